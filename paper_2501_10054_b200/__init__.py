"""Python binding of libtardis (the C ABI in include/tardis.h): argument marshalling only.

Every step of the partially linear FFN forward (TARDIS, arXiv 2501.10054: constant folding,
predictor, speculative folded product, result fixing) runs inside the CUDA library; this
module turns torch tensors into device pointers and status codes into exceptions.  There is
no CPU fallback: importing works anywhere, but any call needs libtardis.so and a CUDA device.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtardis.so")

TARDIS_OK = 0
TARDIS_F32, TARDIS_BF16 = 0, 1
TARDIS_ACT_GELU_TANH, TARDIS_ACT_GELU_ERF, TARDIS_ACT_RELU = 0, 1, 2

EXPORTS = ["tardis_fold", "tardis_ffn_forward", "tardis_ffn_forward_static", "tardis_gemm_bf16", "tardis_stats",
           "tardis_set_debug_capture", "tardis_export_folded", "tardis_set_path", "tardis_set_deterministic", "tardis_stack_forward", "tardis_build_predictor", "tardis_destroy", "tardis_calibrate",
           "tardis_debug_phase_stamps", "tardis_range_search", "tardis_neuron_thresholds", "tardis_debug_wait_timeout", "tardis_clear_error", "tardis_debug_fail_alloc", "tardis_debug_live_allocations", "tardis_debug_damage_guard",
           "tardis_save", "tardis_load", "tardis_status_string", "tardis_last_error"]


class TardisError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


class FoldDesc(ctypes.Structure):
    _fields_ = [("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("act", ctypes.c_int32), ("W1", ctypes.c_void_p), ("W2", ctypes.c_void_p),
                ("b1", ctypes.c_void_p), ("b2", ctypes.c_void_p), ("lo", ctypes.c_void_p),
                ("hi", ctypes.c_void_p), ("a", ctypes.c_void_p), ("c", ctypes.c_void_p),
                ("pred_bits", ctypes.c_int32), ("pred_group", ctypes.c_int32),
                ("pred_codes", ctypes.c_void_p), ("pred_scale", ctypes.c_void_p),
                ("pred_zero", ctypes.c_void_p), ("flags", ctypes.c_uint32)]


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in
                ("calls", "tokens", "flagged_total", "flagged_max", "last_path", "bytes_folded",
                 "bytes_predictor", "bytes_tables", "bytes_w1", "bytes_w2t", "bytes_scratch",
                 "device_error", "exact_rechecks", "launches", "last_union")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads libtardis.so (built in-tree by paper_2501_10054_b200.build).  Fails loudly if absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise TardisError(-1, "libtardis.so not found at %s: run `python -m paper_2501_10054_b200.build` "
                              "(there is no CPU fallback)" % p)
    lib = ctypes.CDLL(p)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
    lib.tardis_fold.argtypes = [ctypes.POINTER(FoldDesc), vp, ctypes.POINTER(vp)]
    lib.tardis_ffn_forward.argtypes = [vp, vp, vp, i64, vp]
    lib.tardis_ffn_forward_static.argtypes = [vp, vp, vp, i64, vp]
    lib.tardis_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.tardis_set_debug_capture.argtypes = [vp, vp, vp]
    lib.tardis_export_folded.argtypes = [vp, vp, vp, vp]
    lib.tardis_set_path.argtypes = [vp, i32]
    lib.tardis_set_deterministic.argtypes = [vp, i32]
    lib.tardis_build_predictor.argtypes = [i32, i32, i32, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.tardis_stack_forward.argtypes = [vp, vp, vp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, ctypes.c_int64, vp]
    lib.tardis_destroy.argtypes = [vp]
    lib.tardis_gemm_bf16.argtypes = [i32, i32, i32, vp, i32, vp, i32, vp, i32, vp]
    lib.tardis_calibrate.argtypes = [i32, i32, vp, i64, vp, ctypes.c_double, ctypes.c_double, i32, vp, vp, vp, vp, vp]
    lib.tardis_debug_phase_stamps.argtypes = [vp, i32]
    lib.tardis_range_search.argtypes = [i32, i32, vp, i64, vp, vp, ctypes.c_double, ctypes.c_double, i32, vp, vp, vp, vp, vp, vp]
    lib.tardis_debug_wait_timeout.argtypes = [vp, i64, vp]
    lib.tardis_neuron_thresholds.argtypes = [i32, i32, vp, i64, vp, vp, vp, i32, ctypes.c_double, ctypes.c_double, ctypes.c_double, vp, vp, vp]
    lib.tardis_clear_error.argtypes = [vp]
    lib.tardis_debug_fail_alloc.argtypes = [i32]
    lib.tardis_debug_live_allocations.argtypes = [ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.tardis_debug_damage_guard.argtypes = [vp, i32, i32]
    lib.tardis_save.argtypes = [vp, ctypes.c_char_p]
    lib.tardis_load.argtypes = [ctypes.c_char_p, vp, ctypes.POINTER(vp)]
    for name in EXPORTS[:-2]:
        getattr(lib, name).restype = ctypes.c_int
    lib.tardis_status_string.argtypes = [ctypes.c_int]
    lib.tardis_status_string.restype = ctypes.c_char_p
    lib.tardis_last_error.argtypes = []
    lib.tardis_last_error.restype = ctypes.c_char_p
    if path is None:
        _lib = lib
    return lib


def _check(status: int, what: str):
    if status != TARDIS_OK:
        lib = load_library()
        msg = lib.tardis_status_string(status).decode()
        detail = lib.tardis_last_error().decode()
        raise TardisError(status, "%s: %s%s" % (what, msg, (" [" + detail + "]") if detail and status == 4 else ""))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise TardisError(1, "tensors must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return TARDIS_F32
    if dt == torch.bfloat16:
        return TARDIS_BF16
    raise TardisError(1, "dtype must be float32 or bfloat16")


def tardis_fold(W1, W2, lo, hi, a, c, pred_codes, pred_scale, pred_zero, pred_group, b1=None, b2=None,
                act=TARDIS_ACT_GELU_TANH, pred_bits=2, stream=None, flags=0) -> int:
    """tardis_fold of the C ABI.  Returns the opaque handle (an integer)."""
    lib = load_library()
    h, d = W1.shape
    desc = FoldDesc(d, h, _dtype_code(W1.dtype), act, _ptr(W1), _ptr(W2), _ptr(b1), _ptr(b2), _ptr(lo), _ptr(hi),
                    _ptr(a), _ptr(c), pred_bits, pred_group, _ptr(pred_codes), _ptr(pred_scale), _ptr(pred_zero), flags)
    out = ctypes.c_void_p()
    _check(lib.tardis_fold(ctypes.byref(desc), _stream(stream), ctypes.byref(out)), "tardis_fold")
    return out.value


def tardis_ffn_forward(handle: int, x: torch.Tensor, y: torch.Tensor, n_tokens: Optional[int] = None, stream=None):
    lib = load_library()
    n = x.shape[0] if n_tokens is None else n_tokens
    _check(lib.tardis_ffn_forward(handle, _ptr(x), _ptr(y), n, _stream(stream)), "tardis_ffn_forward")
    return y


def tardis_ffn_forward_static(handle: int, x: torch.Tensor, y: torch.Tensor, n_tokens: Optional[int] = None, stream=None):
    """tardis_ffn_forward_static of the C ABI: the same forward for callers that may not allocate device
    memory; its scratch is a fixed array inside the library (at most 64 tokens, 4 MiB of scratch)."""
    lib = load_library()
    n = x.shape[0] if n_tokens is None else n_tokens
    st = lib.tardis_ffn_forward_static(handle, _ptr(x), _ptr(y), n, _stream(stream))
    if st == 2:
        raise TardisError(st, "tardis_ffn_forward_static: %s" % lib.tardis_last_error().decode())
    _check(st, "tardis_ffn_forward_static")
    return y


def tardis_gemm_bf16(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, stream=None):
    """C[M, N] (float32) = A[M, K] B[N, K]^T for bfloat16 row-major A, B (last stride 1)."""
    lib = load_library()
    M, K = A.shape
    N = B.shape[0]
    if A.stride(1) != 1 or B.stride(1) != 1 or C.stride(1) != 1 or not (A.is_cuda and B.is_cuda and C.is_cuda):
        raise TardisError(1, "tensors must be CUDA tensors with unit inner stride")
    _check(lib.tardis_gemm_bf16(M, N, K, A.data_ptr(), A.stride(0), B.data_ptr(), B.stride(0), C.data_ptr(), C.stride(0),
                                _stream(stream)), "tardis_gemm_bf16")
    return C


def tardis_calibrate(z: torch.Tensor, b1: Optional[torch.Tensor], q_lo: float, q_hi: float, act: int, stream=None):
    """Per-neuron ranges and linear fits from calibration pre-activations z[d_ff, n_cal] (float32, CUDA, unit inner
    stride): returns (lo, hi, a, c), float32 tensors of d_ff elements on z's device."""
    if z.dtype != torch.float32 or not z.is_cuda or z.stride(1) != 1:
        raise TardisError(1, "z must be a float32 CUDA tensor with unit inner stride")
    h, n = z.shape
    out = [torch.empty(h, dtype=torch.float32, device=z.device) for _ in range(4)]
    _check(load_library().tardis_calibrate(h, n, z.data_ptr(), z.stride(0), _ptr(b1), float(q_lo), float(q_hi), int(act),
                                           out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), out[3].data_ptr(),
                                           _stream(stream)), "tardis_calibrate")
    return tuple(out)


def tardis_range_search(z: torch.Tensor, b1: Optional[torch.Tensor], threshold, step: float, act: int, stream=None, want_steps=False):
    """Algorithm 1's greedy range search per neuron from calibration pre-activations z[d_ff, n_cal] (float32, CUDA, unit
    inner stride, n_cal <= 2048): returns (lo, hi, a, c) (and the step counts with want_steps).  `threshold` is a float
    (one coverage for all neurons) or a float32 CUDA tensor of d_ff per-neuron thresholds."""
    if z.dtype != torch.float32 or not z.is_cuda or z.stride(1) != 1:
        raise TardisError(1, "z must be a float32 CUDA tensor with unit inner stride")
    h, n = z.shape
    out = [torch.empty(h, dtype=torch.float32, device=z.device) for _ in range(4)]
    steps = torch.zeros(h, dtype=torch.int32, device=z.device) if want_steps else None
    thr_t = threshold if isinstance(threshold, torch.Tensor) else None
    _check(load_library().tardis_range_search(h, n, z.data_ptr(), z.stride(0), _ptr(b1), _ptr(thr_t),
                                              0.0 if thr_t is not None else float(threshold), float(step), int(act),
                                              out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), out[3].data_ptr(),
                                              _ptr(steps), _stream(stream)), "tardis_range_search")
    return tuple(out) + ((steps,) if want_steps else ())


def tardis_neuron_thresholds(z: torch.Tensor, b1: Optional[torch.Tensor], lo: torch.Tensor, hi: torch.Tensor, act: int,
                             t_layer: float, t_min: float, t_max: float, stream=None):
    """Per-neuron coverage thresholds of Section 5.1.1 from the neurons' approximation errors inside [lo, hi): returns
    (err, thresholds), float32 tensors of d_ff elements (see tardis_neuron_thresholds in tardis.h)."""
    if z.dtype != torch.float32 or not z.is_cuda or z.stride(1) != 1:
        raise TardisError(1, "z must be a float32 CUDA tensor with unit inner stride")
    h, n = z.shape
    err = torch.empty(h, dtype=torch.float32, device=z.device)
    thr = torch.empty(h, dtype=torch.float32, device=z.device)
    _check(load_library().tardis_neuron_thresholds(h, n, z.data_ptr(), z.stride(0), _ptr(b1), _ptr(lo), _ptr(hi), int(act),
                                                   float(t_layer), float(t_min), float(t_max), _ptr(err), _ptr(thr),
                                                   _stream(stream)), "tardis_neuron_thresholds")
    return err, thr


def tardis_stats(handle: int) -> dict:
    lib = load_library()
    st = Stats()
    _check(lib.tardis_stats(handle, ctypes.byref(st)), "tardis_stats")
    return st.as_dict()


def tardis_set_debug_capture(handle: int, flag_bitmap: Optional[torch.Tensor], scores: Optional[torch.Tensor]):
    _check(load_library().tardis_set_debug_capture(handle, _ptr(flag_bitmap), _ptr(scores)), "tardis_set_debug_capture")


def tardis_export_folded(handle: int, Wf: Optional[torch.Tensor], bf: Optional[torch.Tensor], stream=None):
    _check(load_library().tardis_export_folded(handle, _ptr(Wf), _ptr(bf), _stream(stream)), "tardis_export_folded")


def tardis_set_path(handle: int, path: int):
    _check(load_library().tardis_set_path(handle, path), "tardis_set_path")


def tardis_set_deterministic(handle: int, on: bool):
    _check(load_library().tardis_set_deterministic(handle, 1 if on else 0), "tardis_set_deterministic")


def tardis_debug_phase_stamps(max_ctas: int = 512):
    """Phase stamps of the most recent fused decode launch as a numpy int64 array [max_ctas, 16] (needs a
    library built with TARDIS_PHASE_STAMPS; the ordinary build raises UNSUPPORTED)."""
    import numpy as np
    buf = np.zeros((max_ctas, 16), dtype=np.int64)
    _check(load_library().tardis_debug_phase_stamps(buf.ctypes.data, max_ctas), "tardis_debug_phase_stamps")
    return buf


def tardis_debug_wait_timeout(handle: int, limit_cycles: int, stream=None):
    """Launches one warp whose bounded wait runs out after limit_cycles SM cycles (testing aid for the time-out report)."""
    _check(load_library().tardis_debug_wait_timeout(handle, int(limit_cycles), _stream(stream)), "tardis_debug_wait_timeout")


def tardis_clear_error(handle: int):
    _check(load_library().tardis_clear_error(handle), "tardis_clear_error")


def tardis_build_predictor(W1: torch.Tensor, U: Optional[torch.Tensor], bits: int, group: int, stream=None):
    """Predictor of a layer by error-compensated quantisation on the GPU (see tardis_build_predictor in tardis.h).
    W1 [h, d] float32 or bfloat16, U [d, d] float64 upper Cholesky factor of the inverse Hessian (None: round to nearest).
    Returns (codes int32 [h, d bits / 32], scale [h, d / group] in W1's dtype, zero uint8 [h, d / group])."""
    h, d = W1.shape
    if not W1.is_contiguous() or (U is not None and (U.dtype != torch.float64 or not U.is_contiguous() or tuple(U.shape) != (d, d))):
        raise TardisError(1, "W1 must be contiguous and U a contiguous float64 [d, d] tensor")
    codes = torch.empty(h, d * bits // 32, dtype=torch.int32, device=W1.device)
    scale = torch.empty(h, d // group, dtype=W1.dtype, device=W1.device)
    zero = torch.empty(h, d // group, dtype=torch.uint8, device=W1.device)
    _check(load_library().tardis_build_predictor(h, d, _dtype_code(W1.dtype), _ptr(W1), _ptr(U), bits, group, _ptr(codes),
                                                 _ptr(scale), _ptr(zero), _stream(stream)), "tardis_build_predictor")
    return codes, scale, zero


class StackDesc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("layers", ctypes.POINTER(ctypes.c_void_p)), ("normalise", ctypes.c_int32),
                ("ln_gamma", ctypes.POINTER(ctypes.c_void_p)), ("ln_beta", ctypes.POINTER(ctypes.c_void_p)),
                ("ln_eps", ctypes.c_float), ("residual", ctypes.c_int32)]


def tardis_stack_forward(handles, x: torch.Tensor, y: torch.Tensor, gammas=None, betas=None, eps: float = 1e-5,
                         normalise: bool = True, residual: bool = True, work: Optional[torch.Tensor] = None,
                         keep: Optional[torch.Tensor] = None, stream=None):
    """The layers `handles` chained on one residual stream (see tardis_stack_forward in tardis.h).  `work` is scratch of
    2 n d elements in x's dtype (made here when neither it nor `keep` is given: the C call itself allocates nothing);
    `keep` [n_layers, 2, n, d] receives every layer's input and output."""
    L = len(handles)
    arr = (ctypes.c_void_p * L)(*handles)
    ga = (ctypes.c_void_p * L)(*[_ptr(g) for g in gammas]) if gammas is not None else None
    be = (ctypes.c_void_p * L)(*[_ptr(b) for b in betas]) if betas is not None else None
    desc = StackDesc(L, arr, 1 if normalise else 0, ga, be, eps, 1 if residual else 0)
    n = x.shape[0]
    if work is None and keep is None:
        work = torch.empty(2, *x.shape, dtype=x.dtype, device=x.device)
    wb = work.numel() * work.element_size() if work is not None else 0
    kb = keep.numel() * keep.element_size() if keep is not None else 0
    _check(load_library().tardis_stack_forward(ctypes.byref(desc), _ptr(x), _ptr(y), _ptr(work), wb, _ptr(keep), kb, n,
                                               _stream(stream)), "tardis_stack_forward")


def tardis_debug_damage_guard(handle: int, front: bool, repair: bool):
    """Changes (or restores) four guard bytes next to the handle's fp32 accumulator; tardis_stats then reports CORRUPT."""
    _check(load_library().tardis_debug_damage_guard(handle, 1 if front else 0, 1 if repair else 0), "tardis_debug_damage_guard")


def tardis_debug_live_allocations():
    """(count, bytes) of the library's live device allocations in this process."""
    c, b = ctypes.c_int64(), ctypes.c_int64()
    _check(load_library().tardis_debug_live_allocations(ctypes.byref(c), ctypes.byref(b)), "tardis_debug_live_allocations")
    return c.value, b.value


def tardis_debug_fail_alloc(nth: int):
    """The library's (nth + 1)-th device allocation from now fails once; nth < 0 switches the injection off."""
    _check(load_library().tardis_debug_fail_alloc(nth), "tardis_debug_fail_alloc")


def tardis_save(handle: int, path: str):
    """Writes the handle's state (folded matrix, predictor, original weights, tables) to a binary file."""
    _check(load_library().tardis_save(handle, os.fsencode(path)), "tardis_save")


def tardis_load(path: str, stream=None) -> int:
    """Reads a file written by tardis_save and returns a new handle on the current device."""
    out = ctypes.c_void_p()
    _check(load_library().tardis_load(os.fsencode(path), _stream(stream), ctypes.byref(out)), "tardis_load")
    return out.value


def tardis_destroy(handle: int):
    _check(load_library().tardis_destroy(handle), "tardis_destroy")


def fold_layer(layer, stream=None, flags=0) -> int:
    """Convenience: tardis_fold from an object with the fields W1, W2, b1, b2, lo, hi, a, c, codes, scale,
    zero and cfg.group / cfg.act / cfg.bits (all CUDA tensors)."""
    return tardis_fold(layer.W1, layer.W2, layer.lo, layer.hi, layer.a, layer.c, layer.codes, layer.scale,
                       layer.zero, layer.cfg.group, b1=layer.b1, b2=layer.b2, act=layer.cfg.act,
                       pred_bits=layer.cfg.bits, stream=stream, flags=flags)
