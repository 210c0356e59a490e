"""The C-ABI library builds, loads and exports every symbol the public header declares; argument
validation that needs no device.  CPU only."""
import ctypes
import os
import re

import pytest

import paper_2501_10054_b200 as T
from paper_2501_10054_b200 import build as tbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    tbuild.build()
    return T.load_library()


def test_header_symbols_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "tardis.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(tardis_[a-z0-9_]+)\s*\(", hdr))
    assert {"tardis_fold", "tardis_ffn_forward", "tardis_stats"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert set(T.EXPORTS) == names
    for n in T.EXPORTS:
        assert callable(getattr(T, n, None)) or n in ("tardis_status_string", "tardis_last_error")


def test_status_strings(lib):
    assert lib.tardis_status_string(0) == b"ok"
    assert all(lib.tardis_status_string(i) for i in range(8))
    assert lib.tardis_last_error() == b""


def test_struct_layout_matches_header():
    # 4 int32, 8 pointers, 2 int32, 3 pointers, uint32 (+ padding)
    assert ctypes.sizeof(T.FoldDesc) == 16 + 64 + 8 + 24 + 8
    assert ctypes.sizeof(T.Stats) == 15 * 8


def test_invalid_arguments_return_status_before_any_launch(lib):
    out = ctypes.c_void_p()
    assert lib.tardis_fold(None, None, ctypes.byref(out)) == 1
    d = T.FoldDesc()
    assert lib.tardis_fold(ctypes.byref(d), None, None) == 1
    base = dict(d_model=64, d_ff=64, dtype=1, act=0, W1=16, W2=16, lo=16, hi=16, a=16, c=16, pred_bits=2,
                pred_group=16, pred_codes=16, pred_scale=16, pred_zero=16, flags=0)

    def status(**kw):
        f = dict(base)
        f.update(kw)
        return lib.tardis_fold(ctypes.byref(T.FoldDesc(**f)), None, ctypes.byref(out))

    assert status(d_model=0) == 1
    assert status(d_model=60) == 1            # not a multiple of 8
    assert status(d_ff=48) == 1               # not a multiple of 32
    assert status(pred_group=24) == 1         # not a multiple of 16
    assert status(d_model=80, pred_group=32) == 1   # group does not divide d
    assert status(dtype=7) == 1
    assert status(act=5) == 1
    assert status(W1=None) == 1
    assert status(W1=24) == 1                 # misaligned
    assert status(pred_bits=5) == 2           # valid but not built (2, 3, 4 and 8 are)
    assert status(pred_bits=3, d_model=80, pred_group=16) == 1   # a row of 3-bit codes must fill whole words
    assert status(pred_bits=0) == 1
    assert status(flags=7) == 1               # beyond the fold study modes
    assert out.value is None
    assert lib.tardis_ffn_forward(None, 16, 16, 1, None) == 1
    assert lib.tardis_stats(None, None) == 1
    assert lib.tardis_destroy(None) == 1
    assert lib.tardis_set_path(None, 0) == 1
    assert lib.tardis_set_deterministic(None, 1) == 1
    assert lib.tardis_stack_forward(None, None, None, None, 0, None, 0, 1, None) == 1
    assert lib.tardis_build_predictor(8, 64, 1, None, None, 2, 64, None, None, None, None) == 1
    assert lib.tardis_debug_fail_alloc(-1) == 0
    assert lib.tardis_debug_damage_guard(None, 0, 0) == 1
    assert lib.tardis_debug_live_allocations(None, None) == 1
    assert lib.tardis_neuron_thresholds(4, 4, None, 4, None, None, None, 0, 0.8, 0.7, 0.9, None, None, None) == 1
    # the dense product: an output that is not 16-byte aligned (a view that starts at an odd column) is refused
    assert lib.tardis_gemm_bf16(8, 8, 8, 16, 8, 16, 8, 20, 8, None) == 1
    assert lib.tardis_gemm_bf16(8, 8, 8, 16, 8, 16, 8, None, 8, None) == 1
    assert lib.tardis_debug_phase_stamps(None, 4) == 1
    assert lib.tardis_save(None, b"/tmp/x") == 1 and lib.tardis_load(None, None, None) == 1
    out2 = ctypes.c_void_p()
    assert lib.tardis_load(b"/nonexistent/dir/file", None, ctypes.byref(out2)) == 1 and out2.value is None


def test_binding_fails_loudly_without_library(tmp_path):
    with pytest.raises(T.TardisError):
        T.load_library(str(tmp_path / "missing.so"))
