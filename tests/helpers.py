"""Shared helpers of the GPU parity tests: run the CUDA library and the fp64 oracle on the same
seeded arrays and compare them under the parity rules."""
import numpy as np
import torch

import paper_2501_10054_b200 as T
import workloads as W
from oracle import tardis_oracle as O

TOL = {"f32": 1e-5, "bf16": 2e-2}
BAND = 1e-6


def to_cuda(layer):
    import dataclasses
    kw = {}
    for f in dataclasses.fields(layer):
        v = getattr(layer, f.name)
        kw[f.name] = v.cuda().contiguous() if isinstance(v, torch.Tensor) else v
    return W.Layer(**kw)


def unpack_bitmap(bm: torch.Tensor, h: int) -> np.ndarray:
    words = bm.cpu().numpy().view(np.uint32)
    bits = (words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
    return bits.reshape(words.shape[0], -1)[:, :h].astype(bool)


def gpu_forward(handle, layer, x, calls=None, capture=True):
    """Runs tardis_ffn_forward over x in batches `calls` (list of batch sizes; default one call).
    Returns y, flags (bool [n,h]), scores (float64 [n,h])."""
    n, d = x.shape
    h = layer.cfg.d_ff
    y = torch.full_like(x, float("nan"))
    F = np.zeros((n, h), dtype=bool)
    S = np.zeros((n, h))
    calls = calls or [n]
    t0 = 0
    for b in calls:
        if b == 0:
            T.tardis_ffn_forward(handle, x[:0], y[:0], 0)
            continue
        bm = torch.zeros(b, h // 32, dtype=torch.int32, device="cuda")
        sc = torch.full((b, h), float("nan"), dtype=torch.float64, device="cuda")
        if capture:
            T.tardis_set_debug_capture(handle, bm, sc)
        T.tardis_ffn_forward(handle, x[t0:t0 + b], y[t0:t0 + b])
        torch.cuda.synchronize()
        if capture:
            T.tardis_set_debug_capture(handle, None, None)
            F[t0:t0 + b] = unpack_bitmap(bm, h)
            S[t0:t0 + b] = sc.cpu().numpy()
        t0 += b
    assert t0 == n
    return y, F, S


def oracle_reference(s, x64, F_gpu=None, full_fold=True, folded=None):
    """Oracle outputs on the same inputs.  Returns dict(zhat, F, band, F_use, y).  Flags of neurons
    inside the excluded band follow the GPU (either value is valid there)."""
    zhat = O.predictor_score(x64, s["codes"], s["scale"], s["zero"], s["group"], s["b1"], s["bits"])
    F = O.flags_from_score(zhat, s["lo"], s["hi"])
    band = O.near_threshold(zhat, s["lo"], s["hi"], BAND)
    F_use = F if F_gpu is None else np.where(band, F_gpu, F)
    if full_fold:
        if folded is None:
            folded = O.fold(s["W1"], s["W2"], s["a"], s["c"], s["b1"], s["b2"])
        y = O.fix(O.speculate(folded[0], folded[1], x64), x64, F_use, s["W1"], s["W2"], s["a"], s["c"], s["b1"], s["act"])
    else:
        y = O.direct_partially_linear(x64, F_use, s["W1"], s["W2"], s["a"], s["c"], s["b1"], s["b2"], s["act"])
    return dict(zhat=zhat, F=F, band=band, F_use=F_use, y=y, folded=folded)


def assert_parity(layer, s, x, y_gpu, F_gpu, S_gpu, full_fold=True, folded=None, score_tol=1e-9, label=""):
    x64 = x.double().cpu().numpy()
    ref = oracle_reference(s, x64, F_gpu, full_fold, folded)
    band = ref["band"]
    mism = (F_gpu != ref["F"]) & ~band
    assert not mism.any(), "%s: %d flag mismatches outside the 1e-6 band (band holds %d)" % (label, mism.sum(), band.sum())
    if S_gpu is not None and score_tol is not None:
        fin = np.isfinite(ref["zhat"])
        tol = np.broadcast_to(np.asarray(score_tol, dtype=float).reshape(-1, 1) if np.ndim(score_tol) else score_tol, fin.shape)
        err = np.abs(S_gpu - ref["zhat"])
        bad = fin & (err > tol)
        assert not bad.any(), "%s: score error %.3e" % (label, err[bad].max())
    rel = O.rel_error(y_gpu.double().cpu().numpy(), ref["y"])
    tol = TOL[layer.cfg.dtype]
    assert np.nanmax(rel) <= tol, "%s: max relative error %.3e > %.1e" % (label, np.nanmax(rel), tol)
    return dict(band=int(band.sum()), flag_frac=float(ref["F"].mean()), max_rel=float(np.nanmax(rel)), ref=ref)
