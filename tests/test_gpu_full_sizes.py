"""Parity at the full sizes of the five benchmark configurations, in the launch shapes bench.py times
(batch-1 decode, batched decode, prefill chunks).  The GPU runs every token.  The oracle computes the
predictor scores and flags of EVERY token (one BLAS product per quantisation group) and compares them
bit for bit outside the excluded band; the outputs are checked on a seeded sample of the tokens, one by
one, through the direct definition of the partially linear FFN (no d x d fold needed), which equals the
folded path by the pinned identities."""
import numpy as np
import pytest
import torch

import paper_2501_10054_b200 as T
import workloads as W
from oracle import tardis_oracle as O
from tests import helpers as Hp

pytestmark = pytest.mark.gpu


def _check(cfg, batches, sample_per_call, seed=0, fold_rows=8, flag_tokens=None):
    dev = torch.device("cuda", 0)
    L = W.make_layer(cfg, seed, device=dev)
    s = L.numpy64()
    n = sum(batches)
    x = W.make_tokens(cfg, n, seed, device=dev)
    h = T.fold_layer(L)
    rng = np.random.default_rng(seed)
    try:
        # fold: sampled rows of W_f against the oracle (one bf16 rounding of an fp32-accumulated product)
        d = cfg.d_model
        Wf = torch.empty(d, d, dtype=x.dtype, device=dev)
        bf = torch.empty(d, dtype=torch.float32, device=dev)
        T.tardis_export_folded(h, Wf, bf)
        torch.cuda.synchronize()
        rows = np.sort(rng.choice(d, size=fold_rows, replace=False))
        ref_rows = O.fold_rows(rows, s["W1"], s["W2"], s["a"])
        got_rows = Wf[torch.as_tensor(rows, device=dev)].double().cpu().numpy()
        scale = np.abs(ref_rows).max()
        assert np.abs(got_rows - ref_rows).max() <= 2.0 ** -8 * scale
        y, F, S = Hp.gpu_forward(h, L, x, batches)
        st = T.tardis_stats(h)
        assert st["device_error"] == 0 and st["tokens"] == n
        assert st["flagged_total"] == int(F.sum())
        # flags of every token (or of the first `flag_tokens` tokens of every call, where the full product would take
        # the CPU minutes) against the oracle's scores
        sel, t1 = [], 0
        for b in batches:
            sel += list(range(t1, t1 + (b if flag_tokens is None else min(b, flag_tokens))))
            t1 += b
        sel = np.asarray(sel)
        band_total = 0
        for c0 in range(0, len(sel), 512):
            part = sel[c0:c0 + 512]
            x64 = x[torch.as_tensor(part, device=dev)].double().cpu().numpy()
            zhat = O.predictor_score(x64, s["codes"], s["scale"], s["zero"], s["group"], s["b1"], s["bits"])
            F_ref = O.flags_from_score(zhat, s["lo"], s["hi"])
            band = O.near_threshold(zhat, s["lo"], s["hi"], Hp.BAND)
            mism = (F[part] != F_ref) & ~band
            assert not mism.any(), "%s: %d flag mismatches outside the band over %d tokens" % (cfg.name, mism.sum(), len(part))
            band_total += int(band.sum())
        print("%s: flags of %d tokens compared, %d (token, neuron) pairs inside the 1e-6 band" % (cfg.name, len(sel), band_total))
        # sampled tokens of every call
        idx, t0 = [], 0
        for b in batches:
            k = min(b, sample_per_call)
            idx += list(t0 + np.sort(rng.choice(b, size=k, replace=False)))
            t0 += b
        idx = np.asarray(idx)
        xs = x[torch.as_tensor(idx, device=dev)]
        info = Hp.assert_parity(L, s, xs, y[torch.as_tensor(idx, device=dev)], F[idx], None, full_fold=False,
                                score_tol=None, label=cfg.name)
        return info, float(F.mean())
    finally:
        T.tardis_destroy(h)
        del L
        torch.cuda.empty_cache()


def test_decode_7b_batch1_and_batch64():
    info, frac = _check(W.CONFIGS["decode_7b"], [1] * 6 + [64], sample_per_call=4)
    assert 0.07 < frac < 0.13


@pytest.mark.parametrize("q", [0, 1, 2, 3])
def test_falcon_shape_decode_batches(q):
    import dataclasses
    qlo, qhi = W.FALCON_QUANTILES[q]
    cfg = dataclasses.replace(W.CONFIGS["falcon_7b"], q_lo=qlo, q_hi=qhi)
    info, frac = _check(cfg, [1, 1, 4, 16, 64], sample_per_call=3)
    assert 0.02 < frac < 0.45


@pytest.mark.parametrize("seed", [3, 4])
def test_prefill_layers_4096_tokens_in_one_call(seed):
    # two independently seeded layers of the prefill configuration; one call crosses the 2048-token chunk of the batched
    # path (1024 while the capture is on) several times
    info, frac = _check(W.CONFIGS["prefill_7b"], [4096], sample_per_call=12, seed=seed)
    assert 0.07 < frac < 0.13


def test_large_8k_decode_and_prefill():
    info, frac = _check(W.CONFIGS["large_8k"], [1, 1, 32, 4096], sample_per_call=3, fold_rows=4, flag_tokens=256)
    assert 0.07 < frac < 0.13


@pytest.mark.parametrize("cfgname", ["large_8k", "decode_7b"])
@pytest.mark.parametrize("path", [0, 3])
def test_adversarial_tokens_one_huge_channel_many_tiny(path, cfgname):
    """Tokens built to stress the fast scores: one channel thousands of times larger than the rest, the rest tiny with
    alternating signs, at d_model = 8192 (the longest accumulation) and at the headline shape.  The flags of every such token
    must still equal the oracle's, on the fused kernels and on the batched tensor-core path (whose allowance for its fp32 accumulation is an
    assumed bound: this is the search for a violation)."""
    cfg = W.CONFIGS[cfgname]
    dev = torch.device("cuda", 0)
    L = W.make_layer(cfg, 2, device=dev)
    s = L.numpy64()
    d = cfg.d_model
    g = torch.Generator().manual_seed(99)
    n = 24
    x = torch.empty(n, d)
    sign = torch.tensor([1.0, -1.0]).repeat(d // 2)
    for t in range(n):
        tiny = (10.0 ** -(1 + t % 4)) * (0.5 + torch.rand(d, generator=g)) * sign
        x[t] = tiny
        x[t, int(torch.randint(0, d, (1,), generator=g))] = float(2.0 ** (3 + t % 9)) * (1 if t % 2 else -1)
    x = x.to(torch.bfloat16).to(dev)
    h = T.fold_layer(L)
    try:
        T.tardis_set_path(h, path)
        y, F, S = Hp.gpu_forward(h, L, x, [n] if path == 3 else [1] * n, capture=True)
        x64 = x.double().cpu().numpy()
        zhat = O.predictor_score(x64, s["codes"], s["scale"], s["zero"], s["group"], s["b1"], s["bits"])
        F_ref = O.flags_from_score(zhat, s["lo"], s["hi"])
        band = O.near_threshold(zhat, s["lo"], s["hi"], Hp.BAND)
        mism = (F != F_ref) & ~band
        assert not mism.any(), "%d flag mismatches on adversarial tokens (path %d)" % (mism.sum(), path)
        err = np.abs(S - zhat)
        print("adversarial tokens, " + cfgname + ", path %d: largest score error %.3e (score magnitudes up to %.1f), %d pairs in the band"
              % (path, float(np.nanmax(err)), float(np.abs(zhat).max()), int(band.sum())))
        assert T.tardis_stats(h)["device_error"] == 0
    finally:
        T.tardis_destroy(h)
