"""Pins of the synthetic-input recipes (calibration-as-setup).  CPU only."""
import math

import numpy as np
import pytest
import torch

import workloads as W


def test_seeded_and_dtype():
    cfg = W.CONFIGS["tiny_f32"]
    a = W.make_tokens(cfg, 8, 3)
    b = W.make_tokens(cfg, 8, 3)
    c = W.make_tokens(cfg, 8, 4)
    assert torch.equal(a, b) and not torch.equal(a, c) and a.dtype == torch.float32
    # LayerNorm'd: zero mean, unit variance per token
    assert a.mean(-1).abs().max() < 1e-5 and (a.var(-1, unbiased=False) - 1).abs().max() < 1e-3
    assert W.make_tokens(cfg, 0, 0).shape == (0, 256)


def test_mixture_outlier_channels():
    cfg = W.LayerConfig("mix", 512, 2048, tokens="mixture", bias=False)
    x = W.make_tokens(cfg, 512, 0).float()
    ch = W.outlier_channels(cfg)
    assert len(ch) == 5
    rest = torch.ones(512, dtype=torch.bool)
    rest[ch] = False
    assert x[:, ch].std() > 10 * x[:, rest].std()


def test_quantile_ranges_coverage():
    g = torch.Generator().manual_seed(0)
    z = torch.randn(1001, 7, generator=g)
    zs, _ = torch.sort(z, dim=0)
    lo, hi = W.quantile_ranges(zs, 0.05, 0.95)
    cov = ((z >= lo) & (z < hi)).float().mean(0)
    assert (cov - 0.90).abs().max() <= 2.0 / 1001 + 1e-6
    # position p (N-1) with linear interpolation: matches numpy's default quantile
    np.testing.assert_allclose(lo.numpy(), np.quantile(z.numpy().astype(np.float64), 0.05, axis=0), rtol=1e-6)
    np.testing.assert_allclose(hi.numpy(), np.quantile(z.numpy().astype(np.float64), 0.95, axis=0), rtol=1e-6)


def test_least_squares_fit_properties():
    g = torch.Generator().manual_seed(1)
    z = torch.randn(4000, 3, generator=g) * torch.tensor([1.0, 0.05, 1.0]) + torch.tensor([0.0, 0.7, -9.0])
    lo = torch.tensor([-1.0, 0.6, -12.0])
    hi = torch.tensor([1.5, 0.8, -7.0])
    a, c = W.least_squares_fit(z, lo, hi, W.ACT_GELU_TANH)
    # residual orthogonality of OLS on the in-range samples
    for j in range(3):
        m = (z[:, j] >= lo[j]) & (z[:, j] < hi[j])
        zz = z[m, j].double()
        r = W.gelu_f64(zz, 0) - (a[j].double() * zz + c[j].double())
        assert abs(r.sum().item()) < 1e-3 and abs((r * zz).sum().item()) < 1e-3
    # tiny range: slope -> GELU'(m); deep negative range: (a, c) -> (0, 0)
    e = 1e-5
    d07 = (W.gelu_f64(torch.tensor(0.7 + e), 0) - W.gelu_f64(torch.tensor(0.7 - e), 0)).item() / (2 * e)
    assert a[1].item() == pytest.approx(d07, abs=2e-2)
    assert abs(a[2].item()) < 1e-6 and abs(c[2].item()) < 1e-6
    # degenerate column (no sample in range): tangent at the midpoint
    a2, c2 = W.least_squares_fit(z[:, :1], torch.tensor([50.0]), torch.tensor([52.0]), 0)
    assert a2.item() == pytest.approx(1.0, abs=1e-6) and abs(c2.item()) < 1e-4


def test_rtn_quantiser_and_packing():
    g = torch.Generator().manual_seed(2)
    W1 = (torch.randn(16, 128, generator=g) * 0.02).bfloat16()
    q, s, zp = W.quantise_rtn(W1, 64, 2, torch.bfloat16)
    assert q.max() <= 3 and zp.max() <= 3 and s.dtype == torch.bfloat16 and s.shape == (16, 2)
    deq = W.dequantise(q, s, zp, 64)
    # the grid contains 0 and spans the group: error at most about half a step
    assert ((deq - W1.float()).abs() <= 0.55 * s.float().repeat_interleave(64, dim=1) + 1e-9).all()
    words = W.pack_codes(q).numpy().view(np.uint32)
    assert words.shape == (16, 8)
    for k in (0, 1, 15, 16, 127):
        assert ((words[:, k // 16] >> np.uint32(2 * (k % 16))) & 3).tolist() == q[:, k].tolist()


def test_gptq_no_worse_than_rtn_on_correlated_inputs():
    g = torch.Generator().manual_seed(3)
    d, h, N = 128, 32, 512
    mix = torch.randn(d, d, generator=g) * 0.3 + torch.eye(d)
    X = torch.randn(N, d, generator=g) @ mix
    W1 = torch.randn(h, d, generator=g) * 0.02
    qr, sr, zr = W.quantise_rtn(W1, 64, 2, torch.float32)
    qg, sg, zg = W.quantise_gptq(W1, X, 64, 2, torch.float32, block=64)
    assert qg.max() <= 3
    err = lambda q, s, z: (X @ (W1 - W.dequantise(q, s, z, 64)).t()).norm().item()
    assert err(qg, sg, zg) <= err(qr, sr, zr)


def test_make_layer_target_fraction():
    cfg = W.LayerConfig("t", 128, 512, dtype="bf16", n_calib=1024, target_flag_frac=0.10)
    L = W.make_layer(cfg, 0)
    x = W.make_tokens(cfg, 256, 0, tag="tune")
    zhat = W.preactivations(W.dequantise(
        torch.from_numpy(np.stack([((L.codes.numpy().view(np.uint32) >> np.uint32(2 * p)) & 3) for p in range(16)], -1)
                         .reshape(512, 128).astype(np.uint8)), L.scale, L.zero, cfg.group), L.b1, x)
    frac = (~((zhat >= L.lo) & (zhat < L.hi))).float().mean().item()
    assert abs(frac - 0.10) < 0.01
    assert L.W1.dtype == torch.bfloat16 and L.a.dtype == torch.float32 and L.codes.shape == (512, 8)
