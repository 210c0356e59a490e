"""GPU parity of the offline statistics (tardis_calibrate) against the oracle, through the C ABI.

Both sides get the same float32 pre-activations, so every decision that float arithmetic makes for an integer
(which samples lie inside [lo, hi)) is taken on identical numbers: the ranges must agree bit for bit, the fits
within the float32 rounding of sums taken in a different order."""
import numpy as np
import pytest
import torch

import paper_2501_10054_b200 as T
import workloads as W
from oracle import tardis_oracle as O

pytestmark = pytest.mark.gpu


def _check(z, b1, q_lo, q_hi, act):
    lo, hi, a, c = T.tardis_calibrate(z, b1, q_lo, q_hi, act)
    torch.cuda.synchronize()
    zc = z.cpu().numpy()
    if b1 is not None:
        zc = zc + b1.cpu().numpy()[:, None]                     # float32 sum, as the kernel forms it
    lo_ref, hi_ref = O.quantile_ranges(zc, q_lo, q_hi)
    a_ref, c_ref = O.least_squares_fit(zc, lo_ref, hi_ref, act)
    assert np.array_equal(lo.cpu().numpy(), lo_ref) and np.array_equal(hi.cpu().numpy(), hi_ref)
    a, c = a.cpu().numpy().astype(np.float64), c.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(a - a_ref) <= 2e-6 * np.maximum(1.0, np.abs(a_ref)))
    assert np.all(np.abs(c - c_ref) <= 2e-6 * np.maximum(1.0, np.abs(c_ref)))
    return lo_ref, hi_ref, a_ref, c_ref


@pytest.mark.parametrize("act", [W.ACT_GELU_TANH, W.ACT_GELU_ERF, W.ACT_RELU])
@pytest.mark.parametrize("shape", [(64, 1), (40, 2), (96, 257), (33, 1000), (16, 2048), (8, 8192)])
def test_ranges_and_fits_match_oracle(shape, act):
    h, n = shape
    g = torch.Generator().manual_seed(100 * h + n)
    z = (torch.randn(h, n, generator=g) * torch.linspace(0.3, 3.0, h)[:, None] + torch.linspace(-1, 1, h)[:, None]).cuda()
    b1 = (0.1 * torch.randn(h, generator=g)).cuda()
    _check(z, b1, 0.05, 0.95, act)
    _check(z, None, 0.0, 1.0, act)
    _check(z, None, 0.4, 0.4, act)                              # empty range: every neuron takes the tangent


def test_padded_rows_ties_and_degenerate_neurons():
    # leading dimension larger than n, many equal samples, constant neurons
    g = torch.Generator().manual_seed(7)
    buf = torch.randn(50, 700, generator=g).cuda()
    buf[:10] = torch.round(buf[:10] * 2) / 2                   # ties
    buf[10:13] = 0.25                                           # constant: zero variance in range
    z = buf[:, :613]
    assert z.stride(0) == 700
    _check(z, None, 0.1, 0.9, W.ACT_GELU_TANH)


def test_layer_calibration_through_the_gemm_entry():
    # pre-activations of a bf16 layer from the library's own GEMM, then ranges and fits; the recipe of the synthetic
    # workloads (float32 pre-activations from torch) gives the same statistics up to the accumulation order of z
    cfg = W.LayerConfig("cal", 512, 2048, n_calib=1024)
    L = W.make_layer(cfg, 3)
    xcal = W.make_tokens(cfg, 1024, 3, tag="calib").cuda()
    W1 = L.W1.cuda()
    z = torch.empty(cfg.d_ff, 1024, dtype=torch.float32, device="cuda")
    T.tardis_gemm_bf16(W1, xcal, z)
    b1 = L.b1.cuda() if L.b1 is not None else None
    lo, hi, a, c = _check(z, b1, 0.05, 0.95, cfg.act)
    assert np.all(lo < hi)
    z_ref = xcal.float() @ W1.float().t()
    if b1 is not None:
        z_ref = z_ref + b1[None, :]
    q = torch.quantile(z_ref, torch.tensor([0.05, 0.95], device="cuda"), dim=0).cpu().numpy()
    assert np.abs(lo - q[0]).max() < 1e-3 and np.abs(hi - q[1]).max() < 1e-3


def test_argument_errors():
    lib = T.load_library()
    z = torch.zeros(4, 16, device="cuda")
    o = [torch.zeros(4, device="cuda") for _ in range(4)]
    def call(h, n, zp, ld, qlo, qhi, act):
        return lib.tardis_calibrate(h, n, zp, ld, None, qlo, qhi, act, o[0].data_ptr(), o[1].data_ptr(), o[2].data_ptr(),
                                    o[3].data_ptr(), None)
    assert call(4, 16, z.data_ptr(), 16, 0.1, 0.9, 0) == T.TARDIS_OK
    assert call(4, 16, None, 16, 0.1, 0.9, 0) == 1              # null samples
    assert call(4, 16, z.data_ptr(), 8, 0.1, 0.9, 0) == 1       # leading dimension below n_cal
    assert call(4, 16, z.data_ptr(), 16, 0.9, 0.1, 0) == 1      # q_lo > q_hi
    assert call(4, 16, z.data_ptr(), 16, 0.1, 1.5, 0) == 1
    assert call(4, 16, z.data_ptr(), 16, 0.1, 0.9, 7) == 1      # unknown activation
    assert call(4, 16, z.data_ptr(), 16, 0.1, 0.9, 2) == T.TARDIS_OK   # ReLU
    assert call(4, 9000, z.data_ptr(), 9000, 0.1, 0.9, 0) == 2  # more samples than the kernel sorts
    torch.cuda.synchronize()


def test_full_size_layer_sampled_neurons():
    # the shape bench.py times (16384 neurons x 2048 calibration tokens, pre-activations from the library's GEMM):
    # the GPU does every neuron, the oracle a seeded sample of them
    cfg = W.CONFIGS["decode_7b"]
    dev = torch.device("cuda", 0)
    W1, _, b1, _ = W.make_weights(cfg, 0, device=dev)
    xcal = W.make_tokens(cfg, 2048, 0, device=dev, tag="calib")
    z = torch.empty(cfg.d_ff, 2048, dtype=torch.float32, device=dev)
    T.tardis_gemm_bf16(W1, xcal, z)
    lo, hi, a, c = T.tardis_calibrate(z, b1, 0.05, 0.95, cfg.act)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(0).choice(cfg.d_ff, size=256, replace=False))
    idx = torch.as_tensor(rows, device=dev)
    zc = z[idx].cpu().numpy()
    if b1 is not None:
        zc = zc + b1[idx].cpu().numpy()[:, None]
    lo_ref, hi_ref = O.quantile_ranges(zc, 0.05, 0.95)
    a_ref, c_ref = O.least_squares_fit(zc, lo_ref, hi_ref, cfg.act)
    assert np.array_equal(lo[idx].cpu().numpy(), lo_ref) and np.array_equal(hi[idx].cpu().numpy(), hi_ref)
    assert np.all(np.abs(a[idx].cpu().numpy() - a_ref) <= 2e-6 * np.maximum(1.0, np.abs(a_ref)))
    assert np.all(np.abs(c[idx].cpu().numpy() - c_ref) <= 2e-6 * np.maximum(1.0, np.abs(c_ref)))
    # everywhere: a proper range, about 90 percent of the samples inside, a finite fit
    zb = z + (b1[:, None] if b1 is not None else 0.0)
    inside = ((zb >= lo[:, None]) & (zb < hi[:, None])).float().mean(1)
    assert bool((lo < hi).all()) and float((inside - 0.9).abs().max()) < 2e-3
    assert bool(torch.isfinite(a).all()) and bool(torch.isfinite(c).all())


# ------------------------------------------------------------------ Algorithm 1: the greedy range search
def _check_search(z, b1, thr, step, act, thr_tensor=None):
    """tardis_range_search against the oracle, neuron by neuron.  The ranges must be the same float32 numbers; a neuron
    whose search met a near-tie (the two candidate errors within 1e-7 of each other, or two samples with kernel densities
    within 1e-9) may legitimately go the other way under a different summation order: those are counted, and for them the
    result only has to be a valid outcome (coverage reached, not reached one step earlier)."""
    res = T.tardis_range_search(z, b1, thr_tensor if thr_tensor is not None else thr, step, act, want_steps=True)
    torch.cuda.synchronize()
    lo, hi, a, c, steps = [r.cpu().numpy() for r in res]
    zc = z.cpu().numpy()
    if b1 is not None:
        zc = zc + b1.cpu().numpy()[:, None]
    h, n = zc.shape
    ties = 0
    for j in range(h):
        t = float(thr_tensor[j]) if thr_tensor is not None else thr
        lo_r, hi_r, trace, margin = O.greedy_range_search(zc[j], t, step, act, return_trace=True)
        same = np.float32(lo_r) == lo[j] and np.float32(hi_r) == hi[j] and steps[j] == len(trace)
        if not same:
            zs = np.sort(zc[j].astype(np.float64))
            bw = 1.06 * np.std(zs, ddof=1) * n ** -0.2
            dens = np.array([np.exp(-0.5 * ((zs - v) / bw) ** 2).sum() for v in zs]) if bw > 0 else np.ones(n)
            top = np.sort(dens)[-2:]
            near = margin < 1e-7 or (top[1] - top[0]) <= 1e-9 * top[1]
            assert near, "neuron %d: GPU range (%r, %r) after %d steps, oracle (%r, %r) after %d, margin %.3e" % (
                j, lo[j], hi[j], steps[j], lo_r, hi_r, len(trace), margin)
            ties += 1
            inside = ((zc[j] >= lo[j]) & (zc[j] < hi[j])).mean()
            assert inside >= t - 1e-12
        # the line of the final range, from the float32 bounds the kernel stored
        a_ref, c_ref = O.least_squares_fit(zc[j:j + 1], lo[j:j + 1], hi[j:j + 1], act)
        assert abs(float(a[j]) - float(a_ref[0])) <= 2e-6 * max(1.0, abs(float(a_ref[0])))
        assert abs(float(c[j]) - float(c_ref[0])) <= 2e-6 * max(1.0, abs(float(c_ref[0])))
    return ties


@pytest.mark.parametrize("act", [W.ACT_GELU_TANH, W.ACT_RELU])
@pytest.mark.parametrize("shape", [(48, 64), (24, 257), (12, 1000)])
def test_greedy_range_search_matches_oracle(shape, act):
    h, n = shape
    g = torch.Generator().manual_seed(7 * h + n)
    z = (torch.randn(h, n, generator=g) * torch.linspace(0.3, 2.0, h)[:, None] + torch.linspace(-1, 1, h)[:, None]).cuda()
    b1 = (0.1 * torch.randn(h, generator=g)).cuda()
    ties = _check_search(z, b1, 0.85, 0.05, act)
    thr = torch.linspace(0.5, 0.97, h).cuda()
    ties += _check_search(z, None, None, 0.1, act, thr_tensor=thr)
    print("range search %s: %d near-ties among %d searches" % (shape, ties, 2 * h))
    assert ties <= h // 4


def test_greedy_range_search_edge_cases_and_errors():
    lib = T.load_library()
    # all samples equal, a single sample, threshold 0 (empty range at the centroid) and 1 (every sample)
    z = torch.tensor([[0.3] * 16, list(np.cumsum(np.linspace(0.1, 0.4, 16)) - 2.0)], dtype=torch.float32).cuda()   # (no symmetric ties)
    lo, hi, a, c = T.tardis_range_search(z, None, 1.0, 0.5, W.ACT_GELU_TANH)
    torch.cuda.synchronize()
    zc = z.cpu().numpy()
    for j in range(2):
        lo_r, hi_r = O.greedy_range_search(zc[j], 1.0, 0.5)
        assert np.float32(lo_r) == lo[j].item() and np.float32(hi_r) == hi[j].item()
        assert ((zc[j] >= lo[j].item()) & (zc[j] < hi[j].item())).all()
    lo0, hi0, _, _ = T.tardis_range_search(z, None, 0.0, 0.5, W.ACT_GELU_TANH)
    assert (lo0 == hi0).all()
    one = torch.tensor([[1.25]], dtype=torch.float32).cuda()
    lo1, hi1, _, _ = T.tardis_range_search(one, None, 0.9, 0.25, W.ACT_RELU)
    assert lo1.item() == 1.25 and hi1.item() == 1.5
    big = torch.zeros(2, 4096, device="cuda")
    with pytest.raises(T.TardisError):
        T.tardis_range_search(big, None, 0.9, 0.1, 0)          # more than 2048 samples: unsupported
    p = z.data_ptr()
    assert lib.tardis_range_search(2, 16, p, 16, None, None, 0.9, 0.0, 0, p, p, p, p, None, None) == 1   # step must be positive
    assert lib.tardis_range_search(2, 16, p, 16, None, None, 1.5, 0.1, 0, p, p, p, p, None, None) == 1   # threshold outside [0, 1]


def test_greedy_range_search_full_layer_shape_sampled():
    """The 7B-class shape (16384 neurons x 2048 calibration tokens) runs whole on the GPU; the oracle checks a seeded sample."""
    cfg = W.CONFIGS["decode_7b"]
    dev = torch.device("cuda", 0)
    L = W.make_layer(cfg, 5, device=dev)
    xcal = W.make_tokens(cfg, 2048, 5, device=dev, tag="calib")
    zcal = torch.empty(cfg.d_ff, 2048, dtype=torch.float32, device=dev)
    T.tardis_gemm_bf16(L.W1, xcal, zcal)
    lo, hi, a, c, steps = T.tardis_range_search(zcal, L.b1, 0.85, 0.05, cfg.act, want_steps=True)
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(cfg.d_ff, size=6, replace=False))
    sel = torch.as_tensor(rows, device=dev)
    zs = zcal[sel].contiguous()
    ties = _check_search(zs, L.b1[sel].contiguous() if L.b1 is not None else None, 0.85, 0.05, cfg.act)
    lo_s, hi_s, _, _ = T.tardis_range_search(zs, L.b1[sel].contiguous() if L.b1 is not None else None, 0.85, 0.05, cfg.act)
    assert torch.equal(lo_s, lo[sel]) and torch.equal(hi_s, hi[sel])
    cov = ((zcal + L.b1[:, None] >= lo[:, None]) & (zcal + L.b1[:, None] < hi[:, None])).float().mean(dim=1)
    assert float(cov.min()) >= 0.85 - 1e-6 and float(cov.mean()) < 0.87


# ---- neuron-level thresholds (tardis_neuron_thresholds) ----
@pytest.mark.parametrize("h,n,act", [(96, 257, W.ACT_GELU_TANH), (300, 1000, W.ACT_GELU_ERF), (1024, 2048, W.ACT_RELU), (5, 16, W.ACT_GELU_TANH)])
def test_neuron_thresholds_match_oracle(h, n, act):
    """Errors: each neuron's approx_error of the oracle within the rounding of a float32 and of sums taken in another order.
    Thresholds: the oracle's allocation on its own errors (rounded to float32, the precision the order is taken in); a
    neuron may differ only where its error is so close to the error at which the budget runs out that the two sides
    can order it differently, and then both values must be valid ones (t_min or t_max).  The mean threshold is t_layer."""
    g = torch.Generator().manual_seed(31 * h + n)
    z = (torch.randn(h, n, generator=g) * torch.linspace(0.3, 3.0, h)[:, None] + torch.linspace(-1, 1, h)[:, None]).cuda()
    b1 = (0.1 * torch.randn(h, generator=g)).cuda()
    lo, hi, _, _ = T.tardis_range_search(z, b1, 0.85, 0.05, act)
    for (t_layer, t_min, t_max) in [(0.85, 0.7, 0.95), (0.8, 0.8, 0.9), (0.9, 0.5, 0.9), (0.77, 0.6, 1.0)]:
        err, thr = T.tardis_neuron_thresholds(z, b1, lo, hi, act, t_layer, t_min, t_max)
        torch.cuda.synchronize()
        zc = z.cpu().numpy() + b1.cpu().numpy()[:, None]
        lo_c, hi_c = lo.cpu().numpy().astype(np.float64), hi.cpu().numpy().astype(np.float64)
        e_ref = np.array([O.approx_error(zc[j], lo_c[j], hi_c[j], act) for j in range(h)])
        e_gpu = err.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(e_gpu - e_ref) <= 1e-6 * np.abs(e_ref) + 1e-30), np.abs(e_gpu - e_ref).max()
        e32 = e_ref.astype(np.float32).astype(np.float64)
        t_ref = O.neuron_thresholds(e32, t_layer, t_min, t_max)
        t_gpu = thr.cpu().numpy().astype(np.float64)
        assert abs(t_gpu.mean() - t_layer) <= 1e-6
        assert np.all(t_gpu >= t_min - 1e-7) and np.all(t_gpu <= t_max + 1e-7)
        diff = np.abs(t_gpu - t_ref) > 1e-6
        if diff.any():
            order = np.argsort(e32, kind="stable")
            funded = int(np.floor((t_layer - t_min) * h / (t_max - t_min) + 1e-9)) if t_max > t_min else 0
            cut = e32[order[min(funded, h - 1)]]
            assert np.all(np.abs(e32[diff] - cut) <= 2e-6 * abs(cut) + 1e-30), "thresholds differ away from the cut-off error"
    # a layer whose neurons all have the same error: the smaller index is funded first
    same = torch.zeros(8, 64).cuda()
    same[:, ::2] = 1.0
    err, thr = T.tardis_neuron_thresholds(same, None, torch.full((8,), -5.0).cuda(), torch.full((8,), 5.0).cuda(), W.ACT_RELU, 0.75, 0.5, 1.0)
    assert np.allclose(thr.cpu().numpy(), [1, 1, 1, 1, 0.5, 0.5, 0.5, 0.5])
    with pytest.raises(T.TardisError):
        T.tardis_neuron_thresholds(same, None, err, err, 0, 0.5, 0.6, 0.9)      # t_layer below t_min


def test_offline_pipeline_thresholds_feed_the_range_search():
    """The offline steps of Section 5.1.1 chained on the GPU: a range search at the layer threshold, the neuron-level
    thresholds from the errors of those ranges, a second search with one threshold per neuron.  Properties that must hold
    whatever the data: every neuron's final range covers at least its own threshold of its samples (or all of them), a
    neuron whose threshold went up does not get a narrower range, and the thresholds average to the layer's."""
    h, n, act = 512, 1024, W.ACT_GELU_TANH
    g = torch.Generator().manual_seed(77)
    z = (torch.randn(h, n, generator=g) * torch.linspace(0.4, 2.5, h)[:, None] + torch.linspace(-0.5, 0.5, h)[:, None]).cuda()
    lo0, hi0, _, _ = T.tardis_range_search(z, None, 0.85, 0.05, act)
    err, thr = T.tardis_neuron_thresholds(z, None, lo0, hi0, act, 0.85, 0.75, 0.95)
    lo1, hi1, a1, c1 = T.tardis_range_search(z, None, thr, 0.05, act)
    torch.cuda.synchronize()
    inside = ((z >= lo1[:, None]) & (z < hi1[:, None])).float().mean(dim=1)
    assert bool((inside >= thr - 1e-6).all())
    assert abs(float(thr.mean()) - 0.85) < 1e-5
    up = thr > 0.85 + 1e-6
    assert bool(((hi1 - lo1)[up] >= (hi0 - lo0)[up] - 1e-6).all())
    down = thr < 0.85 - 1e-6
    assert bool(((hi1 - lo1)[down] <= (hi0 - lo0)[down] + 1e-6).all())
    # the neurons with the smallest errors are the ones that were given the widest coverage
    order = torch.argsort(err, stable=True)
    assert bool((thr[order[:h // 4]] >= thr[order[-h // 4:]].max() - 1e-6).all())


# ---- the predictor built on the GPU (tardis_build_predictor) ----
def _upper_factor(X, damp=0.01):
    """Upper Cholesky factor of the inverse of H = (2/N) X^T X + damp mean(diag H) I, by numpy's routines in float64."""
    X = np.asarray(X, dtype=np.float64)
    H = 2.0 / X.shape[0] * X.T @ X
    H += damp * np.mean(np.diag(H)) * np.eye(H.shape[0])
    return np.ascontiguousarray(np.linalg.cholesky(np.linalg.inv(H)).T)


def _build_and_compare(W1, U, bits, G, rows=None):
    """GPU builder against the oracle on the same W1 and U: codes, zero-points and scales must be identical (every rounding
    decision is taken in double precision with the same sequence of rounded operations on both sides)."""
    dtype = "f32" if W1.dtype == torch.float32 else "bf16"
    Ud = None if U is None else torch.from_numpy(U).cuda()
    codes, scale, zero = T.tardis_build_predictor(W1, Ud, bits, G)
    torch.cuda.synchronize()
    h, d = W1.shape
    rows = np.arange(h) if rows is None else rows
    q_ref, s_ref, z_ref, _ = O.gptq_quantise(W1[torch.as_tensor(rows).cuda()].double().cpu().numpy(), U, G, bits, dtype)
    q_gpu = O.unpack_codes(codes.cpu().numpy().view(np.uint32)[rows], d, bits)
    bad = int((q_gpu != q_ref).sum())
    assert bad == 0, "%d of %d codes differ" % (bad, q_ref.size)
    assert np.array_equal(zero.cpu().numpy()[rows].astype(np.float64), z_ref)
    assert np.array_equal(scale.double().cpu().numpy()[rows], s_ref)
    return codes, scale, zero


@pytest.mark.parametrize("dt", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("h,d,G,bits", [(400, 512, 64, 2), (130, 512, 128, 2), (64, 256, 128, 4), (70, 384, 64, 8), (1, 64, 64, 2), (50, 320, 64, 3)])
def test_build_predictor_matches_oracle(h, d, G, bits, dt):
    g = torch.Generator().manual_seed(h * 7 + d + bits)
    W1 = (torch.randn(h, d, generator=g) * 0.05).to(dt).cuda()
    mix = torch.eye(d) + 0.5 * torch.randn(d, d, generator=g) / d ** 0.5
    X = (torch.randn(3 * d, d, generator=g) @ mix).numpy()
    _build_and_compare(W1, _upper_factor(X), bits, G)
    _build_and_compare(W1, None, bits, G)                       # no U: plain rounding to nearest
    W0 = W1.clone()
    W0[0] = 0                                                   # a neuron of zeros: scale 1, every code = zero-point 0
    _build_and_compare(W0, _upper_factor(X), bits, G)


def test_build_predictor_full_size_sampled_rows_and_use_in_a_layer():
    """The 7B-class layer (16384 x 4096, groups of 128, 2 bits): sampled neurons against the oracle (neurons are independent
    given U), then the built predictor goes into tardis_fold and a forward is compared with the oracle run on those codes."""
    cfg = W.CONFIGS["decode_7b"]
    L = W.make_layer(cfg, seed=4, device=torch.device("cuda", 0))
    xcal = W.make_tokens(cfg, 1024, 4, device=torch.device("cuda", 0), tag="calibration").double()
    H = 2.0 / xcal.shape[0] * xcal.t() @ xcal
    H += 0.01 * torch.mean(torch.diagonal(H)) * torch.eye(cfg.d_model, dtype=torch.float64, device=H.device)
    U = torch.linalg.cholesky(torch.cholesky_inverse(torch.linalg.cholesky(H)), upper=True).contiguous()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    codes, scale, zero = T.tardis_build_predictor(L.W1, U, 2, 128)
    e1.record()
    torch.cuda.synchronize()
    print("tardis_build_predictor, 16384 x 4096: %.1f ms" % e0.elapsed_time(e1))
    rows = np.array([0, 1, 63, 64, 4097, 8191, 12345, 16383])
    Un = U.cpu().numpy()
    q_ref, s_ref, z_ref, _ = O.gptq_quantise(L.W1[torch.as_tensor(rows).cuda()].double().cpu().numpy(), Un, 128, 2, "bf16")
    q_gpu = O.unpack_codes(codes.cpu().numpy().view(np.uint32)[rows], cfg.d_model, 2)
    assert np.array_equal(q_gpu, q_ref) and np.array_equal(zero.cpu().numpy()[rows].astype(np.float64), z_ref)
    assert np.array_equal(scale.double().cpu().numpy()[rows], s_ref)
    # the output error on the calibration inputs is below that of plain rounding for these neurons
    r_codes, r_scale, r_zero = T.tardis_build_predictor(L.W1, None, 2, 128)
    def out_err(c, s_, z_):
        qq = O.unpack_codes(c.cpu().numpy().view(np.uint32)[rows], cfg.d_model, 2).astype(np.float64).reshape(len(rows), -1, 128)
        deq = ((qq - z_.cpu().numpy()[rows].astype(np.float64)[:, :, None]) * s_.double().cpu().numpy()[rows][:, :, None]).reshape(len(rows), -1)
        return np.linalg.norm(xcal.cpu().numpy() @ (L.W1[torch.as_tensor(rows).cuda()].double().cpu().numpy() - deq).T)
    assert out_err(codes, scale, zero) < 0.9 * out_err(r_codes, r_scale, r_zero)
    import dataclasses
    from tests import helpers as Hp
    L2 = dataclasses.replace(L, codes=codes, scale=scale, zero=zero)
    h = T.fold_layer(L2)
    try:
        x = W.make_tokens(cfg, 3, 9, device=torch.device("cuda", 0))
        y, F, S = Hp.gpu_forward(h, L2, x, [1, 2])
        Hp.assert_parity(L2, L2.numpy64(), x, y, F, S, score_tol=3e-4, label="built predictor")
    finally:
        T.tardis_destroy(h)
