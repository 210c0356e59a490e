"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same seeded
inputs.  Flags bit-exact outside the 1e-6 score band; outputs within 1e-5 (fp32) / 2e-2 (bf16)
max relative error |dy| / max(|y_ref|, rms(y_ref[t,:]))."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2501_10054_b200 as T
import workloads as W
from oracle import tardis_oracle as O
from tests import helpers as Hp

pytestmark = pytest.mark.gpu


def _layer(cfg, seed=0):
    return Hp.to_cuda(W.make_layer(cfg, seed))


def _run(cfg, n, calls=None, seed=0, path=0, full_fold=True):
    L = _layer(cfg, seed)
    s = L.numpy64()
    x = W.make_tokens(cfg, n, seed).cuda()
    h = T.fold_layer(L)
    try:
        T.tardis_set_path(h, path)
        y, F, S = Hp.gpu_forward(h, L, x, calls)
        # generic kernels: exact fp64 score; fused decode kernel (calls of up to 8 tokens): exact up to the tracked
        # rounding of tiny x elements; batched path: fp32 tensor-core scores (flags are settled exactly near the
        # range ends, the captured score is the fast one)
        if path == 1 or cfg.dtype == "f32":
            tol = 1e-9
        else:
            # the decode kernel rounds x to a 22-bit grid under the token's largest element
            xmax = x.float().abs().amax(dim=1).cpu().numpy()
            small = np.maximum(5e-7, 4e-6 * xmax)
            fused = path != 3 and cfg.bits == 2
            tol = np.concatenate([np.full(b, 0.0 if (b <= 8 and fused) else 3e-4) for b in (calls or [n])])
            tol = np.where(tol == 0.0, small, tol)
        info = Hp.assert_parity(L, s, x, y, F, S, full_fold=full_fold, label=cfg.name, score_tol=tol)
        st = T.tardis_stats(h)
        assert st["tokens"] == n and st["device_error"] == 0
        assert st["flagged_total"] == int(F.sum())
        assert st["flagged_max"] == int(F.sum(1).max()) if n else True
    finally:
        T.tardis_destroy(h)
    return info


def test_tiny_f32_config_all_tokens():
    cfg = W.CONFIGS["tiny_f32"]
    info = _run(cfg, 64)
    assert 0.02 < info["flag_frac"] < 0.4


def test_tiny_f32_fold_matches_oracle_elementwise():
    cfg = W.CONFIGS["tiny_f32"]
    L = _layer(cfg)
    s = L.numpy64()
    h = T.fold_layer(L)
    Wf = torch.empty(cfg.d_model, cfg.d_model, dtype=torch.float32, device="cuda")
    bf = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    T.tardis_export_folded(h, Wf, bf)
    torch.cuda.synchronize()
    Wf_ref, bf_ref = O.fold(s["W1"], s["W2"], s["a"], s["c"], s["b1"], s["b2"])
    assert np.abs(Wf.double().cpu().numpy() - Wf_ref).max() <= 1e-5 * np.abs(Wf_ref).max()
    assert np.abs(bf.double().cpu().numpy() - bf_ref).max() <= 1e-5 * np.abs(bf_ref).max()
    st = T.tardis_stats(h)
    # footprint accounting: folded matrix d^2 against the 2 d h original weights = 12.5 % at h = 4 d,
    # 2-bit codes = 6.25 % of the original weights
    assert (st["bytes_folded"] - 4 * cfg.d_model) / (st["bytes_w1"] + st["bytes_w2t"]) == 0.125
    assert (cfg.d_ff * cfg.d_model // 4) / st["bytes_w1"] == 2 / 32            # 2-bit codes against fp32 W1
    T.tardis_destroy(h)


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("shape", [(512, 2048, 64), (1136, 4544, 16), (768, 3072, 128)])
def test_bf16_small_shapes_ragged_batches(shape, path):
    d, hh, G = shape
    cfg = W.LayerConfig("small_%d" % d, d, hh, group=G, n_calib=512, bias=(d != 1136),
                        tokens="mixture" if d == 1136 else "student_t")
    calls = [1, 1, 3, 8, 9, 0, 2, 64, 65, 5]
    info = _run(cfg, sum(calls), calls, path=path)
    assert 0.02 < info["flag_frac"] < 0.5


def test_batched_path_forced_for_calls_of_a_few_tokens():
    # path 3 sends every call through the tensor-core path, also those the per-token kernel would take
    cfg = W.LayerConfig("small_forced", 512, 2048, group=64, n_calib=512)
    calls = [1, 3, 8, 2, 0, 7]
    info = _run(cfg, sum(calls), calls, path=3)
    assert 0.02 < info["flag_frac"] < 0.5


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_wider_predictor_codes(bits):
    # 3- and 4-bit codes: batched tensor-core path (also for calls of a few tokens) and generic kernels; 8-bit codes: generic
    # kernels only.  The paper sweeps the predictor size (Section 7.6); here each width must give the oracle's flags.
    # (3-bit codes are a bit stream: some cross from one 32-bit word into the next.)
    cfg = W.LayerConfig("bits%d" % bits, 512, 2048, group=64, bits=bits, n_calib=512)
    calls = [1, 3, 20, 8]
    info = _run(cfg, sum(calls), calls, path=3 if bits <= 4 else 0)
    assert 0.02 < info["flag_frac"] < 0.5
    _run(cfg, 6, [1, 5], path=1)
    cfg32 = W.LayerConfig("bits%d_f32" % bits, 128, 512, dtype="f32", group=32, bits=bits, n_calib=512)
    _run(cfg32, 7)


def test_relu_activation_on_every_path():
    # ReLU layer (the OPT model of the paper's evaluation): per-token kernel, batched path, generic kernels, fp32
    cfg = W.LayerConfig("relu", 512, 2048, dtype="bf16", act=W.ACT_RELU, n_calib=512)
    _run(cfg, 30, [1, 5, 24], seed=2)
    _run(cfg, 12, [2, 10], seed=2, path=1)
    cfg = W.LayerConfig("relu32", 128, 512, dtype="f32", act=W.ACT_RELU, n_calib=512)
    _run(cfg, 9, seed=4)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_exact_range_mode_flags_from_true_preactivations(dtype):
    # path 4: the range check runs on z = W1 x + b1 itself (the paper's ablation that takes the predictor out)
    cfg = W.LayerConfig("hybrid_" + dtype, 256, 1024, dtype=dtype, n_calib=512)
    L = _layer(cfg, 1)
    s = L.numpy64()
    x = W.make_tokens(cfg, 11, 1).cuda()
    h = T.fold_layer(L)
    try:
        T.tardis_set_path(h, 4)
        y, F, S = Hp.gpu_forward(h, L, x, [1, 10])
        x64 = x.double().cpu().numpy()
        z = x64 @ s["W1"].T + s["b1"][None, :]
        F_ref = O.flags_from_score(z, s["lo"], s["hi"])
        band = O.near_threshold(z, s["lo"], s["hi"], Hp.BAND)
        assert not ((F != F_ref) & ~band).any()
        assert np.abs(S - z).max() < 1e-9                       # the captured score is the pre-activation
        y_ref = O.direct_partially_linear(x64, np.where(band, F, F_ref), s["W1"], s["W2"], s["a"], s["c"], s["b1"], s["b2"], s["act"])
        assert np.nanmax(O.rel_error(y.double().cpu().numpy(), y_ref)) <= Hp.TOL[dtype]
        # the predictor's flags differ from these on some neurons (that difference is what the mode measures)
        zhat = O.predictor_score(x64, s["codes"], s["scale"], s["zero"], s["group"], s["b1"], s["bits"])
        assert (O.flags_from_score(zhat, s["lo"], s["hi"]) != F_ref).any()
    finally:
        T.tardis_destroy(h)


def test_erf_activation_and_other_seed():
    cfg = W.LayerConfig("erf", 256, 1024, dtype="bf16", act=W.ACT_GELU_ERF, n_calib=512)
    _run(cfg, 17, [1, 16], seed=5)
    cfg = W.LayerConfig("erf32", 128, 512, dtype="f32", act=W.ACT_GELU_ERF, n_calib=512)
    _run(cfg, 9, seed=6)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_degenerate_ranges_all_and_none_flagged(dtype):
    cfg = W.LayerConfig("deg_" + dtype, 256, 1024, dtype=dtype, n_calib=256)
    L = _layer(cfg)
    x = W.make_tokens(cfg, 5, 1).cuda()
    inf = torch.full_like(L.lo, float("inf"))
    for lo, hi, frac in ((inf, inf, 1.0), (-inf, inf, 0.0)):
        L2 = W.Layer(**{**L.__dict__, "lo": lo, "hi": hi})
        s = L2.numpy64()
        h = T.fold_layer(L2)
        y, F, S = Hp.gpu_forward(h, L2, x, [1, 4])
        assert F.mean() == frac
        Hp.assert_parity(L2, s, x, y, F, S, label="degenerate", score_tol=1e-4)
        if frac == 1.0:   # every neuron flagged: the original GELU FFN
            dense = O.dense_ffn(x.double().cpu().numpy(), s["W1"], s["W2"], s["b1"], s["b2"], s["act"])
            assert O.rel_error(y.double().cpu().numpy(), dense).max() <= Hp.TOL[dtype]
        T.tardis_destroy(h)


def test_nan_token_is_flagged_everywhere_and_propagates():
    cfg = W.LayerConfig("nan", 256, 1024, dtype="bf16", n_calib=256)
    L = _layer(cfg)
    x = W.make_tokens(cfg, 3, 2).cuda()
    x[1, 7] = float("nan")
    h = T.fold_layer(L)
    y, F, S = Hp.gpu_forward(h, L, x, [3])
    assert F[1].all() and torch.isnan(y[1]).all()
    assert not torch.isnan(y[0]).any() and not torch.isnan(y[2]).any()
    T.tardis_destroy(h)


def test_forward_argument_errors_and_empty_call():
    cfg = W.LayerConfig("args", 128, 512, dtype="bf16", n_calib=256)
    L = _layer(cfg)
    h = T.fold_layer(L)
    lib = T.load_library()
    x = W.make_tokens(cfg, 2, 0).cuda()
    y = torch.empty_like(x)
    assert lib.tardis_ffn_forward(h, x.data_ptr(), y.data_ptr(), -1, None) == 1
    assert lib.tardis_ffn_forward(h, None, y.data_ptr(), 1, None) == 1
    assert lib.tardis_ffn_forward(h, x.data_ptr() + 2, y.data_ptr(), 1, None) == 1
    assert lib.tardis_ffn_forward(h, None, None, 0, None) == 0          # empty call is a no-op
    assert T.tardis_stats(h)["calls"] == 0
    T.tardis_destroy(h)


def test_run_to_run_flags_identical():
    cfg = W.LayerConfig("rep", 512, 2048, n_calib=512)
    L = _layer(cfg)
    x = W.make_tokens(cfg, 8, 0).cuda()
    h = T.fold_layer(L)
    y1, F1, S1 = Hp.gpu_forward(h, L, x, [8])
    y2, F2, S2 = Hp.gpu_forward(h, L, x, [8])
    # the fused kernel adds its partial scores in a fixed order: the captured scores of two runs are the same numbers
    assert (F1 == F2).all() and (S1 == S2).all()
    assert (y1.float() - y2.float()).abs().max() <= 2e-2 * y1.float().abs().max()
    T.tardis_destroy(h)


@pytest.mark.parametrize("d,h,G", [(512, 2048, 64), (4096, 16384, 128)])
def test_deterministic_mode_same_bits_run_to_run(d, h, G):
    """With tardis_set_deterministic on, y of repeated calls is the same bits (fused path at 1, 3, 4 and 9 tokens, batched
    path at 40 tokens), still agrees with the oracle, and other work in between (a call in the default mode, a call on
    another handle) does not change it."""
    cfg = W.LayerConfig("det", d, h, n_calib=512, group=G)
    L = _layer(cfg)
    s = L.numpy64()
    other = T.fold_layer(L)                                  # a second handle of the same layer, left in the default mode
    hd = T.fold_layer(L)
    try:
        T.tardis_set_deterministic(hd, True)
        for n in (1, 3, 4, 9, 40):
            x = W.make_tokens(cfg, n, 7 + n).cuda()
            outs = []
            for rep in range(4):
                y = torch.empty_like(x)
                T.tardis_ffn_forward(hd, x, y)
                torch.cuda.synchronize()
                outs.append(y.clone())
                yo = torch.empty_like(x)
                T.tardis_ffn_forward(other, x, yo)            # unrelated work between the repetitions
            for y in outs[1:]:
                assert torch.equal(y.view(torch.int16), outs[0].view(torch.int16)), "n = %d" % n
            assert T.tardis_stats(hd)["last_path"] == (2 if n <= 16 else 3)
            yg, F, S = Hp.gpu_forward(hd, L, x, [n])
            assert torch.equal(yg.view(torch.int16), outs[0].view(torch.int16))
            keep = np.arange(n)[: 6]
            ix = torch.as_tensor(keep).cuda()
            Hp.assert_parity(L, s, x[ix], yg[ix], F[keep], S[keep], score_tol=3e-4, label="det n=%d" % n)
        # switching the mode off again gives the default kernels back (same flags, y within the usual tolerance)
        T.tardis_set_deterministic(hd, False)
        x = W.make_tokens(cfg, 4, 99).cuda()
        y0 = torch.empty_like(x); y1 = torch.empty_like(x)
        T.tardis_ffn_forward(hd, x, y0)
        T.tardis_ffn_forward(other, x, y1)
        torch.cuda.synchronize()
        assert (y0.float() - y1.float()).abs().max() <= 2e-2 * y1.float().abs().max()
        assert T.tardis_stats(hd)["device_error"] == 0
    finally:
        T.tardis_destroy(hd)
        T.tardis_destroy(other)


def test_deterministic_mode_refused_where_only_atomic_kernels_serve():
    cfg = W.LayerConfig("detf32", 256, 1024, n_calib=512, dtype="f32")
    L = _layer(cfg)
    h = T.fold_layer(L)
    try:
        with pytest.raises(T.TardisError) as e:
            T.tardis_set_deterministic(h, True)
        assert e.value.status == 2
    finally:
        T.tardis_destroy(h)


@pytest.mark.parametrize("n,normalise,residual", [(1, True, True), (5, True, True), (40, True, True), (3, False, True), (4, True, False)])
def test_stack_forward_layer_by_layer_against_the_oracle(n, normalise, residual):
    """Three independently seeded layers chained on one stream.  With `keep`, every layer's input u_l and output f_l
    are read back: u_l against the oracle's layer normalisation of the stream the GPU itself had (rebuilt from the
    kept outputs, so that a flag that flips downstream of a bf16 rounding does not hide a layer's error), f_l against
    the oracle's forward on exactly u_l (flags and scores captured per layer), the final stream against the rounded
    sums.  The same call without `keep` (two work buffers in turns) gives the same y."""
    cfg = W.LayerConfig("stack", 512, 2048, n_calib=512)
    Ls = [_layer(cfg, seed=10 + l) for l in range(3)]
    hs = [T.fold_layer(L) for L in Ls]
    g = torch.Generator().manual_seed(3)
    gammas = [(1.0 + 0.1 * torch.randn(512, generator=g)).cuda() for _ in Ls]
    betas = [(0.1 * torch.randn(512, generator=g)).cuda() for _ in Ls]
    x = W.make_tokens(cfg, n, 21).cuda()
    try:
        caps = []
        for h in hs:
            bm = torch.zeros(n, 2048 // 32, dtype=torch.int32, device="cuda")
            sc = torch.full((n, 2048), float("nan"), dtype=torch.float64, device="cuda")
            T.tardis_set_debug_capture(h, bm, sc)
            caps.append((bm, sc))
        keep = torch.full((3, 2, n, 512), float("nan"), dtype=x.dtype, device="cuda")
        y = torch.empty_like(x)
        T.tardis_stack_forward(hs, x, y, gammas, betas, 1e-5, normalise, residual, keep=keep)
        torch.cuda.synchronize()
        for h in hs:
            T.tardis_set_debug_capture(h, None, None)
        stream = x.clone()
        for l, L in enumerate(Ls):
            u, f = keep[l, 0], keep[l, 1]
            if normalise:
                ref_u = O.layer_norm(stream.double().cpu().numpy(), gammas[l].double().cpu().numpy(), betas[l].double().cpu().numpy(), 1e-5)
                err = np.abs(u.double().cpu().numpy() - ref_u)
                assert (err <= 2.0 ** -8 * np.abs(ref_u) + 1e-6).all(), "layer %d: normalisation off by %.3e" % (l, err.max())
            else:
                assert torch.equal(u, stream)
            F = Hp.unpack_bitmap(caps[l][0], 2048)
            S = caps[l][1].cpu().numpy()
            Hp.assert_parity(L, L.numpy64(), u, f, F, S, score_tol=3e-4, label="stack layer %d" % l)
            stream = (stream.float() + f.float()).to(x.dtype) if residual else f.clone()
        assert torch.equal(y, stream)
        # without keep: same result from the two work buffers; in place as well
        y2 = torch.empty_like(x)
        T.tardis_stack_forward(hs, x, y2, gammas, betas, 1e-5, normalise, residual)
        x3 = x.clone()
        T.tardis_stack_forward(hs, x3, x3, gammas, betas, 1e-5, normalise, residual)
        torch.cuda.synchronize()
        tol = 2e-2 * float(y.float().abs().max())
        assert float((y2.float() - y.float()).abs().max()) <= tol and float((x3.float() - y.float()).abs().max()) <= tol
        # a buffer that is too small is refused
        with pytest.raises(T.TardisError) as e:
            T.tardis_stack_forward(hs, x, y2, gammas, betas, 1e-5, normalise, residual, work=torch.empty(n * 512, dtype=x.dtype, device="cuda"))
        assert e.value.status == 1
    finally:
        for h in hs:
            T.tardis_destroy(h)


@pytest.mark.parametrize("dtype,d,h", [("bf16", 512, 2048), ("f32", 256, 1024)])
def test_allocation_failures_return_a_status_and_leak_nothing(dtype, d, h):
    """Every device allocation of tardis_fold (and of what it prepares for the kernels) fails once in turn, injected through
    tardis_debug_fail_alloc: the call returns TARDIS_ERR_ALLOC, frees what it had, and a later fold of the same layer works
    and gives correct results.  The same for the buffers of the deterministic mode, the predictor builder and tardis_load."""
    import tempfile, os
    cfg = W.LayerConfig("allocfail", d, h, n_calib=512, dtype=dtype)
    L = _layer(cfg)
    torch.cuda.synchronize()
    live0 = T.tardis_debug_live_allocations()               # (other tests' handles are all destroyed: normally (0, 0))
    failed = 0
    try:
        for nth in range(200):
            T.tardis_debug_fail_alloc(nth)
            try:
                hd = T.fold_layer(L)
            except T.TardisError as e:
                assert e.status == 3, e.status
                failed += 1
                assert T.tardis_debug_live_allocations() == live0, "allocation %d: something left behind" % nth
                continue
            break                                            # nth is past the last allocation of a fold: it went through
        else:
            raise AssertionError("fold never succeeded")
        T.tardis_debug_fail_alloc(-1)
        assert failed >= 10, failed
        x = W.make_tokens(cfg, 3, 1).cuda()
        y, F, S = Hp.gpu_forward(hd, L, x, [3])
        Hp.assert_parity(L, L.numpy64(), x, y, F, S, score_tol=3e-4, label="after failures")
        if dtype == "bf16":
            T.tardis_debug_fail_alloc(0)
            with pytest.raises(T.TardisError):
                T.tardis_set_deterministic(hd, True)
            T.tardis_debug_fail_alloc(-1)
            T.tardis_set_deterministic(hd, True)
            T.tardis_set_deterministic(hd, False)
        path = os.path.join(tempfile.mkdtemp(), "layer.bin")
        T.tardis_save(hd, path)
        T.tardis_destroy(hd)
        hd = None
        assert T.tardis_debug_live_allocations() == live0
        for nth in (0, 3, 9):
            T.tardis_debug_fail_alloc(nth)
            with pytest.raises(T.TardisError) as e:
                T.tardis_load(path)
            assert e.value.status == 3
            assert T.tardis_debug_live_allocations() == live0
        for nth in range(5):
            T.tardis_debug_fail_alloc(nth)
            with pytest.raises(T.TardisError) as e:
                T.tardis_build_predictor(L.W1, None, 2, 64)
            assert e.value.status == 3
        T.tardis_debug_fail_alloc(-1)
        assert T.tardis_debug_live_allocations() == live0
    finally:
        T.tardis_debug_fail_alloc(-1)
        if hd:
            T.tardis_destroy(hd)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_guard_areas_report_a_write_past_a_buffer(dtype):
    """The buffers of a handle lie between guard areas that tardis_stats checks: untouched after real work on every path,
    reported as TARDIS_ERR_CORRUPT once four guard bytes in front of or behind a buffer have changed (changed here by
    tardis_debug_damage_guard, inside the allocation), and fine again after they are restored."""
    cfg = W.LayerConfig("guards", 512, 2048, n_calib=512, dtype=dtype)
    L = _layer(cfg)
    h = T.fold_layer(L)
    try:
        x = W.make_tokens(cfg, 70, 2).cuda()
        y = torch.empty_like(x)
        for n in (1, 4, 9, 70):
            T.tardis_ffn_forward(h, x[:n], y[:n])
        for path in (1, 3, 4, 0):
            T.tardis_set_path(h, path)
            T.tardis_ffn_forward(h, x[:5], y[:5])
        assert T.tardis_stats(h)["device_error"] == 0          # (reads every guard back)
        for front in (True, False):
            T.tardis_debug_damage_guard(h, front, False)
            with pytest.raises(T.TardisError) as e:
                T.tardis_stats(h)
            assert e.value.status == 6
            T.tardis_debug_damage_guard(h, front, True)
            assert T.tardis_stats(h)["device_error"] == 0
        T.tardis_ffn_forward(h, x[:3], y[:3])
        assert T.tardis_stats(h)["device_error"] == 0
    finally:
        T.tardis_destroy(h)


def test_batched_path_chunk_boundary_nan_token_and_empty_ranges():
    """More tokens than one scratch chunk in a single call (chunks hold 1024 tokens while the debug capture is on,
    2048 otherwise), a token holding a NaN in the middle of it, and the result compared token by token with the
    oracle on a seeded sample."""
    cfg = W.LayerConfig("chunks", 256, 1024, n_calib=512)
    L = _layer(cfg)
    s = L.numpy64()
    n = 1030
    x = W.make_tokens(cfg, n, 4).cuda()
    x[1027, 5] = float("nan")
    h = T.fold_layer(L)
    try:
        y, F, S = Hp.gpu_forward(h, L, x, [n])
        assert T.tardis_stats(h)["last_path"] == 3
        assert F[1027].all() and torch.isnan(y[1027]).all()
        keep = np.array([0, 1, 511, 1023, 1024, 1026, 1028, 1029])
        assert not torch.isnan(y[torch.as_tensor(keep).cuda()]).any()
        Hp.assert_parity(L, s, x[torch.as_tensor(keep).cuda()], y[torch.as_tensor(keep).cuda()], F[keep], S[keep],
                         score_tol=3e-4, label="chunks")
        st = T.tardis_stats(h)
        assert st["flagged_total"] == int(F.sum()) and st["device_error"] == 0
        # without the capture the chunks are twice as long: 2055 tokens cross that boundary too, and every token
        # must come out as it does in the captured run (same products, same order of accumulation)
        x2 = torch.cat([x, x[:1025]])
        y2 = torch.empty_like(x2)
        T.tardis_ffn_forward(h, x2, y2)
        torch.cuda.synchronize()
        ref2 = torch.cat([y, y[:1025]])
        ok = (y2 == ref2) | (torch.isnan(y2) & torch.isnan(ref2))
        assert bool(ok.all())
    finally:
        T.tardis_destroy(h)


def test_bounded_wait_runs_out_is_reported_and_cleared():
    """A device-side wait whose data never arrives ends by its limit, sets the error word (no trap, no hang: the kernel
    returns normally), tardis_stats reports the time-out, and after tardis_clear_error the handle works as before."""
    cfg = W.LayerConfig("timeout", 256, 1024, n_calib=256)
    L = _layer(cfg)
    s = L.numpy64()
    x = W.make_tokens(cfg, 3, 4).cuda()
    h = T.fold_layer(L)
    lib = T.load_library()
    y0, F0, _ = Hp.gpu_forward(h, L, x, [3])
    assert lib.tardis_debug_wait_timeout(h, 200000, None) == 0          # about 0.1 ms of waiting
    st = T.Stats()
    assert lib.tardis_stats(h, ctypes.byref(st)) == 5                   # TARDIS_ERR_TIMEOUT
    assert st.device_error == 1
    assert lib.tardis_clear_error(h) == 0
    assert lib.tardis_stats(h, ctypes.byref(st)) == 0 and st.device_error == 0
    y1, F1, _ = Hp.gpu_forward(h, L, x, [3])
    assert (F0 == F1).all()
    Hp.assert_parity(L, s, x, y1, F1, None, score_tol=None, label="after a cleared time-out")
    assert lib.tardis_debug_wait_timeout(h, -1, None) == 1
    T.tardis_destroy(h)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_save_and_load_round_trip(tmp_path, dtype):
    """A handle written to a file and read back gives the same flags and scores bit for bit, outputs within the parity
    tolerance of the oracle, and the same footprint; a damaged file is refused."""
    cfg = W.LayerConfig("saveload_" + dtype, 512, 2048, dtype=dtype, n_calib=512)
    L = _layer(cfg)
    s = L.numpy64()
    x = W.make_tokens(cfg, 21, 6).cuda()
    h = T.fold_layer(L)
    path = str(tmp_path / "layer.tardis")
    T.tardis_save(h, path)
    h2 = T.tardis_load(path)
    calls = [1, 4, 16]
    y1, F1, S1 = Hp.gpu_forward(h, L, x, calls)
    y2, F2, S2 = Hp.gpu_forward(h2, L, x, calls)
    assert (F1 == F2).all() and np.array_equal(S1, S2, equal_nan=True)
    Hp.assert_parity(L, s, x, y2, F2, None, score_tol=None, label="loaded handle")
    st1, st2 = T.tardis_stats(h), T.tardis_stats(h2)
    for k in ("bytes_folded", "bytes_predictor", "bytes_tables", "bytes_w1", "bytes_w2t"):
        assert st1[k] == st2[k]
    Wf1 = torch.empty(cfg.d_model, cfg.d_model, dtype=x.dtype, device="cuda")
    Wf2 = torch.empty_like(Wf1)
    T.tardis_export_folded(h, Wf1, None)
    T.tardis_export_folded(h2, Wf2, None)
    torch.cuda.synchronize()
    assert torch.equal(Wf1, Wf2)
    T.tardis_destroy(h)
    T.tardis_destroy(h2)
    # one flipped byte in the middle, and a truncated file: TARDIS_ERR_CORRUPT (6), no handle
    raw = bytearray(open(path, "rb").read())
    raw[len(raw) // 2] ^= 0x40
    bad = str(tmp_path / "bad.tardis")
    open(bad, "wb").write(raw)
    lib = T.load_library()
    out = ctypes.c_void_p()
    assert lib.tardis_load(bad.encode(), None, ctypes.byref(out)) == 6 and out.value is None
    open(bad, "wb").write(raw[:len(raw) // 3])
    assert lib.tardis_load(bad.encode(), None, ctypes.byref(out)) == 6 and out.value is None
