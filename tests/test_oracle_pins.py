"""Pins of the fp64 oracle against what the paper and the mathematics fix.
CPU only.  Each test states which plausible mistake it is meant to catch."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import tardis_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = np.array([float(t) for t in v])
    return out


def Phi(z):
    """Standard normal CDF through erfc (independent of the oracle's erf call)."""
    return 0.5 * math.erfc(-z / math.sqrt(2.0))


# ------------------------------------------------------------------ GELU
def test_gelu_closed_forms():
    # exact form: GELU(z) = z Phi(z); GELU(-2) = -2 Phi(-2) = -0.0455002639...
    assert O.gelu(-2.0, O.ACT_GELU_ERF) == pytest.approx(-2.0 * Phi(-2.0), abs=1e-15)
    assert -2.0 * Phi(-2.0) == pytest.approx(-0.04550026389635842, abs=1e-12)
    for act in (O.ACT_GELU_TANH, O.ACT_GELU_ERF):
        assert O.gelu(0.0, act) == 0.0
        z = np.linspace(-6, 6, 49)
        # odd-part identity GELU(z) - GELU(-z) = z (Phi(z) + Phi(-z) = 1; tanh is odd)
        np.testing.assert_allclose(O.gelu(z, act) - O.gelu(-z, act), z, atol=1e-14)
        assert O.gelu(30.0, act) == pytest.approx(30.0, abs=1e-12)
        assert abs(float(O.gelu(-30.0, act))) < 1e-12
    # the tanh form is the published approximation of the exact one: they agree to < 1e-3
    z = np.linspace(-8, 8, 4001)
    assert np.max(np.abs(O.gelu(z, O.ACT_GELU_TANH) - O.gelu(z, O.ACT_GELU_ERF))) < 1e-3
    # tanh-form value at -2 quoted to six digits (-0.045402)
    assert float(O.gelu(-2.0, O.ACT_GELU_TANH)) == pytest.approx(-0.0454023, abs=2e-7)
    # derivative at 0 is 1/2 for both forms (catches a dropped 0.5 or a wrong inner constant sign)
    for act in (O.ACT_GELU_TANH, O.ACT_GELU_ERF):
        e = 1e-6
        assert (float(O.gelu(e, act)) - float(O.gelu(-e, act))) / (2 * e) == pytest.approx(0.5, abs=1e-9)
    # second-order coefficient of the tanh form: GELU(z) ~ z/2 + z^2 sqrt(2/pi)/2 near 0
    e = 1e-3
    curv = (float(O.gelu(e)) + float(O.gelu(-e))) / (e * e)
    assert curv == pytest.approx(math.sqrt(2 / math.pi), rel=1e-5)


# ------------------------------------------------------------------ worked example (Section 4.2)
def _worked():
    g = read_golden("worked_example.txt")
    # nn.Linear layout: W1[h,d] row j = neuron j (paper's column j); W2[d,h] column j = paper's row j
    W1 = np.stack([g["W1_col1"], g["W1_col2"]])
    W2 = np.stack([g["W2_row1"], g["W2_row2"]]).T
    a = np.array([g["slope_intercept1"][0], g["slope_intercept2"][0]])
    c = np.array([g["slope_intercept1"][1], g["slope_intercept2"][1]])
    lo = np.array([g["range1"][0], g["range2"][0]])
    hi = np.array([g["range1"][1], g["range2"][1]])
    return g, W1, W2, a, c, lo, hi


def test_worked_example_fold_and_speculate():
    g, W1, W2, a, c, lo, hi = _worked()
    Wf, bf = O.fold(W1, W2, a, c)
    # paper convention C = W_f^T; values derived from the printed numbers
    np.testing.assert_allclose(Wf.T, [[-0.65, 0.1], [0.45, 0.2]], atol=1e-15)
    np.testing.assert_allclose(bf, [0.1, 0.2], atol=1e-15)
    y0 = O.speculate(Wf, bf, g["x"][None, :])
    np.testing.assert_allclose(y0[0], g["xC_plus_B"], atol=1e-15)   # printed: (0.3, -0.1)


def test_worked_example_flags_and_fix():
    g, W1, W2, a, c, lo, hi = _worked()
    x = g["x"][None, :]
    z = x @ W1.T
    np.testing.assert_allclose(z[0], g["z"][1:], atol=0)
    F = O.flags_from_score(z, lo, hi)
    assert F[0].tolist() == [bool(v) for v in g["flagged"]]          # neuron one flagged, two not
    Wf, bf = O.fold(W1, W2, a, c)
    y = O.fix(O.speculate(Wf, bf, x), x, F, W1, W2, a, c, act=O.ACT_GELU_ERF)
    # printed steps: (0.3,-0.1) - (0.4,0) + GELU(-2) (-1,0)
    gelu_m2 = -2.0 * Phi(-2.0)
    expect = g["xC_plus_B"] - g["subtracted"] + gelu_m2 * g["W2_row1"]
    np.testing.assert_allclose(y[0], expect, atol=1e-15)
    np.testing.assert_allclose(y[0], [-0.1 + 0.04550026389635842, -0.1], atol=1e-12)
    # the subtracted term itself: (a1 z1 + c1) * W2 row 1 = (0.4, 0)
    np.testing.assert_allclose((a[0] * z[0, 0] + c[0]) * W2[:, 0], g["subtracted"], atol=1e-15)


def test_fold_example_section_3_1():
    g = read_golden("fold_example.txt")
    W1 = np.stack([g["W1_col1"], g["W1_col2"]])
    W2 = np.stack([g["W2_row1"], g["W2_row2"]]).T
    prod = np.stack([g["W1W2_row1"], g["W1W2_row2"]])            # paper's W1 W2
    for slope in (1.0, 0.3, -2.0):
        Wf, bf = O.fold(W1, W2, np.full(2, slope), np.zeros(2))
        np.testing.assert_allclose(Wf.T, slope * prod, atol=1e-15)
        np.testing.assert_allclose(bf, 0, atol=0)
        x = np.array([[0.7, -1.3]])
        np.testing.assert_allclose(O.speculate(Wf, bf, x)[0],
                                   [slope * (-2 * 0.7 + 3 * -1.3), slope * (0.7 + 2 * -1.3)], atol=1e-15)
    d, h = 7, 28
    assert 1 - d * d / (2 * d * h) == g["param_reduction_h4d"][0]


# ------------------------------------------------------------------ invariants on random small problems
def _random_problem(rng, d, h, n, group=None, bias=True):
    W1 = rng.normal(size=(h, d))
    W2 = rng.normal(size=(d, h))
    b1 = rng.normal(size=h) if bias else None
    b2 = rng.normal(size=d) if bias else None
    a = rng.uniform(-0.2, 1.2, size=h)
    c = rng.normal(size=h) * 0.1
    x = rng.normal(size=(n, d))
    return W1, W2, b1, b2, a, c, x


def _loops_partially_linear(x, F, W1, W2, b1, b2, a, c, act):
    """The definition as scalar Python loops (brute force; no numpy contraction)."""
    n, d, h = len(x), len(x[0]), len(W1)
    y = [[0.0] * d for _ in range(n)]
    for t in range(n):
        for j in range(h):
            z = sum(W1[j][k] * x[t][k] for k in range(d)) + (b1[j] if b1 is not None else 0.0)
            if F[t][j]:
                u = math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)
                phi = 0.5 * z * (1.0 + math.tanh(u)) if act == O.ACT_GELU_TANH else z * Phi(z)
                if act == O.ACT_RELU:
                    phi = z if z > 0.0 else 0.0
            else:
                phi = a[j] * z + c[j]
            for i in range(d):
                y[t][i] += W2[i][j] * phi
        if b2 is not None:
            for i in range(d):
                y[t][i] += b2[i]
    return np.array(y)


@pytest.mark.parametrize("bias", [True, False])
def test_linear_activation_identity(bias):
    """With every activation replaced by its neuron's linear map the unfolded FFN equals
    W_f x + b_f (catches a transposed operand, a dropped a_j b1_j / c_j / b2 term)."""
    rng = np.random.default_rng(1)
    W1, W2, b1, b2, a, c, x = _random_problem(rng, 5, 11, 4, bias=bias)
    Wf, bf = O.fold(W1, W2, a, c, b1, b2)
    none = np.zeros((4, 11), dtype=bool)
    ref = _loops_partially_linear(x.tolist(), none, W1.tolist(), W2.tolist(),
                                  None if b1 is None else b1.tolist(), None if b2 is None else b2.tolist(),
                                  a.tolist(), c.tolist(), O.ACT_GELU_TANH)
    np.testing.assert_allclose(O.speculate(Wf, bf, x), ref, rtol=0, atol=1e-12)
    # no neuron flagged: fixing changes nothing
    np.testing.assert_array_equal(O.fix(O.speculate(Wf, bf, x), x, none, W1, W2, a, c, b1), O.speculate(Wf, bf, x))


@pytest.mark.parametrize("act", [O.ACT_GELU_TANH, O.ACT_GELU_ERF, O.ACT_RELU])
def test_all_flagged_equals_dense_ffn(act):
    rng = np.random.default_rng(2)
    W1, W2, b1, b2, a, c, x = _random_problem(rng, 6, 13, 5)
    Wf, bf = O.fold(W1, W2, a, c, b1, b2)
    allf = np.ones((5, 13), dtype=bool)
    y = O.fix(O.speculate(Wf, bf, x), x, allf, W1, W2, a, c, b1, act)
    ref = _loops_partially_linear(x.tolist(), allf, W1.tolist(), W2.tolist(), b1.tolist(), b2.tolist(),
                                  a.tolist(), c.tolist(), act)
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(O.dense_ffn(x, W1, W2, b1, b2, act), ref, rtol=0, atol=1e-12)


def test_brute_force_every_flag_subset():
    """d = 3, h = 8: for each of the 2^8 flag subsets fold + speculate + fix equals the scalar-loop
    definition, and so does the unfolded numpy definition."""
    rng = np.random.default_rng(3)
    d, h = 3, 8
    W1, W2, b1, b2, a, c, x = _random_problem(rng, d, h, 1)
    Wf, bf = O.fold(W1, W2, a, c, b1, b2)
    y0 = O.speculate(Wf, bf, x)
    for bits in itertools.product([False, True], repeat=h):
        F = np.array([bits])
        ref = _loops_partially_linear(x.tolist(), F, W1.tolist(), W2.tolist(), b1.tolist(), b2.tolist(),
                                      a.tolist(), c.tolist(), O.ACT_GELU_TANH)
        np.testing.assert_allclose(O.fix(y0, x, F, W1, W2, a, c, b1), ref, rtol=0, atol=1e-12)
        np.testing.assert_allclose(O.direct_partially_linear(x, F, W1, W2, a, c, b1, b2), ref, rtol=0, atol=1e-12)


def test_brute_force_d16_h16_random_subsets():
    rng = np.random.default_rng(4)
    d = h = 16
    W1, W2, b1, b2, a, c, x = _random_problem(rng, d, h, 3)
    Wf, bf = O.fold(W1, W2, a, c, b1, b2)
    for _ in range(40):
        F = rng.random((3, h)) < rng.random()
        ref = _loops_partially_linear(x.tolist(), F, W1.tolist(), W2.tolist(), b1.tolist(), b2.tolist(),
                                      a.tolist(), c.tolist(), O.ACT_GELU_TANH)
        np.testing.assert_allclose(O.fix(O.speculate(Wf, bf, x), x, F, W1, W2, a, c, b1), ref, rtol=0, atol=1e-11)


def test_fold_rows_matches_fold():
    rng = np.random.default_rng(5)
    W1, W2, b1, b2, a, c, x = _random_problem(rng, 9, 20, 1)
    Wf, _ = O.fold(W1, W2, a, c, b1, b2)
    np.testing.assert_allclose(O.fold_rows([7, 0, 3], W1, W2, a), Wf[[7, 0, 3]], atol=1e-13)
    # element-wise definition W_f[i,k] = sum_j W2[i,j] a_j W1[j,k]
    i, k = 4, 2
    assert Wf[i, k] == pytest.approx(sum(W2[i, j] * a[j] * W1[j, k] for j in range(20)), abs=1e-13)


# ------------------------------------------------------------------ predictor
def test_unpack_convention():
    # channel 0 in the two lowest bits, channel 15 in the two highest
    word = sum(v << (2 * p) for p, v in enumerate([1, 2, 3, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 3]))
    q = O.unpack_codes(np.array([[word, 0b11]], dtype=np.uint32), 32)
    assert q[0, :4].tolist() == [1, 2, 3, 0] and q[0, 15] == 3 and q[0, 16] == 3 and q[0, 17:].sum() == 0


def test_unpack_convention_4_and_8_bits():
    # The packing rule of the interface: with p = 32 / bits codes per word, channel k sits in word k / p, bits
    # bits * (k % p) upwards.  The words are written out by hand (hex digits = 4-bit codes, bytes = 8-bit codes).
    # 4 bits: word 0 holds channels 0..7 = 1,2,3,4,5,6,7,15 -> hex digits from the low end: 0xF7654321;
    #         word 1 holds channels 8..15 = 0,0,0,0,0,0,0,9 -> 0x90000000
    q4 = O.unpack_codes(np.array([[0xF7654321, 0x90000000]], dtype=np.uint32), 16, bits=4)
    assert q4[0].tolist() == [1, 2, 3, 4, 5, 6, 7, 15, 0, 0, 0, 0, 0, 0, 0, 9]
    # 8 bits: word 0 holds channels 0..3 = 0x01, 0x80, 0xFF, 0x10 -> 0x10FF8001; word 1 channels 4..7 = 7,0,0,200 -> 0xC8000007
    q8 = O.unpack_codes(np.array([[0x10FF8001, 0xC8000007]], dtype=np.uint32), 8, bits=8)
    assert q8[0].tolist() == [0x01, 0x80, 0xFF, 0x10, 7, 0, 0, 200]
    # a transposed field order (channel k in the HIGH bits first) would give other lists: check one against the wrong reading
    assert q4[0].tolist() != [15, 7, 6, 5, 4, 3, 2, 1, 9, 0, 0, 0, 0, 0, 0, 0]


@pytest.mark.parametrize("bits", [4, 8])
def test_predictor_score_scalar_loops_4_and_8_bits(bits):
    # scalar-loop evaluation of zhat = b1 + sum_g s (sum_k (q - zp) x) straight from hand-packed words, against the oracle
    rng = np.random.default_rng(100 + bits)
    per = 32 // bits
    h, d, G = 3, 32, 16
    q = rng.integers(0, 1 << bits, size=(h, d))
    words = np.zeros((h, d // per), dtype=np.uint32)
    for j in range(h):
        for k in range(d):
            words[j, k // per] |= np.uint32(int(q[j, k]) << (bits * (k % per)))
    s = rng.uniform(0.01, 0.1, size=(h, d // G))
    zp = rng.integers(0, 1 << bits, size=(h, d // G)).astype(np.uint8)
    b1 = rng.normal(size=h)
    x = rng.normal(size=(2, d))
    want = np.zeros((2, h))
    for t in range(2):
        for j in range(h):
            acc = b1[j]
            for g in range(d // G):
                inner = 0.0
                for k in range(g * G, (g + 1) * G):
                    inner += (int(q[j, k]) - int(zp[j, g])) * x[t, k]
                acc += s[j, g] * inner
            want[t, j] = acc
    got = O.predictor_score(x, words, s, zp, G, b1, bits)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    assert O.unpack_codes(words, d, bits).tolist() == q.tolist()


def _pack(q):
    h, d = q.shape
    w = np.zeros((h, d // 16), dtype=np.uint64)
    for p in range(16):
        w |= q[:, p::16].astype(np.uint64) << np.uint64(2 * p)
    return w.astype(np.uint32)


def test_predictor_hand_case():
    # 2 neurons, d = 16 = one group.  neuron 0: codes k%4, s = 0.5, zp = 1; neuron 1: all 3, s = 2, zp = 0
    q = np.stack([np.arange(16) % 4, np.full(16, 3)]).astype(np.uint8)
    x = np.arange(16, dtype=np.float64)[None, :] - 4.0
    s = np.array([[0.5], [2.0]])
    zp = np.array([[1], [0]], dtype=np.uint8)
    b1 = np.array([0.25, -1.0])
    zhat = O.predictor_score(x, _pack(q), s, zp, 16, b1)
    e0 = 0.25 + 0.5 * sum((k % 4 - 1) * (k - 4.0) for k in range(16))
    e1 = -1.0 + 2.0 * 3 * sum(k - 4.0 for k in range(16))
    np.testing.assert_allclose(zhat[0], [e0, e1], atol=1e-13)


def test_predictor_exact_special_case_is_a_gemv():
    """With unit scales, zero zero-points and integer weights in 0..3 the predictor's
    "compressed W1" is W1 itself, so the score is the textbook GEMV W1 x + b1."""
    rng = np.random.default_rng(6)
    h, d, G = 12, 64, 16
    q = rng.integers(0, 4, size=(h, d)).astype(np.uint8)
    x = rng.normal(size=(5, d))
    b1 = rng.normal(size=h)
    zhat = O.predictor_score(x, _pack(q), np.ones((h, d // G)), np.zeros((h, d // G), dtype=np.uint8), G, b1)
    ref = np.array([[sum(float(q[j, k]) * x[t, k] for k in range(d)) + b1[j] for j in range(h)] for t in range(5)])
    np.testing.assert_allclose(zhat, ref, atol=1e-12)


def test_predictor_groups_scales_zero_points_and_linearity():
    rng = np.random.default_rng(7)
    h, d, G = 6, 96, 32
    q = rng.integers(0, 4, size=(h, d)).astype(np.uint8)
    s = rng.uniform(0.01, 0.05, size=(h, d // G))
    zp = rng.integers(0, 4, size=(h, d // G)).astype(np.uint8)
    x = rng.normal(size=(3, d))
    zhat = O.predictor_score(x, _pack(q), s, zp, G)
    ref = np.zeros((3, h))
    for t in range(3):
        for j in range(h):
            for k in range(d):
                ref[t, j] += s[j, k // G] * (float(q[j, k]) - float(zp[j, k // G])) * x[t, k]
    np.testing.assert_allclose(zhat, ref, atol=1e-12)
    z2 = O.predictor_score(2.5 * x[:1] - x[1:2], _pack(q), s, zp, G)
    np.testing.assert_allclose(z2, 2.5 * zhat[:1] - zhat[1:2], atol=1e-12)


def test_flag_rule_half_open_and_nan():
    lo = np.array([-1.0, -1.0, -1.0, -1.0, -1.0])
    hi = np.array([2.0, 2.0, 2.0, 2.0, 2.0])
    z = np.array([[-1.0, 2.0, 0.0, np.nan, np.nextafter(2.0, 0.0)]])
    assert O.flags_from_score(z, lo, hi)[0].tolist() == [False, True, False, True, False]
    z = np.array([[-1.0 - 5e-7, 2.0 + 2e-6, 0.0, 1.0, -1.0 + 2e-6]])
    assert O.near_threshold(z, lo, hi)[0].tolist() == [True, False, False, False, False]


def test_full_path_composition():
    """tardis_ffn = the five steps in order; its output equals the unfolded definition under its own flags."""
    rng = np.random.default_rng(8)
    h, d, G = 32, 32, 16
    W1, W2, b1, b2, a, c, x = _random_problem(rng, d, h, 6)
    q = rng.integers(0, 4, size=(h, d)).astype(np.uint8)
    s = rng.uniform(0.3, 0.9, size=(h, d // G))
    zp = rng.integers(0, 4, size=(h, d // G)).astype(np.uint8)
    lo = rng.uniform(-6, -1, size=h)
    hi = rng.uniform(1, 6, size=h)
    y, F, zhat = O.tardis_ffn(x, W1, W2, a, c, lo, hi, _pack(q), s, zp, G, b1, b2)
    assert 0 < F.mean() < 1
    np.testing.assert_array_equal(F, ~((lo <= zhat) & (zhat < hi)))
    np.testing.assert_allclose(y, O.direct_partially_linear(x, F, W1, W2, a, c, b1, b2), atol=1e-11)


def test_rel_error_metric():
    y_ref = np.array([[3.0, 4.0, 0.0, 0.0]])            # rms = 2.5
    y = y_ref + np.array([[0.3, 0.0, 0.25, 0.0]])
    np.testing.assert_allclose(O.rel_error(y, y_ref)[0], [0.1, 0.0, 0.1, 0.0])


# ---- offline range / fit functions -------------------------------------------------------------------
def test_quantile_ranges_match_numpy_and_arithmetic_sequences():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((7, 257)).astype(np.float32)
    lo, hi = O.quantile_ranges(z, 0.05, 0.95)
    ref_lo = np.quantile(z.astype(np.float64), 0.05, axis=1, method="linear")
    ref_hi = np.quantile(z.astype(np.float64), 0.95, axis=1, method="linear")
    assert lo.dtype == np.float32 and hi.dtype == np.float32
    assert np.array_equal(lo, ref_lo.astype(np.float32)) and np.array_equal(hi, ref_hi.astype(np.float32))
    # samples 0, 1, ..., N-1 in any order: the quantile at level p is p (N - 1) itself
    N = 101
    seq = rng.permutation(N).astype(np.float64)[None, :]
    lo, hi = O.quantile_ranges(seq, 0.125, 0.9)
    assert lo[0] == np.float32(12.5) and hi[0] == np.float32(90.0)
    # p = 0 and p = 1 are the extremes; one sample: both ends are that sample
    lo, hi = O.quantile_ranges(z, 0.0, 1.0)
    assert np.array_equal(lo, z.min(1)) and np.array_equal(hi, z.max(1))
    lo, hi = O.quantile_ranges(np.array([[3.0]]), 0.3, 0.6)
    assert lo[0] == 3.0 and hi[0] == 3.0


@pytest.mark.parametrize("act", [O.ACT_GELU_TANH, O.ACT_GELU_ERF, O.ACT_RELU])
def test_least_squares_fit_normal_equations_polyfit_and_range_rule(act):
    rng = np.random.default_rng(6)
    z = (rng.standard_normal((5, 400)) * 1.3).astype(np.float32)
    lo = np.array([-1.0, -0.5, -2.0, 0.0, -3.0], dtype=np.float32)
    hi = np.array([0.5, 0.25, 2.0, 1.5, 3.0], dtype=np.float32)
    a, c = O.least_squares_fit(z, lo, hi, act)
    for j in range(5):
        zz = z[j].astype(np.float64)
        zz = zz[(zz >= lo[j]) & (zz < hi[j])]
        sg = O.gelu(zz, act)
        # library cross-check: degree-1 polynomial least squares
        pa, pc = np.polyfit(zz, sg, 1)
        assert abs(a[j] - pa) <= 2e-6 * max(1.0, abs(pa)) and abs(c[j] - pc) <= 2e-6 * max(1.0, abs(pc))
        # normal equations: the residual is orthogonal to 1 and to z (float32 rounding of a, c allowed for)
        r = sg - (float(a[j]) * zz + float(c[j]))
        assert abs(r.sum()) <= 1e-5 * zz.size and abs((r * zz).sum()) <= 1e-5 * zz.size
    # half-open range: a sample equal to hi is outside, one equal to lo is inside
    zz = np.array([[0.0, 1.0, 2.0, 5.0]])
    a1, c1 = O.least_squares_fit(zz, np.array([0.0], np.float32), np.array([2.0], np.float32), act)
    g0, g1 = O.gelu(0.0, act), O.gelu(1.0, act)
    assert abs(a1[0] - (g1 - g0)) < 1e-6 and abs(c1[0] - g0) < 1e-6          # the line through the two samples in range


@pytest.mark.parametrize("act", [O.ACT_GELU_TANH, O.ACT_GELU_ERF])
def test_least_squares_fit_degenerate_takes_the_tangent_at_the_midpoint(act):
    # no sample in range / a single one / identical ones: tangent of GELU at (lo + hi) / 2
    z = np.array([[5.0, 6.0, 7.0], [0.25, 9.0, 9.5], [0.5, 0.5, 0.5]])
    lo = np.array([-1.0, 0.0, 0.0], np.float32)
    hi = np.array([1.0, 1.0, 1.0], np.float32)
    a, c = O.least_squares_fit(z, lo, hi, act)
    for j in range(3):
        m = 0.5 * (float(lo[j]) + float(hi[j]))
        eps = 1e-6
        slope = (O.gelu(m + eps, act) - O.gelu(m - eps, act)) / (2 * eps)      # derivative pinned numerically
        assert abs(a[j] - slope) < 1e-6 and abs(c[j] - (O.gelu(m, act) - slope * m)) < 1e-6
    # a neuron that is linear where it is sampled: GELU(z) -> z for large z, so a -> 1, c -> 0
    zz = np.linspace(20.0, 30.0, 50)[None, :]
    a, c = O.least_squares_fit(zz, np.array([0.0], np.float32), np.array([100.0], np.float32), act)
    assert abs(a[0] - 1.0) < 1e-6 and abs(c[0]) < 1e-5


def test_relu_values_and_fit_special_cases():
    z = np.array([-3.0, -0.0, 0.0, 1e-300, 2.5])
    np.testing.assert_array_equal(O.gelu(z, O.ACT_RELU), np.array([0.0, 0.0, 0.0, 1e-300, 2.5]))
    assert np.isnan(O.gelu(np.array([np.nan]), O.ACT_RELU))[0]
    np.testing.assert_array_equal(O.gelu_derivative(np.array([-1.0, 0.0, 2.0]), O.ACT_RELU), np.array([0.0, 0.0, 1.0]))
    # a range left of zero fits the zero function, one right of zero the identity: the linear function is then
    # exact inside the range, which is why one function serves ReLU models at every ratio (Section 7.2)
    rng = np.random.default_rng(9)
    zz = rng.standard_normal((2, 300))
    a, c = O.least_squares_fit(zz, np.array([-5.0, 0.0], np.float32), np.array([0.0, 5.0], np.float32), O.ACT_RELU)
    assert a[0] == 0.0 and c[0] == 0.0 and abs(a[1] - 1.0) < 1e-7 and abs(c[1]) < 1e-7
    # degenerate fallback: the tangent at the midpoint is 0 left of zero and the identity right of it
    a, c = O.least_squares_fit(np.array([[9.0], [9.0]]), np.array([-2.0, 1.0], np.float32), np.array([-1.0, 2.0], np.float32),
                               O.ACT_RELU)
    assert (a[0], c[0], a[1], c[1]) == (0.0, 0.0, 1.0, 0.0)


# ------------------------------------------------------------------ Algorithm 1: range search (Section 5.1.1)
def test_kde_centroid_against_library_kde_and_special_cases():
    from scipy.stats import gaussian_kde
    rng = np.random.default_rng(7)
    z = np.concatenate([rng.normal(-1.0, 0.3, 300), rng.normal(2.0, 1.0, 100)])       # dense cluster + sparse cluster
    c = O.kde_centroid(z)
    # library KDE with the same kernel width (factor times the sample standard deviation), evaluated at the samples
    kde = gaussian_kde(z, bw_method=1.06 * z.size ** -0.2)
    zs = np.sort(z)
    assert c == zs[int(np.argmax(kde(zs)))]
    assert -1.6 < c < -0.4                                  # the search starts in the denser cluster
    # shifting the samples shifts the centroid; all-equal samples and a single sample give that value
    assert O.kde_centroid(z + 3.0) == pytest.approx(c + 3.0, abs=1e-12)
    assert O.kde_centroid(np.full(9, 0.25)) == 0.25 and O.kde_centroid([1.5]) == 1.5
    # symmetric samples with one centre point: the centre is the densest point
    sym = np.concatenate([-np.arange(1, 40) ** 1.3, [0.0], np.arange(1, 40) ** 1.3]) * 0.01
    assert O.kde_centroid(sym) == 0.0


def test_approx_error_against_polyfit_and_exact_cases():
    rng = np.random.default_rng(8)
    z = rng.normal(size=400) * 1.5
    lo, hi = -1.0, 0.7
    zin = z[(z >= lo) & (z < hi)]
    g = O.gelu(zin, O.ACT_GELU_TANH)
    coef, res, *_ = np.polyfit(zin, g, 1, full=True)         # library least squares: sum of squared residuals
    assert O.approx_error(z, lo, hi) == pytest.approx(res[0] / zin.size, rel=1e-9)
    # ReLU is a straight line on either side of 0: no error there, some across the kink
    assert O.approx_error(z, 0.0, 5.0, O.ACT_RELU) == pytest.approx(0.0, abs=1e-25)
    assert O.approx_error(z, -5.0, 0.0, O.ACT_RELU) == 0.0
    assert O.approx_error(z, -1.0, 1.0, O.ACT_RELU) > 1e-3
    # half-open range and the fewer-than-two rule
    assert O.approx_error([0.0, 1.0, 2.0], 0.0, 2.0) == O.approx_error([0.0, 1.0], 0.0, 2.0) == pytest.approx(0.0, abs=1e-30)
    assert O.approx_error([0.5], 0.0, 1.0) == 0.0 and O.approx_error([3.0, 4.0], 0.0, 1.0) == 0.0


def test_greedy_range_search_properties_and_closed_form_trace():
    rng = np.random.default_rng(9)
    z = np.sort(rng.standard_t(4, size=300) * 0.8 - 0.3)
    for t, step in ((0.5, 0.05), (0.85, 0.02), (0.97, 0.1)):
        lo, hi, trace, margin = O.greedy_range_search(z, t, step, return_trace=True)
        c = O.kde_centroid(z)
        inside = ((z >= lo) & (z < hi)).mean()
        assert inside >= t                                     # the threshold is reached ...
        kl, kr = trace.count("L"), trace.count("R")
        assert lo == c - kl * step and hi == c + kr * step and lo <= c <= hi
        # ... and was not reached one step earlier (the last step is undone on its side)
        if trace[-1] == "L":
            assert ((z >= lo + step) & (z < hi)).mean() < t
        else:
            assert ((z >= lo) & (z < hi - step)).mean() < t
    # every decision re-derived from a library fit: the side with the smaller mean squared residual (right on ties)
    lo, hi, trace, margin = O.greedy_range_search(z, 0.6, 0.05, return_trace=True)
    c, kl, kr = O.kde_centroid(z), 0, 0

    def mse(a, b):
        zin = z[(z >= a) & (z < b)]
        if zin.size < 2 or np.ptp(zin) == 0:
            return 0.0
        g = O.gelu(zin, O.ACT_GELU_TANH)
        p = np.polyfit(zin, g, 1)
        return float(np.mean((g - np.polyval(p, zin)) ** 2))
    for ch in trace:
        lo_c, hi_c = c - kl * 0.05, c + kr * 0.05
        if hi_c > z[-1]:
            want = "L"
        elif lo_c <= z[0]:
            want = "R"
        else:
            el, er = mse(c - (kl + 1) * 0.05, hi_c), mse(lo_c, c + (kr + 1) * 0.05)
            want = "L" if el < er else "R"
            if abs(el - er) <= 1e-9 * max(el, er):
                want = ch                                  # a near-tie may go either way in another summation order
        assert ch == want
        kl, kr = kl + (ch == "L"), kr + (ch == "R")
    # closed form: ReLU on positive samples has zero error on both sides at every step, ties go right, and once the range
    # has passed the largest sample the left side is taken: R ... R L ... L
    zp = np.linspace(1.0, 3.0, 41)
    lo, hi, trace, _ = O.greedy_range_search(zp, 0.9, 0.25, O.ACT_RELU, return_trace=True)
    s = "".join(trace)
    assert s == "R" * s.count("R") + "L" * s.count("L") and s.count("R") >= 1
    assert hi > zp[-1] and ((zp >= lo) & (zp < hi)).mean() >= 0.9


def test_neuron_thresholds_against_library_lp():
    from scipy.optimize import linprog
    rng = np.random.default_rng(10)
    err = rng.uniform(0.1, 2.0, size=12)
    t = O.neuron_thresholds(err, 0.8, 0.6, 0.95)
    assert t.sum() == pytest.approx(0.8 * 12) and t.min() >= 0.6 - 1e-12 and t.max() <= 0.95 + 1e-12
    lp = linprog(err, A_eq=np.ones((1, 12)), b_eq=[0.8 * 12], bounds=[(0.6, 0.95)] * 12)
    assert float(err @ t) == pytest.approx(lp.fun, rel=1e-9)
    np.testing.assert_allclose(t, lp.x, atol=1e-7)
    # the neurons with the largest error keep the lowest threshold
    assert t[np.argmax(err)] == 0.6 and t[np.argmin(err)] == 0.95


def test_layer_norm_and_stack_against_library_and_closed_forms():
    """layer_norm: the library routine of torch on the same rows (another implementation), rows of known statistics
    (a row a + b k normalises to the standardised ramp whatever a and b > 0 are; a constant row gives beta), invariance
    under shift and positive scaling of the input (eps = 0), mean 0 / variance 1 of the output.  stack_forward: linear
    stand-in layers give a closed form (residual: product of (I + M_l); none: product of M_l), and the kept inputs and
    outputs are consistent with the final stream."""
    import torch
    rng = np.random.default_rng(5)
    v = rng.standard_normal((7, 48)) * 3 + 1.5
    g, b = rng.standard_normal(48), rng.standard_normal(48)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(v), (48,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    np.testing.assert_allclose(O.layer_norm(v, g, b, 1e-5), ref, rtol=1e-12, atol=1e-12)
    out = O.layer_norm(v, None, None, 0.0)
    np.testing.assert_allclose(out.mean(axis=1), 0.0, atol=1e-13)
    np.testing.assert_allclose((out ** 2).mean(axis=1), 1.0, rtol=1e-12)
    np.testing.assert_allclose(O.layer_norm(4.0 * v - 9.0, None, None, 0.0), out, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(O.layer_norm(-v, None, None, 0.0), -out, rtol=1e-12, atol=1e-13)   # a sign error in the centring shows here
    k = np.arange(9.0)
    ramp = (k - 4.0) / math.sqrt(60.0 / 9.0)                       # mean 4, variance (sum (k-4)^2)/9 = 60/9
    np.testing.assert_allclose(O.layer_norm((2.0 + 0.5 * k)[None, :], None, None, 0.0)[0], ramp, rtol=1e-12)
    np.testing.assert_allclose(O.layer_norm(np.full((1, 9), 3.0), g[:9], b[:9], 1e-5)[0], b[:9], atol=1e-12)
    # eps enters under the root: variance 60/9, eps 1 -> divisor sqrt(60/9 + 1)
    np.testing.assert_allclose(O.layer_norm(k[None, :], None, None, 1.0)[0], (k - 4.0) / math.sqrt(60.0 / 9.0 + 1.0), rtol=1e-12)

    Ms = [rng.standard_normal((6, 6)) * 0.3 for _ in range(3)]
    ffns = [lambda u, M=M: u @ M.T for M in Ms]
    x = rng.standard_normal((4, 6))
    y, us, fs = O.stack_forward(x, ffns, normalise=False, residual=True)
    P = np.eye(6)
    for M in Ms:
        P = (np.eye(6) + M) @ P
    np.testing.assert_allclose(y, x @ P.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(y, x + fs[0] + fs[1] + fs[2], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(us[1], x + fs[0], rtol=1e-12, atol=1e-12)
    y2, _, _ = O.stack_forward(x, ffns, normalise=False, residual=False)
    np.testing.assert_allclose(y2, x @ (Ms[2] @ Ms[1] @ Ms[0]).T, rtol=1e-12, atol=1e-12)
    y3, us3, fs3 = O.stack_forward(x, ffns, gammas=[g[:6]] * 3, betas=[b[:6]] * 3, eps=1e-5, normalise=True, residual=True)
    np.testing.assert_allclose(us3[2], O.layer_norm(x + fs3[0] + fs3[1], g[:6], b[:6], 1e-5), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(fs3[2], us3[2] @ Ms[2].T, rtol=1e-12, atol=1e-12)


def test_gptq_quantise_identities_and_special_cases():
    """round_to_storage against torch's conversions (another implementation of the same format); group_grid on a hand
    example; gptq_quantise: with U = identity it is rounding to nearest on the group's grid (and the errors are the plain
    residuals); with a general U the recorded errors reproduce the result exactly through W - E U = dequantised codes
    (the defining recurrence unrolled: a wrong sign, a wrong row of U or an off-by-one in `later channels` breaks it);
    a two-channel case worked by hand; on correlated inputs the output error ||X (W - What)^T|| is smaller than with
    plain rounding (what the procedure is for); pack_codes inverts unpack_codes."""
    import torch
    rng = np.random.default_rng(11)
    v = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-6, 6, 4000), [0.0, 1.0, -2.5, 3.0e-39]])
    np.testing.assert_array_equal(O.round_to_storage(v, "bf16"), torch.from_numpy(v).float().bfloat16().double().numpy())
    np.testing.assert_array_equal(O.round_to_storage(v, "f32"), torch.from_numpy(v).float().double().numpy())
    # grid by hand: weights -1 .. 2, 2 bits: scale 1, zero 1; all positive 0.5 .. 2: range widened to 0: scale 2/3 -> bf16
    s, z = O.group_grid(np.array([[-1.0, 0.25, 2.0, 1.0]]), 2, "f32")
    assert s[0] == 1.0 and z[0] == 1.0
    s, z = O.group_grid(np.array([[0.5, 2.0, 1.0, 1.5]]), 2, "bf16")
    assert s[0] == 0.66796875 and z[0] == 0.0                       # 2/3 in bf16 = 171 / 256
    s, z = O.group_grid(np.zeros((1, 4)), 2, "bf16")
    assert s[0] == 1.0 and z[0] == 0.0

    h, d, G = 6, 32, 16
    W = rng.standard_normal((h, d))
    q, sc, zp, E = O.gptq_quantise(W, None, G, 2, "f32")
    for j in range(h):
        for g in range(d // G):
            wg = W[j, g * G:(g + 1) * G]
            s_, z_ = O.group_grid(wg[None, :], 2, "f32")
            np.testing.assert_array_equal(q[j, g * G:(g + 1) * G], np.clip(np.rint(wg / s_[0] + z_[0]), 0, 3))
    deq = (q.reshape(h, d // G, G) - zp[:, :, None]) * sc[:, :, None]
    np.testing.assert_allclose(E, W - deq.reshape(h, d), rtol=0, atol=1e-15)

    X = rng.standard_normal((200, d)) @ (np.eye(d) + 0.6 * rng.standard_normal((d, d)))      # correlated channels
    H = 2.0 / 200 * X.T @ X + 0.01 * np.mean(np.diag(2.0 / 200 * X.T @ X)) * np.eye(d)
    U = np.linalg.cholesky(np.linalg.inv(H)).T                                                   # upper: U^T U = H^-1
    np.testing.assert_allclose(U.T @ U, np.linalg.inv(H), rtol=1e-9, atol=1e-12)
    q2, sc2, zp2, E2 = O.gptq_quantise(W, U, G, 2, "f32")
    deq2 = ((q2.reshape(h, d // G, G) - zp2[:, :, None]) * sc2[:, :, None]).reshape(h, d)
    np.testing.assert_allclose(W - E2 @ np.triu(U), deq2, rtol=1e-10, atol=1e-10)
    err_rtn = np.linalg.norm(X @ (W - deq.reshape(h, d)).T)
    err_gptq = np.linalg.norm(X @ (W - deq2).T)
    assert err_gptq < 0.9 * err_rtn, (err_gptq, err_rtn)
    # two channels, one group, by hand: w = (0.9, 1.4), 2 bits, range [0, 1.4] -> scale 1.4/3, zero 0;
    # q0 = rint(0.9 / s) = 2, e0 = (0.9 - 2 s) / u00, w1 <- 1.4 - e0 u01, q1 = rint(w1 / s)
    U2 = np.array([[2.0, 0.5], [0.0, 1.0]])
    qh, sh, zh, Eh = O.gptq_quantise(np.array([[0.9, 1.4]]), U2, 2, 2, "f32")
    s_ = float(np.float32(1.4 / 3))
    e0 = (0.9 - 2 * s_) / 2.0
    w1 = 1.4 - e0 * 0.5
    assert sh[0, 0] == s_ and zh[0, 0] == 0 and qh[0, 0] == 2 and qh[0, 1] == int(np.rint(w1 / s_))
    np.testing.assert_allclose(Eh[0], [e0, (w1 - s_ * qh[0, 1]) / 1.0], rtol=1e-15)
    for bits in (2, 3, 4, 8):
        qq = rng.integers(0, 1 << bits, (5, 64)).astype(np.uint8)
        np.testing.assert_array_equal(O.unpack_codes(O.pack_codes(qq, bits), 64, bits), qq)


def test_unpack_convention_3_bits_bit_stream():
    """3-bit codes are a bit stream over the row's words: 32 codes fill three words, code 10 starts at bit 30 of word 0 and
    ends in bit 0 of word 1, code 21 starts at bit 31 of word 1.  Words written out by hand from the codes 0..7 repeating
    (k mod 8), and a scalar-loop score on them."""
    codes = [k % 8 for k in range(32)]
    bits_str = "".join("".join(str((c >> b) & 1) for b in range(3)) for c in codes)       # the stream, first bit first
    words = [int(bits_str[32 * w:32 * (w + 1)][::-1], 2) for w in range(3)]
    # by hand: codes 0,1,2,...: word 0 = 0b10_110_101_100_011_010_001_000 ... the low 9 bits are 0b010_001_000 = 0x88
    assert words[0] & 0x1FF == 0b010001000
    # code 10 (= 2 = 0b010): bits 30, 31 of word 0 are 0, 1; bit 0 of word 1 is 0
    assert (words[0] >> 30) & 3 == 0b10 and words[1] & 1 == 0
    # code 21 (= 5 = 0b101): bit 31 of word 1 is 1, bits 0, 1 of word 2 are 0, 1
    assert (words[1] >> 31) & 1 == 1 and words[2] & 3 == 0b10
    q = O.unpack_codes(np.array([words], dtype=np.uint32), 32, 3)
    assert q.tolist() == [codes]
    assert O.pack_codes(np.array([codes], dtype=np.uint8), 3).tolist() == [words]
    x = np.arange(1.0, 33.0)[None, :] / 7.0
    scale, zero = np.array([[0.25, 0.5]]), np.array([[3.0, 4.0]])
    z = O.predictor_score(x, np.array([words], dtype=np.uint32), scale, zero, 16, np.array([0.125]), 3)
    ref = 0.125
    for g in range(2):
        inner = 0.0
        for k in range(16 * g, 16 * g + 16):
            inner += (codes[k] - zero[0, g]) * x[0, k]
        ref += scale[0, g] * inner
    assert abs(z[0, 0] - ref) < 1e-12
