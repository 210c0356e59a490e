"""fp64 CPU oracle of the TARDIS partially linear FFN forward (arXiv 2501.10054).

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and
the CPU-baseline / reference arm of the benchmark may import this module.  It
shares no code with the CUDA library and never calls it; the CUDA library never
calls this.  Everything here is plain numpy in float64, written in the order
and notation of the paper so it can be checked against the paper by eye.

Notation bridge.  The paper writes row vectors, FFN(x) = sigma(x W1) W2 with
W1 in R^{d x h}, W2 in R^{h x d}; neuron n is column n of W1 and row n of W2
(Section 3.1, Section 5.1).  This module uses the nn.Linear storage layout:

    W1[h, d]  row j    = neuron j's input weights   (paper: column j of W1)
    W2[d, h]  column j = neuron j's output weights  (paper: row j of W2)

so W_f = W2 diag(a) W1 is the transpose of the paper's folded matrix C and
b_f is the paper's B (with the biases b1, b2 the paper drops for presentation,
Section 3.1 footnote).  Slope/intercept (a_j, c_j) are the paper's (a, b) of
the per-neuron linear function on the half-open range [l1, l2) = [lo_j, hi_j)
(Section 5.1.1).

Pins (tests, CPU only): the worked two-neuron example of Section 4.2, the fold
example of Section 3.1, the linear-activation identity, the all-flagged = dense
GELU FFN identity, brute force over every flag subset for d, h <= 16, the
exact-predictor special case, closed forms of GELU, the packing convention;
for the offline range / fit functions: the quantile routine of numpy, arithmetic
sequences, the normal equations, numpy's polynomial fit, two-sample lines and
the analytic tangent.  No function in this file is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

ACT_GELU_TANH = 0
ACT_GELU_ERF = 1
ACT_RELU = 2

_F64 = np.float64


def _as64(v):
    return np.ascontiguousarray(np.asarray(v, dtype=_F64))


# --------------------------------------------------------------------------
# activation
# --------------------------------------------------------------------------
def gelu(z, act=ACT_GELU_TANH):
    """The activation sigma in float64.  The paper only says "GELU" (Section
    3.2); both common forms are provided: tanh form 0.5 z (1 + tanh(sqrt(2/pi)
    (z + 0.044715 z^3))) and the exact form z * Phi(z) with Phi the standard
    normal CDF.  ReLU, max(z, 0), is the activation of the OPT model in the
    paper's evaluation (Section 7.1)."""
    z = np.asarray(z, dtype=_F64)
    if act == ACT_GELU_TANH:
        u = math.sqrt(2.0 / math.pi) * (z + 0.044715 * z * z * z)
        return 0.5 * z * (1.0 + np.tanh(u))
    if act == ACT_GELU_ERF:
        from scipy.special import erf          # library primitive: the error function
        return 0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))
    if act == ACT_RELU:
        return np.where(z > 0.0, z, 0.0 * z)              # 0 * z keeps NaN a NaN
    raise ValueError("unknown activation %r" % (act,))


# --------------------------------------------------------------------------
# predictor state format
# --------------------------------------------------------------------------
def unpack_codes(codes_u32, d, bits=2):
    """Expand packed predictor codes to one integer per weight.

    Packed layout: row j is one bit stream over its 32-bit words, lowest bits first; input channel k holds the bits
    [bits k, bits (k + 1)) of it.  With 2, 4 or 8 bits per code that is 32/bits codes per word; a 3-bit code may start in
    one word and go on in the lowest bits of the next.  Returns uint8 [h, d]."""
    codes_u32 = np.asarray(codes_u32, dtype=np.uint32)
    h, nw = codes_u32.shape
    if nw * 32 != d * bits:
        raise ValueError("codes row has %d words, expected %d" % (nw, d * bits // 32))
    if 32 % bits == 0:                      # a code never leaves its word: 32/bits codes per word
        per = 32 // bits
        q = np.empty((h, d), dtype=np.uint8)
        mask = np.uint32((1 << bits) - 1)
        for p in range(per):
            q[:, p::per] = ((codes_u32 >> np.uint32(bits * p)) & mask).astype(np.uint8)
        return q
    # the stream as single bits, then `bits` of them per channel, the lowest first
    stream = (codes_u32[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & np.uint32(1)
    per_code = stream.reshape(h, d, bits).astype(np.uint32)
    q = np.zeros((h, d), dtype=np.uint32)
    for b in range(bits):
        q |= per_code[:, :, b] << np.uint32(b)
    return q.astype(np.uint8)


def predictor_score(x, codes_u32, scale, zero, group, b1=None, bits=2):
    """Predictor score of Section 5.3: the pre-activation computed from the
    compressed (quantised) copy of W1 instead of W1 itself.

        zhat[t, j] = b1_j + sum_g s[j,g] * sum_{k in g} (q[j,k] - zp[j,g]) * x[t,k]

    x [n, d]; codes packed uint32 [h, d*bits/32]; scale, zero [h, d/group]."""
    x = _as64(x)
    n, d = x.shape
    q = unpack_codes(codes_u32, d, bits).astype(_F64)
    h = q.shape[0]
    scale = _as64(scale)
    zero = _as64(zero)
    ng = d // group
    if scale.shape != (h, ng) or zero.shape != (h, ng):
        raise ValueError("scale/zero must be [h, d/group]")
    zhat = np.zeros((n, h), dtype=_F64)
    for g in range(ng):
        ks = slice(g * group, (g + 1) * group)
        centred = q[:, ks] - zero[:, g:g + 1]            # (q - zp), [h, group]
        zhat += (x[:, ks] @ centred.T) * scale[:, g][None, :]
    if b1 is not None:
        zhat += _as64(b1)[None, :]
    return zhat


def flags_from_score(zhat, lo, hi):
    """A neuron is flagged when its (predicted) pre-activation is outside the
    half-open linear range [lo, hi) of Section 5.1.1.  Written as the negation
    of the in-range test so that NaN scores are flagged."""
    zhat = _as64(zhat)
    lo = _as64(lo)[None, :]
    hi = _as64(hi)[None, :]
    with np.errstate(invalid="ignore"):
        inside = (lo <= zhat) & (zhat < hi)
    return ~inside


def near_threshold(zhat, lo, hi, band=1e-6):
    """Neurons whose score lies within `band` of either range end; their flag
    is excluded from bit-exact comparison and reported instead."""
    zhat = _as64(zhat)
    return (np.abs(zhat - _as64(lo)[None, :]) < band) | (np.abs(zhat - _as64(hi)[None, :]) < band)


# --------------------------------------------------------------------------
# offline: constant folding (Section 5.2)
# --------------------------------------------------------------------------
def fold(W1, W2, a, c, b1=None, b2=None):
    """Constant folding.  Per neuron CF gives (a_j * outer(W2[:,j], W1[j,:]),
    c_j * W2[:,j]); summed over neurons:

        W_f[i,k] = sum_j W2[i,j] a_j W1[j,k]
        b_f[i]   = sum_j W2[i,j] (a_j b1_j + c_j) + b2_i
    """
    W1 = _as64(W1)
    W2 = _as64(W2)
    a = _as64(a)
    c = _as64(c)
    h, d = W1.shape
    b1v = np.zeros(h) if b1 is None else _as64(b1)
    b2v = np.zeros(d) if b2 is None else _as64(b2)
    Wf = (W2 * a[None, :]) @ W1
    bf = W2 @ (a * b1v + c) + b2v
    return Wf, bf


def fold_rows(rows, W1, W2, a):
    """Rows `rows` of W_f only (for sampled checks at sizes where the whole
    d x d fold is too slow on a CPU)."""
    W1 = _as64(W1)
    a = _as64(a)
    W2r = _as64(np.asarray(W2)[np.asarray(rows)])
    return (W2r * a[None, :]) @ W1


# --------------------------------------------------------------------------
# online: speculate, then fix (Section 5.4)
# --------------------------------------------------------------------------
def speculate(Wf, bf, x):
    """Speculative approximation: every neuron assumed in range, y0 = W_f x + b_f."""
    return _as64(x) @ _as64(Wf).T + _as64(bf)[None, :]


def fix(y0, x, F, W1, W2, a, c, b1=None, act=ACT_GELU_TANH):
    """Result fixing.  For every flagged neuron j of token t: recompute the true
    pre-activation z_j from the original W1 row, take away the linear value that
    the folded product already contains and add the true activation:

        y[t,:] += W2[:,j] * (GELU(z_j) - a_j z_j - c_j)

    The predictor's flags define the result: a flagged neuron is replaced even
    if its true z_j is inside the range, an unflagged one keeps the linear value."""
    x = _as64(x)
    W1 = _as64(W1)
    W2 = _as64(W2)
    a = _as64(a)
    c = _as64(c)
    F = np.asarray(F, dtype=bool)
    y = _as64(y0).copy()
    for t in range(x.shape[0]):
        idx = np.nonzero(F[t])[0]
        if idx.size == 0:
            continue
        z = W1[idx] @ x[t]
        if b1 is not None:
            z = z + _as64(b1)[idx]
        delta = gelu(z, act) - a[idx] * z - c[idx]
        y[t] += W2[:, idx] @ delta
    return y


def tardis_ffn(x, W1, W2, a, c, lo, hi, codes_u32, scale, zero, group,
               b1=None, b2=None, act=ACT_GELU_TANH, bits=2, folded=None):
    """The whole path in the paper's order: fold (offline), predictor score,
    flag, speculative folded product, result fixing.  Returns (y, F, zhat).
    `folded` may carry a previously computed (W_f, b_f)."""
    if folded is None:
        folded = fold(W1, W2, a, c, b1, b2)
    Wf, bf = folded
    zhat = predictor_score(x, codes_u32, scale, zero, group, b1, bits)
    F = flags_from_score(zhat, lo, hi)
    y0 = speculate(Wf, bf, x)
    y = fix(y0, x, F, W1, W2, a, c, b1, act)
    return y, F, zhat


# --------------------------------------------------------------------------
# definitions the path is checked against
# --------------------------------------------------------------------------
def dense_ffn(x, W1, W2, b1=None, b2=None, act=ACT_GELU_TANH):
    """The original FFN, W2 GELU(W1 x + b1) + b2 (Section 3.1)."""
    x = _as64(x)
    z = x @ _as64(W1).T
    if b1 is not None:
        z = z + _as64(b1)[None, :]
    y = gelu(z, act) @ _as64(W2).T
    if b2 is not None:
        y = y + _as64(b2)[None, :]
    return y


def direct_partially_linear(x, F, W1, W2, a, c, b1=None, b2=None, act=ACT_GELU_TANH):
    """The partially linear FFN with no folding at all: neuron j contributes
    W2[:,j] * phi_j(z_j), phi_j = GELU when flagged, a_j z + c_j otherwise
    (Section 5.1.1 with the predictor's flags standing in for the range test).
    Costs 4 d h per token and needs no d x d matrix, so it also serves as the
    per-token check at full problem sizes."""
    x = _as64(x)
    z = x @ _as64(W1).T
    if b1 is not None:
        z = z + _as64(b1)[None, :]
    F = np.asarray(F, dtype=bool)
    phi = np.where(F, gelu(z, act), _as64(a)[None, :] * z + _as64(c)[None, :])
    y = phi @ _as64(W2).T
    if b2 is not None:
        y = y + _as64(b2)[None, :]
    return y


def rel_error(y, y_ref):
    """Per-element error |y - y_ref| / max(|y_ref|, rms(y_ref[t,:])); the maximum
    of this over all elements is the "max relative error" of the parity gate."""
    y = _as64(y)
    y_ref = _as64(y_ref)
    rms = np.sqrt(np.mean(y_ref * y_ref, axis=-1, keepdims=True))
    den = np.maximum(np.abs(y_ref), rms)
    den = np.where(den > 0, den, 1.0)
    return np.abs(y - y_ref) / den


# --------------------------------------------------------------------------
# offline: per-neuron range and linear fit from calibration pre-activations
# --------------------------------------------------------------------------
def quantile_ranges(z, q_lo, q_hi):
    """Range of every neuron: the interval that holds a chosen share of the
    activation inputs profiled for it (Section 4.1, Insight 2, describes the procedure; Section 5.1, step 2), taken here as
    the central portion between the q_lo and q_hi quantiles of the neuron's
    calibration pre-activations.  z[h, N]: row j = the N samples of
    neuron j.  The quantile at level p is the linear interpolation between the
    order statistics around position p (N - 1).  (The greedy search of
    Algorithm 1 is a different way to pick the same kind of range; the
    configurations of this repository use quantiles.)  Returns (lo, hi) as
    float32 arrays: the range is stored in single precision."""
    z = _as64(z)
    h, N = z.shape
    zs = np.sort(z, axis=1)
    out = []
    for p in (q_lo, q_hi):
        pos = float(p) * (N - 1)
        i0 = int(math.floor(pos))
        i1 = min(i0 + 1, N - 1)
        w = pos - i0
        out.append((zs[:, i0] * (1.0 - w) + zs[:, i1] * w).astype(np.float32))
    return out[0], out[1]


def gelu_derivative(z, act=ACT_GELU_TANH):
    """d/dz sigma(z), analytic, float64 (ReLU: 1 for z > 0, else 0)."""
    z = np.asarray(z, dtype=_F64)
    if act == ACT_GELU_TANH:
        k = math.sqrt(2.0 / math.pi)
        u = k * (z + 0.044715 * z ** 3)
        t = np.tanh(u)
        return 0.5 * (1.0 + t) + 0.5 * z * (1.0 - t * t) * k * (1.0 + 3.0 * 0.044715 * z * z)
    if act == ACT_GELU_ERF:
        from scipy.special import erf
        return 0.5 * (1.0 + erf(z / math.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)
    if act == ACT_RELU:
        return np.where(z > 0.0, 1.0, 0.0)
    raise ValueError("unknown activation %r" % (act,))


def least_squares_fit(z, lo, hi, act=ACT_GELU_TANH):
    """The linear function y = a z + c of every neuron: the least-squares
    regression (Section 5.1, step 3; Section 4.1, Insight 2) of the activation
    sigma(z) on z over the calibration samples inside the neuron's range
    lo <= z < hi:
        a = cov(z, sigma(z)) / var(z),   c = mean(sigma(z)) - a mean(z).
    A neuron with fewer than two samples in range, or whose in-range samples
    have variance below 1e-30, takes the tangent of sigma at the range midpoint.
    z[h, N] float (samples as stored, i.e. float32 values), lo/hi[h] float32.
    Returns (a, c) as float32 arrays."""
    z = _as64(z)
    lo64, hi64 = _as64(lo), _as64(hi)
    h, N = z.shape
    a = np.empty(h, dtype=np.float32)
    c = np.empty(h, dtype=np.float32)
    for j in range(h):
        zj = z[j]
        inside = (zj >= lo64[j]) & (zj < hi64[j])
        zz = zj[inside]
        ok = False
        if zz.size >= 2:
            sg = gelu(zz, act)
            mz, ms = zz.mean(), sg.mean()
            var = ((zz - mz) ** 2).mean()
            if var > 1e-30:
                cov = ((zz - mz) * (sg - ms)).mean()
                aj = cov / var
                cj = ms - aj * mz
                ok = True
        if not ok:
            mid = 0.5 * (lo64[j] + hi64[j])
            aj = float(gelu_derivative(mid, act))
            cj = float(gelu(mid, act)) - aj * mid
        a[j] = np.float32(aj)
        c[j] = np.float32(cj)
    return a, c


# --------------------------------------------------------------------------
# offline: the greedy range search of Algorithm 1 (Section 5.1.1, "Range Searching")
# --------------------------------------------------------------------------
def kde_centroid(samples):
    """Centroid of a neuron's activation inputs by kernel density estimation (Algorithm 1, find_centroid): the
    sample at which a Gaussian kernel density estimate of the samples is highest.  The paper names KDE but not the
    kernel or its width; the reading taken here: Gaussian kernel, Silverman's rule-of-thumb width
    bw = 1.06 * std * N^(-1/5) (std with N - 1 in the denominator), density evaluated at the samples themselves,
    ties to the smallest sample.  With bw = 0 (all samples equal) or a single sample that value is the centroid."""
    z = np.sort(_as64(samples).ravel())
    n = z.size
    if n == 1:
        return float(z[0])
    bw = 1.06 * np.std(z, ddof=1) * n ** (-0.2)
    if not bw > 0.0:
        return float(z[0])
    dens = np.empty(n)
    for i in range(n):
        u = (z - z[i]) / bw
        dens[i] = np.exp(-0.5 * u * u).sum()
    return float(z[int(np.argmax(dens))])


def approx_error(samples, lo, hi, act=ACT_GELU_TANH):
    """Error of approximating the activation by its least-squares line over the samples inside [lo, hi)
    (Algorithm 1, approx_error; Section 4.1 measures it as a mean squared error): the mean of the squared residuals
    of that line.  Fewer than two samples in range, or samples that do not vary: 0 (a line fits them exactly)."""
    z = _as64(samples).ravel()
    zin = z[(z >= lo) & (z < hi)]
    if zin.size < 2:
        return 0.0
    g = gelu(zin, act)
    mz, mg = zin.mean(), g.mean()
    dz, dg = zin - mz, g - mg
    var = (dz * dz).mean()
    if not var > 1e-30:
        return 0.0
    a = (dz * dg).mean() / var
    r = dg - a * dz
    return float((r * r).mean())


def greedy_range_search(samples, t, step, act=ACT_GELU_TANH, return_trace=False):
    """Range of one neuron by Algorithm 1: start from the empty range at the KDE centroid; while the share of the
    samples inside the range is below the threshold t, form the range extended by `step` to the left and the range
    extended by `step` to the right, measure the approximation error of each, and keep the one with the smaller
    error (the right one on a tie).  Ranges are half-open, [lo, hi).

    The printed listing builds the left candidate as (R.left - s, R.left) and the right one as (R.left, R.right + s);
    taken literally the left candidate would drop everything found so far, so the reading is (R.left - s, R.right)
    and (R.left, R.right + s): each candidate is the current range grown on one side.  Bounds are kept as
    centroid - k_left * step and centroid + k_right * step with integer step counts, so that no rounding accumulates.
    The loop also stops once the range holds every sample, and a side that has passed the outermost sample is not
    grown any further (the other side is taken without comparing errors).

    Returns (lo, hi) as Python floats (and, with return_trace, the list of 'L'/'R' choices and the smallest
    relative margin |err_left - err_right| / max(err_left, err_right) seen, a measure of how close a decision was)."""
    z = np.sort(_as64(samples).ravel())
    n = z.size
    c = kde_centroid(z)
    kl = kr = 0
    trace, margin = [], float("inf")
    while True:
        lo, hi = c - kl * step, c + kr * step
        inside = int(((z >= lo) & (z < hi)).sum())
        if inside >= t * n or inside == n:
            break
        lo_l, hi_r = c - (kl + 1) * step, c + (kr + 1) * step
        # a side that already reaches past the outermost sample has nothing left to add: the other side is taken
        # (as printed, the loop would grow such a side for ever whenever its error stays the smaller one)
        if hi > z[-1]:
            go_left = True
        elif lo <= z[0]:
            go_left = False
        else:
            e_l = approx_error(z, lo_l, hi, act)
            e_r = approx_error(z, lo, hi_r, act)
            m = max(e_l, e_r)
            if m > 0.0:
                margin = min(margin, abs(e_l - e_r) / m)
            go_left = e_l < e_r
        if go_left:
            kl += 1
            trace.append("L")
        else:
            kr += 1
            trace.append("R")
    lo, hi = c - kl * step, c + kr * step
    if return_trace:
        return lo, hi, trace, margin
    return lo, hi


def neuron_thresholds(err, t_layer, t_min, t_max):
    """Neuron-level thresholds of Section 5.1.1: minimise sum_n E_n t_n subject to sum_n t_n = t_layer * h.  As printed
    the problem has no bounds on t_n and is unbounded; the reading taken here adds the box t_min <= t_n <= t_max
    (t_min <= t_layer <= t_max).  A linear objective over a box with one equality constraint is minimised greedily:
    every neuron starts at t_min, and the remaining budget goes, up to t_max each, to the neurons in order of
    increasing error (ties to the smaller index); at most one neuron ends strictly between the bounds."""
    err = _as64(err).ravel()
    h = err.size
    if not (t_min <= t_layer <= t_max):
        raise ValueError("need t_min <= t_layer <= t_max")
    t = np.full(h, float(t_min))
    budget = (t_layer - t_min) * h
    for j in np.argsort(err, kind="stable"):
        give = min(t_max - t_min, budget)
        t[j] += give
        budget -= give
        if budget <= 0.0:
            break
    return t


# ---- a chain of layers on one residual stream (no counterpart in the paper: the stack call of the library) ----
def layer_norm(v, gamma=None, beta=None, eps=1e-5):
    """Layer normalisation of every row of v[n, d] by its definition: subtract the row's mean, divide by the square
    root of the row's variance (divisor d) plus eps, multiply by gamma[d] and add beta[d] (1 and 0 when absent)."""
    v = _as64(v)
    d = v.shape[-1]
    out = np.empty_like(v)
    for t in range(v.shape[0]):
        mean = v[t].sum() / d
        var = ((v[t] - mean) ** 2).sum() / d
        out[t] = (v[t] - mean) / math.sqrt(var + eps)
    if gamma is not None:
        out = out * _as64(gamma)[None, :]
    if beta is not None:
        out = out + _as64(beta)[None, :]
    return out


def stack_forward(x, ffns, gammas=None, betas=None, eps=1e-5, normalise=True, residual=True):
    """s_0 = x; u_l = layer_norm(s_l) or s_l; f_l = ffns[l](u_l); s_{l+1} = s_l + f_l or f_l.  Returns s_L and the
    lists of u_l and f_l.  `ffns` are callables [n, d] -> [n, d] (a layer's partially linear forward)."""
    s = _as64(x)
    us, fs = [], []
    for l, ffn in enumerate(ffns):
        u = layer_norm(s, None if gammas is None else gammas[l], None if betas is None else betas[l], eps) if normalise else s
        f = _as64(ffn(u))
        us.append(u)
        fs.append(f)
        s = s + f if residual else f
    return s, us, fs


# ---- building the predictor: quantisation of W1 with error compensation (Section 6: "GPTQ with 2-bit precision") ----
def round_to_storage(v, dtype):
    """The value a float64 number takes when stored as `dtype` ("f32" or "bf16"): rounded to nearest-even to float32, and
    for bf16 rounded once more, to nearest-even, to the upper 16 bits of the float32 word (finite values)."""
    f = np.asarray(v, dtype=np.float64).astype(np.float32)
    if dtype == "f32":
        return f.astype(np.float64)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def group_grid(wg, bits, dtype):
    """Asymmetric uniform grid of one group of weights wg[..., G]: the range [min, max] widened to contain 0, the scale
    (max - min) / (2^bits - 1) rounded to its storage type before anything else uses it (1 if that is 0), the zero-point
    round(-min / scale) clamped to the code range.  Returns (scale, zero)."""
    levels = (1 << bits) - 1
    wmin = np.minimum(wg.min(axis=-1), 0.0)
    wmax = np.maximum(wg.max(axis=-1), 0.0)
    scale = round_to_storage((wmax - wmin) / levels, dtype)
    scale = np.where(scale > 0.0, scale, 1.0)
    zero = np.clip(np.rint(-wmin / scale), 0, levels)
    return scale, zero


def gptq_quantise(W1, U, group, bits=2, dtype="bf16"):
    """Quantisation of W1[h, d] with the error of every rounded channel spread over the channels not yet rounded (the
    GPTQ procedure the paper uses for its predictor).  U[d, d] is the upper Cholesky factor of the inverse Hessian of the
    layer's inputs (U^T U = H^-1); U = None stands for the identity, which leaves plain rounding to nearest.

    Channels go in ascending order.  When channel k opens a group, the group's grid comes from the weights as they are at
    that moment (earlier errors already spread into them).  Then q_k = clip(rint(w_k / s + z)), the error
    e_k = (w_k - s (q_k - z)) / U[k, k], and every later channel j > k takes w_j <- w_j - e_k U[k, j].
    Returns (q uint8 [h, d], scale [h, d/G], zero [h, d/G], E [h, d] the errors e_k)."""
    W = _as64(W1).copy()
    h, d = W.shape
    levels = (1 << bits) - 1
    q = np.empty((h, d), dtype=np.uint8)
    E = np.empty((h, d))
    scale = np.empty((h, d // group))
    zero = np.empty((h, d // group))
    for k in range(d):
        g = k // group
        if k % group == 0:
            scale[:, g], zero[:, g] = group_grid(W[:, k:k + group], bits, dtype)
        qk = np.clip(np.rint(W[:, k] / scale[:, g] + zero[:, g]), 0, levels)
        q[:, k] = qk.astype(np.uint8)
        ukk = 1.0 if U is None else U[k, k]
        E[:, k] = (W[:, k] - scale[:, g] * (qk - zero[:, g])) / ukk
        if U is not None and k + 1 < d:
            W[:, k + 1:] -= E[:, k][:, None] * U[k, k + 1:][None, :]
    return q, scale, zero, E


def pack_codes(q, bits=2):
    """The inverse of unpack_codes: [h, d] codes into [h, d bits / 32] 32-bit words, one bit stream per row, channel order
    ascending, lowest bits first."""
    q = np.asarray(q, dtype=np.uint32)
    h, d = q.shape
    single = (q[:, :, None] >> np.arange(bits, dtype=np.uint32)[None, None, :]) & np.uint32(1)     # [h, d, bits]
    stream = single.reshape(h, d * bits // 32, 32).astype(np.uint64)
    words = (stream << np.arange(32, dtype=np.uint64)[None, None, :]).sum(axis=2)
    return words.astype(np.uint32)
