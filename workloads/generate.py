"""Seeded synthetic inputs for the partially linear FFN forward.

This module only manufactures INPUT DATA for the path: weights, tokens, and the
frozen per-neuron state (linear range, slope/intercept, quantised-W1 predictor)
that the paper's offline calibration would hand to the fold.  It contains none
of the path's own arithmetic (fold, predictor score, flagging, folded product,
result fixing); both the CPU oracle and the CUDA library receive the arrays made
here, unchanged.

The real workloads of the paper (Falcon-7B weights, C4 calibration text) are not
available; these generators take their shapes (d_ff = 4 d_model, Falcon-7B's
4544/18176) and their structure (heavy-tailed, skewed activation inputs;
outlier channels) instead:

* weights  W ~ N(0, 0.02^2), biases ~ N(0, 0.01^2), rounded once to the dtype
* tokens   iid Student-t (nu = 4) per channel, then LayerNorm (no affine,
           eps 1e-5); the "mixture" kind flips a fair coin per token between
           Gaussian and Student-t and scales a fixed 1 % of channels by 20
           after the LayerNorm (activation-outlier channels)
* ranges   per-neuron [q_lo, q_hi] quantiles of the calibration pre-activations
           (linear interpolation between order statistics, position p (N-1))
* fit      ordinary least squares of GELU on the calibration samples that lie
           in the range (Section 5.1: "linear functions are obtained using
           least squares regression")
* predictor  W1 quantised to 2 bits on an asymmetric uniform grid per (neuron,
           group of G consecutive channels): round-to-nearest, or the GPTQ
           column-by-column error-compensated rounding (Section 6: "GPTQ with
           2-bit precision").

torch is used as the array library so the same code runs on the CPU (tests) or
on a GPU (full-size benchmark set-up).  Random streams differ between devices;
within one run both sides always see the same arrays.
"""
from __future__ import annotations

import dataclasses
import math
import zlib
from typing import Optional

import torch

ACT_GELU_TANH = 0
ACT_GELU_ERF = 1
ACT_RELU = 2


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    d_model: int
    d_ff: int
    dtype: str = "bf16"            # "f32" | "bf16": storage type of W1, W2, x, y, predictor scale
    act: int = ACT_GELU_TANH
    group: int = 64                # predictor group size G
    bits: int = 2
    bias: bool = True
    tokens: str = "student_t"      # "student_t" | "mixture"
    n_calib: int = 4096
    q_lo: float = 0.05
    q_hi: float = 0.95
    target_flag_frac: Optional[float] = None   # if set, (q_lo, 1-q_lo) is bisected to reach it
    quantiser: str = "rtn"         # "rtn" | "gptq"


# The five configurations the benchmark definition names.
CONFIGS = {
    "tiny_f32": LayerConfig("tiny_f32", 256, 1024, dtype="f32", n_calib=4096, q_lo=0.05, q_hi=0.95),
    "decode_7b": LayerConfig("decode_7b", 4096, 16384, n_calib=2048, target_flag_frac=0.10, group=128),
    "falcon_7b": LayerConfig("falcon_7b", 4544, 18176, bias=False, tokens="mixture", n_calib=2048),
    "prefill_7b": LayerConfig("prefill_7b", 4096, 16384, n_calib=2048, target_flag_frac=0.10, group=128),
    "large_8k": LayerConfig("large_8k", 8192, 32768, n_calib=2048, target_flag_frac=0.10, group=128),
}
# quantile pairs of the Falcon-shaped sweep (flagged fraction about 5/10/20/30 %)
FALCON_QUANTILES = [(0.025, 0.975), (0.05, 0.95), (0.10, 0.90), (0.15, 0.85)]


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def seed_for(*parts) -> int:
    """Deterministic 31-bit seed from a tuple of names/numbers."""
    return zlib.crc32("/".join(str(p) for p in parts).encode()) & 0x7FFFFFFF


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


# --------------------------------------------------------------------------
# weights and tokens
# --------------------------------------------------------------------------
def make_weights(cfg: LayerConfig, seed: int, device="cpu"):
    """W1[h,d], W2[d,h] in cfg.dtype; b1[h], b2[d] float32 or None."""
    g = _gen(seed_for(cfg.name, seed, "weights"), device)
    dt = torch_dtype(cfg.dtype)
    h, d = cfg.d_ff, cfg.d_model
    W1 = (torch.randn(h, d, generator=g, device=device, dtype=torch.float32) * 0.02).to(dt)
    W2 = (torch.randn(d, h, generator=g, device=device, dtype=torch.float32) * 0.02).to(dt)
    if cfg.bias:
        b1 = torch.randn(h, generator=g, device=device, dtype=torch.float32) * 0.01
        b2 = torch.randn(d, generator=g, device=device, dtype=torch.float32) * 0.01
    else:
        b1 = b2 = None
    return W1, W2, b1, b2


def _student_t(n, d, nu, g, device):
    z = torch.randn(n, d, generator=g, device=device, dtype=torch.float32)
    v = torch.zeros(n, d, device=device, dtype=torch.float32)
    for _ in range(nu):                       # chi-square(nu) as a sum of squares
        v += torch.randn(n, d, generator=g, device=device, dtype=torch.float32) ** 2
    return z / torch.sqrt(v / nu)


def _layernorm(x, eps=1e-5):
    mu = x.mean(dim=-1, keepdim=True)
    var = x.var(dim=-1, unbiased=False, keepdim=True)
    return (x - mu) / torch.sqrt(var + eps)


def outlier_channels(cfg: LayerConfig, device="cpu"):
    """The fixed 1 % of channels the "mixture" token kind scales by 20."""
    g = _gen(seed_for(cfg.name, "outlier_channels"), "cpu")
    k = max(1, cfg.d_model // 100)
    return torch.randperm(cfg.d_model, generator=g)[:k].to(device)


def make_tokens(cfg: LayerConfig, n: int, seed: int, device="cpu", tag="tokens"):
    """x[n, d] in cfg.dtype."""
    g = _gen(seed_for(cfg.name, seed, tag), device)
    d = cfg.d_model
    out = []
    for s in range(0, n, 4096):               # chunked: bounded temporary memory
        m = min(4096, n - s)
        if cfg.tokens == "student_t":
            x = _layernorm(_student_t(m, d, 4, g, device))
        elif cfg.tokens == "mixture":
            coin = torch.rand(m, 1, generator=g, device=device) < 0.5
            xg = torch.randn(m, d, generator=g, device=device, dtype=torch.float32)
            xt = _student_t(m, d, 4, g, device)
            x = _layernorm(torch.where(coin, xg, xt))
            x[:, outlier_channels(cfg, device)] *= 20.0
        else:
            raise ValueError(cfg.tokens)
        out.append(x.to(torch_dtype(cfg.dtype)))
    return torch.cat(out, dim=0) if out else torch.empty(0, d, dtype=torch_dtype(cfg.dtype), device=device)


# --------------------------------------------------------------------------
# calibration-as-setup: ranges and linear fits
# --------------------------------------------------------------------------
def gelu_f64(z: torch.Tensor, act: int) -> torch.Tensor:
    z = z.double()
    if act == ACT_GELU_TANH:
        return torch.nn.functional.gelu(z, approximate="tanh")
    if act == ACT_RELU:
        return torch.relu(z)
    return torch.nn.functional.gelu(z)


def preactivations(W1, b1, xcal):
    """z[N, h] = xcal W1^T + b1 in float32 (calibration statistics only)."""
    z = xcal.float() @ W1.float().t()
    if b1 is not None:
        z = z + b1[None, :]
    return z


def quantile_ranges(z_sorted: torch.Tensor, q_lo: float, q_hi: float):
    """Per-neuron (lo, hi) = the q_lo and q_hi quantiles of the column, linear
    interpolation between order statistics at position p (N-1); float32 out."""
    N = z_sorted.shape[0]

    def at(p):
        pos = p * (N - 1)
        i0 = int(math.floor(pos))
        i1 = min(i0 + 1, N - 1)
        w = pos - i0
        return (z_sorted[i0].double() * (1.0 - w) + z_sorted[i1].double() * w).float()

    return at(q_lo), at(q_hi)


def least_squares_fit(z: torch.Tensor, lo: torch.Tensor, hi: torch.Tensor, act: int, chunk: int = 2048):
    """Ordinary least squares of GELU(z) on z over the samples with lo <= z < hi,
    per neuron (column): a = cov(z, s)/var(z), c = mean(s) - a mean(z).
    Degenerate columns (< 2 samples or var < 1e-30) take the tangent at the
    range midpoint.  float64 arithmetic, float32 out."""
    N, h = z.shape
    a = torch.empty(h, dtype=torch.float32, device=z.device)
    c = torch.empty(h, dtype=torch.float32, device=z.device)
    for s in range(0, h, chunk):
        e = min(h, s + chunk)
        zz = z[:, s:e].double()
        l = lo[s:e].double()[None, :]
        u = hi[s:e].double()[None, :]
        m = ((zz >= l) & (zz < u)).double()
        sg = gelu_f64(zz, act)
        cnt = m.sum(0)
        safe = cnt.clamp(min=1.0)
        mz = (m * zz).sum(0) / safe
        ms = (m * sg).sum(0) / safe
        dz = (zz - mz[None, :]) * m
        var = (dz * dz).sum(0) / safe
        cov = (dz * (sg - ms[None, :])).sum(0) / safe
        ok = (cnt >= 2) & (var > 1e-30)
        mid = (0.5 * (l + u)).squeeze(0)
        eps = 1e-6
        slope_mid = (gelu_f64(mid + eps, act) - gelu_f64(mid - eps, act)) / (2 * eps)
        a64 = torch.where(ok, cov / var.clamp(min=1e-300), slope_mid)
        c64 = torch.where(ok, ms - a64 * mz, gelu_f64(mid, act) - slope_mid * mid)
        a[s:e] = a64.float()
        c[s:e] = c64.float()
    return a, c


# --------------------------------------------------------------------------
# predictor: 2-bit quantised copy of W1
# --------------------------------------------------------------------------
def _grid(wg: torch.Tensor, levels: int, scale_dtype: torch.dtype):
    """Asymmetric uniform grid of one group: range forced to contain 0; the scale
    is rounded to its storage dtype BEFORE codes are chosen."""
    wmin = wg.amin(dim=-1).clamp(max=0.0)
    wmax = wg.amax(dim=-1).clamp(min=0.0)
    scale = ((wmax - wmin) / (levels - 1)).to(scale_dtype).float()
    scale = torch.where(scale > 0, scale, torch.ones_like(scale))
    zero = torch.round(-wmin / scale).clamp(0, levels - 1)
    return scale, zero


def quantise_rtn(W1: torch.Tensor, group: int, bits: int, scale_dtype: torch.dtype):
    """Round-to-nearest on the per-(neuron, group) grid.  Returns
    q uint8 [h,d], scale [h,d/G] (scale_dtype), zero uint8 [h,d/G]."""
    h, d = W1.shape
    levels = 1 << bits
    w = W1.float().reshape(h, d // group, group)
    scale, zero = _grid(w, levels, scale_dtype)
    q = torch.round(w / scale[..., None] + zero[..., None]).clamp(0, levels - 1)
    return q.reshape(h, d).to(torch.uint8), scale.to(scale_dtype), zero.to(torch.uint8)


def quantise_gptq(W1: torch.Tensor, xcal: torch.Tensor, group: int, bits: int,
                  scale_dtype: torch.dtype, damp: float = 0.01, block: int = 128):
    """GPTQ-style quantisation of W1 (rows = neurons, columns = input channels):
    channels are rounded one at a time in natural order and the rounding error of
    each is spread over the not-yet-rounded channels with the upper Cholesky
    factor of the inverse Hessian H = (2/N) X^T X + damp * mean(diag H) I.  The
    grid of a group is fixed from the error-compensated weights when the group
    starts.  Same outputs as quantise_rtn."""
    h, d = W1.shape
    levels = 1 << bits
    dev = W1.device
    if block % group:
        raise ValueError("block must be a multiple of group")
    X = xcal.double()
    H = (2.0 / X.shape[0]) * (X.t() @ X)
    H += damp * torch.mean(torch.diagonal(H)) * torch.eye(d, dtype=H.dtype, device=dev)
    Hinv = torch.cholesky_inverse(torch.linalg.cholesky(H))
    U = torch.linalg.cholesky(Hinv, upper=True).float()      # upper factor of H^-1
    W = W1.float().clone()
    Q = torch.empty(h, d, dtype=torch.uint8, device=dev)
    scale = torch.empty(h, d // group, dtype=torch.float32, device=dev)
    zero = torch.empty(h, d // group, dtype=torch.float32, device=dev)
    for b0 in range(0, d, block):
        b1_ = min(d, b0 + block)
        Wb = W[:, b0:b1_].clone()
        Eb = torch.zeros_like(Wb)
        Ub = U[b0:b1_, b0:b1_]
        for i in range(b1_ - b0):
            k = b0 + i
            if k % group == 0:
                s_, z_ = _grid(Wb[:, i:i + group], levels, scale_dtype)
                scale[:, k // group] = s_
                zero[:, k // group] = z_
            s_ = scale[:, k // group]
            z_ = zero[:, k // group]
            w = Wb[:, i]
            q = torch.round(w / s_ + z_).clamp(0, levels - 1)
            Q[:, k] = q.to(torch.uint8)
            err = (w - s_ * (q - z_)) / Ub[i, i]
            Wb[:, i:] -= err[:, None] * Ub[i, i:][None, :]
            Eb[:, i] = err
        W[:, b1_:] -= Eb @ U[b0:b1_, b1_:]
    return Q, scale.to(scale_dtype), zero.to(torch.uint8)


def pack_codes(q: torch.Tensor, bits: int = 2) -> torch.Tensor:
    """[h,d] codes -> [h, d*bits/32] 32-bit words: one bit stream per row, channel order
    ascending, lowest bits first (a 3-bit code may cross into the next word).  Returned as
    int32 holding the uint32 bit pattern."""
    h, d = q.shape
    q64 = q.to(torch.int64)
    single = (q64[:, :, None] >> torch.arange(bits, device=q.device, dtype=torch.int64)[None, None, :]) & 1
    stream = single.reshape(h, d * bits // 32, 32)
    word = (stream << torch.arange(32, device=q.device, dtype=torch.int64)[None, None, :]).sum(-1)
    word = torch.where(word >= 2 ** 31, word - 2 ** 32, word)
    return word.to(torch.int32)


def dequantise(q, scale, zero, group):
    h, d = q.shape
    qf = q.float().reshape(h, d // group, group)
    return ((qf - zero.float()[..., None]) * scale.float()[..., None]).reshape(h, d)


# --------------------------------------------------------------------------
# one layer's full frozen state
# --------------------------------------------------------------------------
@dataclasses.dataclass
class Layer:
    cfg: LayerConfig
    W1: torch.Tensor
    W2: torch.Tensor
    b1: Optional[torch.Tensor]
    b2: Optional[torch.Tensor]
    lo: torch.Tensor
    hi: torch.Tensor
    a: torch.Tensor
    c: torch.Tensor
    codes: torch.Tensor     # int32 [h, d*bits/32] (uint32 bit pattern)
    scale: torch.Tensor     # cfg.dtype [h, d/G]
    zero: torch.Tensor      # uint8 [h, d/G]
    q_lo: float
    q_hi: float

    def numpy64(self):
        """The same values widened exactly to float64 numpy arrays (oracle side)."""
        import numpy as np
        f = lambda t: None if t is None else t.detach().double().cpu().numpy()
        return dict(W1=f(self.W1), W2=f(self.W2), b1=f(self.b1), b2=f(self.b2), lo=f(self.lo),
                    hi=f(self.hi), a=f(self.a), c=f(self.c),
                    codes=self.codes.cpu().numpy().view(np.uint32), scale=f(self.scale),
                    zero=self.zero.cpu().numpy(), group=self.cfg.group, bits=self.cfg.bits,
                    act=self.cfg.act)


def make_layer(cfg: LayerConfig, seed: int = 0, device="cpu", eval_tokens: Optional[torch.Tensor] = None) -> Layer:
    """Weights + calibration-as-setup.  With cfg.target_flag_frac set, the
    symmetric quantile pair (q, 1-q) is bisected until the predictor-flagged
    fraction on `eval_tokens` (default: 256 fresh tokens) is about the target."""
    W1, W2, b1, b2 = make_weights(cfg, seed, device)
    xcal = make_tokens(cfg, cfg.n_calib, seed, device, tag="calibration")
    dt = torch_dtype(cfg.dtype)
    if cfg.quantiser == "gptq":
        q, scale, zero = quantise_gptq(W1, xcal, cfg.group, cfg.bits, dt)
    else:
        q, scale, zero = quantise_rtn(W1, cfg.group, cfg.bits, dt)
    z = preactivations(W1, b1, xcal)
    zs, _ = torch.sort(z, dim=0)
    q_lo, q_hi = cfg.q_lo, cfg.q_hi
    if cfg.target_flag_frac is not None:
        if eval_tokens is None:
            eval_tokens = make_tokens(cfg, 256, seed, device, tag="tune")
        zhat = preactivations(dequantise(q, scale, zero, cfg.group), b1, eval_tokens)
        lo_q, hi_q = 1e-4, 0.4999
        for _ in range(20):
            mid = 0.5 * (lo_q + hi_q)
            lo, hi = quantile_ranges(zs, mid, 1.0 - mid)
            frac = (~((zhat >= lo[None, :]) & (zhat < hi[None, :]))).float().mean().item()
            if frac > cfg.target_flag_frac:
                hi_q = mid          # too many flagged -> widen the range -> smaller q
            else:
                lo_q = mid
        q_lo = 0.5 * (lo_q + hi_q)
        q_hi = 1.0 - q_lo
    lo, hi = quantile_ranges(zs, q_lo, q_hi)
    del zs
    a, c = least_squares_fit(z, lo, hi, cfg.act)
    return Layer(cfg, W1, W2, b1, b2, lo, hi, a, c, pack_codes(q, cfg.bits), scale, zero, q_lo, q_hi)
