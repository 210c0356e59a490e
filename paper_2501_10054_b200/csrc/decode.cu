// Fused batch-1 decode kernel of the online path (Section 5.4) for bf16 layers on sm_100a.
//
// One launch does the whole token: predictor score (Section 5.3), flagging and compaction,
// speculative folded product, result fixing.  The grid is two 512-thread CTAs per SM; all
// weight traffic is coalesced 128-bit read-only loads kept several deep per thread (which is
// what reaches the HBM rate on this part: the bytes in flight per SM, not the copy engine).
//
//   * A CTA owns a few 16-neuron tiles.  Its predictor codes are evaluated on the integer
//     tensor cores: codes are masked straight out of the packed words (no shifts: the field
//     position is a power-of-4 weight that the pre-scaling of x undoes) and multiplied with a
//     4-limb signed base-256 fixed-point copy of x (mma.m16n8k32.u8.s8, s32 accumulators,
//     exact); group sums are scaled and accumulated in fp64, so the score equals the
//     mathematical one up to the (tracked) truncation of tiny x elements; a score that close to
//     a range end is re-evaluated exactly from the original codes.  Warps split the tiles and
//     the channel range; partial scores meet in shared memory.
//   * Flags are compacted by ballot + prefix sum into the CTA's ascending list.
//   * Every thread owns 8 output columns (per slot).  For the CTA's flagged neurons it reads
//     its slice of the W1 row (partial dot products meet through warp shuffles and shared
//     memory to give the exact z_j), then its slice of the W2T row, scaled by
//     delta_j = GELU(z_j) - a_j z_j - c_j, into its column accumulators.
//   * The folded matrix C = W_f^T is handed out dynamically: each warp (owning a fixed column
//     range in every CTA) draws row chunks from a global ticket of its column range, so CTAs
//     with few flagged neurons take more of the folded product and all finish together.
//   * Warps add their columns into an fp32 accumulator with vector reductions; the last warp
//     to arrive on a column range adds b_f, rounds to bf16, and re-zeroes the scratch.
#include <stdio.h>

#include <vector>

#include "common.cuh"

namespace tardis {
namespace dec {

constexpr int NW = 16;            // warps per CTA
constexpr int NTH = NW * 32;      // threads per CTA
constexpr int CTAS_PER_SM = 2;
constexpr int KC = 256;           // channels per predictor block
constexpr int MAXROWS = 256;      // predictor rows (neurons) per CTA: at most 16 tiles
constexpr int MAXRC = 64;         // exact re-checks per CTA before the list overflows (rest handled in place)
constexpr int LOADS = 4;          // 128-bit loads per thread and batch (rows x slots)
// control words (unsigned int) in global scratch; all zero between calls
constexpr int CTL_TICKET = 0;     // [NW] stride 32: next folded-matrix row chunk of a warp's column range
constexpr int CTL_DONE = 512;     // [NW] stride 32: warps that have added their columns
constexpr int CTL_NFL = 1024;     // flagged neurons of the token so far
constexpr int CTL_ARRIVED = 1056; // CTAs that have reported their flagged count
constexpr int CTL_WORDS = 1088;

struct Params {
  const uint8_t* pblocks;  // [tile][kchunk] predictor blocks
  int pbs, nkc, G;
  const __nv_bfloat16 *W1, *W2T, *C;
  const float *bf, *lo, *hi, *a, *c, *b1;
  const uint32_t* codes; const __nv_bfloat16* scale; const uint8_t* zero;   // originals (exact re-check)
  const float* smax;       // largest group scale of the layer
  const int2* plan;        // per CTA: first tile, tile count
  const __nv_bfloat16* x; __nv_bfloat16* y;
  float* yacc; unsigned int* ctl; unsigned long long* counters;
  uint32_t* dbg_bitmap; double* dbg_scores;
  int d, dpad, h, ngroups, act;
  int ts_log2;             // tile slots per CTA = 1 << ts_log2; warps per tile = NW >> ts_log2
  int nvec, cw;            // 8-column vectors in a row; vectors per warp
  int ntk;                 // row chunks of the folded matrix (LOADS / VPT rows each)
};

struct Scratch {           // handle-owned device memory of the fused path
  uint8_t* pblocks; int2* plan; float* smax; float* yacc; unsigned int* ctl;
  Params base; size_t smem_bytes; size_t bytes; int grid; int vpt;
};

// ---- small wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ldg_stream(const void* p) {   // read-only, no L1 allocation
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void fma8(float (&acc)[8], float s, const uint4& w) {
  acc[0] += s * bf_lo(w.x); acc[1] += s * bf_hi(w.x);
  acc[2] += s * bf_lo(w.y); acc[3] += s * bf_hi(w.y);
  acc[4] += s * bf_lo(w.z); acc[5] += s * bf_hi(w.z);
  acc[6] += s * bf_lo(w.w); acc[7] += s * bf_hi(w.w);
}
__device__ __forceinline__ float dot8(const uint4& w, const float (&xv)[8]) {
  return bf_lo(w.x) * xv[0] + bf_hi(w.x) * xv[1] + bf_lo(w.y) * xv[2] + bf_hi(w.y) * xv[3] +
         bf_lo(w.z) * xv[4] + bf_hi(w.z) * xv[5] + bf_lo(w.w) * xv[6] + bf_hi(w.w) * xv[7];
}

// ---- shared-memory carve-up (host and device agree through this) -----------------------------------
struct SmemLayout {
  size_t xs, xq, sxd, zpart, wpart, score, tab, fl_j, fl_delta, rc, flagbits, wred, misc, total;
  __host__ __device__ SmemLayout(int d, int dpad, int ngroups) {
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; size_t r = o; o += bytes; return r; };
    xs = take(size_t(dpad) * sizeof(float), 16);
    xq = take(size_t(4) * (dpad + 64), 128);
    sxd = take(size_t(ngroups + 16) * sizeof(double), 8);
    zpart = take(size_t(NW) * 16 * sizeof(double), 8);
    wpart = take(size_t(LOADS) * NW * sizeof(float), 4);
    score = take(MAXROWS * sizeof(double), 8);
    tab = take(size_t(5) * MAXROWS * sizeof(float), 4);
    fl_j = take(MAXROWS * sizeof(int), 4);
    fl_delta = take(MAXROWS * sizeof(float), 4);
    rc = take(MAXRC * sizeof(int), 4);
    flagbits = take(MAXROWS * sizeof(int), 4);
    wred = take(size_t(3) * NW * sizeof(float), 4);
    misc = take(32 * sizeof(int), 8);
    total = o;
    (void)d;
  }
};
enum { MS_NFL = 0, MS_NRC = 1, MS_WCNT = 8 };

// ---- the kernel ---------------------------------------------------------------------------------------
template <int VPT>
__global__ void __launch_bounds__(NTH, CTAS_PER_SM) k_decode(const Params p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout L(p.d, p.dpad, p.ngroups);
  float* xs = reinterpret_cast<float*>(smem + L.xs);
  uint8_t* xq = smem + L.xq;
  double* sxd = reinterpret_cast<double*>(smem + L.sxd);
  double* zpart = reinterpret_cast<double*>(smem + L.zpart);
  float* wpart = reinterpret_cast<float*>(smem + L.wpart);
  double* score = reinterpret_cast<double*>(smem + L.score);
  float* tab = reinterpret_cast<float*>(smem + L.tab);   // [5][MAXROWS]: lo, hi, b1, a, c of the CTA's neurons
  int* fl_j = reinterpret_cast<int*>(smem + L.fl_j);
  float* fl_delta = reinterpret_cast<float*>(smem + L.fl_delta);
  int* rc = reinterpret_cast<int*>(smem + L.rc);
  int* flagbits = reinterpret_cast<int*>(smem + L.flagbits);
  float* wred = reinterpret_cast<float*>(smem + L.wred);
  volatile int* misc = reinterpret_cast<volatile int*>(smem + L.misc);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = p.d;
  const int xq_stride = p.dpad + 64;
  const int2 plan = p.plan[blockIdx.x];
  const int TS = 1 << p.ts_log2, KS = NW >> p.ts_log2;
  const int ts = warp & (TS - 1), ks = warp >> p.ts_log2;
  const bool pred_warp = ts < plan.y;
  const int g = lane >> 2, t4 = lane & 3;

  // ---- first predictor block: independent of x, so its latency hides behind the x preparation ----
  const uint8_t* pb = p.pblocks + (size_t(plan.x + (pred_warp ? ts : 0)) * p.nkc) * p.pbs;
  uint4 cw0 = make_uint4(0u, 0u, 0u, 0u), cw1 = cw0;
  if (pred_warp && ks < p.nkc) {
    const uint8_t* blk = pb + size_t(ks) * p.pbs;
    cw0 = ldg_stream(blk + lane * 16);
    cw1 = ldg_stream(blk + 512 + lane * 16);
  }

  // per-neuron tables of the CTA's rows (their latency also hides behind the x preparation)
  if (tid < plan.y * 16) {
    const int j = plan.x * 16 + tid;
    tab[tid] = p.lo[j]; tab[MAXROWS + tid] = p.hi[j]; tab[2 * MAXROWS + tid] = p.b1[j];
    tab[3 * MAXROWS + tid] = p.a[j]; tab[4 * MAXROWS + tid] = p.c[j];
  }

  // ---- x -> fp32 copy in shared memory, max |x| ----
  {
    float amax = 0.f;
    bool nonfinite = false;
    for (int v = tid; v * 8 < p.dpad; v += NTH) {
      float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (v < p.nvec) {
        const uint4 w = *reinterpret_cast<const uint4*>(p.x + size_t(v) * 8);
        f[0] = bf_lo(w.x); f[1] = bf_hi(w.x); f[2] = bf_lo(w.y); f[3] = bf_hi(w.y);
        f[4] = bf_lo(w.z); f[5] = bf_hi(w.z); f[6] = bf_lo(w.w); f[7] = bf_hi(w.w);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (!(fabsf(f[i]) <= 3.0e38f)) nonfinite = true;
        amax = fmaxf(amax, fabsf(f[i]));
      }
      *reinterpret_cast<float4*>(xs + v * 8) = make_float4(f[0], f[1], f[2], f[3]);
      *reinterpret_cast<float4*>(xs + v * 8 + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    amax = fmaxf(amax, 0.f);   // drops NaN
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const bool any_nf = __any_sync(0xffffffffu, nonfinite);
    if (lane == 0) { wred[warp] = amax; wred[NW + warp] = any_nf ? 1.f : 0.f; }
    if (tid < 32) misc[tid] = 0;
  }
  __syncthreads();
  float amax_all = 0.f;
  bool tok_nonfinite = false;
#pragma unroll
  for (int w = 0; w < NW; ++w) { amax_all = fmaxf(amax_all, wred[w]); tok_nonfinite |= wred[NW + w] != 0.f; }
  // exponent E: |x| 2^-E < 2^24 for every element
  int E = 0;
  if (amax_all > 0.f && !tok_nonfinite) E = max(int((__float_as_uint(amax_all) >> 23) & 0xff) - 127 - 23, -100);

  // ---- fixed-point limbs of x in tensor-core operand order; group sums; truncation residual ----
  {
    const float inv = __uint_as_float(uint32_t(127 - E) << 23);    // 2^-E
    const int units = p.dpad / 16;
    const int lpg = p.G / 16;                                       // lanes (units) per predictor group
    float resid = 0.f;
    for (int u0 = 0; u0 < units; u0 += NTH) {
      const int u = u0 + tid;
      const bool active = u < units;
      uint32_t D[16];
      int sx = 0;
#pragma unroll
      for (int cidx = 0; cidx < 16; ++cidx) {
        const int k = u * 16 + cidx;
        const float v = (active && !tok_nonfinite && k < d) ? xs[k] * inv : 0.f;
        const int X = __float2int_rz(v);
        resid += fabsf(v - float(X));
        sx += X;
        // signed base-256 digits of X 4^(3-f): adding 0x80 to the three low bytes and flipping
        // those bits back leaves byte l = digit l as a signed 8-bit value
        const uint32_t Y = uint32_t(X) << (2 * (3 - (cidx & 3)));
        D[cidx] = (Y + 0x00808080u) ^ 0x00808080u;
      }
      if (active) {
        const int kb = u >> 2, t = u & 3;
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          uint32_t wv[4];   // word f: byte i = digit l of channel 4 i + f
#pragma unroll
          for (int f = 0; f < 4; ++f) {
            const uint32_t lo2 = __byte_perm(D[f], D[4 + f], 0x0040 + l * 0x0011);       // bytes: D[f].l, D[4+f].l
            const uint32_t hi2 = __byte_perm(D[8 + f], D[12 + f], 0x0040 + l * 0x0011);
            wv[f] = __byte_perm(lo2, hi2, 0x5410);
          }
          *reinterpret_cast<uint4*>(xq + size_t(l) * xq_stride + size_t(kb) * 64 + t * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
      // group sums of the integer x (exact)
      for (int o = 1; o < lpg; o <<= 1) sx += __shfl_xor_sync(0xffffffffu, sx, o);
      if (active && (lane & (lpg - 1)) == 0) sxd[u / lpg] = double(sx);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) resid += __shfl_xor_sync(0xffffffffu, resid, o);
    if (lane == 0) wred[2 * NW + warp] = resid;
  }
  __syncthreads();
  // tolerance of the fast score: every dropped fraction (< 1 unit of 2^E) times |code - zero| <= 3 times the scale
  double tau;
  {
    float rs = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) rs += wred[2 * NW + w];
    tau = double(rs) * 1.001 * 3.0 * double(*p.smax) * ldexp(1.0, E);
  }

  // ---- predictor: this warp's tile over its share of the channel chunks ----
  if (pred_warp) {
    double zacc[4] = {0.0, 0.0, 0.0, 0.0}, zt[2] = {0.0, 0.0};
    const int kb_per_group = p.G / 64;
    const int gpc = KC / p.G;
    for (int kc = ks; kc < p.nkc; kc += KS) {
      const uint8_t* blk = pb + size_t(kc) * p.pbs;
      // next block's codes
      uint4 n0 = make_uint4(0u, 0u, 0u, 0u), n1 = n0;
      if (kc + KS < p.nkc) {
        const uint8_t* nb = blk + size_t(KS) * p.pbs;
        n0 = ldg_stream(nb + lane * 16);
        n1 = ldg_stream(nb + 512 + lane * 16);
      }
      const uint2* mp = reinterpret_cast<const uint2*>(blk + 1024);
      uint2 mw[4];
#pragma unroll
      for (int gl = 0; gl < 4; ++gl) mw[gl] = gl < gpc ? __ldg(&mp[gl * 8 + g]) : make_uint2(0u, 0u);
      int ia[4] = {0, 0, 0, 0};
#pragma unroll
      for (int pair = 0; pair < 2; ++pair) {
        const uint4 cw = pair ? cw1 : cw0;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int kbl = pair * 2 + half;              // 64-channel block inside the 256-channel chunk
          const int kb = kc * 4 + kbl;
          const uint32_t A = half ? cw.z : cw.x, B = half ? cw.w : cw.y;
          uint4 xb = make_uint4(0u, 0u, 0u, 0u);
          if (g < 4) xb = *reinterpret_cast<const uint4*>(xq + size_t(g) * xq_stride + size_t(kb) * 64 + t4 * 16);
          mma_u8s8(ia, A & 0x03030303u, B & 0x03030303u, A & 0x0C0C0C0Cu, B & 0x0C0C0C0Cu, xb.x, xb.y);
          mma_u8s8(ia, A & 0x30303030u, B & 0x30303030u, A & 0xC0C0C0C0u, B & 0xC0C0C0C0u, xb.z, xb.w);
          if ((kbl + 1) % kb_per_group == 0) {
            const int gl = kbl / kb_per_group;          // group inside the chunk
            const uint2 m = gl == 0 ? mw[0] : gl == 1 ? mw[1] : gl == 2 ? mw[2] : mw[3];
            const double s0 = double(bf_hi(m.x)), s1 = double(bf_hi(m.y));
            zacc[0] += s0 * double(ia[0]); zacc[1] += s0 * double(ia[1]);
            zacc[2] += s1 * double(ia[2]); zacc[3] += s1 * double(ia[3]);
            const double sx = sxd[min(kb / kb_per_group, p.ngroups - 1)];
            zt[0] += s0 * double(m.x & 3u) * sx;
            zt[1] += s1 * double(m.y & 3u) * sx;
            ia[0] = ia[1] = ia[2] = ia[3] = 0;
          }
        }
      }
      cw0 = n0; cw1 = n1;
    }
    // limbs: lane t4 = 0 holds limbs 0,1 ; t4 = 1 holds limbs 2,3 (columns 4..7 are unused for one token)
    double v0 = 0.0, v1 = 0.0;
    if (t4 == 0) { v0 = zacc[0] + 256.0 * zacc[1]; v1 = zacc[2] + 256.0 * zacc[3]; }
    if (t4 == 1) { v0 = 65536.0 * (zacc[0] + 256.0 * zacc[1]); v1 = 65536.0 * (zacc[2] + 256.0 * zacc[3]); }
    v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
    v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
    if (t4 == 0) {
      zpart[(ks * TS + ts) * 16 + g] = v0 * (1.0 / 64.0) - zt[0];
      zpart[(ks * TS + ts) * 16 + g + 8] = v1 * (1.0 / 64.0) - zt[1];
    }
  }
  __syncthreads();

  // ---- scores, flags ----
  const int nrow = plan.y * 16;
  if (tid < nrow) {
    const int tl = tid >> 4, r = tid & 15;
    const int j = (plan.x + tl) * 16 + r;
    double s = 0.0;
    for (int k = 0; k < KS; ++k) s += zpart[(k * TS + tl) * 16 + r];
    const double zhat = double(tab[2 * MAXROWS + tid]) + ldexp(s, E);
    const double lo = double(tab[tid]), hi = double(tab[MAXROWS + tid]);
    int f = ((lo <= zhat) && (zhat < hi)) ? 0 : 1;
    if (tok_nonfinite) f = 1;
    else if (tau > 0.0 && (fabs(zhat - lo) <= tau || fabs(zhat - hi) <= tau)) {
      const int q = atomicAdd(const_cast<int*>(&misc[MS_NRC]), 1);
      if (q < MAXRC) rc[q] = tid;
      else {                                        // list full: this thread re-evaluates its neuron alone
        const int nwords = d / 16;
        double a64 = 0.0;
        for (int w = 0; w < nwords; ++w) {
          const uint32_t word = p.codes[size_t(j) * nwords + w];
          const int grp = (w * 16) / p.G;
          const double zp = double(p.zero[size_t(j) * p.ngroups + grp]);
          double inner = 0.0;
          for (int q2 = 0; q2 < 16; ++q2) inner += (double((word >> (2 * q2)) & 3u) - zp) * double(xs[w * 16 + q2]);
          a64 += double(__bfloat162float(p.scale[size_t(j) * p.ngroups + grp])) * inner;
        }
        const double z2 = a64 + double(p.b1[j]);
        f = ((lo <= z2) && (z2 < hi)) ? 0 : 1;
        score[tid] = z2;
        flagbits[tid] = f;
        f |= 4;
      }
    }
    if (!(f & 4)) {
      flagbits[tid] = f;
      score[tid] = tok_nonfinite ? __longlong_as_double(0x7ff8000000000000ll) : zhat;
    }
  }
  __syncthreads();
  // exact re-evaluation from the original codes (rare): one warp per listed neuron
  {
    const int nrc = min(int(misc[MS_NRC]), MAXRC);
    const int nwords = d / 16;
    for (int e = warp; e < nrc; e += NW) {
      const int n = rc[e];
      const int j = (plan.x + (n >> 4)) * 16 + (n & 15);
      double a64 = 0.0;
      for (int w = lane; w < nwords; w += 32) {
        const uint32_t word = p.codes[size_t(j) * nwords + w];
        const int grp = (w * 16) / p.G;
        const double zp = double(p.zero[size_t(j) * p.ngroups + grp]);
        double inner = 0.0;
#pragma unroll
        for (int q = 0; q < 16; ++q) inner += (double((word >> (2 * q)) & 3u) - zp) * double(xs[w * 16 + q]);
        a64 += double(__bfloat162float(p.scale[size_t(j) * p.ngroups + grp])) * inner;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a64 += __shfl_xor_sync(0xffffffffu, a64, o);
      if (lane == 0) {
        const double zhat = a64 + double(p.b1[j]);
        flagbits[n] = ((double(p.lo[j]) <= zhat) && (zhat < double(p.hi[j]))) ? 0 : 1;
        score[n] = zhat;
      }
    }
    if (nrc > 0) {
      if (tid == 0) atomicAdd(&p.counters[CTR_RECHECKS], (unsigned long long)nrc);
      __syncthreads();
    }
  }
  // ---- ascending flagged list: ballot + prefix over the (at most 8) warps that hold rows ----
  {
    const int f = (tid < nrow) ? (flagbits[tid] & 1) : 0;
    const uint32_t bal = __ballot_sync(0xffffffffu, f != 0);
    if (lane == 0) misc[MS_WCNT + warp] = __popc(bal);
    __syncthreads();
    int base = 0, total = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) { const int cnt = misc[MS_WCNT + w]; if (w < warp) base += cnt; total += cnt; }
    if (f) fl_j[base + __popc(bal & ((1u << lane) - 1u))] = (plan.x + (tid >> 4)) * 16 + (tid & 15);
    if (tid == 0) misc[MS_NFL] = total;
    // debug capture: 16-bit halves of the flag words, scores
    if (p.dbg_bitmap && tid < nrow && (tid & 15) == 0)
      reinterpret_cast<uint16_t*>(p.dbg_bitmap)[plan.x + (tid >> 4)] = uint16_t((bal >> (lane & 16)) & 0xffffu);
    if (p.dbg_scores && tid < nrow) p.dbg_scores[(plan.x + (tid >> 4)) * 16 + (tid & 15)] = score[tid];
    // flagged-count statistics: the last CTA to report moves the token's total into the counters
    if (tid == 0) {
      if (total) atomicAdd(&p.ctl[CTL_NFL], (unsigned int)total);
      __threadfence();
      if (atomicAdd(&p.ctl[CTL_ARRIVED], 1u) == gridDim.x - 1) {
        __threadfence();
        const unsigned int tot = atomicExch(&p.ctl[CTL_NFL], 0u);
        atomicAdd(&p.counters[CTR_FLAGGED_TOTAL], (unsigned long long)tot);
        atomicMax(&p.counters[CTR_FLAGGED_MAX], (unsigned long long)tot);
        atomicExch(&p.ctl[CTL_ARRIVED], 0u);
      }
    }
  }
  __syncthreads();
  const int nfl = misc[MS_NFL];

  // ---- this thread's columns ----
  int col[VPT];
  bool cval[VPT];
#pragma unroll
  for (int m = 0; m < VPT; ++m) {
    const int vl = m * 32 + lane, vec = warp * p.cw + vl;
    cval[m] = vl < p.cw && vec < p.nvec;
    col[m] = cval[m] ? vec * 8 : 0;
  }
  float acc[VPT][8];
#pragma unroll
  for (int m = 0; m < VPT; ++m)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[m][i] = 0.f;

  // ---- result fixing: W1 rows -> z_j -> delta_j ; W2T rows scaled by delta_j ----
  if (nfl > 0) {
    float xr[VPT][8];
#pragma unroll
    for (int m = 0; m < VPT; ++m) {
      const float4 q0 = *reinterpret_cast<const float4*>(xs + col[m]);
      const float4 q1 = *reinterpret_cast<const float4*>(xs + col[m] + 4);
      xr[m][0] = q0.x; xr[m][1] = q0.y; xr[m][2] = q0.z; xr[m][3] = q0.w;
      xr[m][4] = q1.x; xr[m][5] = q1.y; xr[m][6] = q1.z; xr[m][7] = q1.w;
    }
    constexpr int FB = LOADS / VPT;   // flagged rows per batch
    for (int e0 = 0; e0 < nfl; e0 += FB) {
      uint4 w[FB][VPT];
      int jr[FB];
#pragma unroll
      for (int r = 0; r < FB; ++r) {
        jr[r] = (e0 + r < nfl) ? fl_j[e0 + r] : -1;
#pragma unroll
        for (int m = 0; m < VPT; ++m)
          w[r][m] = (jr[r] >= 0 && cval[m]) ? ldg_stream(p.W1 + size_t(jr[r]) * d + col[m]) : make_uint4(0u, 0u, 0u, 0u);
      }
      float part[FB];
#pragma unroll
      for (int r = 0; r < FB; ++r) {
        part[r] = 0.f;
#pragma unroll
        for (int m = 0; m < VPT; ++m) part[r] += dot8(w[r][m], xr[m]);
      }
      // the W2T rows of the same neurons go in flight while the dot products meet
#pragma unroll
      for (int r = 0; r < FB; ++r)
#pragma unroll
        for (int m = 0; m < VPT; ++m)
          w[r][m] = (jr[r] >= 0 && cval[m]) ? ldg_stream(p.W2T + size_t(jr[r]) * d + col[m]) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int r = 0; r < FB; ++r) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part[r] += __shfl_xor_sync(0xffffffffu, part[r], o);
        if (lane == 0) wpart[r * NW + warp] = part[r];
      }
      __syncthreads();
      if (tid < FB && e0 + tid < nfl) {
        const int row = fl_j[e0 + tid] - plan.x * 16;
        float z = 0.f;
#pragma unroll
        for (int ww = 0; ww < NW; ++ww) z += wpart[tid * NW + ww];
        z += tab[2 * MAXROWS + row];
        fl_delta[tid] = gelu_f32(z, p.act) - tab[3 * MAXROWS + row] * z - tab[4 * MAXROWS + row];
      }
      __syncthreads();
#pragma unroll
      for (int r = 0; r < FB; ++r) {
        const float dl = (jr[r] >= 0) ? fl_delta[r] : 0.f;
#pragma unroll
        for (int m = 0; m < VPT; ++m) fma8(acc[m], dl, w[r][m]);
      }
    }
  }

  // ---- speculative folded product: row chunks of C drawn from this column range's ticket ----
  {
    constexpr int TK = LOADS / VPT;   // rows per chunk
    unsigned int* ticket = p.ctl + CTL_TICKET + warp * 32;
    auto issue = [&]() -> unsigned int {     // lane 0 draws; the value is looked at one step later
      unsigned int t = 0;
      if (lane == 0) t = atomicAdd(ticket, 1u);
      return t;
    };
    auto resolve = [&](unsigned int raw) -> int {
      const unsigned int t = __shfl_sync(0xffffffffu, raw, 0);
      return t < (unsigned int)p.ntk ? int(t) : -1;
    };
    auto load = [&](uint4 (&buf)[TK][VPT], int tk) {
#pragma unroll
      for (int r = 0; r < TK; ++r) {
        const int k = tk * TK + r;
#pragma unroll
        for (int m = 0; m < VPT; ++m)
          buf[r][m] = (k < d && cval[m]) ? ldg_stream(p.C + size_t(k) * d + col[m]) : make_uint4(0u, 0u, 0u, 0u);
      }
    };
    auto consume = [&](const uint4 (&buf)[TK][VPT], int tk) {
#pragma unroll
      for (int r = 0; r < TK; ++r) {
        const int k = tk * TK + r;
        const float sc = k < d ? xs[k] : 0.f;
#pragma unroll
        for (int m = 0; m < VPT; ++m) fma8(acc[m], sc, buf[r][m]);
      }
    };
    uint4 b0[TK][VPT], b1[TK][VPT];
    int t0 = resolve(issue());
    int t1 = t0 >= 0 ? resolve(issue()) : -1;
    if (t0 >= 0) load(b0, t0);
    if (t1 >= 0) load(b1, t1);
    bool more = t1 >= 0;
    while (t0 >= 0) {
      unsigned int raw = more ? issue() : 0xffffffffu;
      consume(b0, t0);
      t0 = more ? resolve(raw) : -1;
      more = t0 >= 0;
      if (t0 >= 0) load(b0, t0);
      if (t1 < 0) break;
      raw = more ? issue() : 0xffffffffu;
      consume(b1, t1);
      t1 = more ? resolve(raw) : -1;
      more = t1 >= 0;
      if (t1 >= 0) load(b1, t1);
    }
  }

  // ---- combine: add this warp's columns; the last warp on a column range finishes it ----
#pragma unroll
  for (int m = 0; m < VPT; ++m)
    if (cval[m]) {
      red_add_v4(p.yacc + col[m], acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
      red_add_v4(p.yacc + col[m] + 4, acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
    }
  __threadfence();
  __syncwarp();
  unsigned int arrived = 0;
  if (lane == 0) arrived = atomicAdd(&p.ctl[CTL_DONE + warp * 32], 1u);
  arrived = __shfl_sync(0xffffffffu, arrived, 0);
  if (arrived == gridDim.x - 1) {
    __threadfence();
#pragma unroll
    for (int m = 0; m < VPT; ++m)
      if (cval[m]) {
        const float4 a0 = __ldcg(reinterpret_cast<const float4*>(p.yacc + col[m]));
        const float4 a1 = __ldcg(reinterpret_cast<const float4*>(p.yacc + col[m] + 4));
        const float4 q0 = *reinterpret_cast<const float4*>(p.bf + col[m]);
        const float4 q1 = *reinterpret_cast<const float4*>(p.bf + col[m] + 4);
        __nv_bfloat162 o[4];
        o[0] = __floats2bfloat162_rn(a0.x + q0.x, a0.y + q0.y);
        o[1] = __floats2bfloat162_rn(a0.z + q0.z, a0.w + q0.w);
        o[2] = __floats2bfloat162_rn(a1.x + q1.x, a1.y + q1.y);
        o[3] = __floats2bfloat162_rn(a1.z + q1.z, a1.w + q1.w);
        *reinterpret_cast<uint4*>(p.y + col[m]) = *reinterpret_cast<const uint4*>(o);
        *reinterpret_cast<float4*>(p.yacc + col[m]) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(p.yacc + col[m] + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    if (lane == 0) {
      p.ctl[CTL_TICKET + warp * 32] = 0u;
      p.ctl[CTL_DONE + warp * 32] = 0u;
    }
  }
}

// ---- set-up kernels --------------------------------------------------------------------------------------
// Predictor blocks: block (tile, kc) = 2 x 32 lanes x {A0,B0,A1,B1} code words + per-group {row g, row g+8} metadata.
__global__ void k_pack_pblocks(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                               const uint8_t* __restrict__ zero, uint8_t* __restrict__ out, int d, int h, int G,
                               int nkc, int pbs) {
  const int tile = blockIdx.x, kc = blockIdx.y;
  uint8_t* blk = out + (size_t(tile) * nkc + kc) * pbs;
  const int nwords = d / 16, ng = d / G;
  for (int e = threadIdx.x; e < 256; e += blockDim.x) {        // 256 code words
    const int pair = e >> 7, ln = (e >> 2) & 31, sub = e & 3;   // sub: 0 A(half0) 1 B(half0) 2 A(half1) 3 B(half1)
    const int gg = ln >> 2, tt = ln & 3;
    const int row = tile * 16 + gg + ((sub & 1) ? 8 : 0);
    const int kbl = pair * 2 + (sub >> 1);
    const int word = (kc * 4 + kbl) * 4 + tt;
    reinterpret_cast<uint32_t*>(blk)[e] = (word < nwords) ? codes[size_t(row) * nwords + word] : 0u;
  }
  const int gpc = KC / G;
  for (int e = threadIdx.x; e < gpc * 16; e += blockDim.x) {
    const int gl = e >> 4, gg = (e >> 1) & 7, hi = e & 1;
    const int row = tile * 16 + gg + (hi ? 8 : 0);
    const int grp = kc * gpc + gl;
    uint32_t w = 0u;
    if (grp < ng) w = (uint32_t(__bfloat16_as_ushort(scale[size_t(row) * ng + grp])) << 16) | uint32_t(zero[size_t(row) * ng + grp] & 3u);
    reinterpret_cast<uint32_t*>(blk + 1024)[e] = w;
  }
  (void)h;
}

__global__ void k_max_scale(const __nv_bfloat16* __restrict__ scale, size_t count, float* out) {
  float m = 0.f;
  for (size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x; e < count; e += size_t(gridDim.x) * blockDim.x)
    m = fmaxf(m, fabsf(__bfloat162float(scale[e])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
}

}  // namespace dec

using namespace dec;

tardis_status_t decode_prepare(Handle* H, cudaStream_t s) {
  H->dscratch = nullptr;
  H->codes_mma = nullptr;
  const int d = H->d, h = H->h, G = H->G;
  if (H->dtype != TARDIS_BF16) return TARDIS_OK;
  if (!(G == 64 || G == 128 || G == 256)) return TARDIS_OK;         // generic kernels serve other group sizes
  const int grid = H->num_sms * CTAS_PER_SM;
  const int NT = h / 16;
  const int tiles_max = (NT + grid - 1) / grid;
  const int nvec = d / 8;
  const int cw = (nvec + NW - 1) / NW;
  const int vpt = (cw + 31) / 32;
  if (tiles_max > NW || vpt > 2 || d < 64) return TARDIS_OK;
  Scratch* S = new (std::nothrow) Scratch();
  if (!S) return TARDIS_ERR_ALLOC;
  memset(S, 0, sizeof(*S));
  Params& p = S->base;
  p.d = d; p.h = h; p.G = G; p.ngroups = H->ngroups; p.act = H->act;
  p.dpad = (d + KC - 1) / KC * KC;
  p.nkc = p.dpad / KC;
  p.pbs = 1024 + 64 * (KC / G);
  p.ts_log2 = 0;
  while ((1 << p.ts_log2) < tiles_max) ++p.ts_log2;
  p.nvec = nvec; p.cw = cw;
  const int tk_rows = LOADS / vpt;
  p.ntk = (d + tk_rows - 1) / tk_rows;
  S->grid = grid; S->vpt = vpt;
  S->smem_bytes = SmemLayout(d, p.dpad, p.ngroups).total;
  int max_smem = 0;
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, H->device));
  if (S->smem_bytes > size_t(max_smem)) { delete S; return TARDIS_OK; }

  auto fail = [&](tardis_status_t st) { H->dscratch = S; decode_release(H); return st; };
  size_t tally = 0;
  const size_t pb_bytes = size_t(NT) * p.nkc * p.pbs;
  cudaError_t e = cudaMalloc(&S->pblocks, pb_bytes); tally += pb_bytes;
  if (e == cudaSuccess) { e = cudaMalloc(&S->plan, sizeof(int2) * grid); tally += sizeof(int2) * grid; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->smax, 16); tally += 16; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->yacc, sizeof(float) * d); tally += sizeof(float) * d; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->ctl, sizeof(unsigned int) * CTL_WORDS); tally += sizeof(unsigned int) * CTL_WORDS; }
  if (e != cudaSuccess) { set_last_error(e, "cudaMalloc"); cudaGetLastError(); return fail(TARDIS_ERR_ALLOC); }
  S->bytes = tally;

  // tiles spread evenly over the CTAs
  std::vector<int2> plan(grid);
  int tile_cum = 0;
  for (int c = 0; c < grid; ++c) {
    const int tc = NT / grid + (c < NT % grid ? 1 : 0);
    plan[c] = make_int2(tile_cum, tc);
    tile_cum += tc;
  }
  e = cudaMemcpyAsync(S->plan, plan.data(), sizeof(int2) * grid, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);   // plan.data() is a stack-owned host buffer
  if (e == cudaSuccess) e = cudaMemsetAsync(S->smax, 0, 16, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(S->yacc, 0, sizeof(float) * d, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(S->ctl, 0, sizeof(unsigned int) * CTL_WORDS, s);
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare"); return fail(TARDIS_ERR_CUDA); }
  k_pack_pblocks<<<dim3(NT, p.nkc), 128, 0, s>>>(H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero,
                                                 S->pblocks, d, h, G, p.nkc, p.pbs);
  k_max_scale<<<64, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->scale), size_t(h) * H->ngroups, S->smax);
  e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_decode<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S->smem_bytes));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_decode<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S->smem_bytes));
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare launch"); return fail(TARDIS_ERR_CUDA); }

  p.pblocks = S->pblocks; p.plan = S->plan; p.smax = S->smax; p.yacc = S->yacc; p.ctl = S->ctl;
  p.W1 = static_cast<const __nv_bfloat16*>(H->W1); p.W2T = static_cast<const __nv_bfloat16*>(H->W2T);
  p.C = static_cast<const __nv_bfloat16*>(H->C); p.bf = H->bf; p.lo = H->lo; p.hi = H->hi; p.a = H->a; p.c = H->c; p.b1 = H->b1;
  p.codes = H->codes; p.scale = static_cast<const __nv_bfloat16*>(H->scale); p.zero = H->zero;
  p.counters = H->counters;
  H->dscratch = S;
  H->dscratch_bytes = S->bytes;
  H->bytes_scratch += S->bytes - pb_bytes;
  H->bytes_predictor += pb_bytes;
  H->codes_mma = reinterpret_cast<uint32_t*>(S->pblocks);
  return TARDIS_OK;
}

tardis_status_t launch_decode_forward(Handle* H, const void* x, void* y, int n, cudaStream_t s) {
  Scratch* S = static_cast<Scratch*>(H->dscratch);
  for (int t = 0; t < n; ++t) {
    Params p = S->base;
    p.x = static_cast<const __nv_bfloat16*>(x) + size_t(t) * H->d;
    p.y = static_cast<__nv_bfloat16*>(y) + size_t(t) * H->d;
    p.dbg_bitmap = H->dbg_bitmap ? H->dbg_bitmap + size_t(t) * (H->h / 32) : nullptr;
    p.dbg_scores = H->dbg_scores ? H->dbg_scores + size_t(t) * H->h : nullptr;
    if (S->vpt == 1) k_decode<1><<<S->grid, NTH, S->smem_bytes, s>>>(p);
    else k_decode<2><<<S->grid, NTH, S->smem_bytes, s>>>(p);
    H->launches += 1;
  }
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

void decode_release(Handle* H) {
  Scratch* S = static_cast<Scratch*>(H->dscratch);
  if (!S) return;
  void* ptrs[] = {S->pblocks, S->plan, S->smax, S->yacc, S->ctl};
  for (void* q : ptrs)
    if (q) cudaFree(q);
  delete S;
  H->dscratch = nullptr;
  H->codes_mma = nullptr;
}

}  // namespace tardis
