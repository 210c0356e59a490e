// Fused decode kernel of the online path (Section 5.4) for calls of 1 to 4 tokens on bf16 layers, sm_100a.
//
// One launch does the whole call: predictor scores (Section 5.3), flagging and compaction, speculative
// folded product, result fixing over the union of the flagged neurons.  One CTA of 32 warps per SM.
//
//   * Prologue (before griddepcontrol.wait, so it overlaps the tail of the previous launch in the stream):
//     the CTA owns a few 16-neuron tiles; their predictor blocks (packed 2-bit codes + one word per
//     neuron and group) are fetched with bulk async copies into shared memory.
//   * x of every token is loaded once: a bf16 copy in shared memory, and a 4-limb signed base-256 fixed-point
//     copy (of two tokens at a time) in tensor-core operand order.
//   * Warps 16..31 then stream the folded matrix (stored in A-fragment order, 8 KB units drawn from one
//     global ticket) through mma.m16n8k16.bf16 with the tokens as operand columns, straight from global
//     memory into registers, and add the partial outputs to an fp32 accumulator in global memory.
//   * Warps 0..15 evaluate the predictor on the integer tensor cores (mma.m16n8k32.u8.s8): the codes are
//     masked out of the packed words (the field position is a power-of-4 weight that the pre-scaling of x
//     undoes); the 8 operand columns are the 4 limbs of two tokens.  The integer group sums are exact; they are
//     scaled by the bf16 group scales and added up in fp32.  The fp32 steps and the truncation of tiny x
//     elements have a bound tau; a score within tau of a range end is re-evaluated in fp64 from the codes, so
//     the flags are the exact ones.  Calls of 3 or 4 tokens run this pass twice.
//   * Result fixing, all 32 warps: W1 rows, then W2^T rows of the union of the flagged neurons arrive by one
//     bulk copy per row in a ring of row slots (the predictor buffers, free by then).  A step of the ring holds
//     up to 16 rows.  Pre-activations: one mma.m16n8k16 chain per warp over its share of the channels (A = 16
//     rows by ldmatrix, B = x of the tokens), partial sums meet in shared memory, delta = act(z) - a z - c
//     for the tokens that flagged the neuron, else 0.  Outputs: A = the W2^T rows transposed by
//     ldmatrix.trans (16 output columns x 16 neurons), B = delta split into two bf16 terms, accumulators
//     for all output columns stay in registers over all steps.
//   * All partial outputs are added (red.global) into one of a few replicas of the fp32 accumulator; CTAs
//     count themselves when done; the last one sums the replicas, adds b_f, rounds to bf16, writes y and
//     re-zeroes the scratch.
#include <stdio.h>

#include <new>
#include <vector>

#include "common.cuh"
#include "exact.cuh"
#include "ptx.cuh"

namespace tardis {
namespace fz {
using namespace ptx;

constexpr int NW = 32;            // warps per CTA
constexpr int NWP = 16;           // of them, predictor warps (the others stream the folded matrix meanwhile)
constexpr int NTH = NW * 32;
constexpr int NTP = NWP * 32;     // threads of the predictor warps
constexpr int KC = 256;           // channels per predictor block
constexpr int MAXT = 4;           // tokens per launch
constexpr int MAXTILES = 10;      // predictor tiles (of 16 neurons) per CTA
constexpr int MAXRC = 64;         // exact re-checks per CTA and pass before the list overflows (rest handled in place)
constexpr int MAXBUF = 10;        // predictor tile buffers in shared memory
constexpr int MAXGROUPS = 4;      // slot groups (one barrier each, one buffer of partial sums each) of the result fixing
constexpr int MAXGS = 16;         // rows per slot group (one MMA tile)
constexpr int NREP = 1;           // replicas of the output accumulator (more replicas spread the reductions, but the last CTA
                                  // reads them all: one measured fastest)
constexpr int CTMAX = 9;          // 16-column output tiles per warp (d <= 32 * 16 * CTMAX = 4608)
// control words (unsigned int) in global scratch; all zero between calls
constexpr int CTL_TICKET = 0;     // next unit of the folded matrix
constexpr int CTL_DONE = 32;      // CTAs that have added all their contributions
constexpr int CTL_NFL = 64;       // [MAXT] flagged neurons per token so far
constexpr int CTL_UNION = 72;     // neurons flagged by any token
constexpr int CTL_WORDS = 96;

struct Params {
  const uint8_t* pblocks;  // [tile][kchunk] predictor blocks
  int pbs, nkc, G;
  const __nv_bfloat16 *W1, *W2T;
  const uint4* Cp;         // folded matrix in tensor-core fragment order
  const float *bf, *lo, *hi, *a, *c, *b1;
  const uint32_t* codes; const __nv_bfloat16* scale; const uint8_t* zero;   // originals (exact re-check)
  const float* smax;       // largest group scale of the layer
  const int2* plan;        // per CTA: first tile, tile count
  const __nv_bfloat16* x; __nv_bfloat16* y;
  float* yacc;             // [NREP][MAXT][dacc] fp32
  float* dpart;            // deterministic mode: [nkc + grid][MAXT][dacc] partial outputs, each written by one owner; else null
  unsigned int* ctl; unsigned long long* counters;
  uint32_t* dbg_bitmap; double* dbg_scores;
  int n;                   // tokens of this call (1..MAXT)
  int d, dpad, dacc, h, ngroups, act;
  int nbuf, unit_bytes, buf_bytes;   // tile buffers in shared memory, bytes of a tile's blocks, bytes between buffers
  int tiles_max;
  int nvec;                // 8-column vectors in a row
  int slot_stride;         // result fixing: bytes between row slots
  int smem_total;          // dynamic shared memory of a CTA
  int gs_cap;              // result fixing: most neurons of a step (16, or 8 where that keeps one more predictor tile in shared memory)
  int nunits;              // folded-matrix units in all
};

struct Scratch {           // handle-owned device memory of this path
  uint8_t* pblocks; int2* plan; float* smax; float* yacc; unsigned int* ctl; uint4* Cp;
  Params base; size_t smem_bytes; size_t bytes; int grid; const void* kernels[2][2]; bool pairs_fit;
  float* dpart;            // partial outputs of the deterministic mode (allocated when the mode is first switched on)
  int nbuf_n[MAXT + 1];    // tile buffers in shared memory for a call of n tokens
  int gs_cap_n[MAXT + 1];  // ... and the most neurons of a step of its result fixing
};

// ---- shared-memory carve-up (host and device agree through this) -----------------------------------
// Small tables first, then x of the call's tokens, then the predictor buffers, the limbs and the partial scores.
// Everything from pbuf to the partial pre-activations at the end of the CTA's shared memory becomes the row slots of
// the result fixing.
struct SmemLayout {
  size_t zeros, sx2, tab, fl_j, fl_mask, fl_delta, rc, flagbits, red, bars, misc, xh, wz, wz_end, pbuf, xq, zpart, pred_end, slots_end;
  int xstride, xq_stride, wz_groups, ztok;
  __host__ __device__ SmemLayout(int dpad, int ngroups, int tiles_max, int nbuf, int buf_bytes, int ntok, size_t total_bytes, int gs_cap) {
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; size_t r = o; o += bytes; return r; };
    const size_t rows = size_t(tiles_max) * 16;
    xstride = dpad + 16;                      // elements between tokens of the bf16 copy (16 zeros behind each token)
    xq_stride = dpad + 64;                    // bytes between limbs
    zeros = take(256, 16);                    // what the lanes that feed unused operand columns read
    sx2 = take(size_t(2) * (ngroups + 16) * sizeof(int2), 8);
    tab = take(5 * rows * sizeof(float), 4);
    fl_j = take(rows * sizeof(int), 4);
    fl_mask = take(rows * sizeof(int), 4);
    fl_delta = take(rows * MAXT * sizeof(float), 16);
    rc = take(MAXRC * sizeof(int), 4);
    flagbits = take(rows * sizeof(int), 4);
    red = take(size_t(2) * ntok * 40 * sizeof(float), 4);  // per token and warp round: sum |x|, rounding residual
    bars = take(size_t(MAXBUF + MAXGROUPS) * sizeof(uint64_t), 8);
    misc = take(64 * sizeof(int), 8);
    xh = take(size_t(ntok) * xstride * 2, 16);
    pbuf = take(size_t(nbuf) * buf_bytes, 128);
    ztok = ntok < 2 ? ntok : 2;                            // tokens of a predictor pass
    xq = take(size_t(ztok) * 4 * xq_stride, 128);          // limbs of the tokens of a pass
    zpart = take(size_t(tiles_max) * NWP * ztok * 16 * sizeof(float), 16);
    pred_end = o;
    // the partial pre-activations of the result fixing sit at the very end: they are not needed while the predictor runs,
    // so they do not compete with its buffers for room.  One buffer per step of MAXGS neurons; as many buffers as fit behind
    // the predictor's state, MAXGROUPS at most (one at least: wz_end tells the caller whether that one fits)
    const size_t per = size_t(gs_cap) * ntok * 33 * sizeof(float);   // (gs_cap: most neurons of a step, 8 or MAXGS)
    size_t nb = total_bytes > o ? (total_bytes - o) / per : 0;
    nb = nb > size_t(MAXGROUPS) ? size_t(MAXGROUPS) : (nb < 1 ? 1 : nb);
    wz_groups = int(nb);
    const size_t wzbytes = nb * per;
    const size_t end = total_bytes > o + wzbytes ? total_bytes : o + wzbytes;
    wz = (end - wzbytes) / 16 * 16;
    wz_end = wz + wzbytes;
    slots_end = wz;
  }
};
enum { MS_NRC = 1, MS_ERR = 2, MS_LAST = 3, MS_NUN = 4, MS_AMAX = 8, MS_NONFIN = 12, MS_TOKCNT = 16, MS_WCNT = 24, MS_BUFCNT = 32 };

// ---- phase stamps (compiled in with -DTARDIS_PHASE_STAMPS only) -----------------------------------------
// Thread 0 of every CTA (and lane 0 of the first streaming warp) writes the global timer at the phase
// boundaries of the last launch; tardis_debug_phase_stamps copies the table to the host.
constexpr int kStampCtas = 512, kStampSlots = 16;
enum { ST_START = 0, ST_X = 1, ST_LIMBS = 2, ST_PRED = 3, ST_STREAM = 4, ST_FLAGS = 5, ST_FIXED = 6, ST_COUNTED = 7,
       ST_FINAL = 8, ST_NFL = 9 };
#ifdef TARDIS_PHASE_STAMPS
__device__ long long g_stamps[kStampCtas * kStampSlots];
__device__ __forceinline__ long long global_timer() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define FZ_STAMP(cond, slot) do { if ((cond) && blockIdx.x < kStampCtas) g_stamps[blockIdx.x * kStampSlots + (slot)] = global_timer(); } while (0)
#define FZ_STAMP_VALUE(cond, slot, v) do { if ((cond) && blockIdx.x < kStampCtas) g_stamps[blockIdx.x * kStampSlots + (slot)] = (long long)(v); } while (0)
#else
#define FZ_STAMP(cond, slot) do { } while (0)
#define FZ_STAMP_VALUE(cond, slot, v) do { } while (0)
#endif

__device__ __forceinline__ void ldmatrix_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr) : "memory");
}
// four 8 x 8 matrices: lanes 8 m .. 8 m + 7 give the row addresses of matrix m, register m receives it
__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
// Exact fp64 predictor sum of one neuron (row r of a tile) from the tile's predictor blocks in shared memory: the same
// terms in the same order as exact_score, which reads the original arrays in global memory.  Lane `lane` of `nl` takes
// the code words lane, lane + nl, ...; the caller adds the lanes up.
__device__ __forceinline__ double exact_from_blocks(const uint8_t* ubase, int pbs, int G, int r, const __nv_bfloat16* xt, int d,
                                                    int lane, int nl) {
  const int nwords = d >> 4, gg = r & 7, up = (r >> 3) & 1;
  double acc = 0.0;
  for (int w = lane; w < nwords; w += nl) {
    const int kc = w >> 4, kbl = (w >> 2) & 3, tt = w & 3;
    const uint8_t* blk = ubase + kc * pbs;
    const uint32_t word = reinterpret_cast<const uint32_t*>(blk)[(kbl >> 1) * 128 + (gg * 4 + tt) * 4 + up + 2 * (kbl & 1)];
    const int gl = ((w & 15) * 16) / G;
    const uint32_t mw = reinterpret_cast<const uint32_t*>(blk + 1024)[gl * 16 + gg * 2 + up];
    const double zp = double(mw & 3u);
    double inner = 0.0;
#pragma unroll
    for (int q = 0; q < 16; ++q) inner += (double((word >> (2 * q)) & 3u) - zp) * double(__bfloat162float(xt[w * 16 + q]));
    acc += double(__uint_as_float(mw & 0xffff0000u)) * inner;
  }
  return acc;
}
__device__ __forceinline__ void bar_sync_pred() { asm volatile("bar.sync 2, %0;" ::"n"(NTP) : "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  return uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(lo))) | (uint32_t(__bfloat16_as_ushort(__float2bfloat16_rn(hi))) << 16);
}

// ---- the kernel ---------------------------------------------------------------------------------------
// G: predictor group size; CT: 16-column output tiles per warp; NTK: 1 = the call has one token (most of the token loops
// fold away), 4 = up to four; FAST: every tile of the CTA has its own buffer and a warp has the same one or two channel
// pairs in every tile (their x operands stay in registers), else the general loop over a ring of tile buffers.
template <int G, int CT, int NTK, bool FAST>
__global__ void __launch_bounds__(NTH, 1) k_fused(const Params p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout L(p.dpad, p.ngroups, p.tiles_max, p.nbuf, p.buf_bytes, p.n, size_t(p.smem_total), p.gs_cap);
  uint8_t* pbuf = smem + L.pbuf;
  uint8_t* xq = smem + L.xq;
  float* zpart = reinterpret_cast<float*>(smem + L.zpart);
  __nv_bfloat16* xh = reinterpret_cast<__nv_bfloat16*>(smem + L.xh);
  int2* sx2 = reinterpret_cast<int2*>(smem + L.sx2);
  float* tab = reinterpret_cast<float*>(smem + L.tab);   // [5][TR]: lo, hi, b1, a, c of the CTA's neurons
  float* wz = reinterpret_cast<float*>(smem + L.wz);
  int* fl_j = reinterpret_cast<int*>(smem + L.fl_j);
  int* fl_mask = reinterpret_cast<int*>(smem + L.fl_mask);
  float* fl_delta = reinterpret_cast<float*>(smem + L.fl_delta);
  int* rc = reinterpret_cast<int*>(smem + L.rc);
  int* flagbits = reinterpret_cast<int*>(smem + L.flagbits);
  float* red = reinterpret_cast<float*>(smem + L.red);    // [3][MAXT][40]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
  volatile int* misc = reinterpret_cast<volatile int*>(smem + L.misc);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = p.d, n = NTK == 1 ? 1 : p.n;
  const int TR = p.tiles_max * 16;
  const int XS = L.xstride, xq_stride = L.xq_stride;
  const int2 plan = p.plan[blockIdx.x];
  const int NU = plan.y;                           // predictor units (tiles) of this CTA
  const int NP = (n + 1) >> 1;                     // predictor passes (two tokens each)
  const int NQ = NU * NP;                          // units in the order they are consumed
  const bool resident = FAST || NU <= p.nbuf;      // every tile has its own buffer: nothing is fetched twice
  const int g = lane >> 2, t4 = lane & 3;
  const int nv = p.dpad >> 3;                      // 8-channel vectors per token (padded)
  const int nrow = plan.y * 16;

  auto issue_unit = [&](int u, int b) {
    const uint32_t bytes = uint32_t(p.unit_bytes);
    mbar_expect_tx(&full[b], bytes);
    bulk_g2s(pbuf + size_t(b) * p.buf_bytes, p.pblocks + size_t(plan.x + u) * p.unit_bytes, bytes, &full[b]);
  };

  FZ_STAMP(tid == 0, ST_START);
  // Programmatic dependent launch: the next launch in the stream may start its own prologue (everything
  // up to its griddepcontrol.wait reads only the layer's constant state) while this one is still running.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid < nrow) {
    const int j = plan.x * 16 + tid;
    tab[tid] = p.lo[j]; tab[TR + tid] = p.hi[j]; tab[2 * TR + tid] = p.b1[j]; tab[3 * TR + tid] = p.a[j]; tab[4 * TR + tid] = p.c[j];
    flagbits[tid] = 0;
  }
  if (tid == 0) {
    for (int b = 0; b < MAXBUF + MAXGROUPS; ++b) mbar_init(&full[b], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 64) misc[tid] = 0;
  if (tid >= 64 && tid < 128) reinterpret_cast<uint32_t*>(smem + L.zeros)[tid - 64] = 0u;
  for (int i = tid; i < 2 * n * 40; i += NTH) red[i] = 0.f;
  __syncthreads();
  // predictor blocks first: nothing of them depends on x.  When every tile has its own buffer, all copies report to
  // one barrier; else the buffers form a ring with one barrier each.
  if (resident) {
    if (tid == 0) mbar_expect_tx(&full[0], uint32_t(NU) * uint32_t(p.unit_bytes));
    if (lane == 0 && warp < NU)
      bulk_g2s(pbuf + size_t(warp) * p.buf_bytes, p.pblocks + size_t(plan.x + warp) * p.unit_bytes, uint32_t(p.unit_bytes), &full[0]);
  } else if (lane == 0 && warp < p.nbuf && warp < NQ) {
    issue_unit(warp % NU, warp);
  }
  // tiles that have to wait for a buffer are asked into L2 meanwhile: their copies then do not queue behind the folded matrix
  if (!resident && NU > p.nbuf) {
    const char* base = reinterpret_cast<const char*>(p.pblocks + size_t(plan.x + p.nbuf) * p.unit_bytes);
    const int lines = ((NU - p.nbuf) * p.unit_bytes + 127) / 128;
    for (int i = tid; i < lines; i += NTH) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + size_t(i) * 128));
  }
  const float smax_f = *p.smax;                    // constant state of the layer: fetched before the wait

  // From here on the kernel touches what earlier work in the stream may still be writing (x, the
  // scratch shared by the calls of one handle): wait until that work has completed and is visible.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- x: bf16 copy in shared memory (channels beyond d and 16 more are zero), max |x|, sum |x| ----
  for (int base = 0; base < n * nv; base += NTH) {
    const int i = base + tid;
    if (i < n * nv) {                                // uniform over a warp (nv is a multiple of 32)
      const int t = i / nv, v = i - t * nv;
      uint4 xw = make_uint4(0u, 0u, 0u, 0u);
      if (v < p.nvec) xw = *reinterpret_cast<const uint4*>(p.x + size_t(t) * d + size_t(v) * 8);
      *reinterpret_cast<uint4*>(xh + t * XS + v * 8) = xw;
      float f[8];
      unpack8(f, xw);
      float amax = 0.f, l1 = 0.f;
      bool nonfinite = false;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (!(fabsf(f[q]) <= 3.0e38f)) nonfinite = true;
        amax = fmaxf(amax, fabsf(f[q]));
        l1 += fabsf(f[q]);
      }
      amax = fmaxf(amax, 0.f);   // drops NaN
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
      }
      const bool any_nf = __any_sync(0xffffffffu, nonfinite);
      if (lane == 0) {
        atomicMax(const_cast<int*>(&misc[MS_AMAX + t]), __float_as_int(amax));
        if (any_nf) misc[MS_NONFIN + t] = 1;
        red[t * 40 + (v >> 5)] = l1;
      }
    }
  }
  if (tid < n * 8) reinterpret_cast<uint32_t*>(xh + (tid >> 3) * XS + p.dpad)[tid & 7] = 0u;
  __syncthreads();
  FZ_STAMP(tid == 0, ST_X);
  // exponent E_t: |x| 2^-E < 2^22 for every element of token t
  auto token_exp = [&](int t) -> int {
    const float am = __int_as_float(misc[MS_AMAX + t]);
    if (!(am > 0.f) || misc[MS_NONFIN + t]) return 0;
    return max(int((__float_as_uint(am) >> 23) & 0xff) - 127 - 21, -100);
  };

  // ---- fixed-point limbs of two tokens in tensor-core operand order; group sums; truncation residual ----
  // A thread takes 8 channels = half of a 16-channel unit; the two halves meet through one shuffle.  X = round(x 2^-E)
  // is pre-scaled by 4^(3 - channel mod 4) (the predictor masks code fields in place, which weights them by 4^field)
  // and split into four signed base-256 digits.
  auto build_limbs = [&](int t0, int ptid, int nthreads) {
    const int ntk = min(2, n - t0);
    constexpr int lpg = G / 8;                                        // lanes per predictor group
    constexpr int g_log2 = G == 64 ? 6 : 7;
    const bool odd = lane & 1;
    for (int base = 0; base < ntk * nv; base += nthreads) {
      const int i = base + ptid;
      if (i >= ntk * nv) break;                                       // uniform over a warp
      const int tl = i / nv, v = i - tl * nv, t = t0 + tl;
      const int E = token_exp(t);
      const bool dead = misc[MS_NONFIN + t] != 0;
      const float inv = __uint_as_float(uint32_t(127 - E) << 23);    // 2^-E
      float f[8];
      unpack8(f, *reinterpret_cast<const uint4*>(xh + t * XS + v * 8));
      uint32_t D[8];
      int sx = 0;
      float resid = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float s = dead ? 0.f : f[c] * inv;
        const float r = s + 12582912.f;                         // 1.5 * 2^23: rounds s to an integer (|s| < 2^22)
        const int X = __float_as_int(r) - 0x4B400000;
        resid += fabsf(s - (r - 12582912.f));
        sx += X;
        // signed base-256 digits of X 4^(3-f): adding 0x80 to the three low bytes and flipping
        // those bits back leaves byte l = digit l as a signed 8-bit value
        const uint32_t Y = uint32_t(X) << (2 * (3 - (c & 3)));
        D[c] = (Y + 0x00808080u) ^ 0x00808080u;
      }
      // H[l][q]: 16-bit pairs (digit l of channels f, 4+f) for f = 2q (low half) and 2q+1 (high half)
      uint32_t H[4][2];
#pragma unroll
      for (int l = 0; l < 4; ++l)
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const uint32_t h0 = __byte_perm(D[2 * q], D[4 + 2 * q], 0x0040 + l * 0x0011);
          const uint32_t h1 = __byte_perm(D[2 * q + 1], D[5 + 2 * q], 0x0040 + l * 0x0011);
          H[l][q] = __byte_perm(h0, h1, 0x5410);
        }
      // the even thread of a pair stores limbs 0,1 and the odd one limbs 2,3
      uint32_t mine[2][2], theirs[2][2];
#pragma unroll
      for (int li = 0; li < 2; ++li)
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          mine[li][q] = odd ? H[2 + li][q] : H[li][q];
          const uint32_t send = odd ? H[li][q] : H[2 + li][q];
          theirs[li][q] = __shfl_xor_sync(0xffffffffu, send, 1);
        }
      {
        const int u = v >> 1, kb = u >> 2, tt = u & 3;
#pragma unroll
        for (int li = 0; li < 2; ++li) {
          const int l = (odd ? 2 : 0) + li;
          uint32_t wv[4];   // word f: byte i = digit l of channel 4 i + f (even thread: i = 0,1; odd: i = 2,3)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const uint32_t lo = odd ? theirs[li][q] : mine[li][q], hi = odd ? mine[li][q] : theirs[li][q];
            wv[2 * q] = __byte_perm(lo, hi, 0x5410);
            wv[2 * q + 1] = __byte_perm(lo, hi, 0x7632);
          }
          *reinterpret_cast<uint4*>(xq + size_t(tl * 4 + l) * xq_stride + size_t(kb) * 64 + tt * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
      // group sums of the integer x (exact); stored as 64 sum = hi 65536 + lo for the two halves of the limbs
#pragma unroll
      for (int o = 1; o < lpg; o <<= 1) sx += __shfl_xor_sync(0xffffffffu, sx, o);
      if ((lane & (lpg - 1)) == 0) {
        const long long S = 64ll * sx;
        sx2[tl * (p.ngroups + 16) + ((v * 8) >> g_log2)] = make_int2(int(S & 0xffff), int(S >> 16));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) resid += __shfl_xor_sync(0xffffffffu, resid, o);
      if (lane == 0) red[(n + t) * 40 + (v >> 5)] = resid;
    }
  };
  build_limbs(0, tid, NTH);
  FZ_STAMP(tid == 0, ST_LIMBS);

  // ---- speculative folded product on the tensor cores (warps NWP..NW-1) ----
  // The folded matrix is stored in units of 16 outputs x 256 channels (8 KB, contiguous, already in A-fragment
  // order), unit u = (output tile u / nkc, channel chunk u % nkc).  A warp draws units from one global ticket
  // (one draw ahead), streams a unit as four blocks of four 128-bit loads per lane (one block ahead of the one
  // being multiplied), multiplies it with x (the B operand: column t = token t, other columns zero) in two
  // independent accumulators, and adds the 16 x n partial outputs to the accumulator replica of its CTA.
  float* const rep = p.yacc + size_t(blockIdx.x % NREP) * MAXT * p.dacc;
  auto stream_c = [&]() {
    unsigned int* ticket = p.ctl + CTL_TICKET;
    auto issue = [&]() -> unsigned int {        // lane 0 draws; the value is looked at one unit later
      unsigned int t = 0;
      if (lane == 0) t = atomicAdd(ticket, 1u);
      return t;
    };
    auto resolve = [&](unsigned int raw) -> int {
      const unsigned int t = __shfl_sync(0xffffffffu, raw, 0);
      return t < (unsigned int)p.nunits ? int(t) : -1;
    };
    // lanes of column g < n read token g, the others the zeros behind token 0
    const __nv_bfloat16* const xrow = g < n ? xh + g * XS + t4 * 16 : xh + p.dpad;
    const int xstep = g < n ? 8 : 0;                    // uint4 per 64-channel block
    const int xchunk = g < n ? KC : 0;                  // elements per channel chunk
    auto load = [&](uint4 (&buf)[4], int u, int bi) {
      const uint4* src = p.Cp + size_t(u) * 512 + lane + bi * 128;
#pragma unroll
      for (int m = 0; m < 4; ++m) buf[m] = ldg_stream(src + m * 32);
    };
    auto multiply = [&](float (&c)[2][4], const uint4 (&buf)[4], const uint4* xp, int bi) {
      const uint4 x0 = xp[bi * xstep], x1 = xp[bi * xstep + 1];
      mma_bf16(c[0], buf[0].x, buf[0].y, buf[0].z, buf[0].w, x0.x, x0.y);
      mma_bf16(c[1], buf[1].x, buf[1].y, buf[1].z, buf[1].w, x0.z, x0.w);
      mma_bf16(c[0], buf[2].x, buf[2].y, buf[2].z, buf[2].w, x1.x, x1.y);
      mma_bf16(c[1], buf[3].x, buf[3].y, buf[3].z, buf[3].w, x1.z, x1.w);
    };
    uint4 ba[4], bb[4];
    int u = resolve(issue());
    bool more = u >= 0;
    unsigned int raw = more ? issue() : 0xffffffffu;
    if (u >= 0) load(ba, u, 0);
    while (u >= 0) {
      const int it = u / p.nkc, kc = u - it * p.nkc;
      const uint4* xp = reinterpret_cast<const uint4*>(xrow + kc * xchunk);
      float c[2][4];
#pragma unroll
      for (int m = 0; m < 2; ++m) c[m][0] = c[m][1] = c[m][2] = c[m][3] = 0.f;
      load(bb, u, 1);
      multiply(c, ba, xp, 0);
      load(ba, u, 2);
      multiply(c, bb, xp, 1);
      load(bb, u, 3);
      multiply(c, ba, xp, 2);
      const int nx = more ? resolve(raw) : -1;        // the next unit: its first block goes in flight now
      more = nx >= 0;
      raw = more ? issue() : 0xffffffffu;
      if (nx >= 0) load(ba, nx, 0);
      multiply(c, bb, xp, 3);
      if (p.dpart) {                                    // deterministic mode: the unit's sums have a place of their own
        float* const o = p.dpart + size_t(kc) * MAXT * p.dacc + it * 16 + g;
        if (2 * t4 < n) { o[(2 * t4) * p.dacc] = c[0][0] + c[1][0]; o[(2 * t4) * p.dacc + 8] = c[0][2] + c[1][2]; }
        if (2 * t4 + 1 < n) { o[(2 * t4 + 1) * p.dacc] = c[0][1] + c[1][1]; o[(2 * t4 + 1) * p.dacc + 8] = c[0][3] + c[1][3]; }
      } else {
        if (2 * t4 < n) {
          red_add_f32(rep + (2 * t4) * p.dacc + it * 16 + g, c[0][0] + c[1][0]);
          red_add_f32(rep + (2 * t4) * p.dacc + it * 16 + g + 8, c[0][2] + c[1][2]);
        }
        if (2 * t4 + 1 < n) {
          red_add_f32(rep + (2 * t4 + 1) * p.dacc + it * 16 + g, c[0][1] + c[1][1]);
          red_add_f32(rep + (2 * t4 + 1) * p.dacc + it * 16 + g + 8, c[0][3] + c[1][3]);
        }
      }
      u = nx;
    }
  };

  // ---- roles ----
  // The limbs are complete once all 32 warps have passed here.  The streaming warps only announce their part
  // (bar.arrive) and go on to the folded product, which needs nothing but x; the predictor warps wait for
  // everybody's limbs (bar.sync).  Both meet again before the result fixing.
  if (warp >= NWP) {
    asm volatile("bar.arrive 1, %0;" ::"n"(NTH) : "memory");
    stream_c();
    FZ_STAMP(tid == NTP, ST_STREAM);
  } else {
    asm volatile("bar.sync 1, %0;" ::"n"(NTH) : "memory");
    // ---- predictor: two tokens per pass; within tile u the warp takes the 128-channel pairs with
    //      (u npairs + pair) mod NWP = warp, so that the pairs of all tiles spread evenly ----
    constexpr int GPC = KC / G;                              // groups per chunk: 4 or 2
    const int npairs = p.nkc * 2;
    const double smax = double(smax_f);
    int q = 0;                                               // units consumed so far (over all passes)
    for (int pass = 0; pass < NP; ++pass) {
      const int t0 = pass * 2, ntk = min(2, n - t0);
      if (pass > 0) {                                        // limbs of the next two tokens replace the old ones
        bar_sync_pred();
        build_limbs(t0, tid, NTP);
        bar_sync_pred();
      }
      // operand side: column g = limb g & 3 of token t0 + (g >> 2); columns of a missing token read zeros
      const bool bcol = (g >> 2) < ntk;
      const uint8_t* const xql = bcol ? xq + size_t(g) * xq_stride + t4 * 16 : smem + L.zeros + t4 * 16;
      const int xon = bcol ? 1 : 0;
      // result side: this lane holds limbs 2 (t4 & 1), 2 (t4 & 1) + 1 of token t0 + (t4 >> 1)
      const int* const sxl = reinterpret_cast<const int*>(sx2 + (t4 >> 1) * (p.ngroups + 16)) + (t4 & 1);
      // one item: 128 channels (pair) x the 16 neurons of a tile.  A group done: integer sums (exact) -> minus zero-point
      // times the sum of x -> times the bf16 scale, accumulated in fp32 (rows g and g + 8 of the tile)
      auto item = [&](const uint8_t* ubase, int pair, const uint4& xb0, const uint4& xb1, int sxa, int sxb, float& fa0, float& fa1) {
        const int kc = pair >> 1, half = pair & 1;
        const uint8_t* const blk = ubase + kc * p.pbs;
        const uint4 cw = reinterpret_cast<const uint4*>(blk)[half * 32 + lane];
        const uint2* const mp = reinterpret_cast<const uint2*>(blk + 1024) + g;
        auto scale_group = [&](const int (&ia)[4], int gl, int sx) {
          const uint2 mw = mp[gl * 8];
          const int w0 = ia[0] + (ia[1] << 8) - int(mw.x & 3u) * sx;
          const int w1 = ia[2] + (ia[3] << 8) - int(mw.y & 3u) * sx;
          fa0 = fmaf(__uint_as_float(mw.x & 0xffff0000u), float(w0), fa0);
          fa1 = fmaf(__uint_as_float(mw.y & 0xffff0000u), float(w1), fa1);
        };
        int qa[4], qb[4];
        mma_u8s8_z(qa, cw.x & 0x03030303u, cw.y & 0x03030303u, cw.x & 0x0C0C0C0Cu, cw.y & 0x0C0C0C0Cu, xb0.x, xb0.y);
        mma_u8s8_z(qb, cw.z & 0x03030303u, cw.w & 0x03030303u, cw.z & 0x0C0C0C0Cu, cw.w & 0x0C0C0C0Cu, xb1.x, xb1.y);
        mma_u8s8(qa, cw.x & 0x30303030u, cw.y & 0x30303030u, cw.x & 0xC0C0C0C0u, cw.y & 0xC0C0C0C0u, xb0.z, xb0.w);
        mma_u8s8(qb, cw.z & 0x30303030u, cw.w & 0x30303030u, cw.z & 0xC0C0C0C0u, cw.w & 0xC0C0C0C0u, xb1.z, xb1.w);
        if (G == 64) {
          scale_group(qa, half * 2, sxa);
          scale_group(qb, half * 2 + 1, sxb);
        } else {                                          // G == 128: one group
#pragma unroll
          for (int e = 0; e < 4; ++e) qa[e] += qb[e];
          scale_group(qa, half, sxa);
        }
      };
      // limbs 2,3 (odd t4) weigh 65536 times limbs 0,1; lanes t4 = 0 / 2 store the partial score of token 0 / 1
      auto store_partial = [&](int u, float fa0, float fa1) {
        const float o0 = __shfl_xor_sync(0xffffffffu, fa0, 1), o1 = __shfl_xor_sync(0xffffffffu, fa1, 1);
        if (!(t4 & 1) && (t4 >> 1) < L.ztok) {
          float* zp = zpart + size_t((u * NWP + warp) * L.ztok + (t4 >> 1)) * 16;
          zp[g] = fmaf(65536.f, o0, fa0);
          zp[g + 8] = fmaf(65536.f, o1, fa1);
        }
      };
      auto wait_unit = [&](int b, uint32_t par) -> bool {
        bool landed = mbar_wait_warp(&full[b], par);
        if (!landed) {                                 // record, give the copy one more bounded wait, skip the work
          if (lane == 0) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ERR] = 1; }
          landed = mbar_wait_warp(&full[b], par);
        }
        return landed && !misc[MS_ERR];
      };
      auto load_x = [&](int pair, uint4& xb0, uint4& xb1, int& sxa, int& sxb) {
        const int kc = pair >> 1, half = pair & 1;
        const uint4* const xp = reinterpret_cast<const uint4*>(xql + (kc * KC + half * 128) * xon);
        xb0 = xp[0]; xb1 = xp[4 * xon];
        const int grp = G == 64 ? kc * GPC + half * 2 : kc * GPC + half;
        sxa = sxl[grp * 2];
        sxb = G == 64 ? sxl[(grp + 1) * 2] : 0;
      };
      if (FAST) {
        // every tile is in shared memory behind one barrier, and a warp has the same one or two pairs in every tile:
        // their x operands stay in registers; pairs beyond 2 NWP (fewer than NWP of them) go round the warps from tile to tile
        // (only rows longer than 16 chunks, CT > 8, have such pairs: the loop over them folds away otherwise)
        const bool two = npairs >= 2 * NWP;
        const int extra = (CT > 8 && two) ? npairs - 2 * NWP : 0;
        const bool usable = wait_unit(0, 0u);
        uint4 xa0, xa1, xc0 = make_uint4(0u, 0u, 0u, 0u), xc1 = xc0;
        int sa0, sa1, sc0 = 0, sc1 = 0;
        load_x(warp, xa0, xa1, sa0, sa1);
        if (two) load_x(warp + NWP, xc0, xc1, sc0, sc1);
        for (int u = 0; u < NU && usable; ++u) {
          const uint8_t* const ubase = pbuf + size_t(u) * p.buf_bytes;
          float fa0 = 0.f, fa1 = 0.f, fc0 = 0.f, fc1 = 0.f;
          item(ubase, warp, xa0, xa1, sa0, sa1, fa0, fa1);
          if (two) item(ubase, warp + NWP, xc0, xc1, sc0, sc1, fc0, fc1);
          for (int e = 0; CT > 8 && e < extra; ++e)
            if ((u * extra + e) % NWP == warp) {
              uint4 xb0, xb1;
              int sxa, sxb;
              load_x(2 * NWP + e, xb0, xb1, sxa, sxb);
              item(ubase, 2 * NWP + e, xb0, xb1, sxa, sxb, fc0, fc1);
            }
          store_partial(u, fa0 + fc0, fa1 + fc1);
        }
        q += NU;
      } else {
        // within tile u the warp takes the pairs with (u npairs + pair) mod NWP = warp, so that the pairs of all tiles
        // spread evenly over the warps
        for (int u = 0; u < NU; ++u, ++q) {
          const int b = resident ? 0 : q % p.nbuf;
          const bool usable = wait_unit(b, resident ? 0u : uint32_t((q / p.nbuf) & 1));
          const uint8_t* const ubase = pbuf + size_t(resident ? u : b) * p.buf_bytes;
          float fa0 = 0.f, fa1 = 0.f;
          int first = (warp - u * npairs) % NWP;
          if (first < 0) first += NWP;
          for (int pair = first; pair < npairs && usable; pair += NWP) {
            uint4 xb0, xb1;
            int sxa, sxb;
            load_x(pair, xb0, xb1, sxa, sxb);
            item(ubase, pair, xb0, xb1, sxa, sxb, fa0, fa1);
          }
          store_partial(u, fa0, fa1);
          // hand the buffer back: the last warp to leave it starts the copy of the unit that reuses it
          if (!resident && q + p.nbuf < NQ) {
            __threadfence_block();
            __syncwarp();
            if (lane == 0) {
              const int old = atomicAdd(const_cast<int*>(&misc[MS_BUFCNT + b]), 1);
              if (old == NWP - 1) {
                misc[MS_BUFCNT + b] = 0;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                issue_unit((q + p.nbuf) % NU, b);
              }
            }
          }
        }
      }
      bar_sync_pred();
      FZ_STAMP(tid == 0 && pass == 0, ST_PRED);
      // ---- scores and flags of this pass ----
      // tau bounds what the fast score can be off by: the rounding residuals of x (each at most 1/2 unit of 2^E)
      // times |code - zero| <= 3 times the scale, plus the fp32 roundings (one per conversion, product-sum and
      // combination: at most 12 per partial score, each at most 2^-24 of 3 smax sum |x|).
      if (tid < ntk * nrow) {
        const int tl = tid / nrow, r = tid - tl * nrow, t = t0 + tl;
        const int tile = r >> 4, rr = r & 15;
        const int j = plan.x * 16 + r;
        const int E = token_exp(t);
        float rs = 0.f, l1 = 0.f;
        for (int w = 0; w < (nv >> 5); ++w) { l1 += red[t * 40 + w]; rs += red[(n + t) * 40 + w]; }
        const double unit = __longlong_as_double((long long)(1023 + E) << 52);   // 2^E
        const double tau = 1.01 * 3.0 * smax * (double(rs) * unit + 12.0 * 5.9604644775390625e-08 * (double(l1) + double(rs) * unit));
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < NWP; ++w) s += double(zpart[size_t((tile * NWP + w) * L.ztok + tl) * 16 + rr]);
        const double b1 = double(tab[2 * TR + r]);
        double zhat = b1 + s * (unit * 0.015625);
        const double lo = double(tab[r]), hi = double(tab[TR + r]);
        int f = ((lo <= zhat) && (zhat < hi)) ? 0 : 1;
        if (misc[MS_NONFIN + t]) { f = 1; zhat = __longlong_as_double(0x7ff8000000000000ll); }
        else if (fabs(zhat - lo) <= tau || fabs(zhat - hi) <= tau) {
          const int e = atomicAdd(const_cast<int*>(&misc[MS_NRC]), 1);
          if (e < MAXRC) { rc[e] = (tl << 16) | r; f = -1; }
          else {                                        // list full: this thread re-evaluates its neuron alone
            const int qu = pass * NU + tile;            // the tile's blocks are still in shared memory unless its buffer was refilled
            const bool here = resident || qu + p.nbuf >= NQ;
            zhat = b1 + (here ? exact_from_blocks(pbuf + size_t(resident ? tile : qu % p.nbuf) * p.buf_bytes, p.pbs, G, rr, xh + t * XS, d, 0, 1)
                              : exact_score_single(p.codes, p.scale, p.zero, xh + t * XS, j, d, G, 2));
            f = ((lo <= zhat) && (zhat < hi)) ? 0 : 1;
          }
        }
        if (f > 0) atomicOr(&flagbits[r], 1 << t);
        if (p.dbg_scores && f >= 0) p.dbg_scores[size_t(t) * p.h + j] = zhat;
      }
      bar_sync_pred();
      // exact re-evaluation from the original codes (rare): one warp per listed (token, neuron)
      {
        const int nrc = min(int(misc[MS_NRC]), MAXRC);
        for (int e = warp; e < nrc; e += NWP) {
          const int tl = rc[e] >> 16, r = rc[e] & 0xffff, t = t0 + tl;
          const int j = plan.x * 16 + r;
          double ex;
          const int qu = pass * NU + (r >> 4);
          if (resident || qu + p.nbuf >= NQ) {  // the tile's blocks are still in shared memory (its buffer was not refilled)
            ex = exact_from_blocks(pbuf + size_t(resident ? (r >> 4) : qu % p.nbuf) * p.buf_bytes, p.pbs, G, r & 15, xh + t * XS, d, lane, 32);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ex += __shfl_xor_sync(0xffffffffu, ex, o);
          } else {
            ex = exact_score(p.codes, p.scale, p.zero, xh + t * XS, j, d, G, 2, lane);
          }
          const double zhat = double(tab[2 * TR + r]) + ex;
          if (lane == 0) {
            if (!((double(tab[r]) <= zhat) && (zhat < double(tab[TR + r])))) atomicOr(&flagbits[r], 1 << t);
            if (p.dbg_scores) p.dbg_scores[size_t(t) * p.h + j] = zhat;
          }
        }
        if (nrc > 0) {                                  // (uniform over the predictor warps)
          bar_sync_pred();
          if (tid == 0) {
            atomicAdd(&p.counters[CTR_RECHECKS], (unsigned long long)nrc);
            misc[MS_NRC] = 0;
          }
        }
      }
    }
    // ---- ascending list of the neurons flagged by any token: ballot + prefix over the warps that hold rows ----
    {
      const int fb = (tid < nrow) ? flagbits[tid] : 0;
      const uint32_t bal = __ballot_sync(0xffffffffu, fb != 0);
      if (lane == 0 && warp < 8) misc[MS_WCNT + warp] = __popc(bal);
      for (int t = 0; t < n; ++t) {
        const uint32_t bt = __ballot_sync(0xffffffffu, (fb >> t) & 1);
        if (lane == 0 && bt) atomicAdd(const_cast<int*>(&misc[MS_TOKCNT + t]), __popc(bt));
        // debug capture: 16-bit halves of the flag words
        if (p.dbg_bitmap && tid < nrow && (tid & 15) == 0)
          reinterpret_cast<uint16_t*>(p.dbg_bitmap + size_t(t) * (p.h / 32))[plan.x + (tid >> 4)] = uint16_t((bt >> (lane & 16)) & 0xffffu);
      }
      bar_sync_pred();
      int base = 0, total = 0;
#pragma unroll
      for (int w = 0; w < 8; ++w) { const int cnt = misc[MS_WCNT + w]; if (w < warp) base += cnt; total += cnt; }
      if (fb) {
        const int pos = base + __popc(bal & ((1u << lane) - 1u));
        fl_j[pos] = plan.x * 16 + tid;
        fl_mask[pos] = fb;
      }
      if (tid == 0) {
        misc[MS_NUN] = total;
        for (int t = 0; t < n; ++t)
          if (misc[MS_TOKCNT + t]) atomicAdd(&p.ctl[CTL_NFL + t], (unsigned int)misc[MS_TOKCNT + t]);
        if (total) atomicAdd(&p.ctl[CTL_UNION], (unsigned int)total);
      }
      bar_sync_pred();
    }
    FZ_STAMP(tid == 0, ST_FLAGS);
  }

  // ---- result fixing ----
  // Everything from pbuf to the end of the CTA's shared memory is free now and becomes row slots (slot_stride
  // bytes apart: a row plus 16 bytes, so that the 8 rows of an ldmatrix tile fall into different banks).  The
  // W1 rows of the listed neurons come first, GS <= 8 per step, then their W2^T rows; a step fills one slot group
  // with one barrier, NG groups are in flight, step s uses group s mod NG.
  uint64_t* const fixbar = &full[MAXBUF];
  const uint32_t rowbytes = uint32_t(d) * 2u;
  uint8_t* const slots = smem + L.pbuf;
  const int nslots = int((L.slots_end - L.pbuf) / size_t(p.slot_stride));
  // (two groups: with three or four, more rows are asked for at once and the rows needed first arrive later; measured)
  const int NG = 2;
  const int GS = min(p.gs_cap, nslots / NG);
  // fills the group of step st: warp `issuer` arms the barrier and its lanes issue one copy each
  auto fill = [&](int st, int nun, int issuer) {
    const int nA = (nun + GS - 1) / GS;                             // steps over W1 rows (as many again over W2^T rows)
    if (st >= 2 * nA || warp != issuer) return;
    const bool second = st >= nA;
    const int i0 = (second ? st - nA : st) * GS, cnt = min(GS, nun - i0);
    const int gr = st % NG;
    if (lane == 0) mbar_expect_tx(&fixbar[gr], uint32_t(cnt) * rowbytes);
    __syncwarp();
    if (lane < cnt) {
      const __nv_bfloat16* src = (second ? p.W2T : p.W1) + size_t(fl_j[i0 + lane]) * d;
      bulk_g2s(slots + size_t(gr * GS + lane) * p.slot_stride, src, rowbytes, &fixbar[gr]);
    }
  };
  auto wait_group = [&](int st) -> bool {
    const int gr = st % NG;
    const uint32_t par = uint32_t((st / NG) & 1);
    bool landed = mbar_wait_warp(&fixbar[gr], par);
    if (!landed) {
      if (lane == 0) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ERR] = 1; }
      landed = mbar_wait_warp(&fixbar[gr], par);
    }
    return landed;
  };
  // the predictor warps start the first copies on their own: the streaming warps may still be busy.  Only W1 rows
  // go out here: the pre-activations are needed first, and W2^T rows asked for at the same moment would share the
  // memory system with them
  if (warp < NWP) {
    const int nun = misc[MS_NUN];
    const int nA0 = (nun + GS - 1) / GS;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the region was read with ordinary loads
    for (int st = 0; st < NG && st < nA0; ++st) fill(st, nun, st);
  }
  __syncthreads();
  const int nun = misc[MS_NUN];
  const int nA = (nun + GS - 1) / GS;
  if (nA < NG) {                                                    // slot groups left over: the first W2^T rows follow
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int st = nA; st < NG; ++st) fill(st, nun, NW - 1 - st);
  }
  const int nks = d >> 4;                                           // 16-channel steps of a row (= 16-column tiles of an output)
  FZ_STAMP_VALUE(tid == 0, ST_NFL, nun);
  // -- pre-activations and deltas: steps over the W1 rows, as many at a time as there are buffers of partial sums (NG at most) --
  {
    // x as the B operand (column g = token g): the warp's k-steps are the same in every step, so their operands are
    // loaded once
    uint32_t xb0[CT], xb1[CT];
    {
      const __nv_bfloat16* const xb = g < n ? xh + g * XS + 2 * t4 : reinterpret_cast<const __nv_bfloat16*>(smem + L.zeros);
      const int xbs = g < n ? 16 : 0;
#pragma unroll
      for (int e = 0; e < CT; ++e) {
        const int ks = warp + e * NW;
        xb0[e] = xb1[e] = 0u;
        if (ks < nks) {
          xb0[e] = *reinterpret_cast<const uint32_t*>(xb + ks * xbs);
          xb1[e] = *reinterpret_cast<const uint32_t*>(xb + ks * xbs + (xbs >> 1));
        }
      }
    }
    const int wzstride = p.gs_cap * n * 33;                         // floats per buffer of partial sums
    const int NCH = min(NG, L.wz_groups);                           // steps summed up together
    for (int c0 = 0; c0 < nA; c0 += NCH) {
      const int c1 = min(nA, c0 + NCH);
      for (int st = c0; st < c1; ++st) {
        const int nw1 = min(GS, nun - st * GS);
        const bool landed = wait_group(st);
        const uint32_t gbase = smem_u32(slots + size_t((st % NG) * GS) * p.slot_stride);
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (NTK == 1) {
          // A operand = up to 16 W1 rows x 16 channels: lanes 0..7 address rows 0..7, lanes 8..15 rows 8..15 (channels 0..7 of the
          // step), lanes 16..31 the same rows at channels 8..15; a row the step does not have reads the step's last row instead
          // (its sums are not used)
          const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8;
          const uint32_t abase = gbase + uint32_t(min(a_row, nw1 - 1)) * p.slot_stride + ((lane >> 4) & 1) * 16 + warp * 32;
  #pragma unroll
          for (int e2 = 0; e2 < CT; e2 += 2) {                        // two tiles in flight
            uint32_t a0[2], a1[2], a2[2], a3[2];
  #pragma unroll
            for (int e = 0; e < 2; ++e)
              if (e2 + e < CT && warp + (e2 + e) * NW < nks && landed) ldmatrix_x4(a0[e], a1[e], a2[e], a3[e], abase + (e2 + e) * (NW * 32));
  #pragma unroll
            for (int e = 0; e < 2; ++e)
              if (e2 + e < CT && warp + (e2 + e) * NW < nks && landed) mma_bf16(c, a0[e], a1[e], a2[e], a3[e], xb0[e2 + e], xb1[e2 + e]);
          }
          // the partial sum of (row, token) pair q = n row + token goes to [33 q + warp]: stores and loads without bank conflicts
          // (c[0], c[1]: row g; c[2], c[3]: row g + 8)
          float* const wzs = wz + size_t(st - c0) * wzstride;
          const bool upper = g + 8 < GS;                              // (a buffer holds the sums of GS rows)
          if (2 * t4 < n) { wzs[(n * g + 2 * t4) * 33 + warp] = c[0]; if (upper) wzs[(n * (g + 8) + 2 * t4) * 33 + warp] = c[2]; }
          if (2 * t4 + 1 < n) { wzs[(n * g + 2 * t4 + 1) * 33 + warp] = c[1]; if (upper) wzs[(n * (g + 8) + 2 * t4 + 1) * 33 + warp] = c[3]; }
        } else {
          // only rows 0..7 of the MMA tile are in use: lane l < 16 gives ldmatrix row l & 7, channels + 8 (l >> 3)
          const uint32_t abase = gbase + uint32_t(min(lane & 7, nw1 - 1)) * p.slot_stride + ((lane >> 3) & 1) * 16 + warp * 32;
  #pragma unroll
          for (int e2 = 0; e2 < CT; e2 += 2) {                        // two tiles in flight
            uint32_t a0[2], a2[2];
  #pragma unroll
            for (int e = 0; e < 2; ++e)
              if (e2 + e < CT && warp + (e2 + e) * NW < nks && landed) ldmatrix_x2(a0[e], a2[e], abase + (e2 + e) * (NW * 32));
  #pragma unroll
            for (int e = 0; e < 2; ++e)
              if (e2 + e < CT && warp + (e2 + e) * NW < nks && landed) mma_bf16(c, a0[e], 0u, a2[e], 0u, xb0[e2 + e], xb1[e2 + e]);
          }
          // the partial sum of (row, token) pair q = n row + token goes to [33 q + warp]: stores and loads without bank conflicts
          float* const wzs = wz + size_t(st - c0) * wzstride;
          if (2 * t4 < n) wzs[(n * g + 2 * t4) * 33 + warp] = c[0];
          if (2 * t4 + 1 < n) wzs[(n * g + 2 * t4 + 1) * 33 + warp] = c[1];
        }
      }
      __syncthreads();                                              // partial sums complete; the rows are used
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      for (int st = c0; st < c1; ++st) fill(st + NG, nun, NW - 1 - (st - c0));
      // a warp adds up the 32 partial sums of a pair (a fixed tree) and turns them into delta
      const int npair = (c1 - c0) * GS * n;
      for (int pq = warp; pq < npair; pq += NW) {
        const int sl = pq / (GS * n), q = pq - sl * (GS * n), row = q / n, t = q - row * n;
        const int idx = (c0 + sl) * GS + row;
        if (idx < nun) {
          float z = wz[size_t(sl) * wzstride + q * 33 + lane];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
          if (lane == 0) {
            float dl = 0.f;
            if ((fl_mask[idx] >> t) & 1) {
              const int r = fl_j[idx] - plan.x * 16;
              z += tab[2 * TR + r];
              dl = gelu_f32(z, p.act) - tab[3 * TR + r] * z - tab[4 * TR + r];
            }
            fl_delta[idx * MAXT + t] = dl;
          }
        }
      }
      if (c1 < nA) __syncthreads();                                 // the partial sums are read before the next steps overwrite them
    }
  }
  __syncthreads();                                                  // every delta is in place
  // -- outputs: steps over the W2^T rows; the accumulators of all output columns stay in registers --
  float acc[CT][4];
#pragma unroll
  for (int ci = 0; ci < CT; ++ci) acc[ci][0] = acc[ci][1] = acc[ci][2] = acc[ci][3] = 0.f;
  {
    // W2^T tiles (transposed on load), 16 output columns x the neurons of the step.  Calls of one token (steps of up to 16
    // neurons): lanes 0..7 address neurons 0..7 at columns 0..7, lanes 8..15 the same neurons at columns 8..15, lanes 16..31
    // neurons 8..15 likewise.  Calls of several tokens (steps of up to 8 neurons): lanes 0..15 only, the other half of the
    // operand is zero.
    constexpr bool WIDE = NTK == 1;
    const int w2_row = (lane & 7) + (WIDE ? ((lane >> 4) & 1) * 8 : 0), w2_cofs = ((lane >> 3) & 1) * 8;
    for (int st = nA; st < 2 * nA; ++st) {
      const int l0 = (st - nA) * GS, nw2 = min(GS, nun - l0);
      const bool landed = wait_group(st);
      const uint32_t gbase = smem_u32(slots + size_t((st % NG) * GS) * p.slot_stride);
      // B operand: delta of the step's neurons (k = neuron), columns 0..3 the leading bf16 term of tokens 0..3, columns 4..7 the
      // rest; b0 holds neurons 2 t4, 2 t4 + 1, b1 neurons 2 t4 + 8, 2 t4 + 9 (a neuron the step does not have counts as 0)
      float dv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int kk = 2 * t4 + (e & 1) + (e >> 1) * 8;
        const float v = ((WIDE || e < 2) && kk < nw2 && (g & 3) < n) ? fl_delta[(l0 + kk) * MAXT + (g & 3)] : 0.f;
        const float hi = __bfloat162float(__float2bfloat16_rn(v));
        dv[e] = (g >> 2) ? v - hi : hi;
      }
      const uint32_t b0 = pack_bf16(dv[0], dv[1]), b1 = WIDE ? pack_bf16(dv[2], dv[3]) : 0u;
      const uint32_t abase = gbase + uint32_t(min(w2_row, nw2 - 1)) * p.slot_stride + w2_cofs * 2;
#pragma unroll
      for (int ci = 0; ci < CT; ++ci) {
        if (warp + ci * NW < nks && landed) {
          uint32_t a0, a1, a2 = 0u, a3 = 0u;
          if constexpr (WIDE) ldmatrix_x4_trans(a0, a1, a2, a3, abase + (warp + ci * NW) * 32);
          else ldmatrix_x2_trans(a0, a1, abase + (warp + ci * NW) * 32);
          mma_bf16(acc[ci], a0, a1, a2, a3, b0, b1);
        }
      }
      if (st + NG < 2 * nA) {
        __syncthreads();                                            // rows used
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        fill(st + NG, nun, NW - 1);
      }
    }
  }
  // The accumulators hold 16 output columns x (leading | remaining term of 4 tokens) per tile: add the two terms,
  // stage the sums in shared memory (the row slots are free) and add them to this CTA's replica with 128-bit reductions.
  if (nun > 0 || p.dpart) {                                         // (deterministic mode: every CTA writes its part, zeros too)
    __syncthreads();
    float* const yst = reinterpret_cast<float*>(slots);           // [n][dpad]
#pragma unroll
    for (int ci = 0; ci < CT; ++ci) {
      const int ct = warp + ci * NW;
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = acc[ci][e] + __shfl_xor_sync(0xffffffffu, acc[ci][e], 2);
      if (ct * 16 < d && t4 < 2) {
        if (2 * t4 < n) { yst[(2 * t4) * p.dpad + ct * 16 + g] = v[0]; yst[(2 * t4) * p.dpad + ct * 16 + g + 8] = v[2]; }
        if (2 * t4 + 1 < n) { yst[(2 * t4 + 1) * p.dpad + ct * 16 + g] = v[1]; yst[(2 * t4 + 1) * p.dpad + ct * 16 + g + 8] = v[3]; }
      }
    }
    __syncthreads();
    const int nq = d >> 2;
    for (int i = tid; i < n * nq; i += NTH) {
      const int t = i / nq, v4 = i - t * nq;
      const float4 s = *reinterpret_cast<const float4*>(yst + t * p.dpad + v4 * 4);
      if (p.dpart) *reinterpret_cast<float4*>(p.dpart + (size_t(p.nkc + blockIdx.x) * MAXT + t) * p.dacc + v4 * 4) = s;
      else red_add_v4(rep + t * p.dacc + v4 * 4, s.x, s.y, s.z, s.w);
    }
  }
  FZ_STAMP(tid == 0, ST_FIXED);

  // Any warp of any CTA may have added to any column, so the columns are complete when the last CTA is:
  // the CTAs count themselves, and the last one turns the accumulator into y.
  __threadfence();
  __syncthreads();
  if (tid == 0) misc[MS_LAST] = int(atomicAdd(&p.ctl[CTL_DONE], 1u));
  __syncthreads();
  FZ_STAMP(tid == 0, ST_COUNTED);
  if (misc[MS_LAST] == int(gridDim.x) - 1) {
    __threadfence();
    for (int i = tid; i < (p.dpart ? 0 : n * p.nvec); i += NTH) {    // (deterministic mode: k_ordered_sum writes y)
      const int t = i / p.nvec, c0 = (i - t * p.nvec) * 8;
      float4 a0[NREP + 1], a1[NREP + 1];
      a0[NREP] = *reinterpret_cast<const float4*>(p.bf + c0);
      a1[NREP] = *reinterpret_cast<const float4*>(p.bf + c0 + 4);
#pragma unroll
      for (int rp = 0; rp < NREP; ++rp) {
        const float* q = p.yacc + (size_t(rp) * MAXT + t) * p.dacc + c0;
        a0[rp] = __ldcg(reinterpret_cast<const float4*>(q));
        a1[rp] = __ldcg(reinterpret_cast<const float4*>(q + 4));
      }
      float4 s0 = a0[NREP], s1 = a1[NREP];
#pragma unroll
      for (int rp = 0; rp < NREP; ++rp) {
        s0.x += a0[rp].x; s0.y += a0[rp].y; s0.z += a0[rp].z; s0.w += a0[rp].w;
        s1.x += a1[rp].x; s1.y += a1[rp].y; s1.z += a1[rp].z; s1.w += a1[rp].w;
        float* q = p.yacc + (size_t(rp) * MAXT + t) * p.dacc + c0;
        *reinterpret_cast<float4*>(q) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(q + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      __nv_bfloat162 o[4];
      o[0] = __floats2bfloat162_rn(s0.x, s0.y);
      o[1] = __floats2bfloat162_rn(s0.z, s0.w);
      o[2] = __floats2bfloat162_rn(s1.x, s1.y);
      o[3] = __floats2bfloat162_rn(s1.z, s1.w);
      *reinterpret_cast<uint4*>(p.y + size_t(t) * d + c0) = *reinterpret_cast<const uint4*>(o);
    }
    FZ_STAMP(tid == 0, ST_FINAL);
    if (tid == 0) {   // every CTA has arrived, so every CTA's counts are in
      p.ctl[CTL_TICKET] = 0u;
      p.ctl[CTL_DONE] = 0u;
      for (int t = 0; t < n; ++t) {
        const unsigned int tot = atomicExch(&p.ctl[CTL_NFL + t], 0u);
        atomicAdd(&p.counters[CTR_FLAGGED_TOTAL], (unsigned long long)tot);
        atomicMax(&p.counters[CTR_FLAGGED_MAX], (unsigned long long)tot);
      }
      p.counters[CTR_LAST_UNION] = (unsigned long long)atomicExch(&p.ctl[CTL_UNION], 0u);
    }
  }
}

// ---- set-up kernels --------------------------------------------------------------------------------------
// Predictor blocks: block (tile, kc) = 2 x 32 lanes x {A0,B0,A1,B1} code words (1 KB, in the order the lanes of the
// integer MMA read them) + per group {row g, row g+8} words: the bf16 scale in the upper half, the zero-point below.
__global__ void k_pack_pblocks(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                               const uint8_t* __restrict__ zero, uint8_t* __restrict__ out, int d, int G, int nkc, int pbs) {
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
    if (grp < ng)
      w = (uint32_t(__bfloat16_as_ushort(scale[size_t(row) * ng + grp])) << 16) | uint32_t(zero[size_t(row) * ng + grp] & 3u);
    reinterpret_cast<uint32_t*>(blk + 1024)[e] = w;
  }
}

// Folded matrix in A-fragment order of mma.m16n8k16 (bf16).  Unit (it, kc) = outputs 16 it .. 16 it + 15
// times channels 256 kc .. 256 kc + 255 = 4 blocks x 4 MMAs x 32 lanes x 16 bytes, contiguous; units are
// ordered it-major.  Register r of lane (g, t4) in MMA m of block bi holds W_f[16 it + g + 8 (r & 1)]
// [256 kc + 64 bi + 16 t4 + 4 m + 2 (r >> 1) + {0, 1}]: a lane's B operands for a block are then 16
// consecutive channels of x.  C is the fold's output, C[k][i] = W_f[i][k]; channels beyond d are zero.
__global__ void k_pack_folded(const __nv_bfloat16* __restrict__ C, uint4* __restrict__ out, int d, int nkc) {
  const int u = blockIdx.x, it = u / nkc, kc = u - it * nkc;
  for (int e = threadIdx.x; e < 16 * 32; e += blockDim.x) {
    const int bm = e >> 5, ln = e & 31, bi = bm >> 2, m = bm & 3, gg = ln >> 2, tt = ln & 3;
    uint32_t r[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int row = it * 16 + gg + ((q & 1) ? 8 : 0);
      const int k = kc * KC + bi * 64 + tt * 16 + m * 4 + ((q >> 1) ? 2 : 0);
      const uint32_t lo = (k < d) ? __bfloat16_as_ushort(C[size_t(k) * d + row]) : 0u;
      const uint32_t hi = (k + 1 < d) ? __bfloat16_as_ushort(C[size_t(k + 1) * d + row]) : 0u;
      r[q] = lo | (hi << 16);
    }
    out[size_t(u) * 512 + e] = make_uint4(r[0], r[1], r[2], r[3]);
  }
}

__global__ void k_max_scale(const __nv_bfloat16* __restrict__ scale, size_t count, float* out) {
  float m = 0.f;
  for (size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x; e < count; e += size_t(gridDim.x) * blockDim.x)
    m = fmaxf(m, fabsf(__bfloat162float(scale[e])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
}

}  // namespace fz

using namespace fz;

// Builds the state of this path for bf16 layers with 2-bit codes, group size 64 or 128 and d_model a multiple of 16
// up to 4608; other layers are left to the other kernels (H->fscratch stays null).
tardis_status_t fused_prepare(Handle* H, cudaStream_t s) {
  H->fscratch = nullptr;
  const int d = H->d, h = H->h, G = H->G;
  if (H->dtype != TARDIS_BF16 || H->bits != 2) return TARDIS_OK;
  if (!(G == 64 || G == 128)) return TARDIS_OK;
  const int NT = h / 16;
  const int dpad = (d + KC - 1) / KC * KC;
  if (d < 64 || d % 16 || dpad > 32 * 16 * CTMAX || h % 16) return TARDIS_OK;
  int max_smem = 0;
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, H->device));

  Scratch* S = new (std::nothrow) Scratch();
  if (!S) return TARDIS_ERR_ALLOC;
  memset(S, 0, sizeof(*S));
  Params& p = S->base;
  p.d = d; p.h = h; p.G = G; p.ngroups = H->ngroups; p.act = H->act;
  p.dpad = dpad; p.dacc = (d + 31) / 32 * 32;
  p.nkc = dpad / KC;
  p.pbs = 1024 + 64 * (KC / G);
  p.unit_bytes = p.nkc * p.pbs;
  p.nvec = d / 8;
  p.nunits = (d / 16) * p.nkc;
  p.slot_stride = dpad * 2 + 16;
  const int grid = H->num_sms < NT ? H->num_sms : NT;
  const int tiles_max = (NT + grid - 1) / grid;
  if (tiles_max > MAXTILES) { delete S; return TARDIS_OK; }
  // per number of tokens of a call: as many tile buffers as fit next to x (all tiles if possible).  The CTA takes all the
  // shared memory there is: what the predictor state leaves free holds row slots (and the output staging of the last step)
  for (int nt = 1; nt <= MAXT; ++nt) {
    const size_t need_slots = size_t(nt) * dpad * 4 > size_t(4) * p.slot_stride ? size_t(nt) * dpad * 4 : size_t(4) * p.slot_stride;
    S->nbuf_n[nt] = 0;
    // steps of up to 16 neurons need twice the room for partial sums: they give way where that room buys another tile buffer
    for (int nbuf = tiles_max < MAXBUF ? tiles_max : MAXBUF; nbuf >= 1 && S->nbuf_n[nt] == 0; --nbuf)
      for (int cap = nt == 1 ? MAXGS : 8; cap >= 8; cap -= 8) {   // (calls of several tokens: 8, measured)
        const SmemLayout L(dpad, p.ngroups, tiles_max, nbuf, p.unit_bytes, nt, size_t(max_smem), cap);
        if (L.pred_end <= size_t(max_smem) && L.wz_end <= size_t(max_smem) && L.slots_end - L.pbuf >= need_slots) {
          S->nbuf_n[nt] = nbuf; S->gs_cap_n[nt] = cap;
          break;
        }
      }
    if (S->nbuf_n[nt] == 0) { delete S; return TARDIS_OK; }
  }
  p.tiles_max = tiles_max; p.buf_bytes = p.unit_bytes; S->smem_bytes = size_t(max_smem); p.smem_total = max_smem;
  S->grid = grid;
  auto fail = [&](tardis_status_t st) { H->fscratch = S; fused_release(H); return st; };
  size_t tally = 0;
  const size_t pb_bytes = size_t(NT) * p.nkc * p.pbs;
  const size_t yacc_bytes = sizeof(float) * NREP * MAXT * p.dacc;
  const size_t cp_bytes = size_t(p.nunits) * 8192;
  cudaError_t e = dev_malloc(&S->pblocks, pb_bytes); tally += pb_bytes;
  if (e == cudaSuccess) { e = dev_malloc(&S->plan, sizeof(int2) * grid); tally += sizeof(int2) * grid; }
  if (e == cudaSuccess) { e = dev_malloc(&S->smax, 16); tally += 16; }
  if (e == cudaSuccess) { e = dev_malloc(&S->Cp, cp_bytes); tally += cp_bytes; }
  if (e == cudaSuccess) { e = dev_malloc(&S->yacc, yacc_bytes); tally += yacc_bytes; }
  if (e == cudaSuccess) { e = dev_malloc(&S->ctl, sizeof(unsigned int) * CTL_WORDS); tally += sizeof(unsigned int) * CTL_WORDS; }
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
  if (e == cudaSuccess) e = cudaMemsetAsync(S->yacc, 0, yacc_bytes, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(S->ctl, 0, sizeof(unsigned int) * CTL_WORDS, s);
  if (e != cudaSuccess) { set_last_error(e, "fused_prepare"); return fail(TARDIS_ERR_CUDA); }
  k_pack_pblocks<<<dim3(NT, p.nkc), 128, 0, s>>>(H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero,
                                                 S->pblocks, d, G, p.nkc, p.pbs);
  k_pack_folded<<<p.nunits, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->C), S->Cp, d, p.nkc);
  k_max_scale<<<64, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->scale), size_t(h) * H->ngroups, S->smax);
  e = cudaGetLastError();
  const bool wide = dpad > 32 * 16 * 8;
  // kernels[one token or more][ring or fast]
  if (G == 64 && wide) { S->kernels[0][0] = (const void*)k_fused<64, 9, 1, false>; S->kernels[0][1] = (const void*)k_fused<64, 9, 1, true>;
                         S->kernels[1][0] = (const void*)k_fused<64, 9, 4, false>; S->kernels[1][1] = (const void*)k_fused<64, 9, 4, true>; }
  else if (G == 64) { S->kernels[0][0] = (const void*)k_fused<64, 8, 1, false>; S->kernels[0][1] = (const void*)k_fused<64, 8, 1, true>;
                      S->kernels[1][0] = (const void*)k_fused<64, 8, 4, false>; S->kernels[1][1] = (const void*)k_fused<64, 8, 4, true>; }
  else if (wide) { S->kernels[0][0] = (const void*)k_fused<128, 9, 1, false>; S->kernels[0][1] = (const void*)k_fused<128, 9, 1, true>;
                   S->kernels[1][0] = (const void*)k_fused<128, 9, 4, false>; S->kernels[1][1] = (const void*)k_fused<128, 9, 4, true>; }
  else { S->kernels[0][0] = (const void*)k_fused<128, 8, 1, false>; S->kernels[0][1] = (const void*)k_fused<128, 8, 1, true>;
         S->kernels[1][0] = (const void*)k_fused<128, 8, 4, false>; S->kernels[1][1] = (const void*)k_fused<128, 8, 4, true>; }
  for (int a = 0; a < 2 && e == cudaSuccess; ++a)
    for (int b = 0; b < 2 && e == cudaSuccess; ++b)
      e = cudaFuncSetAttribute(S->kernels[a][b], cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
  S->pairs_fit = (p.nkc * 2 == NWP || (p.nkc * 2 >= 2 * NWP && p.nkc * 2 < 3 * NWP));
  if (e != cudaSuccess) { set_last_error(e, "fused_prepare launch"); return fail(TARDIS_ERR_CUDA); }

  p.pblocks = S->pblocks; p.plan = S->plan; p.smax = S->smax; p.yacc = S->yacc; p.ctl = S->ctl;
  p.W1 = static_cast<const __nv_bfloat16*>(H->W1); p.W2T = static_cast<const __nv_bfloat16*>(H->W2T);
  p.Cp = S->Cp; p.bf = H->bf; p.lo = H->lo; p.hi = H->hi; p.a = H->a; p.c = H->c; p.b1 = H->b1;
  p.codes = H->codes; p.scale = static_cast<const __nv_bfloat16*>(H->scale); p.zero = H->zero;
  p.counters = H->counters;
  H->fscratch = S;
  // beyond this many tokens the batched tensor-core path is faster (decode_7b: 208 against 212 us at 16 tokens, 245 against
  // 212 at 18; Falcon shape: 253 against 255 us at 13, 272 against 251 at 14)
  H->fused_max_tokens = dpad <= 4096 ? kDecodeMaxTokens : 13;
  H->bytes_scratch += S->bytes - pb_bytes - cp_bytes;
  H->bytes_predictor += pb_bytes;
  H->bytes_folded += cp_bytes;
  return TARDIS_OK;
}

// Deterministic mode: y[t][i] = b_f[i] + the partial outputs of the channel chunks and of the CTAs (parts 0 .. nparts - 1).
// A warp takes four columns of one token: lane l adds parts l, l + 32, ... in ascending order, the 32 lane sums meet
// in a fixed tree.  The same bits whenever the inputs are the same.
__global__ void k_ordered_sum(const float* __restrict__ dpart, const float* __restrict__ bf, __nv_bfloat16* __restrict__ y,
                              int n, int d, int dacc, int nparts) {
  const int nq = d >> 2;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (i >= n * nq) return;                              // (the same for the whole warp)
  const int t = i / nq, q = i - t * nq;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
  for (int part = lane; part < nparts; part += 32) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(dpart + (size_t(part) * fz::MAXT + t) * dacc + q * 4));
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s.x += __shfl_xor_sync(0xffffffffu, s.x, o); s.y += __shfl_xor_sync(0xffffffffu, s.y, o);
    s.z += __shfl_xor_sync(0xffffffffu, s.z, o); s.w += __shfl_xor_sync(0xffffffffu, s.w, o);
  }
  if (lane == 0) {
    const float4 b = *reinterpret_cast<const float4*>(bf + q * 4);
    __nv_bfloat162 o[2] = {__floats2bfloat162_rn(s.x + b.x, s.y + b.y), __floats2bfloat162_rn(s.z + b.z, s.w + b.w)};
    *reinterpret_cast<uint2*>(y + size_t(t) * d + q * 4) = *reinterpret_cast<const uint2*>(o);
  }
}

// Switches the order-independent accumulation of this path on or off; the partial-output buffer is allocated the first time.
tardis_status_t fused_set_deterministic(Handle* H, bool on) {
  Scratch* S = static_cast<Scratch*>(H->fscratch);
  if (!S) return TARDIS_OK;
  if (on && !S->dpart) {
    const size_t bytes = size_t(S->base.nkc + S->grid) * MAXT * S->base.dacc * sizeof(float);
    const cudaError_t e = dev_malloc(&S->dpart, bytes);
    if (e != cudaSuccess) { S->dpart = nullptr; set_last_error(e, "cudaMalloc"); cudaGetLastError(); return TARDIS_ERR_ALLOC; }
    H->bytes_scratch += bytes;
  }
  return TARDIS_OK;
}

tardis_status_t launch_fused_forward(Handle* H, const void* x, void* y, int n, cudaStream_t s) {
  Scratch* S = static_cast<Scratch*>(H->fscratch);
  const bool det = H->deterministic && S->dpart;
  for (int t0 = 0; t0 < n;) {
    // calls of 5 to 8 tokens go as two launches of about equal size
    const int left = n - t0;
    const int nt = left <= MAXT ? left : (left < 2 * MAXT ? (left + 1) / 2 : MAXT);
    Params p = S->base;
    p.n = nt;
    p.nbuf = S->nbuf_n[nt];
    p.gs_cap = S->gs_cap_n[nt];
    p.x = static_cast<const __nv_bfloat16*>(x) + size_t(t0) * H->d;
    p.y = static_cast<__nv_bfloat16*>(y) + size_t(t0) * H->d;
    p.dbg_bitmap = H->dbg_bitmap ? H->dbg_bitmap + size_t(t0) * (H->h / 32) : nullptr;
    p.dbg_scores = H->dbg_scores ? H->dbg_scores + size_t(t0) * H->h : nullptr;
    p.dpart = det ? S->dpart : nullptr;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S->grid); cfg.blockDim = dim3(NTH); cfg.dynamicSmemBytes = S->smem_bytes; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    void* args[] = {&p};
    const bool fast = S->pairs_fit && S->nbuf_n[nt] >= p.tiles_max;
    TARDIS_CUDA_TRY(cudaLaunchKernelExC(&cfg, S->kernels[nt == 1 ? 0 : 1][fast ? 1 : 0], args));
    H->launches += 1;
    if (det) {
      const int work = nt * (H->d >> 2);                    // warps
      k_ordered_sum<<<(work + 3) / 4, 128, 0, s>>>(S->dpart, H->bf, p.y, nt, H->d, p.dacc, p.nkc + S->grid);
      TARDIS_CUDA_TRY(cudaGetLastError());
      H->launches += 1;
    }
    t0 += nt;
  }
  return TARDIS_OK;
}

// A bounded wait that runs out, on purpose and without any fault: one warp arms a barrier for bytes that no copy will ever
// deliver, waits with the given limit, and records the time-out in the handle's error word exactly as the kernels do.
__global__ void k_wait_that_runs_out(long long limit_cycles, unsigned long long* counters) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    fz::mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fz::mbar_expect_tx(&bar, 16u);
  }
  __syncwarp();
  const bool landed = fz::mbar_wait_warp(&bar, 0u, limit_cycles);
  if (!landed && threadIdx.x == 0) atomicExch(&counters[CTR_ERROR], 1ull);
}

tardis_status_t launch_wait_that_runs_out(Handle* H, long long limit_cycles, cudaStream_t s) {
  k_wait_that_runs_out<<<1, 32, 0, s>>>(limit_cycles, H->counters);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t fused_read_stamps(long long* out, int max_ctas) {
#ifdef TARDIS_PHASE_STAMPS
  const int n = max_ctas < kStampCtas ? max_ctas : kStampCtas;
  TARDIS_CUDA_TRY(cudaDeviceSynchronize());
  TARDIS_CUDA_TRY(cudaMemcpyFromSymbol(out, g_stamps, sizeof(long long) * size_t(n) * kStampSlots));
  return TARDIS_OK;
#else
  (void)out; (void)max_ctas;
  return TARDIS_ERR_UNSUPPORTED;
#endif
}

void fused_release(Handle* H) {
  Scratch* S = static_cast<Scratch*>(H->fscratch);
  if (!S) return;
  void* ptrs[] = {S->pblocks, S->plan, S->smax, S->yacc, S->ctl, S->Cp, S->dpart};
  for (void* q : ptrs)
    if (q) dev_free(q);
  delete S;
  H->fscratch = nullptr;
}

}  // namespace tardis
