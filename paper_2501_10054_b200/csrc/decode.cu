// Fused batch-1 decode kernel of the online path (Section 5.4) for bf16 layers on sm_100a.
//
// One launch does the whole token: predictor score (Section 5.3), flagging and compaction,
// speculative folded product, result fixing.  The grid is (up to) two 512-thread CTAs per SM.
//
//   * Prologue (before griddepcontrol.wait, so it overlaps the tail of the previous launch in the
//     stream): a CTA owns a few 16-neuron tiles; their predictor blocks (packed 2-bit codes + group
//     words) are one contiguous region per tile and are fetched with a few large bulk async copies
//     (cp.async.bulk + mbarrier) into shared memory.  They read constant state of the layer only.
//     (Prefetching the folded matrix into L2 here as well was measured: no gain, left out.)
//   * x is loaded once: a bf16 copy in shared memory, and a 4-limb signed base-256 fixed-point copy in
//     tensor-core operand order.
//   * Then the warps split.  Warps 0..7 evaluate the predictor on the integer tensor cores: the codes are
//     masked straight out of the packed words (no shifts: the field position is a power-of-4 weight that
//     the pre-scaling of x undoes) and multiplied with the limbs (mma.m16n8k32.u8.s8, s32 accumulators,
//     exact).  The bf16 group scales of a neuron are held as 16-bit integers over one power of two per
//     neuron, so group sums are scaled and accumulated in 64-bit integers (exact) and the score equals the
//     mathematical one up to the (tracked) truncation of tiny x elements and one fp64 rounding; a score
//     that close to a range end is re-evaluated in fp64 from the original codes.  This phase is bound by
//     the integer pipe, which is why only half of the warps are given to it.
//   * Meanwhile warps 8..15 run the speculative folded product on the bf16 tensor cores: the fold leaves
//     W_f in A-fragment order (units of 16 outputs x 256 channels, 8 KB, contiguous).  A warp works on
//     one channel chunk at a time and draws output tiles from a global ticket of that chunk, so the
//     units spread over all CTAs however busy each one is.
//   * All 16 warps meet; flags are compacted by ballot + prefix sum into the CTA's ascending list.
//   * Result fixing: the predictor buffers are free by now and become row slots.  The W1 rows of the
//     CTA's flagged neurons, then their W2T rows, are fetched by one bulk copy per row, all slots at once
//     (a ring of slot groups when there are more rows than slots).  W1 rows give z_j (the warps split
//     the channels) and delta_j = GELU(z_j) - a_j z_j - c_j; then every thread owns 8 output columns
//     (per slot of 512 vectors) and adds delta_j times its slice of the W2T rows.
//   * All partial outputs are added (red.global) into one of a few replicas of an fp32 accumulator
//     (the replicas keep the number of reductions per address small).  CTAs count themselves when
//     done; the last one sums the replicas, adds b_f, rounds to bf16, and re-zeroes the scratch.
#include <stdio.h>

#include <vector>

#include "common.cuh"
#include "ptx.cuh"

namespace tardis {
namespace dec {
using namespace ptx;

constexpr int NW = 16;            // warps per CTA
constexpr int NWP = 8;            // of them, warps that evaluate the predictor while the others stream the folded matrix
constexpr int NTH = NW * 32;      // threads per CTA
constexpr int KC = 256;           // channels per predictor block
constexpr int MAXTILES = 16;      // predictor tiles (of 16 neurons) per CTA
constexpr int MAXRC = 64;         // exact re-checks per CTA before the list overflows (rest handled in place)
constexpr int MAXBUF = 8;         // predictor unit buffers in shared memory
constexpr int MAXSLOTS = 16;      // rows of W1 / W2T held in shared memory at once by the result fixing
constexpr int MAXGROUPS = 8;      // slot groups (one barrier each) of the result fixing
constexpr int kBadRow = 0x40000000;   // row whose group scales do not fit the integer form: always re-evaluated
constexpr int NREP = 4;           // replicas of the output accumulator
constexpr int XVR = 2;            // 8-channel vectors of x per thread (padded d <= 8192)
// control words (unsigned int) in global scratch; all zero between calls
constexpr int CTL_TICKET = 0;     // [32] stride 32: next output tile of a channel chunk of the folded matrix
constexpr int CTL_DONE = 1024;    // CTAs that have added all their contributions
constexpr int CTL_NFL = 1056;     // flagged neurons of the token so far
constexpr int CTL_WORDS = 1088;

struct Params {
  const uint8_t* pblocks;  // [tile][kchunk] predictor blocks
  int pbs, nkc, G;
  const __nv_bfloat16 *W1, *W2T;
  const uint4* Cp;         // folded matrix in tensor-core fragment order (see k_pack_folded)
  const float *bf, *lo, *hi, *a, *c, *b1;
  const uint32_t* codes; const __nv_bfloat16* scale; const uint8_t* zero;   // originals (exact re-check)
  const float* smax;       // largest group scale of the layer
  const int* rowexp;       // per neuron: power of two its integer group scales are expressed in (kBadRow: none)
  const int2* plan;        // per CTA: first tile, tile count
  const __nv_bfloat16* x; __nv_bfloat16* y;
  float* yacc;             // [NREP][dacc] fp32
  unsigned int* ctl; unsigned long long* counters;
  uint32_t* dbg_bitmap; double* dbg_scores;
  int d, dpad, dacc, h, ngroups, act;
  int nranges, cpr;        // a tile's chunks are taken in nranges units of cpr chunks (cpr <= NW)
  int nbuf, unit_bytes;    // unit buffers in shared memory and their size
  int tiles_max;
  int nvec;                // 8-column vectors in a row
  int fix_gs, fix_ng;      // result fixing: row slots per group, groups (fix_gs * fix_ng rows fit in the predictor buffers)
  int nunits;              // folded-matrix units in all
  int ntk;                 // output tiles of the folded matrix (16 outputs each)
};

struct Scratch {           // handle-owned device memory of the fused path
  uint8_t* pblocks; int2* plan; float* smax; float* yacc; unsigned int* ctl; int* rowexp; uint4* Cp;
  Params base; size_t smem_bytes; size_t bytes; int grid; int vpt; const void* kernel;
};

// ---- shared-memory carve-up (host and device agree through this) -----------------------------------
struct SmemLayout {
  size_t pbuf_bytes, pbuf, xq, zeros, xh, sxi, zpart, wpart, score, tab, fl_j, fl_delta, rc, flagbits, wred, bars, misc, total;
  __host__ __device__ SmemLayout(int dpad, int ngroups, int tiles_max, int nbuf, int unit_bytes) {
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; size_t r = o; o += bytes; return r; };
    const size_t rows = size_t(tiles_max) * 16;
    pbuf_bytes = size_t(nbuf) * unit_bytes;
    if (pbuf_bytes < size_t(4) * dpad) pbuf_bytes = size_t(4) * dpad;   // room for two rows of the result fixing
    pbuf = take(pbuf_bytes, 128);
    xq = take(size_t(4) * (dpad + 64), 128);
    zeros = take(256, 16);                    // what the lanes that feed unused operand columns read
    xh = take(size_t(dpad + 16) * 2, 16);     // + 16 zeros: the B operand of lanes that feed the unused columns
    sxi = take(size_t(ngroups + 16) * sizeof(int), 8);
    zpart = take(rows * NW * sizeof(double), 8);
    wpart = take(size_t(2) * MAXSLOTS * NW * sizeof(float), 4);
    score = take(rows * sizeof(double), 8);
    tab = take(6 * rows * sizeof(float), 4);
    fl_j = take(rows * sizeof(int), 4);
    fl_delta = take(rows * sizeof(float), 4);
    rc = take(MAXRC * sizeof(int), 4);
    flagbits = take(rows * sizeof(int), 4);
    wred = take(size_t(3) * NW * sizeof(float), 4);
    bars = take(size_t(MAXBUF + MAXGROUPS) * sizeof(uint64_t), 8);
    misc = take(48 * sizeof(int), 8);
    total = o;
  }
};
enum { MS_NFL = 0, MS_NRC = 1, MS_ERR = 2, MS_LAST = 3, MS_WCNT = 8, MS_BUFCNT = 32 };


// ---- phase stamps (compiled in with -DTARDIS_PHASE_STAMPS only) -----------------------------------------
// Thread 0 of every CTA (and lane 0 of the first streaming warp) writes the global timer at the phase
// boundaries of the last launch; tardis_debug_phase_stamps copies the table to the host.
constexpr int kStampCtas = 512, kStampSlots = 16;
enum { ST_START = 0, ST_X = 1, ST_LIMBS = 2, ST_PRED = 3, ST_STREAM = 4, ST_FLAGS = 5, ST_FIXED = 6, ST_COUNTED = 7,
       ST_FINAL = 8, ST_NFL = 9 };
#ifdef TARDIS_PHASE_STAMPS
__device__ long long g_stamps[kStampCtas * kStampSlots];
__device__ __forceinline__ long long global_timer() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define TARDIS_STAMP(cond, slot) do { if ((cond) && blockIdx.x < kStampCtas) g_stamps[blockIdx.x * kStampSlots + (slot)] = global_timer(); } while (0)
#define TARDIS_STAMP_VALUE(cond, slot, v) do { if ((cond) && blockIdx.x < kStampCtas) g_stamps[blockIdx.x * kStampSlots + (slot)] = (long long)(v); } while (0)
#else
#define TARDIS_STAMP(cond, slot) do { } while (0)
#define TARDIS_STAMP_VALUE(cond, slot, v) do { } while (0)
#endif

// ---- the kernel ---------------------------------------------------------------------------------------
template <int VPT, int G>
__global__ void __launch_bounds__(NTH, 2) k_decode(const Params p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout L(p.dpad, p.ngroups, p.tiles_max, p.nbuf, p.unit_bytes);
  uint8_t* pbuf = smem + L.pbuf;
  uint8_t* xq = smem + L.xq;
  __nv_bfloat16* xh = reinterpret_cast<__nv_bfloat16*>(smem + L.xh);
  int* sxi = reinterpret_cast<int*>(smem + L.sxi);
  double* zpart = reinterpret_cast<double*>(smem + L.zpart);
  float* wpart = reinterpret_cast<float*>(smem + L.wpart);
  double* score = reinterpret_cast<double*>(smem + L.score);
  float* tab = reinterpret_cast<float*>(smem + L.tab);   // [6][TR]: lo, hi, b1, a, c, scale exponent (int bits) of the CTA's neurons
  int* fl_j = reinterpret_cast<int*>(smem + L.fl_j);
  float* fl_delta = reinterpret_cast<float*>(smem + L.fl_delta);
  int* rc = reinterpret_cast<int*>(smem + L.rc);
  int* flagbits = reinterpret_cast<int*>(smem + L.flagbits);
  float* wred = reinterpret_cast<float*>(smem + L.wred);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
  volatile int* misc = reinterpret_cast<volatile int*>(smem + L.misc);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = p.d;
  const int TR = p.tiles_max * 16;
  const int xq_stride = p.dpad + 64;
  const int2 plan = p.plan[blockIdx.x];
  const int NU = plan.y * p.nranges;            // predictor units of this CTA
  const int g = lane >> 2, t4 = lane & 3;

  // Unit u = (tile u / nranges, chunk range u % nranges): one contiguous piece of the predictor blocks.
  auto issue_unit = [&](int u) {
    const int tl = u / p.nranges, r = u - tl * p.nranges;
    const int nch = min(p.cpr, p.nkc - r * p.cpr);
    const int b = u % p.nbuf;
    const uint32_t bytes = uint32_t(nch) * p.pbs;
    mbar_expect_tx(&full[b], bytes);
    bulk_g2s(pbuf + size_t(b) * p.unit_bytes, p.pblocks + (size_t(plan.x + tl) * p.nkc + size_t(r) * p.cpr) * p.pbs, bytes, &full[b]);
  };

  TARDIS_STAMP(tid == 0, ST_START);
  // Programmatic dependent launch: the next launch in the stream may start its own prologue (everything
  // up to its griddepcontrol.wait reads only the layer's constant state) while this one is still running.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // per-neuron tables of the CTA's rows
  float tl0 = 0.f, tl1 = 0.f, tl2 = 0.f, tl3 = 0.f, tl4 = 0.f;
  int tl5 = 0;
  if (tid < plan.y * 16) {
    const int j = plan.x * 16 + tid;
    tl0 = p.lo[j]; tl1 = p.hi[j]; tl2 = p.b1[j]; tl3 = p.a[j]; tl4 = p.c[j]; tl5 = p.rowexp[j];
  }

  if (tid == 0) {
    for (int b = 0; b < p.nbuf; ++b) mbar_init(&full[b], 1);
    for (int b = 0; b < MAXGROUPS; ++b) mbar_init(&full[MAXBUF + b], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 48) misc[tid] = 0;
  if (tid < 8) reinterpret_cast<uint32_t*>(xh + p.dpad)[tid] = 0u;
  if (tid >= 32 && tid < 96) reinterpret_cast<uint32_t*>(smem + L.zeros)[tid - 32] = 0u;
  __syncthreads();
  // predictor blocks first: nothing of them depends on x
  if (lane == 0 && warp < p.nbuf && warp < NU) issue_unit(warp);

  // From here on the kernel touches what earlier work in the stream may still be writing (x, the
  // scratch shared by the calls of one handle): wait until that work has completed and is visible.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  uint4 xw[XVR];
#pragma unroll
  for (int m = 0; m < XVR; ++m) {
    const int v = tid + m * NTH;
    xw[m] = make_uint4(0u, 0u, 0u, 0u);
    if (v < p.nvec) xw[m] = *reinterpret_cast<const uint4*>(p.x + size_t(v) * 8);
  }

  if (tid < plan.y * 16) {
    tab[tid] = tl0; tab[TR + tid] = tl1; tab[2 * TR + tid] = tl2; tab[3 * TR + tid] = tl3; tab[4 * TR + tid] = tl4; tab[5 * TR + tid] = __int_as_float(tl5);
  }

  // ---- x: registers, bf16 copy in shared memory, max |x| ----
  {
    float amax = 0.f;
    bool nonfinite = false;
#pragma unroll
    for (int m = 0; m < XVR; ++m) {
      const int v = tid + m * NTH;
      if (v * 8 < p.dpad) *reinterpret_cast<uint4*>(xh + v * 8) = xw[m];
      float f[8];
      unpack8(f, xw[m]);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (!(fabsf(f[i]) <= 3.0e38f)) nonfinite = true;
        amax = fmaxf(amax, fabsf(f[i]));
      }
    }
    amax = fmaxf(amax, 0.f);   // drops NaN
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const bool any_nf = __any_sync(0xffffffffu, nonfinite);
    if (lane == 0) { wred[warp] = amax; wred[NW + warp] = any_nf ? 1.f : 0.f; }
  }
  __syncthreads();
  TARDIS_STAMP(tid == 0, ST_X);
  float amax_all = 0.f;
  bool tok_nonfinite = false;
#pragma unroll
  for (int w = 0; w < NW; ++w) { amax_all = fmaxf(amax_all, wred[w]); tok_nonfinite |= wred[NW + w] != 0.f; }
  // exponent E: |x| 2^-E < 2^22 for every element
  int E = 0;
  if (amax_all > 0.f && !tok_nonfinite) E = max(int((__float_as_uint(amax_all) >> 23) & 0xff) - 127 - 21, -100);

  // ---- speculative folded product on the tensor cores ----
  // The folded matrix is stored in units of 16 outputs x 256 channels (8 KB, contiguous, already in
  // A-fragment order).  A warp works on channel chunks first, first + step, ... and draws the output tiles from
  // the global ticket of the chunk; it streams a unit as four blocks of four 128-bit loads per lane (one
  // block ahead of the one being multiplied), multiplies it with x (the B operand: column 0 = x, other
  // columns zero) in two independent accumulators, and adds the 16 partial outputs to the accumulator
  // replica of its CTA.
  float* const rep = p.yacc + size_t(blockIdx.x % NREP) * p.dacc;
  auto stream_c = [&](int first, int step) {
    unsigned int* ticket = p.ctl + CTL_TICKET;
    auto issue = [&]() -> unsigned int {        // lane 0 draws; the value is looked at one unit later
      unsigned int t = 0;
      if (lane == 0) t = atomicAdd(ticket, 1u);
      return t;
    };
    auto resolve = [&](unsigned int raw) -> int {
      const unsigned int t = __shfl_sync(0xffffffffu, raw, 0);
      return t < (unsigned int)p.ntk ? int(t) : -1;
    };
    for (int kc = first; kc < p.nkc; kc += step) {
      ticket = p.ctl + CTL_TICKET + kc * 32;
      // lanes of column 0 read x, the others the zeros behind it
      const uint4* xp = reinterpret_cast<const uint4*>(g == 0 ? xh + kc * KC + t4 * 16 : xh + p.dpad);
      const int xstep = g == 0 ? 8 : 0;                 // uint4 per 64-channel block
      const uint4* cbase = p.Cp + size_t(kc) * 512 + lane;
      const size_t tstride = size_t(p.nkc) * 512;       // uint4 per output tile
      auto load = [&](uint4 (&buf)[4], int it, int bi) {
        const uint4* src = cbase + size_t(it) * tstride + bi * 128;
#pragma unroll
        for (int m = 0; m < 4; ++m) buf[m] = ldg_stream(src + m * 32);
      };
      auto multiply = [&](float (&c)[2][4], const uint4 (&buf)[4], int bi) {
        const uint4 x0 = xp[bi * xstep], x1 = xp[bi * xstep + 1];
        mma_bf16(c[0], buf[0].x, buf[0].y, buf[0].z, buf[0].w, x0.x, x0.y);
        mma_bf16(c[1], buf[1].x, buf[1].y, buf[1].z, buf[1].w, x0.z, x0.w);
        mma_bf16(c[0], buf[2].x, buf[2].y, buf[2].z, buf[2].w, x1.x, x1.y);
        mma_bf16(c[1], buf[3].x, buf[3].y, buf[3].z, buf[3].w, x1.z, x1.w);
      };
      uint4 ba[4], bb[4];
      int it = resolve(issue());
      bool more = it >= 0;
      unsigned int raw = more ? issue() : 0xffffffffu;
      if (it >= 0) load(ba, it, 0);
      while (it >= 0) {
        float c[2][4];
#pragma unroll
        for (int m = 0; m < 2; ++m) c[m][0] = c[m][1] = c[m][2] = c[m][3] = 0.f;
        load(bb, it, 1);
        multiply(c, ba, 0);
        load(ba, it, 2);
        multiply(c, bb, 1);
        load(bb, it, 3);
        multiply(c, ba, 2);
        const int nx = more ? resolve(raw) : -1;        // the next tile: its first block goes in flight now
        more = nx >= 0;
        raw = more ? issue() : 0xffffffffu;
        if (nx >= 0) load(ba, nx, 0);
        multiply(c, bb, 3);
        if (t4 == 0) {
          red_add_f32(rep + it * 16 + g, c[0][0] + c[1][0]);
          red_add_f32(rep + it * 16 + g + 8, c[0][2] + c[1][2]);
        }
        it = nx;
      }
    }
  };

  // ---- fixed-point limbs of x in tensor-core operand order; group sums; truncation residual ----
  // A thread holds 8 channels = half of a 16-channel unit; the two halves meet through one shuffle.
  {
    const float inv = __uint_as_float(uint32_t(127 - E) << 23);    // 2^-E
    const int lpg = p.G / 8;                                        // lanes per predictor group
    const int g_log2 = p.G == 64 ? 6 : (p.G == 128 ? 7 : 8);
    const bool odd = lane & 1;
    float resid = 0.f;
#pragma unroll
    for (int m = 0; m < XVR; ++m) {
      if (m * NTH * 8 >= p.dpad) break;             // uniform over the CTA
      const int v = tid + m * NTH;
      const bool active = v * 8 < p.dpad;
      float f[8];
      unpack8(f, xw[m]);
      uint32_t D[8];
      int sx = 0;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float s = (active && !tok_nonfinite) ? f[c] * inv : 0.f;
        const float t = s + 12582912.f;                         // 1.5 * 2^23: rounds s to an integer (|s| < 2^22)
        const int X = __float_as_int(t) - 0x4B400000;
        resid += fabsf(s - (t - 12582912.f));
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
      if (active) {
        const int u = v >> 1, kb = u >> 2, t = u & 3;
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
          *reinterpret_cast<uint4*>(xq + size_t(l) * xq_stride + size_t(kb) * 64 + t * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
      // group sums of the integer x (exact)
      for (int o = 1; o < lpg; o <<= 1) sx += __shfl_xor_sync(0xffffffffu, sx, o);
      if (active && (lane & (lpg - 1)) == 0) sxi[(v * 8) >> g_log2] = sx;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) resid += __shfl_xor_sync(0xffffffffu, resid, o);
    if (lane == 0) wred[2 * NW + warp] = resid;
  }
  // ---- roles ----
  // The limbs are complete once all 16 warps have passed here.  Warps 8..15 only announce their part
  // (bar.arrive) and go on to the speculative folded product, which needs nothing but x; warps 0..7 wait for
  // everybody's limbs (bar.sync) and evaluate the predictor.  Both meet again at the barrier after it.
  TARDIS_STAMP(tid == 0, ST_LIMBS);
  if (warp >= NWP) {
    asm volatile("bar.arrive 1, %0;" ::"n"(NTH) : "memory");
    stream_c(warp - NWP, NW - NWP);
    TARDIS_STAMP(tid == NWP * 32, ST_STREAM);
  } else {
    asm volatile("bar.sync 1, %0;" ::"n"(NTH) : "memory");
  }
  // ---- predictor: warp w < 8 takes chunks w, w + 8, ... of every unit; partial scores of a tile go to shared memory ----
  if (warp < NWP) {
    long long zacc[4] = {0, 0, 0, 0}, zt[2] = {0, 0};
    constexpr int GPC = KC / G;                              // groups per chunk: 4 or 2
    // Everything a block needs sits at fixed offsets from four per-lane pointers (codes, group words, group sums
    // of x, limbs of x); lanes whose operand columns are unused (g >= 4) read a block of zeros instead.
    const uint8_t* const xql = g < 4 ? xq + size_t(g) * xq_stride + t4 * 16 : smem + L.zeros + t4 * 16;
    const int xqs = g < 4 ? KC : 0;                          // bytes of limbs per chunk
    int b = 0, tl = 0, r = 0;                                // buffer, tile and chunk range of unit u
    uint32_t par = 0u;                                       // phase of the buffer's barrier
    for (int u = 0; u < NU; ++u) {
      bool landed = mbar_wait(&full[b], par);
      if (!landed) {                                 // record, give the copy one more bounded wait, skip the work
        if (lane == 0) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ERR] = 1; }
        landed = mbar_wait(&full[b], par);
      }
      const int nch = min(p.cpr, p.nkc - r * p.cpr);
      const bool usable = landed && !misc[MS_ERR];
      const uint8_t* const ubase = pbuf + size_t(b) * p.unit_bytes;
      for (int cc = warp; cc < nch && usable; cc += NWP) {
        const int kc = r * p.cpr + cc;
        const uint8_t* const blk = ubase + cc * p.pbs;
        const uint4* const cp = reinterpret_cast<const uint4*>(blk) + lane;
        const uint2* const mp = reinterpret_cast<const uint2*>(blk + 1024) + g;
        const int* const sxp = sxi + kc * GPC;
        const uint4* const xp = reinterpret_cast<const uint4*>(xql + kc * xqs);
        // group gl of the chunk done: sums (|.| < 2^22) times the integer scales (|.| < 2^15), all exact
        auto scale_group = [&](const int (&ia)[4], int gl) {
          const uint2 mw = mp[gl * 8];
          const int m0 = int(mw.x) >> 16, m1 = int(mw.y) >> 16;
          zacc[0] += (long long)m0 * ia[0]; zacc[1] += (long long)m0 * ia[1];
          zacc[2] += (long long)m1 * ia[2]; zacc[3] += (long long)m1 * ia[3];
          const int sx = sxp[gl];
          zt[0] += (long long)(m0 * int(mw.x & 3u)) * sx;
          zt[1] += (long long)(m1 * int(mw.y & 3u)) * sx;
        };
#pragma unroll
        for (int pair = 0; pair < 2; ++pair) {            // 128 channels: four independent MMAs
          const uint4 cw = cp[pair * 32];
          const uint4 xb0 = xp[pair * 8], xb1 = xp[pair * 8 + 4];
          // two accumulator chains of two MMAs each (a longer chain through one accumulator would stall the pipe)
          int qa[4], qb[4];
          mma_u8s8_z(qa, cw.x & 0x03030303u, cw.y & 0x03030303u, cw.x & 0x0C0C0C0Cu, cw.y & 0x0C0C0C0Cu, xb0.x, xb0.y);
          mma_u8s8_z(qb, cw.z & 0x03030303u, cw.w & 0x03030303u, cw.z & 0x0C0C0C0Cu, cw.w & 0x0C0C0C0Cu, xb1.x, xb1.y);
          mma_u8s8(qa, cw.x & 0x30303030u, cw.y & 0x30303030u, cw.x & 0xC0C0C0C0u, cw.y & 0xC0C0C0C0u, xb0.z, xb0.w);
          mma_u8s8(qb, cw.z & 0x30303030u, cw.w & 0x30303030u, cw.z & 0xC0C0C0C0u, cw.w & 0xC0C0C0C0u, xb1.z, xb1.w);
          if (G == 64) {
            scale_group(qa, pair * 2);
            scale_group(qb, pair * 2 + 1);
          } else {                                        // G == 128
            int ga[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) ga[i] = qa[i] + qb[i];
            scale_group(ga, pair);
          }
        }
      }
      if (r == p.nranges - 1) {
        // limbs: lane t4 = 0 holds limbs 0,1 ; t4 = 1 holds limbs 2,3 (columns 4..7 are unused for one token)
        double v0 = 0.0, v1 = 0.0;
        // |sums| < 2^47: adding them to the bit pattern of 2^52 + 2^51 and taking that constant off again converts exactly
        const double d0 = __longlong_as_double(zacc[0] + 0x4338000000000000LL) - 6755399441055744.0;
        const double d1 = __longlong_as_double(zacc[1] + 0x4338000000000000LL) - 6755399441055744.0;
        const double d2 = __longlong_as_double(zacc[2] + 0x4338000000000000LL) - 6755399441055744.0;
        const double d3 = __longlong_as_double(zacc[3] + 0x4338000000000000LL) - 6755399441055744.0;
        if (t4 == 0) { v0 = d0 + 256.0 * d1; v1 = d2 + 256.0 * d3; }
        if (t4 == 1) { v0 = 65536.0 * (d0 + 256.0 * d1); v1 = 65536.0 * (d2 + 256.0 * d3); }
        v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
        if (t4 == 0) {
          zpart[(tl * NWP + warp) * 16 + g] = v0 * (1.0 / 64.0) - double(zt[0]);
          zpart[(tl * NWP + warp) * 16 + g + 8] = v1 * (1.0 / 64.0) - double(zt[1]);
        }
        zacc[0] = zacc[1] = zacc[2] = zacc[3] = 0; zt[0] = zt[1] = 0;
      }
      // hand the buffer back: the last warp to leave it starts the copy of the unit that reuses it
      if (u + p.nbuf < NU) {                             // (never with every unit resident from the start)
        __threadfence_block();
        __syncwarp();
        if (lane == 0) {
          const int old = atomicAdd(const_cast<int*>(&misc[MS_BUFCNT + b]), 1);
          if (old == NWP - 1) {
            misc[MS_BUFCNT + b] = 0;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue_unit(u + p.nbuf);
          }
        }
      }
      if (++b == p.nbuf) { b = 0; par ^= 1u; }
      if (++r == p.nranges) { r = 0; ++tl; }
    }
  }
  TARDIS_STAMP(tid == 0, ST_PRED);
  __syncthreads();
  // tolerance of the fast score: every rounding residual (<= 1/2 unit of 2^E) times |code - zero| <= 3 times the scale
  double tau;
  {
    float rs = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) rs += wred[2 * NW + w];
    tau = double(rs) * 1.001 * 3.0 * double(*p.smax) * ldexp(1.0, E);
  }


  // ---- scores, flags ----
  const int nrow = plan.y * 16;
  if (tid < nrow) {
    const int tl = tid >> 4, r = tid & 15;
    const int j = (plan.x + tl) * 16 + r;
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < NWP; ++w) s += zpart[(tl * NWP + w) * 16 + r];
    const int rexp = __float_as_int(tab[5 * TR + tid]);
    const double zhat = double(tab[2 * TR + tid]) + ldexp(s, E + (rexp == kBadRow ? 0 : rexp));
    const double lo = double(tab[tid]), hi = double(tab[TR + tid]);
    int f = ((lo <= zhat) && (zhat < hi)) ? 0 : 1;
    if (tok_nonfinite) f = 1;
    else if (rexp == kBadRow || (tau > 0.0 && (fabs(zhat - lo) <= tau || fabs(zhat - hi) <= tau))) {
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
          for (int q2 = 0; q2 < 16; ++q2) inner += (double((word >> (2 * q2)) & 3u) - zp) * double(__bfloat162float(xh[w * 16 + q2]));
          a64 += double(__bfloat162float(p.scale[size_t(j) * p.ngroups + grp])) * inner;
        }
        const double z2 = a64 + double(tab[2 * TR + tid]);
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
        for (int q = 0; q < 16; ++q) inner += (double((word >> (2 * q)) & 3u) - zp) * double(__bfloat162float(xh[w * 16 + q]));
        a64 += double(__bfloat162float(p.scale[size_t(j) * p.ngroups + grp])) * inner;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a64 += __shfl_xor_sync(0xffffffffu, a64, o);
      if (lane == 0) {
        const double zhat = a64 + double(tab[2 * TR + n]);
        flagbits[n] = ((double(tab[n]) <= zhat) && (zhat < double(tab[TR + n]))) ? 0 : 1;
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
    if (tid == 0) {
      misc[MS_NFL] = total;
      if (total) atomicAdd(&p.ctl[CTL_NFL], (unsigned int)total);   // read by the warp that finishes column range 0
    }
    // debug capture: 16-bit halves of the flag words, scores
    if (p.dbg_bitmap && tid < nrow && (tid & 15) == 0)
      reinterpret_cast<uint16_t*>(p.dbg_bitmap)[plan.x + (tid >> 4)] = uint16_t((bal >> (lane & 16)) & 0xffffu);
    if (p.dbg_scores && tid < nrow) p.dbg_scores[(plan.x + (tid >> 4)) * 16 + (tid & 15)] = score[tid];
  }
  __syncthreads();
  const int nfl = misc[MS_NFL];

  TARDIS_STAMP(tid == 0, ST_FLAGS);
  TARDIS_STAMP_VALUE(tid == 0, ST_NFL, nfl);
  // ---- result fixing ----
  // The predictor buffers are free now and take the rows the fixing needs, one bulk copy per row: item i < nfl
  // is the W1 row of the i-th flagged neuron, item nfl + i its W2T row.  The row slots form a ring of groups
  // with one barrier each; all groups are filled at once (for a typical token that is every row the CTA
  // needs, so the fixing costs one trip to memory), and a group is filled again as soon as its rows have been
  // used.  W1 rows: the warps split the channels, partial dot products meet in shared memory and give
  // delta_j = GELU(z_j) - a_j z_j - c_j.  W2T rows: a thread owns VPT vectors of 8 output columns and adds
  // delta_j times its slice of the row.
  float acc[VPT][8];
#pragma unroll
  for (int m = 0; m < VPT; ++m)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[m][i] = 0.f;
  {
    uint64_t* fixbar = &full[MAXBUF];
    const uint32_t rowbytes = uint32_t(d) * 2u;
    const size_t slot_bytes = size_t(p.dpad) * 2;
    const int nitems = 2 * nfl;
    const int GS = p.fix_gs, NG = p.fix_ng;
    const int kw = p.dpad / NW;                                   // channels per warp (a multiple of 16)
    // fills group gr with the items of step st (all threads call it; thread 0 arms the barrier, lane 0 of
    // warp k issues the copy of the k-th item)
    auto fill = [&](int gr, int st) {
      const int i0 = st * GS, cnt = min(GS, nitems - i0);
      if (cnt <= 0) return;
      if (tid == 0) mbar_expect_tx(&fixbar[gr], uint32_t(cnt) * rowbytes);
      if (lane == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the slots were read with ordinary loads
        for (int k = warp; k < cnt; k += NW) {
          const int i = i0 + k;
          const __nv_bfloat16* src = i < nfl ? p.W1 + size_t(fl_j[i]) * d : p.W2T + size_t(fl_j[i - nfl]) * d;
          bulk_g2s(pbuf + size_t(gr * GS + k) * slot_bytes, src, rowbytes, &fixbar[gr]);
        }
      }
    };
    const int nsteps = (nitems + GS - 1) / GS;
    for (int gr = 0; gr < NG; ++gr) fill(gr, gr);
    int gr = 0;
    uint32_t par = 0u;
    for (int st = 0; st < nsteps; ++st) {
      const int i0 = st * GS, cnt = min(GS, nitems - i0);
      bool landed = mbar_wait(&fixbar[gr], par);
      if (!landed) {
        if (lane == 0) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ERR] = 1; }
        landed = mbar_wait(&fixbar[gr], par);
      }
      const int nw1 = max(0, min(cnt, nfl - i0));                 // items of this step that are W1 rows
      float* wp = wpart + (st & 1) * MAXSLOTS * NW;
      for (int k = 0; k < nw1; ++k) {
        const __nv_bfloat16* row = reinterpret_cast<const __nv_bfloat16*>(pbuf + size_t(gr * GS + k) * slot_bytes);
        float part = 0.f;
        for (int c0 = warp * kw + lane * 8; c0 < (warp + 1) * kw; c0 += 256) {
          if (c0 < d && landed) {
            float xv[8];
            unpack8(xv, *reinterpret_cast<const uint4*>(xh + c0));
            part += dot8(*reinterpret_cast<const uint4*>(row + c0), xv);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if (lane == 0) wp[k * NW + warp] = part;
      }
      if (nw1 > 0) {
        __syncthreads();
        if (tid < nw1) {
          const int rowi = fl_j[i0 + tid] - plan.x * 16;
          float z = 0.f;
#pragma unroll
          for (int ww = 0; ww < NW; ++ww) z += wp[tid * NW + ww];
          z += tab[2 * TR + rowi];
          fl_delta[i0 + tid] = gelu_f32(z, p.act) - tab[3 * TR + rowi] * z - tab[4 * TR + rowi];
        }
        if (nw1 < cnt) __syncthreads();                           // W2T rows of the same step need these deltas
      }
      for (int k = nw1; k < cnt; ++k) {
        const __nv_bfloat16* row = reinterpret_cast<const __nv_bfloat16*>(pbuf + size_t(gr * GS + k) * slot_bytes);
        const float dl = fl_delta[i0 + k - nfl];
#pragma unroll
        for (int m = 0; m < VPT; ++m) {
          const int vec = m * NTH + tid;
          if (vec < p.nvec && landed) fma8(acc[m], dl, *reinterpret_cast<const uint4*>(row + vec * 8));
        }
      }
      if (st + 1 < nsteps) {
        __syncthreads();                                          // rows used, deltas visible
        fill(gr, st + NG);
      }
      if (++gr == NG) { gr = 0; par ^= 1u; }
    }
  }
  if (nfl > 0) {
#pragma unroll
    for (int m = 0; m < VPT; ++m) {
      const int vec = m * NTH + tid;
      if (vec < p.nvec) {
        red_add_v4(rep + vec * 8, acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
        red_add_v4(rep + vec * 8 + 4, acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
      }
    }
  }

  TARDIS_STAMP(tid == 0, ST_FIXED);
  // Any warp of any CTA may have added to any column, so the columns are complete when the last CTA is:
  // the CTAs count themselves, and the last one turns the accumulator into y.
  __threadfence();
  __syncthreads();
  if (tid == 0) misc[MS_LAST] = int(atomicAdd(&p.ctl[CTL_DONE], 1u));
  __syncthreads();
  TARDIS_STAMP(tid == 0, ST_COUNTED);
  if (misc[MS_LAST] == int(gridDim.x) - 1) {
    __threadfence();
    for (int vec = tid; vec < p.nvec; vec += NTH) {
      const int c0 = vec * 8;
      float4 a0[NREP + 1], a1[NREP + 1];
      a0[NREP] = *reinterpret_cast<const float4*>(p.bf + c0);
      a1[NREP] = *reinterpret_cast<const float4*>(p.bf + c0 + 4);
#pragma unroll
      for (int rp = 0; rp < NREP; ++rp) {
        const float* q = p.yacc + size_t(rp) * p.dacc + c0;
        a0[rp] = __ldcg(reinterpret_cast<const float4*>(q));
        a1[rp] = __ldcg(reinterpret_cast<const float4*>(q + 4));
      }
      float4 s0 = a0[NREP], s1 = a1[NREP];
#pragma unroll
      for (int rp = 0; rp < NREP; ++rp) {
        s0.x += a0[rp].x; s0.y += a0[rp].y; s0.z += a0[rp].z; s0.w += a0[rp].w;
        s1.x += a1[rp].x; s1.y += a1[rp].y; s1.z += a1[rp].z; s1.w += a1[rp].w;
        float* q = p.yacc + size_t(rp) * p.dacc + c0;
        *reinterpret_cast<float4*>(q) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(q + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      __nv_bfloat162 o[4];
      o[0] = __floats2bfloat162_rn(s0.x, s0.y);
      o[1] = __floats2bfloat162_rn(s0.z, s0.w);
      o[2] = __floats2bfloat162_rn(s1.x, s1.y);
      o[3] = __floats2bfloat162_rn(s1.z, s1.w);
      *reinterpret_cast<uint4*>(p.y + c0) = *reinterpret_cast<const uint4*>(o);
    }
    TARDIS_STAMP(tid == 0, ST_FINAL);
    if (lane == 0) {
      for (int kc = warp; kc < p.nkc; kc += NW) p.ctl[CTL_TICKET + kc * 32] = 0u;
      if (warp == 0) {   // every CTA has arrived, so every CTA's flagged count is in
        p.ctl[CTL_DONE] = 0u;
        const unsigned int tot = atomicExch(&p.ctl[CTL_NFL], 0u);
        atomicAdd(&p.counters[CTR_FLAGGED_TOTAL], (unsigned long long)tot);
        atomicMax(&p.counters[CTR_FLAGGED_MAX], (unsigned long long)tot);
      }
    }
  }
}

// ---- set-up kernels --------------------------------------------------------------------------------------
// A bf16 scale is m 2^(e-134) with an integer |m| < 256 (e = biased exponent, at least 1).  Over the groups of
// one neuron the exponents differ little, so every scale of the row is an integer of at most 15 bits times
// 2^(emin-134); rowexp[j] = emin - 134, or kBadRow when the spread is too wide (or a scale is inf / nan).
__device__ __forceinline__ void bf16_parts(__nv_bfloat16 v, int* m, int* e) {
  const uint32_t b = __bfloat16_as_ushort(v);
  const int ex = int((b >> 7) & 0xffu), man = int(b & 0x7fu);
  *e = ex ? ex : 1;
  *m = (ex ? (128 | man) : man) * ((b & 0x8000u) ? -1 : 1);
}
__global__ void k_row_exponent(const __nv_bfloat16* __restrict__ scale, int h, int ng, int* __restrict__ rowexp) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= h) return;
  int emin = 1 << 20, emax = 0;
  bool bad = false;
  for (int g = 0; g < ng; ++g) {
    int m, e;
    bf16_parts(scale[size_t(j) * ng + g], &m, &e);
    if (e == 255) bad = true;
    if (m != 0) { emin = min(emin, e); emax = max(emax, e); }
  }
  if (emax == 0) emin = emax = 1;                    // all scales zero
  rowexp[j] = (bad || emax - emin > 7) ? kBadRow : emin - 134;
}

// Predictor blocks: block (tile, kc) = 2 x 32 lanes x {A0,B0,A1,B1} code words + per-group {row g, row g+8}
// words (integer scale << 16 | zero-point).
__global__ void k_pack_pblocks(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                               const uint8_t* __restrict__ zero, const int* __restrict__ rowexp,
                               uint8_t* __restrict__ out, int d, int G, int nkc, int pbs) {
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
    const int re = rowexp[row];
    if (grp < ng && re != kBadRow) {
      int m, ex;
      bf16_parts(scale[size_t(row) * ng + grp], &m, &ex);
      const int M = m * (1 << (m != 0 ? ex - (re + 134) : 0));
      w = (uint32_t(M & 0xffff) << 16) | uint32_t(zero[size_t(row) * ng + grp] & 3u);
    }
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

}  // namespace dec

using namespace dec;

tardis_status_t decode_prepare(Handle* H, cudaStream_t s) {
  H->dscratch = nullptr;
  H->codes_mma = nullptr;
  const int d = H->d, h = H->h, G = H->G;
  if (H->dtype != TARDIS_BF16 || H->bits != 2) return TARDIS_OK;   // (the integer tensor-core predictor is built for 2-bit codes)
  if (!(G == 64 || G == 128)) return TARDIS_OK;                     // generic kernels serve other group sizes
  const int NT = h / 16;
  const int nvec = d / 8;
  const int vpt = nvec > NTH ? 2 : 1;
  const int dpad = (d + KC - 1) / KC * KC;
  if (d < 64 || d % 16 || dpad > XVR * NTH * 8 || dpad / KC > 32) return TARDIS_OK;
  int max_smem = 0, sm_smem = 0;
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, H->device));
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&sm_smem, cudaDevAttrMaxSharedMemoryPerMultiprocessor, H->device));

  Scratch* S = new (std::nothrow) Scratch();
  if (!S) return TARDIS_ERR_ALLOC;
  memset(S, 0, sizeof(*S));
  Params& p = S->base;
  p.d = d; p.h = h; p.G = G; p.ngroups = H->ngroups; p.act = H->act;
  p.dpad = dpad; p.dacc = (d + 31) / 32 * 32;
  p.nkc = dpad / KC;
  p.pbs = 1024 + 64 * (KC / G);
  p.nranges = (p.nkc + NW - 1) / NW;
  p.cpr = (p.nkc + p.nranges - 1) / p.nranges;
  p.unit_bytes = p.cpr * p.pbs;
  p.nvec = nvec;
  p.nunits = (d / 16) * p.nkc;
  p.ntk = d / 16;
  S->vpt = vpt;
  // two CTAs per SM when their shared memory fits (each CTA also reserves 1 KB), else one
  bool placed = false;
  for (int per_sm = 2; per_sm >= 1 && !placed; --per_sm) {
    const int grid = H->num_sms * per_sm;
    const int tiles_max = (NT + grid - 1) / grid;
    if (tiles_max > MAXTILES) continue;
    const int units = tiles_max * p.nranges;
    const size_t budget = per_sm == 2 ? size_t(sm_smem) / 2 - 1024 : size_t(max_smem);
    const int nbuf_hi = units < MAXBUF ? units : MAXBUF;
    const int nbuf_lo = units < 2 ? units : 2;
    for (int nbuf = nbuf_hi; nbuf >= nbuf_lo && nbuf >= 1; --nbuf) {
      const size_t need = SmemLayout(dpad, p.ngroups, tiles_max, nbuf, p.unit_bytes).total;
      if (need <= budget && need <= size_t(max_smem)) {
        S->grid = grid; p.tiles_max = tiles_max; p.nbuf = nbuf; S->smem_bytes = need;
        size_t slots = SmemLayout(dpad, p.ngroups, tiles_max, nbuf, p.unit_bytes).pbuf_bytes / (size_t(dpad) * 2);
        if (slots > size_t(MAXSLOTS)) slots = MAXSLOTS;
        p.fix_gs = slots >= 6 ? int(slots) / 3 : 1;
        p.fix_ng = int(slots) / p.fix_gs;
        if (p.fix_ng > MAXGROUPS) p.fix_ng = MAXGROUPS;
        placed = true;
        break;
      }
    }
  }
  if (!placed) { delete S; return TARDIS_OK; }
  const int grid = S->grid;

  auto fail = [&](tardis_status_t st) { H->dscratch = S; decode_release(H); return st; };
  size_t tally = 0;
  const size_t pb_bytes = size_t(NT) * p.nkc * p.pbs;
  const size_t yacc_bytes = sizeof(float) * NREP * p.dacc;
  cudaError_t e = dev_malloc(&S->pblocks, pb_bytes); tally += pb_bytes;
  if (e == cudaSuccess) { e = dev_malloc(&S->plan, sizeof(int2) * grid); tally += sizeof(int2) * grid; }
  if (e == cudaSuccess) { e = dev_malloc(&S->smax, 16); tally += 16; }
  if (e == cudaSuccess) { e = dev_malloc(&S->rowexp, sizeof(int) * h); tally += sizeof(int) * h; }
  const size_t cp_bytes = size_t(p.nunits) * 8192;
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
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare"); return fail(TARDIS_ERR_CUDA); }
  k_row_exponent<<<(h + 255) / 256, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->scale), h, H->ngroups, S->rowexp);
  k_pack_pblocks<<<dim3(NT, p.nkc), 128, 0, s>>>(H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero, S->rowexp,
                                                 S->pblocks, d, G, p.nkc, p.pbs);
  k_pack_folded<<<p.nunits, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->C), S->Cp, d, p.nkc);
  k_max_scale<<<64, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->scale), size_t(h) * H->ngroups, S->smax);
  e = cudaGetLastError();
  S->kernel = vpt == 1 ? (G == 64 ? (const void*)k_decode<1, 64> : (const void*)k_decode<1, 128>)
                       : (G == 64 ? (const void*)k_decode<2, 64> : (const void*)k_decode<2, 128>);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(S->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare launch"); return fail(TARDIS_ERR_CUDA); }

  p.pblocks = S->pblocks; p.plan = S->plan; p.smax = S->smax; p.rowexp = S->rowexp; p.yacc = S->yacc; p.ctl = S->ctl;
  p.W1 = static_cast<const __nv_bfloat16*>(H->W1); p.W2T = static_cast<const __nv_bfloat16*>(H->W2T);
  p.Cp = S->Cp; p.bf = H->bf; p.lo = H->lo; p.hi = H->hi; p.a = H->a; p.c = H->c; p.b1 = H->b1;
  p.codes = H->codes; p.scale = static_cast<const __nv_bfloat16*>(H->scale); p.zero = H->zero;
  p.counters = H->counters;
  H->dscratch = S;
  H->dscratch_bytes = S->bytes;
  H->bytes_scratch += S->bytes - pb_bytes - cp_bytes;
  H->bytes_predictor += pb_bytes;
  H->bytes_folded += cp_bytes;
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
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S->grid); cfg.blockDim = dim3(NTH); cfg.dynamicSmemBytes = S->smem_bytes; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    void* args[] = {&p};
    TARDIS_CUDA_TRY(cudaLaunchKernelExC(&cfg, S->kernel, args));
    H->launches += 1;
  }
  return TARDIS_OK;
}

tardis_status_t decode_read_stamps(long long* out, int max_ctas) {
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

void decode_release(Handle* H) {
  Scratch* S = static_cast<Scratch*>(H->dscratch);
  if (!S) return;
  void* ptrs[] = {S->pblocks, S->plan, S->smax, S->yacc, S->ctl, S->rowexp, S->Cp};
  for (void* q : ptrs)
    if (q) dev_free(q);
  delete S;
  H->dscratch = nullptr;
  H->codes_mma = nullptr;
}

}  // namespace tardis
