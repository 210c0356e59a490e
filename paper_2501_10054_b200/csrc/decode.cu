// Fused batch-1 decode kernel of the online path (Section 5.4) for bf16 layers on sm_100a.
//
// One persistent CTA per SM.  A producer warp streams everything the token needs through a
// shared-memory ring with bulk async copies (cp.async.bulk + mbarrier): first the CTA's share
// of the predictor (2-bit codes + group scales, Section 5.3), then rows of the folded matrix
// C = W_f^T, and - as soon as the CTA's flags are known - the gathered W1 rows and W2T rows of
// its flagged neurons.  16 consumer warps
//   * evaluate the predictor score on the integer tensor cores: codes are masked straight out of
//     the packed words (no shifts: the field position is a power-of-4 weight that the operand
//     pre-scaling of x undoes) and multiplied with a 4-limb signed base-256 fixed-point copy of x
//     (mma.m16n8k32.u8.s8, s32 accumulators, exact); group sums are scaled and accumulated in fp64,
//     so the score equals the mathematical one up to the (tracked) truncation of tiny x elements;
//     scores that close to a range end are re-evaluated exactly from the original codes;
//   * flag and compact (ballot + prefix sum), recompute z_j from the gathered W1 rows;
//   * own 8 output columns per thread and add  x_k C[k,:]  and  delta_j W2T[j,:]  into registers.
// CTAs combine with vector float atomics into an fp32 accumulator; the last CTA adds b_f, rounds
// to bf16, and re-zeroes the accumulator for the next call.
#include <stdio.h>

#include <vector>

#include "common.cuh"

namespace tardis {
namespace dec {

constexpr int CW = 16;            // consumer warps
constexpr int CT = CW * 32;       // consumer threads
constexpr int NTHREADS = CT + 32; // + one producer warp
constexpr int KC = 256;           // channels per predictor block
constexpr int MAXFL = 256;        // flagged neurons per CTA (16 tiles x 16)
constexpr int MAXRC = 64;         // exact re-checks per CTA before the list overflows (rest handled in order)
constexpr int MAXROWS = 8;        // rows per ring stage
constexpr uint32_t SPIN_LIMIT = 1u << 24;   // polls of a non-blocking test: a fraction of a second

enum StageType { ST_PRED = 0, ST_C = 1, ST_W1 = 2, ST_W2T = 3, ST_END = 4 };

struct Plan { int tile_begin, tile_count, crow_begin, crow_count; };

struct Params {
  const uint8_t* pblocks;  // [tile][kchunk] predictor blocks
  int pbs, nkc, G;
  const __nv_bfloat16 *W1, *W2T, *C;
  const float *bf, *lo, *hi, *a, *c, *b1;
  const uint32_t* codes; const __nv_bfloat16* scale; const uint8_t* zero;   // originals (exact re-check)
  const float* smax;       // largest group scale of the layer
  const Plan* plan;
  const __nv_bfloat16* x; __nv_bfloat16* y;
  float* yacc; unsigned int* sync; unsigned long long* counters;
  uint32_t* dbg_bitmap; double* dbg_scores;
  int d, dpad, h, ngroups, act;
  int ring, stage_bytes, rows_per_stage, kp, tslots, vpt;
};

struct Scratch {          // handle-owned device memory of the fused path
  uint8_t* pblocks; Plan* plan; float* smax; float* yacc; unsigned int* sync;
  Params base; size_t smem_bytes; size_t bytes;
};

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit ran out (the caller records the error and leaves).
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity) {
  for (uint32_t i = 0; i < SPIN_LIMIT; ++i)
    if (mbar_test(b, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(CT) : "memory"); }
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

// ---- shared-memory carve-up (host and device agree through this) -----------------------------------
struct SmemLayout {
  size_t ring, desc, xq, xs, sxd, zpart, fl_j, fl_delta, wpart, rc, flagbits, score, bars, misc, total;
  __host__ __device__ SmemLayout(const Params& p) {
    size_t o = 0;
    auto take = [&](size_t bytes, size_t align) { o = (o + align - 1) / align * align; size_t r = o; o += bytes; return r; };
    ring = take(size_t(p.ring) * p.stage_bytes, 128);
    desc = take(size_t(p.ring) * 16 * sizeof(int), 16);
    xq = take(size_t(4) * (p.dpad + 64), 128);
    xs = take(size_t(p.d) * sizeof(float), 16);
    sxd = take(size_t(p.ngroups) * sizeof(double), 8);
    zpart = take(size_t(CW) * 16 * sizeof(double), 8);
    fl_j = take(MAXFL * sizeof(int), 4);
    fl_delta = take(MAXFL * sizeof(float), 4);
    wpart = take(size_t(MAXFL) * CW * sizeof(float), 4);
    rc = take(MAXRC * sizeof(int), 4);
    flagbits = take(MAXFL * sizeof(int), 4);
    score = take(MAXFL * sizeof(double), 8);
    bars = take(size_t(2 * p.ring + 1) * sizeof(uint64_t), 8);
    misc = take(32 * sizeof(int), 8);
    total = o;
  }
};
// misc slots
enum { MS_E = 0, MS_NONFINITE = 1, MS_NFL = 2, MS_NRC = 3, MS_ABORT = 4, MS_LAST = 5, MS_TAUBITS = 6, MS_RESID = 7, MS_MAXBITS = 8, MS_WCNT = 16 };

// ---- the kernel ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NTHREADS, 1) k_decode(const Params p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout L(p);
  uint8_t* ring = smem + L.ring;
  int* desc = reinterpret_cast<int*>(smem + L.desc);
  uint8_t* xq = smem + L.xq;
  float* xs = reinterpret_cast<float*>(smem + L.xs);
  double* sxd = reinterpret_cast<double*>(smem + L.sxd);
  double* zpart = reinterpret_cast<double*>(smem + L.zpart);
  int* fl_j = reinterpret_cast<int*>(smem + L.fl_j);
  float* fl_delta = reinterpret_cast<float*>(smem + L.fl_delta);
  float* wpart = reinterpret_cast<float*>(smem + L.wpart);
  int* rc = reinterpret_cast<int*>(smem + L.rc);
  int* flagbits = reinterpret_cast<int*>(smem + L.flagbits);
  double* score = reinterpret_cast<double*>(smem + L.score);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
  uint64_t* empty = full + p.ring;
  uint64_t* flags_ready = empty + p.ring;
  volatile int* misc = reinterpret_cast<volatile int*>(smem + L.misc);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Plan plan = p.plan[blockIdx.x];
  const int d = p.d, row_bytes = 2 * d;
  const int xq_stride = p.dpad + 64;

  if (tid == 0) {
    for (int i = 0; i < p.ring; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], CW); }
    mbar_init(flags_ready, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < 32; ++i) misc[i] = 0;
  }
  for (int g = tid; g < p.ngroups; g += NTHREADS) sxd[g] = 0.0;
  __syncthreads();

  // =========================== producer warp ===========================
  if (warp == CW) {
    if (lane != 0) return;
    int stage = 0;
    bool ok = true;
    auto acquire = [&](int& slot) -> bool {
      slot = stage % p.ring;
      const uint32_t par = ((stage / p.ring) & 1) ^ 1;
      if (!mbar_wait(&empty[slot], par)) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ABORT] = 1; return false; }
      return !misc[MS_ABORT];
    };
    auto emit_rows = [&](int type, const __nv_bfloat16* base, const int* ids, int first, int count, bool ids_are_list) -> bool {
      // rows base[id * d ...]; ids: consecutive from `first` (ids == nullptr) or fl_j[first + r]
      int slot;
      if (!acquire(slot)) return false;
      int* ds = desc + slot * 16;
      ds[0] = type; ds[1] = count; ds[2] = first;
      mbar_expect_tx(&full[slot], uint32_t(count) * row_bytes);
      for (int r = 0; r < count; ++r) {
        const int id = ids_are_list ? ids[first + r] : first + r;
        bulk_g2s(ring + size_t(slot) * p.stage_bytes + size_t(r) * row_bytes, base + size_t(id) * d, row_bytes, &full[slot]);
      }
      ++stage;
      return true;
    };
    auto emit_fix = [&]() -> bool {
      const int nfl = misc[MS_NFL];
      for (int e = 0; e < nfl && ok; e += p.rows_per_stage)
        ok = emit_rows(ST_W1, p.W1, fl_j, e, min(p.rows_per_stage, nfl - e), true);
      for (int e = 0; e < nfl && ok; e += p.rows_per_stage)
        ok = emit_rows(ST_W2T, p.W2T, fl_j, e, min(p.rows_per_stage, nfl - e), true);
      return ok;
    };
    // 1. predictor stages
    const int npred = plan.tile_count > 0 ? (p.nkc + p.kp - 1) / p.kp : 0;
    for (int s = 0; s < npred && ok; ++s) {
      int slot;
      if (!(ok = acquire(slot))) break;
      int* ds = desc + slot * 16;
      ds[0] = ST_PRED; ds[1] = s;
      uint32_t bytes = 0;
      for (int ph = 0; ph < p.kp; ++ph)
        if (s * p.kp + ph < p.nkc) bytes += uint32_t(plan.tile_count) * p.pbs;
      mbar_expect_tx(&full[slot], bytes);
      for (int ph = 0; ph < p.kp; ++ph) {
        const int kc = s * p.kp + ph;
        if (kc >= p.nkc) continue;
        for (int t = 0; t < plan.tile_count; ++t)
          bulk_g2s(ring + size_t(slot) * p.stage_bytes + size_t(ph * p.tslots + t) * p.pbs,
                   p.pblocks + (size_t(plan.tile_begin + t) * p.nkc + kc) * p.pbs, p.pbs, &full[slot]);
      }
      ++stage;
    }
    // 2. folded-matrix rows; the flagged rows are slotted in as soon as the flags exist
    bool fixed = false;
    for (int r = 0; r < plan.crow_count && ok; r += p.rows_per_stage) {
      if (!fixed && mbar_test(flags_ready, 0)) { ok = emit_fix(); fixed = true; if (!ok) break; }
      ok = emit_rows(ST_C, p.C, nullptr, plan.crow_begin + r, min(p.rows_per_stage, plan.crow_count - r), false);
    }
    if (ok && !fixed) {
      if (!mbar_wait(flags_ready, 0)) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ABORT] = 1; ok = false; }
      else ok = emit_fix();
    }
    // 3. end marker
    if (ok) {
      int slot;
      if (acquire(slot)) { desc[slot * 16] = ST_END; mbar_arrive(&full[slot]); ++stage; }
    }
    // Leave only when every copy this warp issued has landed (bounded).
    if (!ok) {
      for (int i = 0; i < p.ring; ++i) {
        const int s = stage - 1 - i;
        if (s < 0) break;
        mbar_wait(&full[s % p.ring], (s / p.ring) & 1);
      }
    }
    return;
  }

  // =========================== consumer warps ===========================
  const __nv_bfloat16* xg = p.x;
  // ---- x -> fp32 copy, max |x| ----
  float amax = 0.f;
  bool nonfinite = false;
  for (int k = tid; k < d; k += CT) {
    const float v = __bfloat162float(xg[k]);
    xs[k] = v;
    if (!(fabsf(v) <= 3.0e38f)) nonfinite = true;
    amax = fmaxf(amax, fabsf(v));
  }
  amax = fmaxf(amax, 0.f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) atomicMax(const_cast<int*>(&misc[MS_MAXBITS]), __float_as_int(amax));
  if (nonfinite) misc[MS_NONFINITE] = 1;
  consumer_sync();
  const bool tok_nonfinite = misc[MS_NONFINITE] != 0;
  // exponent E: |x| 2^-E < 2^24 for every element
  int E = 0;
  {
    const float m = __int_as_float(misc[MS_MAXBITS]);
    if (m > 0.f && !tok_nonfinite) E = max(int((__float_as_uint(m) >> 23) & 0xff) - 127 - 23, -100);
  }
  // ---- fixed-point limbs of x in tensor-core operand order; group sums; truncation residual ----
  {
    const float inv = __uint_as_float(uint32_t(127 - E) << 23);    // 2^-E (E in [-149, 104] -> representable when 127-E in 1..254)
    float resid = 0.f;
    const int units = p.dpad / 16;
    for (int u = tid; u < units; u += CT) {
      uint32_t limb[4][4] = {};   // [limb][field] words, byte i = channel 4 i + field
      int sx = 0;
      const int k0 = u * 16;
      if (!tok_nonfinite) {
#pragma unroll
        for (int cidx = 0; cidx < 16; ++cidx) {
          const int k = k0 + cidx;
          const float v = (k < d) ? xs[k] * inv : 0.f;
          const int X = __float2int_rz(v);
          resid += fabsf(v - float(X));
          sx += X;
          const int f = cidx & 3, i = cidx >> 2;
          int Y = X << (2 * (3 - f));
#pragma unroll
          for (int l = 0; l < 4; ++l) {
            const int dig = int(int8_t(Y & 0xff));   // signed low byte
            Y = (Y - dig) >> 8;
            limb[l][f] |= uint32_t(dig & 0xff) << (8 * i);
          }
        }
      }
      const int kb = u >> 2, t = u & 3;
#pragma unroll
      for (int l = 0; l < 4; ++l)
        *reinterpret_cast<uint4*>(xq + size_t(l) * xq_stride + size_t(kb) * 64 + t * 16) =
            make_uint4(limb[l][0], limb[l][1], limb[l][2], limb[l][3]);
      if (k0 < d) atomicAdd(&sxd[k0 / p.G], double(sx));   // integer-valued, exact in any order
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) resid += __shfl_xor_sync(0xffffffffu, resid, o);
    if (lane == 0 && resid > 0.f) atomicAdd(const_cast<int*>(&misc[MS_RESID]), __float2int_ru(resid * 1048576.f));   // 2^-20 units, rounded up
  }
  consumer_sync();
  // tolerance of the fast score: every dropped fraction (< 1 unit of 2^E) times |code - zero| <= 3 times the scale
  const double tau = double(misc[MS_RESID]) * (1.0 / 1048576.0) * 3.0 * double(*p.smax) * ldexp(1.0, E);

  // ---- per-thread state ----
  const int g = lane >> 2, t4 = lane & 3;
  const int tslot = warp % p.tslots, phase = warp / p.tslots;
  const bool pred_warp = tslot < plan.tile_count && phase < p.kp;
  double zacc[4] = {0.0, 0.0, 0.0, 0.0}, zt[2] = {0.0, 0.0};
  float acc[2][8];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[m][i] = 0.f;
  bool pred_done = false, delta_done = false;
  int nfl = 0;

  const int npred = plan.tile_count > 0 ? (p.nkc + p.kp - 1) / p.kp : 0;   // same count the producer issues

  for (int stage = 0;; ++stage) {
    if (stage == npred && !pred_done) {
      // ================= predictor epilogue: scores, flags, compaction =================
      pred_done = true;
      if (pred_warp) {
        // limbs: lane t4 = 0 holds limbs 0,1 ; t4 = 1 holds limbs 2,3 (columns 4..7 are unused for one token)
        double v0 = 0.0, v1 = 0.0;
        if (t4 == 0) { v0 = zacc[0] + 256.0 * zacc[1]; v1 = zacc[2] + 256.0 * zacc[3]; }
        if (t4 == 1) { v0 = 65536.0 * (zacc[0] + 256.0 * zacc[1]); v1 = 65536.0 * (zacc[2] + 256.0 * zacc[3]); }
        v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
        if (t4 == 0) {
          zpart[(phase * p.tslots + tslot) * 16 + g] = v0 * (1.0 / 64.0) - zt[0];
          zpart[(phase * p.tslots + tslot) * 16 + g + 8] = v1 * (1.0 / 64.0) - zt[1];
        }
      }
      consumer_sync();
      const int nrow = plan.tile_count * 16;
      if (tid < nrow) {
        const int tl = tid >> 4, r = tid & 15;
        const int j = (plan.tile_begin + tl) * 16 + r;
        double s = 0.0;
        for (int ph = 0; ph < p.kp; ++ph) s += zpart[(ph * p.tslots + tl) * 16 + r];
        const double zhat = double(p.b1[j]) + ldexp(s, E);
        const double lo = double(p.lo[j]), hi = double(p.hi[j]);
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
      consumer_sync();
      // exact re-evaluation from the original codes (rare): one warp per listed neuron
      {
        const int nrc = min(int(misc[MS_NRC]), MAXRC);
        const int nwords = d / 16;
        for (int e = warp; e < nrc; e += CW) {
          const int n = rc[e];
          const int j = (plan.tile_begin + (n >> 4)) * 16 + (n & 15);
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
        if (lane == 0 && warp == 0 && nrc > 0) atomicAdd(&p.counters[CTR_RECHECKS], (unsigned long long)nrc);
      }
      consumer_sync();
      // ascending flagged list: ballot + prefix over the (at most 8) warps that hold rows
      {
        const int f = (tid < nrow) ? (flagbits[tid] & 1) : 0;
        const uint32_t bal = __ballot_sync(0xffffffffu, f != 0);
        if (lane == 0) misc[MS_WCNT + warp] = __popc(bal);
        consumer_sync();
        int base = 0;
        for (int w = 0; w < warp; ++w) base += misc[MS_WCNT + w];
        if (f) fl_j[base + __popc(bal & ((1u << lane) - 1u))] = (plan.tile_begin + (tid >> 4)) * 16 + (tid & 15);
        if (tid == 0) {
          int total = 0;
          for (int w = 0; w < CW; ++w) total += misc[MS_WCNT + w];
          misc[MS_NFL] = total;
        }
        // debug capture: 16-bit halves of the flag words, scores
        if (p.dbg_bitmap && tid < nrow && (tid & 15) == 0)
          reinterpret_cast<uint16_t*>(p.dbg_bitmap)[plan.tile_begin + (tid >> 4)] = uint16_t((bal >> (lane & 16)) & 0xffffu);
        if (p.dbg_scores && tid < nrow) p.dbg_scores[(plan.tile_begin + (tid >> 4)) * 16 + (tid & 15)] = score[tid];
      }
      consumer_sync();
      nfl = misc[MS_NFL];
      if (tid == 0) mbar_arrive(flags_ready);
    }

    const int slot = stage % p.ring;
    if (!mbar_wait(&full[slot], (stage / p.ring) & 1)) { atomicExch(&p.counters[CTR_ERROR], 1ull); misc[MS_ABORT] = 1; return; }
    const int* ds = desc + slot * 16;
    const int type = ds[0];
    const uint8_t* sbase = ring + size_t(slot) * p.stage_bytes;
    if (type == ST_END) break;

    if (type == ST_PRED) {
      if (pred_warp) {
        const int kc = ds[1] * p.kp + phase;
        if (kc < p.nkc) {
          const uint8_t* blk = sbase + size_t(phase * p.tslots + tslot) * p.pbs;
          const uint4* cp = reinterpret_cast<const uint4*>(blk);
          const uint2* mp = reinterpret_cast<const uint2*>(blk + 1024);
          const int kb_per_group = p.G / 64;
          int ia[4] = {0, 0, 0, 0};
#pragma unroll
          for (int pair = 0; pair < 2; ++pair) {
            const uint4 cw = cp[pair * 32 + lane];
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
                const uint2 mw = mp[gl * 8 + g];
                const double s0 = double(bf_hi(mw.x)), s1 = double(bf_hi(mw.y));
                zacc[0] += s0 * double(ia[0]); zacc[1] += s0 * double(ia[1]);
                zacc[2] += s1 * double(ia[2]); zacc[3] += s1 * double(ia[3]);
                const double sx = sxd[min(kb / kb_per_group, p.ngroups - 1)];
                zt[0] += s0 * double(mw.x & 3u) * sx;
                zt[1] += s1 * double(mw.y & 3u) * sx;
                ia[0] = ia[1] = ia[2] = ia[3] = 0;
              }
            }
          }
        }
      }
    } else if (type == ST_W1) {
      const int cnt = ds[1], first = ds[2];
      for (int r = 0; r < cnt; ++r) {
        const uint8_t* row = sbase + size_t(r) * row_bytes;
        float part = 0.f;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          const int v = tid + m * CT;
          if (m < p.vpt && v * 8 < d) {
            const uint4 w = *reinterpret_cast<const uint4*>(row + size_t(v) * 16);
            const float* xv = xs + v * 8;
            part += bf_lo(w.x) * xv[0] + bf_hi(w.x) * xv[1] + bf_lo(w.y) * xv[2] + bf_hi(w.y) * xv[3] +
                    bf_lo(w.z) * xv[4] + bf_hi(w.z) * xv[5] + bf_lo(w.w) * xv[6] + bf_hi(w.w) * xv[7];
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if (lane == 0) wpart[(first + r) * CW + warp] = part;
      }
    } else {   // ST_C or ST_W2T: scaled row accumulation into the owned columns
      if (type == ST_W2T && !delta_done) {
        delta_done = true;
        consumer_sync();
        if (tid < nfl) {
          const int j = fl_j[tid];
          float z = 0.f;
          for (int w = 0; w < CW; ++w) z += wpart[tid * CW + w];
          z += p.b1[j];
          fl_delta[tid] = gelu_f32(z, p.act) - p.a[j] * z - p.c[j];
        }
        consumer_sync();
      }
      const int cnt = ds[1], first = ds[2];
      for (int r = 0; r < cnt; ++r) {
        const uint8_t* row = sbase + size_t(r) * row_bytes;
        const float sc = (type == ST_C) ? xs[first + r] : fl_delta[first + r];
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          const int v = tid + m * CT;
          if (m < p.vpt && v * 8 < d) {
            const uint4 w = *reinterpret_cast<const uint4*>(row + size_t(v) * 16);
            acc[m][0] += sc * bf_lo(w.x); acc[m][1] += sc * bf_hi(w.x);
            acc[m][2] += sc * bf_lo(w.y); acc[m][3] += sc * bf_hi(w.y);
            acc[m][4] += sc * bf_lo(w.z); acc[m][5] += sc * bf_hi(w.z);
            acc[m][6] += sc * bf_lo(w.w); acc[m][7] += sc * bf_hi(w.w);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[slot]);
  }

  // =========================== epilogue ===========================
#pragma unroll
  for (int m = 0; m < 2; ++m) {
    const int v = tid + m * CT;
    if (m < p.vpt && v * 8 < d) {
      red_add_v4(p.yacc + v * 8, acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
      red_add_v4(p.yacc + v * 8 + 4, acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
    }
  }
  __threadfence();
  consumer_sync();
  if (tid == 0) {
    if (nfl) atomicAdd(&p.sync[1], (unsigned int)nfl);
    __threadfence();
    const unsigned int ticket = atomicAdd(&p.sync[0], 1u);
    misc[MS_LAST] = (ticket == gridDim.x - 1) ? 1 : 0;
  }
  consumer_sync();
  if (misc[MS_LAST]) {
    __threadfence();
    for (int v = tid; v * 8 < d; v += CT) {
      const float4 a0 = __ldcg(reinterpret_cast<const float4*>(p.yacc + v * 8));
      const float4 a1 = __ldcg(reinterpret_cast<const float4*>(p.yacc + v * 8 + 4));
      const float4 b0 = *reinterpret_cast<const float4*>(p.bf + v * 8);
      const float4 b1v = *reinterpret_cast<const float4*>(p.bf + v * 8 + 4);
      __nv_bfloat162 o[4];
      o[0] = __floats2bfloat162_rn(a0.x + b0.x, a0.y + b0.y);
      o[1] = __floats2bfloat162_rn(a0.z + b0.z, a0.w + b0.w);
      o[2] = __floats2bfloat162_rn(a1.x + b1v.x, a1.y + b1v.y);
      o[3] = __floats2bfloat162_rn(a1.z + b1v.z, a1.w + b1v.w);
      *reinterpret_cast<uint4*>(p.y + v * 8) = *reinterpret_cast<const uint4*>(o);
      *reinterpret_cast<float4*>(p.yacc + v * 8) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(p.yacc + v * 8 + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (tid == 0) {
      const unsigned int total = atomicExch(&p.sync[1], 0u);
      atomicAdd(&p.counters[CTR_FLAGGED_TOTAL], (unsigned long long)total);
      atomicMax(&p.counters[CTR_FLAGGED_MAX], (unsigned long long)total);
      __threadfence();
      atomicExch(&p.sync[0], 0u);
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
  const int n = H->num_sms;
  const int NT = h / 16;
  const int tslots = (NT + n - 1) / n;
  if (tslots > 16 || d > 2 * CT * 8 || d < 64) return TARDIS_OK;
  Scratch* S = new (std::nothrow) Scratch();
  if (!S) return TARDIS_ERR_ALLOC;
  memset(S, 0, sizeof(*S));
  Params& p = S->base;
  p.d = d; p.h = h; p.G = G; p.ngroups = H->ngroups; p.act = H->act;
  p.dpad = (d + KC - 1) / KC * KC;
  p.nkc = p.dpad / KC;
  p.pbs = 1024 + 64 * (KC / G);
  p.tslots = tslots;
  p.kp = CW / tslots < p.nkc ? CW / tslots : p.nkc;
  p.vpt = (d / 8 + CT - 1) / CT;
  const int row_bytes = 2 * d;
  int R = 18432 / row_bytes;
  R = R < 1 ? 1 : (R > MAXROWS ? MAXROWS : R);
  p.rows_per_stage = R;
  const int pred_bytes = tslots * p.kp * p.pbs;
  p.stage_bytes = ((pred_bytes > R * row_bytes ? pred_bytes : R * row_bytes) + 127) / 128 * 128;
  int max_smem = 0;
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, H->device));
  p.ring = 12;
  while (p.ring > 2 && SmemLayout(p).total > size_t(max_smem)) --p.ring;
  if (SmemLayout(p).total > size_t(max_smem)) { delete S; return TARDIS_OK; }
  S->smem_bytes = SmemLayout(p).total;

  auto fail = [&](tardis_status_t st) { H->dscratch = S; decode_release(H); return st; };
  size_t tally = 0;
  const size_t pb_bytes = size_t(NT) * p.nkc * p.pbs;
  cudaError_t e = cudaMalloc(&S->pblocks, pb_bytes); tally += pb_bytes;
  if (e == cudaSuccess) { e = cudaMalloc(&S->plan, sizeof(Plan) * n); tally += sizeof(Plan) * n; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->smax, 16); tally += 16; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->yacc, sizeof(float) * d); tally += sizeof(float) * d; }
  if (e == cudaSuccess) { e = cudaMalloc(&S->sync, 16); tally += 16; }
  if (e != cudaSuccess) { set_last_error(e, "cudaMalloc"); cudaGetLastError(); return fail(TARDIS_ERR_ALLOC); }
  S->bytes = tally;

  // byte-balanced static plan: tiles spread evenly, folded-matrix rows fill each CTA up to the mean
  std::vector<Plan> plan(n);
  const double tb = double(p.nkc) * p.pbs, rb = double(row_bytes);
  const double target = (double(NT) * tb + double(d) * rb) / n;
  int tile_cum = 0, row_cum = 0;
  for (int c = 0; c < n; ++c) {
    const int tc = NT / n + (c < NT % n ? 1 : 0);
    plan[c].tile_begin = tile_cum; plan[c].tile_count = tc; tile_cum += tc;
    double want = (target * (c + 1) - tb * tile_cum) / rb;
    int upto = c == n - 1 ? d : int(want + 0.5);
    upto = upto < row_cum ? row_cum : (upto > d ? d : upto);
    plan[c].crow_begin = row_cum; plan[c].crow_count = upto - row_cum; row_cum = upto;
  }
  e = cudaMemcpyAsync(S->plan, plan.data(), sizeof(Plan) * n, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);   // plan.data() is a stack-owned host buffer
  if (e == cudaSuccess) e = cudaMemsetAsync(S->smax, 0, 16, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(S->yacc, 0, sizeof(float) * d, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(S->sync, 0, 16, s);
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare"); return fail(TARDIS_ERR_CUDA); }
  k_pack_pblocks<<<dim3(NT, p.nkc), 128, 0, s>>>(H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero,
                                                 S->pblocks, d, h, G, p.nkc, p.pbs);
  k_max_scale<<<64, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(H->scale), size_t(h) * H->ngroups, S->smax);
  e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_decode, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S->smem_bytes));
  if (e != cudaSuccess) { set_last_error(e, "decode_prepare launch"); return fail(TARDIS_ERR_CUDA); }

  p.pblocks = S->pblocks; p.plan = S->plan; p.smax = S->smax; p.yacc = S->yacc; p.sync = S->sync;
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
    k_decode<<<H->num_sms, NTHREADS, S->smem_bytes, s>>>(p);
    H->launches += 1;
  }
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

void decode_release(Handle* H) {
  Scratch* S = static_cast<Scratch*>(H->dscratch);
  if (!S) return;
  void* ptrs[] = {S->pblocks, S->plan, S->smax, S->yacc, S->sync};
  for (void* q : ptrs)
    if (q) cudaFree(q);
  delete S;
  H->dscratch = nullptr;
  H->codes_mma = nullptr;
}

}  // namespace tardis
