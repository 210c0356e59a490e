// bf16 GEMM on the 5th-generation tensor cores (see gemm.cuh for what it computes).
//
// A CTA computes 128 x BN tiles of the output, one after the other (persistent, one CTA per SM).  Warp 0 stages
// 128 x 64 (A) and BN x 64 (B) operand boxes into a ring of shared-memory stages with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, no multicast); warp 1 issues tcgen05.mma (M = 128, N = BN,
// K = 16 per instruction) from one thread, accumulating in tensor memory (TMEM, 128 lanes x BN fp32 columns,
// two accumulators used in turn) and releasing each stage with tcgen05.commit; warps 2..5 read a finished
// accumulator back with tcgen05.ld (each warp its own 32 lanes) and run the epilogue while the next tile's
// main loop fills the other accumulator.  Every wait on an mbarrier is bounded: when it runs out the waiter
// sets an error word and the CTA falls through to the end, where TMEM is released.
#include "gemm.cuh"

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdio.h>

#include "common.cuh"
#include "exact.cuh"

namespace tardis {
namespace gemm {

constexpr int BM = 128;                 // tile rows (tokens / outputs)
constexpr int BK = 64;                  // channels per stage: 64 bf16 = one 128-byte swizzle row
constexpr int NTHREADS = 192;           // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr uint32_t SPIN_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity) {   // bounded
  for (uint32_t i = 0; i < SPIN_LIMIT; ++i) {
    if (mbar_test(b, parity)) return true;
    if (i > 64) __nanosleep(32);
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, M = 128, N from the instruction descriptor, K = 16
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The barrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 64 bf16 (128 bytes) with the
// 128-byte swizzle TMA applies: start address (>> 4), leading-dimension offset (unused for this layout, 1),
// stride between 8-row groups = 1024 bytes (>> 4), descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFFu) >> 4);
  d |= uint64_t(1) << 16;
  d |= uint64_t(1024 >> 4) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, both K-major, N and M of the tile.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(N >> 3) << 17) | (uint32_t(M >> 4) << 24);
}

struct KParams {
  int M, N, kb1, kb2;          // k blocks (of 64) of the two operand pairs
  int epilogue, ldo, act, splits;
  int fast_m, band;            // tile raster (see decode() in the kernel)
  float* out_f32; __nv_bfloat16* out_bf16;
  const float *bias, *addend, *a, *c;
  const uint32_t* bitmap;
  unsigned long long* error_word;
  const float *lo, *hi, *colscale, *rowscale;
  float keps;
  uint32_t* bitmap_out;
  uint2* rlist; unsigned int* rcount; int rcap;
  const uint32_t* codes; const __nv_bfloat16* scale; const uint8_t* zero;
  const __nv_bfloat16* xsrc; int d, G, bits;
};

template <int BN> struct Cfg {
  static constexpr int STAGE_BYTES = BM * BK * 2 + BN * BK * 2;
  static constexpr int NS = (BN == 256) ? 4 : 6;                      // stages
  static constexpr int SMEM = NS * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */ + 4 * 4096 /* epilogue staging */;
  static constexpr int TMEM_COLS = 2 * BN;                            // two accumulators
};

// The epilogue of 32 consecutive columns n .. n + nv - 1 of output row m (one thread).
// A&S 7.1.26 form of erf (absolute error below 2e-7, far inside the bf16 rounding of the correction it feeds)
__device__ __forceinline__ float gelu_quick(float z, int act) {
  if (act != TARDIS_ACT_GELU_ERF) return gelu_f32(z, act);
  const float x = fabsf(z) * 0.7071067811865476f;
  const float t = __fdividef(1.f, fmaf(0.3275911f, x, 1.f));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float e = 1.f - poly * t * __expf(-x * x);          // erf(|z| / sqrt 2)
  return 0.5f * z * (1.f + copysignf(e, z));
}

// `stage`: 32 x 32 floats of shared memory of the calling warp (element [i][lane]).
__device__ __forceinline__ void epilogue_chunk(const KParams& p, float (&v)[32], int m, int n, int nv, bool first_split, bool have_acc,
                                               float* stage, int lane) {
  if (p.epilogue == GEMM_EPI_FLAGS) {
    const float xn = p.rowscale[m];
    const uint32_t valid = nv == 32 ? 0xffffffffu : ((1u << nv) - 1u);
    uint32_t word = valid;                                   // a non-finite token: every neuron flagged
    if (xn <= 3.0e38f) {
      const float kx = p.keps * xn;
      word = 0u;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        if (i < nv) {
          const float z = v[i] + p.bias[n + i], l = p.lo[n + i], u = p.hi[n + i];
          const float tau = fmaf(p.colscale[n + i], kx, 1e-30f);
          bool flag = !((l <= z) && (z < u));
          if (fabsf(z - l) <= tau || fabsf(z - u) <= tau) {  // rare
            const unsigned int slot = atomicAdd(&p.rcount[0], 1u);
            if (slot < (unsigned int)p.rcap) p.rlist[slot] = make_uint2((unsigned int)m, (unsigned int)(n + i));
            else {                                           // queue full: settle this one here (slow, but exact)
              const double ze = exact_score_single(p.codes, p.scale, p.zero, p.xsrc + size_t(m) * p.d, n + i, p.d, p.G, p.bits) + double(p.bias[n + i]);
              flag = !((double(l) <= ze) && (ze < double(u)));
              atomicAdd(&p.rcount[1], 1u);
            }
          }
          word |= (flag ? 1u : 0u) << i;
          v[i] = z;
        }
      }
    }
    p.bitmap_out[size_t(m) * (p.N / 32) + (n >> 5)] = word;
    if (p.out_f32) {
      float* o = p.out_f32 + size_t(m) * p.ldo + n;
      if (nv == 32 && (p.ldo & 3) == 0) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(o + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
      } else {
        for (int i = 0; i < nv; ++i) o[i] = v[i];
      }
    }
    return;
  }
  if (p.epilogue == GEMM_EPI_F32 && p.splits > 1) {
    float* o = p.out_f32 + size_t(m) * p.ldo + n;
    const bool with_bias = p.bias && first_split;
    if (have_acc || with_bias) {
      if (nv == 32 && (p.ldo & 3) == 0) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          float4 t = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          if (with_bias) { t.x += p.bias[n + i]; t.y += p.bias[n + i + 1]; t.z += p.bias[n + i + 2]; t.w += p.bias[n + i + 3]; }
          asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(o + i), "f"(t.x), "f"(t.y), "f"(t.z), "f"(t.w) : "memory");
        }
      } else {
        for (int i = 0; i < nv; ++i) atomicAdd(o + i, v[i] + (with_bias ? p.bias[n + i] : 0.f));
      }
    }
  } else if (p.epilogue == GEMM_EPI_F32) {
    float* o = p.out_f32 + size_t(m) * p.ldo + n;
    if (nv == 32 && (p.ldo & 3) == 0) {
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        float4 t = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        if (p.bias) { t.x += p.bias[n + i]; t.y += p.bias[n + i + 1]; t.z += p.bias[n + i + 2]; t.w += p.bias[n + i + 3]; }
        *reinterpret_cast<float4*>(o + i) = t;
      }
    } else {
      for (int i = 0; i < nv; ++i) o[i] = v[i] + (p.bias ? p.bias[n + i] : 0.f);
    }
  } else {
    // bf16 outputs: this thread's 32 values become four 16-byte stores
    if (p.epilogue == GEMM_EPI_ADD_BF16) {
      const float* ad = p.addend + size_t(m) * p.ldo + n;
      if (nv == 32 && (p.ldo & 3) == 0) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 t = *reinterpret_cast<const float4*>(ad + i);
          v[i] += t.x; v[i + 1] += t.y; v[i + 2] += t.z; v[i + 3] += t.w;
        }
      } else {
        for (int i = 0; i < nv; ++i) v[i] += ad[i];
      }
    } else {   // GEMM_EPI_DELTA: one flag word covers this thread's 32 columns
      // Only the flagged tenth of the elements needs the activation, at different columns in every row: the
      // accumulators go to shared memory, each thread walks the set bits of its own word, and the corrections come
      // back under the word's mask.
      uint32_t word = p.bitmap[size_t(m) * (p.N / 32) + (n >> 5)];
      if (nv < 32) word &= (1u << nv) - 1u;
#pragma unroll
      for (int i = 0; i < 32; ++i) stage[i * 32 + lane] = v[i];
      for (uint32_t w = word; w; w &= w - 1u) {
        const int i = __ffs(w) - 1;
        const float z = stage[i * 32 + lane] + (p.bias ? p.bias[n + i] : 0.f);
        stage[i * 32 + lane] = gelu_quick(z, p.act) - p.a[n + i] * z - p.c[n + i];
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = ((word >> i) & 1u) ? stage[i * 32 + lane] : 0.f;
    }
    __nv_bfloat16* o = p.out_bf16 + size_t(m) * p.ldo + n;
    if (nv == 32 && (p.ldo & 7) == 0) {
#pragma unroll
      for (int i = 0; i < 32; i += 8) {
        __nv_bfloat162 h[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) h[q] = __floats2bfloat162_rn(v[i + 2 * q], v[i + 2 * q + 1]);
        *reinterpret_cast<uint4*>(o + i) = *reinterpret_cast<const uint4*>(h);
      }
    } else {
      for (int i = 0; i < nv; ++i) o[i] = __float2bfloat16_rn(v[i]);
    }
  }
}

// Persistent: CTA c works on tiles c, c + gridDim.x, ... of a banded raster.  Two accumulators in tensor memory:
// while the epilogue warps drain one, the MMA warp is already filling the other with the next tile.
template <int BN>
__global__ void __launch_bounds__(NTHREADS, 1)
k_gemm(const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
       const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2, const KParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::NS * C::STAGE_BYTES);
  uint64_t* empty = full + C::NS;
  uint64_t* accum_full = empty + C::NS;        // [2]
  uint64_t* accum_empty = accum_full + 2;      // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_empty + 2);
  volatile uint32_t* failed = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nm = (p.M + BM - 1) / BM, nn = (p.N + BN - 1) / BN;
  const int ntiles = nm * nn * p.splits;
  const int nkb_all = p.kb1 + p.kb2;
  const int per = (nkb_all + p.splits - 1) / p.splits;   // k blocks per split of the channel range

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&accum_full[b], 1); mbar_init(&accum_empty[b], 4); }
    *failed = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA1) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB1) : "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);  // the whole warp; a power of two >= 32 fp32 columns
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // tile -> first row, first column, k-block range
  auto decode = [&](int tile, int& m0, int& n0, int& kb_lo, int& nkb, int& z) {
    z = tile / (nm * nn);
    const int rem = tile - z * (nm * nn);
    // raster: bands of `band` tiles along the dimension with fewer tiles, walked across the other dimension, so
    // that the CTAs running at the same time cover a compact block and share its operand tiles in L2
    const int F = p.fast_m ? nm : nn, S = p.fast_m ? nn : nm;
    const int bi = rem / (p.band * S), r2 = rem - bi * (p.band * S);
    const int w = min(p.band, F - bi * p.band);
    const int slow = r2 / w, fast = bi * p.band + (r2 - slow * w);
    const int mi = p.fast_m ? fast : slow, ni = p.fast_m ? slow : fast;
    m0 = mi * BM; n0 = ni * BN;
    kb_lo = z * per;
    nkb = max(0, min(nkb_all, kb_lo + per) - kb_lo);
  };

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;                                 // k blocks staged so far (over all tiles)
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
        int m0, n0, kb_lo, nkb, z;
        decode(tile, m0, n0, kb_lo, nkb, z);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % C::NS;
          if (*failed || !mbar_wait(&empty[s], ((it / C::NS) & 1) ^ 1)) { *failed = 1u; ok = false; break; }
          uint8_t* sa = smem + s * C::STAGE_BYTES;
          uint8_t* sb = sa + BM * BK * 2;
          mbar_expect_tx(&full[s], C::STAGE_BYTES);
          const int kg = kb_lo + kb;                   // k block in the whole channel range
          const bool second = kg >= p.kb1;
          const int kx = (second ? kg - p.kb1 : kg) * BK;
          tma_load_2d(sa, second ? &tmA2 : &tmA1, kx, m0, &full[s]);
          tma_load_2d(sb, second ? &tmB2 : &tmB1, kx, n0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(BM, BN);
      uint32_t it = 0, use = 0;                        // k blocks consumed; accumulator uses so far
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
        int m0, n0, kb_lo, nkb, z;
        decode(tile, m0, n0, kb_lo, nkb, z);
        if (nkb == 0) continue;                        // nothing to add: the epilogue takes zeros
        const uint32_t ab = use & 1u;
        // the epilogue warps have drained this accumulator's previous tile
        if (*failed || !mbar_wait(&accum_empty[ab], ((use >> 1) & 1) ^ 1)) { *failed = 1u; ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + ab * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % C::NS;
          if (!mbar_wait(&full[s], (it / C::NS) & 1)) { *failed = 1u; ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * C::STAGE_BYTES);
          const uint32_t sb = sa + BM * BK * 2;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t adesc = smem_desc_k_major_sw128(sa + k * 32);
            const uint64_t bdesc = smem_desc_k_major_sw128(sb + k * 32);
            umma_f16(tacc, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty[s]);                      // frees the stage when these MMAs have read it
        }
        if (ok) umma_commit(&accum_full[ab]);          // accumulator complete
        ++use;
      }
    }
  } else {
    // ---------------- epilogue: warp q reads TMEM lanes 32 (warp % 4) .. + 31 ----------------
    const int q = warp & 3;
    float* const stage = reinterpret_cast<float*>(smem + C::NS * C::STAGE_BYTES + 256) + q * 1024;
    uint32_t use = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
      int m0, n0, kb_lo, nkb, z;
      decode(tile, m0, n0, kb_lo, nkb, z);
      const int m = m0 + q * 32 + lane;
      const uint32_t ab = use & 1u;
      if (nkb > 0) {
        ok = !*failed && mbar_wait(&accum_full[ab], (use >> 1) & 1);
        if (!ok) { *failed = 1u; break; }
        tc_fence_after();
      }
      for (int ch = 0; ch < BN / 32; ++ch) {
        float v[32];
        if (nkb > 0) tmem_ld32(tmem_base + ab * BN + (uint32_t(q * 32) << 16) + uint32_t(ch * 32), v);
        else {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;
        }
        const int n = n0 + ch * 32;
        const int nv = min(32, p.N - n);
        if (m < p.M && nv > 0) epilogue_chunk(p, v, m, n, nv, z == 0, nkb > 0, stage, lane);   // (no early exit: tcgen05.ld needs the whole warp)
      }
      if (nkb > 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&accum_empty[ab]);  // this warp's lanes of the accumulator may be overwritten
        ++use;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *failed && p.error_word) atomicExch(p.error_word, 1ull);
  if (warp == 1) tmem_dealloc(tmem_base, C::TMEM_COLS);
}

// ---- host side ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      cudaGetLastError();
  }
  return fn;
}

// [rows, K] bf16 row-major with leading dimension ld; box = 64 channels x box_rows rows, 128-byte swizzle;
// elements outside the matrix read as zero.
static bool make_map(CUtensorMap* map, const void* base, int rows, int K, int ld, int box_rows) {
  const cuuint64_t dims[2] = {cuuint64_t(K), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(ld) * 2};
  const cuuint32_t box[2] = {cuuint32_t(BK), cuuint32_t(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
static tardis_status_t launch_bn(const GemmArgs& g, cudaStream_t s) {
  CUtensorMap a1, b1, a2, b2;
  if (!make_map(&a1, g.A1, g.M, g.K1, g.lda1, BM) || !make_map(&b1, g.B1, g.N, g.K1, g.ldb1, BN)) return TARDIS_ERR_INVALID_ARG;
  a2 = a1; b2 = b1;
  if (g.K2 > 0 && (!make_map(&a2, g.A2, g.M, g.K2, g.lda2, BM) || !make_map(&b2, g.B2, g.N, g.K2, g.ldb2, BN)))
    return TARDIS_ERR_INVALID_ARG;
  KParams p;
  p.M = g.M; p.N = g.N; p.kb1 = (g.K1 + BK - 1) / BK; p.kb2 = g.K2 > 0 ? (g.K2 + BK - 1) / BK : 0;
  p.epilogue = g.epilogue; p.ldo = g.ldo; p.act = g.act; p.splits = g.splits > 1 ? g.splits : 1;
  p.out_f32 = g.out_f32; p.out_bf16 = static_cast<__nv_bfloat16*>(g.out_bf16);
  p.bias = g.bias; p.addend = g.addend; p.a = g.a; p.c = g.c; p.bitmap = g.bitmap; p.error_word = g.error_word;
  p.lo = g.lo; p.hi = g.hi; p.colscale = g.colscale; p.rowscale = g.rowscale; p.keps = g.keps; p.bitmap_out = g.bitmap_out;
  p.rlist = g.rlist; p.rcount = g.rcount; p.rcap = g.rcap; p.codes = g.codes; p.scale = static_cast<const __nv_bfloat16*>(g.scale);
  p.zero = g.zero; p.xsrc = static_cast<const __nv_bfloat16*>(g.xsrc); p.d = g.d; p.G = g.G; p.bits = g.bits;
  TARDIS_CUDA_TRY(cudaFuncSetAttribute(k_gemm<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::SMEM));
  const int nm = (g.M + BM - 1) / BM, nn = (g.N + BN - 1) / BN;
  p.fast_m = nm <= nn ? 1 : 0;
  const int fcount = p.fast_m ? nm : nn;
  p.band = fcount <= 16 ? fcount : 12;
  const long tiles = long(nm) * nn * p.splits;
  int dev = 0, sms = 0;
  TARDIS_CUDA_TRY(cudaGetDevice(&dev));
  TARDIS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const unsigned grid = unsigned(tiles < sms ? tiles : sms);          // one CTA per SM (shared memory), persistent
  k_gemm<BN><<<grid, NTHREADS, Cfg<BN>::SMEM, s>>>(a1, b1, a2, b2, p);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

}  // namespace gemm

tardis_status_t launch_gemm(const GemmArgs& g, cudaStream_t s) {
  using namespace gemm;
  if (g.M <= 0 || g.N <= 0 || g.K1 <= 0) return TARDIS_ERR_INVALID_ARG;
  if (!encode_fn()) return TARDIS_ERR_UNSUPPORTED;
  auto bad = [](const void* p, int ld, int K) { return !p || (reinterpret_cast<uintptr_t>(p) & 15u) || (ld & 7) || (K & 7) || ld < K; };
  if (bad(g.A1, g.lda1, g.K1) || bad(g.B1, g.ldb1, g.K1)) return TARDIS_ERR_INVALID_ARG;
  if (g.K2 > 0 && (bad(g.A2, g.lda2, g.K2) || bad(g.B2, g.ldb2, g.K2))) return TARDIS_ERR_INVALID_ARG;
  if ((g.epilogue == GEMM_EPI_DELTA || g.epilogue == GEMM_EPI_FLAGS) && (g.N % 32)) return TARDIS_ERR_INVALID_ARG;
  if (g.epilogue == GEMM_EPI_FLAGS && !(g.bias && g.lo && g.hi && g.colscale && g.rowscale && g.bitmap_out && g.rlist && g.rcount &&
                                         g.codes && g.scale && g.zero && g.xsrc))
    return TARDIS_ERR_INVALID_ARG;
  if (g.splits > 1 && g.epilogue != GEMM_EPI_F32) return TARDIS_ERR_INVALID_ARG;
  // the epilogues store (or reduce) 16 bytes at a time
  auto misaligned = [](const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u); };
  if (misaligned(g.out_f32) || misaligned(g.out_bf16) || misaligned(g.addend)) return TARDIS_ERR_INVALID_ARG;
  // wide tiles when they still fill the machine, narrow ones for skinny problems
  const long tiles256 = long((g.N + 255) / 256) * ((g.M + BM - 1) / BM) * (g.splits > 1 ? g.splits : 1);
  if (tiles256 >= 120) return launch_bn<256>(g, s);
  return launch_bn<128>(g, s);
}

}  // namespace tardis
