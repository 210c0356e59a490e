// Thin wrappers over the PTX the fused kernels use: mbarriers with bounded waits, bulk async copies,
// streaming loads, legacy tensor-core MMAs (integer and bf16), vector reductions to global memory.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace tardis {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
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
// Bounded wait: false when the limit ran out (the caller records the error and goes on without the
// data).  The test is the non-blocking form (the potentially blocking try_wait was measured to take several hundred
// cycles even on a completed phase); the limit is in SM clock cycles (a fraction of a second).
constexpr long long WAIT_LIMIT_CYCLES = 400000000ll;
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, long long limit = WAIT_LIMIT_CYCLES) {
  if (mbar_test(b, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_test(b, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// The same for a whole warp (all 32 lanes must call it): lane 0 polls, the others learn the outcome through a shuffle,
// which also orders their later reads of the copied data after lane 0's observation of the barrier.  (Every lane
// polling the same barrier word serialises: with 32 warps waiting that costs more than the wait itself.)
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* b, uint32_t parity, long long limit = WAIT_LIMIT_CYCLES) {
  int ok = 0;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(b, parity, limit) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint4 ldg_stream(const void* p) {   // read-only, no L1 allocation
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The same with a zero accumulator going in: MMAs of one warp that do not depend on each other pipeline
// four times better than a chain through one accumulator, so each MMA of a group starts its own sum.
__device__ __forceinline__ void mma_u8s8_z(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
               : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void red_add_f32(float* addr, float v) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void unpack8(float (&f)[8], const uint4& w) {
  f[0] = bf_lo(w.x); f[1] = bf_hi(w.x); f[2] = bf_lo(w.y); f[3] = bf_hi(w.y);
  f[4] = bf_lo(w.z); f[5] = bf_hi(w.z); f[6] = bf_lo(w.w); f[7] = bf_hi(w.w);
}
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


}  // namespace ptx
}  // namespace tardis
