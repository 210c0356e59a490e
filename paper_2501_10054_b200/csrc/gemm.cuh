// bf16 tensor-core GEMM of libtardis (tcgen05 + TMEM accumulators + TMA operand staging, sm_100a).
//   acc[m, n] = sum_k A1[m, k] B1[n, k] (+ sum_k A2[m, k] B2[n, k])      A: [M, K] row-major, B: [N, K] row-major
// followed by one of the epilogues below.  Used by the offline fold (Section 5.2), by the batched
// speculative product (Section 5.4) and by the batched predictor / result fixing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "tardis.h"

namespace tardis {

enum GemmEpilogue {
  GEMM_EPI_F32 = 0,        // out_f32[m, n] = acc + (bias ? bias[n] : 0)
  GEMM_EPI_ADD_BF16 = 1,   // out_bf16[m, n] = bf16(acc + addend_f32[m, n])
  GEMM_EPI_DELTA = 2,      // z = acc + bias[n]; out_bf16[m, n] = flagged(m, n) ? GELU(z) - a[n] z - c[n] : 0
  GEMM_EPI_FLAGS = 3       // z = acc + bias[n]; bit (m, n) of bitmap_out = !(lo[n] <= z < hi[n]); a z within
                           // keps * colscale[n] * rowscale[m] of lo[n] or hi[n] is queued in rlist for exact
                           // re-evaluation (settled in place from the codes when the queue is full); a row whose
                           // rowscale is not finite is flagged throughout; z is also stored when out_f32 is given
};

struct GemmArgs {
  int M, N, K1, K2;                 // K2 = 0: one operand pair only.  K1, K2 multiples of 8.
  const void *A1, *B1, *A2, *B2;    // device bf16; leading dimensions lda1 ... in elements (multiples of 8)
  int lda1, ldb1, lda2, ldb2;
  int epilogue;                     // GemmEpilogue
  int splits;                       // > 1 (GEMM_EPI_F32 only): the channel range is split over that many CTAs per tile, which
                                    // ADD their parts to out_f32 (the caller zeroes it first); the bias is added once
  float* out_f32; void* out_bf16;   // row-major, leading dimension ldo
  int ldo;
  const float* bias;                // [N] or null
  const float* addend;              // [M, ldo] fp32 (GEMM_EPI_ADD_BF16)
  const float *a, *c;               // [N] (GEMM_EPI_DELTA)
  const uint32_t* bitmap;           // [M, N / 32] flag words (GEMM_EPI_DELTA)
  int act;
  unsigned long long* error_word;   // device counter slot that receives 1 when a bounded wait runs out
  // GEMM_EPI_FLAGS
  const float *lo, *hi, *colscale, *rowscale;   // [N], [N], [N], [M]
  float keps;
  uint32_t* bitmap_out;             // [M, N / 32]
  uint2* rlist; unsigned int* rcount; int rcap;   // queue of (m, n) pairs, its fill count ([1]: pairs settled in place), capacity
  const uint32_t* codes; const void* scale; const uint8_t* zero;   // the packed predictor (rows n)
  const void* xsrc; int d, G, bits; // the bf16 rows A1 came from (leading dimension d), group size, bits per code
};

// Enqueues the GEMM on `s`.  Returns UNSUPPORTED when the tensor-map entry point of the driver is not
// available, INVALID_ARG on misaligned operands, CUDA on launch failure.
tardis_status_t launch_gemm(const GemmArgs& g, cudaStream_t s);

}  // namespace tardis
