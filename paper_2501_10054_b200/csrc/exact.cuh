// Exact fp64 predictor sums (Section 5.3: s[j,g] (q - zp) x over the channels of neuron j, without the bias) from the
// packed codes (2, 4 or 8 bits each): what decides a flag when a fast score is too close to a range end.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace tardis {

// one warp; every lane returns the sum
__device__ inline double exact_score(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                              const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G,
                              int bits, int lane) {   // one warp; every lane returns the sum
  const int per = 32 / bits;                    // codes per word
  const uint32_t cmask = (1u << bits) - 1u;
  const int nwords = d / per, ng = d / G;
  double acc = 0.0;
  for (int w = lane; w < nwords; w += 32) {
    const uint32_t word = codes[size_t(j) * nwords + w];
    const int g = (w * per) / G;
    const double zp = double(zero[size_t(j) * ng + g]);
    double inner = 0.0;
    for (int q = 0; q < per; ++q) inner += (double((word >> (bits * q)) & cmask) - zp) * double(__bfloat162float(xt[w * per + q]));
    acc += double(__bfloat162float(scale[size_t(j) * ng + g])) * inner;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  return acc;
}

__device__ inline double exact_score_single(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                                     const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G, int bits) {
  const int per = 32 / bits;                    // codes per word
  const uint32_t cmask = (1u << bits) - 1u;
  const int nwords = d / per, ng = d / G;
  double acc = 0.0;
  for (int w = 0; w < nwords; ++w) {
    const uint32_t word = codes[size_t(j) * nwords + w];
    const int g = (w * per) / G;
    const double zp = double(zero[size_t(j) * ng + g]);
    double inner = 0.0;
    for (int q = 0; q < per; ++q) inner += (double((word >> (bits * q)) & cmask) - zp) * double(__bfloat162float(xt[w * per + q]));
    acc += double(__bfloat162float(scale[size_t(j) * ng + g])) * inner;
  }
  return acc;
}

}  // namespace tardis
