// Exact fp64 predictor sums (Section 5.3: s[j,g] (q - zp) x over the channels of neuron j, without the bias) from the
// packed codes (2, 3, 4 or 8 bits each): what decides a flag when a fast score is too close to a range end.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace tardis {

// Code of channel k in a row of packed codes: the row is one bit stream, channel order ascending, lowest bits first (code k
// holds bits [k bits, (k + 1) bits) of it).  With 2, 4 or 8 bits a code never leaves its 32-bit word; a 3-bit code may.
__device__ __forceinline__ uint32_t stream_code(const uint32_t* __restrict__ row, int k, int bits) {
  const int pos = k * bits, w = pos >> 5, sh = pos & 31;
  uint32_t v = row[w] >> sh;
  if (sh + bits > 32) v |= row[w + 1] << (32 - sh);
  return v & ((1u << bits) - 1u);
}

// the same sums for code widths that do not divide 32 (3 bits): channel by channel, lane l takes channels 32 i + l
__device__ inline double exact_score_stream(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                                            const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G,
                                            int bits, int first, int stride) {
  const int ng = d / G;
  const uint32_t* row = codes + size_t(j) * (size_t(d) * bits / 32);
  double acc = 0.0;
  for (int k = first; k < d; k += stride) {
    const int g = k / G;
    const double zp = double(zero[size_t(j) * ng + g]);
    acc += double(__bfloat162float(scale[size_t(j) * ng + g])) * ((double(stream_code(row, k, bits)) - zp) * double(__bfloat162float(xt[k])));
  }
  return acc;
}

// one warp; every lane returns the sum
__device__ inline double exact_score(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                              const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G,
                              int bits, int lane) {   // one warp; every lane returns the sum
  if (32 % bits) {
    double acc = exact_score_stream(codes, scale, zero, xt, j, d, G, bits, lane, 32);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
  }
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

// The same sums for a kernel that does nothing else (k_recheck): with 2-bit codes the 16 channels of a word come in as two
// 128-bit loads and the loads of four words go out before the first is used; same terms in the same order as exact_score.
// (Kept apart from exact_score: inside the fused kernels its registers would spill.)
__device__ inline double exact_score_wide(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                                          const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G,
                                          int bits, int lane) {
  if (bits != 2 || (reinterpret_cast<uintptr_t>(xt) & 15u) != 0) return exact_score(codes, scale, zero, xt, j, d, G, bits, lane);
  const int nwords = d / 16, ng = d / G;
  double acc = 0.0;
  {
    // the 16 channels of a word come in as two 128-bit loads, and the loads of four words go out before the first is used
    // (same terms in the same order as the general loop below)
    for (int w0 = lane; w0 < nwords; w0 += 128) {
      uint32_t word[4];
      uint8_t zr[4];
      __nv_bfloat16 sr[4];
      uint4 xa[4], xb[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int w = w0 + 32 * u;
        if (w < nwords) {
          const int g = (w * 16) / G;
          word[u] = codes[size_t(j) * nwords + w];
          zr[u] = zero[size_t(j) * ng + g];
          sr[u] = scale[size_t(j) * ng + g];
          xa[u] = *reinterpret_cast<const uint4*>(xt + w * 16);
          xb[u] = *reinterpret_cast<const uint4*>(xt + w * 16 + 8);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (w0 + 32 * u < nwords) {
          const double zp = double(zr[u]);
          const uint32_t xw[8] = {xa[u].x, xa[u].y, xa[u].z, xa[u].w, xb[u].x, xb[u].y, xb[u].z, xb[u].w};
          double inner = 0.0;
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const float xf = __uint_as_float((q & 1) ? (xw[q >> 1] & 0xffff0000u) : (xw[q >> 1] << 16));
            inner += (double((word[u] >> (2 * q)) & 3u) - zp) * double(xf);
          }
          acc += double(__bfloat162float(sr[u])) * inner;
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  return acc;
}

__device__ inline double exact_score_single(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                                     const uint8_t* __restrict__ zero, const __nv_bfloat16* __restrict__ xt, int j, int d, int G, int bits) {
  if (32 % bits) return exact_score_stream(codes, scale, zero, xt, j, d, G, bits, 0, 1);
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
