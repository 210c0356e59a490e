// Offline statistics of a layer (Section 5.1, steps 2 and 3; the procedure is described with Insight 2 in Section 4.1): from the calibration pre-activations of every neuron,
// the range that holds the central portion of them (quantiles q_lo, q_hi) and the least-squares line
// y = a z + c of GELU over the samples inside that range.
//
// One CTA per neuron: the N samples are sorted in shared memory (bitonic network over the next power of two,
// padded with +inf), the two quantiles are interpolated between order statistics in fp64 and rounded to fp32,
// and the regression sums run in fp64 in two passes (means, then centred second moments), GELU in fp64.
#include "common.cuh"

namespace tardis {
namespace cal {

constexpr int NT = 256;
constexpr int kMaxSamples = 8192;

__device__ __forceinline__ double block_sum(double v, double* red) {     // every thread gets the sum
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();                                                        // red is free again
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) t += red[w];
  return t;
}

__device__ __forceinline__ double gelu_slope_f64(double z, int act) {
  if (act == TARDIS_ACT_RELU) return z > 0.0 ? 1.0 : 0.0;
  if (act == TARDIS_ACT_GELU_TANH) {
    const double k = 0.7978845608028654;
    const double u = k * (z + 0.044715 * z * z * z), t = tanh(u);
    return 0.5 * (1.0 + t) + 0.5 * z * (1.0 - t * t) * k * (1.0 + 3.0 * 0.044715 * z * z);
  }
  return 0.5 * (1.0 + erf(z * 0.7071067811865476)) + z * exp(-0.5 * z * z) * 0.3989422804014327;
}

__global__ void __launch_bounds__(NT)
k_calibrate(const float* __restrict__ z, long long ldz, const float* __restrict__ b1, int n, int npad, double q_lo, double q_hi,
            int act, float* __restrict__ lo, float* __restrict__ hi, float* __restrict__ a, float* __restrict__ c) {
  extern __shared__ float keys[];                      // [npad]
  __shared__ double red[NT / 32];
  __shared__ float range[2];
  const int j = blockIdx.x, tid = threadIdx.x;
  const float bias = b1 ? b1[j] : 0.f;
  for (int i = tid; i < npad; i += NT) {
    float v = __int_as_float(0x7f800000);              // +inf: padding sorts behind every sample
    if (i < n) v = z[size_t(j) * ldz + i] + bias;
    keys[i] = v;
  }
  __syncthreads();
  // bitonic sorting network, ascending
  for (int k = 2; k <= npad; k <<= 1) {
    for (int s = k >> 1; s > 0; s >>= 1) {
      for (int t = tid; t < npad / 2; t += NT) {
        const int i = 2 * t - (t & (s - 1)), p = i + s;          // pair (i, i + s), i without bit s
        const bool up = (i & k) == 0;
        const float x = keys[i], y = keys[p];
        if ((x > y) == up) { keys[i] = y; keys[p] = x; }
      }
      __syncthreads();
    }
  }
  // quantile at level q: between the order statistics around position q (n - 1)
  if (tid < 2) {
    const double pos = (tid == 0 ? q_lo : q_hi) * double(n - 1);
    const int i0 = int(floor(pos)), i1 = min(i0 + 1, n - 1);
    const double w = pos - double(i0);
    const double v = __dadd_rn(__dmul_rn(double(keys[i0]), 1.0 - w), __dmul_rn(double(keys[i1]), w));
    range[tid] = float(v);
  }
  __syncthreads();
  const double l = double(range[0]), u = double(range[1]);
  // least squares over the samples with l <= z < u
  double cnt = 0.0, sz = 0.0, ss = 0.0;
  for (int i = tid; i < n; i += NT) {
    const double v = double(keys[i]);
    if (v >= l && v < u) { cnt += 1.0; sz += v; ss += gelu_f64(v, act); }
  }
  cnt = block_sum(cnt, red); sz = block_sum(sz, red); ss = block_sum(ss, red);
  const double safe = cnt > 0.0 ? cnt : 1.0;
  const double mz = sz / safe, ms = ss / safe;
  double var = 0.0, cov = 0.0;
  for (int i = tid; i < n; i += NT) {
    const double v = double(keys[i]);
    if (v >= l && v < u) { const double dz = v - mz; var += dz * dz; cov += dz * (gelu_f64(v, act) - ms); }
  }
  var = block_sum(var, red) / safe; cov = block_sum(cov, red) / safe;
  if (tid == 0) {
    double aj, cj;
    if (cnt >= 2.0 && var > 1e-30) { aj = cov / var; cj = ms - aj * mz; }
    else {                                             // too few samples in range: tangent at the midpoint
      const double mid = 0.5 * (l + u);
      aj = gelu_slope_f64(mid, act);
      cj = gelu_f64(mid, act) - aj * mid;
    }
    lo[j] = range[0]; hi[j] = range[1]; a[j] = float(aj); c[j] = float(cj);
  }
}

}  // namespace cal

tardis_status_t launch_calibrate(int h, int n, const float* z, long long ldz, const float* b1, double q_lo, double q_hi, int act,
                                 float* lo, float* hi, float* a, float* c, cudaStream_t s) {
  if (n < 1 || n > cal::kMaxSamples) return TARDIS_ERR_UNSUPPORTED;
  int npad = 2;
  while (npad < n) npad <<= 1;
  cal::k_calibrate<<<h, cal::NT, size_t(npad) * sizeof(float), s>>>(z, ldz, b1, n, npad, q_lo, q_hi, act, lo, hi, a, c);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

}  // namespace tardis
