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

// loads the n samples of neuron j (plus its bias) into keys[0..npad) (+inf beyond n) and sorts them ascending
// (bitonic network; npad a power of two); all threads of the CTA
__device__ __forceinline__ void load_and_sort(const float* __restrict__ z, long long ldz, const float* __restrict__ b1, int j, int n,
                                              int npad, float* keys) {
  const int tid = threadIdx.x;
  const float bias = b1 ? b1[j] : 0.f;
  for (int i = tid; i < npad; i += NT) {
    float v = __int_as_float(0x7f800000);              // +inf: padding sorts behind every sample
    if (i < n) v = z[size_t(j) * ldz + i] + bias;
    keys[i] = v;
  }
  __syncthreads();
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
}

// least squares of the activation over the samples with l <= z < u (fp64, two passes: means, then centred second
// moments); thread 0 writes the line of neuron j; fewer than two samples in range: the tangent at the midpoint
__device__ __forceinline__ void fit_and_store(const float* keys, int n, float lo_f, float hi_f, int act, double* red, int j,
                                              float* __restrict__ lo, float* __restrict__ hi, float* __restrict__ a, float* __restrict__ c) {
  const int tid = threadIdx.x;
  const double l = double(lo_f), u = double(hi_f);
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
    lo[j] = lo_f; hi[j] = hi_f; a[j] = float(aj); c[j] = float(cj);
  }
}

__global__ void __launch_bounds__(NT)
k_calibrate(const float* __restrict__ z, long long ldz, const float* __restrict__ b1, int n, int npad, double q_lo, double q_hi,
            int act, float* __restrict__ lo, float* __restrict__ hi, float* __restrict__ a, float* __restrict__ c) {
  extern __shared__ float keys[];                      // [npad]
  __shared__ double red[NT / 32];
  __shared__ float range[2];
  const int j = blockIdx.x, tid = threadIdx.x;
  load_and_sort(z, ldz, b1, j, n, npad, keys);
  // quantile at level q: between the order statistics around position q (n - 1)
  if (tid < 2) {
    const double pos = (tid == 0 ? q_lo : q_hi) * double(n - 1);
    const int i0 = int(floor(pos)), i1 = min(i0 + 1, n - 1);
    const double w = pos - double(i0);
    const double v = __dadd_rn(__dmul_rn(double(keys[i0]), 1.0 - w), __dmul_rn(double(keys[i1]), w));
    range[tid] = float(v);
  }
  __syncthreads();
  fit_and_store(keys, n, range[0], range[1], act, red, j, lo, hi, a, c);
}

// ---- the greedy range search of Algorithm 1 (Section 5.1.1, "Range Searching") --------------------------------------
// One CTA per neuron.  (1) Sort the samples.  (2) Centroid: the sample with the highest Gaussian kernel density estimate
// (width 1.06 std N^-1/5, density evaluated at every sample, fp64).  (3) The greedy loop, all threads in step: range =
// centroid - k_l step .. centroid + k_r step, grown by one step on the side whose candidate range has the smaller error
// (right on ties; a side that has passed the outermost sample is not grown) until the share of samples inside reaches the
// neuron's threshold.  The error of a candidate is evaluated as its definition says: least-squares line over the samples
// inside (means, centred moments), then the mean of the squared residuals; the samples are sorted, so "inside" is an index
// range found by binary search, and the activation values are computed once.  (Prefix sums would make a candidate O(1),
// but they lose the exact zeros of piecewise-linear activations, on which the tie rule depends.)  (4) The line over the
// final range, as in k_calibrate.
constexpr int kMaxSearchSamples = 2048;

__device__ __forceinline__ void block_sum2(double& v0, double& v1, double* red) {     // every thread gets both sums
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { v0 += __shfl_xor_sync(0xffffffffu, v0, o); v1 += __shfl_xor_sync(0xffffffffu, v1, o); }
  __syncthreads();                                                                    // red is free again
  if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = v0; red[NT / 32 + (threadIdx.x >> 5)] = v1; }
  __syncthreads();
  double t0 = 0.0, t1 = 0.0;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) { t0 += red[w]; t1 += red[NT / 32 + w]; }
  v0 = t0; v1 = t1;
}

__global__ void __launch_bounds__(NT)
k_range_search(const float* __restrict__ z, long long ldz, const float* __restrict__ b1, int n, int npad,
               const float* __restrict__ thr, double t_all, double step, int act, float* __restrict__ lo, float* __restrict__ hi,
               float* __restrict__ a, float* __restrict__ c, int* __restrict__ steps_out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* gs = reinterpret_cast<double*>(smem_raw);                // [n] activation of the sorted samples
  float* keys = reinterpret_cast<float*>(gs + n);                  // [npad]
  __shared__ double red[2 * (NT / 32)];
  __shared__ double bestv[NT / 32];
  __shared__ int besti[NT / 32];
  __shared__ double cen_s;
  const int j = blockIdx.x, tid = threadIdx.x;
  load_and_sort(z, ldz, b1, j, n, npad, keys);
  // mean and standard deviation (N - 1 in the denominator) of the samples; activation values
  double s1 = 0.0;
  for (int i = tid; i < n; i += NT) { s1 += double(keys[i]); gs[i] = gelu_f64(double(keys[i]), act); }
  const double mean = block_sum(s1, red) / double(n);
  double s2 = 0.0;
  for (int i = tid; i < n; i += NT) { const double dz = double(keys[i]) - mean; s2 += dz * dz; }
  s2 = block_sum(s2, red);
  const double bw = n > 1 ? 1.06 * sqrt(s2 / double(n - 1)) * pow(double(n), -0.2) : 0.0;
  // centroid: highest density, the smallest sample among equals
  if (bw > 0.0) {
    const double inv = 1.0 / bw;
    double bv = -1.0;
    int bi = 0x7fffffff;
    for (int i = tid; i < n; i += NT) {
      const double zi = double(keys[i]);
      double dsum = 0.0;
      for (int k = 0; k < n; ++k) { const double u = (double(keys[k]) - zi) * inv; dsum += exp(-0.5 * u * u); }
      if (dsum > bv) { bv = dsum; bi = i; }                 // i ascends within a thread: the first maximum stays
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if ((tid & 31) == 0) { bestv[tid >> 5] = bv; besti[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < NT / 32; ++w)
        if (bestv[w] > bv || (bestv[w] == bv && besti[w] < bi)) { bv = bestv[w]; bi = besti[w]; }
      cen_s = double(keys[bi]);
    }
  } else if (tid == 0) {
    cen_s = double(keys[0]);
  }
  __syncthreads();
  const double cen = cen_s;
  const double t = thr ? double(thr[j]) : t_all;
  auto lower = [&](double v) {                            // number of samples below v
    int l = 0, r = n;
    while (l < r) { const int m = (l + r) >> 1; if (double(keys[m]) < v) l = m + 1; else r = m; }
    return l;
  };
  // mean squared residual of the least-squares line over the sorted samples i0 .. i1 - 1 (every thread gets it)
  auto mse = [&](int i0, int i1) -> double {
    const int cnt = i1 - i0;
    if (cnt < 2) return 0.0;                              // (uniform over the CTA)
    const double q = 1.0 / double(cnt);
    double sz = 0.0, sg = 0.0;
    for (int i = i0 + tid; i < i1; i += NT) { sz += double(keys[i]); sg += gs[i]; }
    block_sum2(sz, sg, red);
    const double mz = sz * q, mg = sg * q;
    double vzz = 0.0, vzg = 0.0;
    for (int i = i0 + tid; i < i1; i += NT) { const double dz = double(keys[i]) - mz; vzz += dz * dz; vzg += dz * (gs[i] - mg); }
    block_sum2(vzz, vzg, red);
    vzz *= q; vzg *= q;
    if (!(vzz > 1e-30)) return 0.0;
    const double sl = vzg / vzz;
    double rr = 0.0, dummy = 0.0;
    for (int i = i0 + tid; i < i1; i += NT) { const double r = (gs[i] - mg) - sl * (double(keys[i]) - mz); rr += r * r; }
    block_sum2(rr, dummy, red);
    return rr * q;
  };
  const double zmin = double(keys[0]), zmax = double(keys[n - 1]);
  int kl = 0, kr = 0, nsteps = 0;
  const int cap = 4 + 2 * int(fmin(1.0e7, (zmax - zmin) / step + 2.0));   // the loop ends long before; a guard against a bad step
  for (; nsteps < cap; ++nsteps) {
    const double l = cen - kl * step, u = cen + kr * step;
    const int i0 = lower(l), i1 = lower(u);
    const int inside = i1 - i0;
    if (double(inside) >= t * double(n) || inside == n) break;
    bool go_left;
    if (u > zmax) go_left = true;
    else if (l <= zmin) go_left = false;
    else {
      const double el = mse(lower(cen - (kl + 1) * step), i1);
      const double er = mse(i0, lower(cen + (kr + 1) * step));
      go_left = el < er;
    }
    if (go_left) ++kl; else ++kr;
  }
  const float lo_f = float(cen - kl * step), hi_f = float(cen + kr * step);
  if (tid == 0 && steps_out) steps_out[j] = nsteps;
  __syncthreads();
  fit_and_store(keys, n, lo_f, hi_f, act, red, j, lo, hi, a, c);
}

// Error contribution of every neuron (Section 5.1.1, the E of the neuron-level thresholds): the mean squared residual of
// the least-squares line over the neuron's samples inside its range [lo_j, hi_j), as Algorithm 1's approx_error measures it.
__global__ void __launch_bounds__(NT)
k_neuron_error(const float* __restrict__ z, long long ldz, const float* __restrict__ b1, int n, int npad, int act,
               const float* __restrict__ lo, const float* __restrict__ hi, float* __restrict__ err) {
  extern __shared__ __align__(16) unsigned char smem_err[];
  double* gs = reinterpret_cast<double*>(smem_err);                // [n] activation of the sorted samples
  float* keys = reinterpret_cast<float*>(gs + n);                  // [npad] sorted samples
  __shared__ double red[2 * (NT / 32)];
  const int j = blockIdx.x, tid = threadIdx.x;
  load_and_sort(z, ldz, b1, j, n, npad, keys);
  for (int i = tid; i < n; i += NT) gs[i] = gelu_f64(double(keys[i]), act);
  __syncthreads();
  auto lower = [&](double v) {
    int l = 0, r = n;
    while (l < r) { const int m = (l + r) >> 1; if (double(keys[m]) < v) l = m + 1; else r = m; }
    return l;
  };
  const int i0 = lower(double(lo[j])), i1 = lower(double(hi[j]));
  const int cnt = i1 - i0;
  double e = 0.0;
  if (cnt >= 2) {                                           // (uniform over the CTA)
    const double q = 1.0 / double(cnt);
    double sz = 0.0, sg = 0.0;
    for (int i = i0 + tid; i < i1; i += NT) { sz += double(keys[i]); sg += gs[i]; }
    block_sum2(sz, sg, red);
    const double mz = sz * q, mg = sg * q;
    double vzz = 0.0, vzg = 0.0;
    for (int i = i0 + tid; i < i1; i += NT) { const double dz = double(keys[i]) - mz; vzz += dz * dz; vzg += dz * (gs[i] - mg); }
    block_sum2(vzz, vzg, red);
    vzz *= q; vzg *= q;
    if (vzz > 1e-30) {
      const double sl = vzg / vzz;
      double rr = 0.0, dummy = 0.0;
      for (int i = i0 + tid; i < i1; i += NT) { const double r = (gs[i] - mg) - sl * (double(keys[i]) - mz); rr += r * r; }
      block_sum2(rr, dummy, red);
      e = rr * q;
    }
  }
  if (tid == 0) err[j] = float(e);
}

// Neuron-level thresholds (Section 5.1.1): minimise sum_j E_j t_j subject to sum_j t_j = t_layer h, read with the box
// t_min <= t_j <= t_max.  A linear objective over a box with one equality: every neuron starts at t_min and the budget
// (t_layer - t_min) h goes, t_max - t_min each, to the neurons in order of increasing error (the smaller index first among
// equals).  A thread finds its neuron's place in that order by counting, then takes its share of what is left for it.
__global__ void __launch_bounds__(NT)
k_neuron_thresholds(const float* __restrict__ err, int h, double t_layer, double t_min, double t_max, float* __restrict__ t) {
  __shared__ float tile[NT];
  const int j = blockIdx.x * NT + threadIdx.x;
  const float ej = j < h ? err[j] : 0.f;
  int rank = 0;
  for (int base = 0; base < h; base += NT) {
    __syncthreads();
    tile[threadIdx.x] = base + threadIdx.x < h ? err[base + threadIdx.x] : 0.f;
    __syncthreads();
    const int m = min(NT, h - base);
    for (int i = 0; i < m; ++i) rank += (tile[i] < ej || (tile[i] == ej && base + i < j)) ? 1 : 0;
  }
  if (j >= h) return;
  const double cap = t_max - t_min, budget = (t_layer - t_min) * double(h);
  const double give = fmin(cap, fmax(0.0, budget - double(rank) * cap));
  t[j] = float(t_min + give);
}

}  // namespace cal

tardis_status_t launch_neuron_thresholds(int h, int n, const float* z, long long ldz, const float* b1, const float* lo, const float* hi,
                                         int act, double t_layer, double t_min, double t_max, float* err, float* t, cudaStream_t s) {
  if (n < 1 || n > cal::kMaxSearchSamples) return TARDIS_ERR_UNSUPPORTED;
  int npad = 2;
  while (npad < n) npad <<= 1;
  const size_t smem = size_t(n) * sizeof(double) + size_t(npad) * sizeof(float);
  cal::k_neuron_error<<<h, cal::NT, smem, s>>>(z, ldz, b1, n, npad, act, lo, hi, err);
  TARDIS_CUDA_TRY(cudaGetLastError());
  cal::k_neuron_thresholds<<<(h + cal::NT - 1) / cal::NT, cal::NT, 0, s>>>(err, h, t_layer, t_min, t_max, t);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t launch_calibrate(int h, int n, const float* z, long long ldz, const float* b1, double q_lo, double q_hi, int act,
                                 float* lo, float* hi, float* a, float* c, cudaStream_t s) {
  if (n < 1 || n > cal::kMaxSamples) return TARDIS_ERR_UNSUPPORTED;
  int npad = 2;
  while (npad < n) npad <<= 1;
  cal::k_calibrate<<<h, cal::NT, size_t(npad) * sizeof(float), s>>>(z, ldz, b1, n, npad, q_lo, q_hi, act, lo, hi, a, c);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t launch_range_search(int h, int n, const float* z, long long ldz, const float* b1, const float* thr, double t_all,
                                    double step, int act, float* lo, float* hi, float* a, float* c, int* steps_out, cudaStream_t s) {
  if (n < 1 || n > cal::kMaxSearchSamples) return TARDIS_ERR_UNSUPPORTED;
  int npad = 2;
  while (npad < n) npad <<= 1;
  const size_t smem = size_t(n) * sizeof(double) + size_t(npad) * sizeof(float);
  TARDIS_CUDA_TRY(cudaFuncSetAttribute(cal::k_range_search, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  cal::k_range_search<<<h, cal::NT, smem, s>>>(z, ldz, b1, n, npad, thr, t_all, step, act, lo, hi, a, c, steps_out);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

}  // namespace tardis
