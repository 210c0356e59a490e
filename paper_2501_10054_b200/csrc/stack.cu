// A chain of partially linear FFN layers on one residual stream: per layer an optional layer normalisation of the
// stream, the layer's forward (tardis_ffn_forward, whatever path it picks), and the addition of its output to the
// stream.  The paper has no counterpart of this call (it replaces the FFN block inside an existing model, Section 6);
// it is the shape in which a decoder hands the FFN blocks of consecutive layers to this library, without attention.
//
// Two small kernels live here.  k_update_norm (one CTA per token, the row in registers, fp32) adds the previous layer's
// output to the stream and normalises the result for the next layer in one pass; k_stream_update adds the last layer's
// output.  Both take part in the programmatic hand-over between launches: they let the next launch start at once
// (the fused decode kernel then loads its predictor blocks while the row is being normalised) and wait for the launch
// before them only where they first touch its results.  Everything else is the per-layer forward.
#include "common.cuh"

namespace tardis {
namespace {

constexpr int LN_THREADS = 256;
constexpr int LN_MAXPER = 48;   // elements per thread: d_model up to 12288

__device__ __forceinline__ float block_sum(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                       // (sh may still be read from the previous sum)
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < LN_THREADS / 32; ++w) t += sh[w];   // every thread adds the same numbers in the same order
  return t;
}

// stream[t][:] takes the previous layer's output f[t][:] (update: added when `residual`, else copied), then
// out[t][i] = (stream[t][i] - mean_t) / sqrt(var_t + eps) * gamma[i] + beta[i]; mean and variance (1/d, not 1/(d-1)) over the
// row; without `normalise` out is the stream itself.
template <typename T>
__global__ void __launch_bounds__(LN_THREADS) k_update_norm(T* __restrict__ stream, const T* __restrict__ f, int update, int residual,
                                                            int normalise, T* __restrict__ out, const float* __restrict__ gamma,
                                                            const float* __restrict__ beta, int d, float eps) {
  __shared__ float sh[LN_THREADS / 32];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");          // the launch before wrote f (or the stream)
  T* row = stream + size_t(blockIdx.x) * d;
  const T* frow = f + size_t(blockIdx.x) * d;
  float v[LN_MAXPER];
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < LN_MAXPER; ++e) {
    const int i = threadIdx.x + e * LN_THREADS;
    v[e] = 0.f;
    if (i < d) {
      if (update) {
        const T nv = residual ? from_f32<T>(to_f32<T>(row[i]) + to_f32<T>(frow[i])) : frow[i];   // rounded as it is stored
        row[i] = nv;
        v[e] = to_f32<T>(nv);
      } else {
        v[e] = to_f32<T>(row[i]);
      }
    }
    s += v[e];
  }
  if (!normalise) {
#pragma unroll
    for (int e = 0; e < LN_MAXPER; ++e) {
      const int i = threadIdx.x + e * LN_THREADS;
      if (i < d) out[size_t(blockIdx.x) * d + i] = from_f32<T>(v[e]);
    }
    return;
  }
  const float mean = block_sum(s, sh) / float(d);
  float q = 0.f;
#pragma unroll
  for (int e = 0; e < LN_MAXPER; ++e) {
    const int i = threadIdx.x + e * LN_THREADS;
    const float c = i < d ? v[e] - mean : 0.f;
    q += c * c;
  }
  const float rstd = rsqrtf(block_sum(q, sh) / float(d) + eps);
#pragma unroll
  for (int e = 0; e < LN_MAXPER; ++e) {
    const int i = threadIdx.x + e * LN_THREADS;
    if (i < d) out[size_t(blockIdx.x) * d + i] = from_f32<T>((v[e] - mean) * rstd * (gamma ? gamma[i] : 1.f) + (beta ? beta[i] : 0.f));
  }
}

// stream += f (residual) or stream = f: after the last layer
template <typename T>
__global__ void k_stream_update(T* __restrict__ stream, const T* __restrict__ f, size_t count, int residual) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < count; i += size_t(gridDim.x) * blockDim.x)
    stream[i] = residual ? from_f32<T>(to_f32<T>(stream[i]) + to_f32<T>(f[i])) : f[i];
}

template <typename... Args>
cudaError_t launch_chained(void (*kernel)(Args...), dim3 grid, dim3 block, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename T>
tardis_status_t run_stack(const tardis_stack_desc_t* desc, const void* x, void* y, void* work, void* keep, int64_t n, cudaStream_t s) {
  Handle* H0 = reinterpret_cast<Handle*>(desc->layers[0]);
  const int d = H0->d;
  const size_t count = size_t(n) * d;
  T* stream = static_cast<T*>(y);
  if (x != y) TARDIS_CUDA_TRY(cudaMemcpyAsync(y, x, count * sizeof(T), cudaMemcpyDeviceToDevice, s));
  const int norm = desc->normalise != 0 ? 1 : 0;
  T* fprev = nullptr;
  for (int l = 0; l < desc->n_layers; ++l) {
    // with `keep`, the layer's input and output stay where the caller can read them; else two buffers for the inputs take
    // turns with one for the output (the update of layer l + 1 reads the output of layer l while writing its own input)
    T* xin = keep ? static_cast<T*>(keep) + size_t(2 * l) * count : static_cast<T*>(work);
    T* fout = keep ? static_cast<T*>(keep) + size_t(2 * l + 1) * count : static_cast<T*>(work) + count;
    const T* layer_in = stream;
    if (norm || keep || l > 0) {
      TARDIS_CUDA_TRY(launch_chained(k_update_norm<T>, dim3(unsigned(n)), dim3(LN_THREADS), s, stream, static_cast<const T*>(fprev ? fprev : stream),
                                     l > 0 ? 1 : 0, desc->residual, norm, xin, norm && desc->ln_gamma ? desc->ln_gamma[l] : static_cast<const float*>(nullptr),
                                     norm && desc->ln_beta ? desc->ln_beta[l] : static_cast<const float*>(nullptr), d, desc->ln_eps));
      layer_in = xin;
    }
    const tardis_status_t st = tardis_ffn_forward(desc->layers[l], layer_in, fout, n, reinterpret_cast<tardis_stream_t>(s));
    if (st != TARDIS_OK) return st;
    fprev = fout;
  }
  const unsigned blocks = unsigned((count + 255) / 256 < 4096 ? (count + 255) / 256 : 4096);
  TARDIS_CUDA_TRY(launch_chained(k_stream_update<T>, dim3(blocks), dim3(256), s, stream, static_cast<const T*>(fprev), count, desc->residual));
  return TARDIS_OK;
}

}  // namespace

tardis_status_t launch_stack_forward(const tardis_stack_desc_t* desc, const void* x, void* y, void* work, void* keep, int64_t n,
                                     cudaStream_t s) {
  Handle* H0 = reinterpret_cast<Handle*>(desc->layers[0]);
  if (H0->d > LN_THREADS * LN_MAXPER) return TARDIS_ERR_UNSUPPORTED;
  return H0->dtype == TARDIS_F32 ? run_stack<float>(desc, x, y, work, keep, n, s) : run_stack<__nv_bfloat16>(desc, x, y, work, keep, n, s);
}

}  // namespace tardis
