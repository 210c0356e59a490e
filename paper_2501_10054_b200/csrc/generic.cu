// Generic kernels of the online path (Section 5.4) for any dtype, shape and token count:
// exact predictor score + flag, folded product, result fixing.  They favour exactness and
// simplicity; the fused decode kernel and the batched tensor-core path are the fast ones.
#include <mutex>

#include "common.cuh"
#include "exact.cuh"

namespace tardis {

// ---- predictor score (Section 5.3) and flag (Section 5.1.1), exact ----------------------
// One warp per neuron, 32 neurons per block, tokens looped.  The products (code - zero) * x
// are exact in fp64 and so, to 1e-16 relative, are the sums, so the comparison with
// [lo, hi) is taken on the mathematically exact score.
template <typename T>
__global__ void __launch_bounds__(1024) k_predictor_exact(
    const uint32_t* __restrict__ codes, const T* __restrict__ scale, const uint8_t* __restrict__ zero,
    const float* __restrict__ b1, const float* __restrict__ lo, const float* __restrict__ hi,
    const T* __restrict__ x, int n, int d, int h, int G, int bits, uint32_t* __restrict__ bitmap,
    uint32_t* __restrict__ dbg_bitmap, double* __restrict__ dbg_scores) {
  __shared__ int flag_s[32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 32 + warp;
  const int per = 32 / bits;                    // codes per word
  const uint32_t cmask = (1u << bits) - 1u;
  const int nwords = d / per, ng = d / G;
  const double lo_j = double(lo[j]), hi_j = double(hi[j]), b1_j = double(b1[j]);
  for (int t = 0; t < n; ++t) {
    const T* xt = x + size_t(t) * d;
    double acc = 0.0;
    if (32 % bits) {                            // 3-bit codes: a bit stream, channel by channel
      const uint32_t* row = codes + size_t(j) * (size_t(d) * bits / 32);
      for (int k = lane; k < d; k += 32) {
        const int g = k / G;
        acc += double(to_f32(scale[size_t(j) * ng + g])) *
               ((double(stream_code(row, k, bits)) - double(zero[size_t(j) * ng + g])) * double(to_f32(xt[k])));
      }
    }
    for (int w = lane; w < nwords && 32 % bits == 0; w += 32) {
      const uint32_t word = codes[size_t(j) * nwords + w];
      const int g = (w * per) / G;
      const double zp = double(zero[size_t(j) * ng + g]);
      double inner = 0.0;
      for (int p = 0; p < per; ++p) {
        const double q = double((word >> (bits * p)) & cmask);
        inner += (q - zp) * double(to_f32(xt[w * per + p]));
      }
      acc += double(to_f32(scale[size_t(j) * ng + g])) * inner;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    const double zhat = acc + b1_j;
    const bool inside = (lo_j <= zhat) && (zhat < hi_j);
    if (lane == 0) {
      flag_s[warp] = inside ? 0 : 1;
      if (dbg_scores) dbg_scores[size_t(t) * h + j] = zhat;
    }
    __syncthreads();
    if (warp == 0) {
      const uint32_t word = __ballot_sync(0xffffffffu, flag_s[lane] != 0);
      if (lane == 0) {
        bitmap[size_t(t) * (h / 32) + blockIdx.x] = word;
        if (dbg_bitmap) dbg_bitmap[size_t(t) * (h / 32) + blockIdx.x] = word;
      }
    }
    __syncthreads();
  }
}

// ---- range check on the true pre-activations ----------------------------------------------
// The third scenario of the precision study (Section 7.7): the flag comes from z_j = W1[j,:] x + b1_j itself,
// evaluated in fp64, instead of from the predictor, which shows what the predictor's mistakes cost.  Same layout
// as the kernel above.
template <typename T>
__global__ void __launch_bounds__(1024) k_range_check_exact(
    const T* __restrict__ W1, const float* __restrict__ b1, const float* __restrict__ lo, const float* __restrict__ hi,
    const T* __restrict__ x, int n, int d, int h, uint32_t* __restrict__ bitmap, uint32_t* __restrict__ dbg_bitmap,
    double* __restrict__ dbg_scores) {
  __shared__ int flag_s[32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 32 + warp;
  const double lo_j = double(lo[j]), hi_j = double(hi[j]), b1_j = double(b1[j]);
  for (int t = 0; t < n; ++t) {
    const T* xt = x + size_t(t) * d;
    double acc = 0.0;
    for (int k = lane; k < d; k += 32) acc += double(to_f32(W1[size_t(j) * d + k])) * double(to_f32(xt[k]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    const double z = acc + b1_j;
    const bool inside = (lo_j <= z) && (z < hi_j);
    if (lane == 0) {
      flag_s[warp] = inside ? 0 : 1;
      if (dbg_scores) dbg_scores[size_t(t) * h + j] = z;
    }
    __syncthreads();
    if (warp == 0) {
      const uint32_t word = __ballot_sync(0xffffffffu, flag_s[lane] != 0);
      if (lane == 0) {
        bitmap[size_t(t) * (h / 32) + blockIdx.x] = word;
        if (dbg_bitmap) dbg_bitmap[size_t(t) * (h / 32) + blockIdx.x] = word;
      }
    }
    __syncthreads();
  }
}

// ---- flagged-count statistics ----------------------------------------------------------------
__global__ void k_flag_stats(const uint32_t* __restrict__ bitmap, int words, unsigned long long* counters) {
  __shared__ unsigned int total;
  if (threadIdx.x == 0) total = 0;
  __syncthreads();
  unsigned int c = 0;
  for (int w = threadIdx.x; w < words; w += blockDim.x) c += __popc(bitmap[size_t(blockIdx.x) * words + w]);
  atomicAdd(&total, c);
  __syncthreads();
  if (threadIdx.x == 0) {
    atomicAdd(&counters[CTR_FLAGGED_TOTAL], (unsigned long long)total);
    atomicMax(&counters[CTR_FLAGGED_MAX], (unsigned long long)total);
  }
}

// ---- speculative folded product (Section 5.4): yacc[t, i] = b_f[i] + sum_k C[k, i] x[t, k] ----
__global__ void k_init_yacc(float* __restrict__ yacc, const float* __restrict__ bf, int n, int d) {
  size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e < size_t(n) * d) yacc[e] = bf[e % d];
}

template <typename T, typename Acc>
__global__ void __launch_bounds__(256) k_folded_product(const T* __restrict__ C, const T* __restrict__ x,
                                                        float* __restrict__ yacc, int n, int d, int kchunk) {
  constexpr int TT = 8, KT = 128;
  __shared__ float xs[TT][KT];
  const int i = blockIdx.x * 256 + threadIdx.x;
  const int t0 = blockIdx.y * TT;
  const int kbeg = blockIdx.z * kchunk, kend = min(d, kbeg + kchunk);
  Acc acc[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) acc[t] = Acc(0);
  for (int k0 = kbeg; k0 < kend; k0 += KT) {
    for (int e = threadIdx.x; e < TT * KT; e += 256) {
      int t = e / KT, kk = e % KT;
      xs[t][kk] = (t0 + t < n && k0 + kk < kend) ? to_f32(x[size_t(t0 + t) * d + k0 + kk]) : 0.f;
    }
    __syncthreads();
    if (i < d) {
      const int klim = min(KT, kend - k0);
      for (int kk = 0; kk < klim; ++kk) {
        const Acc cv = Acc(to_f32(C[size_t(k0 + kk) * d + i]));
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[t] += cv * Acc(xs[t][kk]);
      }
    }
    __syncthreads();
  }
  if (i < d)
#pragma unroll
    for (int t = 0; t < TT; ++t)
      if (t0 + t < n) atomicAdd(&yacc[size_t(t0 + t) * d + i], float(acc[t]));
}

// ---- result fixing (Section 5.4) ---------------------------------------------------------------
// Block = (token t, block of NB neurons).  Pass 1: warps take the block's flagged neurons in turn,
// recompute z_j = W1[j,:] x_t + b1_j and delta_j = GELU(z_j) - a_j z_j - c_j.  Pass 2: each thread
// owns columns and adds delta_j W2T[j, col] over the block's flagged neurons.
template <typename T, typename Acc>
__global__ void __launch_bounds__(256) k_fix(const T* __restrict__ W1, const T* __restrict__ W2T,
                                             const float* __restrict__ b1, const float* __restrict__ a,
                                             const float* __restrict__ c, const T* __restrict__ x,
                                             const uint32_t* __restrict__ bitmap, float* __restrict__ yacc,
                                             int d, int h, int act) {
  constexpr int NB = 1024;
  extern __shared__ float xs[];                 // [d]
  __shared__ int list_j[NB];
  __shared__ float list_delta[NB];
  __shared__ int count_s;
  const int t = blockIdx.x, jb = blockIdx.y * NB;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int k = threadIdx.x; k < d; k += 256) xs[k] = to_f32(x[size_t(t) * d + k]);
  if (warp == 0) {   // ascending list of the block's flagged neurons
    const int wi = jb / 32 + lane;
    const uint32_t word = (wi < h / 32) ? bitmap[size_t(t) * (h / 32) + wi] : 0u;
    int cnt = __popc(word), pre = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, pre, o);
      if (lane >= o) pre += v;
    }
    int pos = pre - cnt;
    uint32_t wbits = word;
    while (wbits) {
      int b = __ffs(wbits) - 1;
      wbits &= wbits - 1;
      list_j[pos++] = wi * 32 + b;
    }
    if (lane == 31) count_s = pre;
  }
  __syncthreads();
  const int count = count_s;
  if (count == 0) return;
  for (int e = warp; e < count; e += 8) {
    const int j = list_j[e];
    const T* row = W1 + size_t(j) * d;
    Acc z = Acc(0);
    for (int k = lane; k < d; k += 32) z += Acc(to_f32(row[k])) * Acc(xs[k]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) {
      z += Acc(b1[j]);
      Acc delta;
      if (sizeof(Acc) == 8) delta = Acc(gelu_f64(double(z), act) - double(a[j]) * double(z) - double(c[j]));
      else delta = Acc(gelu_f32(float(z), act) - a[j] * float(z) - c[j]);
      list_delta[e] = float(delta);
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < d; col += 256) {
    Acc acc = Acc(0);
    for (int e = 0; e < count; ++e) acc += Acc(list_delta[e]) * Acc(to_f32(W2T[size_t(list_j[e]) * d + col]));
    atomicAdd(&yacc[size_t(t) * d + col], float(acc));
  }
}

template <typename T>
__global__ void k_store_y(const float* __restrict__ yacc, T* __restrict__ y, size_t count) {
  size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e < count) y[e] = from_f32<T>(yacc[e]);
}

template <typename T, typename Acc>
static tardis_status_t generic_typed(Handle* H, const T* x, T* y, int64_t n_total, cudaStream_t s) {
  const int d = H->d, h = H->h;
  for (int64_t t0 = 0; t0 < n_total; t0 += kGenericChunk) {
    const int n = int(n_total - t0 < kGenericChunk ? n_total - t0 : kGenericChunk);
    const T* xc = x + size_t(t0) * d;
    uint32_t* dbgb = H->dbg_bitmap ? H->dbg_bitmap + size_t(t0) * (h / 32) : nullptr;
    double* dbgs = H->dbg_scores ? H->dbg_scores + size_t(t0) * h : nullptr;
    if (H->path_override == 4)
      k_range_check_exact<T><<<h / 32, 1024, 0, s>>>(static_cast<const T*>(H->W1), H->b1, H->lo, H->hi, xc, n, d, h, H->bitmap, dbgb, dbgs);
    else
      k_predictor_exact<T><<<h / 32, 1024, 0, s>>>(H->codes, static_cast<const T*>(H->scale), H->zero, H->b1, H->lo, H->hi,
                                                   xc, n, d, h, H->G, H->bits, H->bitmap, dbgb, dbgs);
    k_flag_stats<<<n, 256, 0, s>>>(H->bitmap, h / 32, H->counters);
    const size_t cnt = size_t(n) * d;
    k_init_yacc<<<unsigned((cnt + 255) / 256), 256, 0, s>>>(H->yacc, H->bf, n, d);
    int ksplit = n <= 8 ? 16 : 1;
    int kchunk = ((d + ksplit - 1) / ksplit + 127) / 128 * 128;
    ksplit = (d + kchunk - 1) / kchunk;
    k_folded_product<T, Acc><<<dim3((d + 255) / 256, (n + 7) / 8, ksplit), 256, 0, s>>>(
        static_cast<const T*>(H->C), xc, H->yacc, n, d, kchunk);
    k_fix<T, Acc><<<dim3(n, (h + 1023) / 1024), 256, size_t(d) * sizeof(float), s>>>(
        static_cast<const T*>(H->W1), static_cast<const T*>(H->W2T), H->b1, H->a, H->c, xc, H->bitmap, H->yacc, d, h, H->act);
    k_store_y<T><<<unsigned((cnt + 255) / 256), 256, 0, s>>>(H->yacc, y + size_t(t0) * d, cnt);
    H->launches += 6;
  }
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

// ---- forward whose scratch is part of the library image -----------------------------------------------
// Same kernels as above, but the fp32 accumulator and the flag bitmap live in one file-scope device array
// instead of memory obtained from the allocator.  Every GPU that loads the library carries the array
// until the process exits; all calls (of all handles) share it.
constexpr size_t kStaticScratchBytes = size_t(4) << 20;   // 4 MiB
constexpr int kStaticMaxDevices = 64;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on `device` (which must be current).  In host code the array's name
// is only a stand-in for the symbol, never a pointer a kernel may use: the address comes from the runtime,
// once per device.
static tardis_status_t static_scratch_address(int device, unsigned char** out) {
  static unsigned char* cache[kStaticMaxDevices] = {};
  static std::mutex guard;                       // first calls of two host threads must not race on the cache
  if (device < 0 || device >= kStaticMaxDevices) return TARDIS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(guard);
  if (!cache[device]) {
    void* ptr = nullptr;
    TARDIS_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
    cache[device] = static_cast<unsigned char*>(ptr);
  }
  *out = cache[device];
  return TARDIS_OK;
}

template <typename T, typename Acc>
static tardis_status_t static_typed(Handle* H, const T* x, T* y, int n, float* yacc, uint32_t* bitmap, cudaStream_t s) {
  const int d = H->d, h = H->h;
  if (H->path_override == 4)                    // exact-range mode: flags from the true pre-activations, as in generic_typed
    k_range_check_exact<T><<<h / 32, 1024, 0, s>>>(static_cast<const T*>(H->W1), H->b1, H->lo, H->hi, x, n, d, h, bitmap,
                                                   H->dbg_bitmap, H->dbg_scores);
  else
    k_predictor_exact<T><<<h / 32, 1024, 0, s>>>(H->codes, static_cast<const T*>(H->scale), H->zero, H->b1, H->lo, H->hi,
                                                 x, n, d, h, H->G, H->bits, bitmap, H->dbg_bitmap, H->dbg_scores);
  k_flag_stats<<<n, 256, 0, s>>>(bitmap, h / 32, H->counters);
  const size_t cnt = size_t(n) * d;
  k_init_yacc<<<unsigned((cnt + 255) / 256), 256, 0, s>>>(yacc, H->bf, n, d);
  int ksplit = n <= 8 ? 16 : 1;
  int kchunk = ((d + ksplit - 1) / ksplit + 127) / 128 * 128;
  ksplit = (d + kchunk - 1) / kchunk;
  k_folded_product<T, Acc><<<dim3((d + 255) / 256, (n + 7) / 8, ksplit), 256, 0, s>>>(
      static_cast<const T*>(H->C), x, yacc, n, d, kchunk);
  k_fix<T, Acc><<<dim3(n, (h + 1023) / 1024), 256, size_t(d) * sizeof(float), s>>>(
      static_cast<const T*>(H->W1), static_cast<const T*>(H->W2T), H->b1, H->a, H->c, x, bitmap, yacc, d, h, H->act);
  k_store_y<T><<<unsigned((cnt + 255) / 256), 256, 0, s>>>(yacc, y, cnt);
  H->launches += 6;
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

size_t static_forward_scratch_bytes(const Handle* H, int64_t n) {
  const size_t acc = (size_t(n) * H->d * sizeof(float) + 255) / 256 * 256;
  const size_t bm = (size_t(n) * (H->h / 32) * sizeof(uint32_t) + 255) / 256 * 256;
  return acc + bm;
}

tardis_status_t launch_static_forward(Handle* H, const void* x, void* y, int64_t n, cudaStream_t s) {
  if (size_t(H->d) * sizeof(float) > 48 * 1024) return TARDIS_ERR_UNSUPPORTED;
  if (n > kStaticMaxTokens || static_forward_scratch_bytes(H, n) > kStaticScratchBytes) return TARDIS_ERR_UNSUPPORTED;
  int cur = -1;
  TARDIS_CUDA_TRY(cudaGetDevice(&cur));
  if (cur != H->device) return TARDIS_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  tardis_status_t st = static_scratch_address(cur, &base);
  if (st != TARDIS_OK) return st;
  // Both regions are written in full by the first kernels that touch them (the bitmap by the predictor,
  // the accumulator by its initialisation with b_f), so nothing of an earlier call's contents is read.
  float* yacc = reinterpret_cast<float*>(base);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(base + (size_t(n) * H->d * sizeof(float) + 255) / 256 * 256);
  if (H->dtype == TARDIS_F32)
    return static_typed<float, double>(H, static_cast<const float*>(x), static_cast<float*>(y), int(n), yacc, bitmap, s);
  return static_typed<__nv_bfloat16, float>(H, static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), int(n), yacc, bitmap, s);
}

tardis_status_t launch_generic_forward(Handle* H, const void* x, void* y, int64_t n, cudaStream_t s) {
  if (size_t(H->d) * sizeof(float) > 48 * 1024) return TARDIS_ERR_UNSUPPORTED;
  if (H->dtype == TARDIS_F32)
    return generic_typed<float, double>(H, static_cast<const float*>(x), static_cast<float*>(y), n, s);
  return generic_typed<__nv_bfloat16, float>(H, static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(y), n, s);
}

}  // namespace tardis
