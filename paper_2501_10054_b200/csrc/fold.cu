// Offline constant folding (Section 5.2): C = W1^T diag(a) W2^T-transposed, i.e.
//   C[k, i] = W_f[i, k] = sum_j W2[i, j] a_j W1[j, k],   b_f = W2 (a .* b1 + c) + b2,
// plus the W2 -> W2T[h, d] transpose that makes a neuron's output weights contiguous.
// Accumulation is fp32 for bf16 storage and fp64 for fp32 storage; one rounding at the end
// (the paper's precision study, Section 7.7, shows bf16 intermediates are not good enough).
#include "common.cuh"

namespace tardis {

// ---- W2[d, h] -> W2T[h, d] -------------------------------------------------------------
template <typename T>
__global__ void k_transpose(const T* __restrict__ in, T* __restrict__ out, int rows, int cols) {
  __shared__ T tile[32][33];
  int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int rr = r0 + r, cc = c0 + threadIdx.x;
    if (rr < rows && cc < cols) tile[r][threadIdx.x] = in[size_t(rr) * cols + cc];
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int cc = c0 + r, rr = r0 + threadIdx.x;   // out[cc][rr]
    if (rr < rows && cc < cols) out[size_t(cc) * rows + rr] = tile[threadIdx.x][r];
  }
}

// ---- C[k, i] = sum_j a_j W1[j, k] W2T[j, i] --------------------------------------------
// Both operands are read along their contiguous dimension.  Block 16x16 threads, tile
// (16*TM) x (16*TM), TM x TM outputs per thread, 16 neurons per step.
template <typename T, typename Acc, int TM>
__global__ void __launch_bounds__(256) k_fold_gemm(const T* __restrict__ W1, const T* __restrict__ W2T,
                                                   const float* __restrict__ a, T* __restrict__ C, int d, int h) {
  constexpr int TILE = 16 * TM, JS = 16;
  __shared__ Acc As[JS][TILE];   // a_j * W1[j, k0 + .]
  __shared__ Acc Bs[JS][TILE];   // W2T[j, i0 + .]
  const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * 16 + tx;
  const int k0 = blockIdx.y * TILE, i0 = blockIdx.x * TILE;
  Acc acc[TM][TM];
#pragma unroll
  for (int p = 0; p < TM; ++p)
#pragma unroll
    for (int q = 0; q < TM; ++q) acc[p][q] = Acc(0);
  for (int j0 = 0; j0 < h; j0 += JS) {
    // 16 rows x TILE columns per operand; 256 threads -> TM elements each
    for (int e = tid; e < JS * TILE; e += 256) {
      int r = e / TILE, cc = e % TILE;
      int j = j0 + r;
      Acc va = Acc(0), vb = Acc(0);
      if (j < h) {
        if (k0 + cc < d) va = Acc(a[j]) * Acc(to_f32(W1[size_t(j) * d + k0 + cc]));
        if (i0 + cc < d) vb = Acc(to_f32(W2T[size_t(j) * d + i0 + cc]));
      }
      As[r][cc] = va;
      Bs[r][cc] = vb;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < JS; ++r) {
      Acc av[TM], bv[TM];
#pragma unroll
      for (int p = 0; p < TM; ++p) av[p] = As[r][ty * TM + p];
#pragma unroll
      for (int q = 0; q < TM; ++q) bv[q] = Bs[r][q * 16 + tx];
#pragma unroll
      for (int p = 0; p < TM; ++p)
#pragma unroll
        for (int q = 0; q < TM; ++q) acc[p][q] += av[p] * bv[q];
    }
    __syncthreads();
  }
#pragma unroll
  for (int p = 0; p < TM; ++p) {
    int k = k0 + ty * TM + p;
    if (k >= d) continue;
#pragma unroll
    for (int q = 0; q < TM; ++q) {
      int i = i0 + q * 16 + tx;
      if (i < d) C[size_t(k) * d + i] = from_f32<T>(float(acc[p][q]));
    }
  }
}

// ---- b_f[i] = sum_j W2T[j, i] (a_j b1_j + c_j) + b2_i -----------------------------------
template <typename T>
__global__ void __launch_bounds__(256) k_fold_bias(const T* __restrict__ W2T, const float* __restrict__ a,
                                                   const float* __restrict__ c, const float* __restrict__ b1,
                                                   const float* __restrict__ b2, float* __restrict__ bf, int d, int h) {
  __shared__ double red[8][32];
  const int i = blockIdx.x * 32 + threadIdx.x;
  double acc = 0.0;
  if (i < d)
    for (int j = threadIdx.y; j < h; j += 8)
      acc += double(to_f32(W2T[size_t(j) * d + i])) * (double(a[j]) * double(b1[j]) + double(c[j]));
  red[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.y == 0 && i < d) {
    double s = 0.0;
    for (int r = 0; r < 8; ++r) s += red[r][threadIdx.x];
    bf[i] = float(s + (b2 ? double(b2[i]) : 0.0));
  }
}

template <typename T>
static tardis_status_t fold_typed(Handle* H, const tardis_fold_desc_t* desc, cudaStream_t s, bool skip_product) {
  const int d = H->d, h = H->h;
  dim3 tb(32, 8);
  k_transpose<T><<<dim3((h + 31) / 32, (d + 31) / 32), tb, 0, s>>>(static_cast<const T*>(desc->W2), static_cast<T*>(H->W2T), d, h);
  if (skip_product) {
    // the caller forms the product on the tensor cores
  } else if (sizeof(T) == 4) {
    constexpr int TM = 4;
    dim3 g((d + 16 * TM - 1) / (16 * TM), (d + 16 * TM - 1) / (16 * TM));
    k_fold_gemm<T, double, TM><<<g, dim3(16, 16), 0, s>>>(static_cast<const T*>(H->W1), static_cast<const T*>(H->W2T), H->a,
                                                          static_cast<T*>(H->C), d, h);
  } else {
    constexpr int TM = 8;
    dim3 g((d + 16 * TM - 1) / (16 * TM), (d + 16 * TM - 1) / (16 * TM));
    k_fold_gemm<T, float, TM><<<g, dim3(16, 16), 0, s>>>(static_cast<const T*>(H->W1), static_cast<const T*>(H->W2T), H->a,
                                                         static_cast<T*>(H->C), d, h);
  }
  k_fold_bias<T><<<(d + 31) / 32, tb, 0, s>>>(static_cast<const T*>(H->W2T), H->a, H->c, H->b1, desc->b2, H->bf, d, h);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t launch_fold(Handle* H, const tardis_fold_desc_t* desc, cudaStream_t s, bool skip_product) {
  const size_t h = H->h, d = H->d, ng = H->ngroups;
  const cudaMemcpyKind D2D = cudaMemcpyDeviceToDevice;
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->W1, desc->W1, h * d * H->esize, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->lo, desc->lo, h * 4, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->hi, desc->hi, h * 4, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->a, desc->a, h * 4, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->c, desc->c, h * 4, D2D, s));
  if (desc->b1) TARDIS_CUDA_TRY(cudaMemcpyAsync(H->b1, desc->b1, h * 4, D2D, s));
  else TARDIS_CUDA_TRY(cudaMemsetAsync(H->b1, 0, h * 4, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->codes, desc->pred_codes, h * d / 8 * H->bits, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->scale, desc->pred_scale, h * ng * H->esize, D2D, s));
  TARDIS_CUDA_TRY(cudaMemcpyAsync(H->zero, desc->pred_zero, h * ng, D2D, s));
  TARDIS_CUDA_TRY(cudaMemsetAsync(H->counters, 0, CTR_COUNT * sizeof(unsigned long long), s));
  if (H->dtype == TARDIS_F32) return fold_typed<float>(H, desc, s, skip_product);
  return fold_typed<__nv_bfloat16>(H, desc, s, skip_product);
}

tardis_status_t launch_fold_product(Handle* H, cudaStream_t s) {
  const int d = H->d, h = H->h;
  if (H->dtype != TARDIS_BF16) return TARDIS_ERR_UNSUPPORTED;
  constexpr int TM = 8;
  dim3 g((d + 16 * TM - 1) / (16 * TM), (d + 16 * TM - 1) / (16 * TM));
  k_fold_gemm<__nv_bfloat16, float, TM><<<g, dim3(16, 16), 0, s>>>(static_cast<const __nv_bfloat16*>(H->W1),
                                                                   static_cast<const __nv_bfloat16*>(H->W2T), H->a,
                                                                   static_cast<__nv_bfloat16*>(H->C), d, h);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t launch_export_folded(Handle* H, void* Wf, float* bf, cudaStream_t s) {
  const int d = H->d;
  if (Wf) {
    dim3 g((d + 31) / 32, (d + 31) / 32), tb(32, 8);
    if (H->dtype == TARDIS_F32) k_transpose<float><<<g, tb, 0, s>>>(static_cast<const float*>(H->C), static_cast<float*>(Wf), d, d);
    else k_transpose<__nv_bfloat16><<<g, tb, 0, s>>>(static_cast<const __nv_bfloat16*>(H->C), static_cast<__nv_bfloat16*>(Wf), d, d);
    TARDIS_CUDA_TRY(cudaGetLastError());
  }
  if (bf) TARDIS_CUDA_TRY(cudaMemcpyAsync(bf, H->bf, size_t(d) * 4, cudaMemcpyDeviceToDevice, s));
  return TARDIS_OK;
}

}  // namespace tardis
