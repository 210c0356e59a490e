// Building the predictor on the GPU: quantisation of W1 with the rounding error of every channel spread over the channels
// not yet rounded (GPTQ, which Section 6 of the paper names as the source of its 2-bit predictor).
//
// Per neuron (row of W1), channels in ascending order: when channel k opens a group, the group's grid (scale rounded to
// its storage type, zero-point) comes from the weights as they are then; q_k = clip(rint(w_k / s + z)),
// e_k = (w_k - s (q_k - z)) / U[k][k], and w_j <- w_j - e_k U[k][j] for j > k.  U is the upper Cholesky factor of the
// inverse Hessian of the layer's inputs, made by the caller; no U means the identity (plain rounding to nearest).
//
// Layout of the work: blocks of 64 channels.  k_block rounds the 64 channels of a block one after the other (a thread
// per neuron, the block's weights and the 64 x 64 corner of U in shared memory) and leaves the 64 errors of every neuron;
// k_spread then takes them to all later channels, for each (neuron, channel) in ascending order of k.  A channel thus
// sees exactly the sequence of subtractions of the channel-by-channel procedure, each a rounded product followed by a
// rounded difference in double precision (no fused multiply-add), so the codes equal those of a plain double-precision
// implementation bit for bit.
#include "common.cuh"

namespace tardis {
namespace {

constexpr int QB = 64;            // channels per block (divides the group size)
constexpr int QROWS = 64;         // neurons per CTA

template <typename T>
__global__ void k_widen(const T* __restrict__ W1, double* __restrict__ Wd, size_t count) {
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < count; i += size_t(gridDim.x) * blockDim.x)
    Wd[i] = double(to_f32<T>(W1[i]));
}

__device__ __forceinline__ double storage_round(double v, int dtype) {
  const float f = __double2float_rn(v);
  return dtype == TARDIS_F32 ? double(f) : double(__bfloat162float(__float2bfloat16_rn(f)));
}

// One block of 64 channels, one thread per neuron.
__global__ void __launch_bounds__(QROWS) k_block(double* __restrict__ Wd, const double* __restrict__ U, int h, int d, int b0, int G,
                                                 int levels, int dtype, double* __restrict__ scale64, double* __restrict__ zero64,
                                                 uint8_t* __restrict__ q, double* __restrict__ Eb) {
  extern __shared__ double sm[];
  double* Ws = sm;                          // [QROWS][QB + 1]
  double* Us = sm + QROWS * (QB + 1);       // [QB][QB]
  const int r0 = blockIdx.x * QROWS, tid = threadIdx.x;
  const int ng = d / G, nb = min(QB, d - b0);
  for (int e = tid; e < QROWS * QB; e += QROWS) {
    const int rr = e / QB, c = e - rr * QB;
    Ws[rr * (QB + 1) + c] = (r0 + rr < h && c < nb) ? Wd[size_t(r0 + rr) * d + b0 + c] : 0.0;
  }
  for (int e = tid; e < QB * QB; e += QROWS) {
    const int i = e / QB, j = e - i * QB;
    Us[e] = U ? ((i < nb && j < nb) ? U[size_t(b0 + i) * d + b0 + j] : 0.0) : (i == j ? 1.0 : 0.0);
  }
  __syncthreads();
  const int r = r0 + tid;
  if (r >= h) return;
  double* w = Ws + tid * (QB + 1);
  const int g = b0 / G;
  double s, z;
  if (b0 % G == 0) {                        // the block opens a group: its grid from the weights as they are now
    double wmin = 0.0, wmax = 0.0;
    for (int c = 0; c < G; ++c) {
      const double v = c < nb ? w[c] : Wd[size_t(r) * d + b0 + c];
      wmin = fmin(wmin, v);
      wmax = fmax(wmax, v);
    }
    s = storage_round(__ddiv_rn(__dsub_rn(wmax, wmin), double(levels)), dtype);
    if (!(s > 0.0)) s = 1.0;
    z = fmin(fmax(rint(__ddiv_rn(-wmin, s)), 0.0), double(levels));
    scale64[size_t(r) * ng + g] = s;
    zero64[size_t(r) * ng + g] = z;
  } else {
    s = scale64[size_t(r) * ng + g];
    z = zero64[size_t(r) * ng + g];
  }
  for (int i = 0; i < nb; ++i) {
    const double wi = w[i];
    const double qk = fmin(fmax(rint(__dadd_rn(__ddiv_rn(wi, s), z)), 0.0), double(levels));
    q[size_t(r) * d + b0 + i] = uint8_t(qk);
    const double e = __ddiv_rn(__dsub_rn(wi, __dmul_rn(s, qk - z)), Us[i * QB + i]);
    Eb[size_t(r) * QB + i] = e;
    for (int j = i + 1; j < nb; ++j) w[j] = __dsub_rn(w[j], __dmul_rn(e, Us[i * QB + j]));
  }
}

// W[r][j] <- W[r][j] - e[r][i] U[b0 + i][j], i = 0 .. nb - 1 in this order, for the channels j >= b0 + 64.
// CTA: 64 neurons x 64 channels; thread (tx, ty): channel tx, neurons 16 ty .. 16 ty + 15.
__global__ void __launch_bounds__(256) k_spread(double* __restrict__ Wd, const double* __restrict__ U, const double* __restrict__ Eb,
                                                int h, int d, int b0, int nb) {
  extern __shared__ double sm[];
  double (*Es)[QB] = reinterpret_cast<double (*)[QB]>(sm);                 // [QROWS][QB]
  double (*Ut)[QB] = reinterpret_cast<double (*)[QB]>(sm + QROWS * QB);    // [QB][QB]
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
  const int j0 = b0 + QB + blockIdx.x * QB, r0 = blockIdx.y * QROWS;
  for (int e = threadIdx.x; e < QROWS * QB; e += 256) {
    const int rr = e / QB, i = e - rr * QB;
    Es[rr][i] = (r0 + rr < h && i < nb) ? Eb[size_t(r0 + rr) * QB + i] : 0.0;
    Ut[rr][i] = (rr < nb && j0 + i < d) ? U[size_t(b0 + rr) * d + j0 + i] : 0.0;
  }
  __syncthreads();
  const int j = j0 + tx;
  if (j >= d) return;
  double w[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int r = r0 + ty * 16 + k;
    w[k] = r < h ? Wd[size_t(r) * d + j] : 0.0;
  }
  for (int i = 0; i < nb; ++i) {
    const double u = Ut[i][tx];
#pragma unroll
    for (int k = 0; k < 16; ++k) w[k] = __dsub_rn(w[k], __dmul_rn(Es[ty * 16 + k][i], u));
  }
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int r = r0 + ty * 16 + k;
    if (r < h) Wd[size_t(r) * d + j] = w[k];
  }
}

// codes into 32-bit words (channel order ascending, lowest bits first), scale into its storage type, zero-points into bytes
template <typename T>
__global__ void k_pack_out(const uint8_t* __restrict__ q, const double* __restrict__ scale64, const double* __restrict__ zero64,
                           int h, int d, int G, int bits, uint32_t* __restrict__ codes, T* __restrict__ scale, uint8_t* __restrict__ zero) {
  const int nw = d * bits / 32, ng = d / G;     // the row is one bit stream: code k holds bits [k bits, (k + 1) bits)
  const size_t words = size_t(h) * nw, groups = size_t(h) * ng;
  for (size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x; e < words; e += size_t(gridDim.x) * blockDim.x) {
    const size_t r = e / nw;
    const int wi = int(e - r * nw);
    uint32_t word = 0u;
    const int k0 = (wi * 32) / bits, k1 = min(d - 1, (wi * 32 + 31) / bits);    // codes with a bit in this word
    for (int k = k0; k <= k1; ++k) {
      const int sh = k * bits - wi * 32;                                        // (negative: the code started in the word before)
      const uint32_t c = q[r * d + k];
      word |= sh >= 0 ? c << sh : c >> (-sh);
    }
    codes[e] = word;
  }
  for (size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x; e < groups; e += size_t(gridDim.x) * blockDim.x) {
    scale[e] = from_f32<T>(float(scale64[e]));          // (already a value of the storage type: the conversion is exact)
    zero[e] = uint8_t(zero64[e]);
  }
}

}  // namespace

tardis_status_t launch_build_predictor(int h, int d, int dtype, const void* W1, const double* U, int bits, int G, uint32_t* codes,
                                       void* scale, uint8_t* zero, cudaStream_t s) {
  const int ng = d / G, levels = (1 << bits) - 1;
  double *Wd = nullptr, *Eb = nullptr, *scale64 = nullptr, *zero64 = nullptr;
  uint8_t* q = nullptr;
  auto release = [&]() {
    dev_free(Wd); dev_free(Eb); dev_free(scale64); dev_free(zero64); dev_free(q);
  };
  cudaError_t e = dev_malloc(&Wd, size_t(h) * d * sizeof(double));
  if (e == cudaSuccess) e = dev_malloc(&Eb, size_t(h) * QB * sizeof(double));
  if (e == cudaSuccess) e = dev_malloc(&scale64, size_t(h) * ng * sizeof(double));
  if (e == cudaSuccess) e = dev_malloc(&zero64, size_t(h) * ng * sizeof(double));
  if (e == cudaSuccess) e = dev_malloc(&q, size_t(h) * d);
  if (e != cudaSuccess) { release(); cudaGetLastError(); return TARDIS_ERR_ALLOC; }
  const size_t count = size_t(h) * d;
  if (dtype == TARDIS_F32) k_widen<float><<<2048, 256, 0, s>>>(static_cast<const float*>(W1), Wd, count);
  else k_widen<__nv_bfloat16><<<2048, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(W1), Wd, count);
  const size_t smem = (size_t(QROWS) * (QB + 1) + QB * QB) * sizeof(double);
  const size_t smem2 = (size_t(QROWS) * QB + QB * QB) * sizeof(double);
  e = cudaFuncSetAttribute(k_block, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_spread, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem2));
  for (int b0 = 0; b0 < d && e == cudaSuccess; b0 += QB) {
    const int nb = d - b0 < QB ? d - b0 : QB;
    k_block<<<(h + QROWS - 1) / QROWS, QROWS, smem, s>>>(Wd, U, h, d, b0, G, levels, dtype, scale64, zero64, q, Eb);
    const int later = d - (b0 + QB);
    if (U && later > 0) k_spread<<<dim3((later + QB - 1) / QB, (h + QROWS - 1) / QROWS), 256, smem2, s>>>(Wd, U, Eb, h, d, b0, nb);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) {
    if (dtype == TARDIS_F32) k_pack_out<float><<<1024, 256, 0, s>>>(q, scale64, zero64, h, d, G, bits, codes, static_cast<float*>(scale), zero);
    else k_pack_out<__nv_bfloat16><<<1024, 256, 0, s>>>(q, scale64, zero64, h, d, G, bits, codes, static_cast<__nv_bfloat16*>(scale), zero);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);      // the scratch goes away with this call
  release();
  if (e != cudaSuccess) { set_last_error(e, "tardis_build_predictor"); return TARDIS_ERR_CUDA; }
  return TARDIS_OK;
}

}  // namespace tardis
