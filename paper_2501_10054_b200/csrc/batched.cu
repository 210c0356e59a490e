// Batched / prefill form of the online path (Section 5.4) for bf16 layers: every step is a dense product on
// the tcgen05 tensor cores (gemm.cu) or a light elementwise pass.
//
// For a chunk of up to kChunk tokens X[n, d]:
//   1. fast predictor scores  Zhat = X What^T + b1, What = s (q - zp) (Section 5.3).  What needs 10 significant
//      bits (13 with 4-bit codes), so it is held as an exact sum of two bf16 matrices (hi + lo); one GEMM runs
//      over both and its epilogue turns the scores into flag words (they are stored only for the debug
//      capture).  Products are exact, the fp32 accumulation is not: a score within
//      tau(t, j) = kEps * (2^bits - 1) max_g s[j,g] * |x_t|_1 of a range end is queued by the epilogue and
//      re-evaluated in fp64 from the packed codes (k_recheck), so the flags are the exact ones;
//   2. speculative product    Yacc = X W_f^T + b_f                               (fp32);
//   3. result fixing          Delta = flag .* (GELU(Z) - a Z - c), Z = X W1^T + b1   (GEMM with that epilogue, bf16),
//                             y = bf16(Yacc + Delta W2^T)                            (GEMM over all neurons:
//      with independent ~10 % flags the union over >= 64 tokens is practically every neuron, which is why
//      the paper expects little gain for prompt-heavy requests).
#include <vector>

#include "common.cuh"
#include "exact.cuh"
#include "gemm.cuh"

namespace tardis {
namespace bat {

// Tokens per pass (the scratch is sized for this).  With 2048 the big products have 16 x 64 tiles = 6.9 waves of
// 148 CTAs; 1024-token chunks lost 15 % of the time to their last, partial wave.
constexpr int kChunk = 2048;
constexpr int kChunkCapture = 1024;          // ... while the debug capture is on (the score buffer holds that many)
constexpr float kEps = 7.62939453125e-6f;    // 2^-17: relative accumulation-error allowance of the fast scores
constexpr int kMaxRecheck = 1 << 21;         // (token, neuron) pairs per chunk that can queue for re-evaluation

struct State {
  __nv_bfloat16 *Wf, *W2, *What_hi, *What_lo;     // [d,d], [d,h], [h,d], [h,d]
  float* smaxrow;                                  // [h] largest group scale of a neuron
  float *zhat, *yacc, *x1;                         // [kChunkCapture,h] (scores for the capture; fold temporary), [kChunk,d], [kChunk]
  __nv_bfloat16* delta;                            // [kChunk,h]
  uint32_t* bitmap;                                // [kChunk,h/32]
  uint2* rlist;                                    // [kMaxRecheck] (token, neuron)
  unsigned int* rcount;                            // [2]: queued pairs (may exceed the queue), pairs settled in place
  size_t bytes_state, bytes_scratch;
};

// ---- set-up ---------------------------------------------------------------------------------------------
// What = s (q - zp) split exactly into hi = bf16(What) and lo = What - hi (at most 2 significant bits left).
__global__ void k_dequant_split(const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                                const uint8_t* __restrict__ zero, __nv_bfloat16* __restrict__ hi,
                                __nv_bfloat16* __restrict__ lo, float* __restrict__ smaxrow, int d, int G, int bits) {
  const int per = 32 / bits;                    // codes per word
  const uint32_t cmask = (1u << bits) - 1u;
  const int j = blockIdx.x, ng = d / G, nwords = d / per;
  if (32 % bits) {                              // 3-bit codes: a bit stream, channel by channel
    const uint32_t* row = codes + size_t(j) * (size_t(d) * bits / 32);
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
      const int g = k / G;
      const float v = __bfloat162float(scale[size_t(j) * ng + g]) * (float(stream_code(row, k, bits)) - float(zero[size_t(j) * ng + g]));
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      hi[size_t(j) * d + k] = h;
      lo[size_t(j) * d + k] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
  for (int w = threadIdx.x; w < nwords && 32 % bits == 0; w += blockDim.x) {
    const uint32_t word = codes[size_t(j) * nwords + w];
    const int g = (w * per) / G;
    const float s = __bfloat162float(scale[size_t(j) * ng + g]);
    const float zp = float(zero[size_t(j) * ng + g]);
    for (int q = 0; q < per; ++q) {
      const float v = s * (float((word >> (bits * q)) & cmask) - zp);   // exact: 8-bit significand times |int| <= 15
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      hi[size_t(j) * d + w * per + q] = h;
      lo[size_t(j) * d + w * per + q] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int g = 0; g < ng; ++g) m = fmaxf(m, fabsf(__bfloat162float(scale[size_t(j) * ng + g])));
    smaxrow[j] = m;
  }
}

// ---- per-chunk passes -----------------------------------------------------------------------------------
// |x_t|_1 (inf when the token holds a non-finite value: every neuron of it is then flagged)
__global__ void k_xnorm(const __nv_bfloat16* __restrict__ x, int d, float* __restrict__ x1) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  float s = 0.f;
  bool bad = false;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    const float v = __bfloat162float(x[size_t(t) * d + k]);
    if (!(fabsf(v) <= 3.0e38f)) bad = true;
    s += fabsf(v);
  }
  if (bad) s = __int_as_float(0x7f800000);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < (blockDim.x + 31) / 32; ++w) tot += red[w];
    x1[t] = tot;
  }
}

// One warp per queued pair: exact fp64 score from the packed codes decides the flag.
__global__ void k_recheck(const uint2* __restrict__ rlist, const unsigned int* __restrict__ rcount,
                          const uint32_t* __restrict__ codes, const __nv_bfloat16* __restrict__ scale,
                          const uint8_t* __restrict__ zero, const float* __restrict__ b1, const float* __restrict__ lo,
                          const float* __restrict__ hi, const __nv_bfloat16* __restrict__ x, int d, int h, int G, int bits,
                          uint32_t* __restrict__ bitmap, float* __restrict__ zhat, unsigned long long* counters) {
  const int lane = threadIdx.x & 31;
  const unsigned int total = min(rcount[0], (unsigned int)kMaxRecheck);
  const unsigned int nwarps = (gridDim.x * blockDim.x) >> 5;
  for (unsigned int e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; e < total; e += nwarps) {
    const uint2 pr = rlist[e];
    const int t = int(pr.x), j = int(pr.y);
    const double z = exact_score_wide(codes, scale, zero, x + size_t(t) * d, j, d, G, bits, lane) + double(b1[j]);
    if (lane == 0) {
      const bool inside = (double(lo[j]) <= z) && (z < double(hi[j]));
      uint32_t* wp = bitmap + size_t(t) * (h / 32) + (j >> 5);
      if (inside) atomicAnd(wp, ~(1u << (j & 31)));
      else atomicOr(wp, 1u << (j & 31));
      if (zhat) zhat[size_t(t) * h + j] = float(z);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    atomicAdd(&counters[CTR_RECHECKS], (unsigned long long)total + rcount[1]);
  }
}

__global__ void k_flag_counts(const uint32_t* __restrict__ bitmap, int words, unsigned long long* counters) {
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

__global__ void k_round_store(const float* __restrict__ yacc, __nv_bfloat16* __restrict__ y, size_t count) {
  const size_t e = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
  if (e + 3 < count) {
    const float4 v = *reinterpret_cast<const float4*>(yacc + e);
    __nv_bfloat162 o[2] = {__floats2bfloat162_rn(v.x, v.y), __floats2bfloat162_rn(v.z, v.w)};
    *reinterpret_cast<uint2*>(y + e) = *reinterpret_cast<const uint2*>(o);
  } else {
    for (size_t i = e; i < count; ++i) y[i] = __float2bfloat16_rn(yacc[i]);
  }
}

__global__ void k_capture(const uint32_t* __restrict__ bitmap, const float* __restrict__ zhat, const float* __restrict__ x1,
                          int n, int h, uint32_t* __restrict__ dbg_bitmap, double* __restrict__ dbg_scores) {
  const size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= size_t(n) * h) return;
  if (dbg_scores) {
    const int t = int(e / h);
    dbg_scores[e] = (x1[t] <= 3.0e38f) ? double(zhat[e]) : __longlong_as_double(0x7ff8000000000000ll);
  }
  if (dbg_bitmap && e < size_t(n) * (h / 32)) dbg_bitmap[e] = bitmap[e];
}

}  // namespace bat

using namespace bat;

template <typename T> __global__ void k_transpose_b(const T* __restrict__ in, T* __restrict__ out, int rows, int cols) {
  __shared__ T tile[32][33];
  int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int rr = r0 + r, cc = c0 + threadIdx.x;
    if (rr < rows && cc < cols) tile[r][threadIdx.x] = in[size_t(rr) * cols + cc];
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    int cc = c0 + r, rr = r0 + threadIdx.x;
    if (rr < rows && cc < cols) out[size_t(cc) * rows + rr] = tile[threadIdx.x][r];
  }
}

tardis_status_t batched_prepare(Handle* H) {
  H->bstate = nullptr;
  if (H->dtype != TARDIS_BF16) return TARDIS_OK;
  const int d = H->d, h = H->h;
  if (d % 8 || h % 32) return TARDIS_OK;
  State* S = new (std::nothrow) State();
  if (!S) return TARDIS_ERR_ALLOC;
  memset(S, 0, sizeof(*S));
  H->bstate = S;
  const size_t hd = size_t(h) * d;
  struct Req { void** p; size_t bytes; bool scratch; };
  Req reqs[] = {
      {reinterpret_cast<void**>(&S->Wf), size_t(d) * d * 2, false}, {reinterpret_cast<void**>(&S->W2), hd * 2, false},
      {reinterpret_cast<void**>(&S->What_hi), hd * 2, false},       {reinterpret_cast<void**>(&S->What_lo), hd * 2, false},
      {reinterpret_cast<void**>(&S->smaxrow), size_t(h) * 4, false},
      {reinterpret_cast<void**>(&S->zhat), size_t(kChunkCapture) * h * 4, true}, {reinterpret_cast<void**>(&S->yacc), size_t(kChunk) * d * 4, true},
      {reinterpret_cast<void**>(&S->x1), size_t(kChunk) * 4, true},       {reinterpret_cast<void**>(&S->delta), size_t(kChunk) * h * 2, true},
      {reinterpret_cast<void**>(&S->bitmap), size_t(kChunk) * (h / 32) * 4, true},
      {reinterpret_cast<void**>(&S->rlist), size_t(kMaxRecheck) * 8, true}, {reinterpret_cast<void**>(&S->rcount), 16, true}};
  for (const Req& r : reqs) {
    cudaError_t e = dev_malloc(r.p, r.bytes);
    if (e != cudaSuccess) { set_last_error(e, "cudaMalloc"); cudaGetLastError(); batched_release(H); return TARDIS_ERR_ALLOC; }
    (r.scratch ? S->bytes_scratch : S->bytes_state) += r.bytes;
  }
  H->bytes_folded += size_t(d) * d * 2;
  H->bytes_w2t += hd * 2;                       // second copy of W2 (original orientation)
  H->bytes_predictor += 2 * hd * 2 + size_t(h) * 4;
  H->bytes_scratch += S->bytes_scratch;
  return TARDIS_OK;
}

// a_j W1[j][k] in fp32, transposed to [k][j] and split into bf16 hi + lo (16 significant bits together)
__global__ void k_scale_transpose_split(const __nv_bfloat16* __restrict__ W1, const float* __restrict__ a,
                                        __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo, int h, int d) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int j = j0 + r, k = k0 + threadIdx.x;
    if (j < h && k < d) tile[r][threadIdx.x] = a[j] * __bfloat162float(W1[size_t(j) * d + k]);
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + r, j = j0 + threadIdx.x;
    if (j < h && k < d) {
      const float v = tile[threadIdx.x][r];
      const __nv_bfloat16 hv = __float2bfloat16_rn(v);
      hi[size_t(k) * h + j] = hv;
      lo[size_t(k) * h + j] = __float2bfloat16_rn(v - __bfloat162float(hv));
    }
  }
}

// rows [i0, i0 + rows) of W_f (fp32) rounded once to bf16 and stored as C[k][i]
__global__ void k_store_folded(const float* __restrict__ Wf32, __nv_bfloat16* __restrict__ C, int i0, int rows, int d) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int ii = r0 + r, k = k0 + threadIdx.x;
    if (ii < rows && k < d) tile[r][threadIdx.x] = Wf32[size_t(ii) * d + k];
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + r, ii = r0 + threadIdx.x;
    if (ii < rows && k < d) C[size_t(k) * d + i0 + ii] = __float2bfloat16_rn(tile[threadIdx.x][r]);
  }
}

// Constant folding (Section 5.2) on the tensor cores: W_f = W2 (diag(a) W1), with diag(a) W1 formed in fp32 and
// carried as two bf16 matrices so that the product keeps 16 significant bits of it; fp32 accumulation over
// all neurons, one rounding to bf16.  Uses the batched path's buffers as temporaries (they are filled later).
tardis_status_t launch_fold_tensor(Handle* H, const tardis_fold_desc_t* desc, cudaStream_t s) {
  State* S = static_cast<State*>(H->bstate);
  if (!S || H->dtype != TARDIS_BF16) return TARDIS_ERR_UNSUPPORTED;
  const int d = H->d, h = H->h;
  dim3 tb(32, 8);
  k_scale_transpose_split<<<dim3((d + 31) / 32, (h + 31) / 32), tb, 0, s>>>(static_cast<const __nv_bfloat16*>(H->W1), H->a,
                                                                            S->What_hi, S->What_lo, h, d);
  const size_t cap = size_t(kChunkCapture) * h;              // floats in the score buffer
  int rows_per = int(cap / d);
  rows_per = rows_per / 128 * 128;
  if (rows_per < 128) return TARDIS_ERR_UNSUPPORTED;
  for (int i0 = 0; i0 < d; i0 += rows_per) {
    const int rows = d - i0 < rows_per ? d - i0 : rows_per;
    GemmArgs g = {};
    g.M = rows; g.N = d; g.K1 = h; g.K2 = desc->flags == TARDIS_FOLD_BF16_INTERMEDIATE ? 0 : h;   // (study mode: leading term only)
    g.A1 = static_cast<const __nv_bfloat16*>(desc->W2) + size_t(i0) * h; g.lda1 = h; g.B1 = S->What_hi; g.ldb1 = h;
    g.A2 = g.A1; g.lda2 = h; g.B2 = S->What_lo; g.ldb2 = h;
    g.epilogue = GEMM_EPI_F32; g.out_f32 = S->zhat; g.ldo = d; g.error_word = &H->counters[CTR_ERROR];
    const tardis_status_t st = launch_gemm(g, s);
    if (st != TARDIS_OK) return st;
    k_store_folded<<<dim3((d + 31) / 32, (rows + 31) / 32), tb, 0, s>>>(S->zhat, static_cast<__nv_bfloat16*>(H->C), i0, rows, d);
  }
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

tardis_status_t batched_finish(Handle* H, const void* W2, cudaStream_t s) {
  State* S = static_cast<State*>(H->bstate);
  if (!S) return TARDIS_OK;
  const int d = H->d, h = H->h;
  const size_t hd = size_t(h) * d;
  dim3 tb(32, 8);
  // W_f[i][k] row-major (the GEMMs want the channel index contiguous in both operands): transpose of C
  k_transpose_b<__nv_bfloat16><<<dim3((d + 31) / 32, (d + 31) / 32), tb, 0, s>>>(static_cast<const __nv_bfloat16*>(H->C), S->Wf, d, d);
  if (W2) TARDIS_CUDA_TRY(cudaMemcpyAsync(S->W2, W2, hd * 2, cudaMemcpyDeviceToDevice, s));
  else      // (a handle read back from a file has only the transposed copy)
    k_transpose_b<__nv_bfloat16><<<dim3((d + 31) / 32, (h + 31) / 32), tb, 0, s>>>(static_cast<const __nv_bfloat16*>(H->W2T), S->W2, h, d);
  if (H->bits <= 4)   // (8-bit codes: the batched path is not used, see the dispatch)
    k_dequant_split<<<h, 256, 0, s>>>(H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero, S->What_hi, S->What_lo,
                                    S->smaxrow, d, H->G, H->bits);
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

void batched_release(Handle* H) {
  State* S = static_cast<State*>(H->bstate);
  if (!S) return;
  void* ptrs[] = {S->Wf, S->W2, S->What_hi, S->What_lo, S->smaxrow, S->zhat, S->yacc, S->x1, S->delta, S->bitmap, S->rlist, S->rcount};
  for (void* q : ptrs)
    if (q) dev_free(q);
  delete S;
  H->bstate = nullptr;
}

tardis_status_t launch_batched_forward(Handle* H, const void* xv, void* yv, int64_t n_total, cudaStream_t s) {
  State* S = static_cast<State*>(H->bstate);
  if (!S) return TARDIS_ERR_UNSUPPORTED;
  const int d = H->d, h = H->h;
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(xv);
  __nv_bfloat16* y = static_cast<__nv_bfloat16*>(yv);
  const bool keep_scores = H->dbg_bitmap || H->dbg_scores;
  const int chunk = keep_scores ? kChunkCapture : kChunk;
  for (int64_t t0 = 0; t0 < n_total; t0 += chunk) {
    const int n = int(n_total - t0 < chunk ? n_total - t0 : chunk);
    const __nv_bfloat16* xc = x + size_t(t0) * d;
    TARDIS_CUDA_TRY(cudaMemsetAsync(S->rcount, 0, 16, s));
    k_xnorm<<<n, 256, 0, s>>>(xc, d, S->x1);
    // 1. fast scores: one GEMM over the hi and lo halves of the dequantised predictor
    GemmArgs g = {};
    g.M = n; g.N = h; g.K1 = d; g.K2 = d;
    g.A1 = xc; g.lda1 = d; g.B1 = S->What_hi; g.ldb1 = d; g.A2 = xc; g.lda2 = d; g.B2 = S->What_lo; g.ldb2 = d;
    // its epilogue turns the scores into flag words and queues the pairs too close to a range end; the scores
    // themselves are stored only for the debug capture
    g.epilogue = GEMM_EPI_FLAGS; g.out_f32 = keep_scores ? S->zhat : nullptr; g.ldo = h; g.bias = H->b1;
    g.error_word = &H->counters[CTR_ERROR];
    g.lo = H->lo; g.hi = H->hi; g.colscale = S->smaxrow; g.rowscale = S->x1; g.keps = kEps * float((1 << H->bits) - 1);
    g.bitmap_out = S->bitmap; g.rlist = S->rlist; g.rcount = S->rcount; g.rcap = kMaxRecheck;
    g.codes = H->codes; g.scale = H->scale; g.zero = H->zero; g.xsrc = xc; g.d = d; g.G = H->G; g.bits = H->bits;
    tardis_status_t st = launch_gemm(g, s);
    if (st != TARDIS_OK) return st;
    k_recheck<<<H->num_sms * 4, 256, 0, s>>>(S->rlist, S->rcount, H->codes, static_cast<const __nv_bfloat16*>(H->scale), H->zero, H->b1,
                                             H->lo, H->hi, xc, d, h, H->G, H->bits, S->bitmap, keep_scores ? S->zhat : nullptr, H->counters);
    k_flag_counts<<<n, 256, 0, s>>>(S->bitmap, h / 32, H->counters);
    if (H->dbg_bitmap || H->dbg_scores) {
      const size_t cnt = size_t(n) * h;
      k_capture<<<unsigned((cnt + 255) / 256), 256, 0, s>>>(S->bitmap, S->zhat, S->x1, n, h,
                                                            H->dbg_bitmap ? H->dbg_bitmap + size_t(t0) * (h / 32) : nullptr,
                                                            H->dbg_scores ? H->dbg_scores + size_t(t0) * h : nullptr);
    }
    // A batch of one tile of tokens is bound by weight traffic and its products over d outputs have few
    // tiles: those split their channel range over several CTAs, which add into the fp32 accumulator.
    // (not in deterministic mode: the order of those additions is not fixed)
    const int splits = (n <= 128 && d <= 8192 && !H->deterministic) ? 4 : 1;
    // 2. speculative folded product
    GemmArgs f = {};
    f.M = n; f.N = d; f.K1 = d; f.A1 = xc; f.lda1 = d; f.B1 = S->Wf; f.ldb1 = d;
    f.epilogue = GEMM_EPI_F32; f.out_f32 = S->yacc; f.ldo = d; f.bias = H->bf; f.error_word = &H->counters[CTR_ERROR];
    f.splits = splits;
    if (splits > 1) TARDIS_CUDA_TRY(cudaMemsetAsync(S->yacc, 0, size_t(n) * d * sizeof(float), s));
    st = launch_gemm(f, s);
    if (st != TARDIS_OK) return st;
    // 3. result fixing: exact pre-activations of every neuron, masked correction, output product
    GemmArgs z = {};
    z.M = n; z.N = h; z.K1 = d; z.A1 = xc; z.lda1 = d; z.B1 = H->W1; z.ldb1 = d;
    z.epilogue = GEMM_EPI_DELTA; z.out_bf16 = S->delta; z.ldo = h; z.bias = H->b1; z.a = H->a; z.c = H->c; z.bitmap = S->bitmap;
    z.act = H->act; z.error_word = &H->counters[CTR_ERROR];
    st = launch_gemm(z, s);
    if (st != TARDIS_OK) return st;
    GemmArgs o = {};
    o.M = n; o.N = d; o.K1 = h; o.A1 = S->delta; o.lda1 = h; o.B1 = S->W2; o.ldb1 = h; o.ldo = d; o.error_word = &H->counters[CTR_ERROR];
    if (splits > 1) {
      o.epilogue = GEMM_EPI_F32; o.out_f32 = S->yacc; o.splits = splits;
    } else {
      o.epilogue = GEMM_EPI_ADD_BF16; o.out_bf16 = y + size_t(t0) * d; o.addend = S->yacc;
    }
    st = launch_gemm(o, s);
    if (st != TARDIS_OK) return st;
    if (splits > 1) {
      const size_t cnt = size_t(n) * d;
      k_round_store<<<unsigned((cnt / 4 + 255) / 256 + 1), 256, 0, s>>>(S->yacc, y + size_t(t0) * d, cnt);
    }
    H->launches += 9 + ((H->dbg_bitmap || H->dbg_scores) ? 1 : 0);
  }
  TARDIS_CUDA_TRY(cudaGetLastError());
  return TARDIS_OK;
}

}  // namespace tardis
