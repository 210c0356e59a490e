// Shared declarations of libtardis (internal; the public interface is include/tardis.h).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tardis.h"

namespace tardis {

constexpr uint64_t kMagic = 0x7A2D15F01DULL;
constexpr int kGenericChunk = 256;   // tokens per pass of the generic kernels (scratch is sized for this)
constexpr int kDecodeMaxTokens = 16; // largest batch the fused decode kernel takes (4 tokens per launch) on layers of up to 4096
                                     // channels; 13 on wider ones (measured against the batched path, see fused_max_tokens)
constexpr int kStaticMaxTokens = 64; // largest batch of the forward that keeps its scratch in the library image

// device counter slots
enum { CTR_FLAGGED_TOTAL = 0, CTR_FLAGGED_MAX = 1, CTR_ERROR = 2, CTR_RECHECKS = 3, CTR_TICKET = 4, CTR_LAST_UNION = 5, CTR_COUNT = 8 };

struct Handle {
  uint64_t magic;
  int d, h, dtype, act, G, ngroups;
  int bits;              // bits per predictor code (2, 4 or 8)
  size_t esize;
  int device;
  // state (device)
  void* W1;        // [h, d]   original rows (result fixing recomputes z_j from these)
  void* W2T;       // [h, d]   W2 transposed: row j = output weights of neuron j
  void* C;         // [d, d]   C[k, i] = W_f[i, k]  (the paper's folded matrix, row k = input channel k)
  float* bf;       // [d]
  float *lo, *hi, *a, *c, *b1;   // [h]; b1 is zeros when the layer has no bias
  uint32_t* codes; // [h, d/16]
  void* scale;     // [h, d/G]
  uint8_t* zero;   // [h, d/G]
  // fused-decode state (bf16 only; null otherwise)
  uint32_t* codes_mma;   // predictor codes re-packed into tensor-core fragment order
  float2* pmeta;         // [h/16 tiles][ngroups][16 rows] (scale, scale*zero)
  // scratch (device)
  float* yacc;           // [kGenericChunk, d] fp32 accumulator
  uint32_t* bitmap;      // [kGenericChunk, h/32]
  unsigned long long* counters;  // [CTR_COUNT]
  void* fscratch;        // fused decode state for calls of 1..4 tokens per launch (see fused.cu); null when not built
  int fused_max_tokens;  // calls of up to this many tokens go to that kernel when the path is chosen automatically
  void* dscratch;        // fused decode scratch (see decode.cu)
  size_t dscratch_bytes;
  void* bstate;          // batched / prefill state and scratch (see batched.cu); null when not built
  // debug capture (caller-owned)
  uint32_t* dbg_bitmap;
  double* dbg_scores;
  // host-side bookkeeping
  uint64_t calls, tokens, last_path, launches;
  cudaStream_t last_stream;
  int path_override;
  bool deterministic;    // y must not depend on the order in which partial sums arrive (tardis_set_deterministic)
  size_t bytes_folded, bytes_predictor, bytes_tables, bytes_w1, bytes_w2t, bytes_scratch;
  int num_sms;
};

void set_last_error(cudaError_t e, const char* where);

// Every device allocation of the library goes through here: cudaMalloc, or the failure that tardis_debug_fail_alloc
// has asked for (so that the clean-up after a failed allocation can be tested without exhausting a GPU).  The memory
// handed out sits between two guard areas that tardis_stats checks.
cudaError_t dev_malloc_raw(void** p, size_t bytes);
template <typename T> inline cudaError_t dev_malloc(T** p, size_t bytes) { return dev_malloc_raw(reinterpret_cast<void**>(p), bytes); }
void dev_free(void* p);   // what dev_malloc gave (null is fine)

#define TARDIS_CUDA_TRY(expr)                                  \
  do {                                                         \
    cudaError_t e__ = (expr);                                  \
    if (e__ != cudaSuccess) {                                  \
      ::tardis::set_last_error(e__, #expr);                    \
      return TARDIS_ERR_CUDA;                                  \
    }                                                          \
  } while (0)

// ---- kernels' host launchers (each returns after enqueueing on `s`) ----
tardis_status_t launch_fold(Handle* H, const tardis_fold_desc_t* desc, cudaStream_t s, bool skip_product = false);
tardis_status_t launch_fold_product(Handle* H, cudaStream_t s);   // the SIMT product alone
tardis_status_t launch_export_folded(Handle* H, void* Wf, float* bf, cudaStream_t s);
tardis_status_t launch_generic_forward(Handle* H, const void* x, void* y, int64_t n, cudaStream_t s);
tardis_status_t launch_static_forward(Handle* H, const void* x, void* y, int64_t n, cudaStream_t s);
tardis_status_t decode_prepare(Handle* H, cudaStream_t s);                 // builds codes_mma, pmeta, scratch
tardis_status_t launch_decode_forward(Handle* H, const void* x, void* y, int n, cudaStream_t s);
void decode_release(Handle* H);
tardis_status_t decode_read_stamps(long long* out, int max_ctas);
tardis_status_t fused_prepare(Handle* H, cudaStream_t s);                  // builds the state of fused.cu (bf16, d_model <= 4608)
tardis_status_t launch_fused_forward(Handle* H, const void* x, void* y, int n, cudaStream_t s);
void fused_release(Handle* H);
tardis_status_t fused_set_deterministic(Handle* H, bool on);               // allocates the partial-output buffer of the mode
tardis_status_t fused_read_stamps(long long* out, int max_ctas);
tardis_status_t launch_wait_that_runs_out(Handle* H, long long limit_cycles, cudaStream_t s);   // UNSUPPORTED unless built with TARDIS_PHASE_STAMPS
tardis_status_t batched_prepare(Handle* H);                                                   // bf16 only: allocations
tardis_status_t batched_finish(Handle* H, const void* W2, cudaStream_t s);   // fills the batched state (W2 null: from W2T)
tardis_status_t launch_batched_forward(Handle* H, const void* x, void* y, int64_t n, cudaStream_t s);
void batched_release(Handle* H);
tardis_status_t launch_stack_forward(const tardis_stack_desc_t* desc, const void* x, void* y, void* work, void* keep, int64_t n,
                                     cudaStream_t s);   // stack.cu; arguments checked by the caller
tardis_status_t launch_build_predictor(int h, int d, int dtype, const void* W1, const double* U, int bits, int G, uint32_t* codes,
                                       void* scale, uint8_t* zero, cudaStream_t s);   // gptq.cu; arguments checked by the caller
tardis_status_t launch_fold_tensor(Handle* H, const tardis_fold_desc_t* desc, cudaStream_t s);  // bf16 fold on the tensor cores

// ---- small device helpers ----
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// offline statistics (calibrate.cu)
tardis_status_t launch_neuron_thresholds(int h, int n, const float* z, long long ldz, const float* b1, const float* lo, const float* hi,
                                         int act, double t_layer, double t_min, double t_max, float* err, float* t, cudaStream_t s);
tardis_status_t launch_calibrate(int h, int n, const float* z, long long ldz, const float* b1, double q_lo, double q_hi, int act,
                                 float* lo, float* hi, float* a, float* c, cudaStream_t s);

tardis_status_t launch_range_search(int h, int n, const float* z, long long ldz, const float* b1, const float* thr, double t_all,
                                    double step, int act, float* lo, float* hi, float* a, float* c, int* steps_out, cudaStream_t s);

// the activation (the name is historical: ReLU is served too)
__device__ __forceinline__ float gelu_f32(float z, int act) {
  if (act == TARDIS_ACT_RELU) return z > 0.f ? z : 0.f * z;      // 0 * z keeps NaN a NaN
  if (act == TARDIS_ACT_GELU_TANH) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + tanhf(u));
  }
  return 0.5f * z * (1.0f + erff(z * 0.7071067811865476f));
}
__device__ __forceinline__ double gelu_f64(double z, int act) {
  if (act == TARDIS_ACT_RELU) return z > 0.0 ? z : 0.0 * z;
  if (act == TARDIS_ACT_GELU_TANH) {
    double u = 0.7978845608028654 * (z + 0.044715 * z * z * z);
    return 0.5 * z * (1.0 + tanh(u));
  }
  return 0.5 * z * (1.0 + erf(z * 0.7071067811865476));
}

}  // namespace tardis
