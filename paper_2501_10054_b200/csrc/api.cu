// C ABI of libtardis: argument validation, handle life cycle, dispatch.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include <atomic>
#include <mutex>
#include <unordered_map>
#include <vector>
#include "common.cuh"
#include "gemm.cuh"

namespace tardis {

static thread_local char g_last_error[256] = "";

void set_last_error(cudaError_t e, const char* where) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e), where);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static Handle* check(tardis_handle_t h) {
  Handle* H = reinterpret_cast<Handle*>(h);
  if (!H || H->magic != kMagic) return nullptr;
  return H;
}

// A handle's memory and kernels belong to the device that was current at tardis_fold: a call made with another device
// current would launch there against this handle's pointers.
static std::atomic<int> g_fail_alloc{-1};   // >= 0: that many allocations still succeed, the next one fails (once)

// Every allocation carries 256 guard bytes of a fixed pattern in front of and behind what the caller gets; tardis_stats
// looks at the guards of the handle's allocations and reports TARDIS_ERR_CORRUPT when a kernel has written past an end.
constexpr size_t kGuard = 256;
constexpr int kGuardByte = 0xA5;
struct Allocation { char* base; size_t bytes; const void* owner; int device; };
static std::mutex g_alloc_mutex;
static std::unordered_map<const void*, Allocation> g_allocs;        // keyed by the pointer handed out
static thread_local const void* g_alloc_owner = nullptr;            // the handle whose entry point is running on this thread
struct OwnerScope {
  explicit OwnerScope(const void* o) { g_alloc_owner = o; }
  ~OwnerScope() { g_alloc_owner = nullptr; }
};

cudaError_t dev_malloc_raw(void** p, size_t bytes) {
  *p = nullptr;
  if (g_fail_alloc.load() >= 0 && g_fail_alloc.fetch_sub(1) == 0) return cudaErrorMemoryAllocation;
  char* base = nullptr;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&base), bytes + 2 * kGuard);
  if (e != cudaSuccess) return e;
  e = cudaMemset(base, kGuardByte, kGuard);
  if (e == cudaSuccess) e = cudaMemset(base + kGuard + bytes, kGuardByte, kGuard);
  if (e != cudaSuccess) { cudaFree(base); return e; }
  int dev = -1;
  cudaGetDevice(&dev);
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    g_allocs[base + kGuard] = Allocation{base, bytes, g_alloc_owner, dev};
  }
  *p = base + kGuard;
  return cudaSuccess;
}

void dev_free(void* p) {
  if (!p) return;
  char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    auto it = g_allocs.find(p);
    if (it != g_allocs.end()) { base = it->second.base; g_allocs.erase(it); }
  }
  cudaFree(base ? static_cast<void*>(base) : p);
}

// Number of damaged guards among the allocations of `owner` (both guards of every allocation are read back); -1 on a CUDA error.
static int damaged_guards(const void* owner) {
  std::vector<Allocation> mine;
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    for (const auto& kv : g_allocs)
      if (kv.second.owner == owner) mine.push_back(kv.second);
  }
  int bad = 0;
  unsigned char buf[2 * kGuard];
  for (const Allocation& al : mine) {
    if (cudaMemcpy(buf, al.base, kGuard, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    if (cudaMemcpy(buf + kGuard, al.base + kGuard + al.bytes, kGuard, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    bool ok = true;
    for (size_t i = 0; i < 2 * kGuard; ++i) ok = ok && buf[i] == kGuardByte;
    bad += ok ? 0 : 1;
  }
  return bad;
}

static bool on_handle_device(const Handle* H) {
  int cur = -1;
  return cudaGetDevice(&cur) == cudaSuccess && cur == H->device;
}

template <typename T>
static tardis_status_t dev_alloc(T** p, size_t count, size_t* tally) {
  *p = nullptr;
  size_t bytes = count * sizeof(T);
  cudaError_t e = dev_malloc(reinterpret_cast<void**>(p), bytes ? bytes : 16);
  if (e != cudaSuccess) {
    set_last_error(e, "cudaMalloc");
    cudaGetLastError();
    return TARDIS_ERR_ALLOC;
  }
  if (tally) *tally += bytes;
  return TARDIS_OK;
}

static void free_all(Handle* H) {
  fused_release(H);
  decode_release(H);
  batched_release(H);
  void* ptrs[] = {H->W1, H->W2T, H->C, H->bf, H->lo, H->hi, H->a, H->c, H->b1, H->codes, H->scale,
                  H->zero, H->yacc, H->bitmap, H->counters};
  for (void* p : ptrs)
    if (p) dev_free(p);
  H->magic = 0;
  delete H;
}

// Allocates a handle and its device arrays for a layer of the given shape (nothing is filled in yet).
static tardis_status_t new_handle(int d, int h, int dtype, int act, int G, int bits, cudaStream_t s, Handle** out) {
  *out = nullptr;
  Handle* H = new (std::nothrow) Handle();
  if (!H) return TARDIS_ERR_ALLOC;
  memset(H, 0, sizeof(*H));
  g_alloc_owner = H;                                   // (the entry point that called this resets it when it returns)
  H->magic = kMagic;
  H->d = d; H->h = h; H->dtype = dtype; H->act = act; H->G = G; H->ngroups = d / G;
  H->bits = bits;
  H->esize = dtype == TARDIS_F32 ? 4 : 2;
  H->last_stream = s;
  cudaError_t e = cudaGetDevice(&H->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&H->num_sms, cudaDevAttrMultiProcessorCount, H->device);
  if (e != cudaSuccess) { set_last_error(e, "device query"); delete H; return TARDIS_ERR_CUDA; }
  const size_t hd = size_t(h) * d;
  tardis_status_t st = TARDIS_OK;
  auto A = [&](auto** p, size_t count, size_t* tally) { if (st == TARDIS_OK) st = dev_alloc(p, count, tally); };
  A(reinterpret_cast<char**>(&H->W1), hd * H->esize, &H->bytes_w1);
  A(reinterpret_cast<char**>(&H->W2T), hd * H->esize, &H->bytes_w2t);
  A(reinterpret_cast<char**>(&H->C), size_t(d) * d * H->esize, &H->bytes_folded);
  A(&H->bf, size_t(d), &H->bytes_folded);
  A(&H->lo, size_t(h), &H->bytes_tables);
  A(&H->hi, size_t(h), &H->bytes_tables);
  A(&H->a, size_t(h), &H->bytes_tables);
  A(&H->c, size_t(h), &H->bytes_tables);
  A(&H->b1, size_t(h), &H->bytes_tables);
  A(&H->codes, hd * H->bits / 32, &H->bytes_predictor);
  A(reinterpret_cast<char**>(&H->scale), size_t(h) * H->ngroups * H->esize, &H->bytes_predictor);
  A(&H->zero, size_t(h) * H->ngroups, &H->bytes_predictor);
  A(&H->yacc, size_t(kGenericChunk) * d, &H->bytes_scratch);
  A(&H->bitmap, size_t(kGenericChunk) * (h / 32), &H->bytes_scratch);
  A(&H->counters, size_t(CTR_COUNT), &H->bytes_scratch);
  if (st != TARDIS_OK) { free_all(H); return st; }
  *out = H;
  return TARDIS_OK;
}

}  // namespace tardis

using namespace tardis;

extern "C" {

tardis_status_t tardis_fold(const tardis_fold_desc_t* desc, tardis_stream_t stream, tardis_handle_t* out) {
  if (!desc || !out) return TARDIS_ERR_INVALID_ARG;
  *out = nullptr;
  const int d = desc->d_model, h = desc->d_ff, G = desc->pred_group;
  if (d <= 0 || h <= 0 || G <= 0) return TARDIS_ERR_INVALID_ARG;
  if (desc->dtype != TARDIS_F32 && desc->dtype != TARDIS_BF16) return TARDIS_ERR_INVALID_ARG;
  if (desc->act != TARDIS_ACT_GELU_TANH && desc->act != TARDIS_ACT_GELU_ERF && desc->act != TARDIS_ACT_RELU) return TARDIS_ERR_INVALID_ARG;
  if (desc->flags > TARDIS_FOLD_FP32_PLAIN) return TARDIS_ERR_INVALID_ARG;
  if (d % 8 || h % 32 || G % 16 || d % G) return TARDIS_ERR_INVALID_ARG;
  if (desc->pred_bits != 2 && desc->pred_bits != 3 && desc->pred_bits != 4 && desc->pred_bits != 8)
    return desc->pred_bits > 0 && desc->pred_bits <= 8 ? TARDIS_ERR_UNSUPPORTED : TARDIS_ERR_INVALID_ARG;
  if (desc->pred_bits == 3 && d % 32) return TARDIS_ERR_INVALID_ARG;      // (a row of 3-bit codes is a whole number of words)
  const void* required[] = {desc->W1, desc->W2, desc->lo, desc->hi, desc->a, desc->c,
                            desc->pred_codes, desc->pred_scale, desc->pred_zero};
  for (const void* p : required)
    if (!p) return TARDIS_ERR_INVALID_ARG;
  const void* al[] = {desc->W1, desc->W2, desc->pred_codes, desc->pred_scale};
  for (const void* p : al)
    if (!aligned16(p)) return TARDIS_ERR_INVALID_ARG;

  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  Handle* H = nullptr;
  OwnerScope scope(nullptr);                           // new_handle names the owner of the allocations that follow
  tardis_status_t st = new_handle(d, h, desc->dtype, desc->act, G, desc->pred_bits, s, &H);
  if (st != TARDIS_OK) return st;

  const bool bf16 = H->dtype == TARDIS_BF16;
  if (bf16) st = batched_prepare(H);                          // allocations; its buffers double as fold temporaries
  const bool tensor_fold = st == TARDIS_OK && bf16 && H->bstate != nullptr && desc->flags != TARDIS_FOLD_FP32_PLAIN;
  if (st == TARDIS_OK) st = launch_fold(H, desc, s, tensor_fold);   // (computes the product itself when tensor_fold is false)
  if (st == TARDIS_OK && tensor_fold) {
    st = launch_fold_tensor(H, desc, s);
    if (st == TARDIS_ERR_UNSUPPORTED) st = launch_fold_product(H, s);   // no tensor-map support: plain kernel
  }
  if (st == TARDIS_OK && bf16) st = fused_prepare(H, s);
  if (st == TARDIS_OK && bf16 && !H->fscratch) st = decode_prepare(H, s);   // wider layers: the older per-token kernel
  if (st == TARDIS_OK && bf16) st = batched_finish(H, desc->W2, s);
  if (st != TARDIS_OK) { cudaStreamSynchronize(s); free_all(H); return st; }
  *out = reinterpret_cast<tardis_handle_t>(H);
  return TARDIS_OK;
}

tardis_status_t tardis_ffn_forward(tardis_handle_t handle, const void* x, void* y, int64_t n_tokens,
                                   tardis_stream_t stream) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  if (n_tokens < 0) return TARDIS_ERR_INVALID_ARG;
  if (n_tokens == 0) return TARDIS_OK;
  if (!x || !y || !aligned16(x) || !aligned16(y)) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  H->last_stream = s;
  tardis_status_t st;
  // (deterministic mode: only the kernels of fused.cu and the tensor-core products without a split channel range qualify)
  const bool has_fused = H->fscratch != nullptr || (H->codes_mma != nullptr && !H->deterministic);
  const bool fused = has_fused && ((H->path_override == 0 && n_tokens <= (H->fscratch ? H->fused_max_tokens : 8)) || (H->path_override == 2 && n_tokens <= 4096));
  // (8-bit codes times a bf16 scale do not fit the exact two-term bf16 form the batched scores rely on)
  const bool batched = ((H->path_override == 0 && !fused) || H->path_override == 3) && H->bstate != nullptr && H->bits <= 4;
  if (H->deterministic && !fused && !batched) return TARDIS_ERR_UNSUPPORTED;
  if (fused) {
    st = H->fscratch ? launch_fused_forward(H, x, y, int(n_tokens), s) : launch_decode_forward(H, x, y, int(n_tokens), s);
    H->last_path = 2;
  } else if (batched) {
    st = launch_batched_forward(H, x, y, n_tokens, s);
    H->last_path = 3;
  } else {
    st = launch_generic_forward(H, x, y, n_tokens, s);
    H->last_path = 1;
  }
  if (st == TARDIS_OK) { H->calls += 1; H->tokens += uint64_t(n_tokens); }
  return st;
}

tardis_status_t tardis_ffn_forward_static(tardis_handle_t handle, const void* x, void* y, int64_t n_tokens,
                                         tardis_stream_t stream) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  if (n_tokens < 0) return TARDIS_ERR_INVALID_ARG;
  if (n_tokens == 0) return TARDIS_OK;
  if (!x || !y || !aligned16(x) || !aligned16(y)) return TARDIS_ERR_INVALID_ARG;
  if (n_tokens > kStaticMaxTokens) {
    snprintf(g_last_error, sizeof(g_last_error), "tardis_ffn_forward_static: n_tokens %lld exceeds the limit of %d",
             (long long)n_tokens, kStaticMaxTokens);
    return TARDIS_ERR_UNSUPPORTED;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  H->last_stream = s;
  const tardis_status_t st = launch_static_forward(H, x, y, n_tokens, s);
  if (st == TARDIS_ERR_UNSUPPORTED)
    snprintf(g_last_error, sizeof(g_last_error),
             "tardis_ffn_forward_static: n_tokens * (4 d_model + d_ff / 8) exceeds the 4 MiB of built-in scratch (or d_model > 12288)");
  if (st == TARDIS_OK) { H->last_path = 5; H->calls += 1; H->tokens += uint64_t(n_tokens); }
  return st;
}

tardis_status_t tardis_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int32_t lda, const void* B, int32_t ldb,
                                 float* C, int32_t ldc, tardis_stream_t stream) {
  if (!A || !B || !C || M <= 0 || N <= 0 || K <= 0 || ldc < N) return TARDIS_ERR_INVALID_ARG;
  if (!aligned16(C)) return TARDIS_ERR_INVALID_ARG;   // the epilogue stores (and reduces) 16 bytes at a time when ldc % 4 == 0
  GemmArgs g = {};
  g.M = M; g.N = N; g.K1 = K; g.K2 = 0;
  g.A1 = A; g.B1 = B; g.lda1 = lda; g.ldb1 = ldb;
  g.epilogue = GEMM_EPI_F32; g.out_f32 = C; g.ldo = ldc;
  return launch_gemm(g, reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_calibrate(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1, double q_lo,
                                 double q_hi, int32_t act, float* lo, float* hi, float* a, float* c, tardis_stream_t stream) {
  if (d_ff <= 0 || n_cal <= 0 || !z || ldz < n_cal || !lo || !hi || !a || !c) return TARDIS_ERR_INVALID_ARG;
  if (!(q_lo >= 0.0 && q_lo <= q_hi && q_hi <= 1.0)) return TARDIS_ERR_INVALID_ARG;
  if (act != TARDIS_ACT_GELU_TANH && act != TARDIS_ACT_GELU_ERF && act != TARDIS_ACT_RELU) return TARDIS_ERR_INVALID_ARG;
  return launch_calibrate(d_ff, n_cal, z, ldz, b1, q_lo, q_hi, act, lo, hi, a, c, reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_range_search(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1, const float* thresholds,
                                    double threshold, double step, int32_t act, float* lo, float* hi, float* a, float* c,
                                    int32_t* steps_taken, tardis_stream_t stream) {
  if (d_ff <= 0 || n_cal <= 0 || !z || ldz < n_cal || !lo || !hi || !a || !c) return TARDIS_ERR_INVALID_ARG;
  if (!(step > 0.0) || (!thresholds && !(threshold >= 0.0 && threshold <= 1.0))) return TARDIS_ERR_INVALID_ARG;
  if (act != TARDIS_ACT_GELU_TANH && act != TARDIS_ACT_GELU_ERF && act != TARDIS_ACT_RELU) return TARDIS_ERR_INVALID_ARG;
  return launch_range_search(d_ff, n_cal, z, ldz, b1, thresholds, threshold, step, act, lo, hi, a, c, steps_taken,
                             reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_neuron_thresholds(int32_t d_ff, int32_t n_cal, const float* z, int64_t ldz, const float* b1, const float* lo,
                                         const float* hi, int32_t act, double t_layer, double t_min, double t_max, float* err,
                                         float* thresholds, tardis_stream_t stream) {
  if (d_ff <= 0 || n_cal <= 0 || !z || ldz < n_cal || !lo || !hi || !err || !thresholds) return TARDIS_ERR_INVALID_ARG;
  if (!(t_min >= 0.0 && t_min <= t_layer && t_layer <= t_max && t_max <= 1.0)) return TARDIS_ERR_INVALID_ARG;
  if (act != TARDIS_ACT_GELU_TANH && act != TARDIS_ACT_GELU_ERF && act != TARDIS_ACT_RELU) return TARDIS_ERR_INVALID_ARG;
  return launch_neuron_thresholds(d_ff, n_cal, z, ldz, b1, lo, hi, act, t_layer, t_min, t_max, err, thresholds,
                                  reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_stats(tardis_handle_t handle, tardis_stats_t* out) {
  Handle* H = check(handle);
  if (!H || !out) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  TARDIS_CUDA_TRY(cudaStreamSynchronize(H->last_stream));
  unsigned long long ctr[CTR_COUNT];
  TARDIS_CUDA_TRY(cudaMemcpy(ctr, H->counters, sizeof(ctr), cudaMemcpyDeviceToHost));
  memset(out, 0, sizeof(*out));
  out->calls = H->calls; out->tokens = H->tokens; out->last_path = H->last_path;
  out->flagged_total = ctr[CTR_FLAGGED_TOTAL]; out->flagged_max = ctr[CTR_FLAGGED_MAX];
  out->device_error = ctr[CTR_ERROR]; out->exact_rechecks = ctr[CTR_RECHECKS]; out->last_union = ctr[CTR_LAST_UNION];
  out->bytes_folded = H->bytes_folded; out->bytes_predictor = H->bytes_predictor;
  out->bytes_tables = H->bytes_tables; out->bytes_w1 = H->bytes_w1; out->bytes_w2t = H->bytes_w2t;
  out->bytes_scratch = H->bytes_scratch;
  out->launches = H->launches;
  if (ctr[CTR_ERROR] == 1) return TARDIS_ERR_TIMEOUT;
  if (ctr[CTR_ERROR] != 0) return TARDIS_ERR_CORRUPT;
  const int bad = damaged_guards(H);
  if (bad < 0) { set_last_error(cudaGetLastError(), "guard check"); return TARDIS_ERR_CUDA; }
  if (bad > 0) { out->device_error = 2; return TARDIS_ERR_CORRUPT; }
  return TARDIS_OK;
}

tardis_status_t tardis_set_debug_capture(tardis_handle_t handle, uint32_t* flag_bitmap, double* scores) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  H->dbg_bitmap = flag_bitmap;
  H->dbg_scores = scores;
  return TARDIS_OK;
}

tardis_status_t tardis_export_folded(tardis_handle_t handle, void* Wf, float* bf, tardis_stream_t stream) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  H->last_stream = s;
  return launch_export_folded(H, Wf, bf, s);
}

tardis_status_t tardis_debug_phase_stamps(long long* stamps, int32_t max_ctas) {
  if (!stamps || max_ctas <= 0) return TARDIS_ERR_INVALID_ARG;
  // both fused kernels keep a table; the one whose kernel ran last holds the later entry stamps
  tardis_status_t st = fused_read_stamps(stamps, max_ctas);
  if (st != TARDIS_OK) return st;
  const size_t count = size_t(max_ctas < 512 ? max_ctas : 512) * 16;
  long long* other = new (std::nothrow) long long[count];
  if (!other) return TARDIS_ERR_ALLOC;
  st = decode_read_stamps(other, max_ctas);
  if (st == TARDIS_OK) {
    long long ma = 0, mb = 0;
    for (size_t i = 0; i < count; i += 16) { if (stamps[i] > ma) ma = stamps[i]; if (other[i] > mb) mb = other[i]; }
    if (mb > ma) memcpy(stamps, other, count * sizeof(long long));
  }
  delete[] other;
  return st;
}

tardis_status_t tardis_debug_wait_timeout(tardis_handle_t handle, int64_t limit_cycles, tardis_stream_t stream) {
  Handle* H = check(handle);
  if (!H || limit_cycles < 0 || limit_cycles > 2000000000ll) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  H->last_stream = s;
  return launch_wait_that_runs_out(H, limit_cycles, s);
}

tardis_status_t tardis_clear_error(tardis_handle_t handle) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  TARDIS_CUDA_TRY(cudaStreamSynchronize(H->last_stream));
  TARDIS_CUDA_TRY(cudaMemset(H->counters + CTR_ERROR, 0, sizeof(unsigned long long)));
  return TARDIS_OK;
}

// ---- a handle's state in a file (Section 6: the offline part writes the folded matrix and the predictor to a binary file)
// Layout: 64-byte header {8-byte magic, d, h, dtype, act, G, bits as int32, rest zero}, then the arrays in the order of
// `parts` below as raw bytes, then a 64-bit FNV-1a checksum of all array bytes.
static const char kFileMagic[8] = {'T', 'A', 'R', 'D', 'I', 'S', '0', '1'};

struct FilePart { void* dev; size_t bytes; };
static int file_parts(Handle* H, FilePart* parts) {
  const size_t hd = size_t(H->h) * H->d, h = H->h, d = H->d;
  int n = 0;
  parts[n++] = {H->W1, hd * H->esize};
  parts[n++] = {H->W2T, hd * H->esize};
  parts[n++] = {H->C, d * d * H->esize};
  parts[n++] = {H->bf, d * 4};
  parts[n++] = {H->lo, h * 4}; parts[n++] = {H->hi, h * 4}; parts[n++] = {H->a, h * 4}; parts[n++] = {H->c, h * 4};
  parts[n++] = {H->b1, h * 4};
  parts[n++] = {H->codes, hd / 8 * H->bits};
  parts[n++] = {H->scale, h * size_t(H->ngroups) * H->esize};
  parts[n++] = {H->zero, h * size_t(H->ngroups)};
  return n;
}
static uint64_t fnv1a(uint64_t hsh, const unsigned char* p, size_t n) {
  for (size_t i = 0; i < n; ++i) { hsh ^= p[i]; hsh *= 1099511628211ull; }
  return hsh;
}

tardis_status_t tardis_save(tardis_handle_t handle, const char* path) {
  Handle* H = check(handle);
  if (!H || !path) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  TARDIS_CUDA_TRY(cudaStreamSynchronize(H->last_stream));
  FILE* f = fopen(path, "wb");
  if (!f) { snprintf(g_last_error, sizeof(g_last_error), "tardis_save: cannot open %s", path); return TARDIS_ERR_INVALID_ARG; }
  unsigned char header[64] = {};
  memcpy(header, kFileMagic, 8);
  const int32_t dims[6] = {H->d, H->h, H->dtype, H->act, H->G, H->bits};
  memcpy(header + 8, dims, sizeof(dims));
  bool ok = fwrite(header, 1, 64, f) == 64;
  const size_t chunk = size_t(8) << 20;
  unsigned char* buf = static_cast<unsigned char*>(malloc(chunk));
  if (!buf) { fclose(f); return TARDIS_ERR_ALLOC; }
  FilePart parts[16];
  const int np = file_parts(H, parts);
  uint64_t sum = 14695981039346656037ull;
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < np && ok && e == cudaSuccess; ++i)
    for (size_t o = 0; o < parts[i].bytes && ok && e == cudaSuccess; o += chunk) {
      const size_t nb = parts[i].bytes - o < chunk ? parts[i].bytes - o : chunk;
      e = cudaMemcpy(buf, static_cast<const unsigned char*>(parts[i].dev) + o, nb, cudaMemcpyDeviceToHost);
      if (e == cudaSuccess) { sum = fnv1a(sum, buf, nb); ok = fwrite(buf, 1, nb, f) == nb; }
    }
  if (ok && e == cudaSuccess) ok = fwrite(&sum, 1, 8, f) == 8;
  free(buf);
  ok = (fclose(f) == 0) && ok;
  if (e != cudaSuccess) { set_last_error(e, "tardis_save"); return TARDIS_ERR_CUDA; }
  if (!ok) { snprintf(g_last_error, sizeof(g_last_error), "tardis_save: write to %s failed", path); return TARDIS_ERR_INVALID_ARG; }
  return TARDIS_OK;
}

tardis_status_t tardis_load(const char* path, tardis_stream_t stream, tardis_handle_t* out) {
  if (!path || !out) return TARDIS_ERR_INVALID_ARG;
  *out = nullptr;
  FILE* f = fopen(path, "rb");
  if (!f) { snprintf(g_last_error, sizeof(g_last_error), "tardis_load: cannot open %s", path); return TARDIS_ERR_INVALID_ARG; }
  unsigned char header[64];
  int32_t dims[6];
  if (fread(header, 1, 64, f) != 64 || memcmp(header, kFileMagic, 8) != 0) { fclose(f); return TARDIS_ERR_CORRUPT; }
  memcpy(dims, header + 8, sizeof(dims));
  const int d = dims[0], h = dims[1], dtype = dims[2], act = dims[3], G = dims[4], bits = dims[5];
  const bool sane = d > 0 && h > 0 && G > 0 && d <= (1 << 20) && h <= (1 << 24) && (dtype == TARDIS_F32 || dtype == TARDIS_BF16) &&
                    act >= 0 && act <= TARDIS_ACT_RELU && !(d % 8) && !(h % 32) && !(G % 16) && !(d % G) &&
                    (bits == 2 || bits == 4 || bits == 8 || (bits == 3 && d % 32 == 0));
  if (!sane) { fclose(f); return TARDIS_ERR_CORRUPT; }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  Handle* H = nullptr;
  OwnerScope scope(nullptr);                           // new_handle names the owner of the allocations that follow
  tardis_status_t st = new_handle(d, h, dtype, act, G, bits, s, &H);
  if (st != TARDIS_OK) { fclose(f); return st; }
  const size_t chunk = size_t(8) << 20;
  unsigned char* buf = static_cast<unsigned char*>(malloc(chunk));
  if (!buf) { fclose(f); free_all(H); return TARDIS_ERR_ALLOC; }
  FilePart parts[16];
  const int np = file_parts(H, parts);
  uint64_t sum = 14695981039346656037ull, stored = 0;
  bool ok = true;
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < np && ok && e == cudaSuccess; ++i)
    for (size_t o = 0; o < parts[i].bytes && ok && e == cudaSuccess; o += chunk) {
      const size_t nb = parts[i].bytes - o < chunk ? parts[i].bytes - o : chunk;
      ok = fread(buf, 1, nb, f) == nb;
      if (ok) { sum = fnv1a(sum, buf, nb); e = cudaMemcpy(static_cast<unsigned char*>(parts[i].dev) + o, buf, nb, cudaMemcpyHostToDevice); }
    }
  if (ok) ok = fread(&stored, 1, 8, f) == 8 && stored == sum;
  free(buf);
  fclose(f);
  if (e != cudaSuccess) { set_last_error(e, "tardis_load"); free_all(H); return TARDIS_ERR_CUDA; }
  if (!ok) { free_all(H); return TARDIS_ERR_CORRUPT; }          // truncated file or checksum mismatch
  e = cudaMemsetAsync(H->counters, 0, CTR_COUNT * sizeof(unsigned long long), s);
  if (e != cudaSuccess) { set_last_error(e, "tardis_load"); free_all(H); return TARDIS_ERR_CUDA; }
  // the kernel-specific copies are derived from the stored arrays exactly as tardis_fold derives them
  const bool bf16 = H->dtype == TARDIS_BF16;
  if (bf16) st = batched_prepare(H);
  if (st == TARDIS_OK && bf16) st = fused_prepare(H, s);
  if (st == TARDIS_OK && bf16 && !H->fscratch) st = decode_prepare(H, s);
  if (st == TARDIS_OK && bf16) st = batched_finish(H, nullptr, s);
  if (st != TARDIS_OK) { cudaStreamSynchronize(s); free_all(H); return st; }
  *out = reinterpret_cast<tardis_handle_t>(H);
  return TARDIS_OK;
}

tardis_status_t tardis_debug_damage_guard(tardis_handle_t handle, int32_t front, int32_t repair) {
  Handle* H = check(handle);
  if (!H || !on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  TARDIS_CUDA_TRY(cudaStreamSynchronize(H->last_stream));
  Allocation al{};
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    auto it = g_allocs.find(H->yacc);
    if (it == g_allocs.end()) return TARDIS_ERR_INVALID_ARG;
    al = it->second;
  }
  char* at = front ? al.base + kGuard - 4 : al.base + kGuard + al.bytes;   // the four guard bytes next to the buffer
  TARDIS_CUDA_TRY(cudaMemset(at, repair ? kGuardByte : 0, 4));
  return TARDIS_OK;
}

tardis_status_t tardis_debug_live_allocations(int64_t* count, int64_t* bytes) {
  if (!count || !bytes) return TARDIS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_alloc_mutex);
  *count = int64_t(g_allocs.size());
  *bytes = 0;
  for (const auto& kv : g_allocs) *bytes += int64_t(kv.second.bytes);
  return TARDIS_OK;
}

tardis_status_t tardis_debug_fail_alloc(int32_t nth) {
  g_fail_alloc.store(nth < 0 ? -1 : nth);
  return TARDIS_OK;
}

tardis_status_t tardis_build_predictor(int32_t d_ff, int32_t d_model, tardis_dtype_t dtype, const void* W1, const double* U,
                                       int32_t bits, int32_t group, uint32_t* codes, void* scale, uint8_t* zero, tardis_stream_t stream) {
  if (d_ff < 1 || d_model < 1 || !W1 || !codes || !scale || !zero) return TARDIS_ERR_INVALID_ARG;
  if (!(dtype == TARDIS_F32 || dtype == TARDIS_BF16) || !(bits == 2 || bits == 3 || bits == 4 || bits == 8)) return TARDIS_ERR_INVALID_ARG;
  if (group < 64 || group % 64 || d_model % group) return TARDIS_ERR_INVALID_ARG;
  return launch_build_predictor(d_ff, d_model, dtype, W1, U, bits, group, codes, scale, zero, reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_stack_forward(const tardis_stack_desc_t* desc, const void* x, void* y, void* work, size_t work_bytes,
                                     void* keep, size_t keep_bytes, int64_t n_tokens, tardis_stream_t stream) {
  if (!desc || desc->n_layers < 1 || !desc->layers || n_tokens < 0) return TARDIS_ERR_INVALID_ARG;
  if (!(desc->residual == 0 || desc->residual == 1) || !(desc->normalise == 0 || desc->normalise == 1)) return TARDIS_ERR_INVALID_ARG;
  if (desc->normalise && !(desc->ln_eps >= 0.f)) return TARDIS_ERR_INVALID_ARG;
  Handle* H0 = check(desc->layers[0]);
  if (!H0 || !on_handle_device(H0)) return TARDIS_ERR_INVALID_ARG;
  for (int l = 0; l < desc->n_layers; ++l) {
    Handle* H = check(desc->layers[l]);
    if (!H || H->d != H0->d || H->dtype != H0->dtype || H->device != H0->device) return TARDIS_ERR_INVALID_ARG;
    if (desc->normalise && ((desc->ln_gamma && !desc->ln_gamma[l]) || (desc->ln_beta && !desc->ln_beta[l]))) return TARDIS_ERR_INVALID_ARG;
  }
  if (n_tokens == 0) return TARDIS_OK;
  if (!x || !y || !aligned16(x) || !aligned16(y)) return TARDIS_ERR_INVALID_ARG;
  const size_t count = size_t(n_tokens) * H0->d * H0->esize;
  if (keep) {
    if (!aligned16(keep) || keep_bytes < size_t(2) * desc->n_layers * count) return TARDIS_ERR_INVALID_ARG;
  } else if (!work || !aligned16(work) || work_bytes < 2 * count) {
    return TARDIS_ERR_INVALID_ARG;
  }
  return launch_stack_forward(desc, x, y, work, keep, n_tokens, reinterpret_cast<cudaStream_t>(stream));
}

tardis_status_t tardis_set_deterministic(tardis_handle_t handle, int32_t on) {
  Handle* H = check(handle);
  if (!H || !(on == 0 || on == 1)) return TARDIS_ERR_INVALID_ARG;
  if (!on_handle_device(H)) return TARDIS_ERR_INVALID_ARG;
  if (on && !H->fscratch && !(H->bstate != nullptr && H->bits <= 4)) return TARDIS_ERR_UNSUPPORTED;
  if (on) {
    OwnerScope scope(H);
    const tardis_status_t st = fused_set_deterministic(H, true);
    if (st != TARDIS_OK) return st;
  }
  H->deterministic = on != 0;
  return TARDIS_OK;
}

tardis_status_t tardis_set_path(tardis_handle_t handle, int32_t path) {
  Handle* H = check(handle);
  if (!H || !(path >= 0 && path <= 4)) return TARDIS_ERR_INVALID_ARG;
  H->path_override = path;
  return TARDIS_OK;
}

tardis_status_t tardis_destroy(tardis_handle_t handle) {
  Handle* H = check(handle);
  if (!H) return TARDIS_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  free_all(H);
  if (e != cudaSuccess) { set_last_error(e, "cudaDeviceSynchronize"); return TARDIS_ERR_CUDA; }
  return TARDIS_OK;
}

const char* tardis_status_string(tardis_status_t status) {
  switch (status) {
    case TARDIS_OK: return "ok";
    case TARDIS_ERR_INVALID_ARG: return "invalid argument";
    case TARDIS_ERR_UNSUPPORTED: return "unsupported configuration";
    case TARDIS_ERR_ALLOC: return "device allocation failed";
    case TARDIS_ERR_CUDA: return "CUDA error";
    case TARDIS_ERR_TIMEOUT: return "device-side wait timed out";
    case TARDIS_ERR_CORRUPT: return "handle corrupt";
  }
  return "unknown status";
}

const char* tardis_last_error(void) { return g_last_error; }

}  // extern "C"
