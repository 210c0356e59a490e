// Fused decode kernel (placeholder until the fused path lands: the generic kernels run).
#include "common.cuh"

namespace tardis {
tardis_status_t decode_prepare(Handle* H, cudaStream_t s) { (void)H; (void)s; return TARDIS_OK; }
tardis_status_t launch_decode_forward(Handle* H, const void* x, void* y, int n, cudaStream_t s) {
  return launch_generic_forward(H, x, y, n, s);
}
void decode_release(Handle* H) { (void)H; }
}  // namespace tardis
