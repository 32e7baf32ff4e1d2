// Tensor-core extend attention (tcgen05 / TMEM).  Placeholder translation unit until the kernel lands:
// reports "not supported" so that attn_extend selects the small-tile kernel.
#include "common.cuh"

namespace kvattn {

size_t extend_tc_workspace_bytes(int, int, int, int, int) { return 0; }
bool extend_tc_supported(const kv_pool_t*, int) { return false; }
kv_status_t launch_extend_tc(kv_pool_t*, const void*, int, const int*, const int*, int, const int*, const int*, int,
                             int, int, int, float, void*, float*, void*, size_t, cudaStream_t) {
  return KV_ERR_UNSUPPORTED;
}

}  // namespace kvattn
