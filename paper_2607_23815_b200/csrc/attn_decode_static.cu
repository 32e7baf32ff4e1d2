// attn_decode_static: decode attention for callers that are not allowed to allocate device memory.
//
// The regular attn_decode needs a caller-provided workspace for its split-KV partial results.  Code that
// runs where cudaMalloc is off limits (inside a framework's captured or memory-planned region, in a plugin
// that was handed fixed buffers, in a process whose allocator is frozen after start-up) cannot produce one.
// This variant keeps that scratch in a fixed array that is part of the library image instead.
#include <mutex>

#include "common.cuh"

namespace kvattn {
size_t decode_workspace_bytes(int n_q_heads, int head_dim, int batch, int max_ctx_len);
kv_status_t launch_decode(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                          const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                          void* workspace, size_t workspace_bytes, cudaStream_t st, bool beside = false);

constexpr size_t kStaticScratchBytes = size_t(8) << 20;  // 8 MiB, held by every GPU that loads the library

// The split-KV partials of the last call stay in here; nothing in it has to start at zero, because the
// combine step reads only the slots that the same call wrote before.
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

static std::mutex g_scratch_mu;
static void* g_scratch_ptr[kMaxDevices] = {};  // device address of g_decode_scratch, per device

// In host code the array's name is only a handle; the device address has to be asked for, once per device,
// while that device is current.
static kv_status_t scratch_for_current_device(void** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KV_ERR_CUDA;
  std::lock_guard<std::mutex> g(g_scratch_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return KV_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
  return KV_OK;
}
}  // namespace kvattn

using namespace kvattn;

extern "C" kv_status_t attn_decode_static(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables,
                                          int max_pages, const int* ctx_lens, int batch, int max_ctx_len,
                                          float scale, void* out, float* lse, void* stream) {
  if (p == nullptr || batch < 0 || max_pages < 0 || max_ctx_len < 0) return KV_ERR_INVALID;
  if (n_q_heads <= 0 || n_q_heads % p->n_kv_heads != 0) return KV_ERR_UNSUPPORTED;
  const int g = n_q_heads / p->n_kv_heads;
  if (!(g == 1 || g == 2 || g == 4 || g == 8)) return KV_ERR_UNSUPPORTED;
  if (batch == 0) return KV_OK;
  if (q == nullptr || block_tables == nullptr || ctx_lens == nullptr || out == nullptr || lse == nullptr)
    return KV_ERR_INVALID;
  if ((((uintptr_t)q) | ((uintptr_t)out)) & 15) return KV_ERR_INVALID;
  if (max_ctx_len > (int64_t)max_pages * kPageSize) return KV_ERR_INVALID;
  // the array's address is taken for the current device: that has to be the device that holds the pool's pages
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  if (max_ctx_len == 0) max_ctx_len = 1;
  // the batch must fit the fixed scratch: refuse, do not truncate
  const size_t need = decode_workspace_bytes(n_q_heads, p->head_dim, batch, max_ctx_len);
  if (need > kStaticScratchBytes) return KV_ERR_WORKSPACE;
  void* scratch = nullptr;
  const kv_status_t st = scratch_for_current_device(&scratch);
  if (st != KV_OK) return st;
  return launch_decode(p, q, n_q_heads, block_tables, max_pages, ctx_lens, batch, max_ctx_len, scale, out, lse,
                       scratch, kStaticScratchBytes, (cudaStream_t)stream);
}

extern "C" size_t attn_decode_static_scratch_bytes(void) { return kStaticScratchBytes; }
