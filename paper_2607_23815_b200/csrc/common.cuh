// Shared declarations of the library's translation units: the pool object, the page layout,
// launch accounting.  Not part of the public interface (that is include/kvattn.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "../../include/kvattn.h"

namespace kvattn {

constexpr int kPageSize = 16;

// Device-visible description of the pool, passed to kernels by value.
struct PoolView {
  __nv_bfloat16* k;
  __nv_bfloat16* v;
  int num_pages;
  int n_kv_heads;
  int head_dim;
  int* status;  // device status word: first error seen by a kernel (0 = none)
};

// Byte offset of the 16-byte chunk (slot, dchunk) inside a (page, head) block.  Blocks are made of
// 8-token x 64-dim tiles of 1024 bytes; the chunk index inside a 128-byte row is XORed with the row.
__host__ __device__ __forceinline__ uint32_t chunk_offset_bytes(int slot, int dchunk, int head_dim) {
  const int grp = slot >> 3, r = slot & 7, half = dchunk >> 3, c = dchunk & 7;
  return (uint32_t)(grp * (head_dim * 16) + half * 1024 + r * 128 + ((c ^ r) << 4));
}

__host__ __device__ __forceinline__ size_t block_bytes(int head_dim) { return (size_t)kPageSize * head_dim * 2; }

__device__ __forceinline__ void report(int* status, int code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// The children of the fan-out mode.
struct FanArgs {
  const int* cu_q;         // [n_children + 1]: first row of each child in Q
  const int* cu_children;  // [n_parents + 1]: children of parent g are cu_children[g] .. cu_children[g+1]-1
  const int* tables;       // [n_children][max_pages]: the children's own pages
  int max_pages;
  int n_children;
};

extern std::atomic<int64_t> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

constexpr int kMaxDevices = 64;
// Multiprocessors of the given device (asked once per device).
int sm_count_of(int device);

}  // namespace kvattn

struct kv_pool {
  int num_pages, page_size, n_kv_heads, head_dim;
  int device;
  bool owns_buffers;
  void* k_base;
  void* v_base;
  int64_t bytes_each;
  int* d_status;      // device status word
  int* d_scratch_ids; // device staging for page-id lists (poison fill), num_pages ints
  bool poison;
  // allocator
  std::mutex mu;
  std::vector<int> free_stack;       // back() is handed out next
  std::vector<uint8_t> allocated;    // per page
  std::vector<uint32_t> mark;        // duplicate detection in one release call
  std::vector<uint16_t> refs;        // owners of an allocated page (kv_alloc: 1, kv_ref: +1, kv_free: -1)
  std::vector<uint16_t> pins;        // pin count: a pinned page cannot be evicted
  std::vector<uint64_t> last_use;    // logical clock of the last kv_alloc / kv_touch, for kv_evict_lru
  uint64_t clock;
  uint32_t mark_epoch;
  int64_t evicted_total;
  // attn_extend_host: copies in and out run on streams of their own, so that they overlap the kernels of the
  // neighbouring steps; per staging area (up to kHostSlots in rotation) the events that order its reuse
  static constexpr int kHostSlots = 4;
  cudaStream_t h2d_stream, d2h_stream;
  struct HostSlot {
    void* staging;
    cudaEvent_t in, ran, out;  // inputs copied in; kernels finished; results copied out
  } host_slots[kHostSlots];
  int host_slot_next;

  kvattn::PoolView view() const {
    return kvattn::PoolView{(__nv_bfloat16*)k_base, (__nv_bfloat16*)v_base, num_pages, n_kv_heads, head_dim,
                            d_status};
  }
};

// A pool's kernels are launched on the calling thread's current device and must therefore find the pool's memory
// there: launchers return KV_ERR_INVALID when the current device is not the one the pool was created on.
inline bool on_pool_device(const kv_pool* p) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == p->device;
}

#define KV_CUDA_OK(expr)                      \
  do {                                        \
    cudaError_t _e = (expr);                  \
    if (_e != cudaSuccess) return KV_ERR_CUDA; \
  } while (0)
