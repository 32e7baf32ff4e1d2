// Page pool, allocator and the data-movement kernels (append, gather, bounds check, poison).
#include <algorithm>
#include <new>

#include "common.cuh"
#include "append.cuh"

namespace kvattn {

std::atomic<int64_t> g_launches{0};

// ------------------------------------------------------------------------------------------
// kv_append: one warp moves one token.  Its lanes read consecutive 16-byte chunks of the token's K and V
// rows (coalesced loads, all in flight before the first store); the eight chunks of a 64-dim half land,
// permuted, in one 128-byte row of the page (full-line 16-byte stores).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) append_kernel(PoolView pool, AppendArgs a) {
  append_tokens<8>(pool, a, (blockIdx.x * blockDim.x + threadIdx.x) >> 5, (gridDim.x * blockDim.x) >> 5);
}

__global__ void __launch_bounds__(256) gather_kernel(PoolView pool, const int* __restrict__ block_row, int len,
                                                     uint4* __restrict__ k_out, uint4* __restrict__ v_out) {
  const int chunks_per_row = pool.head_dim >> 3;
  const int chunks_per_token = pool.n_kv_heads * chunks_per_row;
  const int64_t total = (int64_t)len * chunks_per_token;
  const size_t blk = block_bytes(pool.head_dim);
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int token = (int)(idx / chunks_per_token);
    const int rem = (int)(idx - (int64_t)token * chunks_per_token);
    const int head = rem / chunks_per_row;
    const int dchunk = rem - head * chunks_per_row;
    const int page = __ldg(block_row + (token >> 4));
    if (page < 0 || page >= pool.num_pages) { report(pool.status, KV_ERR_BOUNDS); continue; }
    const size_t off = ((size_t)page * pool.n_kv_heads + head) * blk + chunk_offset_bytes(token & 15, dchunk, pool.head_dim);
    k_out[idx] = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(pool.k) + off);
    v_out[idx] = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(pool.v) + off);
  }
}

__global__ void check_batch_kernel(PoolView pool, const int* __restrict__ block_tables, int max_pages,
                                   const int* __restrict__ lens, int batch) {
  for (int i = blockIdx.x; i < batch; i += gridDim.x) {
    const int len = lens[i];
    if (len < 0 || len > max_pages * kPageSize) {
      if (threadIdx.x == 0) report(pool.status, KV_ERR_BOUNDS);
      continue;
    }
    const int nblk = (len + kPageSize - 1) / kPageSize;
    for (int b = threadIdx.x; b < nblk; b += blockDim.x) {
      const int page = block_tables[(int64_t)i * max_pages + b];
      if (page < 0 || page >= pool.num_pages) report(pool.status, KV_ERR_BOUNDS);
    }
  }
}

__global__ void poison_kernel(PoolView pool, const int* __restrict__ page_ids, int n) {
  const size_t per_page16 = (block_bytes(pool.head_dim) * pool.n_kv_heads) >> 4;
  const uint4 nan4 = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
  for (int i = blockIdx.x; i < n; i += gridDim.x) {
    const int page = page_ids[i];
    if (page < 0 || page >= pool.num_pages) continue;
    uint4* kp = reinterpret_cast<uint4*>(pool.k) + (size_t)page * per_page16;
    uint4* vp = reinterpret_cast<uint4*>(pool.v) + (size_t)page * per_page16;
    for (size_t j = threadIdx.x; j < per_page16; j += blockDim.x) { kp[j] = nan4; vp[j] = nan4; }
  }
}

static bool shape_supported(int page_size, int n_kv_heads, int head_dim) {
  return page_size == kPageSize && (head_dim == 64 || head_dim == 128) && n_kv_heads >= 1;
}

int sm_count_of(int device) {
  static std::atomic<int> cached[kMaxDevices];
  if (device < 0 || device >= kMaxDevices) return 1;
  int n = cached[device].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      return 1;
    }
    cached[device].store(n, std::memory_order_relaxed);
  }
  return n;
}

static int grid_for(const kv_pool_t* p, int64_t work_items, int threads) {
  int64_t blocks = (work_items + threads - 1) / threads;
  const int64_t cap = (int64_t)sm_count_of(p->device) * 16;  // a few waves of resident blocks; grid-stride covers the rest
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace kvattn

using namespace kvattn;

extern "C" {

const char* kv_status_str(kv_status_t s) {
  switch (s) {
    case KV_OK: return "ok";
    case KV_ERR_INVALID: return "invalid argument";
    case KV_ERR_OOM: return "out of pages";
    case KV_ERR_NOT_ALLOCATED: return "page not allocated";
    case KV_ERR_BOUNDS: return "block table entry or length out of bounds";
    case KV_ERR_UNSUPPORTED: return "unsupported shape";
    case KV_ERR_CUDA: return "CUDA runtime error";
    case KV_ERR_TIMEOUT: return "device-side wait timed out";
    case KV_ERR_WORKSPACE: return "workspace missing or too small";
    case KV_ERR_PINNED: return "page is pinned";
  }
  return "unknown status";
}

static kv_status_t pool_create_impl(int num_pages, int page_size, int n_kv_heads, int head_dim, void* k_base,
                                    void* v_base, bool owns, kv_pool_t** out) {
  if (out == nullptr) return KV_ERR_INVALID;
  *out = nullptr;
  if (num_pages <= 0 || n_kv_heads <= 0) return KV_ERR_INVALID;
  if (!shape_supported(page_size, n_kv_heads, head_dim)) return KV_ERR_UNSUPPORTED;
  kv_pool* p = new (std::nothrow) kv_pool();
  if (p == nullptr) return KV_ERR_OOM;
  p->num_pages = num_pages; p->page_size = page_size; p->n_kv_heads = n_kv_heads; p->head_dim = head_dim;
  p->owns_buffers = owns; p->k_base = k_base; p->v_base = v_base;
  p->bytes_each = (int64_t)num_pages * n_kv_heads * (int64_t)block_bytes(head_dim);
  p->d_status = nullptr; p->d_scratch_ids = nullptr; p->poison = false;
  p->h2d_stream = nullptr; p->d2h_stream = nullptr; p->host_slot_next = 0;
  for (auto& hs : p->host_slots) hs = kv_pool::HostSlot{nullptr, nullptr, nullptr, nullptr};
  p->mark_epoch = 0; p->evicted_total = 0;
  bool ok = cudaGetDevice(&p->device) == cudaSuccess;
  if (ok && owns) {
    ok = cudaMalloc(&p->k_base, (size_t)p->bytes_each) == cudaSuccess &&
         cudaMalloc(&p->v_base, (size_t)p->bytes_each) == cudaSuccess;
  }
  ok = ok && cudaMalloc(&p->d_status, sizeof(int)) == cudaSuccess &&
       cudaMemset(p->d_status, 0, sizeof(int)) == cudaSuccess &&
       cudaMalloc(&p->d_scratch_ids, sizeof(int) * (size_t)num_pages) == cudaSuccess &&
       cudaStreamCreateWithFlags(&p->h2d_stream, cudaStreamNonBlocking) == cudaSuccess &&
       cudaStreamCreateWithFlags(&p->d2h_stream, cudaStreamNonBlocking) == cudaSuccess;
  for (auto& hs : p->host_slots)
    ok = ok && cudaEventCreateWithFlags(&hs.in, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&hs.ran, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&hs.out, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    kv_pool_destroy(p);
    cudaGetLastError();
    return KV_ERR_CUDA;
  }
  p->free_stack.resize(num_pages);
  for (int i = 0; i < num_pages; ++i) p->free_stack[i] = num_pages - 1 - i;  // back() == 0 first
  p->allocated.assign(num_pages, 0);
  p->refs.assign(num_pages, 0);
  p->pins.assign(num_pages, 0);
  p->last_use.assign(num_pages, 0);
  p->clock = 0;
  p->mark.assign(num_pages, 0);
  *out = p;
  return KV_OK;
}

kv_status_t kv_pool_create(int num_pages, int page_size, int n_kv_heads, int head_dim, kv_pool_t** out) {
  return pool_create_impl(num_pages, page_size, n_kv_heads, head_dim, nullptr, nullptr, true, out);
}

kv_status_t kv_pool_create_ex(int num_pages, int page_size, int n_kv_heads, int head_dim, void* k_base,
                              void* v_base, kv_pool_t** out) {
  if (k_base == nullptr || v_base == nullptr) return KV_ERR_INVALID;
  if (((uintptr_t)k_base & 255) != 0 || ((uintptr_t)v_base & 255) != 0) return KV_ERR_INVALID;
  return pool_create_impl(num_pages, page_size, n_kv_heads, head_dim, k_base, v_base, false, out);
}

kv_status_t kv_pool_destroy(kv_pool_t* p) {
  if (p == nullptr) return KV_ERR_INVALID;
  if (p->owns_buffers) {
    if (p->k_base) cudaFree(p->k_base);
    if (p->v_base) cudaFree(p->v_base);
  }
  if (p->d_status) cudaFree(p->d_status);
  if (p->d_scratch_ids) cudaFree(p->d_scratch_ids);
  if (p->h2d_stream) cudaStreamDestroy(p->h2d_stream);
  if (p->d2h_stream) cudaStreamDestroy(p->d2h_stream);
  for (auto& hs : p->host_slots) {
    if (hs.in) cudaEventDestroy(hs.in);
    if (hs.ran) cudaEventDestroy(hs.ran);
    if (hs.out) cudaEventDestroy(hs.out);
  }
  delete p;
  return KV_OK;
}

kv_status_t kv_pool_stats(const kv_pool_t* p, int* free_pages, int* used_pages, int64_t* evicted_total) {
  if (p == nullptr) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(const_cast<kv_pool_t*>(p)->mu);
  if (free_pages) *free_pages = (int)p->free_stack.size();
  if (used_pages) *used_pages = p->num_pages - (int)p->free_stack.size();
  if (evicted_total) *evicted_total = p->evicted_total;
  return KV_OK;
}

kv_status_t kv_pool_raw(const kv_pool_t* p, void** k_base, void** v_base, int64_t* bytes_each) {
  if (p == nullptr) return KV_ERR_INVALID;
  if (k_base) *k_base = p->k_base;
  if (v_base) *v_base = p->v_base;
  if (bytes_each) *bytes_each = p->bytes_each;
  return KV_OK;
}

int64_t kv_pool_elem_offset(const kv_pool_t* p, int page, int kv_head, int slot, int d) {
  if (p == nullptr || page < 0 || page >= p->num_pages || kv_head < 0 || kv_head >= p->n_kv_heads || slot < 0 ||
      slot >= p->page_size || d < 0 || d >= p->head_dim)
    return -1;
  const int64_t blk_elems = (int64_t)p->page_size * p->head_dim;
  return ((int64_t)page * p->n_kv_heads + kv_head) * blk_elems +
         (int64_t)(chunk_offset_bytes(slot, d >> 3, p->head_dim) >> 1) + (d & 7);
}

kv_status_t kv_pool_set_poison(kv_pool_t* p, int on) {
  if (p == nullptr) return KV_ERR_INVALID;
  p->poison = on != 0;
  return KV_OK;
}

kv_status_t kv_alloc(kv_pool_t* p, int n, int* out_page_ids) {
  if (p == nullptr || n < 0 || (n > 0 && out_page_ids == nullptr)) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  if ((size_t)n > p->free_stack.size()) return KV_ERR_OOM;
  for (int i = 0; i < n; ++i) {
    const int id = p->free_stack.back();
    p->free_stack.pop_back();
    p->allocated[id] = 1;
    p->refs[id] = 1;
    p->pins[id] = 0;
    p->last_use[id] = ++p->clock;
    out_page_ids[i] = id;
  }
  return KV_OK;
}

// Marks the ids of one call; returns false on an id that is out of range, not allocated or (if `unique`) repeated.
static bool check_ids(kv_pool_t* p, const int* ids, int n, bool unique) {
  if (++p->mark_epoch == 0) {  // epoch wrapped: clear the marks
    std::fill(p->mark.begin(), p->mark.end(), 0u);
    p->mark_epoch = 1;
  }
  for (int i = 0; i < n; ++i) {
    const int id = ids[i];
    if (id < 0 || id >= p->num_pages || !p->allocated[id]) return false;
    if (unique && p->mark[id] == p->mark_epoch) return false;
    p->mark[id] = p->mark_epoch;
  }
  return true;
}

static kv_status_t poison_pages(kv_pool_t* p, const int* ids, int n) {
  if (!p->poison || n <= 0) return KV_OK;
  KV_CUDA_OK(cudaMemcpy(p->d_scratch_ids, ids, sizeof(int) * (size_t)n, cudaMemcpyHostToDevice));
  poison_kernel<<<n < 1184 ? n : 1184, 256>>>(p->view(), p->d_scratch_ids, n);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  KV_CUDA_OK(cudaDeviceSynchronize());
  return KV_OK;
}

static kv_status_t release_pages(kv_pool_t* p, const int* ids, int n, bool evict) {
  if (p == nullptr || n < 0 || (n > 0 && ids == nullptr)) return KV_ERR_INVALID;
  {
    std::lock_guard<std::mutex> g(p->mu);
    if (!check_ids(p, ids, n, true)) return KV_ERR_NOT_ALLOCATED;  // nothing has been changed yet
    for (int i = 0; i < n; ++i) {
      // a pinned page is never evicted, and its last owner cannot drop it either
      if (p->pins[ids[i]] > 0 && (evict || p->refs[ids[i]] == 1)) return KV_ERR_PINNED;
    }
    for (int i = 0; i < n; ++i) {
      const int id = ids[i];
      if (!evict && --p->refs[id] > 0) continue;  // other owners remain
      p->allocated[id] = 0;
      p->refs[id] = 0;
      p->free_stack.push_back(id);
    }
    if (evict) p->evicted_total += n;
  }
  return evict ? poison_pages(p, ids, n) : KV_OK;
}

kv_status_t kv_free(kv_pool_t* p, const int* page_ids, int n) { return release_pages(p, page_ids, n, false); }
kv_status_t kv_evict(kv_pool_t* p, const int* page_ids, int n) { return release_pages(p, page_ids, n, true); }

kv_status_t kv_ref(kv_pool_t* p, const int* page_ids, int n) {
  if (p == nullptr || n < 0 || (n > 0 && page_ids == nullptr)) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  if (!check_ids(p, page_ids, n, false)) return KV_ERR_NOT_ALLOCATED;
  for (int i = 0; i < n; ++i)
    if (p->refs[page_ids[i]] >= 0xFFFF) return KV_ERR_INVALID;
  for (int i = 0; i < n; ++i) ++p->refs[page_ids[i]];
  return KV_OK;
}

kv_status_t kv_pin(kv_pool_t* p, const int* page_ids, int n) {
  if (p == nullptr || n < 0 || (n > 0 && page_ids == nullptr)) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  if (!check_ids(p, page_ids, n, false)) return KV_ERR_NOT_ALLOCATED;
  for (int i = 0; i < n; ++i)
    if (p->pins[page_ids[i]] >= 0xFFFF) return KV_ERR_INVALID;
  for (int i = 0; i < n; ++i) ++p->pins[page_ids[i]];
  return KV_OK;
}

kv_status_t kv_unpin(kv_pool_t* p, const int* page_ids, int n) {
  if (p == nullptr || n < 0 || (n > 0 && page_ids == nullptr)) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  if (!check_ids(p, page_ids, n, true)) return KV_ERR_NOT_ALLOCATED;
  for (int i = 0; i < n; ++i)
    if (p->pins[page_ids[i]] == 0) return KV_ERR_INVALID;  // not pinned; nothing has been changed yet
  for (int i = 0; i < n; ++i) --p->pins[page_ids[i]];
  return KV_OK;
}

kv_status_t kv_unpin_all(kv_pool_t* p, int* n_unpinned) {
  if (p == nullptr) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  int cnt = 0;
  for (int id = 0; id < p->num_pages; ++id) {
    if (p->pins[id] > 0) ++cnt;
    p->pins[id] = 0;
  }
  if (n_unpinned) *n_unpinned = cnt;
  return KV_OK;
}

kv_status_t kv_touch(kv_pool_t* p, const int* page_ids, int n) {
  if (p == nullptr || n < 0 || (n > 0 && page_ids == nullptr)) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(p->mu);
  if (!check_ids(p, page_ids, n, false)) return KV_ERR_NOT_ALLOCATED;
  for (int i = 0; i < n; ++i) p->last_use[page_ids[i]] = ++p->clock;
  return KV_OK;
}

kv_status_t kv_evict_lru(kv_pool_t* p, int n, int* out_page_ids, int* n_evicted) {
  if (p == nullptr || n < 0 || n_evicted == nullptr || (n > 0 && out_page_ids == nullptr)) return KV_ERR_INVALID;
  int cnt = 0;
  {
    std::lock_guard<std::mutex> g(p->mu);
    std::vector<int> cand;
    for (int id = 0; id < p->num_pages; ++id)
      if (p->allocated[id] && p->pins[id] == 0) cand.push_back(id);
    cnt = n < (int)cand.size() ? n : (int)cand.size();
    // least recently used first; the clock is strictly increasing, so there are no ties
    std::partial_sort(cand.begin(), cand.begin() + cnt, cand.end(),
                      [&](int a, int b) { return p->last_use[a] < p->last_use[b]; });
    for (int i = 0; i < cnt; ++i) {
      const int id = cand[i];
      p->allocated[id] = 0;
      p->refs[id] = 0;
      p->free_stack.push_back(id);
      out_page_ids[i] = id;
    }
    p->evicted_total += cnt;
  }
  *n_evicted = cnt;
  return poison_pages(p, out_page_ids, cnt);
}

kv_status_t kv_page_info(const kv_pool_t* p, int page, int* allocated, int* refs, int* pins) {
  if (p == nullptr || page < 0 || page >= p->num_pages) return KV_ERR_INVALID;
  std::lock_guard<std::mutex> g(const_cast<kv_pool_t*>(p)->mu);
  if (allocated) *allocated = p->allocated[page];
  if (refs) *refs = p->refs[page];
  if (pins) *pins = p->pins[page];
  return KV_OK;
}

kv_status_t kv_append(kv_pool_t* p, const void* k_new, const void* v_new, const int* cu_new, const int* start_pos,
                      const int* seg_row, const int* block_tables, int max_pages, int n_segments, int total_new,
                      void* stream) {
  if (p == nullptr || n_segments < 0 || total_new < 0 || max_pages < 0) return KV_ERR_INVALID;
  if (n_segments == 0 || total_new == 0) return KV_OK;
  if (k_new == nullptr || v_new == nullptr || cu_new == nullptr || start_pos == nullptr || block_tables == nullptr)
    return KV_ERR_INVALID;
  if ((((uintptr_t)k_new) | ((uintptr_t)v_new)) & 15) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  const AppendArgs a{(const uint4*)k_new, (const uint4*)v_new, cu_new, start_pos, seg_row, block_tables, max_pages, n_segments,
                     total_new};
  append_kernel<<<grid_for(p, (int64_t)total_new * 32, 256), 256, 0, (cudaStream_t)stream>>>(p->view(), a);  // one warp per token
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}

kv_status_t kv_gather(kv_pool_t* p, const int* block_table_row, int len, void* k_out, void* v_out, void* stream) {
  if (p == nullptr || len < 0) return KV_ERR_INVALID;
  if (len == 0) return KV_OK;
  if (block_table_row == nullptr || k_out == nullptr || v_out == nullptr) return KV_ERR_INVALID;
  if ((((uintptr_t)k_out) | ((uintptr_t)v_out)) & 15) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  const int64_t chunks = (int64_t)len * p->n_kv_heads * (p->head_dim >> 3);
  gather_kernel<<<grid_for(p, chunks, 256), 256, 0, (cudaStream_t)stream>>>(p->view(), block_table_row, len,
                                                                         (uint4*)k_out, (uint4*)v_out);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}

kv_status_t kv_last_async_status(kv_pool_t* p) {
  if (p == nullptr || !on_pool_device(p)) return KV_ERR_INVALID;
  int code = 0;
  KV_CUDA_OK(cudaDeviceSynchronize());
  KV_CUDA_OK(cudaMemcpy(&code, p->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (code != 0) KV_CUDA_OK(cudaMemset(p->d_status, 0, sizeof(int)));
  return (kv_status_t)code;
}

kv_status_t kv_check_batch(kv_pool_t* p, const int* block_tables, int max_pages, const int* lens, int batch,
                           void* stream) {
  if (p == nullptr || batch < 0 || max_pages < 0) return KV_ERR_INVALID;
  if (batch == 0) return KV_OK;
  if (block_tables == nullptr || lens == nullptr) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  check_batch_kernel<<<batch < 1184 ? batch : 1184, 128, 0, (cudaStream_t)stream>>>(p->view(), block_tables,
                                                                                  max_pages, lens, batch);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  KV_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  return kv_last_async_status(p);
}

int64_t kvattn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
