// Public attention entry points: argument checks, kernel selection, the mixed-batch launcher.
#include "append.cuh"
#include "common.cuh"

namespace kvattn {
size_t decode_workspace_bytes(int n_q_heads, int head_dim, int batch, int max_ctx_len);
kv_status_t launch_decode(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                          const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                          void* workspace, size_t workspace_bytes, cudaStream_t st, bool beside = false);
kv_status_t launch_extend_small(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                                int max_pages, const int* prefix_lens, const int* extend_lens, int batch,
                                int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                                cudaStream_t st);
size_t extend_tc_workspace_bytes(int n_q_heads, int head_dim, int batch, int total_q, int max_total_len);
bool extend_tc_supported(const kv_pool_t* p, int n_q_heads);
kv_status_t launch_extend_tc(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                             int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                             int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, int cta_cap, int mode, const FanArgs* fan,
                             const AppendArgs* app, int phase, cudaStream_t st);

size_t extend_shared_workspace_bytes(const kv_pool_t* p, int n_q_heads, int n_parents, int n_children, int total_q,
                                     int max_parent_len);
kv_status_t launch_extend_shared(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* cu_children,
                                 const int* parent_tables, int max_pages_parent, const int* parent_lens,
                                 const int* child_tables, int max_pages_child, const int* child_lens, int n_parents,
                                 int n_children, int total_q, int max_child_len, int max_parent_rows, int max_parent_len,
                                 float scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                                 cudaStream_t st);

extern std::atomic<int> g_shared_impl;
extern std::atomic<int> g_decode_impl;

static std::atomic<int> g_extend_impl{0};
static std::atomic<int> g_mixed_extend_ctas{0};  // SMs the extend kernel may take inside attn_mixed (0 = all)

static bool heads_supported(const kv_pool_t* p, int n_q_heads) {
  if (n_q_heads <= 0 || n_q_heads % p->n_kv_heads != 0) return false;
  const int g = n_q_heads / p->n_kv_heads;
  return g == 1 || g == 2 || g == 4 || g == 8;
}

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
}  // namespace kvattn

using namespace kvattn;

extern "C" {

kv_status_t kvattn_set_extend_impl(int impl) {
  if (impl < 0 || impl > 2) return KV_ERR_INVALID;
  g_extend_impl.store(impl);
  return KV_OK;
}

size_t attn_workspace_bytes(const kv_pool_t* p, int n_q_heads, int batch_ext, int total_q, int max_total_len,
                            int batch_dec, int max_ctx_len) {
  if (p == nullptr || n_q_heads <= 0) return 0;
  // the two regions are disjoint so that a mixed step can run both kinds of work at once
  return align256(extend_tc_workspace_bytes(n_q_heads, p->head_dim, batch_ext, total_q, max_total_len)) +
         align256(decode_workspace_bytes(n_q_heads, p->head_dim, batch_dec, max_ctx_len)) + 256;
}

// k_new / v_new non-null: the suffix K/V rows (ragged by cu_q like Q) are first written to positions prefix_lens[i] ..
// of their sequences' pages, in the kernel that also builds the attention kernel's plan.
static kv_status_t extend_impl(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                               int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                               int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                               void* workspace, size_t workspace_bytes, int cta_cap, void* stream,
                               const void* k_new = nullptr, const void* v_new = nullptr, int phase = 0) {
  if (p == nullptr || batch < 0 || total_q < 0 || max_pages < 0 || max_extend_len < 0 || max_total_len < 0)
    return KV_ERR_INVALID;
  if (!heads_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  if (batch == 0 || total_q == 0 || max_extend_len == 0) return KV_OK;
  if (cu_q == nullptr || block_tables == nullptr || prefix_lens == nullptr || extend_lens == nullptr) return KV_ERR_INVALID;
  if (phase != 1 && (q == nullptr || out == nullptr || lse == nullptr)) return KV_ERR_INVALID;
  if ((((uintptr_t)q) | ((uintptr_t)out)) & 15) return KV_ERR_INVALID;
  if (max_total_len < max_extend_len || max_total_len > (int64_t)max_pages * kPageSize) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  const int impl = g_extend_impl.load();
  const bool tc_ok = extend_tc_supported(p, n_q_heads) && scale > 0.f;  // the tensor-core kernel folds a positive scale into the row maximum
  if (impl == 2 && !tc_ok) return KV_ERR_UNSUPPORTED;
  if (phase != 0 && !(impl == 2 || (impl == 0 && tc_ok))) {
    // the small-tile kernel has no plan: planning is a no-op and the planned call is the plain one
    if (phase == 1) return KV_OK;
    phase = 0;
  }
  if (impl == 2 || (impl == 0 && tc_ok)) {
    const AppendArgs app{(const uint4*)k_new, (const uint4*)v_new, cu_q, prefix_lens, nullptr, block_tables, max_pages, batch,
                         total_q};
    return launch_extend_tc(p, q, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch, total_q,
                            max_extend_len, max_total_len, scale, out, lse, workspace, workspace_bytes, cta_cap, 0,
                            nullptr, k_new != nullptr ? &app : nullptr, phase, (cudaStream_t)stream);
  }
  if (k_new != nullptr) {  // the small-tile kernel has no plan to share a launch with: append, then attend
    const kv_status_t as = kv_append(p, k_new, v_new, cu_q, prefix_lens, nullptr, block_tables, max_pages, batch, total_q, stream);
    if (as != KV_OK) return as;
  }
  return launch_extend_small(p, q, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch,
                             max_extend_len, max_total_len, scale, out, lse, (cudaStream_t)stream);
}

kv_status_t attn_extend(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                        int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                        int max_extend_len, int max_total_len, float scale, void* out, float* lse, void* workspace,
                        size_t workspace_bytes, void* stream) {
  return extend_impl(p, q, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch, total_q,
                     max_extend_len, max_total_len, scale, out, lse, workspace, workspace_bytes, 0, stream);
}

kv_status_t attn_extend_append(kv_pool_t* p, const void* q, const void* k_new, const void* v_new, int n_q_heads,
                               const int* cu_q, const int* block_tables, int max_pages, const int* prefix_lens,
                               const int* extend_lens, int batch, int total_q, int max_extend_len, int max_total_len,
                               float scale, void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
  if (p != nullptr && batch > 0 && total_q > 0) {
    if (k_new == nullptr || v_new == nullptr) return KV_ERR_INVALID;
    if ((((uintptr_t)k_new) | ((uintptr_t)v_new)) & 15) return KV_ERR_INVALID;
  }
  return extend_impl(p, q, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch, total_q,
                     max_extend_len, max_total_len, scale, out, lse, workspace, workspace_bytes, 0, stream, k_new, v_new);
}

kv_status_t attn_extend_plan(kv_pool_t* p, int n_q_heads, const int* cu_q, const int* block_tables, int max_pages,
                             const int* prefix_lens, const int* extend_lens, int batch, int total_q, int max_extend_len,
                             int max_total_len, void* workspace, size_t workspace_bytes, void* stream) {
  return extend_impl(p, nullptr, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch, total_q,
                     max_extend_len, max_total_len, 1.f, nullptr, nullptr, workspace, workspace_bytes, 0, stream, nullptr,
                     nullptr, 1);
}

kv_status_t attn_extend_planned(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                                int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                                int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                                void* workspace, size_t workspace_bytes, void* stream) {
  return extend_impl(p, q, n_q_heads, cu_q, block_tables, max_pages, prefix_lens, extend_lens, batch, total_q,
                     max_extend_len, max_total_len, scale, out, lse, workspace, workspace_bytes, 0, stream, nullptr, nullptr,
                     2);
}

size_t attn_extend_shared_workspace_bytes(const kv_pool_t* p, int n_q_heads, int n_parents, int n_children, int total_q,
                                          int max_parent_len) {
  if (p == nullptr || n_q_heads <= 0) return 0;
  return extend_shared_workspace_bytes(p, n_q_heads, n_parents, n_children, total_q, max_parent_len);
}

kv_status_t attn_extend_shared(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* cu_children,
                               const int* parent_tables, int max_pages_parent, const int* parent_lens,
                               const int* child_tables, int max_pages_child, const int* child_lens, int n_parents,
                               int n_children, int total_q, int max_child_len, int max_parent_rows, int max_parent_len,
                               float scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               void* stream) {
  if (p == nullptr || n_parents < 0 || n_children < 0 || total_q < 0 || max_pages_parent < 0 || max_pages_child < 0 ||
      max_child_len < 0 || max_parent_rows < 0 || max_parent_len < 0)
    return KV_ERR_INVALID;
  if (!heads_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  if (n_parents == 0 || n_children == 0 || total_q == 0 || max_child_len == 0) return KV_OK;
  if (q == nullptr || cu_q == nullptr || cu_children == nullptr || parent_tables == nullptr || parent_lens == nullptr ||
      child_tables == nullptr || child_lens == nullptr || out == nullptr || lse == nullptr)
    return KV_ERR_INVALID;
  if ((((uintptr_t)q) & 15) || (((uintptr_t)out) & 31)) return KV_ERR_INVALID;
  if (max_parent_len > (int64_t)max_pages_parent * kPageSize || max_child_len > (int64_t)max_pages_child * kPageSize ||
      max_parent_rows < max_child_len)
    return KV_ERR_INVALID;
  if (!(scale > 0.f) || !extend_tc_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  return launch_extend_shared(p, q, n_q_heads, cu_q, cu_children, parent_tables, max_pages_parent, parent_lens, child_tables,
                              max_pages_child, child_lens, n_parents, n_children, total_q, max_child_len, max_parent_rows,
                              max_parent_len, scale, out, lse, workspace, workspace_bytes, (cudaStream_t)stream);
}

// ---- one call from host buffers ---------------------------------------------------------------
// Layout of the staging area: the device copies of the inputs and results, each 256-byte aligned, followed by the
// attention workspace.
namespace {
struct HostStepLayout {
  size_t q, k, v, cu, bt, pl, el, out, lse, ws, total;
};
HostStepLayout host_step_layout(const kv_pool_t* p, int n_q_heads, int batch, int total_q, int max_pages, int max_total_len) {
  HostStepLayout L{};
  const size_t D = (size_t)p->head_dim;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t at = o; o += align256(bytes); return at; };
  L.q = take((size_t)total_q * n_q_heads * D * 2);
  L.k = take((size_t)total_q * p->n_kv_heads * D * 2);
  L.v = take((size_t)total_q * p->n_kv_heads * D * 2);
  L.cu = take(sizeof(int) * ((size_t)batch + 1));
  L.bt = take(sizeof(int) * (size_t)batch * max_pages);
  L.pl = take(sizeof(int) * (size_t)batch);
  L.el = take(sizeof(int) * (size_t)batch);
  L.out = take((size_t)total_q * n_q_heads * D * 2);
  L.lse = take((size_t)total_q * n_q_heads * 4);
  L.ws = o;
  L.total = o + attn_workspace_bytes(p, n_q_heads, batch, total_q, max_total_len, 0, 0);
  return L;
}
}  // namespace

size_t attn_extend_host_staging_bytes(const kv_pool_t* p, int n_q_heads, int batch, int total_q, int max_pages,
                                      int max_total_len) {
  if (p == nullptr || n_q_heads <= 0 || batch <= 0 || total_q <= 0 || max_pages <= 0) return 0;
  return host_step_layout(p, n_q_heads, batch, total_q, max_pages, max_total_len).total;
}

kv_status_t attn_extend_host(kv_pool_t* p, const void* q, const void* k_new, const void* v_new, int n_q_heads,
                             const int* cu_q, const int* block_tables, int max_pages, const int* prefix_lens,
                             const int* extend_lens, int batch, int total_q, int max_extend_len, int max_total_len,
                             float scale, void* out, float* lse, void* staging, size_t staging_bytes, void* stream) {
  if (p == nullptr || batch < 0 || total_q < 0 || max_pages < 0) return KV_ERR_INVALID;
  if (!heads_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  if (batch == 0 || total_q == 0) return KV_OK;
  if (q == nullptr || k_new == nullptr || v_new == nullptr || cu_q == nullptr || block_tables == nullptr ||
      prefix_lens == nullptr || extend_lens == nullptr || out == nullptr || lse == nullptr || staging == nullptr)
    return KV_ERR_INVALID;
  if (((uintptr_t)staging) & 255) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  const HostStepLayout L = host_step_layout(p, n_q_heads, batch, total_q, max_pages, max_total_len);
  if (staging_bytes < L.total) return KV_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* d = reinterpret_cast<char*>(staging);
  const size_t D = (size_t)p->head_dim;
  const size_t q_bytes = (size_t)total_q * n_q_heads * D * 2, kv_bytes = (size_t)total_q * p->n_kv_heads * D * 2;
  // The copies run on the pool's own copy streams: a stream that carries copies in both directions and kernels
  // serialises them, which costs a third of the throughput of back-to-back steps (measured).  Per staging area:
  // copy in after the kernels that last used it; kernels (caller's stream) after the copy in; copy out after the
  // kernels; the caller's stream waits for the copy out, so it still orders everything the caller does next.
  kv_pool::HostSlot* hs = nullptr;
  {
    std::lock_guard<std::mutex> g(p->mu);
    for (auto& c : p->host_slots)
      if (c.staging == staging) hs = &c;
    if (hs == nullptr) {
      hs = &p->host_slots[p->host_slot_next];
      p->host_slot_next = (p->host_slot_next + 1) % kv_pool::kHostSlots;
      // the slot's previous staging area is forgotten: wait for what was still using its events
      if (hs->staging != nullptr) KV_CUDA_OK(cudaEventSynchronize(hs->out));
      hs->staging = staging;
    }
  }
  KV_CUDA_OK(cudaStreamWaitEvent(p->h2d_stream, hs->ran, 0));  // (a never-recorded event counts as complete)
  KV_CUDA_OK(cudaMemcpyAsync(d + L.k, k_new, kv_bytes, cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.v, v_new, kv_bytes, cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.q, q, q_bytes, cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.cu, cu_q, sizeof(int) * ((size_t)batch + 1), cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.bt, block_tables, sizeof(int) * (size_t)batch * max_pages, cudaMemcpyHostToDevice,
                             p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.pl, prefix_lens, sizeof(int) * (size_t)batch, cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaMemcpyAsync(d + L.el, extend_lens, sizeof(int) * (size_t)batch, cudaMemcpyHostToDevice, p->h2d_stream));
  KV_CUDA_OK(cudaEventRecord(hs->in, p->h2d_stream));
  KV_CUDA_OK(cudaStreamWaitEvent(st, hs->in, 0));
  const int* d_cu = reinterpret_cast<const int*>(d + L.cu);
  const int* d_bt = reinterpret_cast<const int*>(d + L.bt);
  const int* d_pl = reinterpret_cast<const int*>(d + L.pl);
  const int* d_el = reinterpret_cast<const int*>(d + L.el);
  // the suffix K/V rows of sequence i go to positions prefix_lens[i] .. of its pages, then the suffix attends
  kv_status_t s = attn_extend_append(p, d + L.q, d + L.k, d + L.v, n_q_heads, d_cu, d_bt, max_pages, d_pl, d_el, batch, total_q,
                                     max_extend_len, max_total_len, scale, d + L.out, reinterpret_cast<float*>(d + L.lse),
                                     d + L.ws, L.total - L.ws, stream);
  KV_CUDA_OK(cudaEventRecord(hs->ran, st));
  if (s != KV_OK) return s;
  KV_CUDA_OK(cudaStreamWaitEvent(p->d2h_stream, hs->ran, 0));
  KV_CUDA_OK(cudaMemcpyAsync(out, d + L.out, q_bytes, cudaMemcpyDeviceToHost, p->d2h_stream));
  KV_CUDA_OK(cudaMemcpyAsync(lse, d + L.lse, (size_t)total_q * n_q_heads * 4, cudaMemcpyDeviceToHost, p->d2h_stream));
  KV_CUDA_OK(cudaEventRecord(hs->out, p->d2h_stream));
  KV_CUDA_OK(cudaStreamWaitEvent(st, hs->out, 0));
  return KV_OK;
}

kv_status_t kvattn_set_shared_impl(int impl) {
  if (impl < 0 || impl > 2) return KV_ERR_INVALID;
  g_shared_impl.store(impl);
  return KV_OK;
}

kv_status_t kvattn_set_decode_impl(int impl) {
  if (impl < 0 || impl > 2) return KV_ERR_INVALID;
  g_decode_impl.store(impl);
  return KV_OK;
}

kv_status_t kvattn_set_mixed_extend_ctas(int n) {
  if (n < 0) return KV_ERR_INVALID;
  g_mixed_extend_ctas.store(n);
  return KV_OK;
}

static kv_status_t decode_impl(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                               const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                               void* workspace, size_t workspace_bytes, void* stream, bool beside) {
  if (p == nullptr || batch < 0 || max_pages < 0 || max_ctx_len < 0) return KV_ERR_INVALID;
  if (!heads_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  if (batch == 0) return KV_OK;
  if (q == nullptr || block_tables == nullptr || ctx_lens == nullptr || out == nullptr || lse == nullptr)
    return KV_ERR_INVALID;
  if ((((uintptr_t)q) | ((uintptr_t)out)) & 15) return KV_ERR_INVALID;
  if (max_ctx_len > (int64_t)max_pages * kPageSize) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  if (max_ctx_len == 0) max_ctx_len = 1;  // every row is empty: still defines O = 0, LSE = -inf
  // the decode region of a combined workspace starts after the extend region; a caller that sized
  // the workspace for decode only passes (0, 0) for the extend part, so the offset is 0 there
  return launch_decode(p, q, n_q_heads, block_tables, max_pages, ctx_lens, batch, max_ctx_len, scale, out, lse,
                       workspace, workspace_bytes, (cudaStream_t)stream, beside);
}

kv_status_t attn_decode(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                        const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream) {
  return decode_impl(p, q, n_q_heads, block_tables, max_pages, ctx_lens, batch, max_ctx_len, scale, out, lse, workspace,
                     workspace_bytes, stream, false);
}

kv_status_t attn_mixed(kv_pool_t* p, int n_q_heads, float scale, const attn_extend_args_t* ext,
                       const attn_decode_args_t* dec, void* workspace, size_t workspace_bytes, void* stream) {
  if (p == nullptr || !on_pool_device(p)) return KV_ERR_INVALID;
  if (!heads_supported(p, n_q_heads)) return KV_ERR_UNSUPPORTED;
  // (an extend set that launches nothing must not count: the decode kernel may only be queued to start early behind a
  // kernel of this call, never behind whatever the caller ran before)
  const bool has_ext = ext != nullptr && ext->batch > 0 && ext->total_q > 0 && ext->max_extend_len > 0;
  const bool has_dec = dec != nullptr && dec->batch > 0;
  cudaStream_t st = (cudaStream_t)stream;
  size_t ext_bytes = 0;
  if (has_ext)
    ext_bytes = align256(extend_tc_workspace_bytes(n_q_heads, p->head_dim, ext->batch, ext->total_q, ext->max_total_len));
  if (ext_bytes > workspace_bytes) return KV_ERR_WORKSPACE;
  char* ws = reinterpret_cast<char*>(workspace);
  if (has_ext && has_dec) {
    // Both kernels go to the caller's stream.  The persistent extend kernel (tensor-bound) is limited to a share of
    // the SMs and lets the kernel queued behind it start as soon as its own CTAs are resident; the decode kernel
    // (HBM-bound) is queued with the early-start attribute, fills the other SMs at once and, block after block, the
    // SMs the extend CTAs give back.  It waits for nothing: it reads and writes nothing the extend kernel writes.
    int cap = g_mixed_extend_ctas.load();
    if (cap <= 0) {
      // Share of the SMs by the two kinds of work, from the host-side bounds: extend costs its flops at the rate the
      // kernel reaches per SM, decode its bytes at the rate at which about two thirds of the SMs saturate the memory.
      const int sms = sm_count_of(p->device);
      const double flops = 4.0 * p->head_dim * n_q_heads * (double)ext->total_q * 0.75 * ext->max_total_len;
      const double bytes = (double)dec->batch * 0.62 * dec->max_ctx_len * 2.0 * p->n_kv_heads * p->head_dim * 2.0;
      const double sm_s_ext = flops / 800e12 * sms, sm_s_dec = bytes / 6e12 * (sms * 0.68);
      cap = (int)(sms * sm_s_ext / (sm_s_ext + sm_s_dec) + 0.5);
      cap = cap < 16 ? 16 : (cap > sms - 32 ? sms - 32 : cap);
    }
    kv_status_t s = extend_impl(p, ext->q, n_q_heads, ext->cu_q, ext->block_tables, ext->max_pages, ext->prefix_lens,
                                ext->extend_lens, ext->batch, ext->total_q, ext->max_extend_len, ext->max_total_len,
                                scale, ext->out, ext->lse, ws, ext_bytes, cap, st);
    if (s != KV_OK) return s;
    return decode_impl(p, dec->q, n_q_heads, dec->block_tables, dec->max_pages, dec->ctx_lens, dec->batch, dec->max_ctx_len,
                       scale, dec->out, dec->lse, ws ? ws + ext_bytes : nullptr, workspace_bytes - ext_bytes, st, true);
  }
  if (has_ext)
    return attn_extend(p, ext->q, n_q_heads, ext->cu_q, ext->block_tables, ext->max_pages, ext->prefix_lens,
                       ext->extend_lens, ext->batch, ext->total_q, ext->max_extend_len, ext->max_total_len, scale,
                       ext->out, ext->lse, ws, ext_bytes, st);
  if (has_dec)
    return attn_decode(p, dec->q, n_q_heads, dec->block_tables, dec->max_pages, dec->ctx_lens, dec->batch,
                       dec->max_ctx_len, scale, dec->out, dec->lse, ws, workspace_bytes, st);
  return KV_OK;
}

}  // extern "C"
