// Extend attention for children that share a parent's prefix (the dependent tasks of a Cartesian
// product, Sections 5.1 and 5.3: every child task reuses its parent task's prefix and adds a short
// suffix of its own).
//
// Keys of child c of parent g: the first P_g tokens of the parent's pages, then the child's own
// E_c tokens in its private pages.  All suffix queries of all children of a parent are stacked row
// after row, so that the parent's pages are read once, with full query tiles, instead of once per
// child with mostly empty tiles.  Two ways to add the children's own keys:
//   fused   the tensor-core kernel's fan-out mode: after the parent's KV tiles an item walks the
//           tiles of every child that has a row in it, with all other rows masked.  One kernel, no
//           intermediate results.  Good when a child's suffix fills a fair part of a 128-row tile.
//   split   part A: the stacked rows over the parent's keys only; part B: every child's suffix
//           over its own pages; then the two partial results of a row are merged with the
//           log-sum-exp rule.  For very short suffixes (many children per tile).
#include "append.cuh"
#include "common.cuh"

namespace kvattn {

size_t extend_tc_workspace_bytes(int n_q_heads, int head_dim, int batch, int total_q, int max_total_len);
bool extend_tc_supported(const kv_pool_t* p, int n_q_heads);
kv_status_t launch_extend_tc(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                             int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                             int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, int cta_cap, int mode, const FanArgs* fan,
                             const AppendArgs* app, int phase, cudaStream_t st);
kv_status_t launch_extend_small(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                                int max_pages, const int* prefix_lens, const int* extend_lens, int batch,
                                int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                                cudaStream_t st);

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

std::atomic<int> g_shared_impl{0};  // 0: choose by the mean suffix length, 1: split, 2: fused

// Row ranges of the parents in Q (their children are consecutive) and a vector of zeros (the prefix
// lengths of part B).
__global__ void shared_prep_kernel(const int* __restrict__ cu_q, const int* __restrict__ cu_children, int n_parents,
                                   int n_children, int* __restrict__ cu_q_parent, int* __restrict__ rows_parent,
                                   int* __restrict__ zeros) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_parents) {
    const int r0 = __ldg(cu_q + __ldg(cu_children + i)), r1 = __ldg(cu_q + __ldg(cu_children + i + 1));
    cu_q_parent[i] = r0;
    rows_parent[i] = r1 - r0;
  }
  if (i == n_parents) cu_q_parent[n_parents] = __ldg(cu_q + n_children);
  if (i < n_children) zeros[i] = 0;
}

__device__ __forceinline__ int last_le(const int* __restrict__ a, int n, int x) {  // largest i < n with a[i] <= x
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (__ldg(a + mid) <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// out / lse hold part B (the child's own suffix) on entry and the merged result on exit.  One warp per
// (row, query head); lane l owns D/32 consecutive elements.
template <int D>
__global__ void __launch_bounds__(256) shared_merge_kernel(const __nv_bfloat16* __restrict__ o_a,
                                                           const float* __restrict__ lse_a, __nv_bfloat16* __restrict__ out,
                                                           float* __restrict__ lse, const int* __restrict__ cu_q,
                                                           const int* __restrict__ cu_children,
                                                           const int* __restrict__ parent_lens, int n_parents, int n_children,
                                                           int n_q_heads, int64_t total) {
  const int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (w >= total) return;
  const int lane = threadIdx.x & 31;
  const int row = (int)(w / n_q_heads);
  const int child = last_le(cu_q, n_children, row);
  const int parent = last_le(cu_children, n_parents, child);
  if (__ldg(parent_lens + parent) <= 0) return;  // nothing shared: part B is the result
  const float la = __ldg(lse_a + w), lb = lse[w];
  const float mx = fmaxf(la, lb);
  const float wa = __expf(la - mx), wb = __expf(lb - mx);  // lb = -inf only if the child has no suffix row here
  const float inv = 1.f / (wa + wb);
  constexpr int EPL = D / 32;  // elements per lane
  const __nv_bfloat16* pa = o_a + w * D + lane * EPL;
  __nv_bfloat16* po = out + w * D + lane * EPL;
  if (EPL == 4) {
    const uint2 va = __ldg(reinterpret_cast<const uint2*>(pa));
    const uint2 vb = *reinterpret_cast<const uint2*>(po);
    const uint32_t xa[2] = {va.x, va.y}, xb[2] = {vb.x, vb.y};
    uint32_t r[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float a0 = __uint_as_float(xa[i] << 16), a1 = __uint_as_float(xa[i] & 0xffff0000u);
      const float b0 = __uint_as_float(xb[i] << 16), b1 = __uint_as_float(xb[i] & 0xffff0000u);
      const float lo = (a0 * wa + b0 * wb) * inv, hi = (a1 * wa + b1 * wb) * inv;
      asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r[i]) : "f"(hi), "f"(lo));
    }
    *reinterpret_cast<uint2*>(po) = make_uint2(r[0], r[1]);
  } else {
    const uint32_t xa = __ldg(reinterpret_cast<const uint32_t*>(pa)), xb = *reinterpret_cast<const uint32_t*>(po);
    const float a0 = __uint_as_float(xa << 16), a1 = __uint_as_float(xa & 0xffff0000u);
    const float b0 = __uint_as_float(xb << 16), b1 = __uint_as_float(xb & 0xffff0000u);
    const float lo = (a0 * wa + b0 * wb) * inv, hi = (a1 * wa + b1 * wb) * inv;
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    *reinterpret_cast<uint32_t*>(po) = r;
  }
  if (lane == 0) lse[w] = mx + __logf(wa + wb);
}

size_t extend_shared_workspace_bytes(const kv_pool_t* p, int n_q_heads, int n_parents, int n_children, int total_q,
                                     int max_parent_len) {
  if (n_parents <= 0 || n_children <= 0 || total_q <= 0) return 0;
  return align256(sizeof(int) * (size_t)(2 * n_parents + 1 + n_children)) +
         align256((size_t)total_q * n_q_heads * p->head_dim * 2) + align256((size_t)total_q * n_q_heads * 4) +
         align256(extend_tc_workspace_bytes(n_q_heads, p->head_dim, n_children > n_parents ? n_children : n_parents, total_q,
                                            max_parent_len)) +
         256;
}

kv_status_t launch_extend_shared(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* cu_children,
                                 const int* parent_tables, int max_pages_parent, const int* parent_lens,
                                 const int* child_tables, int max_pages_child, const int* child_lens, int n_parents,
                                 int n_children, int total_q, int max_child_len, int max_parent_rows, int max_parent_len,
                                 float scale, void* out, float* lse, void* workspace, size_t workspace_bytes,
                                 cudaStream_t st) {
  if (workspace == nullptr ||
      workspace_bytes < extend_shared_workspace_bytes(p, n_q_heads, n_parents, n_children, total_q, max_parent_len))
    return KV_ERR_WORKSPACE;
  char* ws = reinterpret_cast<char*>(workspace);
  int* cu_q_parent = reinterpret_cast<int*>(ws);
  int* rows_parent = cu_q_parent + n_parents + 1;
  int* zeros = rows_parent + n_parents;
  ws += align256(sizeof(int) * (size_t)(2 * n_parents + 1 + n_children));
  __nv_bfloat16* o_a = reinterpret_cast<__nv_bfloat16*>(ws);
  ws += align256((size_t)total_q * n_q_heads * p->head_dim * 2);
  float* lse_a = reinterpret_cast<float*>(ws);
  ws += align256((size_t)total_q * n_q_heads * 4);
  const size_t tc_bytes = extend_tc_workspace_bytes(n_q_heads, p->head_dim, n_children > n_parents ? n_children : n_parents,
                                                    total_q, max_parent_len);

  const int n_prep = (n_parents + 1 > n_children ? n_parents + 1 : n_children);
  shared_prep_kernel<<<(n_prep + 255) / 256, 256, 0, st>>>(cu_q, cu_children, n_parents, n_children, cu_q_parent, rows_parent,
                                                           zeros);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  kv_status_t s;
  const int impl = g_shared_impl.load();
  const bool fused = impl == 2 || (impl == 0 && (int64_t)total_q >= 16 * (int64_t)n_children);
  if (fused) {
    FanArgs fan{cu_q, cu_children, child_tables, max_pages_child, n_children};
    return launch_extend_tc(p, q, n_q_heads, cu_q_parent, parent_tables, max_pages_parent, parent_lens, rows_parent,
                            n_parents, total_q, max_parent_rows, max_parent_len + max_parent_rows, scale, out, lse, ws,
                            tc_bytes, 0, 2, &fan, nullptr, 0, st);
  }
  // part B first, straight into the caller's buffers: each child's suffix over its private pages
  if (!extend_tc_supported(p, n_q_heads))
    s = launch_extend_small(p, q, n_q_heads, cu_q, child_tables, max_pages_child, zeros, child_lens, n_children,
                            max_child_len, max_child_len, scale, out, lse, st);
  else
    s = launch_extend_tc(p, q, n_q_heads, cu_q, child_tables, max_pages_child, zeros, child_lens, n_children, total_q,
                         max_child_len, max_child_len, scale, out, lse, ws, tc_bytes, 0, 0, nullptr, nullptr, 0, st);
  if (s != KV_OK) return s;
  if (max_parent_len <= 0) return KV_OK;
  // part A: the stacked suffix rows of each parent over the parent's prefix pages
  s = launch_extend_tc(p, q, n_q_heads, cu_q_parent, parent_tables, max_pages_parent, parent_lens, rows_parent, n_parents,
                       total_q, max_parent_rows, max_parent_len, scale, o_a, lse_a, ws, tc_bytes, 0, 1, nullptr, nullptr, 0, st);
  if (s != KV_OK) return s;
  const int64_t total = (int64_t)total_q * n_q_heads;
  const unsigned blocks = (unsigned)((total + 7) / 8);
  if (p->head_dim == 128)
    shared_merge_kernel<128><<<blocks, 256, 0, st>>>(o_a, lse_a, (__nv_bfloat16*)out, lse, cu_q, cu_children, parent_lens,
                                                     n_parents, n_children, n_q_heads, total);
  else
    shared_merge_kernel<64><<<blocks, 256, 0, st>>>(o_a, lse_a, (__nv_bfloat16*)out, lse, cu_q, cu_children, parent_lens,
                                                    n_parents, n_children, n_q_heads, total);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvattn
