// Tensor-core extend attention for sm_100a: suffix queries over reused prefix pages.
//
// Work item = (sequence, KV head, pair of 128-row query tiles).  The rows of a tile are the
// (suffix token, query head of the KV head's group) pairs, token-major, so the G query heads that
// share a KV head share every K/V tile that is brought on chip (GQA) and the causal diagonal is
// only 128/G tokens wide.  One persistent CTA per SM; the items are sorted by cost and taken heaviest
// first from a global counter, so a CTA that finishes early simply takes more.
// Besides extend, the kernel has a prefix-only mode and a fan-out mode (see TcArgs::mode).
//
// Roles (warp-specialised, 16 warps):
//   warps 0-3   softmax of query tile 0: one thread per row (= TMEM lane): masks, running max and
//   warps 4-7   softmax of query tile 1: sum, exp2, P as bf16 back to TMEM, lazy rescale of O.
//   warps 8-11  epilogue of both tiles: O / l -> bf16 -> global, while the softmax warps are already
//               at the next item.
//   warp 12     producer: per 128-token KV tile, one 1-D bulk copy per 16-token page block
//               (the pool keeps blocks in the MMA's 128-byte-swizzle operand layout) into a ring of
//               shared-memory stages; completion is signalled on mbarriers.
//   warp 13     MMA issuer (one elected lane): S = Q K^T and O += P V on tcgen05 with accumulators in
//               tensor memory; P is read straight from tensor memory (it overwrites S in place).
//   warp 14     Q loader: one tensor-map (TMA) copy per 64-dim half brings a query tile into shared
//               memory in the swizzled operand layout, as soon as the MMAs that read the previous
//               item's tile have finished.
//   warp 15     idle (launched for the registers it hands to the others).
// The two query tiles ping-pong: while one tile's softmax runs, the tensor core works on the other.
// All waits are bounded; on expiry the CTA records KV_ERR_TIMEOUT, drains its copies, frees its
// tensor memory and returns.
#include <type_traits>

#include <cuda.h>  // CUtensorMap and its enums (types only: the encoder is looked up at run time)

#include "append.cuh"
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace kvattn {
using namespace ptx;

// The roles' register budgets are set with setmaxnreg.  What the warps hold afterwards must not exceed what the
// CTA was launched with (512 threads x 128 registers), in total and per scheduler (warp index mod 4):
// 8 x 192 (softmax) + 4 x 72 (epilogue) + 56 + 56 + 40 + 24 = 2000 <= 2048 per lane.
constexpr int kTcThreads = 512;
constexpr int kWarpEpilogue = 8, kWarpProducer = 12, kWarpMma = 13, kWarpQ = 14;
constexpr int kPlanBuckets = 2048;
constexpr int kPlanSeqBuckets = 1024;   // length buckets for ranking the sequences (one per plan thread)
constexpr int kPlanMaxRanked = 8192;    // batches up to this size are ranked by length; larger ones keep their order
constexpr float kRescaleThreshold = 8.0f;  // log2 units: O is rescaled only when the max grows by more than this
constexpr int kOptimisticMinLen = 4096;     // batches with a sequence this long use the kernel that skips the maximum search
constexpr float kOptimisticSum = 65536.0f;  // a row sum of one tile beyond this sends the step to the exact maximum

struct TcArgs {
  PoolView pool;
  const __nv_bfloat16* q;
  const int* cu_q;
  const int* block_tables;
  int max_pages;
  const int* prefix_lens;
  const int* extend_lens;
  int batch, n_q_heads, group, lg_group;
  // mode 0: row t of sequence i sees the keys 0 .. P_i + t (extend).
  // mode 1: every row sees the keys [0, P_i) only.
  // mode 2 (fan-out): a "sequence" is a parent, its rows are the suffix tokens of its children stacked one
  //         after the other; a row sees the parent's keys [0, P) and then its own child's keys up to itself.
  //         The KV steps of an item are the parent's tiles followed by the tiles of every child that has a
  //         row in the item, each from the child's own pages.
  int mode;
  FanArgs fan;
  float scale_log2;
  __nv_bfloat16* out;
  float* lse;
  const int4* items;   // two int4 per entry (see ItemRec), cost-sorted
  const int* n_items;  // number of valid entries in items
  int* next_item;      // work counter: the next item of the global list nobody has taken yet
};

// ------------------------------------------------------------------------------------------
// Plan: list the (sequence, tile pair) entries that have rows, heaviest first (counting sort on
// the number of KV tile steps).  Only the order of execution depends on it, never a result.
// ------------------------------------------------------------------------------------------
// One entry of the plan: everything a CTA needs to know about a (sequence, tile pair), so that the
// roles read one 32-byte record per item instead of chasing the length arrays.
struct ItemRec {
  int seq, tp, P, E;
  int row0, n_kv0, n_kv1, kv_end;  // first query row; KV tile steps of the two tiles; keys the item sees at most
                                   // (fan-out mode: kv_end holds the first child that has a row in the item)
};

__device__ __forceinline__ ItemRec make_item(int seq, int tp, int P, int E, int row0, int lg, int max_pages, int mode,
                                             const FanArgs& fan) {
  ItemRec r{seq, tp, P, E, row0, 0, 0, 0};
  int tok_hi_t[2] = {-1, -1};
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r_lo = tp * 256 + t * 128;
    const int tok_lo = r_lo >> lg;
    if (tok_lo >= E) break;
    const int tok_hi = min(E - 1, (r_lo + 127) >> lg);
    tok_hi_t[t] = tok_hi;
    const int sees = mode != 0 ? P : P + tok_hi + 1;
    (t ? r.n_kv1 : r.n_kv0) = (sees + 127) >> 7;
    r.kv_end = sees;
  }
  if ((mode != 0 ? P : P + E) > max_pages * kPageSize) r.n_kv0 = r.n_kv1 = 0;  // longer than its block-table row: skipped (reported by the plan)
  if (mode == 2 && tok_hi_t[0] >= 0) {
    // children with a row in this item: the first one whose last token lies at or after the item's first token,
    // then on until a child starts after the item's last token
    const int c0 = __ldg(fan.cu_children + seq), c1 = __ldg(fan.cu_children + seq + 1);
    const int tok_lo = (tp * 256) >> lg;
    int lo = c0, hi = c1;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(fan.cu_q + mid + 1) - row0 > tok_lo) hi = mid; else lo = mid + 1;
    }
    const int c_first = lo;
    const int tok_hi_item = max(tok_hi_t[0], tok_hi_t[1]);
    int extra0 = 0, extra = 0;
    bool fits = true;
    for (int c = c_first; c < c1; ++c) {
      const int start = __ldg(fan.cu_q + c) - row0, len = __ldg(fan.cu_q + c + 1) - __ldg(fan.cu_q + c);
      if (start > tok_hi_item) break;
      if (len > fan.max_pages * kPageSize) fits = false;
      const int st = (len + 127) >> 7;
      extra += st;
      if (start <= tok_hi_t[0]) extra0 += st;
    }
    r.kv_end = c_first;
    if (!fits) {
      r.n_kv0 = r.n_kv1 = 0;
    } else if (r.n_kv0 > 0 || P == 0) {
      r.n_kv0 = ((P + 127) >> 7) + extra0;
      r.n_kv1 = tok_hi_t[1] >= 0 ? ((P + 127) >> 7) + extra : 0;
    }
  }
  return r;
}

struct PlanArgs {
  const int* prefix_lens;
  const int* extend_lens;
  const int* cu_q;
  int batch, max_tp, lg, max_steps, capacity, max_pages, mode;
  FanArgs fan;
  int groups;
  int* status;
  int4* items;
  int* n_items;
  int* next_item;
  int first_free_item;
};

// Runs in one block of 1024 threads.
__device__ __forceinline__ void plan_body(const PlanArgs& pa) {
  const int* __restrict__ prefix_lens = pa.prefix_lens;
  const int* __restrict__ extend_lens = pa.extend_lens;
  const int* __restrict__ cu_q = pa.cu_q;
  const int batch = pa.batch, max_tp = pa.max_tp, lg = pa.lg, max_steps = pa.max_steps, capacity = pa.capacity;
  const int max_pages = pa.max_pages, mode = pa.mode, groups = pa.groups, first_free_item = pa.first_free_item;
  const FanArgs& fan = pa.fan;
  int* status = pa.status;
  int4* __restrict__ items = pa.items;
  int* __restrict__ n_items = pa.n_items;
  int* __restrict__ next_item = pa.next_item;
  if (threadIdx.x == 0) {
    next_item[0] = first_free_item;  // the CTAs start on items 0 .. grid-1 without asking
    next_item[1] = 0;                // CTAs of the attention kernel that have finished
  }
  __shared__ int hist[kPlanBuckets];
  for (int i = threadIdx.x; i < kPlanBuckets; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const int64_t n = (int64_t)batch * max_tp;
  // A sequence with more suffix tokens than the host-side bound the grid was sized with would lose its last rows
  // without a trace: it is reported instead.
  for (int seq = threadIdx.x; seq < batch; seq += blockDim.x) {
    const int E = __ldg(extend_lens + seq);
    if (__ldg(prefix_lens + seq) >= 0 && (int64_t)E > (((int64_t)max_tp * 256) >> lg)) report(status, KV_ERR_BOUNDS);
  }
  // The sequences are put into groups longest first, so that the last groups, which decide how evenly the CTAs
  // finish, hold the cheapest items: a counting sort of the sequences on their length (ties in arrival order: only
  // the order of execution depends on it).
  __shared__ int seq_hist[kPlanSeqBuckets];
  __shared__ unsigned short seq_rank[kPlanMaxRanked];
  const bool ranked = groups > 1 && batch <= kPlanMaxRanked;
  if (ranked) {
    __shared__ int seq_warp_tot[32];
    seq_hist[threadIdx.x] = 0;
    __syncthreads();
    const int64_t span = (int64_t)max(max_steps, 1) * 64 + 1;  // longer than any sequence the tables can hold
    auto bucket_of = [&](int P, int E) {
      return (int)min((int64_t)(kPlanSeqBuckets - 1), (int64_t)(P + E) * kPlanSeqBuckets / span);
    };
    for (int seq = threadIdx.x; seq < batch; seq += blockDim.x) {
      const int P = __ldg(prefix_lens + seq), E = __ldg(extend_lens + seq);
      if (P >= 0 && E > 0) atomicAdd(&seq_hist[bucket_of(P, E)], 1);
    }
    __syncthreads();
    {  // exclusive prefix, longest bucket first: thread i owns bucket B-1-i
      const int b = kPlanSeqBuckets - 1 - (int)threadIdx.x;
      const int c = seq_hist[b];
      int incl = c;
      const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
      }
      if (lane == 31) seq_warp_tot[w] = incl;
      __syncthreads();
      if (w == 0) {
        int t = seq_warp_tot[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, t, off);
          if (lane >= off) t += v;
        }
        seq_warp_tot[lane] = t;
      }
      __syncthreads();
      seq_hist[b] = (w > 0 ? seq_warp_tot[w - 1] : 0) + incl - c;
    }
    __syncthreads();
    for (int seq = threadIdx.x; seq < batch; seq += blockDim.x) {
      const int P = __ldg(prefix_lens + seq), E = __ldg(extend_lens + seq);
      seq_rank[seq] = (P >= 0 && E > 0) ? (unsigned short)atomicAdd(&seq_hist[bucket_of(P, E)], 1) : 0;
    }
    __syncthreads();
  }
  // Sort key, larger = earlier: the sequences are taken group after group (a group's K/V stays in L2 while its items
  // run, and the tile pairs of a sequence read the same pages), heaviest item first inside a group.
  const int per_group = kPlanBuckets / groups;
  auto key_of = [&](int steps, int seq) {
    const int64_t k = (int64_t)steps * (per_group - 1) / max(max_steps, 1);
    const int cost = (int)min((int64_t)(per_group - 1), k);
    const int grp = (int)((int64_t)(ranked ? (int)seq_rank[seq] : seq) * groups / batch);
    return (groups - 1 - grp) * per_group + cost;
  };
  for (int64_t e = threadIdx.x; e < n; e += blockDim.x) {
    const int seq = (int)(e / max_tp), tp = (int)(e % max_tp);
    const int P = __ldg(prefix_lens + seq), E = __ldg(extend_lens + seq);
    if (P < 0 || E <= 0) continue;
    if (((tp * 256) >> lg) >= E) continue;
    const ItemRec r = make_item(seq, tp, P, E, __ldg(cu_q + seq), lg, max_pages, mode, fan);
    const int steps = r.n_kv0 + r.n_kv1;
    if (steps > 0) atomicAdd(&hist[key_of(steps, seq)], 1);
  }
  __syncthreads();
  // exclusive prefix over the buckets, heaviest first: thread i owns buckets B-1-2i and B-2-2i
  {
    __shared__ int warp_tot[32];
    const int b0 = kPlanBuckets - 1 - 2 * (int)threadIdx.x, b1 = b0 - 1;
    const int c0 = hist[b0], c1 = hist[b1];
    int incl = c0 + c1;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += v;
    }
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    if (w == 0) {
      int t = warp_tot[lane];
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, t, off);
        if (lane >= off) t += v;
      }
      warp_tot[lane] = t;  // inclusive totals of the warps
    }
    __syncthreads();
    const int base = (w > 0 ? warp_tot[w - 1] : 0) + incl - (c0 + c1);
    hist[b0] = base;
    hist[b1] = base + c0;
    if (threadIdx.x == blockDim.x - 1) *n_items = min(base + c0 + c1, capacity);
  }
  __syncthreads();
  for (int64_t e = threadIdx.x; e < n; e += blockDim.x) {
    const int seq = (int)(e / max_tp), tp = (int)(e % max_tp);
    const int P = __ldg(prefix_lens + seq), E = __ldg(extend_lens + seq);
    if (P < 0 || E <= 0) continue;
    if (((tp * 256) >> lg) >= E) continue;
    const ItemRec r = make_item(seq, tp, P, E, __ldg(cu_q + seq), lg, max_pages, mode, fan);
    const int steps = r.n_kv0 + r.n_kv1;
    if (steps == 0 && (mode == 0 || P > 0 || mode == 2)) report(status, KV_ERR_BOUNDS);  // rows exist but the lengths do not fit the tables
    if (steps > 0) {
      const int pos = atomicAdd(&hist[key_of(steps, seq)], 1);
      if (pos < capacity) {
        items[2 * pos] = make_int4(r.seq, r.tp, r.P, r.E);
        items[2 * pos + 1] = make_int4(r.row0, r.n_kv0, r.n_kv1, r.kv_end);
      } else {
        report(status, KV_ERR_BOUNDS);  // more rows on the device than the total the host gave: the entry is dropped
      }
    }
  }
}

__global__ void __launch_bounds__(1024) extend_tc_plan_kernel(const PlanArgs pa) {
  launch_dependents();  // the attention kernel may set itself up meanwhile; it waits for this kernel before it reads the plan
  plan_body(pa);
}

// Prologue of the fused append + extend call: block 0 builds the plan while the other blocks scatter the suffix K/V
// rows into their pages (one warp per token), so the step has one small kernel in front of the attention kernel
// instead of two in a row, and the attention kernel's launch and set-up overlap it.
__global__ void __launch_bounds__(1024) extend_prologue_kernel(const PlanArgs pa, const PoolView pool, const AppendArgs ap) {
  launch_dependents();
  if (blockIdx.x == 0) {
    plan_body(pa);
  } else {
    const int warps_per_block = blockDim.x >> 5;
    append_tokens<4>(pool, ap, (blockIdx.x - 1) * warps_per_block + (threadIdx.x >> 5), (gridDim.x - 1) * warps_per_block);
  }
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// ------------------------------------------------------------------------------------------
template <int D>
struct TcCfg {
  static constexpr int kTileBytes = 128 * D * 2;   // a 128-row tile of Q, K or V
  static constexpr int kBlockBytes = 16 * D * 2;   // one (page, head) block
  static constexpr int kStages = D == 128 ? 5 : 8;
  static constexpr uint32_t kGroupStride = D * 16;  // bytes between 8-token groups inside the K/V tiles
  static constexpr int kHalves = D / 64;
  static constexpr int kQHalfStride = 128 * 128;    // Q tile: [half][row][128 B]
};

template <int D>
struct __align__(1024) TcSmem {
  unsigned char q[2][TcCfg<D>::kTileBytes];
  unsigned char kv[TcCfg<D>::kStages][TcCfg<D>::kTileBytes];
  unsigned long long kv_full[TcCfg<D>::kStages], kv_empty[TcCfg<D>::kStages];
  unsigned long long q_full[2], q_empty[2], s_full[2], p_full[2], o_full[2], o_empty[2], l_full[2];
  // Item queue of the CTA: the producer takes items off the global list (heaviest first, whoever is free
  // takes the next) and announces them here; every role walks the same sequence.
  unsigned long long sched_full[4], sched_empty[4];
  int sched_idx[4];
  float inv_l[2][2][128];  // [tile][item parity][row]: 1 / row sum, handed from the softmax to the epilogue warps
  uint32_t tmem_base;
  int abort_flag;
};

struct Item {
  int seq, kvh, tp, P, E, row0;
  int n_kv[2];   // KV tile steps of the two query tiles (0 = tile has no rows)
  int ld_tiles;  // KV tiles the producer brings in
  int kv_end;    // keys the item can see at most (fan-out mode: the parent's keys)
  int c_first;   // fan-out mode: first child with a row in the item
};

// Fan-out mode: position in the children's part of an item's KV steps.
struct ChildCur {
  int c, jc;        // child and 128-key tile inside the child's suffix
  int start, len;   // the child's first token among the parent's stacked rows, and its length
};
__device__ __forceinline__ void child_load(const TcArgs& a, int row0, ChildCur& k) {
  // children without tokens contribute no step
  int r0 = __ldg(a.fan.cu_q + k.c), r1 = __ldg(a.fan.cu_q + k.c + 1);
  while (r1 == r0 && k.c + 1 < a.fan.n_children) {
    ++k.c;
    r0 = r1;
    r1 = __ldg(a.fan.cu_q + k.c + 1);
  }
  k.start = r0 - row0;
  k.len = r1 - r0;
}
__device__ __forceinline__ void child_first(const TcArgs& a, const Item& it, ChildCur& k) {
  k.c = it.c_first;
  k.jc = 0;
  child_load(a, it.row0, k);
}
__device__ __forceinline__ void child_next(const TcArgs& a, const Item& it, ChildCur& k) {
  if ((k.jc + 1) * 128 < k.len) {
    ++k.jc;
  } else if (k.c + 1 < a.fan.n_children) {
    ++k.c;
    k.jc = 0;
    child_load(a, it.row0, k);
  }
}
__device__ __forceinline__ int child_pages(const ChildCur& k) { return min(8, (k.len - k.jc * 128 + 15) >> 4); }

// Item k of the global list: entry k / Hkv of the plan, KV head k % Hkv.  Returns false past the end.
template <bool FAN>
__device__ __forceinline__ bool fetch_item(const TcArgs& a, int k, int n_total, Item& it) {
  if (k >= n_total) return false;
  const int Hkv = a.pool.n_kv_heads;
  const int e = k / Hkv;
  const int4 r0 = __ldcg(a.items + 2 * e), r1 = __ldcg(a.items + 2 * e + 1);  // written by the kernel before this one: read through L2
  it.seq = r0.x; it.tp = r0.y; it.P = r0.z; it.E = r0.w;
  it.row0 = r1.x; it.n_kv[0] = r1.y; it.n_kv[1] = r1.z; it.kv_end = r1.w;
  it.c_first = 0;
  if (FAN) {
    it.c_first = r1.w;
    it.kv_end = it.P;
  }
  it.kvh = k - e * Hkv;
  it.ld_tiles = max(it.n_kv[0], it.n_kv[1]);
  return true;
}

// Operand descriptors differ only in their low word (start address >> 4 plus the leading-dimension
// offset field); the high word is a constant.  Issuing an MMA then costs one add, so a single thread
// keeps the tensor pipe fed.
__device__ __forceinline__ uint64_t make_desc(uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; }

// S[128 rows x 128 keys] = Q_t (K-major, shared) x K_stage (K-major, shared); q_lo / k_lo: low descriptor words
template <int D>
__device__ __forceinline__ void issue_s_mmas(uint32_t s_tmem, uint32_t q_lo, uint32_t k_lo) {
  constexpr uint32_t kHiQ = (1024u >> 4) | (1u << 14) | (2u << 29);        // SBO 1024, sm_100 descriptor, 128B swizzle
  constexpr uint32_t kHiK = ((uint32_t)(D * 16) >> 4) | (1u << 14) | (2u << 29);  // SBO = 8-token group stride
  constexpr uint32_t idesc = idesc_bf16(128, 128, 0, 0);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks)
    mma_ss(s_tmem, make_desc(kHiQ, q_lo + (ks >> 2) * 1024 + (ks & 3) * 2), make_desc(kHiK, k_lo + (ks >> 2) * 64 + (ks & 3) * 2),
           idesc, ks > 0);
}

// O[128 rows x D] (+)= P (bf16 in tensor memory) x V_stage (MN-major, shared), one MMA per 16-token page
template <int D>
__device__ __forceinline__ void issue_pv_mmas(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_lo, int np, bool first) {
  constexpr uint32_t kHiV = ((uint32_t)(D * 16) >> 4) | (1u << 14) | (2u << 29);
  constexpr uint32_t idesc = idesc_bf16(128, D, 0, 1);
  mma_ts(o_tmem, p_tmem, make_desc(kHiV, v_lo), idesc, first ? 0u : 1u);
#pragma unroll
  for (int p = 1; p < 8; ++p)
    if (p < np) mma_ts(o_tmem, p_tmem + p * 8, make_desc(kHiV, v_lo + p * (D * 2)), idesc, 1u);
}

// OPT: the softmax warps skip the search for the row maximum after an item's first tile (see there); chosen by the
// host for batches whose sequences are long, where nearly every step is such a step.
// FAN: the fan-out mode (TcArgs::mode 2); the other modes are compiled without the walk over the children's tiles.
template <int D, bool OPT, bool FAN>
__global__ void __launch_bounds__(kTcThreads, 1) attn_extend_tc_kernel(const TcArgs a, const __grid_constant__ CUtensorMap q_map) {
  using Cfg = TcCfg<D>;
  extern __shared__ unsigned char smem_raw[];
  // Dynamic shared memory starts on a 1024-byte boundary (this kernel has no static shared memory); the swizzled
  // operand tiles need that.  Checked instead of padded for: the tiles leave no room for padding.
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) report(a.pool.status, KV_ERR_CUDA);
    return;
  }
  // A kernel queued behind this one with the early-start attribute may take the SMs this grid leaves free as soon as
  // every CTA of this grid is resident (the mixed step queues the decode kernel that way).
  launch_dependents();
  TcSmem<D>& sm = *reinterpret_cast<TcSmem<D>*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abortp = &sm.abort_flag;

  if (tid == 0) {
    sm.abort_flag = 0;
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(smem_u32(&sm.kv_full[s]), 1);
      mbar_init(smem_u32(&sm.kv_empty[s]), 1);
    }
    for (int s4 = 0; s4 < 4; ++s4) {
      mbar_init(smem_u32(&sm.sched_full[s4]), 1);    // the producer wrote the slot
      mbar_init(smem_u32(&sm.sched_empty[s4]), 14);  // MMA warp, Q loader, 8 softmax and 4 epilogue warps have read it
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&sm.q_full[t]), 1);    // the Q tile's bytes have landed (transaction count)
      mbar_init(smem_u32(&sm.q_empty[t]), 1);   // tensor core finished the item's last S: the Q buffer may be refilled
      mbar_init(smem_u32(&sm.s_full[t]), 1);    // tensor core finished S (and everything issued before it)
      mbar_init(smem_u32(&sm.p_full[t]), 128);  // every softmax thread wrote its row of P
      mbar_init(smem_u32(&sm.o_full[t]), 1);    // tensor core finished the item's last PV
      mbar_init(smem_u32(&sm.o_empty[t]), 128); // every epilogue thread has read its row of O: the next item may overwrite it
      mbar_init(smem_u32(&sm.l_full[t]), 128);  // every softmax thread has published 1 / row sum
    }
    fence_mbar_init();
  }
  if (warp == kWarpProducer) {
    tmem_alloc(smem_u32(&sm.tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_base;
  // Everything up to here touched only this CTA's own shared and tensor memory and may have run while the kernel in
  // front of this one (the plan, or the plan and the suffix append) was still at work; its results are needed now.
  dependency_wait();
  const int n_total = __ldcg(a.n_items) * a.pool.n_kv_heads;
  const int Hkv = a.pool.n_kv_heads;
  // Round r of this CTA works on item sched_get(r) of the global list (>= n_total: no more work).  A warp
  // calls sched_release(r) once it no longer needs the slot.
  auto sched_get = [&](int round) -> int {
    const bool got = mbar_wait(smem_u32(&sm.sched_full[round & 3]), (round >> 2) & 1, abortp);
    const int idx = *reinterpret_cast<volatile int*>(&sm.sched_idx[round & 3]);
    return got ? idx : 0x7fffffff;
  };
  auto sched_release = [&](int round) {
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&sm.sched_empty[round & 3]));
  };

  if (warp == kWarpProducer) {
    // =============================== producer =============================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    const char* kpool = reinterpret_cast<const char*>(a.pool.k);
    const char* vpool = reinterpret_cast<const char*>(a.pool.v);
    uint32_t loads = 0;  // stage loads issued so far (ring position)
    bool ok = true;
    // Announces item idx as round r (waits until every reader is done with the slot's previous round).
    auto announce = [&](int r, int idx) {
      if (lane == 0) {
        ok = mbar_wait(smem_u32(&sm.sched_empty[r & 3]), ((r >> 2) & 1) ^ 1, abortp);
        *reinterpret_cast<volatile int*>(&sm.sched_idx[r & 3]) = idx;
        mbar_arrive(smem_u32(&sm.sched_full[r & 3]));
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
    };
    int cur = blockIdx.x;
    announce(0, cur);
    for (int round = 0; ok && cur < n_total; ++round) {
      // The next item is taken and announced one item ahead, so that nobody waits for the counter.  (Taking it
      // two items ahead would hide the counter's latency from this warp too, but an item that is committed early
      // cannot go to a CTA that runs out of work: measured slower.)
      int nxt_idx = 0;
      if (lane == 0) nxt_idx = atomicAdd(a.next_item, 1);
      nxt_idx = __shfl_sync(0xffffffffu, nxt_idx, 0);
      announce(round + 1, nxt_idx);
      Item it;
      fetch_item<FAN>(a, cur, n_total, it);
      cur = nxt_idx;
      if (!ok) break;
      const int* bt = a.block_tables + (int64_t)it.seq * a.max_pages;
      const size_t head_off = (size_t)it.kvh * Cfg::kBlockBytes;
      const int n_own = FAN ? (it.P + 127) >> 7 : it.ld_tiles;  // tiles from the sequence's (parent's) own pages
      ChildCur cc{0, 0, 0, 0};
      for (int j = 0; j < it.ld_tiles && ok; ++j) {
        int np = min(8, (it.kv_end - j * 128 + 15) >> 4);
        const int* src_bt = bt + j * 8;
        if (FAN && j >= n_own) {  // fan-out mode: a tile of a child's own keys
          if (j == n_own) child_first(a, it, cc); else child_next(a, it, cc);
          np = child_pages(cc);
          src_bt = a.fan.tables + (int64_t)cc.c * a.fan.max_pages + cc.jc * 8;
        }
        int page = 0;
        if (lane < np) {
          page = __ldg(src_bt + lane);
          if ((unsigned)page >= (unsigned)a.pool.num_pages) {
            report(a.pool.status, KV_ERR_BOUNDS);
            page = 0;
          }
        }
        const size_t src_off = ((size_t)page * Hkv) * Cfg::kBlockBytes + head_off;
#pragma unroll
        for (int which = 0; which < 2; ++which) {  // 0: K tile, 1: V tile
          const uint32_t s = loads % Cfg::kStages, par = (loads / Cfg::kStages) & 1;
          const uint32_t full = smem_u32(&sm.kv_full[s]);
          if (lane == 0) {
            ok = mbar_wait(smem_u32(&sm.kv_empty[s]), par ^ 1, abortp);
            if (ok) mbar_arrive_expect_tx(full, (uint32_t)np * Cfg::kBlockBytes);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
          if (lane < np)
            bulk_g2s(smem_u32(sm.kv[s]) + lane * Cfg::kBlockBytes, (which ? vpool : kpool) + src_off, Cfg::kBlockBytes,
                     full);
          ++loads;
        }
      }
    }
    if (!ok && lane == 0) {
      // give copies that were already issued time to land before the CTA's shared memory goes away
      const uint32_t first = loads > (uint32_t)Cfg::kStages ? loads - Cfg::kStages : 0;
      for (uint32_t i = first; i < loads; ++i) {
        const uint32_t s = i % Cfg::kStages, par = (i / Cfg::kStages) & 1;
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(smem_u32(&sm.kv_full[s]), par) && globaltimer_ns() - t0 < 100000000ull) {
        }
      }
    }
  } else if (warp == kWarpMma) {
    // =============================== MMA issuer ===========================================
    // One thread issues every MMA of the CTA.  Per KV tile j and query tile t:  O_t (+)= P_t V(j) as soon as
    // the softmax warps have written P_t, then S_t = Q_t K(j+1)^T into the columns P_t occupied (the tensor
    // core runs MMAs in issue order), so the other tile's MMAs fill the time this tile's softmax takes.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    const uint32_t q_lo0 = (smem_u32(sm.q[0]) >> 4) | (1u << 16);             // low descriptor words: LBO field 16 B
    const uint32_t k_lo0 = (smem_u32(sm.kv[0]) >> 4) | (1u << 16);
    const uint32_t v_lo0 = (smem_u32(sm.kv[0]) >> 4) | ((1024u >> 4) << 16);  // V tiles: LBO = 64-dim half
    const uint32_t bar_s_full = smem_u32(&sm.s_full[0]), bar_p_full = smem_u32(&sm.p_full[0]);
    const uint32_t bar_q_full = smem_u32(&sm.q_full[0]), bar_o_full = smem_u32(&sm.o_full[0]);
    const uint32_t bar_q_empty = smem_u32(&sm.q_empty[0]), bar_o_empty = smem_u32(&sm.o_empty[0]);
    uint32_t o_uses[2] = {0, 0};        // items per tile whose PV has started (phase of o_empty)
    bool early0 = false;                // tile 0's first S of the coming item has been issued already
    uint32_t loads = 0;                 // ring position, mirrors the producer
    uint32_t steps[2] = {0, 0};         // softmax steps per tile so far (phase of p_full)
    uint32_t items_done[2] = {0, 0};    // items per tile so far (phase of q_full)
    bool ok = true;
    Item nxt;
    bool has_nxt = fetch_item<FAN>(a, sched_get(0), n_total, nxt);
    for (int round = 0; ok && has_nxt; ++round) {
      const Item it = nxt;
      has_nxt = fetch_item<FAN>(a, sched_get(round + 1), n_total, nxt);
      sched_release(round);
      if (it.ld_tiles == 0) continue;
      {
        // The whole warp runs this control flow (all values are warp-uniform); one elected lane issues.
        // first K tile: S(0) of each query tile as soon as its Q tile is in shared memory
        uint32_t stage = loads % Cfg::kStages;
        ok = mbar_wait(smem_u32(&sm.kv_full[stage]), (loads / Cfg::kStages) & 1, abortp);
        ++loads;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (!ok || it.n_kv[t] == 0) continue;
          if (t == 0 && early0) {
            early0 = false;
            continue;
          }
          ok = mbar_wait(bar_q_full + 8 * t, items_done[t] & 1, abortp);
          ++items_done[t];
          if (!ok) continue;
          if (elect_one_sync()) {
            issue_s_mmas<D>(tmem + t * 128, q_lo0 + t * (Cfg::kTileBytes >> 4), k_lo0 + stage * (Cfg::kTileBytes >> 4));
            mma_commit(bar_s_full + 8 * t);
            if (it.n_kv[t] == 1) mma_commit(bar_q_empty + 8 * t);
          }
          __syncwarp();
        }
        if (ok && elect_one_sync()) mma_commit(smem_u32(&sm.kv_empty[stage]));
        __syncwarp();
        const int n_own = FAN ? (it.P + 127) >> 7 : it.ld_tiles;
        ChildCur cc{0, 0, 0, 0};
        for (int j = 0; j < it.ld_tiles && ok; ++j) {
          int np = min(8, (it.kv_end - j * 128 + 15) >> 4);
          if (FAN && j >= n_own) {  // fan-out mode: a tile of a child's own keys
            if (j == n_own) child_first(a, it, cc); else child_next(a, it, cc);
            np = child_pages(cc);
          }
          const uint32_t v_stage = loads % Cfg::kStages;
          ok = mbar_wait(smem_u32(&sm.kv_full[v_stage]), (loads / Cfg::kStages) & 1, abortp);
          ++loads;
          if (!ok) break;
          const bool more = j + 1 < it.ld_tiles;
          uint32_t k_stage = 0;
          if (more) {
            k_stage = loads % Cfg::kStages;
            ok = mbar_wait(smem_u32(&sm.kv_full[k_stage]), (loads / Cfg::kStages) & 1, abortp);
            ++loads;
            if (!ok) break;
          }
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            if (j >= it.n_kv[t]) continue;
            ok = mbar_wait(bar_p_full + 8 * t, steps[t] & 1, abortp);
            ++steps[t];
            if (ok && j == 0) {  // the first PV overwrites O: the previous item's rows must have been read out
              ok = mbar_wait(bar_o_empty + 8 * t, (o_uses[t] & 1) ^ 1, abortp);
              ++o_uses[t];
            }
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one_sync()) {
              issue_pv_mmas<D>(tmem + 256 + t * 128, tmem + t * 128, v_lo0 + v_stage * (Cfg::kTileBytes >> 4), np, j == 0);
              if (j + 1 < it.n_kv[t]) {
                issue_s_mmas<D>(tmem + t * 128, q_lo0 + t * (Cfg::kTileBytes >> 4), k_lo0 + k_stage * (Cfg::kTileBytes >> 4));
                mma_commit(bar_s_full + 8 * t);
                if (j + 2 == it.n_kv[t]) mma_commit(bar_q_empty + 8 * t);  // that was the item's last S of this tile
              } else {
                mma_commit(bar_o_full + 8 * t);
              }
            }
            __syncwarp();
            if (t == 0 && j + 1 == it.n_kv[0] && has_nxt && nxt.n_kv[0] > 0 && nxt.ld_tiles > 0) {
              // Tile 0 is done with this item while tile 1 still has a step or more to go: if the next item's Q
              // tile and first K tile are already there, its first S is issued now instead of after tile 1.
              const uint32_t k0 = loads + (more ? 0 : 0) + 2 * (uint32_t)(it.ld_tiles - 1 - j) - (more ? 1 : 0);
              const uint32_t st0 = k0 % Cfg::kStages;
              // (A stage's barrier may only be asked about load k0 once the stage's previous load, k0 - kStages, has
              // been waited for: otherwise the parity test would be answered by the phase before that one.  In the
              // fan-out mode tile 1 can have several steps more than tile 0, which puts k0 that far ahead.)
              if (k0 < loads + Cfg::kStages &&
                  __all_sync(0xffffffffu, mbar_test_wait(bar_q_full, items_done[0] & 1) &&
                                              mbar_test_wait(smem_u32(&sm.kv_full[st0]), (k0 / Cfg::kStages) & 1))) {
                ++items_done[0];
                early0 = true;
                if (elect_one_sync()) {
                  issue_s_mmas<D>(tmem, q_lo0, k_lo0 + st0 * (Cfg::kTileBytes >> 4));
                  mma_commit(bar_s_full);
                  if (nxt.n_kv[0] == 1) mma_commit(bar_q_empty);
                }
                __syncwarp();
              }
            }
          }
          if (!ok) break;
          if (elect_one_sync()) {
            mma_commit(smem_u32(&sm.kv_empty[v_stage]));
            if (more) mma_commit(smem_u32(&sm.kv_empty[k_stage]));
          }
          __syncwarp();
        }
      }
      ok = __all_sync(0xffffffffu, ok);
    }
  } else if (warp == kWarpQ) {
    // =============================== Q loader ============================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    uint32_t fills[2] = {0, 0};  // tiles loaded so far per buffer (phase of q_empty)
    bool ok = true;
    Item it;
    for (int round = 0; ok && fetch_item<FAN>(a, sched_get(round), n_total, it); ++round) {
      sched_release(round);
      if (it.ld_tiles == 0) continue;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        if (it.n_kv[t] == 0 || !ok) continue;
        if (lane == 0) {
          // the buffer is free once the previous item's last S of this tile has been computed
          ok = mbar_wait(smem_u32(&sm.q_empty[t]), (fills[t] & 1) ^ 1, abortp);
          if (ok) {
            const uint32_t full = smem_u32(&sm.q_full[t]);
            mbar_arrive_expect_tx(full, Cfg::kTileBytes);
            const int tok0 = it.row0 + ((it.tp * 256 + t * 128) >> a.lg_group);
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h)
              tma_load_3d(smem_u32(sm.q[t]) + h * Cfg::kQHalfStride, &q_map, h * 64, it.kvh * a.group, tok0, full);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        ++fills[t];
      }
      // the next item's query tiles are asked into L2 now, a whole item ahead of their copy to shared memory
      Item nx;
      if (fetch_item<FAN>(a, sched_get(round + 1), n_total, nx) && nx.ld_tiles > 0 && lane == 0) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (nx.n_kv[t] == 0) continue;
          const int tok0 = nx.row0 + ((nx.tp * 256 + t * 128) >> a.lg_group);
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h) tma_prefetch_3d(&q_map, h * 64, nx.kvh * a.group, tok0);
        }
      }
    }
  } else if (warp == 15) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 24;");  // idle warp
  } else if (warp >= kWarpEpilogue) {
    // =============================== epilogue warpgroup ====================================
    // One thread per row (= TMEM lane), both tiles in turn: O / l -> bf16 -> global.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    const int w4 = warp & 3;
    const int m = w4 * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)(w4 * 32) << 16);
    const int G = a.group, lg = a.lg_group, Hq = a.n_q_heads;
    uint32_t done[2] = {0, 0};  // items finished per tile (phase of o_full / l_full, parity of inv_l)
    bool ok = true;
    Item it;
    for (int round = 0; ok && fetch_item<FAN>(a, sched_get(round), n_total, it); ++round) {
      sched_release(round);
      if (it.ld_tiles == 0) continue;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        if (it.n_kv[t] == 0 || !ok) continue;
        const int rg = it.tp * 256 + t * 128 + m;
        const int tok = rg >> lg;
        const bool valid = tok < it.E;
        const int64_t orow_idx = (int64_t)(it.row0 + tok) * Hq + it.kvh * G + (rg & (G - 1));
        ok = mbar_wait(smem_u32(&sm.l_full[t]), done[t] & 1, abortp);
        if (ok) ok = mbar_wait(smem_u32(&sm.o_full[t]), done[t] & 1, abortp);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const float inv = sm.inv_l[t][done[t] & 1][m];
        ++done[t];
        const uint32_t o_addr = lane_base + 256 + t * 128;
        // A row is 2 * D contiguous bytes, but a warp holds 32 different rows: 16-byte stores from the thread
        // that owns the row touch 32 cache lines per instruction and half a sector each.  Instead two
        // neighbouring lanes exchange 32-byte pieces, so that every store instruction writes 64 contiguous
        // bytes per lane pair, in 32-byte (whole sector) pieces.
        const int q = lane & 1;
        char* row_ptr = reinterpret_cast<char*>(a.out + orow_idx * D);
        // the neighbour's row and whether it exists
        const uint32_t n_lo = __shfl_xor_sync(0xffffffffu, (uint32_t)reinterpret_cast<uintptr_t>(row_ptr), 1);
        const uint32_t n_hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(reinterpret_cast<uintptr_t>(row_ptr) >> 32), 1);
        char* nb_ptr = reinterpret_cast<char*>(((uint64_t)n_hi << 32) | n_lo);
        const bool nb_valid = __shfl_xor_sync(0xffffffffu, (int)valid, 1) != 0;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t orow[32];
          tmem_ld32(o_addr + c * 32, orow);
          tmem_wait_ld();
          if (c == D / 32 - 1) {  // all of the row has been read: the next item's PV may overwrite O
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&sm.o_empty[t]));
          }
          uint32_t pk[16];  // columns [32c, 32c + 32) as bf16 pairs: two pieces of eight words
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float lo = __uint_as_float(orow[2 * i]) * inv, hi = __uint_as_float(orow[2 * i + 1]) * inv;
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[i]) : "f"(hi), "f"(lo));
          }
          // piece q of the own row is stored by this lane, piece 1-q by the neighbour, and vice versa
          uint32_t w[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint32_t give = q == 0 ? pk[8 + i] : pk[i];
            w[i] = __shfl_xor_sync(0xffffffffu, give, 1);
          }
          // first store: the even lane's row (its own piece 0, and piece 1 handed to the odd lane);
          // second store: the odd lane's row
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const bool own = (q == r);
            if (own ? valid : nb_valid) {
              char* dst = (own ? row_ptr : nb_ptr) + c * 64 + q * 32;
              uint32_t d[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) d[i] = own ? (r == 0 ? pk[i] : pk[8 + i]) : w[i];
              asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(d[0]), "r"(d[1]), "r"(d[2]), "r"(d[3]),
                           "r"(d[4]), "r"(d[5]), "r"(d[6]), "r"(d[7])
                           : "memory");
            }
          }
        }
      }
    }
  } else {
    // =============================== softmax warpgroups ======================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 192;");
    const int t = warp >> 2;                       // query tile of this warpgroup (warps 0-3: tile 0, 4-7: tile 1)
    const int w4 = warp & 3;                       // TMEM lane quarter this warp may access
    const int m = w4 * 32 + lane;                  // row inside the tile
    const uint32_t lane_base = tmem + ((uint32_t)(w4 * 32) << 16);
    const uint32_t s_addr = lane_base + t * 128, o_addr = lane_base + 256 + t * 128;
    const uint32_t bar_s_full = smem_u32(&sm.s_full[t]), bar_l_full = smem_u32(&sm.l_full[t]);
    const uint32_t bar_p_full = smem_u32(&sm.p_full[t]);
    const int G = a.group, lg = a.lg_group, Hq = a.n_q_heads;
    uint32_t steps = 0, items_done = 0;            // phase of s_full / p_full; items finished (parity of inv_l)
    bool ok = true;

    // The item records are read where they are needed (they stay in L1) instead of being carried in registers
    // through the softmax loop, which needs the registers for the score row.
    for (int round = 0; ok; ++round) {
      int n_t, limit;
      bool valid;
      int64_t orow_idx;
      // fan-out mode: the steps from n_own on walk the children's own keys; tok_s is this row's token among the
      // parent's stacked rows (-1: no such row) and (f_row0, f_child) start the walk
      int n_own, tok_s = -1, f_row0 = 0;
      ChildCur cc{0, 0, 0, 0};
      {
        Item it;
        const bool more_items = fetch_item<FAN>(a, sched_get(round), n_total, it);
        if (!more_items) break;
        sched_release(round);
        if (it.ld_tiles == 0) continue;
        n_t = it.n_kv[t];
        if (n_t == 0) continue;
        const int rg = it.tp * 256 + t * 128 + m;
        const int tok = rg >> lg;
        valid = tok < it.E;
        limit = valid && a.mode == 0 ? it.P + tok + 1 : it.kv_end;  // keys this row sees (rows past the end: any)
        orow_idx = (int64_t)(it.row0 + tok) * Hq + it.kvh * G + (rg & (G - 1));  // row of the LSE
        n_own = FAN ? (it.P + 127) >> 7 : n_t;
        if (FAN) {
          tok_s = valid ? tok : -1;
          f_row0 = it.row0;
          cc.c = it.c_first;
        }
      }
      float m_run = -INFINITY, l_run = 0.f;

      for (int j = 0; j < n_t; ++j) {
        ok = mbar_wait(bar_s_full, steps & 1, abortp);
        ++steps;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        // One trip to tensor memory: the row's 128 scores are read into registers, reduced to the row
        // maximum, exponentiated in place and written back as bf16 P.
        // vis: how many of the tile's 128 key columns this row sees (diagonal / last tile: keys past the row's
        // limit are hidden; fan-out mode: only the row's own child, up to the row's own token)
        int vis = limit - j * 128;
        if (FAN && j >= n_own) {
          if (j == n_own) {
            cc.jc = 0;
            child_load(a, f_row0, cc);
          } else if ((cc.jc + 1) * 128 < cc.len) {
            ++cc.jc;
          } else if (cc.c + 1 < a.fan.n_children) {
            ++cc.c;
            cc.jc = 0;
            child_load(a, f_row0, cc);
          }
          const int t_local = tok_s - cc.start;
          vis = (tok_s >= 0 && t_local >= 0 && t_local < cc.len) ? t_local + 1 - cc.jc * 128 : 0;
        }
        const bool ragged = vis < 128;
        uint32_t sr[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, sr[c]);
        tmem_wait_ld();
        if (ragged) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c * 32 + i >= vis) sr[c][i] = 0xff800000u;  // -inf by select: NaN-safe
        }
        if constexpr (OPT) {
          // The row maximum is needed only to keep the exponentials in range, and after the first tile it rarely
          // moves by much: the step first assumes that the maximum in use still serves (no search for the new one) and
          // looks at the row sum it gets.  A sum beyond kOptimisticSum (or not a number) in any row of the warp means
          // some score exceeds the maximum in use by up to 16 or more binades: the warp then takes the step again
          // with the exact maximum.  Both ways are a deterministic function of the inputs.
          // exponentials of the row against a given maximum: P (bf16) goes to tensor memory, the row sum comes back
          auto exp_pass = [&](float m_use) -> float {
            const float neg_m = (m_use == -INFINITY) ? 0.f : -m_use;
            const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nm2 = make_float2(neg_m, neg_m);
            float2 ls2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t pk[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[c][2 * i]), __uint_as_float(sr[c][2 * i + 1])), sc2, nm2);
                float2 pr;
                asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(pr.x) : "f"(x.x));
                asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(pr.y) : "f"(x.y));
                ls2[i & 1] = __fadd2_rn(ls2[i & 1], pr);
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[i]) : "f"(pr.y), "f"(pr.x));
              }
              // P (bf16 pairs) goes over score columns [16c, 16c+16): all scores are in registers by now
              tmem_st16(s_addr + c * 16, pk);
            }
            return (ls2[0].x + ls2[0].y) + (ls2[1].x + ls2[1].y);
          };
          // the exact way: row maximum of the tile, and O and the row sum brought to it if it has grown by much
          auto exact_max = [&]() {
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int i = 0; i < 32; i += 2)
                mx4[c] = fmax3(mx4[c], __uint_as_float(sr[c][i]), __uint_as_float(sr[c][i + 1]));
            const float mx = fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * a.scale_log2;
            const float m_new = fmaxf(m_run, mx);
            const bool grow = m_new > m_run + kRescaleThreshold;  // also true on the first tile (m_run = -inf)
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
              // O holds sums scaled by 2^-m_run: bring them to the new maximum (the PV that produced them
              // has finished: the S this step waited for was committed after it)
              const float alpha = grow ? exp2f(m_run - m_new) : 1.f;
              l_run *= alpha;
#pragma unroll 1
              for (int c = 0; c < D / 16; ++c) {
                uint32_t orow[16];
                tmem_ld16(o_addr + c * 16, orow);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * alpha);
                tmem_st16(o_addr + c * 16, orow);
              }
            }
            if (grow) m_run = m_new;
          };
          const bool first = j == 0 || __any_sync(0xffffffffu, m_run == -INFINITY);
          if (first) exact_max();
          float row_sum = exp_pass(m_run);
          if (!first && !__all_sync(0xffffffffu, row_sum <= kOptimisticSum)) {  // rare: the maximum has moved a long way
            exact_max();
            row_sum = exp_pass(m_run);
          }
          l_run += row_sum;
        } else {
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; i += 2)
              mx4[c] = fmax3(mx4[c], __uint_as_float(sr[c][i]), __uint_as_float(sr[c][i + 1]));
          const float mx = fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * a.scale_log2;
          const float m_new = fmaxf(m_run, mx);
          const bool grow = m_new > m_run + kRescaleThreshold;  // also true on the first tile (m_run = -inf)
          const float m_use = grow ? m_new : m_run;
          if (j > 0 && __any_sync(0xffffffffu, grow)) {
            // O holds sums scaled by 2^-m_run: bring them to the new maximum (the PV that produced them
            // has finished: the S this step waited for was committed after it)
            const float alpha = grow ? exp2f(m_run - m_new) : 1.f;
            l_run *= alpha;
#pragma unroll 1
            for (int c = 0; c < D / 16; ++c) {
              uint32_t orow[16];
              tmem_ld16(o_addr + c * 16, orow);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * alpha);
              tmem_st16(o_addr + c * 16, orow);
            }
          }
          m_run = m_use;
          const float neg_m = (m_use == -INFINITY) ? 0.f : -m_use;
          const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nm2 = make_float2(neg_m, neg_m);
          float2 ls2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[c][2 * i]), __uint_as_float(sr[c][2 * i + 1])), sc2, nm2);
              float2 pr;
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(pr.x) : "f"(x.x));
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(pr.y) : "f"(x.y));
              ls2[i & 1] = __fadd2_rn(ls2[i & 1], pr);
              asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[i]) : "f"(pr.y), "f"(pr.x));
            }
            // P (bf16 pairs) goes over score columns [16c, 16c+16): all scores are in registers by now
            tmem_st16(s_addr + c * 16, pk);
          }
          l_run += (ls2[0].x + ls2[0].y) + (ls2[1].x + ls2[1].y);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(bar_p_full);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      // ---- hand the row to the epilogue warps: 1 / row sum through shared memory; the LSE is written here.
      // The softmax of an item needs only S, so with one-step items it could finish two items before the
      // epilogue warps have looked at the first: a barrier must not get two phases ahead of its waiters, so
      // this hand-over waits until the previous item's rows of this tile have been read out.
      if (items_done > 0) {
        ok = mbar_wait(smem_u32(&sm.o_empty[t]), (items_done - 1) & 1, abortp);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      sm.inv_l[t][items_done & 1][m] = 1.f / l_run;
      mbar_arrive(bar_l_full);
      ++items_done;
      if (valid) a.lse[orow_idx] = (m_run + log2f(l_run)) * 0.6931471805599453f;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && sm.abort_flag != 0) report(a.pool.status, KV_ERR_TIMEOUT);
  if (warp == kWarpProducer) tmem_dealloc(tmem, 512);
  // The last CTA to finish puts the work counter back where the plan left it, so that the same plan can serve
  // another launch (a model runs every layer of a step over the same lengths).  a.next_item + 1 counts the CTAs done.
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(a.next_item + 1, 1) == (int)gridDim.x - 1) {
      a.next_item[0] = (int)gridDim.x;
      a.next_item[1] = 0;
      __threadfence();
    }
  }
}

// ------------------------------------------------------------------------------------------
static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static int64_t item_capacity(int n_q_heads, int n_kv_heads, int batch, int total_q) {
  const int G = n_q_heads / n_kv_heads;
  return (int64_t)total_q * G / 256 + batch + 1;
}

size_t extend_tc_workspace_bytes(int n_q_heads, int head_dim, int batch, int total_q, int max_total_len) {
  (void)head_dim; (void)max_total_len;
  if (batch <= 0 || total_q <= 0) return 0;
  // n_kv_heads is not known here: G <= 8 bounds the list
  return 256 + align256(2 * sizeof(int4) * (size_t)((int64_t)total_q * 8 / 256 + batch + 1));
}

bool extend_tc_supported(const kv_pool_t* p, int n_q_heads) {
  if (p->head_dim != 64 && p->head_dim != 128) return false;
  const int g = n_q_heads / p->n_kv_heads;
  return g == 1 || g == 2 || g == 4 || g == 8;
}

// Tensor map over Q [total_q][Hq][D] (bf16): a box is one 64-dim half of a query tile, that is 128/G tokens x the
// G heads of one KV head x 64 dims, written to shared memory with the 128-byte swizzle the MMA expects.  Rows past
// the end of Q read as zeros.
static kv_status_t make_q_map(CUtensorMap* map, const void* q, int total_q, int n_q_heads, int head_dim, int group) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn encode = nullptr;
  if (encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    KV_CUDA_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return KV_ERR_CUDA;
    encode = reinterpret_cast<encode_fn>(fn);
  }
  const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_q_heads, (cuuint64_t)total_q};
  const cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)n_q_heads * head_dim * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)group, (cuuint32_t)(128 / group)};
  const cuuint32_t elem_strides[3] = {1, 1, 1};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, elem_strides,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? KV_OK : KV_ERR_INVALID;
}

// One persistent CTA per SM, fewer if there are fewer items or the caller caps the kernel.
static kv_status_t tc_grid(const kv_pool_t* p, int n_items_bound, int cta_cap, int* grid_out) {
  const int sm_count = sm_count_of(p->device);
  int grid = n_items_bound < sm_count ? (n_items_bound < 1 ? 1 : n_items_bound) : sm_count;
  if (cta_cap > 0 && grid > cta_cap) grid = cta_cap;  // leave the other SMs to work that runs beside this kernel (< 0: no
                                                      // cap, and the kernel is launched without the early start)
  *grid_out = grid;
  return KV_OK;
}

template <int D, bool OPT, bool FAN>
static kv_status_t launch_tc(const TcArgs& a, const CUtensorMap& q_map, int grid, int device, bool early_start, cudaStream_t st) {
  const size_t smem = sizeof(TcSmem<D>);
  static std::atomic<bool> configured[kMaxDevices];  // the attribute belongs to the function on one device
  if (device < 0 || device >= kMaxDevices) return KV_ERR_INVALID;
  if (!configured[device].load(std::memory_order_acquire)) {
    KV_CUDA_OK(cudaFuncSetAttribute(attn_extend_tc_kernel<D, OPT, FAN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured[device].store(true, std::memory_order_release);
  }
  // early_start: launched so that it may start while the plan kernel in front of it still runs (it waits for it
  // inside).  Not wanted when another kernel is meant to take the SMs first (the mixed step's decode kernel): CTAs
  // that sit on an SM waiting for the plan keep that kernel's blocks away.
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start ? 1 : 0;
  KV_CUDA_OK(cudaLaunchKernelEx(&cfg, attn_extend_tc_kernel<D, OPT, FAN>, a, q_map));
  count_launch();
  return KV_OK;
}

kv_status_t launch_extend_tc(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                             int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                             int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, int cta_cap, int mode, const FanArgs* fan,
                             const AppendArgs* app, int phase, cudaStream_t st) {
  // phase 0: plan (with the suffix append, if any) and attention; 1: the plan only; 2: attention over the plan that a
  // phase-1 call with the same arguments left in the workspace
  const size_t need = extend_tc_workspace_bytes(n_q_heads, p->head_dim, batch, total_q, max_total_len);
  if (workspace == nullptr || workspace_bytes < need) return KV_ERR_WORKSPACE;
  const int G = n_q_heads / p->n_kv_heads;
  // Q is read through a tensor map (16-byte base), O is written with 32-byte stores
  if ((reinterpret_cast<uintptr_t>(q) & 15) != 0 || (reinterpret_cast<uintptr_t>(out) & 31) != 0) return KV_ERR_INVALID;
  CUtensorMap q_map;
  if (phase != 1) {
    const kv_status_t ms = make_q_map(&q_map, q, total_q, n_q_heads, p->head_dim, G);
    if (ms != KV_OK) return ms;
  }
  int lg = 0;
  while ((1 << lg) < G) ++lg;
  int* n_items = reinterpret_cast<int*>(workspace);
  int4* items = reinterpret_cast<int4*>(reinterpret_cast<char*>(workspace) + 256);
  const int64_t capacity = item_capacity(n_q_heads, p->n_kv_heads, batch, total_q);
  const int max_tp = (int)(((int64_t)max_extend_len * G + 255) / 256);
  const int max_steps = 2 * ((max_total_len + 127) / 128);
  const int64_t bound = (int64_t)batch * max_tp * p->n_kv_heads;
  const int n_bound = bound > (1 << 30) ? (1 << 30) : (int)bound;
  int grid = 1;
  {
    const kv_status_t gs = tc_grid(p, n_bound, cta_cap, &grid);
    if (gs != KV_OK) return gs;
  }
  // about a hundred items per group (measured on the 8B extend, long-document and fan-out shapes: fewer and larger
  // groups lose the L2 reuse, one sequence per group loses balance when a sequence has few items)
  // (a batch with fewer than a dozen items per SM is left in pure cost order: there the balance matters more)
  int groups = n_bound >= 12 * sm_count_of(p->device) ? n_bound / 96 : 1;
  groups = groups < 1 ? 1 : groups;
  groups = groups > batch ? batch : groups;
  groups = groups > kPlanBuckets / 16 ? kPlanBuckets / 16 : groups;
  const PlanArgs pa{prefix_lens, extend_lens, cu_q, batch, max_tp, lg, max_steps, (int)capacity, max_pages, mode,
                    fan != nullptr ? *fan : FanArgs{}, groups, p->d_status, items, n_items, n_items + 1, grid};
  if (phase == 2) {
    // the plan is in the workspace already
  } else if (app != nullptr && app->total_new > 0) {
    // plan block + append blocks (32 warps each, one warp per token, all blocks resident at once)
    const int64_t want = ((int64_t)app->total_new + 31) / 32;
    const int64_t cap = 2 * (int64_t)sm_count_of(p->device) - 1;
    const int blocks = (int)(want < cap ? want : cap);
    extend_prologue_kernel<<<1 + blocks, 1024, 0, st>>>(pa, p->view(), *app);
  } else {
    extend_tc_plan_kernel<<<1, 1024, 0, st>>>(pa);
  }
  if (phase != 2) {
    count_launch();
    KV_CUDA_OK(cudaGetLastError());
  }
  if (phase == 1) return KV_OK;

  TcArgs a{};
  a.pool = p->view();
  a.q = (const __nv_bfloat16*)q;
  a.cu_q = cu_q;
  a.block_tables = block_tables;
  a.max_pages = max_pages;
  a.prefix_lens = prefix_lens;
  a.extend_lens = extend_lens;
  a.batch = batch;
  a.n_q_heads = n_q_heads;
  a.group = G;
  a.lg_group = lg;
  a.mode = mode;
  a.fan = fan != nullptr ? *fan : FanArgs{};
  a.scale_log2 = scale * 1.4426950408889634f;
  a.out = (__nv_bfloat16*)out;
  a.lse = lse;
  a.items = items;
  a.n_items = n_items;
  a.next_item = n_items + 1;
  // Skipping the search for the row maximum pays where items have many KV steps (measured: +2 % on the
  // long-document shapes, -1 % on the 8B extend batch whose items have a dozen steps)
  const bool opt = max_total_len >= kOptimisticMinLen;
  const bool early = cta_cap >= 0;
  auto go = [&](auto d, auto o, auto f) {
    return launch_tc<decltype(d)::value, decltype(o)::value, decltype(f)::value>(a, q_map, grid, p->device, early, st);
  };
  using I128 = std::integral_constant<int, 128>;
  using I64 = std::integral_constant<int, 64>;
  const bool fan_mode = mode == 2;
  if (p->head_dim == 128) {
    if (fan_mode) return opt ? go(I128{}, std::true_type{}, std::true_type{}) : go(I128{}, std::false_type{}, std::true_type{});
    return opt ? go(I128{}, std::true_type{}, std::false_type{}) : go(I128{}, std::false_type{}, std::false_type{});
  }
  if (fan_mode) return opt ? go(I64{}, std::true_type{}, std::true_type{}) : go(I64{}, std::false_type{}, std::true_type{});
  return opt ? go(I64{}, std::true_type{}, std::false_type{}) : go(I64{}, std::false_type{}, std::false_type{});
}

}  // namespace kvattn
