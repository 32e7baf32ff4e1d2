// kv_append's data movement as a device function, shared by the stand-alone append kernel and by the prologue kernel
// of the fused append + extend call.
#pragma once

#include "common.cuh"

namespace kvattn {

struct AppendArgs {
  const uint4* k_new;   // [total_new][n_kv_heads][head_dim] bf16, as 16-byte chunks
  const uint4* v_new;
  const int* cu_new;    // [n_segments + 1]
  const int* start_pos; // [n_segments]
  const int* seg_row;   // [n_segments] or nullptr (segment s writes block-table row s)
  const int* block_tables;
  int max_pages, n_segments, total_new;
};

// One warp moves one token: `warp_index` of `n_warps` warps take the tokens warp_index, warp_index + n_warps, ...
// kMaxPerLane: 16-byte chunks of K (and of V) a lane holds at once, i.e. 32 * kMaxPerLane chunks of a token per pass.
template <int kMaxPerLane>
__device__ __forceinline__ void append_tokens(const PoolView& pool, const AppendArgs& a, int warp_index, int n_warps) {
  const uint4* __restrict__ k_new = a.k_new;
  const uint4* __restrict__ v_new = a.v_new;
  const int* __restrict__ cu_new = a.cu_new;
  const int* __restrict__ start_pos = a.start_pos;
  const int* __restrict__ seg_row = a.seg_row;
  const int* __restrict__ block_tables = a.block_tables;
  const int max_pages = a.max_pages, n_segments = a.n_segments, total_new = a.total_new;
  // One warp per token: the token's segment, position and page are looked up once, then the lanes copy the
  // token's 16-byte chunks (n_kv_heads * head_dim / 8 of them), all loads of a token in flight before its stores.
  const int chunks_per_row = pool.head_dim >> 3;               // 16-byte chunks per (token, head)
  const int chunks_per_token = pool.n_kv_heads * chunks_per_row;
  const size_t blk = block_bytes(pool.head_dim);
  const int lane = threadIdx.x & 31;
  const int warps = n_warps;
  for (int token = warp_index; token < total_new; token += warps) {
    // The token's first chunks are asked for before anything else: where they go is found meanwhile (the loads do not
    // depend on it, and a token's warp otherwise spends its time on a chain of small dependent loads).
    const uint4* ksrc = k_new + (int64_t)token * chunks_per_token;
    const uint4* vsrc = v_new + (int64_t)token * chunks_per_token;
    uint4 kk[kMaxPerLane], vv[kMaxPerLane];
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      const int c = i * 32 + lane;
      if (c < chunks_per_token) {
        kk[i] = __ldg(ksrc + c);
        vv[i] = __ldg(vsrc + c);
      }
    }
    // segment of this token: last s with cu_new[s] <= token.  The lanes probe 32 evenly spaced entries at a time, so
    // the search is one dependent load per factor of 32 in the number of segments instead of one per factor of 2
    // (the chain of dependent loads is what a token's warp spends its time on).
    int lo = 0, span = n_segments;
    while (span > 1) {
      const int step = (span + 31) >> 5;
      const int idx = lo + lane * step;
      const bool le = idx < lo + span && __ldg(cu_new + idx) <= token;
      const int k = __popc(__ballot_sync(0xffffffffu, le)) - 1;   // >= 0: cu_new[lo] <= token
      const int end = lo + span;
      lo += max(k, 0) * step;
      span = min(step, end - lo);
    }
    const int seg = lo;
    const int seg_begin = __ldg(cu_new + seg), seg_end = __ldg(cu_new + seg + 1);
    if (token >= seg_end) continue;                            // cu_new not covering this row: skip
    const int pos = __ldg(start_pos + seg) + (token - seg_begin);
    const int row = seg_row ? __ldg(seg_row + seg) : seg;
    const int blk_idx = pos >> 4;
    if (pos < 0 || blk_idx >= max_pages) { report(pool.status, KV_ERR_BOUNDS); continue; }
    const int page = __ldg(block_tables + (int64_t)row * max_pages + blk_idx);
    if (page < 0 || page >= pool.num_pages) { report(pool.status, KV_ERR_BOUNDS); continue; }
    const size_t page_off = (size_t)page * pool.n_kv_heads * blk;
    const bool last = token + 1 == seg_end;
    for (int c0 = 0; c0 < chunks_per_token; c0 += 32 * kMaxPerLane) {
      if (c0 > 0) {  // (the first pass's chunks are in flight already)
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i) {
          const int c = c0 + i * 32 + lane;
          if (c < chunks_per_token) {
            kk[i] = __ldg(ksrc + c);
            vv[i] = __ldg(vsrc + c);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kMaxPerLane; ++i) {
        const int c = c0 + i * 32 + lane;
        if (c < chunks_per_token) {
          const int head = c / chunks_per_row, dchunk = c - head * chunks_per_row;
          const size_t blk_off = page_off + (size_t)head * blk;
          const size_t off = blk_off + chunk_offset_bytes(pos & 15, dchunk, pool.head_dim);
          *reinterpret_cast<uint4*>(reinterpret_cast<char*>(pool.k) + off) = kk[i];
          *reinterpret_cast<uint4*>(reinterpret_cast<char*>(pool.v) + off) = vv[i];
          // The segment's last token also clears the slots behind it in its page.  Slots past a sequence's
          // end therefore never hold NaN/Inf bit patterns, which the tensor-core kernel relies on: it
          // multiplies those V rows by probabilities that are exactly 0.
          if (last) {
            const uint4 z = make_uint4(0, 0, 0, 0);
            for (int slot = (pos & 15) + 1; slot < kPageSize; ++slot) {
              const size_t o2 = blk_off + chunk_offset_bytes(slot, dchunk, pool.head_dim);
              *reinterpret_cast<uint4*>(reinterpret_cast<char*>(pool.k) + o2) = z;
              *reinterpret_cast<uint4*>(reinterpret_cast<char*>(pool.v) + o2) = z;
            }
          }
        }
      }
    }
  }
}

}  // namespace kvattn
