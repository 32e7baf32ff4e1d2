// Small-tile paged attention: the HBM-bound path.
//
// One warp owns one work item = (sequence, KV head, tile of 8 query rows, chunk of the KV range)
// and streams that chunk's pages straight from HBM into registers with coalesced 16-byte loads.
// The 8 query rows are the G query heads that share the KV head (decode: one token; extend: 8/G
// consecutive suffix tokens).  Scores are computed as S^T = K Q^T with tokens in the M dimension
// of mma.sync.m16n8k16 (one 16-token page per MMA row block, the 8 query rows in N), so the K
// fragments are exactly the 16-byte chunks as loaded and no padding of the query rows to 16 is
// needed; O^T = V^T P^T uses the same trick with byte permutes pairing two tokens.  The running
// maximum is shared with three shuffles per page, the row sum is reduced once at the end.
// Partial results of the chunks are merged by combine_kernel with the log-sum-exp rule.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace kvattn {

constexpr int kChunkPages = 32;                       // pages per batch of block-table entries (one per lane)
constexpr int kDecodeChunkTokens = kChunkPages * 16 * 2;  // split size of decode: a function of nothing but this constant

struct SmallArgs {
  PoolView pool;
  const __nv_bfloat16* q;  // [rows][Hq][D]
  const int* block_tables;
  int max_pages;
  const int* len_a;  // decode: ctx_lens; extend: prefix_lens
  const int* len_b;  // extend: extend_lens
  const int* cu_q;   // extend: row offsets
  int n_q_heads, group, batch;
  int max_row_tiles;  // decode: 1; extend: ceil(max_extend_len / (8/G))
  int max_chunks;     // KV chunks per row (1 when writing the result directly)
  int chunk_tokens;   // tokens per chunk (multiple of 512)
  float scale_log2;   // scale * log2(e)
  float* part_o;      // [(row*Hq + head)*max_chunks + chunk][D], normalised within the chunk
  float* part_lse;    // same index; log2-domain log-sum-exp of the chunk
  __nv_bfloat16* out;  // direct mode
  float* lse;          // direct mode
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

template <int D>
struct PageRegs {
  uint4 k[2][D / 32];     // [token group][j]   : slot 8g + r, chunk 4j + c
  uint4 v[2][2][D / 64];  // [token group][parity][u]: slot 8g + 2c + parity, chunk 8u + r
};

template <int D>
__device__ __forceinline__ void load_page(PageRegs<D>& pr, const char* kblk, const char* vblk, int r, int c) {
#pragma unroll
  for (int g = 0; g < 2; ++g) {
#pragma unroll
    for (int j = 0; j < D / 32; ++j) {
      const int ch = 4 * j + c;
      pr.k[g][j] = ldg_stream(kblk + g * (D * 16) + (ch >> 3) * 1024 + r * 128 + (((ch & 7) ^ r) << 4));
    }
  }
#pragma unroll
  for (int g = 0; g < 2; ++g) {
#pragma unroll
    for (int par = 0; par < 2; ++par) {
      const int row = 2 * c + par;
#pragma unroll
      for (int u = 0; u < D / 64; ++u)
        pr.v[g][par][u] = ldg_stream(vblk + g * (D * 16) + u * 1024 + row * 128 + ((r ^ row) << 4));
    }
  }
}

// ---- ring variant (decode): pages come through shared memory -----------------------------------------------
// The register-streaming loader above keeps one page per warp in flight, which is what the registers allow; a warp
// then waits out most of every page's latency, and only all SMs together reach the memory's bandwidth.  In the ring
// variant every warp owns kRingStages page slots in shared memory that it fills with bulk copies (one 16-token K block
// and one V block per slot, exactly as they lie in the pool), so kRingStages - 1 pages per warp are in flight while one
// is consumed, whatever the register budget: fewer SMs saturate HBM, which leaves the others to the tensor-core
// kernel in a mixed step.  The arithmetic on a page is the same code, so the results are the same bits.
constexpr int kRingWarps = 8;
constexpr int kRingStages = 3;

template <int D>
constexpr int ring_smem_bytes() { return kRingWarps * kRingStages * 2 * 16 * D * 2 + kRingWarps * kRingStages * 8 + 16; }

// Fragments of one page from a shared-memory slot (K block, then V block).  Within a quarter warp the K loads of the
// lanes with an odd row take the other 64-byte half first (j ^ 1), so that the eight lanes touch eight different
// 16-byte bank groups; the registers are swapped back afterwards.
template <int D>
__device__ __forceinline__ void load_page_smem(PageRegs<D>& pr, uint32_t slot, int r, int c) {
  auto lds = [](uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
  };
  const int flip = r & 1;
#pragma unroll
  for (int g = 0; g < 2; ++g) {
#pragma unroll
    for (int j = 0; j < D / 32; ++j) {
      const int ch = 4 * (j ^ flip) + c;
      pr.k[g][j] = lds(slot + g * (D * 16) + (ch >> 3) * 1024 + r * 128 + (((ch & 7) ^ r) << 4));
    }
    if (flip) {
#pragma unroll
      for (int j = 0; j < D / 32; j += 2) {
        const uint4 t = pr.k[g][j];
        pr.k[g][j] = pr.k[g][j + 1];
        pr.k[g][j + 1] = t;
      }
    }
  }
  const uint32_t vslot = slot + 16 * D * 2;
#pragma unroll
  for (int g = 0; g < 2; ++g) {
#pragma unroll
    for (int par = 0; par < 2; ++par) {
      const int row = 2 * c + par;
#pragma unroll
      for (int u = 0; u < D / 64; ++u)
        pr.v[g][par][u] = lds(vslot + g * (D * 16) + u * 1024 + row * 128 + ((r ^ row) << 4));
    }
  }
}

template <int D, bool EXTEND, bool DIRECT, bool RING = false>
__global__ void __launch_bounds__(RING ? kRingWarps * 32 : 256, 1) attn_small_kernel(SmallArgs a, int64_t total_items) {
  // the kernel queued behind this one (the combine) may be launched while this one runs; it waits for it inside
  ptx::launch_dependents();
  constexpr int kWarps = RING ? kRingWarps : 8;
  constexpr int kBatchPages = RING ? 2 * kChunkPages : kChunkPages;  // block-table entries held per lane pair / lane
  extern __shared__ __align__(1024) unsigned char ring_raw[];
  unsigned long long* ring_bars = reinterpret_cast<unsigned long long*>(ring_raw + kRingWarps * kRingStages * 2 * 16 * D * 2);
  int* ring_abort = reinterpret_cast<int*>(ring_bars + kRingWarps * kRingStages);
  if (RING) {
    if (threadIdx.x == 0) *ring_abort = 0;
    if ((threadIdx.x & 31) == 0)
      for (int s = 0; s < kRingStages; ++s) ptx::mbar_init(ptx::smem_u32(&ring_bars[(threadIdx.x >> 5) * kRingStages + s]), 1);
    ptx::fence_mbar_init();
    __syncthreads();
  }
  constexpr int NJ = D / 32;  // K chunk loads per token row per lane
  constexpr int NU = D / 64;  // 64-dim halves
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int64_t item = (int64_t)blockIdx.x * kWarps + warp;
  if (item >= total_items) return;

  const int Hkv = a.pool.n_kv_heads, G = a.group, Hq = a.n_q_heads;
  int chunk, rt, kvh, seq;
  if (EXTEND) {
    chunk = (int)(item % a.max_chunks);
    int64_t rest = item / a.max_chunks;
    rt = (int)(rest % a.max_row_tiles);
    rest /= a.max_row_tiles;
    kvh = (int)(rest % Hkv);
    seq = (int)(rest / Hkv);
  } else {
    // Decode: the chunk index is the slowest dimension.  Blocks start in index order, so every sequence's first
    // (full) chunks go first and the last, partly filled or empty chunks of the longer sequences go last: the
    // kernel's tail, when the SMs run out of work one by one, is made of the smallest pieces.
    const int64_t per_chunk = (int64_t)a.batch * Hkv;
    chunk = (int)(item / per_chunk);
    const int rest = (int)(item % per_chunk);
    rt = 0;
    kvh = rest % Hkv;
    seq = rest / Hkv;
  }

  int P = 0, E = 1, L, row0;
  if (EXTEND) {
    P = __ldg(a.len_a + seq);
    E = __ldg(a.len_b + seq);
    L = P + E;
    row0 = __ldg(a.cu_q + seq);
  } else {
    L = __ldg(a.len_a + seq);
    P = L - 1;
    row0 = seq;
  }
  const int tpt = EXTEND ? 8 / G : 1;  // query tokens per tile
  // more suffix tokens than the host-side bound the grid covers: the rows beyond it would never be written
  if (EXTEND && rt == 0 && lane == 0 && (int64_t)E > (int64_t)a.max_row_tiles * tpt) report(a.pool.status, KV_ERR_BOUNDS);
  const int t_first = rt * tpt;
  if (t_first >= E || L <= 0 || P < 0) return;
  if (L > a.max_pages * kPageSize) { report(a.pool.status, KV_ERR_BOUNDS); return; }
  const int t_last = min(E, t_first + tpt) - 1;
  const int tile_limit = P + t_last + 1;  // keys visible to the tile's last token
  // the host-side bounds (max_ctx_len / max_total_len) were too small for this sequence
  if ((int64_t)tile_limit > (int64_t)a.max_chunks * a.chunk_tokens) { report(a.pool.status, KV_ERR_BOUNDS); return; }
  const int chunk_begin = chunk * a.chunk_tokens;
  if (chunk_begin >= tile_limit) return;
  const int chunk_end = min(chunk_begin + a.chunk_tokens, tile_limit);

  // the two query rows whose scores this lane holds (n = 2c, 2c+1) and the row it loads (n = r)
  auto row_token = [&](int n) { return EXTEND ? t_first + n / G : 0; };
  auto row_head = [&](int n) { return kvh * G + (EXTEND ? n % G : n); };
  auto row_valid = [&](int n) { return EXTEND ? (t_first + n / G) < E : n < G; };
  const int n0 = 2 * c, n1 = 2 * c + 1;
  const bool valid0 = row_valid(n0), valid1 = row_valid(n1);
  const int limit0 = valid0 ? P + row_token(n0) + 1 : 0;
  const int limit1 = valid1 ? P + row_token(n1) + 1 : 0;

  uint4 qf[NJ];
  {
    const bool vr = row_valid(r);
    const __nv_bfloat16* qp = a.q + ((int64_t)(row0 + row_token(r)) * Hq + row_head(r)) * D;
#pragma unroll
    for (int j = 0; j < NJ; ++j)
      qf[j] = vr ? __ldg(reinterpret_cast<const uint4*>(qp) + 4 * j + c) : make_uint4(0, 0, 0, 0);
  }

  float acc[NU][4][4];
#pragma unroll
  for (int u = 0; u < NU; ++u)
#pragma unroll
    for (int w = 0; w < 4; ++w)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[u][w][i] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  const size_t blk = block_bytes(D);
  const char* kbase = reinterpret_cast<const char*>(a.pool.k) + (size_t)kvh * blk;
  const char* vbase = reinterpret_cast<const char*>(a.pool.v) + (size_t)kvh * blk;
  const size_t page_stride = (size_t)Hkv * blk;
  const int* bt_row = a.block_tables + (int64_t)seq * a.max_pages;

  const int first_page = chunk_begin >> 4;
  const int n_pages = (chunk_end - chunk_begin + 15) >> 4;

  const uint64_t ring_policy = RING ? ptx::l2_evict_first_policy() : 0;
  uint32_t ring_issued = 0, ring_used = 0;  // ring variant: pages asked for / consumed so far (slot and phase follow)
  for (int pb = 0; pb < n_pages; pb += kBatchPages) {
    const int np = min(kBatchPages, n_pages - pb);
    int my_page = 0, my_page_hi = 0;
    auto table_entry = [&](int idx) {
      int pg = 0;
      if (idx < np) {
        const int b = first_page + pb + idx;
        pg = (b < a.max_pages) ? __ldg(bt_row + b) : -1;
        if ((unsigned)pg >= (unsigned)a.pool.num_pages) {
          report(a.pool.status, KV_ERR_BOUNDS);
          pg = 0;  // stay inside the pool; the result of this row is flagged, not trusted
        }
      }
      return pg;
    };
    my_page = table_entry(lane);
    if (RING) my_page_hi = table_entry(lane + 32);
    // one page of work on the registers in `pr`
    auto process = [&](PageRegs<D>& pr, int p) {
      const int tok0 = chunk_begin + ((pb + p) << 4);  // first token of this page

      // ---- S^T[16 tokens][8 rows] = K Q^T
      float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        mma_bf16_16816(s, pr.k[0][j].x, pr.k[1][j].x, pr.k[0][j].y, pr.k[1][j].y, qf[j].x, qf[j].y);
        mma_bf16_16816(s, pr.k[0][j].z, pr.k[1][j].z, pr.k[0][j].w, pr.k[1][j].w, qf[j].z, qf[j].w);
      }
      // s[0]: (token r, row n0)  s[1]: (token r, n1)  s[2]: (token r+8, n0)  s[3]: (token r+8, n1)
      const int ta = tok0 + r, tb = tok0 + r + 8;
      const float s00 = ta < limit0 ? s[0] * a.scale_log2 : -INFINITY;
      const float s01 = ta < limit1 ? s[1] * a.scale_log2 : -INFINITY;
      const float s10 = tb < limit0 ? s[2] * a.scale_log2 : -INFINITY;
      const float s11 = tb < limit1 ? s[3] * a.scale_log2 : -INFINITY;
      float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
      }
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
      const float al0 = fast_exp2(m0 - mu0), al1 = fast_exp2(m1 - mu1);
      const float p00 = fast_exp2(s00 - mu0), p01 = fast_exp2(s01 - mu1);
      const float p10 = fast_exp2(s10 - mu0), p11 = fast_exp2(s11 - mu1);
      l0 = l0 * al0 + (p00 + p10);
      l1 = l1 * al1 + (p01 + p11);
      const bool changed = (mn0 != m0) || (mn1 != m1);
      m0 = mn0;
      m1 = mn1;
      if (__any_sync(0xffffffffu, changed)) {
#pragma unroll
        for (int u = 0; u < NU; ++u)
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            acc[u][w][0] *= al0; acc[u][w][2] *= al0;
            acc[u][w][1] *= al1; acc[u][w][3] *= al1;
          }
      }
      // P^T fragments: transpose the 8x8 (token, row) tiles held as packed bf16 pairs
      const uint32_t pt0 = movmatrix_trans(pack_bf16x2(p00, p01));
      const uint32_t pt1 = movmatrix_trans(pack_bf16x2(p10, p11));

      // stale slots past the sequence end may hold NaN/Inf bits: select them away (0 * NaN != 0)
      if (tok0 + 16 > L) {
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
          for (int par = 0; par < 2; ++par)
            if (tok0 + 8 * g + 2 * c + par >= L) {
#pragma unroll
              for (int u = 0; u < NU; ++u) pr.v[g][par][u] = make_uint4(0, 0, 0, 0);
            }
      }
      // ---- O^T[D][8 rows] += V^T P^T
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        const uint4 va = pr.v[0][0][u], vb = pr.v[0][1][u], vc = pr.v[1][0][u], vd = pr.v[1][1][u];
        const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
        const uint32_t wc[4] = {vc.x, vc.y, vc.z, vc.w}, wd[4] = {vd.x, vd.y, vd.z, vd.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          mma_bf16_16816(acc[u][w], __byte_perm(wa[w], wb[w], 0x5410), __byte_perm(wa[w], wb[w], 0x7632),
                         __byte_perm(wc[w], wd[w], 0x5410), __byte_perm(wc[w], wd[w], 0x7632), pt0, pt1);
        }
      }
    };
    auto fetch = [&](PageRegs<D>& pr, int p) {
      const int pg = __shfl_sync(0xffffffffu, my_page, p);
      load_page<D>(pr, kbase + (size_t)pg * page_stride, vbase + (size_t)pg * page_stride, r, c);
    };

    if constexpr (RING) {
      const uint32_t slots = ptx::smem_u32(ring_raw) + warp * (kRingStages * 2 * 16 * D * 2);
      const uint32_t bars = ptx::smem_u32(&ring_bars[warp * kRingStages]);
      // asks for page p of the batch into the next slot of the ring (whole warp calls; lane 0 issues)
      auto issue = [&](int p) {
        const int pg = p < 32 ? __shfl_sync(0xffffffffu, my_page, p & 31) : __shfl_sync(0xffffffffu, my_page_hi, p & 31);
        if (lane == 0) {
          const uint32_t s = ring_issued % kRingStages;
          const uint32_t slot = slots + s * (2 * 16 * D * 2), bar = bars + s * 8;
          ptx::mbar_arrive_expect_tx(bar, 2 * 16 * D * 2);
          // (every page is read once: its lines are the first to leave L2, not the K/V that the extend kernel beside
          // this one re-reads)
          ptx::bulk_g2s_hint(slot, kbase + (size_t)pg * page_stride, 16 * D * 2, bar, ring_policy);
          ptx::bulk_g2s_hint(slot + 16 * D * 2, vbase + (size_t)pg * page_stride, 16 * D * 2, bar, ring_policy);
        }
        ++ring_issued;
      };
      for (int p = 0; p < min(kRingStages, np); ++p) issue(p);
      PageRegs<D> pr;
      bool ok = true;
      for (int p = 0; p < np && ok; ++p) {
        const uint32_t s = ring_used % kRingStages;
        ok = ptx::mbar_wait(bars + s * 8, (ring_used / kRingStages) & 1, ring_abort);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ++ring_used;
        load_page_smem<D>(pr, slots + s * (2 * 16 * D * 2), r, c);
        // every lane has its copy of the slot in registers: the slot can take the page kRingStages ahead
        __syncwarp();
        ptx::fence_proxy_async_smem();
        if (p + kRingStages < np) issue(p + kRingStages);
        process(pr, p);
      }
      if (!ok) {
        // a wait gave up: flag it, let the copies that were asked for land (bounded), and leave
        if (lane == 0) {
          report(a.pool.status, KV_ERR_TIMEOUT);
          int never = 0;
          for (; ring_used < ring_issued; ++ring_used)
            ptx::mbar_wait_limit(bars + (ring_used % kRingStages) * 8, (ring_used / kRingStages) & 1, &never, 100000000ull);
        }
        return;
      }
    } else {
      // two register sets alternate: the next page's loads are in flight while this one is consumed
      PageRegs<D> ra, rb;
      fetch(ra, 0);
      for (int p = 0; p < np; p += 2) {
        if (p + 1 < np) fetch(rb, p + 1);
        process(ra, p);
        if (p + 1 < np) {
          if (p + 2 < np) fetch(ra, p + 2);
          process(rb, p + 1);
        }
      }
    }
  }

  // ---- finish: reduce the row sums over the token lanes, normalise, store
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
  const float lse0 = l0 > 0.f ? m0 + log2f(l0) : -INFINITY, lse1 = l1 > 0.f ? m1 + log2f(l1) : -INFINITY;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const bool valid = half ? valid1 : valid0;
    if (!valid) continue;
    const int n = half ? n1 : n0;
    const float inv = half ? inv1 : inv0;
    const int64_t orow = (int64_t)(row0 + row_token(n)) * Hq + row_head(n);
    if (DIRECT) {
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        uint4 o;
        o.x = pack_bf16x2(acc[u][0][half] * inv, acc[u][0][half + 2] * inv);
        o.y = pack_bf16x2(acc[u][1][half] * inv, acc[u][1][half + 2] * inv);
        o.z = pack_bf16x2(acc[u][2][half] * inv, acc[u][2][half + 2] * inv);
        o.w = pack_bf16x2(acc[u][3][half] * inv, acc[u][3][half + 2] * inv);
        *reinterpret_cast<uint4*>(a.out + orow * D + (8 * u + r) * 8) = o;
      }
      if (r == 0) a.lse[orow] = (half ? lse1 : lse0) * 0.6931471805599453f;
    } else {
      float* po = a.part_o + (orow * a.max_chunks + chunk) * D;
#pragma unroll
      for (int u = 0; u < NU; ++u) {
        float4* dst = reinterpret_cast<float4*>(po + (8 * u + r) * 8);
        dst[0] = make_float4(acc[u][0][half] * inv, acc[u][0][half + 2] * inv, acc[u][1][half] * inv,
                             acc[u][1][half + 2] * inv);
        dst[1] = make_float4(acc[u][2][half] * inv, acc[u][2][half + 2] * inv, acc[u][3][half] * inv,
                             acc[u][3][half + 2] * inv);
      }
      if (r == 0) a.part_lse[orow * a.max_chunks + chunk] = half ? lse1 : lse0;
    }
  }
}

// One warp merges the chunk results of one (row, head): lse = log2 sum_s 2^lse_s,
// O = sum_s 2^(lse_s - lse) O_s, in chunk order (deterministic).
template <int D>
__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ part_o,
                                                      const float* __restrict__ part_lse,
                                                      const int* __restrict__ lens, int n_rows, int n_q_heads,
                                                      int max_chunks, int chunk_tokens,
                                                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  ptx::dependency_wait();  // launched early: the partial results of the kernel in front are complete from here on
  if (warp >= n_rows * n_q_heads) return;
  const int row = warp / n_q_heads;
  const int len = __ldg(lens + row);
  const int nch = len <= 0 ? 0 : min(max_chunks, (len + chunk_tokens - 1) / chunk_tokens);
  constexpr int PER = D / 32;
  float o[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) o[i] = 0.f;
  float m = -INFINITY;
  for (int s = 0; s < nch; ++s) m = fmaxf(m, __ldg(part_lse + (int64_t)warp * max_chunks + s));
  float wsum = 0.f;
  if (m > -INFINITY) {
    for (int s = 0; s < nch; ++s) {
      const float w = exp2f(__ldg(part_lse + (int64_t)warp * max_chunks + s) - m);
      wsum += w;
      const float* po = part_o + ((int64_t)warp * max_chunks + s) * D + lane * PER;
#pragma unroll
      for (int i = 0; i < PER; ++i) o[i] += w * __ldg(po + i);
    }
  }
  const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
  __nv_bfloat16* dst = out + (int64_t)warp * D + lane * PER;
#pragma unroll
  for (int i = 0; i < PER; i += 2)
    *reinterpret_cast<uint32_t*>(dst + i) = pack_bf16x2(o[i] * inv, o[i + 1] * inv);
  if (lane == 0) lse[warp] = wsum > 0.f ? (m + log2f(wsum)) * 0.6931471805599453f : -INFINITY;
}

// Rows that no work item touches (ctx_len <= 0) still get a defined result in direct mode.
__global__ void fill_empty_rows_kernel(const int* __restrict__ lens, int n_rows, int row_elems,
                                       __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int n_q_heads) {
  const int row = blockIdx.x;
  if (row >= n_rows || __ldg(lens + row) > 0) return;
  for (int i = threadIdx.x; i < row_elems; i += blockDim.x) out[(int64_t)row * row_elems + i] = __float2bfloat16(0.f);
  for (int h = threadIdx.x; h < n_q_heads; h += blockDim.x) lse[(int64_t)row * n_q_heads + h] = -INFINITY;
}

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t decode_workspace_bytes(int n_q_heads, int head_dim, int batch, int max_ctx_len) {
  if (batch <= 0 || max_ctx_len <= 0) return 0;
  const int max_chunks = (max_ctx_len + kDecodeChunkTokens - 1) / kDecodeChunkTokens;
  if (max_chunks <= 1) return 0;
  const size_t slots = (size_t)batch * n_q_heads * max_chunks;
  return align256(slots * head_dim * sizeof(float)) + align256(slots * sizeof(float));
}

std::atomic<int> g_decode_impl{0};  // 0: default (the ring), 1: pages stream through registers, 2: pages go through a shared-memory ring

// Launches the partial (or direct) decode kernel in the chosen variant.
template <int D, bool DIRECT>
// beside: the kernel is launched so that it may start while the kernel in front of it in the stream still runs (it does
// not wait for it: nothing it touches is written there).  The mixed step uses this to run decode next to the extend kernel.
static kv_status_t launch_decode_kernel(kv_pool_t* p, const SmallArgs& a, int64_t items, bool ring, bool beside, cudaStream_t st) {
  cudaLaunchConfig_t cfg{};
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = beside ? 1 : 0;
  if (ring) {
    constexpr int smem = ring_smem_bytes<D>();
    static std::atomic<bool> configured[kMaxDevices];
    if (p->device < 0 || p->device >= kMaxDevices) return KV_ERR_INVALID;
    if (!configured[p->device].load(std::memory_order_acquire)) {
      KV_CUDA_OK(cudaFuncSetAttribute(attn_small_kernel<D, false, DIRECT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
      configured[p->device].store(true, std::memory_order_release);
    }
    cfg.gridDim = dim3((unsigned)((items + kRingWarps - 1) / kRingWarps));
    cfg.blockDim = dim3(kRingWarps * 32);
    cfg.dynamicSmemBytes = smem;
    KV_CUDA_OK(cudaLaunchKernelEx(&cfg, attn_small_kernel<D, false, DIRECT, true>, a, items));
  } else {
    cfg.gridDim = dim3((unsigned)((items + 7) / 8));
    cfg.blockDim = dim3(256);
    KV_CUDA_OK(cudaLaunchKernelEx(&cfg, attn_small_kernel<D, false, DIRECT, false>, a, items));
  }
  return KV_OK;
}

template <int D>
static kv_status_t launch_decode_d(kv_pool_t* p, const SmallArgs& base, int batch, int max_ctx_len, void* workspace,
                                   size_t workspace_bytes, bool beside, cudaStream_t st) {
  SmallArgs a = base;
  // The ring variant is the default: it keeps more bytes in flight per SM, which holds the bandwidth up on the SMs the
  // tensor-core kernel leaves free in a mixed step (0.46 -> 0.42 ms) and, alone, is worth 1.5 % on long contexts
  // (6190 vs 6100 GB/s on 256 sequences of 1024-4096 tokens) and nothing either way on shorter ones.
  const bool ring = g_decode_impl.load() != 1;
  a.max_row_tiles = 1;
  a.chunk_tokens = kDecodeChunkTokens;
  a.max_chunks = (max_ctx_len + kDecodeChunkTokens - 1) / kDecodeChunkTokens;
  const int64_t items = (int64_t)batch * p->n_kv_heads * a.max_chunks;
  if (a.max_chunks == 1) {
    // (the two kernels write disjoint rows: the second need not wait for the first either)
    if (beside) {
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3((unsigned)batch);
      cfg.blockDim = dim3(128);
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      KV_CUDA_OK(cudaLaunchKernelEx(&cfg, fill_empty_rows_kernel, a.len_a, batch, a.n_q_heads * D, a.out, a.lse, a.n_q_heads));
    } else {
      fill_empty_rows_kernel<<<batch, 128, 0, st>>>(a.len_a, batch, a.n_q_heads * D, a.out, a.lse, a.n_q_heads);
    }
    const kv_status_t ks = launch_decode_kernel<D, true>(p, a, items, ring, beside, st);
    if (ks != KV_OK) return ks;
    count_launch(2);
  } else {
    const size_t need = decode_workspace_bytes(a.n_q_heads, D, batch, max_ctx_len);
    if (workspace == nullptr || workspace_bytes < need) return KV_ERR_WORKSPACE;
    const size_t slots = (size_t)batch * a.n_q_heads * a.max_chunks;
    a.part_o = reinterpret_cast<float*>(workspace);
    a.part_lse = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + align256(slots * D * sizeof(float)));
    const kv_status_t ks = launch_decode_kernel<D, false>(p, a, items, ring, beside, st);
    if (ks != KV_OK) return ks;
    const int rows = batch * a.n_q_heads;
    {
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3((unsigned)((rows + 7) / 8));
      cfg.blockDim = dim3(256);
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      KV_CUDA_OK(cudaLaunchKernelEx(&cfg, combine_kernel<D>, (const float*)a.part_o, (const float*)a.part_lse, a.len_a, batch,
                                    a.n_q_heads, a.max_chunks, a.chunk_tokens, a.out, a.lse));
    }
    count_launch(2);
  }
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}

kv_status_t launch_decode(kv_pool_t* p, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                          const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                          void* workspace, size_t workspace_bytes, cudaStream_t st, bool beside) {
  SmallArgs a{};
  a.pool = p->view();
  a.q = (const __nv_bfloat16*)q;
  a.block_tables = block_tables;
  a.max_pages = max_pages;
  a.len_a = ctx_lens;
  a.n_q_heads = n_q_heads;
  a.group = n_q_heads / p->n_kv_heads;
  a.batch = batch;
  a.scale_log2 = scale * 1.4426950408889634f;
  a.out = (__nv_bfloat16*)out;
  a.lse = lse;
  if (p->head_dim == 128) return launch_decode_d<128>(p, a, batch, max_ctx_len, workspace, workspace_bytes, beside, st);
  return launch_decode_d<64>(p, a, batch, max_ctx_len, workspace, workspace_bytes, beside, st);
}

// Extend on the small-tile kernel: every tile of 8 query rows walks its whole visible KV range
// (no split), so K/V are re-read once per 8/G suffix tokens.  Meant for short suffixes and as the
// reference implementation inside the library for the tensor-core kernel's tests.
kv_status_t launch_extend_small(kv_pool_t* p, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                                int max_pages, const int* prefix_lens, const int* extend_lens, int batch,
                                int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                                cudaStream_t st) {
  SmallArgs a{};
  a.pool = p->view();
  a.q = (const __nv_bfloat16*)q;
  a.block_tables = block_tables;
  a.max_pages = max_pages;
  a.len_a = prefix_lens;
  a.len_b = extend_lens;
  a.cu_q = cu_q;
  a.n_q_heads = n_q_heads;
  a.group = n_q_heads / p->n_kv_heads;
  a.batch = batch;
  a.scale_log2 = scale * 1.4426950408889634f;
  a.out = (__nv_bfloat16*)out;
  a.lse = lse;
  const int tpt = 8 / a.group;
  a.max_row_tiles = (max_extend_len + tpt - 1) / tpt;
  a.max_chunks = 1;
  a.chunk_tokens = ((max_total_len + kDecodeChunkTokens - 1) / kDecodeChunkTokens) * kDecodeChunkTokens;
  const int64_t items = (int64_t)batch * p->n_kv_heads * a.max_row_tiles;
  if (items == 0) return KV_OK;
  const int64_t blocks = (items + 7) / 8;
  if (blocks > 0x7fffffffLL) return KV_ERR_UNSUPPORTED;
  if (p->head_dim == 128)
    attn_small_kernel<128, true, true><<<(int)blocks, 256, 0, st>>>(a, items);
  else
    attn_small_kernel<64, true, true><<<(int)blocks, 256, 0, st>>>(a, items);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}

}  // namespace kvattn
