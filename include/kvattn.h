/*
 * kvattn.h - C ABI of a B200 (sm_100a) library for attention over a paged KV-cache pool.
 *
 * The calls follow the problem as the paper states it (arxiv 2607.23815, "Kalypso:
 * Relational LLM Serving"): an inference engine keeps K/V tensors in a global pool of
 * fixed-size blocks (pages) that are handed out when a request is admitted and returned
 * when it completes (Section 2.1, "vLLM memory model"); when a downstream semantic
 * operator's prompt shares its prefix with the upstream operator's prompt for the same
 * tuple, the cached KV entries are reused and only the new suffix is prefilled
 * (Section 2.1, "Prefix caching" and "Prefix sharing in semantic operators"); short
 * answers are then decoded one token at a time over all stored K/V (Section 2.1, first
 * paragraph); the scheduler releases a task's memory when the tuple is filtered or has
 * left the last stage (Algorithm 1, Complete), and unpinned blocks may be evicted under
 * memory pressure (Section 2.1; Section 6, "Explicit and virtual pinning").
 *
 * Conventions that hold for every call
 *  - Pointers are marked [host] or [dev].  The library never keeps a caller pointer past
 *    the call, and never frees or reallocates caller memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *    that take a stream enqueue work and return without synchronising.
 *  - Every call returns a kv_status_t.  Errors that the host can see (NULL pointers,
 *    negative sizes, unsupported shapes, a workspace that is too small) are returned at
 *    once with nothing launched.  Problems only the device can see (a block-table entry
 *    outside the pool) make the kernel skip the access and record KV_ERR_BOUNDS in a
 *    device status word that kv_last_async_status() reads.  Nothing aborts, traps or throws.
 *  - A pool lives on the device that was current when it was created; calls that launch work must be
 *    made with that device current (KV_ERR_INVALID otherwise).
 *  - Supported shapes: bf16 K/V/Q/O, page_size 16, head_dim 64 or 128,
 *    group G = n_q_heads / n_kv_heads in {1, 2, 4, 8}.  Anything else: KV_ERR_UNSUPPORTED.
 *  - All integer arrays are int32.  Block tables are row-major [rows][max_pages]; entry b
 *    of a row is the physical page of logical block b (tokens 16b .. 16b+15); entries past
 *    ceil(len/16) are never read (pad with -1).
 *
 * Page layout in device memory (private to the library, documented for tests)
 *    K and V are two buffers of num_pages * n_kv_heads blocks; block (page, head) holds the
 *    16 tokens x head_dim bf16 values of that page and KV head, contiguous, 16*head_dim*2
 *    bytes.  Inside a block, element (slot, d) lives at byte offset
 *        (slot/8) * (8*head_dim*2) + (d/64) * 1024 + (slot%8) * 128
 *            + ((((d%64)/8) ^ (slot%8)) * 16) + (d%8) * 2
 *    i.e. 8-token x 64-dim tiles of 1024 bytes whose 16-byte chunks are XOR-swizzled by the
 *    row index.  This is the 128-byte-swizzle shared-memory operand layout of the sm_100
 *    tensor-core MMA, so one bulk copy brings a block into shared memory ready for use.
 *    kv_pool_elem_offset() evaluates the formula.
 */
#ifndef KVATTN_H_
#define KVATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kv_pool kv_pool_t; /* opaque: owns the K/V page memory and the host free list */

typedef enum {
  KV_OK = 0,
  KV_ERR_INVALID = 1,       /* NULL pointer, negative size, inconsistent arguments            */
  KV_ERR_OOM = 2,           /* kv_alloc: not enough free pages (the caller defers the request) */
  KV_ERR_NOT_ALLOCATED = 3, /* kv_free / kv_evict of a page that is not allocated               */
  KV_ERR_BOUNDS = 4,        /* device saw a block-table entry or length outside the pool      */
  KV_ERR_UNSUPPORTED = 5,   /* shape outside the supported set                                 */
  KV_ERR_CUDA = 6,          /* a CUDA runtime call failed (allocation, launch)                 */
  KV_ERR_TIMEOUT = 7,       /* a bounded device-side wait gave up                              */
  KV_ERR_WORKSPACE = 8,     /* workspace pointer NULL or smaller than attn_workspace_bytes()   */
  KV_ERR_PINNED = 9         /* kv_evict, or the last kv_free, of a page that is pinned          */
} kv_status_t;

const char* kv_status_str(kv_status_t s);

/* ---- pool: one pool of equally sized pages for all requests (Section 2.1, vLLM memory model) -- */

/* Creates a pool on the current CUDA device and allocates its K and V buffers with cudaMalloc
 * (2 * num_pages * n_kv_heads * page_size * head_dim * 2 bytes).  *out receives the handle. */
kv_status_t kv_pool_create(int num_pages, int page_size, int n_kv_heads, int head_dim, kv_pool_t** out);
/* Same, over caller-owned device buffers k_base/v_base [dev] of at least that size each, 256-byte
 * aligned; the pool does not free them.  Lets a framework place the pages in its own allocator. */
kv_status_t kv_pool_create_ex(int num_pages, int page_size, int n_kv_heads, int head_dim, void* k_base,
                              void* v_base, kv_pool_t** out);
/* Frees what the pool owns.  The caller makes sure no kernel using the pool is still running. */
kv_status_t kv_pool_destroy(kv_pool_t* pool);
/* Occupancy as the scheduler reads it from the engine (Section 3): any pointer may be NULL. */
kv_status_t kv_pool_stats(const kv_pool_t* pool, int* free_pages, int* used_pages, int64_t* evicted_total);
/* Test surface: device base pointers and the size in bytes of each of the two buffers. */
kv_status_t kv_pool_raw(const kv_pool_t* pool, void** k_base, void** v_base, int64_t* bytes_each);
/* Test surface: ELEMENT offset (bf16 units) of (page, kv_head, slot, d) from k_base / v_base per
 * the layout formula above; -1 if out of range. */
int64_t kv_pool_elem_offset(const kv_pool_t* pool, int page, int kv_head, int slot, int d);
/* Debug aid: when on, kv_evict() overwrites the evicted pages with NaN bit patterns (on the legacy
 * default stream, synchronously) so that a stale read shows up in outputs. */
kv_status_t kv_pool_set_poison(kv_pool_t* pool, int on);

/* ---- allocator (host; mutex-guarded) ------------------------------------------------------ */

/* Hands out n page ids into out_page_ids [host].  All-or-nothing: KV_ERR_OOM leaves the pool
 * unchanged; the caller holds the request back until pages are free again (Section 2.1).
 * Order is deterministic: a fresh pool gives 0,1,2,...; released pages come back last-in-first-out. */
kv_status_t kv_alloc(kv_pool_t* pool, int n, int* out_page_ids);
/* Returns pages whose owner is done (Algorithm 1, Complete: releaseMemory).  A page id that is out
 * of range, not allocated, or listed twice gives KV_ERR_NOT_ALLOCATED with no partial effect. */
kv_status_t kv_free(kv_pool_t* pool, const int* page_ids /*host*/, int n);
/* Returns pages reclaimed under memory pressure (Section 2.1: the blocks of a finished request stay
 * cached only until the engine needs the room).  Same as kv_free plus the eviction counter and the optional poison fill;
 * the former owner must treat its prefix as lost and re-prefill (Section 2.2). */
kv_status_t kv_evict(kv_pool_t* pool, const int* page_ids /*host*/, int n);

/* ---- sharing, pinning, eviction order (host; mutex-guarded) --------------------------------
 * A join creates many dependent tasks over one parent tuple, whose prefix pages they all read (Section 5.1;
 * Algorithm 1, Complete: the parent's memory is released when all its children are done): kv_ref adds an owner
 * to allocated pages, and kv_free only returns a page to the free list when its last owner frees it.
 * Explicit pinning (Section 6, "Explicit and virtual pinning"): a pinned block cannot be evicted until the
 * scheduler unpins it; kv_evict / kv_evict_lru never take a pinned page (kv_evict: KV_ERR_PINNED, nothing
 * changed), and the last owner cannot kv_free it while it is pinned either.  Pins are counted.
 * Deadlock recovery (Section 6): when requests wait while nothing runs, the scheduler unpins everything and
 * falls back to virtual pinning: kv_unpin_all.
 * Eviction order: the engine evicts least-recently-used blocks (Section 2.2, Section 6).  The pool keeps a
 * logical clock per page, set by kv_alloc and kv_touch; kv_evict_lru(n) evicts up to n unpinned allocated
 * pages, least recently used first, whoever owns them (their owners must treat that prefix as lost), and
 * reports which.  All calls validate first and change nothing on error (KV_ERR_NOT_ALLOCATED for a page that
 * is not allocated, KV_ERR_INVALID for kv_unpin of a page that is not pinned).                              */
kv_status_t kv_ref(kv_pool_t* pool, const int* page_ids /*host*/, int n);
kv_status_t kv_pin(kv_pool_t* pool, const int* page_ids /*host*/, int n);
kv_status_t kv_unpin(kv_pool_t* pool, const int* page_ids /*host, no repeats*/, int n);
kv_status_t kv_unpin_all(kv_pool_t* pool, int* n_unpinned /*host, may be NULL: pages that were pinned*/);
kv_status_t kv_touch(kv_pool_t* pool, const int* page_ids /*host*/, int n);
kv_status_t kv_evict_lru(kv_pool_t* pool, int n, int* out_page_ids /*host [n]*/, int* n_evicted /*host*/);
/* Test surface: state of one page (any pointer may be NULL). */
kv_status_t kv_page_info(const kv_pool_t* pool, int page, int* allocated, int* refs, int* pins);

/* ---- kv_append: store new tokens' K/V in their pages (Section 2.1: prefill produces the K/V
 *      tensors of every prompt token, layer by layer) ---------------------------------------- */
/* n_segments segments; segment s holds rows cu_new[s] .. cu_new[s+1]-1 of k_new/v_new
 * ([dev] bf16 [total_new][n_kv_heads][head_dim]) and writes them to token positions
 * start_pos[s] .. of the sequence whose block-table row is seg_row[s] (seg_row NULL: row s).
 * cu_new [dev][n_segments+1], start_pos [dev][n_segments], seg_row [dev][n_segments] or NULL,
 * block_tables [dev][rows][max_pages].  Pure data movement: the stored bits equal the input bits.
 * A segment also clears (to zero bits) the slots that follow its last token in that token's page, so
 * the tail of a sequence's last page never holds stale NaN/Inf patterns; tokens are therefore appended
 * to a page in increasing position order, and two segments of one call must not write into the same
 * page (segments that meet at a page boundary are fine). */
kv_status_t kv_append(kv_pool_t* pool, const void* k_new, const void* v_new, const int* cu_new,
                      const int* start_pos, const int* seg_row, const int* block_tables, int max_pages,
                      int n_segments, int total_new, void* stream);

/* Debug/test surface: copies tokens 0..len-1 of one sequence out of its pages into contiguous
 * k_out/v_out [dev] bf16 [len][n_kv_heads][head_dim].  block_table_row [dev][>= ceil(len/16)]. */
kv_status_t kv_gather(kv_pool_t* pool, const int* block_table_row, int len, void* k_out, void* v_out,
                      void* stream);

/* ---- attention ---------------------------------------------------------------------------- */
/* Common definition (Section 2.1; the plain softmax attention the engine computes): for a query
 * row q of head h at absolute position p, with KV head g = h / G,
 *     s_j = scale * <q, k_j>,  j = 0..p;   O = sum_j softmax(s)_j v_j;   LSE = ln sum_j exp(s_j).
 * O is written as bf16 (fp32 accumulation, one rounding at the store), LSE as fp32 (natural log). */

/* Bytes of scratch [dev] the attention calls need for the given batch (256-byte aligned). */
size_t attn_workspace_bytes(const kv_pool_t* pool, int n_q_heads, int batch_ext, int total_q, int max_total_len,
                            int batch_dec, int max_ctx_len);

/* Extend (the downstream operator prefills nothing but its own suffix, Section 2.1): sequence i has prefix_lens[i] reused tokens
 * and extend_lens[i] new ones, all already in its pages (kv_append first).  Suffix token t sits at
 * position prefix_lens[i]+t and sees keys 0..prefix_lens[i]+t.  prefix_lens[i]=0 is a from-scratch
 * prefill (the cache-miss path of Section 2.2); extend_lens[i]=0 contributes no rows.
 * q/out [dev] bf16 [total_q][n_q_heads][head_dim], ragged by cu_q [dev][batch+1]; lse [dev] fp32
 * [total_q][n_q_heads]; prefix_lens, extend_lens [dev][batch].  max_extend_len / max_total_len are
 * host-side upper bounds on extend_lens[i] and prefix_lens[i]+extend_lens[i] (they size the grid); a
 * sequence that exceeds them on the device, or suffix rows beyond total_q, is recorded as KV_ERR_BOUNDS
 * (kv_last_async_status) and its rows beyond the bound are left unwritten. */
kv_status_t attn_extend(kv_pool_t* pool, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                        int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                        int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream);

/* kv_append of the suffix and attn_extend in one call (Section 2.1: the downstream operator's prefill both
 * stores the suffix tokens' K/V and attends with them): k_new / v_new [dev] bf16 [total_q][n_kv_heads][head_dim],
 * ragged by cu_q like q, are written to positions prefix_lens[i] .. prefix_lens[i]+extend_lens[i]-1 of sequence
 * i's pages exactly as kv_append(k_new, v_new, cu_q, prefix_lens, NULL, block_tables, ...) would (same bits, same
 * clearing of the last page's tail), then the suffix attends exactly as attn_extend would (same bits).  What it
 * saves is launches: the rows are scattered by the kernel that also prepares the attention kernel's work list, and
 * the attention kernel is launched so that its start-up overlaps that kernel.  Arguments, workspace and errors as
 * for kv_append and attn_extend. */
kv_status_t attn_extend_append(kv_pool_t* pool, const void* q, const void* k_new, const void* v_new, int n_q_heads,
                               const int* cu_q, const int* block_tables, int max_pages, const int* prefix_lens,
                               const int* extend_lens, int batch, int total_q, int max_extend_len, int max_total_len,
                               float scale, void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* The same batch passes through every layer of the model with the same lengths and block tables (Section 2.1: K/V
 * are kept per layer), so what attn_extend derives from the lengths alone - its list of work items - can be built
 * once per step and reused by every layer.  attn_extend_plan builds it into the workspace; attn_extend_planned is
 * attn_extend without that part and must get the arguments (lengths, tables, bounds, workspace) the plan was built
 * with; the plan stays valid for any number of attn_extend_planned calls, one at a time, until the workspace is
 * written by another call.  Results are bit-identical to attn_extend.  The pages need not hold the K/V yet when the
 * plan is built. */
kv_status_t attn_extend_plan(kv_pool_t* pool, int n_q_heads, const int* cu_q, const int* block_tables, int max_pages,
                             const int* prefix_lens, const int* extend_lens, int batch, int total_q, int max_extend_len,
                             int max_total_len, void* workspace, size_t workspace_bytes, void* stream);
kv_status_t attn_extend_planned(kv_pool_t* pool, const void* q, int n_q_heads, const int* cu_q, const int* block_tables,
                                int max_pages, const int* prefix_lens, const int* extend_lens, int batch, int total_q,
                                int max_extend_len, int max_total_len, float scale, void* out, float* lse,
                                void* workspace, size_t workspace_bytes, void* stream);

/* One pipeline step from host memory: the call for a caller whose suffix Q/K/V, lengths and block tables live
 * in host buffers (pinned, if the call is to return before the copies are done).  On the given stream it
 * copies the inputs into `staging` [dev], appends the suffix K/V rows of sequence i at positions
 * prefix_lens[i].. of its pages (kv_append), runs attn_extend, and copies O and LSE back into out / lse
 * [host].  All array arguments except staging are HOST pointers with the shapes of kv_append / attn_extend;
 * staging [dev, 256-byte aligned] holds attn_extend_host_staging_bytes() bytes; it and the host buffers belong
 * to the call until the stream has passed it.  The copies run on copy streams of the pool, ordered against the
 * kernels (on `stream`) by events, and the stream waits for the copy out; with two staging areas used in turn
 * one step's copies overlap its neighbour's kernels.  The copy in starts at once: the host inputs must be
 * final when the call is made.  At most four staging areas are tracked at a time.  Errors as for kv_append and attn_extend, KV_ERR_WORKSPACE for a staging area that is too
 * small.  (In the paper the requests reach the engine from host-side operators, Section 3; the paper has
 * no counterpart of this exact call.) */
size_t attn_extend_host_staging_bytes(const kv_pool_t* pool, int n_q_heads, int batch, int total_q, int max_pages,
                                      int max_total_len);
kv_status_t attn_extend_host(kv_pool_t* pool, const void* q, const void* k_new, const void* v_new, int n_q_heads,
                             const int* cu_q, const int* block_tables, int max_pages, const int* prefix_lens,
                             const int* extend_lens, int batch, int total_q, int max_extend_len, int max_total_len,
                             float scale, void* out, float* lse, void* staging, size_t staging_bytes, void* stream);

/* Extend for children that share a parent's prefix (the dependent tasks a Cartesian product creates
 * over one parent task, Sections 5.1 and 5.3).  Parent g owns parent_lens[g] tokens in the pages of
 * parent_tables[g]; its children are the sequences cu_children[g] .. cu_children[g+1]-1.  Child c has
 * child_lens[c] tokens of its own in the pages of child_tables[c] (kv_append first) and its suffix
 * token t sees the parent's parent_lens[g] keys followed by its own keys 0..t.  (For parent lengths
 * that are multiples of the page size this equals attn_extend with every child's block table = the
 * parent's pages followed by its own; other parent lengths are fine here, the children's keys never
 * share a page with the parent's.)  The shared pages are read once per parent for all its children
 * (their query rows are stacked), not once per child.
 * q/out [dev] bf16 [total_q][n_q_heads][head_dim] (out 32-byte aligned), rows ragged by cu_q
 * [dev][n_children+1], children of a parent consecutive; lse [dev] fp32 [total_q][n_q_heads];
 * cu_children [dev][n_parents+1]; parent_tables [dev][n_parents][max_pages_parent]; parent_lens
 * [dev][n_parents]; child_tables [dev][n_children][max_pages_child]; child_lens [dev][n_children].
 * Host-side upper bounds: max_child_len >= child_lens[c]; max_parent_rows >= the suffix tokens of
 * all children of one parent; max_parent_len >= parent_lens[g].  Scratch:
 * attn_extend_shared_workspace_bytes().  Errors: KV_ERR_INVALID (NULL pointers, misaligned q/out, bounds
 * that do not fit the tables), KV_ERR_UNSUPPORTED (head geometry outside the set above, head_dim other
 * than 64/128, scale <= 0), KV_ERR_WORKSPACE; a table entry or length outside the pool is skipped on
 * the device and recorded as KV_ERR_BOUNDS (kv_last_async_status).  Nothing is allocated or retained.
 * With kvattn_set_shared_impl(1) the two partial results of a row (shared part, own part) are each
 * rounded to bf16 before they are merged; the default for suffixes of 16 tokens and more on average
 * accumulates both in one fp32 accumulator. */
size_t attn_extend_shared_workspace_bytes(const kv_pool_t* pool, int n_q_heads, int n_parents, int n_children,
                                          int total_q, int max_parent_len);
kv_status_t attn_extend_shared(kv_pool_t* pool, const void* q, int n_q_heads, const int* cu_q, const int* cu_children,
                               const int* parent_tables, int max_pages_parent, const int* parent_lens,
                               const int* child_tables, int max_pages_child, const int* child_lens, int n_parents,
                               int n_children, int total_q, int max_child_len, int max_parent_rows,
                               int max_parent_len, float scale, void* out, float* lse, void* workspace,
                               size_t workspace_bytes, void* stream);

/* Decode (each new token attends over every K/V stored so far, Section 2.1): one query
 * per sequence at position ctx_lens[i]-1 over keys 0..ctx_lens[i]-1 (its own K/V already appended).
 * q/out [dev] bf16 [batch][n_q_heads][head_dim]; lse [dev] fp32 [batch][n_q_heads]; ctx_lens [dev]
 * [batch]; max_ctx_len: host upper bound.  ctx_lens[i] <= 0 writes O = 0, LSE = -inf. */
kv_status_t attn_decode(kv_pool_t* pool, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                        const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream);

/* (No counterpart in the paper: an addition for callers that must not allocate.)
 * Same result as attn_decode, but without a workspace argument: the split-KV scratch lives in a fixed array
 * inside the library (attn_decode_static_scratch_bytes() = 8 MiB, resident on every GPU that loads the library
 * until the process exits).  Meant for code that runs where device allocation is forbidden or unavailable - a
 * plugin that was handed fixed buffers, a memory-planned or captured region of a framework, a service whose
 * allocator is frozen after start-up - and that therefore cannot size and allocate attn_decode's workspace.
 * The call itself performs no cudaMalloc/cudaFree and calls no allocating routine.
 *  - Limit: a batch whose scratch need (the same formula attn_workspace_bytes() uses for decode; 0 when
 *    max_ctx_len <= 1024) exceeds the array is refused with KV_ERR_WORKSPACE; nothing is launched.
 *  - The first call on each device looks up the array's device address (one cudaGetSymbolAddress with that
 *    device current) and caches it; make that first call before any stream capture begins.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.  Nothing in it needs
 *    to be zero at entry (every slot that is read is written earlier in the same call), but two calls that
 *    overlap on the GPU (different streams, or threads using different streams) race on it: serialise them. */
kv_status_t attn_decode_static(kv_pool_t* pool, const void* q, int n_q_heads, const int* block_tables, int max_pages,
                               const int* ctx_lens, int batch, int max_ctx_len, float scale, void* out, float* lse,
                               void* stream);
size_t attn_decode_static_scratch_bytes(void);

typedef struct {
  const void* q; const int* cu_q; const int* block_tables; int max_pages;
  const int* prefix_lens; const int* extend_lens; int batch; int total_q;
  int max_extend_len; int max_total_len; void* out; float* lse;
} attn_extend_args_t;

typedef struct {
  const void* q; const int* block_tables; int max_pages; const int* ctx_lens;
  int batch; int max_ctx_len; void* out; float* lse;
} attn_decode_args_t;

/* One pipeline step of two chained operators (e.g. sem_map feeding sem_filter, Section 1): the
 * extend set and the decode set are launched so that the tensor-bound and the HBM-bound work
 * share the GPU.  Either argument may be NULL or have batch 0.  The workspace must be sized by
 * attn_workspace_bytes() with both batches.  Work is ordered after prior work on `stream`, and
 * later work on `stream` is ordered after it: both kernels are queued on `stream` itself, the decode kernel so that
 * it starts beside the extend kernel instead of behind it.  The extend kernel takes a share of the SMs that is
 * derived from the host-side bounds of the two batches (kvattn_set_mixed_extend_ctas overrides it). */
kv_status_t attn_mixed(kv_pool_t* pool, int n_q_heads, float scale, const attn_extend_args_t* ext,
                       const attn_decode_args_t* dec, void* workspace, size_t workspace_bytes, void* stream);

/* ---- checks ------------------------------------------------------------------------------- */
/* Validates on the device that every block-table entry a batch would read (blocks 0..ceil(len/16)-1
 * of each row) is a page of this pool and that 0 <= lens[i] <= 16*max_pages; synchronises; returns
 * KV_ERR_BOUNDS if not.  lens, block_tables [dev]. */
kv_status_t kv_check_batch(kv_pool_t* pool, const int* block_tables, int max_pages, const int* lens, int batch,
                           void* stream);
/* Synchronises the device, returns and clears the device status word (KV_OK if nothing was seen). */
kv_status_t kv_last_async_status(kv_pool_t* pool);

/* Selects the extend kernel: 0 = automatic, 1 = the small-tile kernel (rows of one KV head read K/V
 * straight from HBM), 2 = the tcgen05 tensor-core kernel.  Process-wide; for tests and benchmarks. */
kv_status_t kvattn_set_extend_impl(int impl);
/* Test/tuning hook for attn_extend_shared: 0 = choose by the mean suffix length (default), 1 = three kernels
 * (shared part, own part, merge), 2 = one kernel that walks the parent's and then the children's tiles. */
kv_status_t kvattn_set_shared_impl(int impl);
/* Selects how the decode kernel brings pages on chip: 1 = straight into registers (one page per warp in flight), 2 =
 * through a per-warp ring of page slots in shared memory filled by bulk copies (several pages per warp in flight);
 * 0 = the default, which is 2.  Same arithmetic, same bits.  Process-wide; for tests and benchmarks. */
kv_status_t kvattn_set_decode_impl(int impl);
/* Tuning: inside attn_mixed (both sets present) the persistent extend kernel takes at most n SMs, so that the
 * HBM-bound decode kernel runs beside it on the others instead of after it.  0 = derived from the bounds of the two
 * batches (the default).  Process-wide. */
kv_status_t kvattn_set_mixed_extend_ctas(int n);
/* Test surface (the paper has no counterpart): runs a one-CTA kernel whose warps wait, with the same bounded
 * wait the attention kernels use, on barriers that nothing completes; the first gives up after limit_ns
 * (1 .. 1e8), raises the CTA's abort flag, which releases the others, the kernel frees its tensor memory and
 * records KV_ERR_TIMEOUT, which kv_last_async_status() then returns (and clears).  The device stays usable.
 * trace [dev][4] receives: bulk copy landed (1), lanes that gave up (32), parked warp released by the flag (1),
 * nanoseconds waited. */
kv_status_t kvattn_selftest_bounded_wait(kv_pool_t* pool, unsigned long long limit_ns, int* trace, void* stream);
/* Number of kernels this library has launched since load (all pools); for benchmark accounting. */
int64_t kvattn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KVATTN_H_ */
