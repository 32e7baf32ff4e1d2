"""CPU oracle for attention over a paged KV-cache pool.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA path is checked against.
It is independent of the CUDA path: it shares no code, header, table or helper
with it, and nothing in the product imports it (only tests, the smoke check
and the benchmark's CPU-baseline leg do).

What it computes, and the passages it restates:

* The KV cache is one pool of equally sized blocks (pages) for all requests; a
  request's logical blocks map to physical pages through a block table, pages
  are handed out on admission and given back on completion (paper Section 2.1, "vLLM memory
  model").  -> ``FreeList``, ``PagePool``, ``append``, ``gather``.
* Prefill materialises K/V for all prompt tokens; decode attends one new token
  over all stored K/V (Section 2.1, first paragraph).  -> ``attn_decode``.
* With prefix caching the engine reuses the cached KV entries of a shared
  prompt prefix and computes only the novel suffix (Section 2.1, "Prefix
  caching"; Section 2.1, "Prefix sharing in semantic operators": the map
  operator prefills nothing but its own suffix).  -> ``attn_extend``.
  The suffix token t of a prompt [S | C(t) | I] sits at absolute position
  P + t, sees every prefix key and the suffix keys up to itself.
* A Cartesian product turns one finished task into several dependent tasks
  that all reuse the parent's prefix (Section 5.1, "dependent tasks";
  Section 5.3, the Complete procedure).  -> ``attn_extend_shared``: child c of
  parent g sees the parent's P_g keys followed by its own suffix so far.
* Reuse does not change results (Section 1: scheduling leaves the query's
  meaning and the accuracy of its output untouched).  So the result has a plain definition,
  softmax(q K^T * scale) V over the visible keys, and this oracle is that
  definition written out: gather the sequence's pages into contiguous K/V,
  then three separate passes (max, sum of exponentials, weighted sum) in
  float64.  There is no tiling, no online softmax, no split-KV here.

Precision: inputs are bf16 values widened exactly to float64; nothing is
rounded on the oracle side.  LSE is the natural log of sum_j exp(scale*q.k_j).

Readings taken where the paper is silent (it gives no kernel-level detail):
scale is passed explicitly (callers use 1/sqrt(D) rounded to float32); KV head
of query head h is h // G with G = Hq // Hkv; slots at positions >= length hold
arbitrary bits and never influence a result; a decode row with ctx_len <= 0 and
an extend sequence with extend_len == 0 produce O = 0 / LSE = -inf resp. no
rows.

Pins (tests/test_oracle_pins.py): hand-worked closed form, brute force with an
independently written evaluation, K == 0 closed form (mean of V, LSE = ln n),
planted needle, rows of probabilities sum to 1, reuse == from-scratch prefill,
page-permutation invariance, GQA == MHA on repeated KV heads, decode ==
extend(E=1), split-and-combine identity, torch's fp64 SDPA as a black box;
children sharing a parent == every child on a private copy of the prefix.
No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- #
# bf16 <-> float64 (exact widening)
# --------------------------------------------------------------------------- #
def widen(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 values (exact)."""
    b = np.ascontiguousarray(bits).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- #
# page pool (host image) and allocator
# --------------------------------------------------------------------------- #
class PinnedError(Exception):
    """kv_evict, or the last kv_free, of a pinned page."""


class FreeList:
    """LIFO free list over page ids 0..num_pages-1, with owners, pins and an LRU clock.

    Documented order: a fresh list hands out 0, 1, 2, ...; released pages are pushed in the order given and
    popped last-in-first-out.  ``alloc`` is all-or-nothing.  Every call validates first and changes nothing
    on error.

    Sharing (paper Section 5.1; Algorithm 1, Complete: a parent's memory is released when all of its children
    are done): ``ref`` adds an owner, ``free`` removes one, and the page goes back when the last owner frees it.
    Explicit pinning (Section 6): a pinned page is never evicted (``evict`` raises, ``evict_lru`` skips it) and
    its last owner cannot free it; ``unpin_all`` is the deadlock fallback.  Eviction order (Sections 2.2, 6):
    least recently used first, by a logical clock that ``alloc`` and ``touch`` advance.
    """

    def __init__(self, num_pages: int):
        self.num_pages = num_pages
        self.stack = list(range(num_pages - 1, -1, -1))   # pop() gives 0 first
        self.allocated = np.zeros(num_pages, dtype=bool)
        self.refs = [0] * num_pages
        self.pins = [0] * num_pages
        self.last_use = [0] * num_pages
        self.clock = 0
        self.evicted_total = 0

    def alloc(self, n: int):
        if n < 0:
            raise ValueError("negative count")
        if n > len(self.stack):
            return None                                    # out of pages: caller defers
        ids = [self.stack.pop() for _ in range(n)]
        for p in ids:
            self.allocated[p] = True
            self.refs[p], self.pins[p] = 1, 0
            self.clock += 1
            self.last_use[p] = self.clock
        return ids

    def _check(self, ids, unique):
        seen = set()
        for p in ids:
            if p < 0 or p >= self.num_pages or not self.allocated[p] or (unique and p in seen):
                raise KeyError(f"page {p} is not allocated")
            seen.add(p)

    def _drop(self, p):
        self.allocated[p] = False
        self.refs[p] = 0
        self.stack.append(p)

    def free(self, ids):
        ids = list(ids)
        self._check(ids, unique=True)
        if any(self.pins[p] > 0 and self.refs[p] == 1 for p in ids):
            raise PinnedError()
        for p in ids:
            self.refs[p] -= 1
            if self.refs[p] == 0:
                self._drop(p)

    def evict(self, ids):
        ids = list(ids)
        self._check(ids, unique=True)
        if any(self.pins[p] > 0 for p in ids):
            raise PinnedError()
        for p in ids:
            self._drop(p)
        self.evicted_total += len(ids)

    def ref(self, ids):
        ids = list(ids)
        self._check(ids, unique=False)
        for p in ids:
            self.refs[p] += 1

    def pin(self, ids):
        ids = list(ids)
        self._check(ids, unique=False)
        for p in ids:
            self.pins[p] += 1

    def unpin(self, ids):
        ids = list(ids)
        self._check(ids, unique=True)
        if any(self.pins[p] == 0 for p in ids):
            raise ValueError("page is not pinned")
        for p in ids:
            self.pins[p] -= 1

    def unpin_all(self) -> int:
        n = sum(1 for c in self.pins if c > 0)
        self.pins = [0] * self.num_pages
        return n

    def touch(self, ids):
        ids = list(ids)
        self._check(ids, unique=False)
        for p in ids:
            self.clock += 1
            self.last_use[p] = self.clock

    def evict_lru(self, n: int):
        cand = [p for p in range(self.num_pages) if self.allocated[p] and self.pins[p] == 0]
        cand.sort(key=lambda p: self.last_use[p])
        out = cand[:n]
        for p in out:
            self._drop(p)
        self.evicted_total += len(out)
        return out

    @property
    def free_pages(self) -> int:
        return len(self.stack)


class PagePool:
    """Host image of the pool in LOGICAL layout [page][kv_head][slot][dim].

    Values are kept as bf16 bit patterns (uint16) because append and gather
    are pure data movement and are compared bit for bit.
    """

    def __init__(self, num_pages: int, page_size: int, n_kv_heads: int, head_dim: int, fill: int = 0):
        self.num_pages, self.page_size = num_pages, page_size
        self.n_kv_heads, self.head_dim = n_kv_heads, head_dim
        shape = (num_pages, n_kv_heads, page_size, head_dim)
        self.k = np.full(shape, fill, dtype=np.uint16)
        self.v = np.full(shape, fill, dtype=np.uint16)

    def append(self, block_row, start_pos: int, k_new: np.ndarray, v_new: np.ndarray):
        """Write tokens start_pos .. start_pos+n-1 of one sequence.

        k_new, v_new: uint16 [n][Hkv][D].  Token at position pos goes to page
        block_row[pos // ps], slot pos % ps.
        """
        ps = self.page_size
        for i in range(k_new.shape[0]):
            pos = start_pos + i
            page = int(block_row[pos // ps])
            if page < 0 or page >= self.num_pages:
                raise IndexError("block table entry out of range")
            self.k[page, :, pos % ps, :] = k_new[i]
            self.v[page, :, pos % ps, :] = v_new[i]

    def gather(self, block_row, length: int):
        """Contiguous K, V bit arrays [length][Hkv][D] of one sequence."""
        ps = self.page_size
        k = np.empty((length, self.n_kv_heads, self.head_dim), dtype=np.uint16)
        v = np.empty_like(k)
        for b in range((length + ps - 1) // ps):
            page = int(block_row[b])
            n = min(ps, length - b * ps)
            k[b * ps:b * ps + n] = self.k[page, :, :n, :].transpose(1, 0, 2)
            v[b * ps:b * ps + n] = self.v[page, :, :n, :].transpose(1, 0, 2)
        return k, v


# --------------------------------------------------------------------------- #
# attention: the definition
# --------------------------------------------------------------------------- #
def softmax_rows(q: np.ndarray, k: np.ndarray, visible: np.ndarray, scale: float):
    """Probabilities and LSE for query rows q [R][D] over keys k [L][D].

    Row r sees keys j < visible[r].  Returns (p [R][L], lse [R]); p is 0 at
    hidden keys; a row with visible == 0 gets p = 0 and lse = -inf.
    """
    R, L = q.shape[0], k.shape[0]
    s = float(scale) * (q @ k.T)                                   # s_j = scale * q . k_j
    hidden = np.arange(L)[None, :] >= np.asarray(visible)[:, None]
    s = np.where(hidden, -np.inf, s)
    if L == 0:
        return np.zeros((R, 0)), np.full(R, -np.inf)
    empty = np.asarray(visible) <= 0                               # rows that see no key at all
    m = np.max(s, axis=1)                                          # pass 1: row max
    m = np.where(empty, 0.0, m)
    e = np.exp(s - m[:, None])                                     # hidden keys: exp(-inf) = 0
    l = np.sum(e, axis=1)                                          # pass 2: row sum
    with np.errstate(divide="ignore", invalid="ignore"):
        p = np.where(empty[:, None], 0.0, e / l[:, None])
        lse = np.where(empty, -np.inf, m + np.log(l))
    return p, lse


def attention_rows(q, k, v, visible, scale):
    """O [R][D] = sum_j p_rj v_j and LSE [R] for query rows of one head."""
    p, lse = softmax_rows(q, k, visible, scale)
    return p @ v, lse                                              # pass 3: weighted sum


def attn_extend(pool: PagePool, q_bits, n_q_heads, cu_q, block_tables, prefix_lens, extend_lens, scale):
    """Suffix tokens attend over reused prefix pages plus the suffix so far.

    q_bits: uint16 [T_q][Hq][D], ragged by cu_q [B+1]; the suffix K/V are
    already in the pages (appended before this call).  Returns float64
    O [T_q][Hq][D], LSE [T_q][Hq].
    """
    T_q, D = q_bits.shape[0], pool.head_dim
    G = n_q_heads // pool.n_kv_heads
    qf = widen(q_bits)
    out = np.zeros((T_q, n_q_heads, D))
    lse = np.full((T_q, n_q_heads), -np.inf)
    for i in range(len(prefix_lens)):
        P, E = int(prefix_lens[i]), int(extend_lens[i])
        if E <= 0:
            continue
        kb, vb = pool.gather(block_tables[i], P + E)
        kf, vf = widen(kb), widen(vb)
        r0 = int(cu_q[i])
        visible = P + np.arange(E) + 1                              # token t sees keys 0 .. P+t
        for h in range(n_q_heads):
            g = h // G
            o, l = attention_rows(qf[r0:r0 + E, h, :], kf[:, g, :], vf[:, g, :], visible, scale)
            out[r0:r0 + E, h, :] = o
            lse[r0:r0 + E, h] = l
    return out, lse


def attn_extend_shared(pool: PagePool, q_bits, n_q_heads, cu_q, cu_children, parent_tables, parent_lens,
                       child_tables, child_lens, scale):
    """Children of one parent attend over the parent's prefix and their own suffix.

    Parent g holds parent_lens[g] tokens in the pages of parent_tables[g]; its
    children are cu_children[g] .. cu_children[g+1]-1.  Child c holds
    child_lens[c] tokens of its own in child_tables[c]; its suffix token t sees
    the parent's keys 0..P_g-1 and then its own keys 0..t (Section 5.1: the
    dependent tasks of a Cartesian product reuse the upstream task's prefix).
    q_bits: uint16 [T_q][Hq][D], child c's rows are cu_q[c] .. cu_q[c+1]-1.
    Returns float64 O [T_q][Hq][D], LSE [T_q][Hq].
    """
    T_q, D = q_bits.shape[0], pool.head_dim
    G = n_q_heads // pool.n_kv_heads
    qf = widen(q_bits)
    out = np.zeros((T_q, n_q_heads, D))
    lse = np.full((T_q, n_q_heads), -np.inf)
    for g in range(len(parent_lens)):
        P = int(parent_lens[g])
        kp, vp = pool.gather(parent_tables[g], P)
        for c in range(int(cu_children[g]), int(cu_children[g + 1])):
            E = int(child_lens[c])
            if E <= 0:
                continue
            kc, vc = pool.gather(child_tables[c], E)
            kf = widen(np.concatenate([kp, kc], axis=0))     # the child's keys: parent's, then its own
            vf = widen(np.concatenate([vp, vc], axis=0))
            r0 = int(cu_q[c])
            visible = P + np.arange(E) + 1
            for h in range(n_q_heads):
                o, l = attention_rows(qf[r0:r0 + E, h, :], kf[:, h // G, :], vf[:, h // G, :], visible, scale)
                out[r0:r0 + E, h, :] = o
                lse[r0:r0 + E, h] = l
    return out, lse


def attn_decode(pool: PagePool, q_bits, n_q_heads, block_tables, ctx_lens, scale):
    """One query token per sequence at position C-1 attends over keys 0..C-1.

    q_bits: uint16 [B][Hq][D].  Returns float64 O [B][Hq][D], LSE [B][Hq].
    """
    B, D = q_bits.shape[0], pool.head_dim
    G = n_q_heads // pool.n_kv_heads
    qf = widen(q_bits)
    out = np.zeros((B, n_q_heads, D))
    lse = np.full((B, n_q_heads), -np.inf)
    for i in range(B):
        C = int(ctx_lens[i])
        if C <= 0:
            continue
        kb, vb = pool.gather(block_tables[i], C)
        kf, vf = widen(kb), widen(vb)
        for g in range(pool.n_kv_heads):
            hs = slice(g * G, (g + 1) * G)
            o, l = attention_rows(qf[i, hs, :], kf[:, g, :], vf[:, g, :], np.full(G, C), scale)
            out[i, hs, :] = o
            lse[i, hs] = l
    return out, lse


def combine_partials(o_parts: np.ndarray, lse_parts: np.ndarray):
    """Merge attention results computed over a partition of the keys.

    o_parts [S][D] (each normalised over its own part), lse_parts [S].
    lse = ln sum_s exp(lse_s);  O = sum_s exp(lse_s - lse) O_s.
    Used only by the oracle's self-tests (it pins the split-KV combine rule).
    """
    m = np.max(lse_parts)
    w = np.exp(lse_parts - m)
    lse = m + np.log(np.sum(w))
    return (w[:, None] * o_parts).sum(axis=0) / np.sum(w), lse
