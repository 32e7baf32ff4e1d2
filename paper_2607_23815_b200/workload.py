"""Device-resident synthetic workloads for the benchmark and the full-size parity tests.

Plays the (out-of-scope) engine around the library: allocates pages from the pool, scatters them
over the pool with a seeded permutation, builds block tables, draws K/V/Q with synth and writes
K/V into the pages with kv_append.  Contains no attention arithmetic.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np
import torch

from . import kvattn, ranks, synth


@dataclasses.dataclass
class ExtendSet:
    prefix: List[int]
    extend: List[int]
    rows: List[List[int]]
    uids: List[int]
    q: torch.Tensor
    k_new: torch.Tensor
    v_new: torch.Tensor
    cu_q: torch.Tensor
    block_tables: torch.Tensor
    prefix_lens: torch.Tensor
    extend_lens: torch.Tensor
    out: torch.Tensor
    lse: torch.Tensor

    @property
    def max_extend(self): return max(self.extend)
    @property
    def max_total(self): return max(p + e for p, e in zip(self.prefix, self.extend))
    @property
    def total_q(self): return int(sum(self.extend))

    def flops(self, geom: synth.Geometry) -> float:
        """Algorithmic work: 4*D*Hq per visible (query, key) pair."""
        pairs = sum(e * p + e * (e + 1) // 2 for p, e in zip(self.prefix, self.extend))
        return 4.0 * geom.head_dim * geom.n_q_heads * pairs

    def kv_bytes(self, geom: synth.Geometry) -> int:
        return sum(p + e for p, e in zip(self.prefix, self.extend)) * geom.kv_bytes_per_token


@dataclasses.dataclass
class DecodeSet:
    ctx: List[int]
    rows: List[List[int]]
    uids: List[int]
    q: torch.Tensor
    block_tables: torch.Tensor
    ctx_lens: torch.Tensor
    out: torch.Tensor
    lse: torch.Tensor

    @property
    def max_ctx(self): return max(self.ctx)

    def kv_bytes(self, geom: synth.Geometry) -> int:
        return sum(self.ctx) * geom.kv_bytes_per_token


class DeviceWorkload:
    """One workload instance on one GPU: a pool plus an extend set and/or a decode set."""

    def __init__(self, w: synth.Workload, device="cuda", seed_offset: int = 0, write_suffix: bool = True):
        self.w, self.geom, self.device = w, w.geom, device
        self.seed = ranks.replica_seed(w.seed, seed_offset)
        g = w.geom
        self.pool = kvattn.kv_pool_create(w.num_pages, g.page_size, g.n_kv_heads, g.head_dim)
        ids = kvattn.kv_alloc(self.pool, w.num_pages)
        perm = synth.page_permutation(self.seed, w.num_pages)
        self.placement = [ids[i] for i in perm.tolist()]
        self.cursor = 0
        ext, dec = synth.draw_lengths(dataclasses.replace(w, seed=self.seed))
        self.ext: Optional[ExtendSet] = self._make_extend(ext, write_suffix) if ext else None
        self.dec: Optional[DecodeSet] = self._make_decode(dec) if dec else None
        unused = self.placement[self.cursor:]
        if unused:
            kvattn.kv_free(self.pool, unused)                       # pages the batch does not need
        nbytes = kvattn.attn_workspace_bytes(
            self.pool, g.n_q_heads, len(ext), self.ext.total_q if self.ext else 0,
            self.ext.max_total if self.ext else 0, len(dec), self.dec.max_ctx if self.dec else 0)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        torch.cuda.synchronize()

    # ------------------------------------------------------------------ helpers
    def _take(self, n):
        assert self.cursor + n <= len(self.placement), "pool too small for this batch"
        out = self.placement[self.cursor:self.cursor + n]
        self.cursor += n
        return out

    def _i32(self, x):
        return torch.tensor(x, dtype=torch.int32, device=self.device)

    def _append(self, rows_bt, uid_list, ranges):
        """ranges: (row, lo, hi).  Appends in slabs to bound temporary memory."""
        g, dev = self.geom, self.device
        slab, tok = [], 0
        def flush():
            nonlocal slab, tok
            if not slab:
                return
            ks = [synth.normal_bf16(self.seed, synth.TAG_K, uid_list[r], lo, hi - lo, g.n_kv_heads, g.head_dim, dev)
                  for r, lo, hi in slab]
            vs = [synth.normal_bf16(self.seed, synth.TAG_V, uid_list[r], lo, hi - lo, g.n_kv_heads, g.head_dim, dev)
                  for r, lo, hi in slab]
            cu = self._i32(np.concatenate([[0], np.cumsum([hi - lo for _, lo, hi in slab])]).tolist())
            kvattn.kv_append(self.pool, torch.cat(ks), torch.cat(vs), cu, self._i32([lo for _, lo, _ in slab]),
                             self._i32([r for r, _, _ in slab]), rows_bt)
            torch.cuda.synchronize()
            slab, tok = [], 0
        for r, lo, hi in ranges:
            if hi <= lo:
                continue
            slab.append((r, lo, hi)); tok += hi - lo
            if tok >= 65536:
                flush()
        flush()

    def _make_extend(self, ext, write_suffix) -> ExtendSet:
        g, dev = self.geom, self.device
        P, E = [p for p, _ in ext], [e for _, e in ext]
        rows = [self._take(synth.pages_needed(p + e, g.page_size)) for p, e in ext]
        uids = list(range(len(ext)))
        bt = torch.from_numpy(synth.block_table(rows)).to(dev)
        self._append(bt, uids, [(i, 0, P[i]) for i in range(len(ext))])                 # upstream operator
        k_new = torch.cat([synth.normal_bf16(self.seed, synth.TAG_K, uids[i], P[i], E[i], g.n_kv_heads, g.head_dim, dev)
                           for i in range(len(ext))])
        v_new = torch.cat([synth.normal_bf16(self.seed, synth.TAG_V, uids[i], P[i], E[i], g.n_kv_heads, g.head_dim, dev)
                           for i in range(len(ext))])
        q = torch.cat([synth.normal_bf16(self.seed, synth.TAG_Q, uids[i], P[i], E[i], g.n_q_heads, g.head_dim, dev)
                       for i in range(len(ext))])
        cu = self._i32(np.concatenate([[0], np.cumsum(E)]).tolist())
        es = ExtendSet(P, E, rows, uids, q, k_new, v_new, cu, bt, self._i32(P), self._i32(E),
                       torch.empty_like(q), torch.empty((q.shape[0], g.n_q_heads), dtype=torch.float32, device=dev))
        if write_suffix:
            kvattn.kv_append(self.pool, k_new, v_new, cu, es.prefix_lens, None, bt)
        return es

    def _make_decode(self, dec) -> DecodeSet:
        g, dev = self.geom, self.device
        rows = [self._take(synth.pages_needed(c, g.page_size)) for c in dec]
        uids = [1_000_000 + i for i in range(len(dec))]
        bt = torch.from_numpy(synth.block_table(rows)).to(dev)
        self._append(bt, uids, [(i, 0, dec[i]) for i in range(len(dec))])
        q = torch.cat([synth.normal_bf16(self.seed, synth.TAG_Q, uids[i], dec[i] - 1, 1, g.n_q_heads, g.head_dim, dev)
                       for i in range(len(dec))])
        return DecodeSet(list(dec), rows, uids, q, bt, self._i32(dec), torch.empty_like(q),
                         torch.empty((len(dec), g.n_q_heads), dtype=torch.float32, device=dev))

    # ------------------------------------------------------------------ the calls
    def append_suffix(self, stream=None):
        e = self.ext
        kvattn.kv_append(self.pool, e.k_new, e.v_new, e.cu_q, e.prefix_lens, None, e.block_tables, stream)

    def extend(self, stream=None):
        e = self.ext
        kvattn.attn_extend(self.pool, e.q, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens, e.max_extend,
                           e.max_total, self.geom.scale, e.out, e.lse, self.workspace, stream)

    def extend_append(self, stream=None):
        """The downstream operator's prefill as one call: the suffix K/V rows go into their pages and the suffix attends."""
        e = self.ext
        kvattn.attn_extend_append(self.pool, e.q, e.k_new, e.v_new, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens,
                                  e.max_extend, e.max_total, self.geom.scale, e.out, e.lse, self.workspace, stream)

    def extend_plan(self, stream=None):
        e = self.ext
        kvattn.attn_extend_plan(self.pool, self.geom.n_q_heads, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens,
                                e.total_q, e.max_extend, e.max_total, self.workspace, stream)

    def extend_planned(self, stream=None):
        """attn_extend over the plan extend_plan() left in the workspace (what every layer after the first would call)."""
        e = self.ext
        kvattn.attn_extend_planned(self.pool, e.q, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens, e.max_extend,
                                   e.max_total, self.geom.scale, e.out, e.lse, self.workspace, stream)

    def decode(self, stream=None):
        d = self.dec
        kvattn.attn_decode(self.pool, d.q, d.block_tables, d.ctx_lens, d.max_ctx, self.geom.scale, d.out, d.lse,
                           self.workspace, stream)

    def mixed(self, stream=None):
        e, d = self.ext, self.dec
        ea = kvattn.extend_args(e.q, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens, e.max_extend, e.max_total,
                                e.out, e.lse) if e else None
        da = kvattn.decode_args(d.q, d.block_tables, d.ctx_lens, d.max_ctx, d.out, d.lse) if d else None
        kvattn.attn_mixed(self.pool, self.geom.n_q_heads, self.geom.scale, ea, da, self.workspace, stream)

    def source_kv(self, kind: str, i: int):
        """K/V bits of sequence i of the extend ("ext") or decode ("dec") set, re-drawn from the input
        generator (not read back from the pool): the oracle's inputs come from here."""
        g, dev = self.geom, self.device
        if kind == "ext":
            uid, length = self.ext.uids[i], self.ext.prefix[i] + self.ext.extend[i]
        else:
            uid, length = self.dec.uids[i], self.dec.ctx[i]
        k = synth.normal_bf16(self.seed, synth.TAG_K, uid, 0, length, g.n_kv_heads, g.head_dim, dev)
        v = synth.normal_bf16(self.seed, synth.TAG_V, uid, 0, length, g.n_kv_heads, g.head_dim, dev)
        return synth.bf16_bits(k), synth.bf16_bits(v)

    def gather_host(self, rows, length):
        """Contiguous K/V bits of one sequence, read back through kv_gather (for the oracle's input)."""
        g, dev = self.geom, self.device
        k = torch.empty((length, g.n_kv_heads, g.head_dim), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k)
        kvattn.kv_gather(self.pool, self._i32(rows), length, k, v)
        torch.cuda.synchronize()
        return synth.bf16_bits(k), synth.bf16_bits(v)

    def close(self):
        """Destroys the pool; raises if a kernel recorded an error (bounds, a wait that gave up) while it lived."""
        torch.cuda.synchronize()
        status = kvattn.kv_last_async_status(self.pool)
        self.pool.destroy()
        if status != kvattn.KV_OK:
            raise kvattn.KvError(status, "device status at close")


class FanoutWorkload:
    """Children that share their parent's prefix pages (the dependent tasks of a Cartesian product, Section 5.1):
    n_parents parents with a prefix that is a multiple of the page size, n_children children each with a short
    suffix of its own on private pages.  Stands in for the paper's join workload (contracts of about 2,145 tokens
    with 17 right-side tuples each, Section 7.3); lengths are seeded draws around the given centres."""

    def __init__(self, geom: synth.Geometry, n_parents=32, n_children=17, prefix_centre=2144, prefix_spread=224,
                 suffix_range=(30, 44), seed=260723820, device="cuda"):
        self.geom, self.device, self.seed = geom, device, seed
        g, ps = geom, geom.page_size
        self.parent_lens = [ps * (synth.uniform_int(seed, 201, i, prefix_centre - prefix_spread,
                                                    prefix_centre + prefix_spread) // ps) for i in range(n_parents)]
        self.child_lens = [synth.uniform_int(seed, 202, c, suffix_range[0], suffix_range[1])
                           for c in range(n_parents * n_children)]
        self.n_parents, self.n_children = n_parents, n_parents * n_children
        n_pages = sum(L // ps for L in self.parent_lens) + sum(synth.pages_needed(E, ps) for E in self.child_lens)
        self.pool = kvattn.kv_pool_create(n_pages, ps, g.n_kv_heads, g.head_dim)
        ids = kvattn.kv_alloc(self.pool, n_pages)
        placement = [ids[i] for i in synth.page_permutation(seed, n_pages).tolist()]
        cur = 0
        self.parent_rows, self.child_rows = [], []
        for L in self.parent_lens:
            self.parent_rows.append(placement[cur:cur + L // ps]); cur += L // ps
        for E in self.child_lens:
            n = synth.pages_needed(E, ps)
            self.child_rows.append(placement[cur:cur + n]); cur += n
        i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=device)
        self.parent_tables, self.child_tables = i32(synth.block_table(self.parent_rows)), i32(synth.block_table(self.child_rows))
        # K/V: parents carry uids 0.., children 100000..
        for rows, lens, uid0, bt in ((self.parent_rows, self.parent_lens, 0, self.parent_tables),
                                     (self.child_rows, self.child_lens, 100000, self.child_tables)):
            ks = [synth.normal_bf16(seed, synth.TAG_K, uid0 + i, 0, L, g.n_kv_heads, g.head_dim, device) for i, L in enumerate(lens)]
            vs = [synth.normal_bf16(seed, synth.TAG_V, uid0 + i, 0, L, g.n_kv_heads, g.head_dim, device) for i, L in enumerate(lens)]
            kvattn.kv_append(self.pool, torch.cat(ks), torch.cat(vs), i32(np.concatenate([[0], np.cumsum(lens)])),
                             i32([0] * len(lens)), i32(list(range(len(lens)))), bt)
        self.q = torch.cat([synth.normal_bf16(seed, synth.TAG_Q, 100000 + c, 0, E, g.n_q_heads, g.head_dim, device)
                            for c, E in enumerate(self.child_lens)])
        self.cu_q = i32(np.concatenate([[0], np.cumsum(self.child_lens)]))
        self.cu_children = i32(np.arange(n_parents + 1) * n_children)
        self.parent_lens_d, self.child_lens_d = i32(self.parent_lens), i32(self.child_lens)
        self.max_parent_rows = max(sum(self.child_lens[g0 * n_children:(g0 + 1) * n_children]) for g0 in range(n_parents))
        self.out = torch.empty_like(self.q)
        self.lse = torch.empty((self.q.shape[0], g.n_q_heads), dtype=torch.float32, device=device)
        self.ws_shared = torch.empty(max(256, kvattn.attn_extend_shared_workspace_bytes(
            self.pool, g.n_q_heads, n_parents, self.n_children, int(self.q.shape[0]), max(self.parent_lens))),
            dtype=torch.uint8, device=device)
        # the same children as independent sequences: block table = the parent's pages, then the child's own
        child_parent = np.repeat(np.arange(n_parents), n_children)
        self.alias_tables = i32(synth.block_table([self.parent_rows[gp] + self.child_rows[c] for c, gp in enumerate(child_parent)]))
        self.alias_prefix = i32([self.parent_lens[gp] for gp in child_parent])
        self.max_total = max(self.parent_lens[gp] + self.child_lens[c] for c, gp in enumerate(child_parent))
        self.out2, self.lse2 = torch.empty_like(self.q), torch.empty_like(self.lse)
        self.ws_alias = torch.empty(max(256, kvattn.attn_workspace_bytes(self.pool, g.n_q_heads, self.n_children,
                                                                         int(self.q.shape[0]), self.max_total, 0, 0)),
                                    dtype=torch.uint8, device=device)
        torch.cuda.synchronize()

    def flops(self) -> float:
        g = self.geom
        child_parent = np.repeat(np.arange(self.n_parents), self.n_children // self.n_parents)
        pairs = sum(E * self.parent_lens[gp] + E * (E + 1) // 2 for E, gp in zip(self.child_lens, child_parent))
        return 4.0 * g.head_dim * g.n_q_heads * pairs

    def shared(self):
        kvattn.attn_extend_shared(self.pool, self.q, self.cu_q, self.cu_children, self.parent_tables, self.parent_lens_d,
                                  self.child_tables, self.child_lens_d, max(self.child_lens), self.max_parent_rows,
                                  max(self.parent_lens), self.geom.scale, self.out, self.lse, self.ws_shared)

    def independent(self):
        kvattn.attn_extend(self.pool, self.q, self.cu_q, self.alias_tables, self.alias_prefix, self.child_lens_d,
                           max(self.child_lens), self.max_total, self.geom.scale, self.out2, self.lse2, self.ws_alias)

    def close(self):
        """Destroys the pool; raises if a kernel recorded an error (bounds, a wait that gave up) while it lived."""
        torch.cuda.synchronize()
        status = kvattn.kv_last_async_status(self.pool)
        self.pool.destroy()
        if status != kvattn.KV_OK:
            raise kvattn.KvError(status, "device status at close")


class PipelineLoop:
    """The two-operator pipeline step (sem_map feeding sem_filter, Section 1) as a loop over several steps at full
    size: a decode set whose contexts grow by one token per step, an extend set that is redrawn every step, one
    kv_append of each step's new tokens (the extend suffixes and one token per decode sequence), attn_mixed, and
    between steps a seeded fraction of the live pages evicted, re-allocated and re-filled (an evicted block's owner
    recomputes it, Section 2.2).  Plays the engine around the library; holds no attention arithmetic.

    The K/V "source" tensors stand for what the model would recompute: values are keyed on (sequence uid, position),
    so a re-append after an eviction writes the same bits again.
    """

    def __init__(self, w: synth.Workload, device="cuda", seed_offset: int = 0, steps: int = 8, poison: bool = False):
        self.w, self.geom, self.device, self.steps = w, w.geom, device, steps
        self.seed = ranks.replica_seed(w.seed, seed_offset)
        g = w.geom
        self.pool = kvattn.kv_pool_create(w.num_pages, g.page_size, g.n_kv_heads, g.head_dim)
        if poison:
            kvattn.kv_pool_set_poison(self.pool, True)
        # random physical placement: take every page and give them back in a seeded order, so that the library's
        # last-in-first-out free list hands them out in that order
        ids = kvattn.kv_alloc(self.pool, w.num_pages)
        perm = synth.page_permutation(self.seed, w.num_pages)
        kvattn.kv_free(self.pool, [ids[i] for i in perm.tolist()])
        _, dec = synth.draw_lengths(dataclasses.replace(w, seed=self.seed))
        self.n_ext, self.n_dec = w.n_extend, len(dec)
        self.ctx = list(dec)                                                   # current decode context lengths
        self.max_pages = synth.pages_needed(max(max(dec) + steps, w.prefix_range[1] + w.extend_range[1]), g.page_size)
        self.rows = [[] for _ in range(self.n_ext)] + \
                    [kvattn.kv_alloc(self.pool, synth.pages_needed(c + steps, g.page_size)) for c in dec]
        self.dec_uids = [1_000_000 + i for i in range(self.n_dec)]
        self.dec_src_off = np.concatenate([[0], np.cumsum([c + steps for c in dec])]).astype(np.int64)
        self.dec_k_src = torch.cat([synth.normal_bf16(self.seed, synth.TAG_K, u, 0, c + steps, g.n_kv_heads, g.head_dim, device)
                                    for u, c in zip(self.dec_uids, dec)])
        self.dec_v_src = torch.cat([synth.normal_bf16(self.seed, synth.TAG_V, u, 0, c + steps, g.n_kv_heads, g.head_dim, device)
                                    for u, c in zip(self.dec_uids, dec)])
        self.bt_host = np.full((self.n_ext + self.n_dec, self.max_pages), -1, dtype=np.int32)
        for j in range(self.n_dec):
            r = self.rows[self.n_ext + j]
            self.bt_host[self.n_ext + j, :len(r)] = r
        self.bt = torch.from_numpy(self.bt_host).to(device)
        # the decode sequences' contexts so far (an earlier operator's work, not part of a step)
        self._append_ranges([(self.n_ext + j, 0, dec[j]) for j in range(self.n_dec)])
        self.step_index = -1
        self.prefix, self.extend = [], []
        nb = kvattn.attn_workspace_bytes(self.pool, g.n_q_heads, self.n_ext, self.n_ext * w.extend_range[1],
                                         w.prefix_range[1] + w.extend_range[1], self.n_dec, max(dec) + steps)
        self.workspace = torch.empty(max(nb, 256), dtype=torch.uint8, device=device)
        torch.cuda.synchronize()

    def _i32(self, x):
        return torch.tensor(np.asarray(x), dtype=torch.int32, device=self.device)

    # -- where a row's K/V come from ---------------------------------------------------------------
    def _src(self, row):
        """(k_src, v_src, offset of the row's token 0, tokens held)"""
        if row < self.n_ext:
            return self.ext_k_src, self.ext_v_src, int(self.ext_src_off[row]), self.prefix[row] + self.extend[row]
        j = row - self.n_ext
        return self.dec_k_src, self.dec_v_src, int(self.dec_src_off[j]), self.ctx[j]

    def _append_ranges(self, ranges, slab_tokens=1 << 17):
        """kv_append of (row, lo, hi) token ranges, rows gathered from the source tensors (extend rows and decode rows
        in separate calls, in slabs that bound the temporary memory)."""
        for is_ext in (True, False):
            part = [(r, lo, hi) for r, lo, hi in ranges if (r < self.n_ext) == is_ext and hi > lo]
            while part:
                take, tok = [], 0
                while part and tok < slab_tokens:
                    take.append(part.pop()); tok += take[-1][2] - take[-1][1]
                k_src, v_src = (self.ext_k_src, self.ext_v_src) if is_ext else (self.dec_k_src, self.dec_v_src)
                idx = np.concatenate([np.arange(self._src(r)[2] + lo, self._src(r)[2] + hi) for r, lo, hi in take])
                idx_d = torch.from_numpy(idx).to(self.device)
                cu = np.concatenate([[0], np.cumsum([hi - lo for _, lo, hi in take])])
                kvattn.kv_append(self.pool, k_src.index_select(0, idx_d), v_src.index_select(0, idx_d), self._i32(cu),
                                 self._i32([lo for _, lo, _ in take]), self._i32([r for r, _, _ in take]), self.bt)
                torch.cuda.synchronize()

    # -- one step -----------------------------------------------------------------------------------
    def begin_step(self):
        """Draws this step's extend set, places it, writes the upstream operator's prefixes (not part of the step) and
        stages the step's new tokens: the extend suffixes followed by one token per decode sequence."""
        self.step_index += 1
        s, w, g, dev = self.step_index, self.w, self.geom, self.device
        n = self.n_ext
        self.prefix = [synth.uniform_int(self.seed, synth.TAG_LEN_A, 10_000 * (s + 1) + i, *w.prefix_range) for i in range(n)]
        self.extend = [synth.uniform_int(self.seed, synth.TAG_LEN_B, 10_000 * (s + 1) + i, *w.extend_range) for i in range(n)]
        self.ext_uids = [10_000 * (s + 1) + i for i in range(n)]
        L = [p + e for p, e in zip(self.prefix, self.extend)]
        self.ext_src_off = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
        self.ext_k_src = torch.cat([synth.normal_bf16(self.seed, synth.TAG_K, u, 0, l, g.n_kv_heads, g.head_dim, dev)
                                    for u, l in zip(self.ext_uids, L)])
        self.ext_v_src = torch.cat([synth.normal_bf16(self.seed, synth.TAG_V, u, 0, l, g.n_kv_heads, g.head_dim, dev)
                                    for u, l in zip(self.ext_uids, L)])
        for i in range(n):
            self.rows[i] = kvattn.kv_alloc(self.pool, synth.pages_needed(L[i], g.page_size))
            self.bt_host[i] = -1
            self.bt_host[i, :len(self.rows[i])] = self.rows[i]
        self.bt.copy_(torch.from_numpy(self.bt_host))
        self._append_ranges([(i, 0, self.prefix[i]) for i in range(n)])
        # the step's inputs
        self.q_ext = torch.cat([synth.normal_bf16(self.seed, synth.TAG_Q, self.ext_uids[i], self.prefix[i], self.extend[i],
                                                  g.n_q_heads, g.head_dim, dev) for i in range(n)])
        self.q_dec = torch.cat([synth.normal_bf16(self.seed, synth.TAG_Q, self.dec_uids[j], self.ctx[j], 1, g.n_q_heads,
                                                  g.head_dim, dev) for j in range(self.n_dec)])
        new_idx_e = np.concatenate([np.arange(self.ext_src_off[i] + self.prefix[i], self.ext_src_off[i + 1]) for i in range(n)])
        new_idx_d = np.asarray([self.dec_src_off[j] + self.ctx[j] for j in range(self.n_dec)])
        self.k_new = torch.cat([self.ext_k_src.index_select(0, torch.from_numpy(new_idx_e).to(dev)),
                                self.dec_k_src.index_select(0, torch.from_numpy(new_idx_d).to(dev))])
        self.v_new = torch.cat([self.ext_v_src.index_select(0, torch.from_numpy(new_idx_e).to(dev)),
                                self.dec_v_src.index_select(0, torch.from_numpy(new_idx_d).to(dev))])
        self.cu_new = self._i32(np.concatenate([[0], np.cumsum(self.extend + [1] * self.n_dec)]))
        self.start_new = self._i32(self.prefix + self.ctx)
        self.cu_q = self._i32(np.concatenate([[0], np.cumsum(self.extend)]))
        self.prefix_d, self.extend_d = self._i32(self.prefix), self._i32(self.extend)
        self.ctx_after = [c + 1 for c in self.ctx]
        self.ctx_d = self._i32(self.ctx_after)
        self.out_ext, self.out_dec = torch.empty_like(self.q_ext), torch.empty_like(self.q_dec)
        self.lse_ext = torch.empty((self.q_ext.shape[0], g.n_q_heads), dtype=torch.float32, device=dev)
        self.lse_dec = torch.empty((self.n_dec, g.n_q_heads), dtype=torch.float32, device=dev)
        torch.cuda.synchronize()

    def append_new(self, stream=None):
        """kv_append of the step's new tokens (sum of the extend lengths + one per decode sequence), one call."""
        kvattn.kv_append(self.pool, self.k_new, self.v_new, self.cu_new, self.start_new, None, self.bt, stream)

    def mixed(self, stream=None):
        g, n = self.geom, self.n_ext
        ea = kvattn.extend_args(self.q_ext, self.cu_q, self.bt[:n], self.prefix_d, self.extend_d, max(self.extend),
                                max(p + e for p, e in zip(self.prefix, self.extend)), self.out_ext, self.lse_ext)
        da = kvattn.decode_args(self.q_dec, self.bt[n:], self.ctx_d, max(self.ctx_after), self.out_dec, self.lse_dec)
        kvattn.attn_mixed(self.pool, g.n_q_heads, g.scale, ea, da, self.workspace, stream)

    def commit_new(self):
        """The decode sequences now hold one token more."""
        self.ctx = list(self.ctx_after)

    def live_blocks(self):
        """(row, logical block) of every page that holds tokens (call after commit_new)."""
        out = []
        for r in range(self.n_ext + self.n_dec):
            out += [(r, b) for b in range(synth.pages_needed(self._src(r)[3], self.geom.page_size))]
        return out

    def churn(self, fraction=0.2):
        """Evicts a seeded fraction of the live pages, takes as many new ones, and re-fills those logical blocks.
        Returns the number of pages that moved."""
        live = self.live_blocks()
        rng = np.random.default_rng(self.seed % (1 << 31) + self.step_index)
        pick = rng.choice(len(live), size=int(len(live) * fraction), replace=False)
        victims = [live[k] for k in pick]
        old = [self.rows[r][b] for r, b in victims]
        kvattn.kv_evict(self.pool, old)
        new = kvattn.kv_alloc(self.pool, len(old))                       # last-in-first-out: the same ids, another order
        new = [new[k] for k in rng.permutation(len(new))]
        for (r, b), pg in zip(victims, new):
            self.rows[r][b] = pg
            self.bt_host[r, b] = pg
        self.bt.copy_(torch.from_numpy(self.bt_host))
        self._append_ranges([(r, 16 * b, min(16 * b + 16, self._src(r)[3])) for r, b in victims])
        return len(old)

    def end_step(self):
        """The extend set's tuples leave the pipeline: their pages are released (Algorithm 1, Complete)."""
        for i in range(self.n_ext):
            kvattn.kv_free(self.pool, self.rows[i])
            self.rows[i] = []

    def source_bits(self, row):
        """K/V bit patterns of a row's tokens from the source tensors (the oracle's input)."""
        k_src, v_src, off, n = self._src(row)
        return synth.bf16_bits(k_src[off:off + n]), synth.bf16_bits(v_src[off:off + n])

    def step_new_tokens(self) -> int:
        return int(sum(self.extend)) + self.n_dec

    def close(self):
        torch.cuda.synchronize()
        status = kvattn.kv_last_async_status(self.pool)
        self.pool.destroy()
        if status != kvattn.KV_OK:
            raise kvattn.KvError(status, "device status at close")
