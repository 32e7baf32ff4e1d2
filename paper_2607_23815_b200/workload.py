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
