"""Test harness: keeps a device pool (through the C ABI) and the oracle's host pool in lockstep.

The harness plays the out-of-scope scheduler/engine: it owns block tables, decides which physical
page backs which logical block (a seeded permutation of the pool), draws inputs from synth, feeds
the same bits to both sides, and compares results.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np
import torch

from oracle import paged_attention as orc
from paper_2607_23815_b200 import kvattn, synth

NAN_BITS = 0x7FC0
O_TOL = 2e-2      # max |delta| on bf16 outputs (the stated bound)
LSE_TOL = 1e-3    # max |delta| on fp32 LSE (the stated bound)


def tight_ok(o_gpu: np.ndarray, o_ref: np.ndarray) -> float:
    """Worst ratio of |delta| to the tighter element-wise gate 4e-3 + 2^-6 |ref| (<= 1 passes).

    bf16 rounding of O alone is 2^-9 |ref|; the rest comes from P rounded to bf16 before PV.
    """
    gate = 4e-3 + (2.0 ** -6) * np.abs(o_ref)
    return float(np.max(np.abs(o_gpu - o_ref) / gate)) if o_ref.size else 0.0


class DualPool:
    def __init__(self, geom: synth.Geometry, num_pages: int, seed: int, device="cuda", fill=NAN_BITS,
                 with_oracle=True):
        self.geom, self.num_pages, self.seed, self.device = geom, num_pages, seed, device
        self.gen_device = "cpu"         # the input generator runs on the host, so that nearly every kernel a test launches is the library's
        n_elem = num_pages * geom.n_kv_heads * geom.page_size * geom.head_dim
        # caller-owned buffers, pre-filled (NaN by default) so that any stale read shows up
        self.k_buf = torch.full((n_elem,), fill, dtype=torch.int16, device=device)
        self.v_buf = torch.full((n_elem,), fill, dtype=torch.int16, device=device)
        self.pool = kvattn.kv_pool_create_ex(num_pages, geom.page_size, geom.n_kv_heads, geom.head_dim,
                                             self.k_buf, self.v_buf)
        self.host = orc.PagePool(num_pages, geom.page_size, geom.n_kv_heads, geom.head_dim, fill=fill) \
            if with_oracle else None
        ids = kvattn.kv_alloc(self.pool, num_pages)            # the harness manages placement itself
        assert ids == list(range(num_pages))
        self.placement = synth.page_permutation(seed, num_pages).tolist()
        self.cursor = 0

    def take_pages(self, n: int) -> List[int]:
        assert self.cursor + n <= self.num_pages, "test pool too small"
        out = self.placement[self.cursor:self.cursor + n]
        self.cursor += n
        return out

    def append(self, rows: Sequence[Sequence[int]], segs, k_list, v_list):
        """segs: list of (row_index, start_pos); k_list/v_list: bf16 tensors [n][Hkv][D] per segment."""
        dev = self.device
        bt = torch.from_numpy(synth.block_table([list(r) for r in rows])).to(dev)
        lens = [int(k.shape[0]) for k in k_list]
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=dev)
        start = torch.tensor([s for _, s in segs], dtype=torch.int32, device=dev)
        seg_row = torch.tensor([r for r, _ in segs], dtype=torch.int32, device=dev)
        k_all = torch.cat([k.to(dev) for k in k_list]).contiguous()
        v_all = torch.cat([v.to(dev) for v in v_list]).contiguous()
        if k_all.shape[0] > 0:
            kvattn.kv_append(self.pool, k_all, v_all, cu, start, seg_row, bt)
        if self.host is not None:
            for (r, s), k, v in zip(segs, k_list, v_list):
                self.host.append(rows[r], s, synth.bf16_bits(k), synth.bf16_bits(v))

    def device_image(self):
        """Device K and V buffers un-swizzled to the logical layout [page][head][slot][dim] (uint16).

        The mapping is written out here from the documented formula, independently of the library.
        """
        g = self.geom
        D, ps = g.head_dim, g.page_size
        slot = np.arange(ps)[:, None]
        d = np.arange(D)[None, :]
        off = ((slot // 8) * (8 * D * 2) + (d // 64) * 1024 + (slot % 8) * 128
               + ((((d % 64) // 8) ^ (slot % 8)) * 16) + (d % 8) * 2) // 2          # element offset in a block
        out = []
        for buf in (self.k_buf, self.v_buf):
            raw = buf.cpu().numpy().view(np.uint16).reshape(self.num_pages, g.n_kv_heads, ps * D)
            out.append(raw[:, :, off.reshape(-1)].reshape(self.num_pages, g.n_kv_heads, ps, D))
        return out

    def close(self):
        torch.cuda.synchronize()
        self.pool.destroy()


class Batch:
    """A batch of sequences with K/V in a DualPool, Q drawn per sequence."""

    def __init__(self, dp: DualPool, lengths: Sequence[int], uid0: int = 0):
        self.dp = dp
        g = dp.geom
        self.lengths = list(lengths)
        self.uids = [uid0 + i for i in range(len(lengths))]
        self.rows = [dp.take_pages(synth.pages_needed(L, g.page_size)) for L in lengths]

    def kv(self, i: int, lo: int, hi: int):
        g, dp = self.dp.geom, self.dp
        k = synth.normal_bf16(dp.seed, synth.TAG_K, self.uids[i], lo, hi - lo, g.n_kv_heads, g.head_dim, dp.gen_device)
        v = synth.normal_bf16(dp.seed, synth.TAG_V, self.uids[i], lo, hi - lo, g.n_kv_heads, g.head_dim, dp.gen_device)
        return k.to(dp.device), v.to(dp.device)

    def q(self, i: int, lo: int, hi: int):
        g, dp = self.dp.geom, self.dp
        return synth.normal_bf16(dp.seed, synth.TAG_Q, self.uids[i], lo, hi - lo, g.n_q_heads, g.head_dim,
                                 dp.gen_device).to(dp.device)

    def write(self, ranges):
        """ranges: list of (seq index, lo, hi): append tokens lo..hi-1 of those sequences."""
        segs, ks, vs = [], [], []
        for i, lo, hi in ranges:
            if hi <= lo:
                continue
            k, v = self.kv(i, lo, hi)
            segs.append((i, lo)); ks.append(k); vs.append(v)
        if segs:
            self.dp.append(self.rows, segs, ks, vs)

    def block_tables(self, max_pages=None):
        return synth.block_table(self.rows, max_pages)


def run_extend(dp: DualPool, batch: Batch, prefix_lens, extend_lens, impl=0, oracle=True, workspace=None):
    """attn_extend on the device and (optionally) the oracle; returns dict of numpy results."""
    g, dev = dp.geom, dp.device
    B = len(prefix_lens)
    qs = [batch.q(i, prefix_lens[i], prefix_lens[i] + extend_lens[i]) for i in range(B)]
    q = torch.cat(qs).contiguous() if qs else torch.empty((0, g.n_q_heads, g.head_dim), dtype=torch.bfloat16, device=dev)
    cu = np.concatenate([[0], np.cumsum(extend_lens)]).astype(np.int32)
    bt_np = batch.block_tables()
    bt = torch.from_numpy(bt_np).to(dev)
    pl = torch.tensor(prefix_lens, dtype=torch.int32, device=dev)
    el = torch.tensor(extend_lens, dtype=torch.int32, device=dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], g.n_q_heads), float("nan"), dtype=torch.float32, device=dev)
    max_e = max(extend_lens) if B else 0
    max_l = max([p + e for p, e in zip(prefix_lens, extend_lens)]) if B else 0
    nbytes = kvattn.attn_workspace_bytes(dp.pool, g.n_q_heads, B, int(q.shape[0]), max_l, 0, 0)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev) if workspace is None else workspace
    kvattn.kvattn_set_extend_impl(impl)
    try:
        kvattn.attn_extend(dp.pool, q, torch.from_numpy(cu).to(dev), bt, pl, el, max_e, max_l, g.scale, out, lse, ws)
    finally:
        kvattn.kvattn_set_extend_impl(0)
    torch.cuda.synchronize()
    res = {"o": out.float().cpu().numpy().astype(np.float64), "lse": lse.cpu().numpy().astype(np.float64),
           "o_bits": synth.bf16_bits(out), "lse_raw": lse.cpu().numpy().copy(), "q": q, "cu": cu}
    if oracle:
        o_ref, l_ref = orc.attn_extend(dp.host, synth.bf16_bits(q), g.n_q_heads, cu, bt_np, prefix_lens, extend_lens,
                                       g.scale)
        res["o_ref"], res["lse_ref"] = o_ref, l_ref
    return res


def run_decode(dp: DualPool, batch: Batch, ctx_lens, oracle=True):
    g, dev = dp.geom, dp.device
    B = len(ctx_lens)
    qs = [batch.q(i, max(ctx_lens[i] - 1, 0), max(ctx_lens[i] - 1, 0) + 1) for i in range(B)]
    q = torch.cat(qs).contiguous()
    bt_np = batch.block_tables()
    bt = torch.from_numpy(bt_np).to(dev)
    cl = torch.tensor(ctx_lens, dtype=torch.int32, device=dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((B, g.n_q_heads), float("nan"), dtype=torch.float32, device=dev)
    max_c = max(max(ctx_lens), 0)
    nbytes = kvattn.attn_workspace_bytes(dp.pool, g.n_q_heads, 0, 0, 0, B, max_c)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
    kvattn.attn_decode(dp.pool, q, bt, cl, max_c, g.scale, out, lse, ws)
    torch.cuda.synchronize()
    res = {"o": out.float().cpu().numpy().astype(np.float64), "lse": lse.cpu().numpy().astype(np.float64),
           "o_bits": synth.bf16_bits(out), "lse_raw": lse.cpu().numpy().copy(), "q": q}
    if oracle:
        o_ref, l_ref = orc.attn_decode(dp.host, synth.bf16_bits(q), g.n_q_heads, bt_np, ctx_lens, g.scale)
        res["o_ref"], res["lse_ref"] = o_ref, l_ref
    return res


def assert_close(res, what=""):
    o, o_ref, lse, lse_ref = res["o"], res["o_ref"], res["lse"], res["lse_ref"]
    assert not np.isnan(o).any(), f"{what}: NaN in O"
    finite = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), np.isneginf(lse_ref)), f"{what}: -inf pattern of LSE differs"
    d_o = float(np.max(np.abs(o - o_ref))) if o.size else 0.0
    d_l = float(np.max(np.abs(lse[finite] - lse_ref[finite]))) if finite.any() else 0.0
    t = tight_ok(o, o_ref)
    assert d_o <= O_TOL, f"{what}: max|dO| = {d_o:.3e} > {O_TOL}"
    assert d_l <= LSE_TOL, f"{what}: max|dLSE| = {d_l:.3e} > {LSE_TOL}"
    assert t <= 1.0, f"{what}: element-wise gate exceeded by {t:.2f}x (max|dO| {d_o:.3e})"
    return d_o, d_l, t
