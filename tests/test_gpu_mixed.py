"""One pipeline step of two chained operators (extend set + decode set) with appends and page churn."""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, O_TOL, LSE_TOL, tight_ok
from oracle import paged_attention as orc

pytestmark = pytest.mark.gpu


def _mixed(dp, eb, P, E, db, C):
    """attn_mixed on the device; oracle extend + decode on the host."""
    g, dev = dp.geom, dp.device
    q_e = torch.cat([eb.q(i, P[i], P[i] + E[i]) for i in range(len(P))]).contiguous()
    q_d = torch.cat([db.q(i, C[i] - 1, C[i]) for i in range(len(C))]).contiguous()
    cu = np.concatenate([[0], np.cumsum(E)]).astype(np.int32)
    bt_e_np, bt_d_np = eb.block_tables(), db.block_tables()
    t = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
    bt_e, bt_d = torch.from_numpy(bt_e_np).to(dev), torch.from_numpy(bt_d_np).to(dev)
    cu_d, pl, el, cl = t(cu.tolist()), t(P), t(E), t(C)
    o_e, l_e = torch.full_like(q_e, float("nan")), torch.full((q_e.shape[0], g.n_q_heads), float("nan"), device=dev)
    o_d, l_d = torch.full_like(q_d, float("nan")), torch.full((len(C), g.n_q_heads), float("nan"), device=dev)
    max_l = max(p + e for p, e in zip(P, E))
    nbytes = kvattn.attn_workspace_bytes(dp.pool, g.n_q_heads, len(P), int(q_e.shape[0]), max_l, len(C), max(C))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    ea = kvattn.extend_args(q_e, cu_d, bt_e, pl, el, max(E), max_l, o_e, l_e)
    da = kvattn.decode_args(q_d, bt_d, cl, max(C), o_d, l_d)
    kvattn.attn_mixed(dp.pool, g.n_q_heads, g.scale, ea, da, ws)
    torch.cuda.synchronize()
    ref_e = orc.attn_extend(dp.host, synth.bf16_bits(q_e), g.n_q_heads, cu, bt_e_np, P, E, g.scale)
    ref_d = orc.attn_decode(dp.host, synth.bf16_bits(q_d), g.n_q_heads, bt_d_np, C, g.scale)
    return (o_e, l_e, o_d, l_d), (ref_e, ref_d)


def _check(got, ref, what):
    (o_e, l_e, o_d, l_d), (ref_e, ref_d) = got, ref
    for o, l, (ro, rl), name in ((o_e, l_e, ref_e, "extend"), (o_d, l_d, ref_d, "decode")):
        on, ln = o.float().cpu().numpy().astype(np.float64), l.cpu().numpy().astype(np.float64)
        assert not np.isnan(on).any() and not np.isnan(ln).any(), f"{what} {name}: NaN"
        assert np.max(np.abs(on - ro)) <= O_TOL and np.max(np.abs(ln - rl)) <= LSE_TOL, f"{what} {name}"
        assert tight_ok(on, ro) <= 1.0, f"{what} {name}: element-wise gate"


def test_pipeline_steps_with_appends_and_page_churn():
    # Scaled-down sem_map -> sem_filter step: extend sequences over reused prefixes plus decode sequences that
    # grow by one token per step; 20% of the live pages are evicted (poisoned), re-allocated and re-filled
    # between steps.  Attention over unchanged logical content must not change by a single bit.
    geom = synth.Geometry(32, 8, 128)
    dev = "cuda"
    dp = DualPool(geom, 2048, seed=404)
    kvattn.kv_pool_set_poison(dp.pool, True)
    rng = np.random.default_rng(404)
    n_ext, n_dec, steps = 6, 10, 3
    C = [int(c) for c in rng.integers(100, 1500, n_dec)]
    dec = Batch(dp, [c + steps for c in C], uid0=10_000)                   # room for the tokens to come
    dec.write([(i, 0, C[i]) for i in range(n_dec)])
    for step in range(steps):
        P = [int(p) for p in rng.integers(64, 900, n_ext)]
        E = [int(e) for e in rng.integers(8, 150, n_ext)]
        ext = Batch(dp, [p + e for p, e in zip(P, E)], uid0=1000 * (step + 1))
        ext.write([(i, 0, P[i]) for i in range(n_ext)])                     # upstream operator's prefill
        # this step's new tokens: extend suffixes and one decode token per sequence
        ext.write([(i, P[i], P[i] + E[i]) for i in range(n_ext)])
        dec.write([(i, C[i], C[i] + 1) for i in range(n_dec)])
        C = [c + 1 for c in C]
        got, ref = _mixed(dp, ext, P, E, dec, C)
        _check(got, ref, f"step {step}")
        # ---- churn: evict 20% of the live pages, take new ones, re-append the same logical blocks
        live = [(b, i, blk) for b, lens in ((ext, [p + e for p, e in zip(P, E)]), (dec, C))
                for i in range(len(b.rows)) for blk in range(synth.pages_needed(lens[i], 16))]
        pick = rng.choice(len(live), size=len(live) // 5, replace=False)
        victims = [live[k] for k in pick]
        old_pages = [b.rows[i][blk] for b, i, blk in victims]
        kvattn.kv_evict(dp.pool, old_pages)
        for pg in old_pages:
            dp.host.k[pg] = 0x7FC0; dp.host.v[pg] = 0x7FC0                  # the oracle's image forgets them too
        new_pages = kvattn.kv_alloc(dp.pool, len(old_pages))
        assert sorted(new_pages) == sorted(old_pages)                       # last-in-first-out: the same ids come back
        new_pages = [new_pages[k] for k in rng.permutation(len(new_pages))]
        for (b, i, blk), pg in zip(victims, new_pages):
            b.rows[i][blk] = pg
        for b, lens in ((ext, [p + e for p, e in zip(P, E)]), (dec, C)):
            ranges = [(i, 16 * blk, min(16 * blk + 16, lens[i])) for bb, i, blk in victims if bb is b]
            b.write(ranges)
        got2, ref2 = _mixed(dp, ext, P, E, dec, C)
        _check(got2, ref2, f"step {step} after churn")
        for a_, b_ in zip(got, got2):
            assert torch.equal(a_.view(torch.int32) if a_.dtype == torch.float32 else a_.view(torch.int16),
                               b_.view(torch.int32) if b_.dtype == torch.float32 else b_.view(torch.int16))
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    free, used, evicted = kvattn.kv_pool_stats(dp.pool)
    assert evicted > 0 and used == 2048
    dp.close()


def test_mixed_with_one_side_empty():
    geom = synth.Geometry(8, 2, 128)
    dp = DualPool(geom, 128, seed=5)
    b = Batch(dp, [200, 77])
    b.write([(0, 0, 200), (1, 0, 77)])
    dev = "cuda"
    t = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
    bt = torch.from_numpy(b.block_tables()).to(dev)
    q = torch.cat([b.q(0, 199, 200), b.q(1, 76, 77)]).contiguous()
    out, lse = torch.empty_like(q), torch.empty((2, 8), device=dev)
    ws = torch.empty(kvattn.attn_workspace_bytes(dp.pool, 8, 0, 0, 0, 2, 200), dtype=torch.uint8, device=dev)
    kvattn.attn_mixed(dp.pool, 8, geom.scale, None, kvattn.decode_args(q, bt, t([200, 77]), 200, out, lse), ws)
    torch.cuda.synchronize()
    ref_o, ref_l = orc.attn_decode(dp.host, synth.bf16_bits(q), 8, b.block_tables(), [200, 77], geom.scale)
    assert np.max(np.abs(out.float().cpu().numpy() - ref_o)) <= O_TOL
    kvattn.attn_mixed(dp.pool, 8, geom.scale, None, None, ws)               # nothing to do is fine
    dp.close()
