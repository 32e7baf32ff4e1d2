"""Seeded random batch shapes: the tensor-core extend kernel and the small-tile kernel on the same device pool, each
against the oracle and against each other; the two ways attn_extend_shared can run, likewise."""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from oracle import paged_attention as orc
from harness import Batch, DualPool, LSE_TOL, O_TOL, assert_close, run_extend

pytestmark = pytest.mark.gpu
GEOMS = [(32, 8, 128), (8, 8, 128), (16, 8, 64), (8, 1, 128), (4, 2, 64), (64, 8, 128)]


@pytest.mark.parametrize("seed", range(8))
def test_random_batches_tensor_core_vs_small_tile(seed):
    rng = np.random.default_rng(4000 + seed)
    hq, hkv, d = GEOMS[seed % len(GEOMS)]
    geom = synth.Geometry(hq, hkv, d)
    B = int(rng.integers(1, 40))
    kind = seed % 4
    if kind == 0:
        P, E = rng.integers(0, 600, size=B), rng.integers(0, 70, size=B)
    elif kind == 1:
        P, E = rng.integers(0, 40, size=B), rng.integers(1, 400, size=B)
    elif kind == 2:
        P, E = rng.integers(100, 3000, size=B), rng.integers(1, 20, size=B)
    else:
        P, E = rng.integers(0, 300, size=B) * (rng.random(B) < 0.5), rng.integers(0, 300, size=B)
    P, E = [int(x) for x in P], [int(x) for x in E]
    if sum(E) == 0:
        E[0] = 1
    pages = sum(synth.pages_needed(p + e, 16) for p, e in zip(P, E)) + 4
    dp = DualPool(geom, pages, seed=4100 + seed)
    b = Batch(dp, [p + e for p, e in zip(P, E)])
    b.write([(i, 0, P[i] + E[i]) for i in range(B)])
    tc = run_extend(dp, b, P, E, impl=2)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    assert_close(tc, f"random batch {seed}, tensor-core kernel")
    small = run_extend(dp, b, P, E, impl=1, oracle=False)
    small["o_ref"], small["lse_ref"] = tc["o_ref"], tc["lse_ref"]
    assert_close(small, f"random batch {seed}, small-tile kernel")
    assert np.max(np.abs(tc["o"] - small["o"])) <= O_TOL
    assert np.max(np.abs(tc["lse"] - small["lse"])) <= LSE_TOL
    dp.close()


@pytest.mark.parametrize("seed", range(6))
def test_random_fan_outs_one_kernel_vs_three(seed):
    rng = np.random.default_rng(4200 + seed)
    hq, hkv, d = GEOMS[seed % 5]
    geom = synth.Geometry(hq, hkv, d)
    n_par = int(rng.integers(1, 8))
    parent_lens = [int(x) for x in rng.integers(0, 1500, size=n_par)]
    n_child = [int(x) for x in rng.integers(0, 25, size=n_par)]
    if sum(n_child) == 0:
        n_child[0] = 3
    mx = [3, 50, 300][seed % 3]
    child_lens = [int(x) for x in rng.integers(0, mx + 1, size=sum(n_child))]
    if sum(child_lens) == 0:
        child_lens[0] = 2
    pages = sum(synth.pages_needed(L, 16) for L in parent_lens + child_lens) + 8
    dp = DualPool(geom, pages, seed=4300 + seed)
    parents = Batch(dp, parent_lens, uid0=0)
    parents.write([(g, 0, parent_lens[g]) for g in range(n_par)])
    children = Batch(dp, child_lens, uid0=1000)
    children.write([(c, 0, child_lens[c]) for c in range(len(child_lens))])
    cu_children = np.concatenate([[0], np.cumsum(n_child)]).astype(np.int32)
    cu_q = np.concatenate([[0], np.cumsum(child_lens)]).astype(np.int32)
    q = torch.cat([children.q(c, 0, child_lens[c]) for c in range(len(child_lens)) if child_lens[c] > 0]).contiguous()
    i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device="cuda")
    rows = [int(cu_q[cu_children[g + 1]] - cu_q[cu_children[g]]) for g in range(n_par)]
    ws = torch.empty(max(256, kvattn.attn_extend_shared_workspace_bytes(dp.pool, hq, n_par, len(child_lens), int(q.shape[0]),
                                                                        max(parent_lens))), dtype=torch.uint8, device="cuda")
    res = {}
    for impl in (1, 2):
        out = torch.full_like(q, float("nan"))
        lse = torch.full((q.shape[0], hq), float("nan"), dtype=torch.float32, device="cuda")
        kvattn.kvattn_set_shared_impl(impl)
        try:
            kvattn.attn_extend_shared(dp.pool, q, i32(cu_q), i32(cu_children), i32(parents.block_tables()), i32(parent_lens),
                                      i32(children.block_tables()), i32(child_lens), max(child_lens), max(rows),
                                      max(parent_lens), geom.scale, out, lse, ws)
        finally:
            kvattn.kvattn_set_shared_impl(0)
        torch.cuda.synchronize()
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
        res[impl] = (out.float().cpu().numpy(), lse.cpu().numpy())
    o_ref, l_ref = orc.attn_extend_shared(dp.host, synth.bf16_bits(q), hq, cu_q, cu_children, parents.block_tables(),
                                          parent_lens, children.block_tables(), child_lens, geom.scale)
    for impl in (1, 2):
        assert_close({"o": res[impl][0].astype(np.float64), "lse": res[impl][1].astype(np.float64), "o_ref": o_ref,
                      "lse_ref": l_ref}, f"random fan-out {seed}, impl {impl}")
    assert not np.isnan(res[2][0]).any() and not np.isnan(res[1][0]).any()
    assert np.max(np.abs(res[2][0] - res[1][0])) <= O_TOL
    assert np.max(np.abs(res[2][1] - res[1][1])) <= LSE_TOL
    dp.close()
