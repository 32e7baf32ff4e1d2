"""attn_extend_shared (children over a parent's pages) through the C ABI against the oracle and against
attn_extend on aliased block tables."""
import numpy as np
import pytest
import torch

from oracle import paged_attention as orc
from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, assert_close

pytestmark = pytest.mark.gpu


def _run_shared(geom, parent_lens, n_child, child_lens, seed, also_aliased=True, impl=0):
    """Parents and children on one pool; returns device result, oracle result, and attn_extend on aliased tables."""
    dev = "cuda"
    ps = geom.page_size
    n_par, n_ch = len(parent_lens), len(child_lens)
    pages = sum(synth.pages_needed(L, ps) for L in parent_lens) + sum(synth.pages_needed(E, ps) for E in child_lens)
    dp = DualPool(geom, pages + 8, seed=seed)
    parents = Batch(dp, parent_lens, uid0=0)
    parents.write([(g, 0, parent_lens[g]) for g in range(n_par)])
    children = Batch(dp, child_lens, uid0=1000)
    children.write([(c, 0, child_lens[c]) for c in range(n_ch)])
    cu_children = np.concatenate([[0], np.cumsum(n_child)]).astype(np.int32)
    cu_q = np.concatenate([[0], np.cumsum(child_lens)]).astype(np.int32)
    qs = [children.q(c, 0, child_lens[c]) for c in range(n_ch) if child_lens[c] > 0]
    q = torch.cat(qs).contiguous()
    pt_np, ct_np = parents.block_tables(), children.block_tables()
    i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=dev)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], geom.n_q_heads), float("nan"), dtype=torch.float32, device=dev)
    rows_per_parent = [int(cu_q[cu_children[g + 1]] - cu_q[cu_children[g]]) for g in range(n_par)]
    ws = torch.empty(max(256, kvattn.attn_extend_shared_workspace_bytes(dp.pool, geom.n_q_heads, n_par, n_ch, int(q.shape[0]),
                                                                        max(parent_lens))), dtype=torch.uint8, device=dev)
    kvattn.kvattn_set_shared_impl(impl)
    try:
        kvattn.attn_extend_shared(dp.pool, q, i32(cu_q), i32(cu_children), i32(pt_np), i32(parent_lens), i32(ct_np),
                                  i32(child_lens), max(child_lens), max(rows_per_parent), max(parent_lens), geom.scale, out,
                                  lse, ws)
    finally:
        kvattn.kvattn_set_shared_impl(0)
    torch.cuda.synchronize()
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    o_ref, l_ref = orc.attn_extend_shared(dp.host, synth.bf16_bits(q), geom.n_q_heads, cu_q, cu_children, pt_np, parent_lens,
                                          ct_np, child_lens, geom.scale)
    res = {"o": out.float().cpu().numpy().astype(np.float64), "lse": lse.cpu().numpy().astype(np.float64),
           "o_ref": o_ref, "lse_ref": l_ref}
    if also_aliased:
        # the same children as independent sequences whose block tables start with the parent's pages
        child_parent = np.repeat(np.arange(n_par), n_child)
        rows = [list(parents.rows[g][:parent_lens[g] // ps]) + list(children.rows[c]) for c, g in enumerate(child_parent)]
        bt = i32(synth.block_table(rows))
        pl = [parent_lens[g] for g in child_parent]
        max_total = max(p_ + e_ for p_, e_ in zip(pl, child_lens))
        out2, lse2 = torch.full_like(q, float("nan")), torch.full_like(lse, float("nan"))
        ws2 = torch.empty(max(256, kvattn.attn_workspace_bytes(dp.pool, geom.n_q_heads, n_ch, int(q.shape[0]),
                                                               max_total, 0, 0)), dtype=torch.uint8, device=dev)
        kvattn.attn_extend(dp.pool, q, i32(cu_q), bt, i32(pl), i32(child_lens), max(child_lens), max_total, geom.scale,
                           out2, lse2, ws2)
        torch.cuda.synchronize()
        res["o_alias"] = out2.float().cpu().numpy().astype(np.float64)
        res["lse_alias"] = lse2.cpu().numpy().astype(np.float64)
    dp.close()
    return res


IMPLS = [1, 2]   # 1 = shared part / own part / merge, 2 = one kernel walking parent and children tiles


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("hq,hkv,d", [(32, 8, 128), (4, 2, 64), (8, 1, 128), (4, 4, 64)])
def test_shared_prefix_children_match_the_oracle(impl, hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    # parents with page-multiple prefixes (one of them empty), 0..5 children each, ragged suffixes (one empty)
    parent_lens = [48, 400, 0, 16, 2144]
    n_child = [3, 5, 2, 0, 4]
    child_lens = [5, 1, 37, 16, 17, 0, 33, 130, 9, 2, 37, 36, 1, 64]
    res = _run_shared(geom, parent_lens, n_child, child_lens, seed=900 + hq + d, impl=impl)
    assert_close(res, f"shared impl{impl} {hq}/{hkv}/{d}")
    # and it agrees with the independent-sequences path on aliased block tables (both are bf16 results)
    assert np.max(np.abs(res["o"] - res["o_alias"])) <= 2e-2
    assert np.max(np.abs(res["lse"] - res["lse_alias"])) <= 1e-3


@pytest.mark.parametrize("impl", IMPLS)
def test_parent_lengths_need_not_be_page_multiples(impl):
    # the children's keys come from their own pages, so the parent may end anywhere inside a page
    geom = synth.Geometry(32, 8, 128)
    res = _run_shared(geom, [37, 301, 129], [2, 3, 1], [40, 7, 33, 64, 1, 200], seed=931, also_aliased=False, impl=impl)
    assert_close(res, f"ragged parents impl{impl}")


@pytest.mark.parametrize("impl", IMPLS)
def test_many_short_children_per_tile(impl):
    # suffixes of 1..6 tokens: dozens of children share one query tile, some of them empty
    geom = synth.Geometry(8, 2, 128)
    rng = np.random.default_rng(23)
    n_child = [40, 1, 25]
    child_lens = rng.integers(0, 7, size=sum(n_child)).tolist()
    child_lens[0] = 3
    res = _run_shared(geom, [160, 0, 1024], n_child, child_lens, seed=923, impl=impl)
    assert_close(res, f"short children impl{impl}")


@pytest.mark.parametrize("impl", IMPLS)
def test_fanout_workload_shape(impl):
    # a slice of the fan-out workload: 3 parents x 17 children, prefix 2144, suffixes around 37
    geom = synth.Geometry(32, 8, 128)
    rng = np.random.default_rng(17)
    parent_lens = [2144, 2080, 2208]
    n_child = [17, 17, 17]
    child_lens = rng.integers(30, 45, size=51).tolist()
    res = _run_shared(geom, parent_lens, n_child, child_lens, seed=917, also_aliased=False, impl=impl)
    assert_close(res, f"fan-out slice impl{impl}")


@pytest.mark.parametrize("impl", IMPLS)
def test_long_parents_use_the_long_sequence_kernel(impl):
    # parents of 4096 tokens and more select the kernel variant that does not search for the row maximum after an
    # item's first tile; one parent is empty, so its children's rows see nothing until their own tile arrives
    geom = synth.Geometry(16, 4, 128)
    rng = np.random.default_rng(41)
    parent_lens = [4400, 0, 4112]
    n_child = [6, 3, 9]
    child_lens = rng.integers(1, 70, size=18).tolist()
    res = _run_shared(geom, parent_lens, n_child, child_lens, seed=941, impl=impl)
    assert_close(res, f"long parents impl{impl}")
    assert np.max(np.abs(res["o"] - res["o_alias"])) <= 2e-2
    assert np.max(np.abs(res["lse"] - res["lse_alias"])) <= 1e-3
