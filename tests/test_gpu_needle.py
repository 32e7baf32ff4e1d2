"""Indexing tests with O(1) outputs for the tensor-core extend path (attn_extend and attn_extend_shared).

With N(0,1) inputs and thousands of keys an output element is about 0.01, so a V tile taken from the wrong page,
a row of a 128-row tile that looks at the wrong head of its group, or a child that reads another child's keys
moves the output by less than the tolerance.  Here every row's answer is a value that names what was read:

* position-coded keys: key j carries three one-hot codes (j mod 32, j div 32 mod 32, j div 1024) scaled so that
  a query carrying the codes of its target j* scores 43 nats (62 binades) above every other key; the row's
  softmax is then one-hot on j* and O equals v_{j*} (to 1e-15);
* position-coded values: v_j of KV head g holds (j mod 256)/256, (j div 256)/64, g/8 and an owner code, all exact
  in bf16, so the output says which key, which KV head and whose pages were read;
* K == 0: every visible key weighs the same, O = mean of the visible values and LSE = ln(number of visible
  keys), which counts the keys each row sees (causal diagonal, ragged last page, empty prefix).

Every case is also compared with the oracle element by element.
"""
import numpy as np
import pytest
import torch

from oracle import paged_attention as orc
from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, assert_close, run_extend

pytestmark = pytest.mark.gpu

KAPPA = 22.0      # 22^2 * 128^-1/2 = 42.8 nats per matching code


def _codes(j, D):
    """The three code positions of key j inside a head of D dims (D/4 dims per code; the last quarter is unused)."""
    w = D // 4
    j = np.asarray(j)
    return j % w, w + (j // w) % w, 2 * w + (j // (w * w)) % w


def coded_keys(pos, n_kv_heads, D):
    """float32 [n][Hkv][D]: kappa at the three code positions of each key's position, the same for every KV head."""
    pos = np.asarray(pos)
    k = np.zeros((len(pos), n_kv_heads, D), np.float32)
    for c in _codes(pos, D):
        k[np.arange(len(pos)), :, c] = KAPPA
    return k


def coded_values(pos, n_kv_heads, D, owner):
    """float32 [n][Hkv][D]; d mod 4 selects: (j mod 256)/256, (j div 256)/64, g/8, owner/64.  All exact in bf16."""
    pos = np.asarray(pos)
    v = np.zeros((len(pos), n_kv_heads, D), np.float32)
    v[:, :, 0::4] = ((pos % 256) / 256.0)[:, None, None]
    v[:, :, 1::4] = ((pos // 256) / 64.0)[:, None, None]
    v[:, :, 2::4] = (np.arange(n_kv_heads) / 8.0)[None, :, None]
    v[:, :, 3::4] = (owner % 64) / 64.0
    return v


def target_of(seq, p, h, n_heads):
    """The key that query (sequence, absolute position p, head h) looks for: walks through the causal diagonal,
    the first KV tile, a middle tile, the start of the last KV tile, the last page boundary and a pseudo-random key."""
    kind = (p * n_heads + h + seq) % 6
    if kind == 0:
        return p                                   # itself: the causal diagonal
    if kind == 1:
        return (7 * p + 3 * h) % min(128, p + 1)   # first KV tile
    if kind == 2:
        return p // 2                              # a middle tile
    if kind == 3:
        return 128 * (p // 128)                    # first key of the last KV tile
    if kind == 4:
        return 16 * (p // 16)                      # first slot of the last page
    return (p * 2654435761 + h * 40503 + seq * 97) % (p + 1)


def bf(x):
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)


class CodedBatch(Batch):
    """Keys carry their position, values name (position, KV head, sequence); a query carries its target's codes.
    With zero_k the keys are all zero and the queries random (the K == 0 closed form)."""

    def __init__(self, dp, lengths, zero_k=False):
        super().__init__(dp, lengths)
        self.zero_k = zero_k

    def kv(self, i, lo, hi):
        g = self.dp.geom
        pos = np.arange(lo, hi)
        k = np.zeros((hi - lo, g.n_kv_heads, g.head_dim), np.float32) if self.zero_k else \
            coded_keys(pos, g.n_kv_heads, g.head_dim)
        return bf(k).to(self.dp.device), bf(coded_values(pos, g.n_kv_heads, g.head_dim, i)).to(self.dp.device)

    def q(self, i, lo, hi):
        g = self.dp.geom
        if self.zero_k:
            return super().q(i, lo, hi)
        q = np.zeros((hi - lo, g.n_q_heads, g.head_dim), np.float32)
        for t, p in enumerate(range(lo, hi)):
            for h in range(g.n_q_heads):
                for c in _codes(target_of(i, p, h, g.n_q_heads), g.head_dim):
                    q[t, h, c] = KAPPA
        return bf(q).to(self.dp.device)


def _expected_needle(geom, P, E):
    """bf16 bit patterns of v_{j*} for every (row, head) of the batch."""
    G = geom.group
    rows = []
    for i, (p0, e) in enumerate(zip(P, E)):
        for t in range(e):
            p = p0 + t
            tgt = np.array([target_of(i, p, h, geom.n_q_heads) for h in range(geom.n_q_heads)])
            v = coded_values(tgt, geom.n_kv_heads, geom.head_dim, i)          # [Hq][Hkv][D]
            rows.append(v[np.arange(geom.n_q_heads), np.arange(geom.n_q_heads) // G])
    return synth.bf16_bits(bf(np.stack(rows))) if rows else np.zeros((0, geom.n_q_heads, geom.head_dim), np.uint16)


def _needle_case(geom, P, E, impl, what):
    L = [p + e for p, e in zip(P, E)]
    dp = DualPool(geom, sum(synth.pages_needed(x, 16) for x in L) + 8, seed=7000 + len(P) + geom.n_q_heads)
    b = CodedBatch(dp, L)
    b.write([(i, 0, P[i]) for i in range(len(P))])                 # the upstream operator's pages
    b.write([(i, P[i], L[i]) for i in range(len(P))])              # the suffix
    res = run_extend(dp, b, P, E, impl=impl)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    assert_close(res, what)
    # every element of v[j*] is exact in bf16, and the other keys weigh less than 1e-15 together: the output equals
    # v[j*] (a zero element may come out as that residue instead of 0, hence the absolute bound and not the bits)
    want = orc.widen(_expected_needle(geom, P, E))
    bad = np.argwhere(np.abs(res["o"] - want) > 1e-6)
    assert bad.size == 0, f"{what}: {len(bad)} elements differ from v[j*]; first (row, head, dim) = {bad[0]}"
    # LSE = scale * 3 kappa^2 up to the weight of the other keys (< 1e-15)
    lse_want = 3 * KAPPA * KAPPA * geom.scale
    assert np.max(np.abs(res["lse"] - lse_want)) <= 1e-3, what
    dp.close()


GEOMS = [(4, 4, 128), (8, 2, 128), (8, 1, 128), (32, 8, 128), (4, 2, 64)]


@pytest.mark.parametrize("impl", [2, 1])
@pytest.mark.parametrize("hq,hkv,d", GEOMS)
def test_needle_short_edge_lengths(impl, hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    P = [0, 1, 15, 16, 17, 31, 32, 0, 100, 5, 130, 127, 128]
    E = [1, 2, 15, 16, 17, 33, 1, 70, 0, 129, 300, 129, 33]
    _needle_case(geom, P, E, impl, f"needle short impl{impl} {hq}/{hkv}/{d}")


@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 128), (8, 2, 128), (8, 1, 128), (16, 2, 128)])
def test_needle_long_sequences_use_the_long_sequence_kernel(hq, hkv, d):
    # a sequence of 4096 keys or more selects the kernel instantiation whose softmax does not look for the row maximum
    # after an item's first tile: the needle of most rows arrives tens of binades above everything seen before
    geom = synth.Geometry(hq, hkv, d)
    P = [4090, 5000, 37]
    E = [70, 129, 260]
    _needle_case(geom, P, E, 2, f"needle long {hq}/{hkv}/{d}")


@pytest.mark.parametrize("impl", [2, 1])
@pytest.mark.parametrize("hq,hkv,d", GEOMS)
def test_zero_keys_give_the_mean_of_the_visible_values(impl, hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    P = [0, 1, 15, 16, 17, 250, 4100 if d == 128 else 700, 129]
    E = [1, 33, 2, 129, 64, 140, 40, 257]
    L = [p + e for p, e in zip(P, E)]
    dp = DualPool(geom, sum(synth.pages_needed(x, 16) for x in L) + 8, seed=7100 + hq)
    b = CodedBatch(dp, L, zero_k=True)
    b.write([(i, 0, L[i]) for i in range(len(P))])
    res = run_extend(dp, b, P, E, impl=impl)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    assert_close(res, f"K=0 impl{impl}")
    # closed form, written out here from the values themselves: running mean of v over the visible keys, ln(count)
    G = geom.group
    r = 0
    for i in range(len(P)):
        v = coded_values(np.arange(L[i]), geom.n_kv_heads, geom.head_dim, i).astype(np.float64)
        run = np.cumsum(v, axis=0) / np.arange(1, L[i] + 1)[:, None, None]
        for t in range(E[i]):
            n = P[i] + t + 1
            want = run[n - 1][np.arange(geom.n_q_heads) // G]                         # [Hq][D]
            assert np.max(np.abs(res["o"][r] - want)) <= 2.0 ** -8 * 1.0 + 1e-4, (i, t)   # one bf16 rounding of O(1) values
            assert np.max(np.abs(res["lse"][r] - np.log(n))) <= 2e-5, (i, t, n)
            r += 1
    dp.close()


# ---------------------------------------------------------------------------------------------------------------
# attn_extend_shared: a row's target is either one of the parent's keys or one of its own child's keys
# ---------------------------------------------------------------------------------------------------------------
def _shared_target(c, t, h, P, n_heads):
    """(in_parent, index): parent's key index, or the child's own key index <= t."""
    kind = (t * n_heads + h + c) % 4
    if P > 0 and kind == 0:
        return True, (5 * t + 11 * h + c) % P
    if P > 0 and kind == 1:
        return True, P - 1 - ((t + h) % min(P, 16))                  # the parent's last page
    if kind == 2:
        return False, t                                              # itself
    return False, (3 * t + h) % (t + 1)


@pytest.mark.parametrize("impl", [1, 2])
@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 128), (8, 2, 128), (8, 1, 128)])
def test_needle_children_over_a_shared_parent(impl, hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    dev = "cuda"
    parent_lens = [48, 400, 0, 2144, 4112]          # the last one selects the long-sequence kernel
    n_child = [3, 5, 2, 4, 3]
    child_lens = [5, 1, 37, 16, 17, 0, 33, 130, 9, 2, 37, 36, 1, 64, 40, 3, 140]
    n_par, n_ch = len(parent_lens), len(child_lens)
    child_parent = np.repeat(np.arange(n_par), n_child)
    pages = sum(synth.pages_needed(x, 16) for x in parent_lens + child_lens)
    dp = DualPool(geom, pages + 8, seed=7200 + hq)
    # a child's own key t sits at coded position P + t, its values are owned by 32 + child (a parent's by its index)
    parents, children = Batch(dp, parent_lens), Batch(dp, child_lens)
    segs_p = [(g, 0) for g in range(n_par) if parent_lens[g] > 0]
    dp.append(parents.rows, segs_p,
              [bf(coded_keys(np.arange(parent_lens[g]), hkv, d)) for g, _ in segs_p],
              [bf(coded_values(np.arange(parent_lens[g]), hkv, d, g)) for g, _ in segs_p])
    segs_c = [(c, 0) for c in range(n_ch) if child_lens[c] > 0]
    dp.append(children.rows, segs_c,
              [bf(coded_keys(parent_lens[child_parent[c]] + np.arange(child_lens[c]), hkv, d)) for c, _ in segs_c],
              [bf(coded_values(parent_lens[child_parent[c]] + np.arange(child_lens[c]), hkv, d, 32 + c)) for c, _ in segs_c])
    q_rows, want_rows = [], []
    for c in range(n_ch):
        P = parent_lens[child_parent[c]]
        for t in range(child_lens[c]):
            q = np.zeros((hq, d), np.float32)
            want = np.zeros((hq, d), np.float32)
            for h in range(hq):
                in_parent, idx = _shared_target(c, t, h, P, hq)
                pos = idx if in_parent else P + idx
                for cd in _codes(pos, d):
                    q[h, cd] = KAPPA
                want[h] = coded_values([pos], hkv, d, child_parent[c] if in_parent else 32 + c)[0, h // geom.group]
            q_rows.append(q); want_rows.append(want)
    q = bf(np.stack(q_rows)).to(dev).contiguous()
    cu_children = np.concatenate([[0], np.cumsum(n_child)]).astype(np.int32)
    cu_q = np.concatenate([[0], np.cumsum(child_lens)]).astype(np.int32)
    i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=dev)
    pt_np, ct_np = parents.block_tables(), children.block_tables()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], hq), float("nan"), dtype=torch.float32, device=dev)
    rows_per_parent = [int(cu_q[cu_children[g + 1]] - cu_q[cu_children[g]]) for g in range(n_par)]
    ws = torch.empty(max(256, kvattn.attn_extend_shared_workspace_bytes(dp.pool, hq, n_par, n_ch, int(q.shape[0]),
                                                                        max(parent_lens))), dtype=torch.uint8, device=dev)
    kvattn.kvattn_set_shared_impl(impl)
    try:
        kvattn.attn_extend_shared(dp.pool, q, i32(cu_q), i32(cu_children), i32(pt_np), i32(parent_lens), i32(ct_np),
                                  i32(child_lens), max(child_lens), max(rows_per_parent), max(parent_lens), geom.scale,
                                  out, lse, ws)
    finally:
        kvattn.kvattn_set_shared_impl(0)
    torch.cuda.synchronize()
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    o_ref, l_ref = orc.attn_extend_shared(dp.host, synth.bf16_bits(q), hq, cu_q, cu_children, pt_np, parent_lens, ct_np,
                                          child_lens, geom.scale)
    res = {"o": out.float().cpu().numpy().astype(np.float64), "lse": lse.cpu().numpy().astype(np.float64),
           "o_ref": o_ref, "lse_ref": l_ref}
    assert_close(res, f"shared needle impl{impl}")
    bad = np.argwhere(np.abs(res["o"] - np.stack(want_rows).astype(np.float64)) > 1e-6)
    assert bad.size == 0, f"shared needle impl{impl}: {len(bad)} elements differ from v[j*]; first = {bad[0]}"
    dp.close()
