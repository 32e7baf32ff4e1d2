"""Pins for the CPU oracle: what the paper and the mathematics fix.

Each test would fail for a plausible mistake in oracle/paged_attention.py (a
dropped term, a wrong sign or index, a transposed operand, an off-by-one in the
causal boundary, a wrong head mapping, a wrong page/slot computation).
None of them touches the CUDA path.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import paged_attention as orc
from paper_2607_23815_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bits(rng, shape):
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    return synth.bf16_bits(x)


# ---------------------------------------------------------------- closed forms
def test_hand_worked_example():
    # D=2, scale=1/sqrt(2), q=(1,0); k0=(0,0), k1=(sqrt2*ln2, 0): scores (0, ln2)
    # -> weights (1/3, 2/3); v0=(3,0), v1=(0,3) -> O=(1,2), LSE=ln 3.
    q = np.array([[1.0, 0.0]])
    k = np.array([[0.0, 0.0], [math.sqrt(2.0) * math.log(2.0), 0.0]])
    v = np.array([[3.0, 0.0], [0.0, 3.0]])
    o, lse = orc.attention_rows(q, k, v, np.array([2]), 1.0 / math.sqrt(2.0))
    assert np.allclose(o, [[1.0, 2.0]], atol=1e-14)
    assert abs(lse[0] - math.log(3.0)) < 1e-14
    p, _ = orc.softmax_rows(q, k, np.array([2]), 1.0 / math.sqrt(2.0))
    assert np.allclose(p, [[1 / 3, 2 / 3]], atol=1e-15)
    # the second key hidden: the only visible key takes all the weight
    o1, lse1 = orc.attention_rows(q, k, v, np.array([1]), 1.0 / math.sqrt(2.0))
    assert np.allclose(o1, [[3.0, 0.0]]) and abs(lse1[0]) < 1e-15


def _brute(q, k, v, visible, scale):
    """Second, independently written evaluation: explicit exp(s_j)/sum_k exp(s_k), python loops."""
    R, D = len(q), len(q[0])
    O = [[0.0] * D for _ in range(R)]
    LSE = [0.0] * R
    for r in range(R):
        ws = []
        for j in range(visible[r]):
            dot = 0.0
            for d in range(D):
                dot += q[r][d] * k[j][d]
            ws.append(math.exp(scale * dot))
        tot = sum(ws)
        for j, w in enumerate(ws):
            for d in range(D):
                O[r][d] += (w / tot) * v[j][d]
        LSE[r] = math.log(tot)
    return np.array(O), np.array(LSE)


@pytest.mark.parametrize("L,D,R", [(1, 1, 1), (2, 3, 2), (4, 4, 3), (7, 2, 5), (13, 8, 4)])
def test_brute_force_tiny(L, D, R):
    rng = np.random.default_rng(100 + L * 10 + D)
    q, k, v = rng.standard_normal((R, D)), rng.standard_normal((L, D)), rng.standard_normal((L, D))
    visible = rng.integers(1, L + 1, size=R)
    o, lse = orc.attention_rows(q, k, v, visible, 0.7)
    ob, lb = _brute(q.tolist(), k.tolist(), v.tolist(), visible.tolist(), 0.7)
    assert np.max(np.abs(o - ob)) < 1e-13 and np.max(np.abs(lse - lb)) < 1e-13


def test_probability_rows_sum_to_one_and_outputs_are_convex():
    rng = np.random.default_rng(7)
    q, k, v = rng.standard_normal((9, 16)), 3.0 * rng.standard_normal((50, 16)), rng.standard_normal((50, 16))
    visible = np.array([1, 2, 5, 16, 17, 31, 32, 49, 50])
    p, lse = orc.softmax_rows(q, k, visible, 0.25)
    assert np.max(np.abs(p.sum(axis=1) - 1.0)) < 1e-12
    for r, n in enumerate(visible):
        assert np.all(p[r, n:] == 0.0) and np.all(p[r, :n] > 0.0)
    o, _ = orc.attention_rows(q, k, v, visible, 0.25)
    for r, n in enumerate(visible):
        assert np.all(o[r] <= v[:n].max(axis=0) + 1e-12) and np.all(o[r] >= v[:n].min(axis=0) - 1e-12)


def _build_pool(rng, lens, Hkv, D, ps=16, num_pages=64, perm_seed=3, fill=0x7FC0):
    """Pool with sequences of the given lengths on permuted pages; unwritten slots hold NaN bits."""
    pool = orc.PagePool(num_pages, ps, Hkv, D, fill=fill)
    perm = synth.page_permutation(perm_seed, num_pages).tolist()
    rows, kv = [], []
    for L in lens:
        n = synth.pages_needed(L, ps)
        pages, perm = perm[:n], perm[n:]
        k, v = _rand_bits(rng, (L, Hkv, D)), _rand_bits(rng, (L, Hkv, D))
        pool.append(pages, 0, k, v)
        rows.append(pages)
        kv.append((k, v))
    return pool, rows, kv


@pytest.mark.parametrize("P,E", [(0, 1), (0, 17), (1, 1), (15, 2), (16, 16), (17, 15), (31, 33), (32, 1)])
def test_zero_keys_closed_form(P, E):
    # K == 0: every score is 0, so row t is the mean of v_0..v_{P+t} and LSE = ln(P+t+1):
    # checks each row's visible-key count, partial pages included.
    rng = np.random.default_rng(P * 100 + E)
    Hq, Hkv, D, ps = 4, 2, 8, 16
    L = P + E
    pool = orc.PagePool(16, ps, Hkv, D, fill=0x7FC0)                # NaN everywhere
    pages = synth.page_permutation(5, 16).tolist()[:synth.pages_needed(L, ps)]
    v = _rand_bits(rng, (L, Hkv, D))
    pool.append(pages, 0, np.zeros((L, Hkv, D), np.uint16), v)
    q = _rand_bits(rng, (E, Hq, D))
    o, lse = orc.attn_extend(pool, q, Hq, [0, E], synth.block_table([pages]), [P], [E], 0.3)
    vf = orc.widen(v)
    for t in range(E):
        n = P + t + 1
        for h in range(Hq):
            assert np.max(np.abs(o[t, h] - vf[:n, h // 2].mean(axis=0))) < 1e-12
            assert abs(lse[t, h] - math.log(n)) < 1e-12


def test_planted_needle_names_the_key_that_was_read():
    # One key per (row, head) is made to dominate; V is position-coded, so the output reveals which (page, slot, kv
    # head) was read.  Key j carries two one-hot codes (j mod 8 and j div 8) of height 8; a query that carries the
    # codes of its target scores 128 there and at most 64 anywhere else, so every row of every head is decided by a
    # margin of 64 and every one of them is checked.
    Hq, Hkv, D, ps, P, E = 4, 2, 16, 16, 37, 21
    G, L = Hq // Hkv, P + E
    kf = np.zeros((L, Hkv, D), np.float32)
    v = np.zeros((L, Hkv, D), np.float32)
    for j in range(L):
        kf[j, :, j % 8] = 8.0
        kf[j, :, 8 + j // 8] = 8.0
        for g in range(Hkv):
            v[j, g, 0::2] = j
            v[j, g, 1::2] = 100 + g
    qf = np.zeros((E, Hq, D), np.float32)
    target = {}
    for t in range(E):
        for h in range(Hq):
            j = [P + t, 0, (7 * t + 5 * h) % (P + t + 1), 16 * ((P + t) // 16)][(t + h) % 4]   # diagonal, first, any, page start
            target[(t, h)] = j
            qf[t, h, j % 8] = 8.0
            qf[t, h, 8 + j // 8] = 8.0
    bits = lambda x: synth.bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
    pool = orc.PagePool(32, ps, Hkv, D, fill=0x7FC0)
    pages = synth.page_permutation(9, 32).tolist()[:synth.pages_needed(L, ps)]
    pool.append(pages, 0, bits(kf), bits(v))
    o, lse = orc.attn_extend(pool, bits(qf), Hq, [0, E], synth.block_table([pages]), [P], [E], 1.0)
    checked = 0
    for (t, h), j in target.items():
        assert abs(o[t, h, 0] - j) < 1e-9 and abs(o[t, h, 1] - (100 + h // G)) < 1e-9, (t, h, j)
        assert abs(lse[t, h] - 128.0) < 1e-9
        checked += 1
    assert checked == E * Hq


# ------------------------------------------------------ the paper's invariant
def test_reuse_equals_from_scratch_prefill():
    # Extend over reused prefix pages must equal the last E rows of a from-scratch
    # prefill of prefix+suffix placed on different pages.
    w = synth.WORKLOADS["tiny"]
    g = w.geom
    ext, _ = synth.draw_lengths(w)
    perm = synth.page_permutation(w.seed, w.num_pages).tolist()
    pool = orc.PagePool(w.num_pages, g.page_size, g.n_kv_heads, g.head_dim, fill=0x7FC0)
    for i, (P, E) in enumerate(ext[:4]):
        L = P + E
        k = synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_K, i, 0, L, g.n_kv_heads, g.head_dim))
        v = synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_V, i, 0, L, g.n_kv_heads, g.head_dim))
        q = synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_Q, i, 0, L, g.n_q_heads, g.head_dim))
        n = synth.pages_needed(L, g.page_size)
        reuse_pages, scratch_pages, perm = perm[:n], perm[n:2 * n], perm[2 * n:]
        # upstream operator wrote the prefix; downstream appends its suffix
        pool.append(reuse_pages, 0, k[:P], v[:P])
        pool.append(reuse_pages, P, k[P:], v[P:])
        o_reuse, l_reuse = orc.attn_extend(pool, q[P:], g.n_q_heads, [0, E], synth.block_table([reuse_pages]),
                                           [P], [E], g.scale)
        pool.append(scratch_pages, 0, k, v)
        o_full, l_full = orc.attn_extend(pool, q, g.n_q_heads, [0, L], synth.block_table([scratch_pages]),
                                         [0], [L], g.scale)
        assert np.max(np.abs(o_reuse - o_full[P:])) < 1e-12
        assert np.max(np.abs(l_reuse - l_full[P:])) < 1e-12


def test_children_sharing_a_parent_equal_private_copies_and_brute_force():
    # Section 5.1: the dependent tasks of a Cartesian product reuse the parent's prefix.  Sharing the
    # parent's pages must give what every child gets on a private copy of prefix + own suffix, and what
    # the independently written evaluation gives on the concatenated keys.
    rng = np.random.default_rng(515)
    Hkv, Hq, D, ps = 2, 4, 8, 16
    parent_lens, n_child, child_lens = [37, 16, 0], [3, 2, 1], [5, 1, 9, 17, 2, 4]
    pool, parent_rows, parent_kv = _build_pool(rng, parent_lens, Hkv, D, ps=ps, num_pages=96)
    used = {p for row in parent_rows for p in row}
    free = [p for p in synth.page_permutation(11, 96).tolist() if p not in used]
    cu_children = np.concatenate([[0], np.cumsum(n_child)])
    cu_q = np.concatenate([[0], np.cumsum(child_lens)])
    q = _rand_bits(rng, (int(cu_q[-1]), Hq, D))
    child_rows, child_kv, private_rows = [], [], []
    for g in range(len(parent_lens)):
        for c in range(cu_children[g], cu_children[g + 1]):
            E = child_lens[c]
            k, v = _rand_bits(rng, (E, Hkv, D)), _rand_bits(rng, (E, Hkv, D))
            n = synth.pages_needed(E, ps)
            pages, free = free[:n], free[n:]
            pool.append(pages, 0, k, v)
            child_rows.append(pages)
            child_kv.append((k, v))
            # the private copy: parent's tokens and the child's on pages of its own
            n2 = synth.pages_needed(parent_lens[g] + E, ps)
            priv, free = free[:n2], free[n2:]
            pool.append(priv, 0, np.concatenate([parent_kv[g][0], k]), np.concatenate([parent_kv[g][1], v]))
            private_rows.append(priv)
    scale = 0.3
    o, lse = orc.attn_extend_shared(pool, q, Hq, cu_q, cu_children, synth.block_table(parent_rows), parent_lens,
                                    synth.block_table(child_rows), child_lens, scale)
    child_parent = np.repeat(np.arange(len(parent_lens)), n_child)
    o2, lse2 = orc.attn_extend(pool, q, Hq, cu_q, synth.block_table(private_rows),
                               [parent_lens[g] for g in child_parent], child_lens, scale)
    assert np.max(np.abs(o - o2)) < 1e-12 and np.max(np.abs(lse - lse2)) < 1e-12
    for c, g in enumerate(child_parent):
        P, E = parent_lens[g], child_lens[c]
        keys = orc.widen(np.concatenate([parent_kv[g][0], child_kv[c][0]]))
        vals = orc.widen(np.concatenate([parent_kv[g][1], child_kv[c][1]]))
        for h in range(Hq):
            ob, lb = _brute(orc.widen(q[cu_q[c]:cu_q[c + 1], h]).tolist(), keys[:, h // 2].tolist(),
                            vals[:, h // 2].tolist(), [P + t + 1 for t in range(E)], scale)
            assert np.max(np.abs(o[cu_q[c]:cu_q[c + 1], h] - ob)) < 1e-12
            assert np.max(np.abs(lse[cu_q[c]:cu_q[c + 1], h] - lb)) < 1e-12


def test_page_permutation_invariance_is_bit_exact():
    rng = np.random.default_rng(21)
    lens = [40, 17, 64, 1]
    Hq, Hkv, D = 4, 2, 16
    outs = []
    for perm_seed in (1, 2):
        pool, rows, kv = _build_pool(np.random.default_rng(21), lens, Hkv, D, perm_seed=perm_seed)
        q = _rand_bits(np.random.default_rng(22), (len(lens), Hq, D))
        outs.append(orc.attn_decode(pool, q, Hq, synth.block_table(rows), lens, 0.25) + (rows,))
    assert outs[0][2] != outs[1][2]
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_gqa_equals_mha_on_repeated_kv_heads():
    rng = np.random.default_rng(31)
    Hq, Hkv, D, L = 8, 2, 16, 45
    G = Hq // Hkv
    pool, rows, kv = _build_pool(rng, [L], Hkv, D)
    q = _rand_bits(rng, (1, Hq, D))
    o, lse = orc.attn_decode(pool, q, Hq, synth.block_table(rows), [L], 0.25)
    # MHA pool: kv head h of the wide pool is kv head h // G of the narrow one
    k, v = kv[0]
    wide = orc.PagePool(64, 16, Hq, D)
    wide.append(rows[0], 0, np.repeat(k, G, axis=1), np.repeat(v, G, axis=1))
    o2, lse2 = orc.attn_decode(wide, q, Hq, synth.block_table(rows), [L], 0.25)
    # (the library matmul may round differently for G rows at once vs one row)
    assert np.max(np.abs(o - o2)) < 1e-13 and np.max(np.abs(lse - lse2)) < 1e-13


def test_decode_equals_extend_of_one_token():
    rng = np.random.default_rng(41)
    lens = [1, 2, 16, 17, 95]
    Hq, Hkv, D = 4, 2, 16
    pool, rows, _ = _build_pool(rng, lens, Hkv, D, num_pages=32)
    q = _rand_bits(rng, (len(lens), Hq, D))
    bt = synth.block_table(rows)
    od, ld = orc.attn_decode(pool, q, Hq, bt, lens, 0.25)
    oe, le = orc.attn_extend(pool, q, Hq, list(range(len(lens) + 1)), bt, [c - 1 for c in lens], [1] * len(lens), 0.25)
    assert np.max(np.abs(od - oe)) < 1e-13 and np.max(np.abs(ld - le)) < 1e-13


def test_split_and_combine_identity():
    rng = np.random.default_rng(51)
    D, L = 8, 200
    q, k, v = rng.standard_normal((1, D)), 2 * rng.standard_normal((L, D)), rng.standard_normal((L, D))
    o, lse = orc.attention_rows(q, k, v, np.array([L]), 0.5)
    for cuts in ([0, 200], [0, 1, 200], [0, 64, 128, 192, 200], sorted({0, 200, *rng.integers(1, 200, 6).tolist()})):
        parts = [orc.attention_rows(q, k[a:b], v[a:b], np.array([b - a]), 0.5) for a, b in zip(cuts[:-1], cuts[1:])]
        oc, lc = orc.combine_partials(np.stack([p[0][0] for p in parts]), np.array([p[1][0] for p in parts]))
        assert np.max(np.abs(oc - o[0])) < 1e-12 and abs(lc - lse[0]) < 1e-12


def test_against_library_sdpa_black_box():
    # torch's fp64 scaled_dot_product_attention with an explicit boolean mask as a second opinion.
    rng = np.random.default_rng(61)
    Hq, Hkv, D, P, E = 8, 2, 32, 70, 29
    G, L = Hq // Hkv, P + E
    pool, rows, kv = _build_pool(rng, [L], Hkv, D)
    q = _rand_bits(rng, (E, Hq, D))
    o, lse = orc.attn_extend(pool, q, Hq, [0, E], synth.block_table(rows), [P], [E], 0.2)
    k, v = kv[0]
    Q = torch.from_numpy(orc.widen(q)).permute(1, 0, 2)[None]                          # [1][Hq][E][D]
    K = torch.from_numpy(orc.widen(k)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    V = torch.from_numpy(orc.widen(v)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    mask = (torch.arange(L)[None, :] <= (P + torch.arange(E))[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask, scale=0.2)[0].permute(1, 0, 2)
    assert np.max(np.abs(o - ref.numpy())) < 1e-12
    ref_lse = torch.logsumexp(torch.where(mask, 0.2 * (Q[0] @ K[0].transpose(1, 2)), -torch.inf), dim=-1).T
    assert np.max(np.abs(lse - ref_lse.numpy())) < 1e-12


# ------------------------------------------------ data movement and allocator
def test_append_gather_roundtrip_and_untouched_slots():
    rng = np.random.default_rng(71)
    Hkv, D, ps = 2, 8, 16
    pool = orc.PagePool(8, ps, Hkv, D, fill=0xABCD)
    k, v = _rand_bits(rng, (37, Hkv, D)), _rand_bits(rng, (37, Hkv, D))
    pages = [5, 2, 7]
    pool.append(pages, 0, k[:20], v[:20])
    pool.append(pages, 20, k[20:], v[20:])                       # append in the middle of a page
    gk, gv = pool.gather(pages, 37)
    assert np.array_equal(gk, k) and np.array_equal(gv, v)
    # token 18 lives in page pages[1], slot 2, per kv head
    assert np.array_equal(pool.k[2, 1, 2], k[18, 1]) and np.array_equal(pool.v[2, 0, 2], v[18, 0])
    # slots past the length and pages never named keep the fill
    assert np.all(pool.k[7, :, 5:, :] == 0xABCD) and np.all(pool.v[[0, 1, 3, 4, 6]] == 0xABCD)


def test_stale_slots_do_not_influence_results():
    rng = np.random.default_rng(81)
    Hq, Hkv, D = 4, 2, 16
    res = []
    for fill in (0x7FC0, 0x7F80, 0x0000):                        # NaN, +Inf, 0 in the unwritten slots
        pool, rows, _ = _build_pool(np.random.default_rng(81), [21, 33], Hkv, D, fill=fill)
        q = _rand_bits(np.random.default_rng(82), (2, Hq, D))
        res.append(orc.attn_decode(pool, q, Hq, synth.block_table(rows), [21, 33], 0.25))
    for o, l in res[1:]:
        assert np.array_equal(o, res[0][0]) and np.array_equal(l, res[0][1])
    assert np.all(np.isfinite(res[0][0]))


def test_zero_length_conventions():
    pool = orc.PagePool(4, 16, 1, 8)
    q = np.zeros((1, 2, 8), np.uint16)
    o, lse = orc.attn_decode(pool, q, 2, synth.block_table([[]]), [0], 1.0)
    assert np.all(o == 0) and np.all(np.isneginf(lse))
    o, lse = orc.attn_extend(pool, np.zeros((0, 2, 8), np.uint16), 2, [0, 0], synth.block_table([[]]), [5], [0], 1.0)
    assert o.shape == (0, 2, 8)


def test_free_list_order_and_errors():
    fl = orc.FreeList(6)
    assert fl.alloc(3) == [0, 1, 2]
    assert fl.alloc(4) is None and fl.free_pages == 3            # all-or-nothing
    fl.free([1, 0])
    assert fl.alloc(3) == [0, 1, 3]                               # last freed comes back first
    with pytest.raises(KeyError):
        fl.free([5])                                              # never allocated
    with pytest.raises(KeyError):
        fl.free([2, 2])                                           # duplicate in one call, no partial effect
    assert fl.allocated[2]
    fl.evict([2, 3])
    assert fl.evicted_total == 2 and fl.free_pages == 4


def test_kv_bytes_per_token_matches_the_paper_figure():
    for line in open(os.path.join(GOLDEN, "kv_bytes_per_token.txt")):
        if line.startswith("#") or not line.strip():
            continue
        layers, hkv, d, nbytes, kib, tokens, mb = [int(x) for x in line.split()]
        per_layer = synth.Geometry(hkv, hkv, d).kv_bytes_per_token
        assert nbytes == 2 and layers * per_layer == kib * 1024
        assert abs(layers * per_layer * tokens / 1e6 - mb) / mb < 0.03
    assert synth.WORKLOADS["extend_8b"].geom.kv_bytes_per_token == 4096


def test_widen_is_exact():
    bits = np.array([0x0000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F], np.uint16)
    ref = synth.bits_to_bf16(bits).to(torch.float64).numpy()
    assert np.array_equal(orc.widen(bits), ref)


# ------------------------------------------------ owners, pins, eviction order
def test_shared_pages_return_with_their_last_owner():
    fl = orc.FreeList(8)
    parent = fl.alloc(3)                                          # [0, 1, 2]
    for _ in range(2):                                            # two children read the parent's prefix
        fl.ref(parent)
    fl.free(parent)                                               # the parent is done: pages stay
    assert fl.free_pages == 5 and all(fl.allocated[p] for p in parent)
    fl.free(parent[:2])                                           # first child done with two of them
    assert fl.free_pages == 5
    fl.free(parent)                                               # second child: pages 0 and 1 go back, 2 has one owner left
    assert fl.free_pages == 7 and not fl.allocated[0] and not fl.allocated[1] and fl.allocated[2]
    assert fl.alloc(2) == [1, 0]                                  # last in, first out
    with pytest.raises(KeyError):
        fl.ref([5])                                               # not allocated


def test_pinned_pages_are_never_evicted_and_unpin_all_is_the_fallback():
    fl = orc.FreeList(6)
    ids = fl.alloc(4)
    fl.pin([ids[1]]); fl.pin([ids[1]]); fl.pin([ids[3]])          # pins are counted
    with pytest.raises(orc.PinnedError):
        fl.evict([ids[0], ids[1]])
    assert fl.allocated[ids[0]]                                   # no partial effect
    with pytest.raises(orc.PinnedError):
        fl.free([ids[3]])                                         # the last owner cannot drop a pinned page
    fl.unpin([ids[1]])
    with pytest.raises(orc.PinnedError):
        fl.evict([ids[1]])                                        # still pinned once
    with pytest.raises(ValueError):
        fl.unpin([ids[0]])                                        # was never pinned
    assert fl.evict_lru(10) == [ids[0], ids[2]]                   # skips the pinned ones
    assert fl.unpin_all() == 2
    assert fl.evict_lru(10) == [ids[1], ids[3]] and fl.evicted_total == 4 and fl.free_pages == 6


def test_lru_order_follows_alloc_and_touch():
    fl = orc.FreeList(8)
    a = fl.alloc(5)                                               # clock 1..5
    fl.touch([a[0], a[2]])                                        # now the most recent
    assert fl.evict_lru(2) == [a[1], a[3]]
    b = fl.alloc(1)                                               # reuses a[3] (LIFO), newest of all
    assert b == [a[3]]
    assert fl.evict_lru(3) == [a[4], a[0], a[2]]
    assert fl.evict_lru(3) == [a[3]] and fl.evict_lru(1) == []


def test_free_list_invariants_under_random_operations():
    rng = np.random.default_rng(17)
    fl = orc.FreeList(16)
    for _ in range(3000):
        op = rng.integers(0, 8)
        live = [p for p in range(16) if fl.allocated[p]]
        pick = [int(p) for p in rng.choice(live, size=min(len(live), int(rng.integers(1, 4))), replace=False)] if live else []
        try:
            if op == 0: fl.alloc(int(rng.integers(0, 5)))
            elif op == 1 and pick: fl.free(pick)
            elif op == 2 and pick: fl.evict(pick)
            elif op == 3 and pick: fl.ref(pick)
            elif op == 4 and pick: fl.pin(pick)
            elif op == 5 and pick: fl.unpin(pick)
            elif op == 6 and pick: fl.touch(pick)
            elif op == 7: fl.evict_lru(int(rng.integers(0, 3)))
        except (orc.PinnedError, ValueError):
            pass
        alloc = {p for p in range(16) if fl.allocated[p]}
        assert alloc.isdisjoint(fl.stack) and len(alloc) + len(fl.stack) == 16 and len(set(fl.stack)) == len(fl.stack)
        assert all((fl.refs[p] >= 1) == (p in alloc) for p in range(16))
        assert all(fl.pins[p] == 0 for p in fl.stack)             # nothing pinned is ever on the free list
