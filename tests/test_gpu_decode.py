"""attn_decode through the C ABI against the oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, assert_close, run_decode, run_extend

pytestmark = pytest.mark.gpu


@pytest.fixture(params=[1, 2], ids=["pages-through-registers", "pages-through-shared-memory-ring"], autouse=True)
def decode_variant(request):
    """Every test of this file runs with both ways the decode kernel brings pages on chip."""
    kvattn.kvattn_set_decode_impl(request.param)
    yield request.param
    kvattn.kvattn_set_decode_impl(0)


@pytest.mark.parametrize("hq,hkv,d", [(4, 2, 64), (8, 8, 64), (8, 1, 64), (32, 8, 128), (8, 2, 128), (4, 4, 128)])
def test_decode_edge_lengths(hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    lens = [1, 2, 15, 16, 17, 31, 33, 511, 513, 1023, 1024, 1025, 0, 100]
    dp = DualPool(geom, 512, seed=100 + hq + d)
    b = Batch(dp, lens)
    b.write([(i, 0, L) for i, L in enumerate(lens)])
    res = run_decode(dp, b, lens)
    d_o, d_l, t = assert_close(res, f"decode {hq}/{hkv}/{d}")
    # the empty sequence: O = 0, LSE = -inf
    assert np.all(res["o"][12] == 0) and np.all(np.isneginf(res["lse"][12]))
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


def test_decode_long_context_and_split_combine():
    geom = synth.Geometry(32, 8, 128)
    lens = [4096, 4095, 2049, 777]
    dp = DualPool(geom, 1024, seed=7)
    b = Batch(dp, lens)
    b.write([(i, 0, L) for i, L in enumerate(lens)])
    res = run_decode(dp, b, lens)
    assert_close(res, "decode long")
    # run-to-run bit determinism
    res2 = run_decode(dp, b, lens, oracle=False)
    assert np.array_equal(res["o_bits"], res2["o_bits"]) and np.array_equal(res["lse_raw"], res2["lse_raw"])
    dp.close()


def test_decode_is_bit_invariant_under_page_placement():
    geom = synth.Geometry(32, 8, 128)
    lens = [1500, 37, 640]
    outs = []
    for seed_perm in (1, 2):
        dp = DualPool(geom, 256, seed=55)
        dp.placement = synth.page_permutation(seed_perm, 256).tolist()       # same values, other pages
        b = Batch(dp, lens)
        b.write([(i, 0, L) for i, L in enumerate(lens)])
        outs.append((run_decode(dp, b, lens, oracle=False), b.rows))
        dp.close()
    assert outs[0][1] != outs[1][1]
    assert np.array_equal(outs[0][0]["o_bits"], outs[1][0]["o_bits"])
    assert np.array_equal(outs[0][0]["lse_raw"], outs[1][0]["lse_raw"])


def test_decode_equals_extend_of_one_token():
    geom = synth.Geometry(8, 2, 128)
    lens = [1, 16, 200, 513]
    dp = DualPool(geom, 128, seed=9)
    b = Batch(dp, lens)
    b.write([(i, 0, L) for i, L in enumerate(lens)])
    dec = run_decode(dp, b, lens)
    ext = run_extend(dp, b, [L - 1 for L in lens], [1] * len(lens), impl=1)
    assert_close(dec, "decode"); assert_close(ext, "extend E=1")
    assert np.max(np.abs(dec["o"] - ext["o"])) <= 2 ** -7 and np.max(np.abs(dec["lse"] - ext["lse"])) <= 1e-4
    dp.close()


def test_decode_needle_and_position_coded_values():
    # One key dominates each row; V carries its own position, so an indexing slip changes O by >= 1/16.
    geom = synth.Geometry(8, 2, 128)
    dev = "cuda"
    lens = [300, 45]
    dp = DualPool(geom, 64, seed=21)
    b = Batch(dp, lens)
    needles = [(173, 0), (44, 1)]
    qs, segs, ks, vs = [], [], [], []
    for i, L in enumerate(lens):
        q = b.q(i, L - 1, L)                                             # [1][Hq][D]
        j, _ = needles[i]
        k = torch.zeros((L, geom.n_kv_heads, geom.head_dim), dtype=torch.float32, device=dev)
        v = torch.zeros_like(k)
        pos = torch.arange(L, device=dev, dtype=torch.float32)
        v[:, :, 0::3] = ((pos % 16) / 16)[:, None, None]                 # base-16 digits of the position,
        v[:, :, 1::3] = ((pos // 16 % 16) / 16)[:, None, None]           # exact in bf16 and O(1), so the
        v[:, :, 2::3] = ((pos // 256) / 16)[:, None, None]               # 2e-2 bound separates neighbours
        for g in range(geom.n_kv_heads):
            qh = q[0, g * geom.group].float()                            # first head of the group
            k[j, g] = 300.0 * qh / (qh @ qh)                             # scaled score 300/sqrt(128) ~ 26.5
        segs.append((i, 0)); ks.append(k.to(torch.bfloat16)); vs.append(v.to(torch.bfloat16))
    dp.append(b.rows, segs, ks, vs)
    res = run_decode(dp, b, lens)
    assert_close(res, "needle")
    for i, (j, _) in enumerate(needles):
        for g in range(geom.n_kv_heads):
            o = res["o"][i, g * geom.group]
            assert abs(o[0] - (j % 16) / 16) < 0.02 and abs(o[1] - (j // 16 % 16) / 16) < 0.02
            assert abs(o[2] - (j // 256) / 16) < 0.02
    dp.close()


def test_the_two_decode_variants_give_the_same_bits():
    geom = synth.Geometry(32, 8, 128)
    lens = [4096, 1, 16, 17, 1025, 2049, 3, 700, 0, 48]
    dp = DualPool(geom, 1024, seed=17)
    b = Batch(dp, [max(x, 1) for x in lens])
    b.write([(i, 0, L) for i, L in enumerate(lens) if L > 0])
    outs = []
    for impl in (1, 2):
        kvattn.kvattn_set_decode_impl(impl)
        outs.append(run_decode(dp, b, lens, oracle=(impl == 1)))
    assert_close(outs[0], "register variant")
    assert np.array_equal(outs[0]["o_bits"], outs[1]["o_bits"]) and np.array_equal(outs[0]["lse_raw"], outs[1]["lse_raw"])
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()
