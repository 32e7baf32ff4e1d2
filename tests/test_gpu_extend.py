"""attn_extend through the C ABI against the oracle: edge cases, the reuse invariant, aliasing."""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, assert_close, run_extend

pytestmark = pytest.mark.gpu
IMPLS = [1, 2]   # 1 = small-tile kernel, 2 = tcgen05 kernel


def _skip_if_no_tc(impl, geom):
    if impl == 2:
        dp = DualPool(geom, 4, seed=0, with_oracle=False)
        try:
            q = torch.zeros((1, geom.n_q_heads, geom.head_dim), dtype=torch.bfloat16, device="cuda")
            z = torch.zeros(1, dtype=torch.int32, device="cuda")
            kvattn.kvattn_set_extend_impl(2)
            try:
                kvattn.attn_extend(dp.pool, q, torch.tensor([0, 0], dtype=torch.int32, device="cuda"),
                                   torch.zeros((1, 1), dtype=torch.int32, device="cuda"), z, z, 1, 1, 1.0,
                                   torch.empty_like(q), torch.empty((1, geom.n_q_heads), device="cuda"),
                                   torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
            except kvattn.KvError as e:
                if e.status == kvattn.KV_ERR_UNSUPPORTED:
                    pytest.skip("tensor-core extend kernel does not support this shape")
                raise
            finally:
                kvattn.kvattn_set_extend_impl(0)
        finally:
            dp.close()


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("hq,hkv,d", [(4, 2, 64), (32, 8, 128), (8, 1, 128), (4, 4, 64), (16, 2, 128)])
def test_extend_edge_cases(impl, hq, hkv, d):
    geom = synth.Geometry(hq, hkv, d)
    _skip_if_no_tc(impl, geom)
    P = [0, 1, 15, 16, 17, 31, 32, 0, 100, 5, 130]
    E = [1, 2, 15, 16, 17, 33, 1, 70, 0, 129, 300]
    dp = DualPool(geom, 256, seed=200 + hq + d)
    b = Batch(dp, [p + e for p, e in zip(P, E)])
    b.write([(i, 0, P[i]) for i in range(len(P))])                     # upstream operator's prefill
    b.write([(i, P[i], P[i] + E[i]) for i in range(len(P))])           # downstream suffix
    res = run_extend(dp, b, P, E, impl=impl)
    assert_close(res, f"extend impl{impl} {hq}/{hkv}/{d}")
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


@pytest.mark.parametrize("impl", IMPLS)
def test_tiny_config_reuse_equals_from_scratch_prefill(impl):
    # Config "tiny": 8 tuples, P ~ U[32,128], E ~ U[16,48], 256-page pool, random placement.
    w = synth.WORKLOADS["tiny"]
    _skip_if_no_tc(impl, w.geom)
    ext, _ = synth.draw_lengths(w)
    P, E = [p for p, _ in ext], [e for _, e in ext]
    dp = DualPool(w.geom, w.num_pages, seed=w.seed)
    reuse = Batch(dp, [p + e for p, e in ext])
    reuse.write([(i, 0, P[i]) for i in range(len(P))])
    reuse.write([(i, P[i], P[i] + E[i]) for i in range(len(P))])
    r = run_extend(dp, reuse, P, E, impl=impl)
    assert_close(r, "tiny reuse")
    scratch = Batch(dp, [p + e for p, e in ext])                       # same uids -> same values, new pages
    scratch.write([(i, 0, P[i] + E[i]) for i in range(len(P))])
    f = run_extend(dp, scratch, [0] * len(P), [p + e for p, e in ext], impl=impl)
    assert_close(f, "tiny from-scratch")
    # last E rows of the from-scratch prefill == the reuse run (both within tolerance of the same oracle rows)
    worst_o = worst_l = 0.0
    for i in range(len(P)):
        a0, a1 = r["cu"][i], r["cu"][i + 1]
        b0 = f["cu"][i] + P[i]
        assert np.max(np.abs(r["o_ref"][a0:a1] - f["o_ref"][b0:b0 + E[i]])) < 1e-12
        worst_o = max(worst_o, float(np.max(np.abs(r["o"][a0:a1] - f["o"][b0:b0 + E[i]]))))
        worst_l = max(worst_l, float(np.max(np.abs(r["lse"][a0:a1] - f["lse"][b0:b0 + E[i]]))))
    assert worst_o <= 2e-2 and worst_l <= 1e-3
    dp.close()


@pytest.mark.parametrize("impl", IMPLS)
def test_shared_prefix_fan_out(impl):
    # A join's children share the parent's prefix pages (full blocks only) and append private suffixes.
    geom = synth.Geometry(8, 2, 128)
    _skip_if_no_tc(impl, geom)
    dp = DualPool(geom, 128, seed=31)
    fan, P, E = 17, 208, [5 + (3 * c) % 30 for c in range(17)]
    parent = Batch(dp, [P])
    parent.write([(0, 0, P)])
    kids = Batch(dp, E, uid0=100)                                       # private suffix pages only
    kids.rows = [parent.rows[0] + r for r in kids.rows]                 # alias the parent's pages
    segs, ks, vs = [], [], []
    for c in range(fan):
        k, v = kids.kv(c, P, P + E[c])
        segs.append((c, P)); ks.append(k); vs.append(v)
    dp.append(kids.rows, segs, ks, vs)
    res = run_extend(dp, kids, [P] * fan, E, impl=impl)
    assert_close(res, "fan-out")
    dp.close()


@pytest.mark.parametrize("impl", IMPLS)
def test_extend_bit_determinism_and_placement_invariance(impl):
    geom = synth.Geometry(32, 8, 128)
    _skip_if_no_tc(impl, geom)
    P, E = [300, 17, 0], [40, 129, 65]
    outs = []
    for seed_perm in (1, 1, 2):
        dp = DualPool(geom, 128, seed=77)
        dp.placement = synth.page_permutation(seed_perm, 128).tolist()
        b = Batch(dp, [p + e for p, e in zip(P, E)])
        b.write([(i, 0, P[i] + E[i]) for i in range(3)])
        outs.append(run_extend(dp, b, P, E, impl=impl, oracle=False))
        dp.close()
    for o in outs[1:]:
        assert np.array_equal(outs[0]["o_bits"], o["o_bits"]) and np.array_equal(outs[0]["lse_raw"], o["lse_raw"])


def test_many_one_step_items_on_the_tensor_core_kernel():
    # Hundreds of sequences whose keys fit one 128-key tile: every work item is a single softmax step, so the
    # roles of the kernel run as far ahead of each other as their hand-overs allow.  Repeated, because the
    # failure this guards against (a hand-over barrier two phases ahead of its waiters) depended on timing.
    geom = synth.Geometry(32, 8, 128)
    _skip_if_no_tc(2, geom)
    rng = np.random.default_rng(77)
    n = 300
    E = rng.integers(30, 45, size=n).tolist()
    P = [0] * n
    dp = DualPool(geom, 3 * n + 8, seed=277)
    b = Batch(dp, E)
    b.write([(i, 0, E[i]) for i in range(n)])
    for rep in range(6):
        res = run_extend(dp, b, P, E, impl=2, oracle=(rep == 0))
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
        if rep == 0:
            assert_close(res, "one-step items")
            first = res["o_bits"].copy()
        else:
            assert np.array_equal(res["o_bits"], first)
    dp.close()


def test_one_call_from_host_buffers_matches_append_then_extend():
    # attn_extend_host = copies in + kv_append(suffix) + attn_extend + copies out: bit-identical to doing the
    # same with device tensors, and within tolerance of the oracle.
    geom = synth.Geometry(32, 8, 128)
    P = [0, 17, 160, 500, 31]
    E = [40, 1, 129, 64, 300]
    dp = DualPool(geom, 128, seed=311)
    b = Batch(dp, [p + e for p, e in zip(P, E)])
    b.write([(i, 0, P[i]) for i in range(len(P))])                       # the upstream operator's prefix only
    ks, vs = zip(*[b.kv(i, P[i], P[i] + E[i]) for i in range(len(P))])
    q = torch.cat([b.q(i, P[i], P[i] + E[i]) for i in range(len(P))]).contiguous()
    k_new, v_new = torch.cat(ks).contiguous(), torch.cat(vs).contiguous()
    cu = torch.tensor(np.concatenate([[0], np.cumsum(E)]), dtype=torch.int32)
    bt = torch.from_numpy(b.block_tables()).to(torch.int32).contiguous()
    pl, el = torch.tensor(P, dtype=torch.int32), torch.tensor(E, dtype=torch.int32)
    pin = lambda t: t.cpu().contiguous().pin_memory()
    h = [pin(t) for t in (q, k_new, v_new, cu, bt, pl, el)]
    out_h = torch.full(q.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    lse_h = torch.full((q.shape[0], geom.n_q_heads), float("nan"), dtype=torch.float32).pin_memory()
    max_l = max(p + e for p, e in zip(P, E))
    staging = torch.empty(kvattn.attn_extend_host_staging_bytes(dp.pool, geom.n_q_heads, len(P), int(q.shape[0]),
                                                                bt.shape[1], max_l), dtype=torch.uint8, device="cuda")
    kvattn.attn_extend_host(dp.pool, h[0], h[1], h[2], h[3], h[4], h[5], h[6], max(E), max_l, geom.scale, out_h, lse_h,
                            staging)
    torch.cuda.synchronize()
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    # the oracle's pool gets the same suffix rows; the device rows were written by the call itself
    for i in range(len(P)):
        dp.host.append(b.rows[i], P[i], synth.bf16_bits(ks[i]), synth.bf16_bits(vs[i]))
    res = run_extend(dp, b, P, E, impl=0)
    assert np.array_equal(synth.bf16_bits(out_h), res["o_bits"])
    assert np.array_equal(lse_h.numpy(), res["lse_raw"])
    assert_close(res, "host-buffer step")
    dp.close()


class _SpikyBatch(Batch):
    """Keys at a few chosen positions are large and aligned with every query, so that the row maximum jumps by
    tens of binades when their tile arrives."""

    def __init__(self, dp, lengths, spikes):
        super().__init__(dp, lengths)
        self.spikes = spikes  # {position: gain}
        g = dp.geom
        rng = np.random.default_rng(4242)
        self.pattern = torch.tensor(rng.choice([-1.0, 1.0], size=g.head_dim), dtype=torch.float32, device=dp.device)

    def kv(self, i, lo, hi):
        k, v = super().kv(i, lo, hi)
        for pos, gain in self.spikes.items():
            if lo <= pos < hi:
                k[pos - lo] = (gain * self.pattern).to(torch.bfloat16)
        return k, v

    def q(self, i, lo, hi):
        return (super().q(i, lo, hi).float() + self.pattern).to(torch.bfloat16)


@pytest.mark.parametrize("total", [2300, 4500])
def test_scores_that_jump_far_above_the_running_maximum(total):
    # q.k at the spikes is about gain * head_dim, i.e. tens of binades above everything seen before: the kernel
    # variant for long sequences (total >= 4096), which assumes that the maximum in use still serves, has to notice
    # and take such a step again with the exact maximum; the variant for short ones rescales.  Each later spike is
    # larger than the one before, one of them sits among the suffix tokens.
    geom = synth.Geometry(8, 2, 128)
    _skip_if_no_tc(2, geom)
    E = 48
    P = total - E
    # the last one lifts the score by more than 128 binades: without the second look its exponential is infinite
    spikes = {700: 0.75, 1500: 1.5, total - 900: 2.5, total - 20: 9.0}
    dp = DualPool(geom, synth.pages_needed(total, 16) + 4, seed=991)
    b = _SpikyBatch(dp, [total], spikes)
    b.write([(0, 0, total)])
    for impl in (2, 1):
        res = run_extend(dp, b, [P], [E], impl=impl)
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
        assert_close(res, f"spikes, impl {impl}")
    dp.close()


def test_more_sequences_than_the_plan_ranks():
    # The plan kernel ranks the sequences of a batch by length up to a fixed batch size and keeps the batch order
    # beyond it; groups are formed (and the ranking used) only when the batch has a dozen items per SM or more.
    # Both sides of that size are run on the tensor-core kernel and compared with the oracle.
    geom = synth.Geometry(8, 2, 64)
    _skip_if_no_tc(2, geom)
    rng = np.random.default_rng(5)
    for n in (8300, 2200):
        E = rng.integers(1, 5, size=n).tolist()
        P = rng.integers(0, 40, size=n).tolist()
        L = [p + e for p, e in zip(P, E)]
        dp = DualPool(geom, sum(synth.pages_needed(x, 16) for x in L) + 8, seed=300 + n)
        b = Batch(dp, L)
        b.write([(i, 0, L[i]) for i in range(n)])
        res = run_extend(dp, b, P, E, impl=2)
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
        assert_close(res, f"{n} sequences")
        dp.close()


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("hq,hkv,d", [(32, 8, 128), (4, 2, 64), (8, 1, 128)])
def test_append_and_extend_in_one_call_is_bit_identical_to_the_two_calls(impl, hq, hkv, d):
    # attn_extend_append = kv_append(suffix) + attn_extend with fewer launches: the whole pool image, O and LSE must
    # come out bit for bit as from the two calls, and O / LSE within tolerance of the oracle.
    geom = synth.Geometry(hq, hkv, d)
    _skip_if_no_tc(impl, geom)
    # prefixes that end anywhere inside a page and inside a group of eight slots, suffixes of one token, of exactly a
    # group or a page, empty ones, and ones that span several KV tiles
    P = [0, 17, 160, 500, 31, 16, 1000, 5, 123, 8, 64, 127, 250]
    E = [40, 1, 129, 64, 300, 16, 7, 0, 9, 8, 1, 2, 270]
    L = [p + e for p, e in zip(P, E)]
    imgs, outs = [], []
    for fused in (False, True):
        dp = DualPool(geom, 256, seed=321)
        b = Batch(dp, [max(x, 1) for x in L])
        b.write([(i, 0, P[i]) for i in range(len(P))])                       # the upstream operator's prefix only
        ks, vs = zip(*[b.kv(i, P[i], L[i]) for i in range(len(P))])
        if not fused:
            dp.append(b.rows, [(i, P[i]) for i in range(len(P))], list(ks), list(vs))
            res = run_extend(dp, b, P, E, impl=impl)
            assert_close(res, "append then extend")
        else:
            q = torch.cat([b.q(i, P[i], L[i]) for i in range(len(P))]).contiguous()
            k_new, v_new = torch.cat(ks).contiguous(), torch.cat(vs).contiguous()
            t = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device="cuda")
            out = torch.full_like(q, float("nan"))
            lse = torch.full((q.shape[0], hq), float("nan"), dtype=torch.float32, device="cuda")
            ws = torch.empty(kvattn.attn_workspace_bytes(dp.pool, hq, len(P), int(q.shape[0]), max(L), 0, 0), dtype=torch.uint8,
                             device="cuda")
            kvattn.kvattn_set_extend_impl(impl)
            try:
                kvattn.attn_extend_append(dp.pool, q, k_new, v_new, t(np.concatenate([[0], np.cumsum(E)])),
                                          torch.from_numpy(b.block_tables()).to("cuda"), t(P), t(E), max(E), max(L), geom.scale,
                                          out, lse, ws)
            finally:
                kvattn.kvattn_set_extend_impl(0)
            torch.cuda.synchronize()
            res = {"o_bits": synth.bf16_bits(out), "lse_raw": lse.cpu().numpy().copy()}
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
        imgs.append(dp.device_image())
        outs.append(res)
        dp.close()
    assert np.array_equal(imgs[0][0], imgs[1][0]) and np.array_equal(imgs[0][1], imgs[1][1])   # K and V pool images
    assert np.array_equal(outs[0]["o_bits"], outs[1]["o_bits"])
    assert np.array_equal(outs[0]["lse_raw"], outs[1]["lse_raw"])


@pytest.mark.parametrize("impl", IMPLS)
def test_one_plan_serves_several_attention_calls(impl):
    # attn_extend_plan once, attn_extend_planned several times (a model's layers share the lengths): each call gives
    # the bits of attn_extend, also when the queries change between the calls.
    geom = synth.Geometry(32, 8, 128)
    _skip_if_no_tc(impl, geom)
    P, E = [0, 300, 17, 1200, 64], [129, 40, 300, 7, 64]
    L = [p + e for p, e in zip(P, E)]
    dp = DualPool(geom, 200, seed=555)
    b = Batch(dp, L)
    b.write([(i, 0, L[i]) for i in range(len(P))])
    ref = run_extend(dp, b, P, E, impl=impl)
    assert_close(ref, "plain call")
    t = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device="cuda")
    cu, bt, pl, el = t(np.concatenate([[0], np.cumsum(E)])), torch.from_numpy(b.block_tables()).to("cuda"), t(P), t(E)
    q = ref["q"]
    ws = torch.empty(kvattn.attn_workspace_bytes(dp.pool, 32, len(P), int(q.shape[0]), max(L), 0, 0), dtype=torch.uint8,
                     device="cuda")
    kvattn.kvattn_set_extend_impl(impl)
    try:
        kvattn.attn_extend_plan(dp.pool, 32, cu, bt, pl, el, int(q.shape[0]), max(E), max(L), ws)
        for rep in range(4):
            qq = q if rep != 2 else (-q).contiguous()                # another layer's queries over the same plan
            out = torch.full_like(q, float("nan"))
            lse = torch.full((q.shape[0], 32), float("nan"), dtype=torch.float32, device="cuda")
            kvattn.attn_extend_planned(dp.pool, qq, cu, bt, pl, el, max(E), max(L), geom.scale, out, lse, ws)
            torch.cuda.synchronize()
            if rep != 2:
                assert np.array_equal(synth.bf16_bits(out), ref["o_bits"]) and np.array_equal(lse.cpu().numpy(), ref["lse_raw"])
            else:
                assert torch.isfinite(out.float()).all() and not np.array_equal(synth.bf16_bits(out), ref["o_bits"])
    finally:
        kvattn.kvattn_set_extend_impl(0)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()
