"""Pool, allocator, append/gather and the checks, through the C ABI, against the oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import paged_attention as orc
from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, NAN_BITS

pytestmark = pytest.mark.gpu
GEOMS = [synth.Geometry(4, 2, 64), synth.Geometry(32, 8, 128)]


def test_allocator_matches_the_documented_order():
    pool = kvattn.kv_pool_create(12, 16, 2, 64)
    ref = orc.FreeList(12)
    rng = np.random.default_rng(3)
    live = []
    for step in range(200):
        if live and rng.random() < 0.45:
            k = int(rng.integers(1, len(live) + 1))
            idx = rng.choice(len(live), size=k, replace=False)
            ids = [live[i] for i in idx]
            live = [p for i, p in enumerate(live) if i not in set(idx.tolist())]
            if rng.random() < 0.5:
                kvattn.kv_free(pool, ids); ref.free(ids)
            else:
                kvattn.kv_evict(pool, ids); ref.evict(ids)
        else:
            n = int(rng.integers(0, 6))
            want = ref.alloc(n)
            if want is None:
                with pytest.raises(kvattn.KvError) as e:
                    kvattn.kv_alloc(pool, n)
                assert e.value.status == kvattn.KV_ERR_OOM
            else:
                assert kvattn.kv_alloc(pool, n) == want
                live += want
        free, used, ev = kvattn.kv_pool_stats(pool)
        assert (free, used, ev) == (ref.free_pages, 12 - ref.free_pages, ref.evicted_total)
    pool.destroy()


def test_release_errors_have_no_partial_effect():
    pool = kvattn.kv_pool_create(8, 16, 2, 64)
    ids = kvattn.kv_alloc(pool, 4)
    for bad in ([ids[0], 7], [ids[1], ids[1]], [-1], [8]):
        with pytest.raises(kvattn.KvError) as e:
            kvattn.kv_free(pool, bad)
        assert e.value.status == kvattn.KV_ERR_NOT_ALLOCATED
        assert kvattn.kv_pool_stats(pool)[:2] == (4, 4)
    kvattn.kv_free(pool, ids)
    with pytest.raises(kvattn.KvError):
        kvattn.kv_evict(pool, [ids[0]])                              # double release
    pool.destroy()


def test_unsupported_shapes_are_refused():
    for args in ((8, 32, 2, 64), (8, 16, 2, 96), (8, 16, 2, 256)):
        with pytest.raises(kvattn.KvError) as e:
            kvattn.kv_pool_create(*args)
        assert e.value.status == kvattn.KV_ERR_UNSUPPORTED
    pool = kvattn.kv_pool_create(8, 16, 2, 64)
    q = torch.zeros((1, 6, 64), dtype=torch.bfloat16, device="cuda")  # G = 3
    with pytest.raises(kvattn.KvError) as e:
        kvattn.attn_decode(pool, q, torch.zeros((1, 1), dtype=torch.int32, device="cuda"),
                           torch.ones(1, dtype=torch.int32, device="cuda"), 1, 1.0, torch.empty_like(q),
                           torch.empty((1, 6), device="cuda"))
    assert e.value.status == kvattn.KV_ERR_UNSUPPORTED
    pool.destroy()


@pytest.mark.parametrize("geom", GEOMS, ids=["d64", "d128"])
def test_append_is_bit_exact_over_the_whole_pool_image(geom):
    dp = DualPool(geom, 64, seed=11)
    lens = [1, 15, 16, 17, 100, 33]
    b = Batch(dp, lens)
    # first the prefixes (upstream operator), then the rest from the middle of a page (downstream suffix)
    cut = [0, 7, 16, 3, 41, 32]
    b.write([(i, 0, cut[i]) for i in range(len(lens))])
    b.write([(i, cut[i], lens[i]) for i in range(len(lens))])
    torch.cuda.synchronize()
    k_img, v_img = dp.device_image()
    # every written slot is bit-exact; the slots behind a sequence's last token in its last page are zero
    # (the library clears them, as the header documents); pages the batch never named still hold the fill
    for i, L in enumerate(lens):
        gk, gv = dp.host.gather(b.rows[i], L)
        dk = np.concatenate([k_img[pg].transpose(1, 0, 2) for pg in b.rows[i]])
        dv = np.concatenate([v_img[pg].transpose(1, 0, 2) for pg in b.rows[i]])
        assert np.array_equal(dk[:L], gk) and np.array_equal(dv[:L], gv)
        assert np.all(dk[L:] == 0) and np.all(dv[L:] == 0)
    used = sorted(p for r in b.rows for p in r)
    unused = [p for p in range(64) if p not in used]
    assert len(unused) > 0 and np.all(k_img[unused] == NAN_BITS) and np.all(v_img[unused] == NAN_BITS)
    # the library's own offset helper agrees with the formula used by device_image()
    rng = np.random.default_rng(5)
    kflat = dp.k_buf.cpu().numpy().view(np.uint16)
    for _ in range(200):
        p, h, s, d = (int(rng.integers(0, n)) for n in (64, geom.n_kv_heads, 16, geom.head_dim))
        off = kvattn.kv_pool_elem_offset(dp.pool, p, h, s, d)
        assert kflat[off] == k_img[p, h, s, d]
    assert kvattn.kv_pool_elem_offset(dp.pool, 64, 0, 0, 0) == -1
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


@pytest.mark.parametrize("n_seq", [1, 31, 33, 1025, 3000])
def test_append_with_many_and_empty_segments_is_bit_exact(n_seq):
    # The segment of a token is found by a search over cu_new in which the lanes probe 32 entries per step: segment
    # counts around the powers of 32, runs of empty segments (equal entries of cu_new) and one-token segments.
    geom = synth.Geometry(2, 1, 64)
    rng = np.random.default_rng(n_seq)
    lens = [int(x) for x in rng.choice([0, 0, 1, 2, 5, 16, 17], size=n_seq)]
    if sum(lens) == 0:
        lens[-1] = 3
    pages = sum(synth.pages_needed(max(L, 1), 16) for L in lens) + 4
    dp = DualPool(geom, pages, seed=600 + n_seq)
    b = Batch(dp, [max(L, 1) for L in lens])
    ks, vs = zip(*[b.kv(i, 0, lens[i]) for i in range(n_seq)])
    dp.append(b.rows, [(i, 0) for i in range(n_seq)], list(ks), list(vs))          # one call, n_seq segments
    torch.cuda.synchronize()
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    k_img, v_img = dp.device_image()
    for i, L in enumerate(lens):
        if L == 0:
            assert np.all(k_img[b.rows[i]] == NAN_BITS)                            # an empty segment writes nothing
            continue
        gk, gv = dp.host.gather(b.rows[i], L)
        dk = np.concatenate([k_img[pg].transpose(1, 0, 2) for pg in b.rows[i]])
        dv = np.concatenate([v_img[pg].transpose(1, 0, 2) for pg in b.rows[i]])
        assert np.array_equal(dk[:L], gk) and np.array_equal(dv[:L], gv), i
        assert np.all(dk[L:] == 0) and np.all(dv[L:] == 0), i
    dp.close()


@pytest.mark.parametrize("geom", GEOMS, ids=["d64", "d128"])
def test_gather_returns_what_was_appended(geom):
    dp = DualPool(geom, 32, seed=12)
    b = Batch(dp, [77, 5])
    b.write([(0, 0, 77), (1, 0, 5)])
    for i, L in enumerate([77, 5]):
        k_out = torch.empty((L, geom.n_kv_heads, geom.head_dim), dtype=torch.bfloat16, device="cuda")
        v_out = torch.empty_like(k_out)
        row = torch.tensor(b.rows[i], dtype=torch.int32, device="cuda")
        kvattn.kv_gather(dp.pool, row, L, k_out, v_out)
        k, v = b.kv(i, 0, L)
        assert torch.equal(k_out.view(torch.int16), k.view(torch.int16))
        assert torch.equal(v_out.view(torch.int16), v.view(torch.int16))
        hk, hv = dp.host.gather(b.rows[i], L)
        assert np.array_equal(hk, synth.bf16_bits(k_out)) and np.array_equal(hv, synth.bf16_bits(v_out))
    dp.close()


def test_bad_block_table_is_reported_not_dereferenced():
    geom = GEOMS[0]
    dp = DualPool(geom, 16, seed=13, with_oracle=False)
    dev = "cuda"
    bt = torch.tensor([[3, 99, -1], [2, 1, -1]], dtype=torch.int32, device=dev)     # 99 is outside the pool
    lens = torch.tensor([20, 20], dtype=torch.int32, device=dev)
    assert kvattn.kv_check_batch(dp.pool, bt, lens) == kvattn.KV_ERR_BOUNDS
    assert kvattn.kv_check_batch(dp.pool, bt, torch.tensor([16, 20], dtype=torch.int32, device=dev)) == kvattn.KV_OK
    assert kvattn.kv_check_batch(dp.pool, bt, torch.tensor([16, 49], dtype=torch.int32, device=dev)) == kvattn.KV_ERR_BOUNDS
    # append through the bad entry: the store is skipped and the status word set
    k = synth.normal_bf16(1, synth.TAG_K, 0, 0, 20, geom.n_kv_heads, geom.head_dim, dev)
    before = dp.k_buf.clone()
    kvattn.kv_append(dp.pool, k, k, torch.tensor([0, 20], dtype=torch.int32, device=dev),
                     torch.tensor([0], dtype=torch.int32, device=dev), None, bt)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_ERR_BOUNDS
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK                     # cleared by the read
    changed = (dp.k_buf != before).nonzero().flatten()
    blk = 16 * geom.head_dim * geom.n_kv_heads
    assert set((changed // blk).tolist()) == {3}                                    # only page 3 was written
    # decode through the bad entry: flagged, no fault
    q = synth.normal_bf16(1, synth.TAG_Q, 0, 0, 2, geom.n_q_heads, geom.head_dim, dev)
    out, lse = torch.empty_like(q), torch.empty((2, geom.n_q_heads), device=dev)
    kvattn.attn_decode(dp.pool, q, bt, lens, 20, geom.scale, out, lse)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_ERR_BOUNDS
    dp.close()


def test_evict_with_poison_overwrites_the_pages():
    geom = GEOMS[0]
    pool = kvattn.kv_pool_create(8, 16, geom.n_kv_heads, geom.head_dim)
    kvattn.kv_pool_set_poison(pool, True)
    ids = kvattn.kv_alloc(pool, 3)
    k = synth.normal_bf16(2, synth.TAG_K, 0, 0, 48, geom.n_kv_heads, geom.head_dim, "cuda")
    bt = torch.tensor([ids], dtype=torch.int32, device="cuda")
    kvattn.kv_append(pool, k, k, torch.tensor([0, 48], dtype=torch.int32, device="cuda"),
                     torch.tensor([0], dtype=torch.int32, device="cuda"), None, bt)
    kvattn.kv_evict(pool, [ids[1]])
    out = torch.empty_like(k)
    kvattn.kv_gather(pool, bt[0].contiguous(), 48, out, torch.empty_like(k))
    torch.cuda.synchronize()
    assert torch.isnan(out[16:32].float()).all() and torch.equal(out[:16], k[:16]) and torch.equal(out[32:], k[32:])
    pool.destroy()


def test_owners_pins_and_lru_follow_the_oracle():
    # Random walk over every allocator call; the library and the oracle must agree on each result, each error
    # and the state of every page after each call.
    n_pages = 24
    pool = kvattn.kv_pool_create(n_pages, 16, 2, 64)
    ref = orc.FreeList(n_pages)
    rng = np.random.default_rng(23)
    errs = {kvattn.KV_ERR_NOT_ALLOCATED: KeyError, kvattn.KV_ERR_PINNED: orc.PinnedError, kvattn.KV_ERR_INVALID: ValueError}
    calls = [("free", kvattn.kv_free, ref.free), ("evict", kvattn.kv_evict, ref.evict), ("ref", kvattn.kv_ref, ref.ref),
             ("pin", kvattn.kv_pin, ref.pin), ("unpin", kvattn.kv_unpin, ref.unpin), ("touch", kvattn.kv_touch, ref.touch)]
    seen_errors = set()
    for step in range(1500):
        op = int(rng.integers(0, 9))
        if op == 0:
            n = int(rng.integers(0, 6))
            want = ref.alloc(n)
            if want is None:
                with pytest.raises(kvattn.KvError) as e:
                    kvattn.kv_alloc(pool, n)
                assert e.value.status == kvattn.KV_ERR_OOM
            else:
                assert kvattn.kv_alloc(pool, n) == want
        elif op == 7:
            n = int(rng.integers(0, 4))
            assert kvattn.kv_evict_lru(pool, n) == ref.evict_lru(n)
        elif op == 8:
            if rng.random() < 0.1:
                assert kvattn.kv_unpin_all(pool) == ref.unpin_all()
        else:
            name, lib_fn, ref_fn = calls[op - 1]
            # mostly live pages, sometimes a stray or repeated id
            live = [p for p in range(n_pages) if ref.allocated[p]]
            k = int(rng.integers(1, 4))
            ids = [int(rng.choice(live)) if live and rng.random() < 0.9 else int(rng.integers(0, n_pages)) for _ in range(k)]
            try:
                ref_fn(list(ids))
                expect = None
            except (KeyError, orc.PinnedError, ValueError) as ex:
                expect = type(ex)
            if expect is None:
                lib_fn(pool, ids)
            else:
                with pytest.raises(kvattn.KvError) as e:
                    lib_fn(pool, ids)
                assert errs[e.value.status] is expect, (name, ids, e.value.status)
                seen_errors.add(e.value.status)
        free, used, ev = kvattn.kv_pool_stats(pool)
        assert (free, ev) == (ref.free_pages, ref.evicted_total)
        for p in range(n_pages):
            assert kvattn.kv_page_info(pool, p) == (int(ref.allocated[p]), ref.refs[p], ref.pins[p] if ref.allocated[p] else 0) \
                or not ref.allocated[p]
    assert seen_errors == set(errs)                                   # every kind of refusal was exercised
    pool.destroy()
