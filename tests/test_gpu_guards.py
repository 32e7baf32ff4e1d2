"""The guards that a healthy run never exercises: a bounded device-side wait that runs out, guard bands around every
buffer the attention kernels write, and the report for host-side bounds that the device finds too small."""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, assert_close, run_decode, run_extend

pytestmark = pytest.mark.gpu

GUARD = 4096                      # bytes before and after each buffer
PATTERN = 0xA5


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    # One CTA of a test-only kernel waits, with the wait the attention kernels use, on barriers that nothing completes
    # (limit 1 ms): the first waiter gives up and raises the abort flag, the parked warp leaves because of the flag,
    # the bulk copy in flight lands, tensor memory is freed, KV_ERR_TIMEOUT is recorded.  Then real work runs.
    geom = synth.Geometry(8, 2, 128)
    dp = DualPool(geom, 64, seed=77)
    trace = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    kvattn.kvattn_selftest_bounded_wait(dp.pool, 1_000_000, trace)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_ERR_TIMEOUT      # synchronises, returns and clears
    t = trace.cpu().tolist()
    assert t[0] == 1 and t[1] == 32 and t[2] == 1, t
    assert 1_000_000 <= t[3] < 50_000_000, t                                  # gave up after the limit, not much later
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK               # cleared
    # the context is alive: tensor memory was returned (the extend kernel takes all 512 columns) and results are right
    P, E = [100, 0], [40, 130]
    b = Batch(dp, [p + e for p, e in zip(P, E)])
    b.write([(i, 0, P[i] + E[i]) for i in range(2)])
    assert_close(run_extend(dp, b, P, E, impl=2), "extend after a timed-out wait")
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


class Guarded:
    """A device buffer of n bytes with a band of a fixed byte pattern on either side."""

    def __init__(self, nbytes, dtype, shape, align=256):
        pad = (-nbytes) % align
        self.raw = torch.full((GUARD + nbytes + pad + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.nbytes = nbytes
        self.view = self.raw[GUARD:GUARD + nbytes].view(dtype).view(shape)

    def intact(self):
        return bool((self.raw[:GUARD] == PATTERN).all() and (self.raw[GUARD + self.nbytes:] == PATTERN).all())


@pytest.mark.parametrize("hq,hkv,d", [(32, 8, 128), (8, 1, 128), (4, 2, 64), (4, 4, 64)])
def test_guard_bands_around_outputs_and_workspace_stay_untouched(hq, hkv, d):
    # compute-sanitizer is not available here, so stray stores are looked for the plain way: O, LSE and the workspace
    # sit between bands of a byte pattern, and the bands must survive extend (tensor-core kernel, ragged last tiles,
    # suffix lengths that are no multiple of 32/G), decode (several chunks per row) and the fan-out call.
    geom = synth.Geometry(hq, hkv, d)
    dev = "cuda"
    P, E = [0, 17, 300, 5, 1030], [33, 1, 77, 129, 5]
    L = [p + e for p, e in zip(P, E)]
    dp = DualPool(geom, sum(synth.pages_needed(x, 16) for x in L) + 160, seed=8000 + hq)
    b = Batch(dp, L)
    b.write([(i, 0, L[i]) for i in range(len(L))])
    i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=dev)
    # ---- extend
    q = torch.cat([b.q(i, P[i], L[i]) for i in range(len(L))]).contiguous()
    T = q.shape[0]
    out = Guarded(T * hq * d * 2, torch.bfloat16, (T, hq, d))
    lse = Guarded(T * hq * 4, torch.float32, (T, hq))
    ws = Guarded(kvattn.attn_workspace_bytes(dp.pool, hq, len(L), T, max(L), 0, 0), torch.uint8, (-1,))
    bt = torch.from_numpy(b.block_tables()).to(dev)
    for impl in (2, 1):
        kvattn.kvattn_set_extend_impl(impl)
        try:
            kvattn.attn_extend(dp.pool, q, i32(np.concatenate([[0], np.cumsum(E)])), bt, i32(P), i32(E), max(E), max(L),
                               geom.scale, out.view, lse.view, ws.view)
        finally:
            kvattn.kvattn_set_extend_impl(0)
        torch.cuda.synchronize()
        assert out.intact() and lse.intact() and ws.intact(), f"extend impl {impl} wrote outside its buffers"
        assert torch.isfinite(out.view.float()).all() and torch.isfinite(lse.view).all()
    # ---- decode over the same sequences (contexts of up to three chunks)
    qd = torch.cat([b.q(i, L[i] - 1, L[i]) for i in range(len(L))]).contiguous()
    od = Guarded(len(L) * hq * d * 2, torch.bfloat16, (len(L), hq, d))
    ld = Guarded(len(L) * hq * 4, torch.float32, (len(L), hq))
    wd = Guarded(max(256, kvattn.attn_workspace_bytes(dp.pool, hq, 0, 0, 0, len(L), max(L))), torch.uint8, (-1,))
    kvattn.attn_decode(dp.pool, qd, bt, i32(L), max(L), geom.scale, od.view, ld.view, wd.view)
    torch.cuda.synchronize()
    assert od.intact() and ld.intact() and wd.intact(), "decode wrote outside its buffers"
    # ---- fan-out: two parents, ragged children
    parent_lens, n_child, child_lens = [48, 304], [3, 4], [5, 37, 1, 16, 33, 130, 9]
    parents = Batch(dp, parent_lens, uid0=500)
    parents.write([(g, 0, parent_lens[g]) for g in range(2)])
    kids = Batch(dp, child_lens, uid0=600)
    kids.write([(c, 0, child_lens[c]) for c in range(len(child_lens))])
    qs = torch.cat([kids.q(c, 0, child_lens[c]) for c in range(len(child_lens))]).contiguous()
    Ts = qs.shape[0]
    cu_children, cu_q = np.concatenate([[0], np.cumsum(n_child)]), np.concatenate([[0], np.cumsum(child_lens)])
    rows = [int(cu_q[cu_children[g + 1]] - cu_q[cu_children[g]]) for g in range(2)]
    for impl in (1, 2):
        os_ = Guarded(Ts * hq * d * 2, torch.bfloat16, (Ts, hq, d))
        ls_ = Guarded(Ts * hq * 4, torch.float32, (Ts, hq))
        wss = Guarded(kvattn.attn_extend_shared_workspace_bytes(dp.pool, hq, 2, len(child_lens), Ts, max(parent_lens)),
                      torch.uint8, (-1,))
        kvattn.kvattn_set_shared_impl(impl)
        try:
            kvattn.attn_extend_shared(dp.pool, qs, i32(cu_q), i32(cu_children), i32(parents.block_tables()), i32(parent_lens),
                                      i32(kids.block_tables()), i32(child_lens), max(child_lens), max(rows), max(parent_lens),
                                      geom.scale, os_.view, ls_.view, wss.view)
        finally:
            kvattn.kvattn_set_shared_impl(0)
        torch.cuda.synchronize()
        assert os_.intact() and ls_.intact() and wss.intact(), f"fan-out impl {impl} wrote outside its buffers"
        assert torch.isfinite(os_.view.float()).all()
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


@pytest.mark.parametrize("impl", [1, 2])
def test_host_bounds_that_are_too_small_are_reported(impl):
    # max_extend_len sizes the grid: a sequence with more suffix tokens than that would lose its last rows without a
    # trace, so the device records KV_ERR_BOUNDS; the rows inside the bound are still right and nothing outside the
    # buffers is touched.  The same for a total_q that is smaller than the rows the device finds.
    geom = synth.Geometry(8, 2, 128)
    dev = "cuda"
    P, E = [40, 0], [300, 20]
    L = [p + e for p, e in zip(P, E)]
    dp = DualPool(geom, 64, seed=8100)
    b = Batch(dp, L)
    b.write([(i, 0, L[i]) for i in range(2)])
    i32 = lambda x: torch.tensor(np.asarray(x), dtype=torch.int32, device=dev)
    q = torch.cat([b.q(i, P[i], L[i]) for i in range(2)]).contiguous()
    T = q.shape[0]
    out = Guarded(T * 8 * 128 * 2, torch.bfloat16, (T, 8, 128))
    lse = Guarded(T * 8 * 4, torch.float32, (T, 8))
    ws = Guarded(kvattn.attn_workspace_bytes(dp.pool, 8, 2, T, max(L), 0, 0), torch.uint8, (-1,))
    bt = torch.from_numpy(b.block_tables()).to(dev)
    kvattn.kvattn_set_extend_impl(impl)
    try:
        kvattn.attn_extend(dp.pool, q, i32([0, 300, 320]), bt, i32(P), i32(E), 64, max(L), geom.scale, out.view, lse.view,
                           ws.view)                                               # 64 < 300
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_ERR_BOUNDS
        assert out.intact() and lse.intact() and ws.intact()
        kvattn.attn_extend(dp.pool, q, i32([0, 300, 320]), bt, i32(P), i32(E), 300, max(L), geom.scale, out.view, lse.view,
                           ws.view)                                               # the right bound: clean
        assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    finally:
        kvattn.kvattn_set_extend_impl(0)
    dp.close()
