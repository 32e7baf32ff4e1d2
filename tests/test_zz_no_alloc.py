"""attn_decode_static: the decode entry point for callers that are not allowed to allocate device memory.

Some users of this library run where cudaMalloc is off the table: a plugin that only gets the buffers its host
hands it, a region a framework has memory-planned or is capturing, a serving process that freezes its allocator
after start-up.  They cannot build the workspace attn_decode wants, so the library carries a fixed scratch array
for them.  The test drives the entry point through the C ABI twice in a row (the array keeps the first call's
contents, and the second call must not care), asks for the same bits as the regular entry point, compares both
with the oracle and watches the free device memory across the call.  It sits in a file that sorts last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from oracle import paged_attention as orc
from harness import Batch, DualPool, assert_close

pytestmark = pytest.mark.gpu


def _decode_both(dp, batch, ctx):
    """The same batch through attn_decode (caller's workspace) and attn_decode_static (the library's array); the
    free device memory is read around the second call: the static entry point must not change it."""
    g, dev = dp.geom, dp.device
    q = torch.cat([batch.q(i, max(c - 1, 0), max(c - 1, 0) + 1) for i, c in enumerate(ctx)]).contiguous()
    bt_np = batch.block_tables()
    bt = torch.from_numpy(bt_np).to(dev)
    cl = torch.tensor(ctx, dtype=torch.int32, device=dev)
    max_c = max(max(ctx), 0)
    ref_o, ref_l = torch.full_like(q, float("nan")), torch.full((len(ctx), g.n_q_heads), float("nan"), device=dev)
    ws = torch.empty(max(kvattn.attn_workspace_bytes(dp.pool, g.n_q_heads, 0, 0, 0, len(ctx), max_c), 256),
                     dtype=torch.uint8, device=dev)
    kvattn.attn_decode(dp.pool, q, bt, cl, max_c, g.scale, ref_o, ref_l, ws)
    got_o, got_l = torch.full_like(q, float("nan")), torch.full_like(ref_l, float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    kvattn.attn_decode_static(dp.pool, q, bt, cl, max_c, g.scale, got_o, got_l)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    o_ref, l_ref = orc.attn_decode(dp.host, synth.bf16_bits(q), g.n_q_heads, bt_np, ctx, g.scale)
    return (got_o, got_l), (ref_o, ref_l), (o_ref, l_ref), free_before - free_after


def _check_case(dp, batch, ctx, warm):
    (got_o, got_l), (ref_o, ref_l), (o_ref, l_ref), grew = _decode_both(dp, batch, ctx)
    # the two entry points launch the same kernels with the same split sizes and merge order: same bits
    assert torch.equal(got_o.view(torch.int16), ref_o.view(torch.int16))
    assert torch.equal(got_l.view(torch.int32), ref_l.view(torch.int32))
    # and both are right: against the oracle, within the tolerances every other decode test uses
    res = {"o": got_o.float().cpu().numpy().astype(np.float64), "lse": got_l.cpu().numpy().astype(np.float64),
           "o_ref": o_ref, "lse_ref": l_ref}
    assert_close(res, "attn_decode_static")
    if warm:   # (the first call on a device may make the driver load the module that holds the array)
        assert grew == 0, f"free device memory shrank by {grew} bytes across attn_decode_static"


def test_static_scratch_decode_matches_the_workspace_version_twice_in_a_row():
    geom = synth.Geometry(32, 8, 128)
    dp = DualPool(geom, 1024, seed=909)
    # first call: long contexts (several split-KV chunks per row fill the shared array) ...
    ctx_a = [4096, 1300, 513, 2049, 17]
    a = Batch(dp, ctx_a)
    a.write([(i, 0, c) for i, c in enumerate(ctx_a)])
    # ... second call: other sequences with fewer chunks, so stale partials of the first call lie next to its own
    ctx_b = [700, 1025, 90, 3000]
    b = Batch(dp, ctx_b, uid0=50)
    b.write([(i, 0, c) for i, c in enumerate(ctx_b)])
    _check_case(dp, a, ctx_a, warm=False)
    _check_case(dp, b, ctx_b, warm=True)
    _check_case(dp, a, ctx_a, warm=True)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
    dp.close()


def test_static_scratch_short_contexts_and_empty_rows():
    # contexts of at most one chunk need no scratch at all (the kernel writes the result directly), and rows with a
    # context length of zero or less get O = 0, LSE = -inf; both through the static entry point
    geom = synth.Geometry(8, 2, 128)
    dp = DualPool(geom, 512, seed=911)
    ctx_a = [1024, 1, 0, 513, 16]
    a = Batch(dp, [max(c, 1) for c in ctx_a])
    a.write([(i, 0, c) for i, c in enumerate(ctx_a) if c > 0])
    _check_case(dp, a, ctx_a, warm=False)
    ctx_b = [1500, 0, -3, 1025]
    b = Batch(dp, [max(c, 1) for c in ctx_b], uid0=70)
    b.write([(i, 0, c) for i, c in enumerate(ctx_b) if c > 0])
    (got_o, got_l), _, _, _ = _decode_both(dp, b, ctx_b)
    assert torch.all(got_o[1:3].float() == 0) and torch.all(torch.isneginf(got_l[1:3]))
    _check_case(dp, b, ctx_b, warm=True)
    dp.close()


def test_static_scratch_refuses_batches_beyond_its_limit():
    geom = synth.Geometry(32, 8, 128)
    dp = DualPool(geom, 512, seed=910, with_oracle=False)
    limit = kvattn.attn_decode_static_scratch_bytes()
    assert limit == 8 << 20
    batch, max_ctx = 256, 4096                                           # needs about 17 MB of partials
    assert kvattn.attn_workspace_bytes(dp.pool, geom.n_q_heads, 0, 0, 0, batch, max_ctx) > limit
    q = torch.zeros((batch, geom.n_q_heads, geom.head_dim), dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros((batch, 256), dtype=torch.int32, device="cuda")
    cl = torch.ones(batch, dtype=torch.int32, device="cuda")            # (lengths are small; the bound is what counts)
    before = kvattn.kvattn_launch_count()
    with pytest.raises(kvattn.KvError) as e:
        kvattn.attn_decode_static(dp.pool, q, bt, cl, max_ctx, geom.scale, torch.empty_like(q),
                                  torch.empty((batch, geom.n_q_heads), device="cuda"))
    assert e.value.status == kvattn.KV_ERR_WORKSPACE
    assert kvattn.kvattn_launch_count() == before                        # nothing was launched
    dp.close()
