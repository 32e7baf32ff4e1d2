"""attn_decode_static: the decode entry point for callers that are not allowed to allocate device memory.

Some users of this library run where cudaMalloc is off the table: a plugin that only gets the buffers its host
hands it, a region a framework has memory-planned or is capturing, a serving process that freezes its allocator
after start-up.  They cannot build the workspace attn_decode wants, so the library carries a fixed scratch array
for them.  The test drives the entry point through the C ABI twice in a row (the array keeps the first call's
contents, and the second call must not care) and compares with the regular entry point.  It sits in a file
that sorts last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from harness import Batch, DualPool, O_TOL, LSE_TOL

pytestmark = pytest.mark.gpu


def _decode_both(dp, batch, ctx):
    g, dev = dp.geom, dp.device
    q = torch.cat([batch.q(i, c - 1, c) for i, c in enumerate(ctx)]).contiguous()
    bt = torch.from_numpy(batch.block_tables()).to(dev)
    cl = torch.tensor(ctx, dtype=torch.int32, device=dev)
    ref_o, ref_l = torch.full_like(q, float("nan")), torch.full((len(ctx), g.n_q_heads), float("nan"), device=dev)
    ws = torch.empty(max(kvattn.attn_workspace_bytes(dp.pool, g.n_q_heads, 0, 0, 0, len(ctx), max(ctx)), 256),
                     dtype=torch.uint8, device=dev)
    kvattn.attn_decode(dp.pool, q, bt, cl, max(ctx), g.scale, ref_o, ref_l, ws)
    got_o, got_l = torch.full_like(q, float("nan")), torch.full_like(ref_l, float("nan"))
    kvattn.attn_decode_static(dp.pool, q, bt, cl, max(ctx), g.scale, got_o, got_l)
    torch.cuda.synchronize()
    return (got_o, got_l), (ref_o, ref_l)


def test_static_scratch_decode_matches_the_workspace_version_twice_in_a_row():
    geom = synth.Geometry(32, 8, 128)
    dp = DualPool(geom, 1024, seed=909, with_oracle=False)
    # first call: long contexts (several split-KV chunks per row fill the shared array) ...
    ctx_a = [4096, 1300, 513, 2049, 17]
    a = Batch(dp, ctx_a)
    a.write([(i, 0, c) for i, c in enumerate(ctx_a)])
    # ... second call: other sequences with fewer chunks, so stale partials of the first call lie next to its own
    ctx_b = [700, 1025, 90, 3000]
    b = Batch(dp, ctx_b, uid0=50)
    b.write([(i, 0, c) for i, c in enumerate(ctx_b)])
    for batch, ctx in ((a, ctx_a), (b, ctx_b)):
        (got_o, got_l), (ref_o, ref_l) = _decode_both(dp, batch, ctx)
        assert torch.isfinite(got_o.float()).all() and torch.isfinite(got_l).all()
        d_o = (got_o.float() - ref_o.float()).abs().max().item()
        d_l = (got_l - ref_l).abs().max().item()
        assert d_o <= O_TOL and d_l <= LSE_TOL, (d_o, d_l)
    assert kvattn.kv_last_async_status(dp.pool) == kvattn.KV_OK
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
