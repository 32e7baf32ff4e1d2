"""The scheduler simulator driving the library: its page bookkeeping goes through kv_alloc / kv_ref / kv_pin / kv_unpin /
kv_free / kv_evict_lru / kv_unpin_all of a real pool, and every scheduled prefill and decode step runs the attention
calls on the GPU.  The same schedule on the host stand-in must take the same decisions."""
import dataclasses

import pytest
import torch

from paper_2607_23815_b200 import kvattn, synth
from paper_2607_23815_b200.scheduler import HostEngine, LibraryEngine, LibraryExecutor, Scheduler, StageSpec

pytestmark = pytest.mark.gpu

PLAN = [StageSpec("sem_filter", (500, 900), (1, 1), 8, 0.7, 5), StageSpec("join + sem_map", (20, 50), (3, 9), 16, 1.0, 1)]


def _stats(s):
    return {k: v for k, v in dataclasses.asdict(s).items() if k != "budget_trace"}


@pytest.mark.parametrize("pinning,policy,pages", [("explicit", "memory_aware", 1024), ("virtual", "memory_aware", 1024),
                                                  ("virtual", "breadth_first", 640)])
def test_scheduler_drives_the_pool_and_the_attention_calls(pinning, policy, pages):
    geom = synth.Geometry(8, 2, 128)
    pool = kvattn.kv_pool_create(pages, 16, geom.n_kv_heads, geom.head_dim)
    ex = LibraryExecutor(pool, geom, seed=21)
    sch = Scheduler(PLAN, 24, LibraryEngine(pool), pinning=pinning, policy=policy, seed=21, executor=ex, tokens_per_tick=4096)
    st = sch.run()
    torch.cuda.synchronize()
    assert kvattn.kv_last_async_status(pool) == kvattn.KV_OK                     # no table entry or length out of bounds
    assert torch.isfinite(ex.last_out.float()).all()
    free, used, evicted = kvattn.kv_pool_stats(pool)
    assert free == pages and used == 0 and evicted == st.evicted_pages
    assert ex.calls["extend_append"] > 0 and ex.calls["decode"] > 0
    assert ex.rows["prefill"] == st.prefilled_tokens
    # the library's allocator and the host stand-in give the scheduler the same answers: same schedule
    ref = Scheduler(PLAN, 24, HostEngine(pages), pinning=pinning, policy=policy, seed=21, tokens_per_tick=4096).run()
    assert _stats(ref) == _stats(st) and ref.budget_trace == st.budget_trace
    if policy == "breadth_first":
        assert st.prefix_misses > 0 and st.evicted_pages > 0                       # prefixes lost, prefilled again
    else:
        assert st.prefix_misses == 0
    pool.destroy()
