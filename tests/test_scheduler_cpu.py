"""The host-side scheduler simulator (Algorithm 1 of the paper) on the host stand-in for the page pool: no GPU."""
import dataclasses

import pytest

from paper_2607_23815_b200.scheduler import HostEngine, PAGE, Scheduler, StageSpec, _unit, pages_for

JOIN = [StageSpec("sem_filter", (1800, 2400), (1, 1), 8, 0.6, 17), StageSpec("join + sem_map", (20, 50), (4, 12), 16, 1.0, 1)]
THREE = [StageSpec("sem_map", (300, 500), (8, 40), 48, 1.0, 3), StageSpec("sem_filter", (10, 30), (1, 1), 8, 0.5, 4),
         StageSpec("sem_map", (10, 40), (2, 10), 16, 1.0, 1)]


def _stats(s):
    return {k: v for k, v in dataclasses.asdict(s).items() if k != "budget_trace"}


@pytest.mark.parametrize("pinning", ["explicit", "virtual"])
@pytest.mark.parametrize("plan,n", [(JOIN, 40), (THREE, 80)])
def test_every_task_runs_once_and_every_page_comes_back(plan, n, pinning):
    eng = HostEngine(4096)
    sch = Scheduler(plan, n, eng, pinning=pinning, seed=11)
    st = sch.run()
    assert eng.free_pages() == 4096 and not sch.live and all(s.used == 0 for s in sch.stages)
    assert all(c == 0 for c in eng.pins)
    # expected outputs by replaying the same draws stage by stage (filter decisions are keyed on the task)
    tasks = [t for t in sch.by_uid.values()]
    assert all(t.done and t.released for t in tasks)
    per_stage = [sum(1 for t in tasks if t.stage == i) for i in range(len(plan))]
    assert per_stage[0] == n
    for i in range(1, len(plan)):
        survivors = sum(1 for t in tasks if t.stage == i - 1 and _unit(3, 11, t.uid) < plan[i - 1].pass_rate)
        assert per_stage[i] == survivors * plan[i - 1].fanout
    assert st.outputs == sum(1 for t in tasks if t.stage == len(plan) - 1 and _unit(3, 11, t.uid) < plan[-1].pass_rate)
    assert st.completed == len(tasks) and st.launched == len(tasks) + st.retries
    # with enough budget nothing the dependants need is ever evicted
    assert st.prefix_misses == 0 and st.recomputed_tokens == 0
    # budgets: conserved, never below a stage's minimum
    total = sum(st.budget_trace[0])
    for row in st.budget_trace:
        assert sum(row) == total and all(b >= s.min_budget for b, s in zip(row, sch.stages))


def test_children_reuse_full_pages_of_the_parent_and_prefill_the_rest():
    eng = HostEngine(2048)
    sch = Scheduler(JOIN, 6, eng, seed=2)
    sch.run()
    for t in sch.by_uid.values():
        if t.parent is None:
            assert t.reuse_tokens == 0 and t.extend_tokens == t.new_tokens
        else:
            assert t.reuse_tokens == PAGE * (t.parent.ctx_tokens // PAGE)                 # block-granular prefix hit
            assert t.extend_tokens == t.parent.ctx_tokens % PAGE + t.new_tokens
            assert t.table[:t.reuse_tokens // PAGE] == t.parent.table[:t.reuse_tokens // PAGE]
        assert len(t.own_pages) == 0 or len(t.own_pages) == pages_for(t.extend_tokens + t.bound)
        assert t.ctx_tokens == t.reuse_tokens + t.extend_tokens + t.out_tokens


def test_parent_pages_stay_until_the_last_dependant_is_released():
    eng = HostEngine(2048)
    sch = Scheduler(JOIN, 3, eng, pinning="explicit", seed=5)
    seen_pinned_parent = False
    while sch.has_waiting() or sch.running:
        sch.tick()
        for t in sch.by_uid.values():
            if t.done and not t.released:
                assert t.children_left > 0
                assert all(eng.refs[p] >= 1 and eng.pins[p] >= 1 for p in t.own_pages)   # explicit pinning
                seen_pinned_parent = True
            if t.released:
                assert all(sch.live.get(p) != t.uid for p in t.own_pages)
    assert seen_pinned_parent


def test_thresholds_and_budget_moves():
    eng = HostEngine(8192)
    sch = Scheduler(THREE, 0, eng, alpha=1.0, beta=0.5, seed=1)
    s0, s1, s2 = sch.stages
    assert s0.budget == s0.min_budget and s1.budget == s1.min_budget
    assert s2.budget == 8192 - s0.min_budget - s1.min_budget                   # the rest goes to the last stage
    assert s2.high(1.0) == s2.budget / s2.min_budget and s2.low(0.5) == 0.5 * s2.budget / s2.min_budget
    # starvation: the last stage has far fewer waiting tasks than low, upstream has work -> budget walks upstream
    s0.waiting.extend(sch._make_task(0, None, i) for i in range(5))
    b = [s.budget for s in sch.stages]
    sch.rebalance()
    # 2 -> 1: one block (a minimum budget of the receiver); then 1 -> 0: what stage 1 can spare above its own minimum
    assert s2.budget == b[2] - s1.min_budget and s1.budget == b[1] and s0.budget == b[0] + s1.min_budget
    assert sch.stats.starvation_moves == 2 and sch.stats.saturation_moves == 0
    # saturation: stage 1 has more waiting tasks than high and spare budget -> a block goes to the last stage
    s1.budget += 10 * s2.min_budget
    parent = sch._make_task(0, None, 99)
    s1.waiting.extend(sch._make_task(1, parent, i) for i in range(int(s1.high(1.0)) + 2))
    s2.waiting.extend(sch._make_task(2, parent, i) for i in range(int(s2.low(0.5)) + 5))      # not starving
    b = [s.budget for s in sch.stages]
    sch.rebalance()
    assert s1.budget == b[1] - s2.min_budget and s2.budget == b[2] + s2.min_budget
    assert sch.stats.saturation_moves == 1
    # the first stage is never treated as saturated
    s1.waiting.clear()
    s0.waiting.extend(sch._make_task(0, None, 100 + i) for i in range(500))
    moves = sch.stats.saturation_moves
    sch.rebalance()
    assert sch.stats.saturation_moves == moves


def test_a_task_that_reaches_its_token_bound_is_queued_again_with_a_larger_one():
    plan = [StageSpec("sem_map", (100, 100), (40, 40), 16, 1.0, 1)]
    eng = HostEngine(256)
    sch = Scheduler(plan, 4, eng, seed=0)
    st = sch.run()
    assert st.retries == 8 and st.outputs == 4                   # 16 -> 32 -> 64 >= 40: two retries per task
    assert all(t.bound == 64 and t.retries == 2 for t in sch.by_uid.values())
    assert eng.free_pages() == 256


def test_memory_aware_admission_keeps_prefixes_under_virtual_pinning_where_breadth_first_loses_them():
    res = {}
    for policy in ("memory_aware", "breadth_first"):
        eng = HostEngine(4096)
        res[policy] = Scheduler(JOIN, 60, eng, pinning="virtual", policy=policy, seed=3).run()
        assert eng.free_pages() == 4096
    assert res["memory_aware"].prefix_misses == 0 and res["memory_aware"].evicted_pages == 0
    assert res["breadth_first"].prefix_misses > 100 and res["breadth_first"].recomputed_tokens > 100_000
    assert res["memory_aware"].ticks < res["breadth_first"].ticks
    assert res["memory_aware"].outputs == res["breadth_first"].outputs


def test_deadlock_falls_back_to_virtual_pinning_and_finishes():
    # retries double the bound beyond what the stage budgets were sized for while explicit pins hold the parents'
    # pages: at some point requests wait and nothing runs; everything is unpinned and the run completes
    plan = [StageSpec("sem_filter", (200, 260), (1, 1), 8, 1.0, 6), StageSpec("sem_map", (10, 20), (100, 140), 16, 1.0, 1)]
    eng = HostEngine(40)
    sch = Scheduler(plan, 12, eng, pinning="explicit", seed=9)
    st = sch.run()
    assert st.deadlocks >= 1 and sch.pinning == "virtual"
    assert st.outputs == 72 and eng.free_pages() == 40 and all(c == 0 for c in eng.pins)


def test_same_seed_same_schedule():
    a = Scheduler(THREE, 50, HostEngine(1024), seed=4).run()
    b = Scheduler(THREE, 50, HostEngine(1024), seed=4).run()
    c = Scheduler(THREE, 50, HostEngine(1024), seed=5).run()
    assert _stats(a) == _stats(b) and a.budget_trace == b.budget_trace and _stats(a) != _stats(c)
