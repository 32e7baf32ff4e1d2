"""Host-side simulator of the paper's memory-aware scheduler (Algorithm 1: Schedule / Launch / Complete /
Rebalance; Section 5.3) on top of the page pool this library provides.

The scheduler is the part of the paper that decides WHEN the calls of this library are made: it admits a task
(one stage of the query plan on one tuple) only while its stage has budget left, keeps a finished task's prefix
pages alive until the dependent tasks that a Cartesian product created from it are done, releases them then
(kv_free), and moves budget between stages when a stage's waiting queue says it starves or saturates.  It does no
attention arithmetic.  Everything here is plain host Python; the pool it drives is either the library's
(LibraryEngine: kv_alloc / kv_ref / kv_pin / kv_unpin / kv_free / kv_evict_lru / kv_unpin_all, optionally with the
attention calls of every step executed on the GPU) or a host stand-in with the same allocator rules (HostEngine),
so that the policy can be tested without a GPU.

What is restated from the paper, and where:
  * stages, tasks, dependent tasks of a Cartesian product, one waiting queue per stage          Section 5.1
  * Schedule loop, Launch (first-in-first-out admission per stage while the memory manager admits),
    Complete (retry on a token-bound overflow, children through the Cartesian product, dependency tracking,
    release when filtered or in the last stage, a parent released with its last child), Rebalance          Algorithm 1
  * budgets: every stage at least minBudget_s (one task plus its cached prefix), all the rest to the last stage
    at the start; thresholds high_s = alpha * budget_s / minBudget_s, low_s = beta * budget_s / minBudget_s;
    saturation moves a block Delta to the last stage (from the saturated stage if it has Delta unused, else from
    the first stage, scanning downstream, that has), never for the first stage; starvation moves budget from the
    starving stage to the stage upstream of it, walking from the last stage to the first                    Section 5.3
  * token bound per task, interrupted and re-enqueued with a larger bound when it is reached               Section 6
  * explicit pinning (prefix pages of a task with unfinished dependants are pinned) and virtual pinning (nothing is
    pinned; admission alone keeps the engine's least-recently-used eviction away from needed prefixes)     Section 6
  * deadlock: requests waiting, none running -> unpin everything and continue with virtual pinning         Section 6
Readings where the paper leaves a choice (alpha = 1, beta = 0.5 are its evaluation's values, Section 7.1):
  * Delta is not given: one minBudget of the receiving stage by default;
  * the amount moved on starvation is not given: Delta as well, and never below the giver's minBudget or its
    memory in use;
  * time is a discrete tick; a running task needs ceil(prefill_tokens / tokens_per_tick) ticks plus one tick per
    generated token.
"""
from __future__ import annotations

import collections
import dataclasses
import math
from typing import Callable, Deque, Dict, List, Optional, Sequence

PAGE = 16


def pages_for(tokens: int) -> int:
    return (tokens + PAGE - 1) // PAGE


# --------------------------------------------------------------------------------------------------------------
# the pool the scheduler drives
# --------------------------------------------------------------------------------------------------------------
class HostEngine:
    """Host stand-in for the library's page pool with the same allocator rules: all-or-nothing alloc, counted
    owners (ref / free), counted pins, least-recently-used eviction of unpinned pages, unpin_all."""

    def __init__(self, num_pages: int):
        self.num_pages = num_pages
        self.free_list: List[int] = list(range(num_pages - 1, -1, -1))
        self.refs = [0] * num_pages
        self.pins = [0] * num_pages
        self.last_use = [0] * num_pages
        self.clock = 0
        self.evicted_total = 0

    def free_pages(self) -> int:
        return len(self.free_list)

    def alloc(self, n: int) -> Optional[List[int]]:
        if n > len(self.free_list):
            return None
        ids = [self.free_list.pop() for _ in range(n)]
        for p in ids:
            self.refs[p], self.pins[p] = 1, 0
            self.clock += 1
            self.last_use[p] = self.clock
        return ids

    def ref(self, ids: Sequence[int]):
        for p in ids:
            assert self.refs[p] > 0
            self.refs[p] += 1

    def free(self, ids: Sequence[int]):
        for p in ids:
            assert self.refs[p] > 0 and not (self.pins[p] > 0 and self.refs[p] == 1)
            self.refs[p] -= 1
            if self.refs[p] == 0:
                self.free_list.append(p)

    def pin(self, ids: Sequence[int]):
        for p in ids:
            assert self.refs[p] > 0
            self.pins[p] += 1

    def unpin(self, ids: Sequence[int]):
        for p in ids:
            assert self.pins[p] > 0
            self.pins[p] -= 1

    def unpin_all(self) -> int:
        n = sum(1 for c in self.pins if c > 0)
        self.pins = [0] * self.num_pages
        return n

    def touch(self, ids: Sequence[int]):
        for p in ids:
            self.clock += 1
            self.last_use[p] = self.clock

    def evict_lru(self, n: int) -> List[int]:
        cand = sorted((p for p in range(self.num_pages) if self.refs[p] > 0 and self.pins[p] == 0),
                      key=lambda p: self.last_use[p])[:n]
        for p in cand:
            self.refs[p] = 0
            self.free_list.append(p)
        self.evicted_total += len(cand)
        return cand


class LibraryEngine:
    """The same interface over a pool of the CUDA library (needs a GPU: the pool owns device memory)."""

    def __init__(self, pool):
        from . import kvattn
        self.kv, self.pool = kvattn, pool
        self.num_pages = pool.num_pages

    def free_pages(self) -> int:
        return self.kv.kv_pool_stats(self.pool)[0]

    def alloc(self, n):
        try:
            return self.kv.kv_alloc(self.pool, n)
        except self.kv.KvError as e:
            if e.status == self.kv.KV_ERR_OOM:
                return None
            raise

    def ref(self, ids): self.kv.kv_ref(self.pool, ids)
    def free(self, ids): self.kv.kv_free(self.pool, ids)
    def pin(self, ids): self.kv.kv_pin(self.pool, ids)
    def unpin(self, ids): self.kv.kv_unpin(self.pool, ids)
    def unpin_all(self): return self.kv.kv_unpin_all(self.pool)
    def touch(self, ids): self.kv.kv_touch(self.pool, ids)
    def evict_lru(self, n): return self.kv.kv_evict_lru(self.pool, n)


# --------------------------------------------------------------------------------------------------------------
# query plan, tasks
# --------------------------------------------------------------------------------------------------------------
def _mix(*xs: int) -> int:
    """Counter-based hash (splitmix64 steps) of a few integers: every random draw of the simulator is a function of
    (seed, what, which task) and does not depend on the order of execution."""
    z = 0x9E3779B97F4A7C15
    for x in xs:
        z = (z ^ (x & 0xFFFFFFFFFFFFFFFF)) * 0xBF58476D1CE4E5B9 & 0xFFFFFFFFFFFFFFFF
        z = (z ^ (z >> 29)) * 0x94D049BB133111EB & 0xFFFFFFFFFFFFFFFF
        z ^= z >> 32
    return z


def _unit(*xs: int) -> float:
    return (_mix(*xs) >> 11) / float(1 << 53)


@dataclasses.dataclass
class StageSpec:
    """One stage of a pipeline: the operators that run on a tuple between two Cartesian products.

    new_tokens: (lo, hi) tokens the stage's prompt adds to the tuple's context (the operator instruction and, behind a
    Cartesian product, the right-side tuple); for stage 0 this is the scanned tuple itself.  out_tokens: (lo, hi)
    tokens the task generates.  token_bound: tokens of output memory reserved at admission.  pass_rate: probability
    that the stage's predicate keeps the tuple.  fanout: dependent tasks the Cartesian product behind this stage
    creates per surviving tuple (ignored for the last stage)."""
    name: str
    new_tokens: tuple
    out_tokens: tuple = (1, 1)
    token_bound: int = 8
    pass_rate: float = 1.0
    fanout: int = 1


@dataclasses.dataclass
class Task:
    uid: int
    stage: int
    parent: Optional["Task"]
    new_tokens: int                 # tokens this task's prompt adds behind its parent's context
    out_tokens: int                 # tokens it will generate (unknown to the scheduler)
    bound: int                      # output tokens reserved for it
    # filled at launch
    reuse_tokens: int = 0           # leading tokens found in the parent's pages (full pages only)
    extend_tokens: int = 0          # tokens prefilled by this task (the rest of the parent's context + its own)
    table: List[int] = dataclasses.field(default_factory=list)   # block table: reused pages, then own pages
    own_pages: List[int] = dataclasses.field(default_factory=list)
    table_owner: List[int] = dataclasses.field(default_factory=list)  # uid of the task that wrote each page of `table`
    reserved: int = 0               # pages charged to the stage's budget
    ctx_tokens: int = 0             # context length when done
    remaining_prefill: int = 0
    generated: int = 0
    children_left: int = 0
    done: bool = False
    released: bool = False
    pinned: bool = False            # its own pages are pinned by the scheduler (running, or explicit pinning)
    lost: bool = False              # some of its pages were evicted after it finished
    retries: int = 0


@dataclasses.dataclass
class StageState:
    spec: StageSpec
    min_budget: int
    budget: int
    used: int = 0
    waiting: Deque[Task] = dataclasses.field(default_factory=collections.deque)

    def high(self, alpha: float) -> float:
        return alpha * self.budget / self.min_budget

    def low(self, beta: float) -> float:
        return beta * self.budget / self.min_budget


@dataclasses.dataclass
class Stats:
    ticks: int = 0
    launched: int = 0
    completed: int = 0
    filtered: int = 0
    outputs: int = 0
    retries: int = 0
    prefix_hits: int = 0            # launches of dependent tasks that found all reusable pages
    prefix_misses: int = 0          # ... that found fewer (the rest is prefilled again)
    reused_tokens: int = 0
    prefilled_tokens: int = 0
    recomputed_tokens: int = 0      # tokens prefilled again because their pages had been evicted
    evicted_pages: int = 0
    saturation_moves: int = 0
    starvation_moves: int = 0
    deadlocks: int = 0
    peak_pages: int = 0
    budget_trace: List[List[int]] = dataclasses.field(default_factory=list)


# --------------------------------------------------------------------------------------------------------------
# the scheduler
# --------------------------------------------------------------------------------------------------------------
class Scheduler:
    """Algorithm 1 for one pipeline.  `engine` is a HostEngine or a LibraryEngine; `executor` (optional) is told which
    tasks prefill and which decode in every tick and may run the library's attention calls for them.

    policy "memory_aware" is the paper's; "breadth_first" admits whatever the pool can hold, first stage first, with no
    stage budgets (the strawman of Section 5.2 that saturates the cache)."""

    def __init__(self, stages: Sequence[StageSpec], n_tuples: int, engine, budget_pages: Optional[int] = None,
                 alpha: float = 1.0, beta: float = 0.5, delta: Optional[int] = None, pinning: str = "explicit",
                 tokens_per_tick: int = 8192, seed: int = 0, executor=None, policy: str = "memory_aware"):
        assert pinning in ("explicit", "virtual") and policy in ("memory_aware", "breadth_first")
        assert 0 < beta < alpha <= 1.0
        self.engine, self.executor, self.seed = engine, executor, seed
        self.alpha, self.beta, self.pinning, self.policy = alpha, beta, pinning, policy
        self.tokens_per_tick = tokens_per_tick
        total = engine.num_pages if budget_pages is None else budget_pages
        self.stages: List[StageState] = []
        for i, sp in enumerate(stages):
            carry = PAGE - 1 if i > 0 else 0                   # tokens of the parent's last, partly filled page
            mb = pages_for(carry + sp.new_tokens[1] + sp.token_bound)
            self.stages.append(StageState(sp, mb, mb))
        rest = total - sum(s.min_budget for s in self.stages[:-1])
        if rest < self.stages[-1].min_budget:
            raise ValueError("the budget does not hold one task per stage")
        self.stages[-1].budget = rest
        if policy == "breadth_first":
            for s in self.stages:
                s.budget = total
        self.delta = delta
        self.running: List[Task] = []
        self.out: List[Task] = []
        self.stats = Stats()
        self.live: Dict[int, int] = {}                         # page -> uid of the task whose tokens it holds
        self.by_uid: Dict[int, Task] = {}
        self._next_uid = 0
        for t in range(n_tuples):
            self.stages[0].waiting.append(self._make_task(0, None, t))

    # ---- tasks ------------------------------------------------------------------------------------------------
    def _make_task(self, stage: int, parent: Optional[Task], index: int) -> Task:
        sp = self.stages[stage].spec
        uid = self._next_uid
        self._next_uid += 1
        key = (self.seed, stage, parent.uid if parent else -1, index)
        lo, hi = sp.new_tokens
        new = lo + _mix(1, *key) % (hi - lo + 1)
        lo, hi = sp.out_tokens
        out = lo + _mix(2, *key) % (hi - lo + 1)
        t = Task(uid, stage, parent, new, out, sp.token_bound)
        self.by_uid[uid] = t
        return t

    def _hit_pages(self, task: Task) -> int:
        """Leading full pages of the parent's context that are still in the pool."""
        p = task.parent
        if p is None:
            return 0
        n = 0
        for page, owner in zip(p.table[:p.ctx_tokens // PAGE], p.table_owner):
            if self.live.get(page) != owner:
                break
            n += 1
        return n

    def _need(self, task: Task) -> int:
        """Pages the task's own part takes if launched now (what admission charges to the stage)."""
        ctx = task.parent.ctx_tokens if task.parent else 0
        return pages_for(ctx - self._hit_pages(task) * PAGE + task.new_tokens + task.bound)

    # ---- pool with eviction -------------------------------------------------------------------------------------
    def _alloc(self, n: int) -> Optional[List[int]]:
        ids = self.engine.alloc(n)
        if ids is None:
            # the engine makes room the way a prefix cache does: least recently used pages that nothing pins
            evicted = self.engine.evict_lru(n - self.engine.free_pages())
            self.stats.evicted_pages += len(evicted)
            for pg in evicted:
                owner = self.by_uid.get(self.live.pop(pg, -1))
                if owner is not None:
                    owner.lost = True
            ids = self.engine.alloc(n)
        return ids

    # ---- Launch ---------------------------------------------------------------------------------------------------
    def _try_launch(self, st: StageState, ignore_budget: bool = False) -> bool:
        task = st.waiting[0]
        need = self._need(task)
        if not ignore_budget and st.used + need > st.budget:
            return False
        hit = self._hit_pages(task)
        reused = task.parent.table[:hit] if task.parent else []
        if reused:                                   # a running request's pages are never evicted: hold them first
            self.engine.ref(reused)
            self.engine.pin(reused)
        own = self._alloc(need)
        if own is None:
            if reused:
                self.engine.unpin(reused)
                self.engine.free(reused)
            return False
        st.waiting.popleft()
        self.engine.pin(own)
        task.pinned = True
        ctx = task.parent.ctx_tokens if task.parent else 0
        task.reuse_tokens = hit * PAGE
        task.extend_tokens = ctx - task.reuse_tokens + task.new_tokens
        task.own_pages, task.table = own, list(reused) + own
        task.table_owner = (task.parent.table_owner[:hit] if task.parent else []) + [task.uid] * len(own)
        for pg in own:
            self.live[pg] = task.uid
        task.reserved = need
        st.used += need
        task.remaining_prefill, task.generated = task.extend_tokens, 0
        self.running.append(task)
        s = self.stats
        s.launched += 1
        s.reused_tokens += task.reuse_tokens
        s.prefilled_tokens += task.extend_tokens
        if task.parent is not None:
            full = task.parent.ctx_tokens // PAGE
            if hit == full:
                s.prefix_hits += 1
            else:
                s.prefix_misses += 1
                s.recomputed_tokens += (full - hit) * PAGE
        return True

    def launch(self) -> List[Task]:
        started = []
        for st in self.stages:
            while st.waiting:
                before = len(self.running)
                if not self._try_launch(st):
                    break
                started.append(self.running[before])
        return started

    # ---- Complete ---------------------------------------------------------------------------------------------------
    def _drop_reused(self, task: Task):
        n = task.reuse_tokens // PAGE
        if n:
            self.engine.unpin(task.table[:n])
            self.engine.free(task.table[:n])

    def _own_live(self, task: Task) -> List[int]:
        return [pg for pg in task.own_pages if self.live.get(pg) == task.uid]

    def _release(self, task: Task):
        """releaseMemory: the task's pages go back to the pool, its stage gets the budget back, and its parent follows
        when this was the parent's last dependent task."""
        if task.released:
            return
        task.released = True
        mine = self._own_live(task)
        pinned = task.pinned
        if pinned:
            self.engine.unpin(mine)
            task.pinned = False
        if mine:
            self.engine.free(mine)
        for pg in mine:
            del self.live[pg]
        self.stages[task.stage].used -= task.reserved
        if task.parent is not None:
            task.parent.children_left -= 1
            if task.parent.children_left == 0 and task.parent.done:
                self._release(task.parent)

    def complete(self, task: Task):
        st, sp = self.stages[task.stage], self.stages[task.stage].spec
        last = task.stage == len(self.stages) - 1
        self._drop_reused(task)
        if task.out_tokens > task.bound:
            # the request hit its token bound and was interrupted: give it a larger one and queue it again
            self.engine.unpin(task.own_pages)
            self.engine.free(task.own_pages)
            for pg in task.own_pages:
                del self.live[pg]
            st.used -= task.reserved
            task.bound *= 2
            task.retries += 1
            task.own_pages, task.table, task.table_owner, task.reserved = [], [], [], 0
            self.stats.retries += 1
            st.waiting.append(task)
            return
        task.done, task.pinned = True, True
        task.ctx_tokens = task.reuse_tokens + task.extend_tokens + task.out_tokens
        self.stats.completed += 1
        filtered = _unit(3, self.seed, task.uid) >= sp.pass_rate
        if filtered:
            self.stats.filtered += 1
        elif not last:
            nxt = self.stages[task.stage + 1]
            children = [self._make_task(task.stage + 1, task, c) for c in range(sp.fanout)]   # the Cartesian product
            nxt.waiting.extend(children)
            task.children_left = len(children)                                                 # trackDependency
            if self.pinning == "virtual":
                # nothing stays pinned: the prefix is cached, and stays only as long as admission leaves the engine room
                self.engine.unpin(task.own_pages)
                task.pinned = False
                self.engine.touch(task.own_pages)
        else:
            self.out.append(task)
            self.stats.outputs += 1
        if filtered or last or task.children_left == 0:
            self._release(task)

    # ---- Rebalance ----------------------------------------------------------------------------------------------------
    def _delta(self, receiver: StageState) -> int:
        return self.delta if self.delta is not None else receiver.min_budget

    def _spare(self, st: StageState) -> int:
        return st.budget - max(st.used, st.min_budget)

    def rebalance(self):
        if self.policy != "memory_aware":
            return
        last = self.stages[-1]
        for st in self.stages[1:]:
            if len(st.waiting) > st.high(self.alpha):                        # saturated
                d = self._delta(last)
                giver = st if (st is not last and self._spare(st) >= d) else \
                    next((g for g in self.stages[:-1] if self._spare(g) >= d), None)
                if giver is not None:
                    giver.budget -= d
                    last.budget += d
                    self.stats.saturation_moves += 1
        for i in range(len(self.stages) - 1, 0, -1):
            st, prev = self.stages[i], self.stages[i - 1]
            # (a stage whose upstream stages have nothing left to run cannot be fed by giving them budget)
            upstream_work = any(u.waiting for u in self.stages[:i])
            if upstream_work and len(st.waiting) < st.low(self.beta):        # starving
                d = min(self._delta(prev), self._spare(st))
                if d > 0:
                    st.budget -= d
                    prev.budget += d
                    self.stats.starvation_moves += 1

    # ---- the engine's side: one tick ----------------------------------------------------------------------------------
    def _advance(self) -> List[Task]:
        """One tick of the serving engine: the tick's prefill tokens go to the running tasks in launch order, every task
        that is past its prefill generates one token.  Returns the tasks that finished (or hit their bound)."""
        room, finished, decoding = self.tokens_per_tick, [], []
        for t in self.running:
            if t.remaining_prefill > 0:
                take = min(room, t.remaining_prefill)
                t.remaining_prefill -= take
                room -= take
            elif t.generated < min(t.out_tokens, t.bound):
                t.generated += 1
                decoding.append(t)
                if t.generated == min(t.out_tokens, t.bound):
                    finished.append(t)
            else:
                finished.append(t)
        if self.executor is not None and decoding:
            self.executor.decode(decoding)
        return finished

    # ---- Schedule -----------------------------------------------------------------------------------------------------
    def has_waiting(self) -> bool:
        return any(st.waiting for st in self.stages)

    def tick(self):
        started = self.launch()
        if not started and not self.running and self.has_waiting():
            self._break_deadlock()
            started = self.launch() or self._force_one()
        if self.executor is not None and started:
            self.executor.prefill(started)
        for t in self._advance():
            self.running.remove(t)
            self.complete(t)
        self.rebalance()
        s = self.stats
        s.ticks += 1
        s.peak_pages = max(s.peak_pages, self.engine.num_pages - self.engine.free_pages())
        s.budget_trace.append([st.budget for st in self.stages])

    def _break_deadlock(self):
        """Requests wait and nothing runs: with explicit pinning, pinned prefixes may be what keeps them out.  Everything
        is unpinned and the run goes on with virtual pinning (Section 6)."""
        self.stats.deadlocks += 1
        if self.pinning == "explicit":
            self.engine.unpin_all()
            for t in self.by_uid.values():
                t.pinned = False
            self.pinning = "virtual"

    def _force_one(self) -> List[Task]:
        """Still nothing admitted: the most downstream waiting task goes in regardless of its stage's budget, so that
        the pipeline drains from the end (every stage can always run one task)."""
        for st in reversed(self.stages):
            if st.waiting:
                before = len(self.running)
                if self._try_launch(st, ignore_budget=True):
                    return [self.running[before]]
        raise RuntimeError("the pool cannot hold a single waiting task")

    def run(self, max_ticks: int = 10_000_000) -> Stats:
        while self.has_waiting() or self.running:
            if self.stats.ticks >= max_ticks:
                raise RuntimeError("the schedule did not finish")
            self.tick()
        return self.stats


# --------------------------------------------------------------------------------------------------------------
# running the library's calls for the scheduled tasks
# --------------------------------------------------------------------------------------------------------------
class LibraryExecutor:
    """Executes, on the GPU, what the scheduled tasks would ask of one attention layer: a launched task's prefill is
    attn_extend_append of its extend tokens over the pages it reuses, every generated token is a kv_append of that
    token's K/V and an attn_decode over the task's context.  Q/K/V are seeded synthetic values keyed on (task,
    position); nothing here checks numerics (the parity tests do), it checks that the scheduler's page bookkeeping is
    what the kernels can run on: every call must leave the device status clean."""

    def __init__(self, pool, geom, seed: int = 0, device="cuda"):
        import torch
        from . import kvattn, synth
        self.torch, self.kv, self.synth = torch, kvattn, synth
        self.pool, self.geom, self.seed, self.device = pool, geom, seed, device
        self.calls = {"extend_append": 0, "append": 0, "decode": 0}
        self.rows = {"prefill": 0, "decode": 0}

    def _i32(self, x):
        return self.torch.tensor(x, dtype=self.torch.int32, device=self.device)

    def _draw(self, tag, task, pos0, n, heads):
        return self.synth.normal_bf16(self.seed, tag, task.uid, pos0, n, heads, self.geom.head_dim, self.device)

    def _tables(self, tasks):
        width = max(len(t.table) for t in tasks)
        return self._i32([t.table + [-1] * (width - len(t.table)) for t in tasks])

    def prefill(self, tasks):
        g, sy, torch = self.geom, self.synth, self.torch
        tasks = [t for t in tasks if t.extend_tokens > 0]
        if not tasks:
            return
        E, P = [t.extend_tokens for t in tasks], [t.reuse_tokens for t in tasks]
        q = torch.cat([self._draw(sy.TAG_Q, t, t.reuse_tokens, t.extend_tokens, g.n_q_heads) for t in tasks])
        k = torch.cat([self._draw(sy.TAG_K, t, t.reuse_tokens, t.extend_tokens, g.n_kv_heads) for t in tasks])
        v = torch.cat([self._draw(sy.TAG_V, t, t.reuse_tokens, t.extend_tokens, g.n_kv_heads) for t in tasks])
        cu = self._i32([0] + list(__import__("itertools").accumulate(E)))
        out = torch.empty_like(q)
        lse = torch.empty((q.shape[0], g.n_q_heads), dtype=torch.float32, device=self.device)
        max_l = max(p + e for p, e in zip(P, E))
        ws = torch.empty(max(256, self.kv.attn_workspace_bytes(self.pool, g.n_q_heads, len(tasks), int(q.shape[0]), max_l, 0, 0)),
                         dtype=torch.uint8, device=self.device)
        self.kv.attn_extend_append(self.pool, q, k, v, cu, self._tables(tasks), self._i32(P), self._i32(E), max(E), max_l,
                                   g.scale, out, lse, ws)
        self.calls["extend_append"] += 1
        self.rows["prefill"] += int(q.shape[0])
        self.last_out = out

    def decode(self, tasks):
        g, sy, torch = self.geom, self.synth, self.torch
        pos = [t.reuse_tokens + t.extend_tokens + t.generated - 1 for t in tasks]      # the new token's position
        k = torch.cat([self._draw(sy.TAG_K, t, p, 1, g.n_kv_heads) for t, p in zip(tasks, pos)])
        v = torch.cat([self._draw(sy.TAG_V, t, p, 1, g.n_kv_heads) for t, p in zip(tasks, pos)])
        q = torch.cat([self._draw(sy.TAG_Q, t, p, 1, g.n_q_heads) for t, p in zip(tasks, pos)])
        bt = self._tables(tasks)
        self.kv.kv_append(self.pool, k, v, self._i32(list(range(len(tasks) + 1))), self._i32(pos), None, bt)
        ctx = [p + 1 for p in pos]
        out = torch.empty_like(q)
        lse = torch.empty((len(tasks), g.n_q_heads), dtype=torch.float32, device=self.device)
        ws = torch.empty(max(256, self.kv.attn_workspace_bytes(self.pool, g.n_q_heads, 0, 0, 0, len(tasks), max(ctx))),
                         dtype=torch.uint8, device=self.device)
        self.kv.attn_decode(self.pool, q, bt, self._i32(ctx), max(ctx), g.scale, out, lse, ws)
        self.calls["append"] += 1
        self.calls["decode"] += 1
        self.rows["decode"] += len(tasks)
        self.last_out = out
