#!/usr/bin/env python
"""Benchmark of the paged-KV attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the hot path over one batch of the headline workload (a downstream
operator's suffixes over reused prefix pages): the suffix K/V rows are appended to their pages and the
suffix attends over prefix + suffix, through the one call that does both (attn_extend_append).
`value` is the extend algorithmic TFLOP/s over the whole step with inputs resident in HBM; `e2e`
is the same with host buffers (pinned host -> device copies and the device -> host read of O/LSE
inside the timed region).  The same line carries the decode (HBM GB/s), bulk-append and mixed
pipeline-step figures, the roofline of the dominant kernel and the CPU oracle timed on a sample.

Multi-GPU: the path has no exchange step, so N ranks run N independent replicas of the workload
(different seeds); time is the max over ranks and value the sum of the ranks' work over that time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_23815_b200 import synth  # noqa: E402

METRIC = "paged extend-attn TFLOP/s"
HEADLINE = "extend_8b"

# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the
# ncu captures summarised under profiles/; None until a capture of that kernel/workload exists.
NCU_TRAFFIC_BYTES = {"extend_8b": 603_000_000, "decode_8b": 2_652_000_000}  # profiles/attn_*_kernel_*.md


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only) in a thread while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, index: int):
        import threading
        self.sm, self.mx, self.reasons, self.err = [], None, set(), None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(visible.split(",")[index]) if visible and visible.split(",")[index].isdigit() else index
            self.nv, self.h = pynvml, pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.mx = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # noqa: BLE001
            self.nv, self.err = None, f"NVML unavailable: {e}"
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        while not self._stop.is_set():
            try:
                self.sm.append(float(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                try:
                    mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:  # noqa: BLE001
                    mask = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception as e:  # noqa: BLE001
                self.err = str(e)
                return
            time.sleep(0.001)

    def stop(self):
        if self.nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": [self.err]}
        self._stop.set()
        self.thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.mx,
                "samples": len(self.sm), "reasons": sorted(self.reasons)}


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return world, rank, local


def max_over_ranks(x: float, world: int) -> float:
    from paper_2607_23815_b200 import ranks
    return ranks.aggregate(x, 0.0, world)[0]


def sum_over_ranks(x: float, world: int) -> float:
    from paper_2607_23815_b200 import ranks
    return ranks.aggregate(0.0, x, world)[1]


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


class L2Flusher:
    def __init__(self, device):
        self.buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)   # 2x the 126 MB L2

    def __call__(self):
        self.buf.zero_()


def time_steps(fn, steps, warmup, flush, world, split=None, on_timed_start=None):
    """Runs warmup + steps calls of fn(); returns per-step ms (device events) and, if fn records a
    mid-step event through `split`, the ms of the part after it."""
    for _ in range(warmup):
        flush(); fn(None)
    barrier(world)
    if on_timed_start is not None:
        on_timed_start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i in range(steps):
        flush()
        ev[i][0].record()
        fn(ev[i][1])
        ev[i][2].record()
    barrier(world)
    total = [e[0].elapsed_time(e[2]) for e in ev]
    tail = [e[1].elapsed_time(e[2]) for e in ev] if split else None
    return total, tail


# --------------------------------------------------------------------------------------------- #
def cpu_oracle_sample(wl, n_seq, kind):
    """Times the oracle, as it stands, on the first n_seq sequences of the workload (host cores)."""
    from oracle import paged_attention as orc
    g = wl.geom
    if kind == "extend":
        s = wl.ext
        lens = [s.prefix[i] + s.extend[i] for i in range(n_seq)]
    else:
        s = wl.dec
        lens = s.ctx[:n_seq]
    pages = sum(synth.pages_needed(L, g.page_size) for L in lens)
    host = orc.PagePool(pages, g.page_size, g.n_kv_heads, g.head_dim)
    rows, nxt = [], 0
    for i, L in enumerate(lens):
        n = synth.pages_needed(L, g.page_size)
        rows.append(list(range(nxt, nxt + n))); nxt += n
        kb, vb = wl.source_kv("ext" if kind == "extend" else "dec", i)   # from the input generator, not the pool
        host.append(rows[-1], 0, kb, vb)
    bt = synth.block_table(rows)
    if kind == "extend":
        E = s.extend[:n_seq]
        cu = np.concatenate([[0], np.cumsum(E)]).astype(np.int32)
        qb = synth.bf16_bits(s.q[:int(cu[-1])])
        t0 = time.perf_counter()
        o, lse = orc.attn_extend(host, qb, g.n_q_heads, cu, bt, s.prefix[:n_seq], E, g.scale)
        dt = time.perf_counter() - t0
        pairs = sum(e * p + e * (e + 1) // 2 for p, e in zip(s.prefix[:n_seq], E))
        work = 4.0 * g.head_dim * g.n_q_heads * pairs
        got_o = s.out[:int(cu[-1])].float().cpu().numpy()
        got_l = s.lse[:int(cu[-1])].cpu().numpy()
    else:
        qb = synth.bf16_bits(s.q[:n_seq])
        t0 = time.perf_counter()
        o, lse = orc.attn_decode(host, qb, g.n_q_heads, bt, lens, g.scale)
        dt = time.perf_counter() - t0
        work = float(sum(lens) * g.kv_bytes_per_token)
        got_o = s.out[:n_seq].float().cpu().numpy()
        got_l = s.lse[:n_seq].cpu().numpy()
    err_o = float(np.max(np.abs(got_o - o)))
    err_l = float(np.max(np.abs(got_l - lse)))
    return dt, work, err_o, err_l


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_ours(args):
    world, rank, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    torch.cuda.set_device(dev)
    from paper_2607_23815_b200 import kvattn
    from paper_2607_23815_b200.workload import DeviceWorkload
    kvattn.lib()                                                   # fail loudly if the library is missing
    peaks = load_peaks()
    flush = L2Flusher(dev)
    w = synth.WORKLOADS[args.workload]
    g = w.geom
    wl = DeviceWorkload(w, dev, seed_offset=rank, write_suffix=True)

    # ---- headline: suffix append + extend attention, one call ---------------------------------
    def step(_):
        wl.extend_append()

    box = {}
    if rank == 0:
        # the clocks are sampled from before the warm-up to the end of the end-to-end measurement: the timed region
        # of the headline step alone lasts a few milliseconds, too short for more than a handful of samples
        box["sampler"] = ClockSampler(dev.index or 0)

    # ---- the dominant kernel on its own, BEFORE the long step loop: one launch of the attention kernel over the pages
    # as a step leaves them, through attn_extend_planned (the work list is built once, outside the timed region, as for
    # the layers after the first).  At most 30 launches, and in front of the step loop rather than behind it: the
    # denominator is the burst figure of the matmul peak, i.e. of a kernel timed alone on a GPU that has not been at
    # its power cap for tens of milliseconds; back-to-back launches of this kernel behind a 100-step loop settle 3 %
    # lower, like the sustained matmul figure does (inside a step, where the prologue kernel gives the tensor cores a
    # pause, the kernel takes step minus prologue = the time measured here).
    wl.extend_plan()
    kernel_steps = min(args.steps, 30)
    ker_ms, _ = time_steps(lambda _: wl.extend_planned(), kernel_steps, args.warmup, flush, world)
    ext_kernel_ms = statistics.mean(ker_ms)

    def timed_start():
        box["l0"] = kvattn.kvattn_launch_count()

    total_ms, _ = time_steps(step, args.steps, args.warmup, flush, world, on_timed_start=timed_start)
    launches = kvattn.kvattn_launch_count() - box["l0"]
    ms_step = max_over_ranks(statistics.mean(total_ms), world)
    flops = wl.ext.flops(g)
    all_flops = sum_over_ranks(flops, world)
    value = all_flops / (ms_step * 1e-3) / 1e12
    ext_tflops = flops / (ext_kernel_ms * 1e-3) / 1e12
    side_steps = min(args.steps, 20)   # the two comparison figures need no long runs
    call_ms, _ = time_steps(lambda _: wl.extend(), side_steps, args.warmup, flush, world)   # attn_extend: plan + kernel
    # the same step as two calls (kv_append, then attn_extend), for comparison
    two_ms, _ = time_steps(lambda _: (wl.append_suffix(), wl.extend()), min(args.steps, 20), args.warmup, flush, world)

    # ---- e2e: host buffers, copies inside the timed region ---------------------------------
    e = wl.ext
    host_in = [t.cpu().pin_memory() for t in (e.q, e.k_new, e.v_new, e.cu_q, e.block_tables, e.prefix_lens, e.extend_lens)]
    host_out = [torch.empty_like(e.out, device="cpu").pin_memory(), torch.empty_like(e.lse, device="cpu").pin_memory()]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    stage_bytes = kvattn.attn_extend_host_staging_bytes(wl.pool, g.n_q_heads, len(e.prefix), e.total_q,
                                                        int(e.block_tables.shape[1]), e.max_total)
    staging = [torch.empty(stage_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]

    def host_call(b, stream=None):
        # the library's one-call step: host buffers in, host buffers out (copies, kv_append, attn_extend inside)
        kvattn.attn_extend_host(wl.pool, host_in[0], host_in[1], host_in[2], host_in[3], host_in[4], host_in[5],
                                host_in[6], e.max_extend, e.max_total, g.scale, outs[b][0], outs[b][1], staging[b], stream)

    outs = [host_out, [torch.empty_like(t).pin_memory() for t in host_out]]

    def e2e_step(_):
        host_call(0)

    e2e_ms, _ = time_steps(e2e_step, max(3, args.steps // 2), 3, flush, world)
    e2e_serial_ms = max_over_ranks(statistics.mean(e2e_ms), world)

    # The same call the way a caller with host buffers would drive it: two staging areas in turn, so that one step's
    # copies (which the library runs on copy streams of its own) overlap its neighbour's kernels.  Every step still
    # moves all of its inputs in and its results out inside the timed region; the figure is the time of K such
    # steps divided by K.  (Both staging areas append the same suffix rows to the same pages: same bits, no conflict.)
    def piped(n_steps):
        for i in range(n_steps):
            flush()
            host_call(i & 1)

    n_e2e = max(6, args.steps // 2)
    piped(4)
    torch.cuda.synchronize()
    barrier(world)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    piped(n_e2e)
    t1.record()
    torch.cuda.synchronize()
    barrier(world)
    e2e_step_ms = max_over_ranks(t0.elapsed_time(t1) / n_e2e, world)
    e2e_value = all_flops / (e2e_step_ms * 1e-3) / 1e12
    clocks = box["sampler"].stop() if "sampler" in box else None
    if clocks is not None:
        clocks["window"] = "warm-up, timed steps, kernel-only steps and end-to-end steps of the headline workload"
    same = torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][0], e.out.cpu())
    if not same:
        raise RuntimeError("end-to-end steps: the two buffer sets disagree")

    line = {
        "metric": METRIC, "value": round(value, 3), "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: {w.n_extend} tuples, Hq={g.n_q_heads} Hkv={g.n_kv_heads} D={g.head_dim} "
                               f"page=16, prefix U{list(w.prefix_range)}, extend U{list(w.extend_range)}, "
                               f"{w.num_pages}-page pool, random placement",
                   "step": "attn_extend_append = kv_append(suffix) + attn_extend in one call", "l2": "flushed between steps (256 MiB memset, untimed)",
                   "multi_gpu": "replicas only (no exchange step)"},
        "e2e": {"value": round(e2e_value, 3), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_step_ms, 5), "how": "attn_extend_host with two staging areas in turn (a step's copies overlap its neighbour's kernels)",
                "one_step_at_a_time_ms": round(e2e_serial_ms, 5)},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "attn_extend_tc_kernel (attn_extend_planned)", "achieved": round(ext_tflops, 3),
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": round(ext_tflops / peaks["bf16_tflops"], 4),
                     "peak_source": f"{peaks['source']} (burst bf16 matmul)", "frac_of_nominal_2250": round(ext_tflops / 2250.0, 4),
                     "kernel_ms": round(ext_kernel_ms, 5), "kernel_launches_timed": kernel_steps,
                     "kernel_loop": "attn_extend_planned alone, timed in front of the step loop", "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                     "target_frac_of_dense_bf16_peak": 0.60,
                     "target_met_vs_measured_peak": bool(ext_tflops / peaks["bf16_tflops"] >= 0.60),
                     "target_met_vs_nominal_2250": bool(ext_tflops / 2250.0 >= 0.60)},
        "attn_extend_call_ms": round(statistics.mean(call_ms), 5),
        "step_as_two_calls_ms": round(max_over_ranks(statistics.mean(two_ms), world), 5),
        "clocks": clocks,
    }

    if rank == 0 and world == 1:
        if not args.no_cpu:
            # ---- CPU oracle on a bounded sample of the same workload -----------------------
            n_s = min(args.cpu_sample, len(e.prefix))
            dt, work, err_o, err_l = cpu_oracle_sample(wl, n_s, "extend")
            line["cpu_baseline"] = {"value": round(work / dt / 1e12, 6), "unit": "TFLOP/s", "cores": blas_threads(),
                                    "kind": "oracle", "sample": f"first {n_s} of {len(e.prefix)} tuples, {dt:.1f} s",
                                    "max_abs_err_o_vs_gpu": err_o, "max_abs_err_lse_vs_gpu": err_l}
        wl.close(); del wl
        torch.cuda.empty_cache()
        line.update(extra_measurements(args, dev, peaks, flush))
    else:
        wl.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def extra_measurements(args, dev, peaks, flush):
    """Decode (HBM-bound), bulk append and the mixed pipeline step, each on its own workload."""
    from paper_2607_23815_b200 import kvattn
    from paper_2607_23815_b200.workload import DeviceWorkload
    out = {}
    sections = set(x for x in args.sections.split(",") if x and x != "none")
    steps, warm = max(5, args.steps), 3
    if "reuse" in sections:
        out.update(reuse_vs_recompute(args, dev, peaks, flush))
    if "fanout" in sections:
        out.update(fanout_measurement(args, dev, peaks, flush))
    if not sections & {"decode", "append"}:
        if "mixed" in sections:
            out.update(mixed_measurement(args, dev, flush, steps, warm))
        return out
    # decode
    w = synth.WORKLOADS["decode_8b"]
    wl = DeviceWorkload(w, dev)
    ms, _ = time_steps(lambda _: wl.decode(), steps, warm, flush, 1)
    t = statistics.mean(ms)
    gbs = wl.dec.kv_bytes(w.geom) / (t * 1e-3) / 1e9
    if args.no_cpu:
        dt, work, err_o, err_l = float("nan"), float("nan"), None, None
    else:
        dt, work, err_o, err_l = cpu_oracle_sample(wl, min(128, len(wl.dec.ctx)), "decode")
    out["decode"] = {"workload": f"{w.name}: {w.n_decode} seqs, ctx U{list(w.ctx_range)}, {w.num_pages}-page pool",
                     "value": round(gbs, 1), "unit": "GB/s", "ms_per_step": round(t, 5), "min_ms": round(min(ms), 5),
                     "roofline": {"bound": "hbm", "kernel": "attn_decode", "achieved": round(gbs, 1),
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
                                  "peak_source": f"{peaks['source']} (copy)", "frac_of_nominal_8000": round(gbs / 8000.0, 4),
                                  "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
                     "cpu_baseline": None if args.no_cpu else {
                         "value": round(work / dt / 1e9, 4), "unit": "GB/s", "cores": blas_threads(), "kind": "oracle",
                         "sample": f"first {min(128, w.n_decode)} of {w.n_decode} sequences, {dt:.1f} s",
                         "max_abs_err_o_vs_gpu": err_o, "max_abs_err_lse_vs_gpu": err_l}}
    # bulk append: re-write every decode sequence's K/V (read + write bytes)
    d = wl.dec
    n_tok = sum(d.ctx)
    if "append" in sections and n_tok * w.geom.kv_bytes_per_token < 6 << 30:
        k_all = torch.empty((n_tok, w.geom.n_kv_heads, w.geom.head_dim), dtype=torch.bfloat16, device=dev).normal_()
        v_all = torch.empty_like(k_all).normal_()
        cu = torch.tensor(np.concatenate([[0], np.cumsum(d.ctx)]), dtype=torch.int32, device=dev)
        zero = torch.zeros(len(d.ctx), dtype=torch.int32, device=dev)
        ms, _ = time_steps(lambda _: kvattn.kv_append(wl.pool, k_all, v_all, cu, zero, None, d.block_tables),
                           steps, warm, flush, 1)
        t = statistics.mean(ms)
        moved = 2.0 * n_tok * w.geom.kv_bytes_per_token
        cpu = None
        if not args.no_cpu:
            from oracle import paged_attention as orc
            n_s = 4
            kv_src = [wl.source_kv("dec", i) for i in range(n_s)]
            host = orc.PagePool(sum(synth.pages_needed(c, 16) for c in d.ctx[:n_s]), 16, w.geom.n_kv_heads, w.geom.head_dim)
            t0 = time.perf_counter()
            nxt = 0
            for i in range(n_s):
                n = synth.pages_needed(d.ctx[i], 16)
                host.append(list(range(nxt, nxt + n)), 0, kv_src[i][0], kv_src[i][1]); nxt += n
            dt = time.perf_counter() - t0
            cpu = {"value": round(2.0 * sum(d.ctx[:n_s]) * w.geom.kv_bytes_per_token / dt / 1e9, 4), "unit": "GB/s (read+write)",
                   "cores": 1, "kind": "oracle", "sample": f"append of the first {n_s} sequences ({sum(d.ctx[:n_s])} tokens) "
                   f"into the oracle's host page image, {dt:.2f} s"}
        out["append"] = {"cpu_baseline": cpu, "workload": f"bulk append of {n_tok} tokens ({moved / 2e9:.2f} GB of K/V)",
                         "value": round(moved / (t * 1e-3) / 1e9, 1), "unit": "GB/s (read+write)",
                         "ms_per_step": round(t, 5),
                         "frac_of_measured_copy": round(moved / (t * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}
        del k_all, v_all
    wl.close(); del wl
    torch.cuda.empty_cache()
    if "mixed" in sections:
        out.update(mixed_measurement(args, dev, flush, steps, warm))
    return out


def reuse_vs_recompute(args, dev, peaks, flush):
    """Long-document reuse (70B shape): extend over the reused prefix pages against the from-scratch prefill of
    prefix+suffix that a cache miss costs (the kernel-level face of the paper's pipelined-vs-blocking gap)."""
    from paper_2607_23815_b200 import kvattn
    from paper_2607_23815_b200.workload import DeviceWorkload
    w = synth.WORKLOADS["long_doc_70b"]
    g = w.geom
    wl = DeviceWorkload(w, dev)
    e = wl.ext
    ms_reuse, _ = time_steps(lambda _: wl.extend(), 5, 3, flush, 1)
    t_reuse = statistics.mean(ms_reuse)
    # the same sequences from scratch: prefix 0, every token is a query (K/V are already in the pages)
    L = [p + x for p, x in zip(e.prefix, e.extend)]
    q_full = torch.cat([synth.normal_bf16(wl.seed, synth.TAG_Q, e.uids[i], 0, L[i], g.n_q_heads, g.head_dim, dev)
                        for i in range(len(L))])
    out_full = torch.empty_like(q_full)
    lse_full = torch.empty((q_full.shape[0], g.n_q_heads), dtype=torch.float32, device=dev)
    i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
    cu, zero, lens = i32(np.concatenate([[0], np.cumsum(L)]).tolist()), i32([0] * len(L)), i32(L)
    ws = torch.empty(kvattn.attn_workspace_bytes(wl.pool, g.n_q_heads, len(L), int(q_full.shape[0]), max(L), 0, 0),
                     dtype=torch.uint8, device=dev)
    fn = lambda _: kvattn.attn_extend(wl.pool, q_full, cu, e.block_tables, zero, lens, max(L), max(L), g.scale,
                                      out_full, lse_full, ws)
    ms_full, _ = time_steps(fn, 3, 1, flush, 1)
    t_full = statistics.mean(ms_full)
    # the last E rows of the recompute are the reuse run's rows: the invariant the paper relies on
    r0, f0 = int(e.cu_q[1].item()), int(cu[1].item())
    d_o = (out_full[f0 - e.extend[0]:f0].float() - e.out[:r0].float()).abs().max().item()
    cpu = None
    if not args.no_cpu:
        dt, work, err_o, err_l = cpu_oracle_sample(wl, 2, "extend")
        cpu = {"value": round(work / dt / 1e12, 6), "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle",
               "sample": f"first 2 of {len(L)} tuples of the reuse run, all rows and heads, {dt:.1f} s",
               "max_abs_err_o_vs_gpu": err_o, "max_abs_err_lse_vs_gpu": err_l}
    flops_reuse = e.flops(g)
    flops_full = 4.0 * g.head_dim * g.n_q_heads * sum(l * (l + 1) // 2 for l in L)
    res = {"reuse_vs_recompute": {
        "workload": f"{w.name}: {w.n_extend} tuples, Hq={g.n_q_heads} Hkv={g.n_kv_heads}, prefix U{list(w.prefix_range)}, "
                    f"extend U{list(w.extend_range)}",
        "reuse_ms": round(t_reuse, 4), "reuse_tflops": round(flops_reuse / t_reuse / 1e9, 1),
        "reuse_frac_of_measured_peak": round(flops_reuse / t_reuse / 1e9 / peaks["bf16_tflops"], 4),
        "recompute_ms": round(t_full, 3), "recompute_tflops": round(flops_full / t_full / 1e9, 1),
        "recompute_frac_of_measured_peak": round(flops_full / t_full / 1e9 / peaks["bf16_tflops"], 4),
        "time_ratio": round(t_full / t_reuse, 2), "flop_ratio": round(flops_full / flops_reuse, 2),
        "max_abs_diff_last_rows_tuple0": d_o, "cpu_baseline": cpu}}
    del q_full, out_full, lse_full, ws
    wl.close(); del wl
    torch.cuda.empty_cache()
    return res


def fanout_measurement(args, dev, peaks, flush):
    """Children over a shared parent prefix (32 parents x 17 children, prefix ~2144, suffix ~37): one call that reads
    the shared pages once per parent against the same children run as independent sequences on aliased block tables."""
    from paper_2607_23815_b200.workload import FanoutWorkload
    fw = FanoutWorkload(synth.Geometry(32, 8, 128), device=dev)
    from paper_2607_23815_b200 import kvattn
    ms_ind, _ = time_steps(lambda _: fw.independent(), 10, 3, flush, 1)
    kvattn.kvattn_set_shared_impl(1)   # shared part, own part, merge: three kernels
    ms_split, _ = time_steps(lambda _: fw.shared(), 10, 3, flush, 1)
    kvattn.kvattn_set_shared_impl(0)   # the default picks the one-kernel walk for this suffix length
    ms_sh, _ = time_steps(lambda _: fw.shared(), 10, 3, flush, 1)
    t_ind, t_sh, t_split = statistics.mean(ms_ind), statistics.mean(ms_sh), statistics.mean(ms_split)
    d_o = (fw.out.float() - fw.out2.float()).abs().max().item()
    d_l = (fw.lse - fw.lse2).abs().max().item()
    st = kvattn.kv_last_async_status(fw.pool)
    if st != kvattn.KV_OK:
        raise RuntimeError(f"fan-out section: device status {st} (a kernel reported an error)")
    fl = fw.flops()
    res = {"fanout": {
        "workload": f"{fw.n_parents} parents x {fw.n_children // fw.n_parents} children, Hq=32 Hkv=8 D=128, prefix "
                    f"{min(fw.parent_lens)}..{max(fw.parent_lens)}, suffix {min(fw.child_lens)}..{max(fw.child_lens)}",
        "independent_ms": round(t_ind, 4), "shared_ms": round(t_sh, 4), "speedup": round(t_ind / t_sh, 2),
        "shared_three_kernel_ms": round(t_split, 4),
        "independent_tflops": round(fl / t_ind / 1e9, 1), "shared_tflops": round(fl / t_sh / 1e9, 1),
        "shared_frac_of_measured_peak": round(fl / t_sh / 1e9 / peaks["bf16_tflops"], 4),
        "max_abs_diff_o": d_o, "max_abs_diff_lse": d_l}}
    fw.close()
    del fw
    torch.cuda.empty_cache()
    return res


def mixed_measurement(args, dev, flush, steps, warm):
    """One sem_map -> sem_filter pipeline step: extend set and decode set together; then the same configuration as a
    loop of steps with the per-step kv_append of the new tokens and page churn in between (churn not timed)."""
    from paper_2607_23815_b200.workload import DeviceWorkload, PipelineLoop
    peaks = load_peaks()
    out = {}
    w = synth.WORKLOADS["pipeline_step"]
    wl = DeviceWorkload(w, dev)
    ms_mixed, _ = time_steps(lambda _: wl.mixed(), steps, warm, flush, 1)
    ms_ext, _ = time_steps(lambda _: wl.extend(), steps, warm, flush, 1)
    ms_dec, _ = time_steps(lambda _: wl.decode(), steps, warm, flush, 1)
    t_mixed, t_ext, t_dec = statistics.mean(ms_mixed), statistics.mean(ms_ext), statistics.mean(ms_dec)
    # bounds: the two kinds of work perfectly overlapped (the slower of tensor time and HBM time at the measured
    # peaks), and the two calls one after the other
    hbm_ms = (wl.dec.kv_bytes(w.geom) + wl.ext.kv_bytes(w.geom)) / peaks["hbm_gbs"] / 1e6
    tensor_ms = wl.ext.flops(w.geom) / peaks["bf16_tflops"] / 1e9
    cpu = None
    if not args.no_cpu:
        dt_e, work_e, err_oe, err_le = cpu_oracle_sample(wl, 8, "extend")
        dt_d, work_d, err_od, err_ld = cpu_oracle_sample(wl, 32, "decode")
        est = dt_e * wl.ext.flops(w.geom) / work_e + dt_d * wl.dec.kv_bytes(w.geom) / work_d
        cpu = {"value": round(est * 1e3, 1), "unit": "ms per step (extrapolated from the sample by work)", "cores": blas_threads(),
               "kind": "oracle", "sample": f"first 8 of {w.n_extend} extend tuples ({dt_e:.1f} s) and first 32 of {w.n_decode} "
               f"decode sequences ({dt_d:.1f} s)", "max_abs_err_o_vs_gpu": max(err_oe, err_od),
               "max_abs_err_lse_vs_gpu": max(err_le, err_ld)}
    out["pipeline_step"] = {"workload": f"{w.name}: {w.n_extend} extend + {w.n_decode} decode sequences",
                            "mixed_ms": round(t_mixed, 5),
                            "extend_alone_ms": round(t_ext, 5),
                            "decode_alone_ms": round(t_dec, 5),
                            "bound_overlapped_ms": round(max(hbm_ms, tensor_ms), 5),
                            "bound_sum_of_calls_ms": round(t_ext + t_dec, 5),
                            "mixed_over_overlapped_bound": round(t_mixed / max(hbm_ms, tensor_ms), 3),
                            "extend_tflops_alone": round(wl.ext.flops(w.geom) / t_ext / 1e9, 2),
                            "decode_gbs_alone": round(wl.dec.kv_bytes(w.geom) / t_dec / 1e6, 1),
                            "cpu_baseline": cpu}
    wl.close(); del wl
    torch.cuda.empty_cache()
    # the loop: per step one kv_append of the new tokens + attn_mixed, timed together; 20 % page churn between steps
    n_steps = 8
    loop = PipelineLoop(w, dev, steps=n_steps)
    per_step, appended = [], []
    for _ in range(n_steps):
        loop.begin_step()
        ms, _ = time_steps(lambda _: (loop.append_new(), loop.mixed()), 5, 2, flush, 1)   # re-appending the same rows is idempotent
        per_step.append(statistics.mean(ms)); appended.append(loop.step_new_tokens())
        loop.commit_new()
        loop.churn(0.2)
        loop.end_step()
    loop.close()
    out["pipeline_step"]["loop"] = {"steps": n_steps, "step": "kv_append(new tokens) + attn_mixed", "churn": "20 % of the live pages "
                                    "evicted, re-allocated and re-filled between steps (untimed)",
                                    "median_step_ms": round(statistics.median(per_step), 5),
                                    "step_ms": [round(x, 4) for x in per_step], "new_tokens_per_step": appended}
    return out


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import paged_attention as orc
    w = synth.WORKLOADS[args.workload]
    g = w.geom
    ext, _ = synth.draw_lengths(w)
    # The sample shrinks with the number of steps asked for, so that the whole run stays near two minutes: a tuple
    # of this workload costs the oracle about 0.12 s on 8-16 host threads.
    per_step_budget_s = 150.0 / max(1, args.steps + args.warmup)
    n_s = max(1, min(args.cpu_sample, 16, len(ext), int(per_step_budget_s / 0.12)))
    P, E = [p for p, _ in ext[:n_s]], [e for _, e in ext[:n_s]]
    pages = sum(synth.pages_needed(p + e, g.page_size) for p, e in zip(P, E))
    host = orc.PagePool(pages, g.page_size, g.n_kv_heads, g.head_dim)
    perm = synth.page_permutation(w.seed, pages).tolist()
    rows, qs = [], []
    for i in range(n_s):
        L = P[i] + E[i]
        n = synth.pages_needed(L, g.page_size)
        rows.append(perm[:n]); perm = perm[n:]
        host.append(rows[-1], 0,
                    synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_K, i, 0, L, g.n_kv_heads, g.head_dim)),
                    synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_V, i, 0, L, g.n_kv_heads, g.head_dim)))
        qs.append(synth.bf16_bits(synth.normal_bf16(w.seed, synth.TAG_Q, i, P[i], E[i], g.n_q_heads, g.head_dim)))
    q = np.concatenate(qs)
    cu = np.concatenate([[0], np.cumsum(E)]).astype(np.int32)
    bt = synth.block_table(rows)
    flops = 4.0 * g.head_dim * g.n_q_heads * sum(e * p + e * (e + 1) // 2 for p, e in zip(P, E))
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        orc.attn_extend(host, q, g.n_q_heads, cu, bt, P, E, g.scale)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    t = statistics.mean(times)
    v = round(flops / t / 1e12, 6)
    sample = f"first {n_s} of {len(ext)} tuples per step (gather + attention, K/V already in host pages)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(t * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name} (sample)", "sample": sample},
        "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=[k for k, v in synth.WORKLOADS.items() if v.n_extend])
    ap.add_argument("--cpu-sample", type=int, default=64, help="tuples in the CPU-oracle sample")
    ap.add_argument("--sections", default="decode,append,mixed,reuse,fanout",
                    help="extra measurements after the headline: comma list of decode, append, mixed, reuse, fanout "
                         "(or 'none')")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle legs (for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
