"""The benchmark's multi-rank plumbing (replicas only: barrier, max-over-ranks time, summed work) on CPU with
two gloo ranks.  The data path itself has no collective, so this is all there is to the N > 1 case."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2607_23815_b200 import ranks, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank owns a replica of the workload with its own seed: different lengths, same shapes
        w = synth.WORKLOADS["tiny"]
        ext, _ = synth.draw_lengths(synth.scaled(w, seed=ranks.replica_seed(w.seed, rank)))
        work = float(sum(p * e for p, e in ext))
        ms = 10.0 + 5.0 * rank                                   # pretend rank 1 is slower
        agg = ranks.aggregate(ms, work, world, device="cpu")
        out[rank] = (agg, ext)
    finally:
        dist.destroy_process_group()


def test_two_ranks_aggregate_max_time_and_summed_work():
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    (agg0, ext0), (agg1, ext1) = out[0], out[1]
    assert ext0 != ext1                                          # replicas differ by seed
    assert agg0 == agg1                                          # every rank sees the same aggregate
    ms_max, total_work = agg0
    assert ms_max == 15.0
    assert total_work == float(sum(p * e for p, e in ext0) + sum(p * e for p, e in ext1))


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2607_23815_b200 import ranks
    assert ranks.aggregate(3.5, 7.0, 1, device="cpu") == (3.5, 7.0)
    assert ranks.replica_seed(100, 0) == 100 and ranks.replica_seed(100, 3) != 100
