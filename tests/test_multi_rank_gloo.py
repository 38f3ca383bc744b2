"""The N > 1 path of the benchmark on CPU: two gloo ranks plan their batches, time a stand-in
step and reduce the timings.  The GPU work itself does not shard (users are independent
replicas), so what needs covering is the host logic: disjoint seeds per rank, identical
replay plans, max-over-ranks timing, whole-job aggregation."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_02561_b200 import bench_plan as bp
from paper_2603_02561_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.CONFIGS["c2"].with_(B=2, N=64, M=8)
    seeds = bp.rank_seed_indices(w.seed_index, rank, 3)
    # the batches themselves: first user's history of every batch, hashed
    sig = [float(np.abs(wl.history(w.with_(seed_index=s), 0)).sum()) for s in seeds]
    plan = bp.replay_plan(100, 4, 0.02)
    ms = 10.0 + 5.0 * rank                         # rank 1 is the slow one
    reduced = bp.max_over_ranks([ms, 1.0 + rank, 7.0], dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, {"seeds": seeds, "sig": sig, "plan": plan, "reduced": reduced})
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_plan_disjoint_batches_and_reduce_times():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    a, b = res
    assert not set(a["seeds"]) & set(b["seeds"])                  # no batch is shared
    assert wl.CONFIGS["c2"].seed_index not in a["seeds"] + b["seeds"]
    assert not set(a["sig"]) & set(b["sig"])                      # and the data differ
    assert a["plan"] == b["plan"] == (48, 521, 521 * 48)     # 0.5 s at 20 us per step
    assert a["reduced"] == b["reduced"] == [15.0, 2.0, 7.0]        # max over ranks, on both
    assert bp.aggregate_throughput(1000, world, 2.0) == 2 * 1000 / 2e-3


def test_single_process_helpers():
    assert bp.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bp.replay_plan(10, 1, 0.1) == (12, 417, 417 * 12)         # at least half a second
    assert bp.replay_plan(10 ** 6, 24, 0.01)[2] >= 10 ** 6           # the steps asked for are a minimum
    assert bp.replay_plan(10, 24, 50.0) == (288, 3, 864)             # long steps: capped, at least three replays
    nbuf = bp.distinct_buffers(24, 7)
    assert nbuf == 55
    # steps that can run together (same round, or neighbouring rounds of different lanes) never share a buffer
    for rnd in range(6):
        now = [bp.buffer_of_step(rnd, l, 24, nbuf) for l in range(24)]
        nxt = [bp.buffer_of_step(rnd + 1, l, 24, nbuf) for l in range(24)]
        assert len(set(now + nxt)) == 48
    sp = bp.spread([2.0, 4.0, 3.0], 2)
    assert sp == {"median": 1.5, "min": 1.0, "max": 2.0, "replays": 3}
    assert bp.batches_to_exceed_l2(29650944, 126 * 2 ** 20) == 7
    assert bp.rank_seed_indices(3, 0, 2) == [1003, 2003] and bp.rank_seed_indices(3, 1, 2) == [3003, 4003]
