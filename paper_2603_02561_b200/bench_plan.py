"""Host-side planning of the benchmark: which seeded batches a rank generates, how many
graph replays make up the timed region, and the max-over-ranks reduction of the timings.

Users are independent units of work, so N ranks run N independent replicas: each rank
draws its OWN batches (disjoint seed indices) and no data crosses between ranks; the only
collective is the reduction of the measured times after the timed region.  Nothing here
touches the method's arithmetic.
"""
from __future__ import annotations

import math


def rank_seed_indices(base_seed_index: int, rank: int, batches_per_rank: int) -> list[int]:
    """Seed indices of the batches of `rank`: disjoint across ranks, never the base index
    (which the parity tests use)."""
    return [base_seed_index + 1000 * (rank * batches_per_rank + i + 1) for i in range(batches_per_rank)]


def batches_to_exceed_l2(bytes_per_step: int, l2_bytes: int, factor: float = 1.5) -> int:
    """Distinct batches to rotate over so that a step's inputs are never L2-resident."""
    return max(2, math.ceil(factor * l2_bytes / bytes_per_step))


def replay_plan(steps_wanted: int, n_batches: int, in_flight: int) -> tuple[int, int, int]:
    """(steps per graph, replays, steps actually timed).  A graph deals its steps round-robin
    to the in-flight lanes; with several lanes it holds four passes over the batches so the
    join at the end of a graph is amortised."""
    per_graph = 4 * n_batches * in_flight if in_flight > 1 else n_batches
    replays = max(1, math.ceil(steps_wanted / per_graph))
    return per_graph, replays, replays * per_graph


def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum over ranks of a list of floats (the job is as slow as its slowest
    rank).  `dist` is torch.distributed (initialised) or None for a single process."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_throughput(pairs_per_step_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job candidates x positions per second: every rank processed its own step in the
    (max-over-ranks) step time."""
    return world * pairs_per_step_per_rank / (ms_per_step * 1e-3)
