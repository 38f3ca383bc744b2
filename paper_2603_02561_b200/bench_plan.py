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


def distinct_buffers(in_flight: int, l2_batches: int) -> int:
    """Input/output buffer sets to rotate over so that (a) a step's inputs are never L2-resident
    and (b) no two steps that can be in flight together touch the same buffers: lanes drift by
    up to one round against each other, so two rounds' worth of lanes plus the L2 margin."""
    return 2 * max(1, in_flight) + l2_batches


def buffer_of_step(round_index: int, lane: int, in_flight: int, n_buffers: int) -> int:
    """Buffer set used by `lane` in round `round_index` of a graph (rounds are dealt lane by lane)."""
    return (round_index * in_flight + lane) % n_buffers


def replay_plan(steps_wanted: int, in_flight: int, ms_per_step_estimate: float, min_seconds: float = 0.5,
                rounds_per_graph: int = 12, min_replays: int = 50, max_seconds: float = 3.0) -> tuple[int, int, int]:
    """(steps per graph, replays, steps actually timed).  A graph holds `rounds_per_graph` steps
    on each of the in-flight lanes (the join at its end is amortised over them).  The timed
    region honours `steps_wanted` as a minimum and lasts at least `min_seconds` and
    `min_replays` replays by the estimate from the warm-up, capped at `max_seconds`."""
    per_graph = rounds_per_graph * max(1, in_flight)
    est = max(ms_per_step_estimate, 1e-6) * 1e-3 * per_graph              # seconds per replay
    replays = max(min_replays, math.ceil(steps_wanted / per_graph), math.ceil(min_seconds / est))
    cap = max(math.ceil(steps_wanted / per_graph), math.ceil(max_seconds / est), 3)
    replays = max(1, min(replays, cap))
    return per_graph, replays, replays * per_graph


def spread(ms_per_replay, steps_per_replay: int) -> dict:
    """Median, minimum and maximum of the per-replay step times (ms per step)."""
    v = sorted(float(x) / steps_per_replay for x in ms_per_replay)
    n = len(v)
    med = v[n // 2] if n % 2 else 0.5 * (v[n // 2 - 1] + v[n // 2])
    return {"median": med, "min": v[0], "max": v[-1], "replays": n}


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
