#!/usr/bin/env python
"""Benchmark of the SVD-Attention forward pass (solar_lowrank_factor + solar_svd_attention_fwd).

One "step" = one pass of the whole hot path over one batch of B users: streaming Gram of
H, eigensolve, factor-token projections, candidate attention.  Metric: candidates x
sequence positions per second = B*M*N / step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--in-flight S]
                    [--path fused|two_call] [--impl ours|reference]

The timed region replays CUDA graphs of whole steps (no host work between kernels).  With
--in-flight S > 1, S independent batches are in flight on S streams (each with its own
workspace and factors), which is how a serving process overlaps one request's eigensolve
(B CTAs) with another's streaming passes; S = 1 gives the single-call latency.  Both
figures are printed; `value` is the one at the S given (default 30: the step time falls up
to 31 streams and jumps by a fifth at 32, where streams start to share a hardware queue).  Every step in flight
reads and writes buffers of its own (2 S + 7 buffer sets), --steps is a minimum, and the
timed region lasts at least half a second; the spread over the graph replays is printed.
The steps in flight run under solar_set_slice_limit(--slice-limit, default 2: few long slices
per user, the setting for throughput); `single_call` is taken under the library's default
slicing (the setting for latency), the other combination of each is printed beside it.
`value` is measured through solar_svd_attention_fused (three launches per step); the same
measurement through solar_lowrank_factor + solar_svd_attention_fwd (four launches) is
printed beside it as `two_call`.

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own batches of B
users (users are independent: no data-path collective), timing is max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_02561_b200 import bench_plan as bp  # noqa: E402
from paper_2603_02561_b200 import workloads as wl  # noqa: E402

L2_BYTES = 126 * 2 ** 20
KERNELS_PER_STEP = {"fused": 3, "two_call": 4}   # gram, eigensolve (+ projections), [projections,] attention
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # 148 SMs x 128 FMA lanes x 2 flop at 1965 MHz
SFU_TEXPS = 148 * 16 * 1.965e9 / 1e12              # 148 SMs x 16 special-function lanes at 1965 MHz
def measured_traffic(workload: str, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture recorded in
    the traffic file -- or None when there is no capture for this workload and kernel, or the
    kernel's source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        rec = json.load(open(path)).get(f"{workload}/{kernel}")
        if rec is None:
            return None
        src = os.path.join(ROOT, rec["source"])
        if hashlib.sha1(open(src, "rb").read()).hexdigest()[:16] != rec["source_sha1"]:
            return None
        return rec["dram_bytes_per_launch"]
    except Exception:
        return None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def algorithmic_bytes(w: wl.Workload) -> dict:
    es = 2 if w.dtype == "bf16" else 4
    gram = w.B * w.N * w.d * es                      # H read once
    attn = 2 * w.B * w.M * w.d * es                  # C read, O written
    small = 3 * es * w.d * w.d + 8 * w.B * (w.r + w.d * w.r)
    return {"gram": gram, "attn": attn, "total": gram + attn + small}


def algorithmic_flops(w: wl.Workload) -> int:
    return (2 * w.B * w.N * w.d * w.d + 2 * w.B * w.M * w.d * w.d + 4 * w.B * w.M * w.d * w.r
            + 4 * w.B * w.r * w.d * w.d)


# ---------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)),
                   "reasons": sorted(reasons), "samples": len(sm)}
        return out


# ---------------------------------------------------------------------------------------
def oracle_step(w: wl.Workload, users):
    """The CPU oracle (as it stands) on the listed users of the workload; returns seconds."""
    import oracle as o
    Wq, Wk, Wv = wl.weights(w)
    inputs = [(wl.history(w, b).astype(np.float64), wl.candidates(w, b).astype(np.float64))
              for b in users]
    t0 = time.perf_counter()
    for H, C in inputs:
        o.svd_attention(H, C, Wq, Wk, Wv, w.r, w.scale)
    return time.perf_counter() - t0


def cpu_threads() -> int:
    """Threads of the BLAS pool numpy's matrix products run on (the oracle's Jacobi loop itself
    is Python-level and serial)."""
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_step_single_thread(w: wl.Workload, users):
    """The same with every BLAS pool limited to one thread: the condition of the paper's own
    latency experiment (Section 5.2: CPU, a single thread)."""
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        return None
    with threadpool_limits(limits=1):
        return oracle_step(w, users)


def run_reference(args, w: wl.Workload):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # a bounded sample per step: fewer users per step when many steps are asked for, so that the
    # whole run stays within a few minutes of host time
    per_step = args.ref_users if args.steps <= 8 else 1
    sample_users = list(range(min(w.B, per_step)))
    for _ in range(min(args.warmup, 1)):
        oracle_step(w, sample_users[:1])
    ts = [oracle_step(w, sample_users) for _ in range(args.steps)]
    t = float(np.mean(ts))
    pairs = len(sample_users) * w.M * w.N
    value = pairs / t
    line = {
        "impl": "reference", "metric": "svd_attention_fwd_candidates_x_positions_per_sec",
        "value": value, "unit": "pairs/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3 * w.B / len(sample_users),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "d": w.d, "r": w.r, "M": w.M,
                   "storage": w.dtype},
        "cpu_baseline": {"value": value, "unit": "pairs/s", "cores": cpu_threads(), "kind": "oracle",
                         "sample": f"{len(sample_users)} of {w.B} users per step, all {w.M} candidates; "
                                   "ms_per_step is scaled to the full batch"},
        "e2e": {"value": value, "unit": "pairs/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
def eig_flops(w: wl.Workload, route: int, detail: float, sweeps: float) -> float:
    """Useful floating-point operations of the eigensolver for one batch, counted from loop
    bounds.  Route 3 (tridiagonal): reduction 4/3 d^3, back-transformation 2 d^2 r, each
    orthogonalisation pass 4 d r^2, residuals 2 d^2 r, multisection 3 d r per point and step
    (26 bits), twisted factorisation ~20 d r.  Route 1 / 2 (range finder, Jacobi): dense
    products 2mnk, a 2x2 Jacobi block update 24 flop for the matrix and 12 for the vectors."""
    d, r = w.d, w.r
    if route == 3:
        passes = sweeps
        return w.B * (4.0 * d ** 3 / 3 + 4.0 * d * d * r + (passes + 1) * 2.0 * d * r * r + passes * 2.0 * d * r * r
                      + 3.0 * d * r * 4 * 12 + 20.0 * d * r)
    if route == 2:
        return w.B * sweeps * (d - 1) * (d * d / 4) * 36.0
    p = (r + 7) // 8 * 8
    iters = detail
    power = (iters + 1) * 2 * d * d * p + iters * (2 * d * p * p + p ** 3 / 3 + 2 * d * p * p) + 2 * d * p * p
    jac = sweeps * (p - 1) * (p * p / 4) * 36.0
    return w.B * (power + jac + 4 * d * p * p)


class Lane:
    """One in-flight slot: a stream with its own workspace and factor buffers."""

    def __init__(self, torch, solar, w, tdt):
        self.stream = torch.cuda.Stream()
        self.S = torch.empty(w.B, w.r, device="cuda")
        self.V = torch.empty(w.B, w.d, w.r, device="cuda")
        self.ws = solar.alloc_fused_workspace(w.B, w.M, w.N, w.d, w.r, tdt)   # covers the two-call sizes too


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--slice-limit", type=int, default=2,
                    help="solar_set_slice_limit for the steps in flight (0 = the library's own slicing, chosen for the "
                         "latency of one call); the single-call figure is always taken with 0")
    ap.add_argument("--rounds", type=int, default=24,
                    help="consecutive steps of a lane in one CUDA graph (the lanes drain and refill between replays)")
    ap.add_argument("--in-flight", type=int, default=30, help="independent batches in flight (streams)")
    ap.add_argument("--path", default="fused", choices=["fused", "two_call"],
                    help="which public call `value` is measured through (the other is printed beside it)")
    ap.add_argument("--cpu-users", type=int, default=8, help="users in the cpu_baseline sample")
    ap.add_argument("--ref-users", type=int, default=2, help="users per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--light", action="store_true",
                    help="the forward path only (no backward / factored-exact sections, short timed region): "
                         "what the profiler captures are taken on")
    ap.add_argument("--sweep", action="store_true",
                    help="the c5 sweep: one JSON line per (N, r) point, with a brute-force softmax "
                         "attention time on the host beside it")
    ap.add_argument("--sweep-lengths", default="2048,4096,8192,16384,32768")
    ap.add_argument("--sweep-ranks", default="8,16,32,64")
    args = ap.parse_args()
    w = wl.lookup(args.workload)

    if args.impl == "reference":
        if args.steps == 2000:
            args.steps = 3
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2603_02561_b200 import build as solar_build
    from paper_2603_02561_b200 import solar

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        solar_build.build()
    if world > 1:
        dist.barrier()
    solar.lib()

    if args.sweep:
        lengths = [int(x) for x in args.sweep_lengths.split(",")]
        ranks = [int(x) for x in args.sweep_ranks.split(",")]
        args.no_cpu_baseline = True
        for wp in wl.sweep_configs(lengths=lengths, ranks=ranks):
            line = measure(args, wp, torch, dist, solar, world, rank, local, light=True)
            if rank == 0:
                line["brute_force_cpu"] = brute_force_point(wp)
                print(json.dumps(line), flush=True)
            torch.cuda.empty_cache()
    else:
        line = measure(args, w, torch, dist, solar, world, rank, local, light=args.light)
        if rank == 0:
            print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def brute_force_point(w: wl.Workload) -> dict:
    """Brute-force softmax attention over the N positions (Eq. 6-7, O(N M d)) of ONE user of
    the point on the host cores, as candidates x positions per second."""
    import oracle as o
    Wq, Wk, Wv = wl.weights(w)
    H = wl.history(w, 0).astype(np.float64)
    C = wl.candidates(w, 0).astype(np.float64)
    t0 = time.perf_counter()
    o.softmax_attention(H, C, Wq, Wk, Wv, w.scale)
    t = time.perf_counter() - t0
    return {"value": w.M * w.N / t, "unit": "pairs/s", "seconds": t, "cores": cpu_threads(),
            "sample": f"1 of {w.B} users, all {w.M} candidates", "kind": "oracle softmax_attention"}


def measure(args, w, torch, dist, solar, world, rank, local, light=False):
    """Times workload w on this rank's GPU; returns the JSON line (rank 0) or None."""
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    ab = algorithmic_bytes(w)
    # Distinct data: enough seeded batches that a step's inputs are never L2-resident.  Distinct
    # BUFFERS: every step that can be in flight together with another reads and writes buffers of
    # its own (2 x lanes + the L2 margin); buffers beyond the seeded batches hold device copies
    # of them with the users rotated, which is all the DRAM traffic cares about.
    n_lanes = max(1, args.in_flight)
    nseed = bp.batches_to_exceed_l2(ab["total"], L2_BYTES)
    nb = bp.distinct_buffers(n_lanes, nseed)
    batches = [wl.generate(w.with_(seed_index=si)) for si in bp.rank_seed_indices(w.seed_index, rank, nseed)]
    Wq, Wk, Wv = (torch.from_numpy(batches[0][k]).cuda().to(tdt) for k in ("Wq", "Wk", "Wv"))
    dH = [torch.from_numpy(b["H"]).cuda().to(tdt) for b in batches]
    dC = [torch.from_numpy(b["C"]).cuda().to(tdt) for b in batches]
    for k in range(nseed, nb):
        dH.append(torch.roll(dH[k % nseed], 1 + k // nseed, 0).contiguous())
        dC.append(torch.roll(dC[k % nseed], 1 + k // nseed, 0).contiguous())
    dO = [torch.empty_like(c) for c in dC]
    main_stream = torch.cuda.Stream()
    lanes = [Lane(torch, solar, w, tdt) for _ in range(n_lanes)]

    def step(k, lane, stream, path=None):
        if (path or args.path) == "fused":
            solar.svd_attention_fused(dH[k], dC[k], Wq, Wk, Wv, w.r, w.scale, 0, S=lane.S, V=lane.V, O=dO[k],
                                      workspace=lane.ws, stream=stream)
        else:
            solar.lowrank_factor(dH[k], w.r, S=lane.S, V=lane.V, workspace=lane.ws, M=w.M, stream=stream)
            solar.svd_attention_fwd(dC[k], lane.S, lane.V, Wq, Wk, Wv, w.scale, 0, O=dO[k], workspace=lane.ws,
                                    N=w.N, stream=stream)

    def capture(rounds, use_lanes, path=None):
        """A CUDA graph of `rounds` whole steps on each of the lanes' streams."""
        L = len(use_lanes)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(main_stream):
            with torch.cuda.graph(g, stream=main_stream, capture_error_mode="relaxed"):
                if L == 1:
                    for i in range(rounds):
                        step(bp.buffer_of_step(i, 0, 1, nb), use_lanes[0], main_stream, path)
                else:
                    fork = torch.cuda.Event()
                    fork.record(main_stream)
                    for li, lane in enumerate(use_lanes):
                        lane.stream.wait_event(fork)
                        for i in range(rounds):
                            step(bp.buffer_of_step(i, li, L, nb), lane, lane.stream, path)
                        join = torch.cuda.Event()
                        join.record(lane.stream)
                        main_stream.wait_event(join)
        return g

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_replays(g, n):
        """n replays back to back; an event after each, so the spread over replays is known."""
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        with torch.cuda.stream(main_stream):
            ev[0].record(main_stream)
            for i in range(n):
                g.replay()
                ev[i + 1].record(main_stream)
        return ev

    def per_replay_ms(ev):
        return [ev[i].elapsed_time(ev[i + 1]) for i in range(len(ev) - 1)]

    # the first call on a device sets kernel attributes: keep it outside any capture
    for lane in lanes[:2]:
        for path in ("fused", "two_call"):
            step(0, lane, main_stream, path)
    torch.cuda.synchronize()

    ROUNDS = max(1, args.rounds)
    other = "two_call" if args.path == "fused" else "fused"
    # The slicing of the streaming passes is baked into a graph when it is captured.  Requests in
    # flight run under the throughput setting (few, long slices); one call at a time under the
    # library's default (slices that fill the GPU once).  Workspaces were sized under the default,
    # which is the larger.
    slice_cap = max(0, args.slice_limit) if n_lanes > 1 else 0
    solar.set_slice_limit(slice_cap)
    slices_in_flight = solar.gram_slices(w.B, w.N, w.d, tdt)
    g_main = capture(ROUNDS, lanes)
    g_other = capture(ROUNDS, lanes, other) if not light else None
    g_single_cap = capture(nb, lanes[:1]) if (n_lanes > 1 and slice_cap > 0) else None
    solar.set_slice_limit(0)
    slices_default = solar.gram_slices(w.B, w.N, w.d, tdt)
    g_main_default = capture(ROUNDS, lanes) if (slice_cap > 0 and not light) else None
    g_single = capture(nb, lanes[:1]) if n_lanes > 1 else g_main
    # warm-up (at least 3 steps and the --warmup asked for), which also calibrates the plan
    warm = max(1, -(-max(args.warmup, 3) // (ROUNDS * n_lanes)))
    with torch.cuda.stream(main_stream):
        for _ in range(warm):
            g_main.replay()
            g_single.replay()
            if g_other is not None:
                g_other.replay()
    sync_all()
    cal = timed_replays(g_main, 2)
    sync_all()
    est_ms = min(per_replay_ms(cal)) / (ROUNDS * n_lanes)
    steps_per_graph, replays, steps = bp.replay_plan(args.steps, n_lanes, est_ms, rounds_per_graph=ROUNDS,
                                                     min_seconds=0.1 if light else 0.5,
                                                     min_replays=10 if light else 50)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    sync_all()
    ev = timed_replays(g_main, replays)
    sync_all()
    ms = ev[0].elapsed_time(ev[-1])
    spread_main = bp.spread(per_replay_ms(ev), steps_per_graph)
    ms_other, spread_other = None, None
    if g_other is not None:
        evo = timed_replays(g_other, max(10, replays // 4))
        sync_all()
        ms_other = evo[0].elapsed_time(evo[-1]) / ((len(evo) - 1) * steps_per_graph)
        spread_other = bp.spread(per_replay_ms(evo), steps_per_graph)
    # single-call latency: one step at a time on one stream
    single_reps = max(3, min(replays * steps_per_graph // nb, 100))
    sev = timed_replays(g_single, single_reps)
    sync_all()
    ms_single = sev[0].elapsed_time(sev[-1]) / (single_reps * (nb if n_lanes > 1 else steps_per_graph))
    ms_single_cap = None
    if g_single_cap is not None:
        g_single_cap.replay()
        sevc = timed_replays(g_single_cap, single_reps)
        sync_all()
        ms_single_cap = sevc[0].elapsed_time(sevc[-1]) / (single_reps * nb)
    default_plan = None
    if g_main_default is not None:
        g_main_default.replay()
        evd = timed_replays(g_main_default, max(10, replays // 4))
        sync_all()
        default_plan = {"ms_per_step": evd[0].elapsed_time(evd[-1]) / ((len(evd) - 1) * steps_per_graph),
                        "spread": bp.spread(per_replay_ms(evd), steps_per_graph), "gram_slices": slices_default,
                        "what": "the same steps in flight under the library's default slicing (slice limit 0)"}
    # ... and as plain calls (no graph): what a caller without graphs pays per step, host work included
    plain_n = 50
    for _ in range(5):
        step(0, lanes[0], main_stream)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(plain_n):
        step(i % nb, lanes[0], main_stream)
    torch.cuda.synchronize()
    ms_plain = (time.perf_counter() - t0) * 1e3 / plain_n

    def timed_graph_ms(g, reps):
        e = timed_replays(g, reps)
        torch.cuda.synchronize()
        return e[0].elapsed_time(e[-1])

    # per-stage timing: each kernel alone, nb launches (rotating batches) per graph replay
    lane0 = lanes[0]
    info = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    taken = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    stages = {
        "gram": lambda k, st: solar.gram_partials(dH[k], lane0.ws, stream=st),
        "eig": lambda k, st: solar.eig_from_partials_ex(w.B, w.N, w.d, w.r, tdt, solar.ROUTE_AUTO, lane0.S,
                                                        lane0.V, info, taken, lane0.ws, stream=st),
        "attn_prepare": lambda k, st: solar.attn_prepare(lane0.S, lane0.V, Wq, Wk, Wv, w.scale, lane0.ws, stream=st),
        "attn_apply": lambda k, st: solar.attn_apply(dC[k], w.r, 0, dO[k], lane0.ws, stream=st),
    }
    stage_ms = {}
    route_words = None
    for name in ("gram", "eig", "attn_prepare", "attn_apply"):
        fn = stages[name]
        with torch.cuda.stream(main_stream):
            if name in ("eig", "attn_prepare"):    # valid inputs for the stage under test
                solar.gram_partials(dH[0], lane0.ws, stream=main_stream)
            if name == "attn_prepare":
                stages["eig"](0, main_stream)
            if name == "attn_apply":
                solar.gram_partials(dH[0], lane0.ws, stream=main_stream)
                stages["eig"](0, main_stream)
                stages["attn_prepare"](0, main_stream)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(main_stream):
            with torch.cuda.graph(g, stream=main_stream, capture_error_mode="relaxed"):
                for k in range(nb):
                    fn(k, main_stream)
            for _ in range(3):
                g.replay()
        torch.cuda.synchronize()
        reps = 20
        stage_ms[name] = timed_graph_ms(g, reps) / (reps * nb)
        if name == "eig":
            route_words = taken.cpu().numpy()
    # the factored-exact softmax attention over the N positions (beside the hot path, not part
    # of `value`): factorization with U Sigma, then the flash-style kernel; timed alone
    factored = None
    if not light and w.dtype == "bf16" and w.d in (64, 128) and w.r in (16, 32, 64):
        US = torch.empty(w.B, w.N, w.r, dtype=tdt, device="cuda")
        with torch.cuda.stream(main_stream):
            solar.lowrank_factor(dH[0], w.r, S=lane0.S, V=lane0.V, US=US, workspace=lane0.ws, M=w.M,
                                 stream=main_stream)
            for _ in range(2):
                solar.factored_softmax_attention_fwd(dC[0], US, lane0.V, Wq, Wk, Wv, w.scale, O=dO[0],
                                                     workspace=lane0.ws, stream=main_stream)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(main_stream):
            with torch.cuda.graph(g, stream=main_stream, capture_error_mode="relaxed"):
                for k in range(nb):
                    solar.factored_softmax_attention_fwd(dC[k], US, lane0.V, Wq, Wk, Wv, w.scale, O=dO[k],
                                                         workspace=lane0.ws, stream=main_stream)
            g.replay()
        torch.cuda.synchronize()
        f_ms = timed_graph_ms(g, 5) / (5 * nb)
        exps = float(w.pairs)
        factored = {"ms_per_call": f_ms, "value": w.pairs / (f_ms * 1e-3), "unit": "pairs/s",
                    "what": "solar_factored_softmax_attention_fwd (operand set-up + flash kernel), US resident",
                    "roofline": {"bound": "alu", "achieved": exps / (f_ms * 1e-3) / 1e12, "peak": SFU_TEXPS,
                                 "unit": "Texp/s", "frac": exps / (f_ms * 1e-3) / 1e12 / SFU_TEXPS,
                                 "note": "one exp2 per candidate x position on the special-function units"}}
    # the backward pass (beside the hot path, not part of `value`): attention part, then the
    # SVD's gradient as one more streaming pass over H; graph replay over the same batches
    backward = None
    if not light:
        bws = solar.alloc_backward_workspace(w.B, w.M, w.N, w.d, w.r, tdt)
        dHg = torch.empty_like(dH[0])
        gO = [torch.randn(w.B, w.M, w.d, device="cuda").to(tdt) for _ in range(min(nb, 8))]
        grads = solar.alloc_attention_grads(dC[0], w.r)

        def bwd_part(k, which):
            if which in (0, 2):
                solar.svd_attention_bwd(dC[k], lane0.S, lane0.V, Wq, Wk, Wv, w.scale, gO[k % len(gO)], bws, out=grads,
                                        stream=main_stream)
            if which in (1, 2):
                solar.svd_backward(dH[k], lane0.S, lane0.V, grads[4], grads[5], dHg, bws, stream=main_stream)

        with torch.cuda.stream(main_stream):
            solar.lowrank_factor(dH[0], w.r, S=lane0.S, V=lane0.V, workspace=lane0.ws, M=w.M, stream=main_stream)
            bwd_part(0, 2)
        torch.cuda.synchronize()
        b_ms = []
        for which in (0, 1, 2):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(main_stream):
                with torch.cuda.graph(g, stream=main_stream, capture_error_mode="relaxed"):
                    for k in range(nb):
                        bwd_part(k, which)
                g.replay()
            torch.cuda.synchronize()
            b_ms.append(timed_graph_ms(g, 5) / (5 * nb))
        es = 2 if w.dtype == "bf16" else 4
        bwd_bytes = es * w.B * (3 * w.M * w.d + 2 * w.N * w.d)        # C, dO, dC; H, dH
        backward = {"ms_per_call": b_ms[2], "attention_bwd_ms": b_ms[0], "svd_backward_ms": b_ms[1],
                    "what": "solar_svd_attention_bwd + solar_svd_backward, one batch at a time on one stream",
                    "roofline": {"bound": "hbm", "achieved": bwd_bytes / (b_ms[2] * 1e-3) / 1e9,
                                 "peak": peaks()["hbm_gbs"], "unit": "GB/s",
                                 "frac": bwd_bytes / (b_ms[2] * 1e-3) / 1e9 / peaks()["hbm_gbs"],
                                 "algorithmic_bytes": bwd_bytes,
                                 "note": "eight short kernels back to back: latency- and launch-bound"}}
    clocks = sampler.stop() if rank == 0 else None

    # end to end through the public API with host buffers (pinned), copies inside the timed region
    hH = torch.from_numpy(batches[0]["H"]).to(tdt).pin_memory()
    hC = torch.from_numpy(batches[0]["C"]).to(tdt).pin_memory()
    # Requests are independent, so consecutive steps go to E slots (stream, device buffers, host
    # result buffer of their own): the copies of one step overlap the kernels of another, as a
    # serving loop would run them.  Every step still pays its own H2D and D2H inside the timed region.
    E = max(1, min(3, nb))
    e2e_lanes = lanes[:E] + [Lane(torch, solar, w, tdt) for _ in range(E - len(lanes[:E]))]
    hOs = [torch.empty_like(hC).pin_memory() for _ in range(E)]
    hO = hOs[0]
    e2e_steps = 3 if light else max(3, min(steps, 60))
    e2e_count = [0]

    def e2e_step():
        k = e2e_count[0] % E
        e2e_count[0] += 1
        st = e2e_lanes[k].stream
        with torch.cuda.stream(st):
            dH[k].copy_(hH, non_blocking=True); dC[k].copy_(hC, non_blocking=True)
            step(k, e2e_lanes[k], st)
            hOs[k].copy_(dO[k], non_blocking=True)

    for _ in range(3):
        e2e_step()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    ms, e2e_s, ms_single = bp.max_over_ranks([ms, e2e_s, ms_single], dist if world > 1 else None, "cuda")
    if rank != 0:
        return None

    pk = peaks()
    ms_step = ms / steps
    value = bp.aggregate_throughput(w.pairs, world, ms_step)
    roof_s = max(ab["total"] / (pk["hbm_gbs"] * 1e9), algorithmic_flops(w) / (pk["bf16_tflops"] * 1e12))
    dominant = max(stage_ms, key=stage_ms.get)
    tot = sum(stage_ms.values())
    routes = sorted(set(int(x) & 0xFF for x in route_words))
    iters = float(np.mean([(int(x) >> 8) & 0xFF for x in route_words]))
    sweeps = float(np.mean([(int(x) >> 16) & 0xFF for x in route_words]))
    eflops = eig_flops(w, max(routes), iters, sweeps)
    per_kernel = {
        "gram": {"bound": "hbm", "achieved": ab["gram"] / (stage_ms["gram"] * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
                 "unit": "GB/s"},
        "attn_apply": {"bound": "hbm", "achieved": ab["attn"] / (stage_ms["attn_apply"] * 1e-3) / 1e9,
                       "peak": pk["hbm_gbs"], "unit": "GB/s"},
        "eig": {"bound": "alu", "achieved": eflops / (stage_ms["eig"] * 1e-3) / 1e12, "peak": FP32_ALU_TFLOPS,
                "unit": "TFLOP/s", "note": "one CTA per user on B of 148 SMs, a chain of dependent steps (Householder reflections, Sturm counts, "
                        "orthogonalisation, or Jacobi rounds in the fallback): latency-bound"},
        "attn_prepare": {"bound": "alu", "achieved": 6.0 * w.B * w.r * w.d * w.d / (stage_ms["attn_prepare"] * 1e-3) / 1e12,
                         "peak": FP32_ALU_TFLOPS, "unit": "TFLOP/s"},
    }
    for k, v in per_kernel.items():
        v["frac"] = v["achieved"] / v["peak"]
        v["traffic"] = measured_traffic(w.name, k)
    traffic = measured_traffic(w.name, dominant)
    roof = dict(per_kernel[dominant], kernel=dominant, traffic=traffic, peak_source=pk["source"])
    line = {
        "metric": "svd_attention_fwd_candidates_x_positions_per_sec",
        "value": value, "unit": "pairs/s", "n_gpus": world, "steps": steps,
        "warmup": warm * steps_per_graph + 2 * steps_per_graph, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "d": w.d, "r": w.r, "M": w.M,
                   "storage": w.dtype, "users_per_gpu": w.B, "in_flight": n_lanes, "path": args.path,
                   "launch": f"CUDA graphs of {steps_per_graph} steps ({ROUNDS} per lane), {replays} replays, "
                             f"{ms * 1e-3:.2f} s timed",
                   "slice_limit": slice_cap, "gram_slices": slices_in_flight,
                   "distinct_batches": nb, "seeded_batches": nseed,
                   "l2": f"every step in flight has its own input and output buffers: {nb} buffer sets "
                         f"({nb * ab['total'] / 2**20:.0f} MiB > 126 MiB L2), {nseed} seeded batches and device "
                         "copies of them with the users rotated"},
        "ms_per_step_spread": spread_main,
        "single_call": {"ms_per_step": ms_single, "value": world * w.pairs / (ms_single * 1e-3),
                        "note": "one step at a time on one stream (in_flight = 1), graph replay, the library's "
                                "default slicing (slice limit 0)",
                        "gram_slices": slices_default,
                        "ms_per_step_with_slice_limit": ms_single_cap,
                        "plain_calls_ms_per_step": ms_plain,
                        "plain_calls_note": "the same without a graph: host launch work included"},
        ("two_call" if args.path == "fused" else "fused"): (None if ms_other is None else {
            "ms_per_step": ms_other, "value": world * w.pairs / (ms_other * 1e-3), "spread": spread_other,
            "frac": (w.pairs / (ms_other * 1e-3)) / (w.pairs / roof_s),
            "what": ("solar_lowrank_factor + solar_svd_attention_fwd (four launches per step)"
                     if args.path == "fused" else "solar_svd_attention_fused (three launches per step)")}),
        "default_slicing_in_flight": default_plan,
        "path_roofline": {"bound": "hbm", "algorithmic_bytes": ab["total"],
                          "algorithmic_flops": algorithmic_flops(w),
                          "roofline_pairs_per_s": w.pairs / roof_s, "frac": value / world / (w.pairs / roof_s),
                          "frac_single_call": (w.pairs / (ms_single * 1e-3)) / (w.pairs / roof_s),
                          "peak_source": pk["source"]},
        "roofline": roof,
        "roofline_by_kernel": per_kernel,
        "stage_ms": stage_ms, "stage_share": {k: v / tot for k, v in stage_ms.items()},
        "dominant_stage": dominant,
        "eig_route": {"routes": routes, "power_steps": iters, "sweeps_or_passes": sweeps,
                      "note": "route 3 = tridiagonal (orthogonalisation passes), 2 = Jacobi (sweeps), 1 = range finder"},
        "gpu_launches": KERNELS_PER_STEP[args.path] * steps,
        "clocks": clocks,
        "factored_exact": factored,
        "backward": backward,
        "e2e": {"value": world * w.pairs * e2e_steps / e2e_s, "unit": "pairs/s",
                "h2d_bytes_per_step": hH.numel() * hH.element_size() + hC.numel() * hC.element_size(),
                "d2h_bytes_per_step": hO.numel() * hO.element_size(), "steps": e2e_steps,
                "slots": E, "note": "pinned host buffers; consecutive steps alternate over `slots` streams"},
    }
    if not args.no_cpu_baseline and world >= 1:
        users = list(range(min(w.B, args.cpu_users)))
        t = oracle_step(w, users)
        one = users[:max(1, len(users) // 4)]
        t1 = oracle_step_single_thread(w, one)
        line["cpu_baseline"] = {"value": len(users) * w.M * w.N / t, "unit": "pairs/s",
                                "cores": cpu_threads(), "host_cpus": os.cpu_count(), "kind": "oracle", "seconds": t,
                                "sample": f"{len(users)} of {w.B} users, all {w.M} candidates",
                                "note": "numpy fp64; the Jacobi sweeps are a Python loop, only its matrix "
                                        "products use the BLAS pool of `cores` threads",
                                "single_thread": None if t1 is None else {
                                    "value": len(one) * w.M * w.N / t1, "unit": "pairs/s", "cores": 1, "seconds": t1,
                                    "sample": f"{len(one)} of {w.B} users, all {w.M} candidates, BLAS pools limited to 1 thread"}}
    return line


if __name__ == "__main__":
    main()
