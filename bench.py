#!/usr/bin/env python
"""Benchmark of the SVD-Attention forward pass (solar_lowrank_factor + solar_svd_attention_fwd).

One "step" = one pass of the whole hot path over one batch of B users: streaming Gram of
H, Jacobi eigensolve, factor-token projections, candidate attention.  Metric: candidates x
sequence positions per second = B*M*N / step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own batch of B
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

from paper_2603_02561_b200 import workloads as wl  # noqa: E402

L2_BYTES = 126 * 2 ** 20
KERNELS_PER_STEP = 4          # gram, eigensolve, factor-token projections, attention


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
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def run_reference(args, w: wl.Workload):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_users = list(range(min(w.B, args.ref_users)))
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
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--cpu-users", type=int, default=8, help="users in the cpu_baseline sample")
    ap.add_argument("--ref-users", type=int, default=2, help="users per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    w = wl.CONFIGS[args.workload]

    if args.impl == "reference":
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

    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    ab = algorithmic_bytes(w)
    # rotate over enough distinct batches that a step's inputs are never L2-resident
    nb = max(2, -(-int(1.5 * L2_BYTES) // ab["total"]))
    batches = []
    for i in range(nb):
        wi = w.with_(seed_index=w.seed_index + 1000 * (rank * nb + i + 1))
        inp = wl.generate(wi)
        batches.append(inp)
    Wq, Wk, Wv = (torch.from_numpy(batches[0][k]).cuda().to(tdt) for k in ("Wq", "Wk", "Wv"))
    dH = [torch.from_numpy(b["H"]).cuda().to(tdt) for b in batches]
    dC = [torch.from_numpy(b["C"]).cuda().to(tdt) for b in batches]
    dO = [torch.empty_like(c) for c in dC]
    S = torch.empty(w.B, w.r, device="cuda"); V = torch.empty(w.B, w.d, w.r, device="cuda")
    ws = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, tdt)
    stream = torch.cuda.current_stream()

    def step(i):
        k = i % nb
        solar.lowrank_factor(dH[k], w.r, S=S, V=V, workspace=ws, M=w.M, stream=stream)
        solar.svd_attention_fwd(dC[k], S, V, Wq, Wk, Wv, w.scale, 0, O=dO[k], workspace=ws, N=w.N,
                                stream=stream)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)

    # per-stage timing (same inputs, same launch configuration), CUDA events on the launch stream
    info = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    stages = {
        "gram": lambda k: solar.gram_partials(dH[k], ws, stream=stream),
        "eig": lambda k: solar.eig_from_partials(w.B, w.N, w.d, w.r, tdt, S, V, info, ws, stream=stream),
        "attn_prepare": lambda k: solar.attn_prepare(S, V, Wq, Wk, Wv, w.scale, ws, stream=stream),
        "attn_apply": lambda k: solar.attn_apply(dC[k], w.r, 0, dO[k], ws, stream=stream),
    }
    reps = max(10, min(args.steps, 50))
    stage_ms = {}
    for name in ("gram", "eig", "attn_prepare", "attn_apply"):
        fn = stages[name]
        if name == "attn_prepare":        # restore valid factors after timing the eigensolver
            solar.gram_partials(dH[0], ws, stream=stream)
            solar.eig_from_partials(w.B, w.N, w.d, w.r, tdt, S, V, info, ws, stream=stream)
        for k in range(3):
            fn(k % nb)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for k in range(reps):
            fn(k % nb)
        b.record(stream)
        torch.cuda.synchronize()
        stage_ms[name] = a.elapsed_time(b) / reps
    clocks = sampler.stop() if rank == 0 else None

    # end to end through the public API with host buffers (pinned), copies inside the timed region
    hH = torch.from_numpy(batches[0]["H"]).to(tdt).pin_memory()
    hC = torch.from_numpy(batches[0]["C"]).to(tdt).pin_memory()
    hO = torch.empty_like(hC).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step():
        dH[0].copy_(hH, non_blocking=True); dC[0].copy_(hC, non_blocking=True)
        solar.lowrank_factor(dH[0], w.r, S=S, V=V, workspace=ws, M=w.M, stream=stream)
        solar.svd_attention_fwd(dC[0], S, V, Wq, Wk, Wv, w.scale, 0, O=dO[0], workspace=ws, N=w.N,
                                stream=stream)
        hO.copy_(dO[0], non_blocking=True)

    for _ in range(3):
        e2e_step()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    tmax = torch.tensor([ms, e2e_s], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    ms, e2e_s = float(tmax[0]), float(tmax[1])
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    ms_step = ms / args.steps
    value = world * w.pairs / (ms_step * 1e-3)
    roof_s = max(ab["total"] / (pk["hbm_gbs"] * 1e9), algorithmic_flops(w) / (pk["bf16_tflops"] * 1e12))
    dominant = max(stage_ms, key=stage_ms.get)
    gram_gbs = ab["gram"] / (stage_ms["gram"] * 1e-3) / 1e9
    tot = sum(stage_ms.values())
    line = {
        "metric": "svd_attention_fwd_candidates_x_positions_per_sec",
        "value": value, "unit": "pairs/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "d": w.d, "r": w.r, "M": w.M,
                   "storage": w.dtype, "users_per_gpu": w.B,
                   "l2": f"inputs rotate over {nb} distinct batches ({nb * ab['total'] / 2**20:.0f} MiB > 126 MiB L2)"},
        "path_roofline": {"bound": "hbm", "algorithmic_bytes": ab["total"],
                          "algorithmic_flops": algorithmic_flops(w),
                          "roofline_pairs_per_s": w.pairs / roof_s, "frac": value / world / (w.pairs / roof_s),
                          "peak_source": pk["source"]},
        "roofline": {"kernel": "gram", "bound": "hbm", "achieved": gram_gbs, "peak": pk["hbm_gbs"],
                     "unit": "GB/s", "frac": gram_gbs / pk["hbm_gbs"], "traffic": None,
                     "peak_source": pk["source"]},
        "stage_ms": stage_ms, "stage_share": {k: v / tot for k, v in stage_ms.items()},
        "dominant_stage": dominant,
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "clocks": clocks,
        "e2e": {"value": world * w.pairs * e2e_steps / e2e_s, "unit": "pairs/s",
                "h2d_bytes_per_step": hH.numel() * hH.element_size() + hC.numel() * hC.element_size(),
                "d2h_bytes_per_step": hO.numel() * hO.element_size(), "steps": e2e_steps},
    }
    if not args.no_cpu_baseline and world >= 1:
        users = list(range(min(w.B, args.cpu_users)))
        t = oracle_step(w, users)
        line["cpu_baseline"] = {"value": len(users) * w.M * w.N / t, "unit": "pairs/s",
                                "cores": cpu_threads(), "kind": "oracle", "seconds": t,
                                "sample": f"{len(users)} of {w.B} users, all {w.M} candidates"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
