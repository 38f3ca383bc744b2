"""Where the step time goes with many requests in flight: the time per step of chains made of a
SUBSET of the step's kernels (stage-level calls), measured like the benchmark measures the whole
step -- one CUDA graph with `lanes` streams, every step on buffers of its own.

    python -m paper_2603_02561_b200.mix_probe [--workload c3] [--slice-limit 2] [--lanes 30] [--out FILE.md]

Chains: g = Gram pass, e = eigensolver (without the projection epilogue), p = stand-alone projections,
a = candidate attention; "fused" = solar_svd_attention_fused.  A chain without `e` or `p` runs on
the factors and operands a complete call left in the lane's buffers.
"""
from __future__ import annotations

import argparse
import sys

import torch

from . import bench_plan as bp
from . import solar
from . import workloads as wl


def _dev(a, dtype):
    t = torch.from_numpy(a)
    return (t.to(torch.bfloat16) if dtype == "bf16" else t.float()).cuda().contiguous()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--slice-limit", type=int, default=2)
    ap.add_argument("--lanes", type=int, default=30)
    ap.add_argument("--rounds", type=int, default=24)
    ap.add_argument("--replays", type=int, default=30)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()
    w = wl.lookup(args.workload)
    inp = wl.generate(w)
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    H0, C0 = _dev(inp["H"], w.dtype), _dev(inp["C"], w.dtype)
    Wq, Wk, Wv = (_dev(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    L, rounds = args.lanes, args.rounds
    nb = bp.distinct_buffers(L, 7)
    dH = [torch.roll(H0, i, 0).contiguous() for i in range(nb)]
    dC = [torch.roll(C0, i, 0).contiguous() for i in range(nb)]
    dO = [torch.empty_like(C0) for _ in range(nb)]
    solar.set_slice_limit(0)
    lanes = []
    for _ in range(L):
        lane = {"stream": torch.cuda.Stream(), "ws": solar.alloc_fused_workspace(w.B, w.M, w.N, w.d, w.r, tdt),
                "S": torch.empty(w.B, w.r, device="cuda"), "V": torch.empty(w.B, w.d, w.r, device="cuda"),
                "info": torch.zeros(w.B, dtype=torch.int32, device="cuda")}
        solar.svd_attention_fused(dH[0], dC[0], Wq, Wk, Wv, w.r, inp["scale"], S=lane["S"], V=lane["V"], O=dO[0],
                                  workspace=lane["ws"])
        lanes.append(lane)
    torch.cuda.synchronize()
    solar.set_slice_limit(args.slice_limit)
    main_stream = torch.cuda.Stream()

    def step(kinds, k, lane):
        st = lane["stream"]
        if kinds == "fused":
            solar.svd_attention_fused(dH[k], dC[k], Wq, Wk, Wv, w.r, inp["scale"], 0, S=lane["S"], V=lane["V"],
                                      O=dO[k], workspace=lane["ws"], stream=st)
            return
        if "g" in kinds:
            solar.gram_partials(dH[k], lane["ws"], stream=st)
        if "e" in kinds:
            solar.eig_from_partials(w.B, w.N, w.d, w.r, tdt, lane["S"], lane["V"], lane["info"], lane["ws"], stream=st)
        if "p" in kinds:
            solar.attn_prepare(lane["S"], lane["V"], Wq, Wk, Wv, inp["scale"], lane["ws"], stream=st)
        if "a" in kinds:
            solar.attn_apply(dC[k], w.r, 0, dO[k], lane["ws"], stream=st)

    def run(kinds):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(main_stream):
            with torch.cuda.graph(g, stream=main_stream, capture_error_mode="relaxed"):
                fork = torch.cuda.Event()
                fork.record(main_stream)
                for li, lane in enumerate(lanes):
                    lane["stream"].wait_event(fork)
                    for i in range(rounds):
                        step(kinds, bp.buffer_of_step(i, li, L, nb), lane)
                    join = torch.cuda.Event()
                    join.record(lane["stream"])
                    main_stream.wait_event(join)
        with torch.cuda.stream(main_stream):
            for _ in range(3):
                g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(main_stream)
            for _ in range(args.replays):
                g.replay()
            e1.record(main_stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (args.replays * rounds * L) * 1e3

    rows = [(k, run(k)) for k in ("g", "a", "e", "ga", "ge", "gea", "gepa", "fused")]
    solar.set_slice_limit(0)
    nan = sum(int(torch.isnan(o.float()).any()) for o in dO)
    lines = [f"# Kernel mix in flight: {w.name}, {L} lanes, slice limit {args.slice_limit}", "",
             f"Command: `python -m paper_2603_02561_b200.mix_probe {' '.join(sys.argv[1:])}`".replace("  ", " "), "",
             "Time per step of a chain made of some of the step's kernels (g Gram, e eigensolver, p projections,",
             "a attention; stage-level calls), every step on buffers of its own, one CUDA graph over all lanes.", "",
             "| chain | us per step |", "|---|---|"]
    lines += [f"| {k} | {t:.2f} |" for k, t in rows]
    lines += ["", f"Output buffers with NaN rows after the runs: {nan} of {nb}.", ""]
    text = "\n".join(lines)
    print(text)
    if args.out:
        open(args.out, "w").write(text)


if __name__ == "__main__":
    main()
