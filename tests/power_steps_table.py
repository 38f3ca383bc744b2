"""Accuracy of Algorithm 1 (randomized range finder with power iteration, run on the Gram matrix
by the CUDA library) as a function of the number of power steps, against the CPU oracle's exact
truncated SVD.  Not a test: a tool that needs a GPU and writes a table.

    python tests/power_steps_table.py [--out profiles/power_steps.md]

For n_iter = 0 .. 4 (the library's forced count is n_iter + 1 orthonormalised steps) and a few
users of c2, c3 and two c5 points: largest singular-value error relative to sigma_1, smallest
|<v_gpu, v_oracle>| over the kept vectors, largest row-normalised output error of the attention
that uses these factors, and how many of the users the library's own residual / trace bounds
certify."""
import argparse
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle as o  # noqa: E402
import parity_harness as ph  # noqa: E402
from paper_2603_02561_b200 import solar  # noqa: E402
from paper_2603_02561_b200 import workloads as wl  # noqa: E402


def rows_for(w, users):
    inp = wl.generate(w, users=users)
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    H = ph.to_device(inp["H"], w.dtype); C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    B = len(users)
    ws = solar.alloc_workspace(B, w.M, w.N, w.d, w.r, tdt)
    ref = [o.truncated_svd(inp["H"][k].astype(np.float64), w.r) for k in range(B)]
    out = []
    for n_iter in range(5):
        S = torch.empty(B, w.r, device="cuda"); V = torch.empty(B, w.d, w.r, device="cuda")
        info = torch.zeros(B, dtype=torch.int32, device="cuda")
        solar.gram_partials(H, ws)
        solar.eig_from_partials_ex(B, w.N, w.d, w.r, tdt, solar.route_with(solar.ROUTE_SUBSPACE, power_steps=n_iter + 1),
                                   S, V, info, None, ws)
        O = solar.svd_attention_fwd(C, S, V, Wq, Wk, Wv, inp["scale"], workspace=ws, N=w.N)
        torch.cuda.synchronize()
        Sg, Vg = S.cpu().numpy().astype(np.float64), V.cpu().numpy().astype(np.float64)
        Og = O.float().cpu().numpy().astype(np.float64)
        s_err = dot = o_err = 0.0
        dot = 1.0
        for k in range(B):
            s, Vr, _ = ref[k]
            s_err = max(s_err, float(np.abs(Sg[k] - s).max() / s[0]))
            d = np.abs(np.sum(Vg[k] * Vr, axis=0))
            dot = min(dot, float(d.min()))
            flips = np.where(np.sum(Vg[k] * Vr, axis=0) < 0, -1.0, 1.0)
            O_ref = o.svd_attention_from_factors(inp["C"][k].astype(np.float64), s, Vr * flips, inp["Wq"], inp["Wk"],
                                                 inp["Wv"], inp["scale"], True)
            o_err = max(o_err, o.max_rel_err_rows(Og[k], O_ref))
        certified = int((info.cpu().numpy() == 0).sum())
        out.append(f"| {w.name} (N={w.N}, d={w.d}, r={w.r}) | {n_iter} | {s_err:.2e} | {dot:.6f} | {o_err:.2e} | {certified} of {B} |")
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=os.path.join(ROOT, "profiles", "power_steps.md"))
    args = ap.parse_args()
    sweep = {x.name: x for x in wl.sweep_configs()}
    cases = [(wl.CONFIGS["c2"], [0, 1, 2, 3]), (wl.CONFIGS["c3"], [0, 1, 2, 3]),
             (sweep["c5_N8192_r16"], [0, 1, 2, 3]), (sweep["c5_N8192_r32"], [0, 1, 2, 3]),
             (wl.CONFIGS["serve27"], [0, 1])]
    lines = ["# Algorithm 1 on the Gram matrix: accuracy against the number of power steps", "",
             "Command: `python tests/power_steps_table.py` (one B200; the oracle is the exact truncated SVD in fp64).", "",
             "`n_iter` is Algorithm 1's count (the range is span(G^(n_iter+1) Omega), re-orthonormalised every step); ",
             "sigma error is relative to sigma_1; the dot product is the smallest over the kept vectors and users; the ",
             "output error is max over rows of |dO|_inf / |O|_inf (tolerance 2e-2 in bf16); `certified` counts the users ",
             "whose result the library's residual and trace bounds accept.", "",
             "| workload | n_iter | max sigma error | min abs(v_gpu . v_oracle) | max output error | certified |",
             "|---|---|---|---|---|---|"]
    for w, users in cases:
        lines += rows_for(w, users)
    lines.append("")
    open(args.out, "w").write("\n".join(lines))
    print("\n".join(lines))


if __name__ == "__main__":
    main()
