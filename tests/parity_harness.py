"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI
binding and compare with the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import oracle as o
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

# Tolerances on max_m |O_gpu[m]-O_ref[m]|_inf / |O_ref[m]|_inf (rows m), per storage type.
TOL = {"f32": 1e-4, "bf16": 2e-2}
# |v| gap below which the largest component of a vector is "tied" and either sign obeys the gauge
TIE = {"f32": 1e-5, "bf16": 1e-3}


def to_device(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t      # exact: values are bf16-representable


def run_gpu(w: wl.Workload, inp: dict, flags: int = 0, want_us: bool = False, poison: bool = True):
    """Whole forward through solar_lowrank_factor + solar_svd_attention_fwd."""
    H = to_device(inp["H"], w.dtype); C = to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    B, N, d = H.shape
    M = C.shape[1]
    ws = solar.alloc_workspace(B, M, N, d, w.r, H.dtype)
    S = torch.empty(B, w.r, dtype=torch.float32, device="cuda")
    V = torch.empty(B, d, w.r, dtype=torch.float32, device="cuda")
    O = torch.empty_like(C)
    info = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    US = torch.empty(B, N, w.r, dtype=H.dtype, device="cuda") if want_us else None
    if poison:                       # unwritten outputs must show up as NaN
        ws.fill_(0xFF); S.fill_(float("nan")); V.fill_(float("nan")); O.fill_(float("nan"))
        if US is not None:
            US.fill_(float("nan"))
    solar.lowrank_factor(H, w.r, S=S, V=V, US=US, info=info, workspace=ws, M=M)
    solar.svd_attention_fwd(C, S, V, Wq, Wk, Wv, inp["scale"], flags, O=O, workspace=ws, N=N)
    torch.cuda.synchronize()
    out = {"S": S.cpu().numpy().astype(np.float64), "V": V.cpu().numpy().astype(np.float64),
           "O": O.float().cpu().numpy().astype(np.float64), "info": info.cpu().numpy()}
    if US is not None:
        out["US"] = US.float().cpu().numpy().astype(np.float64)
    return out


def gauge_flips(V_gpu, V_ref, dtype):
    """Signs that align the oracle's vectors with the GPU's; a disagreement is only
    accepted where the gauge is numerically tied (top two |components| within TIE)."""
    dots = np.sum(V_gpu * V_ref, axis=0)
    flips = np.where(dots < 0, -1.0, 1.0)
    for i in np.nonzero(flips < 0)[0]:
        a = np.sort(np.abs(V_ref[:, i]))[::-1]
        assert a[0] - a[1] <= TIE[dtype] * 4, f"vector {i}: sign gauge violated (|v| top two {a[:2]})"
    return flips


def check_gauge_rule(V_gpu):
    """The GPU's own V obeys the rule: largest-magnitude component is positive."""
    idx = np.argmax(np.abs(V_gpu), axis=0)
    lead = V_gpu[idx, np.arange(V_gpu.shape[1])]
    assert np.all(lead > 0), "gauge: largest component not positive"


def compare_user(w: wl.Workload, inp: dict, got: dict, k: int, softmax: bool = True):
    """Oracle for user k of the batch; returns a dict of error figures."""
    H = inp["H"][k].astype(np.float64); C = inp["C"][k].astype(np.float64)
    Wq, Wk, Wv = (inp[n].astype(np.float64) for n in ("Wq", "Wk", "Wv"))
    s, V, U = o.truncated_svd(H, w.r)
    Vg = got["V"][k]
    check_gauge_rule(Vg)
    nz = s > 1e-6 * s[0]                       # vectors of zero singular values are arbitrary
    flips = np.ones(w.r)
    flips[nz] = gauge_flips(Vg[:, nz], V[:, nz], w.dtype)
    O_ref = o.svd_attention_from_factors(C, s, V * flips, Wq, Wk, Wv, inp["scale"], softmax)
    err = o.max_rel_err_rows(got["O"][k], O_ref)
    s_err = float(np.abs(got["S"][k] - s).max() / s[0])
    return {"o_err": err, "s_err": s_err, "s": s, "V": V * flips, "U": U * flips, "O_ref": O_ref}
