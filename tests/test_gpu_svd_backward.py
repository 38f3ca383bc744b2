"""solar_svd_backward (Eq. 13-15: dH = U [diag(dS) + 2 Sigma sym(F o (dV^T V))] V^T with
U = H V Sigma^-1) against the CPU oracle, element by element, on the factors the CUDA
factorization itself returns; and, end to end, against finite differences of the
forward oracle."""
import numpy as np
import pytest
import torch

import oracle as o
from oracle import svd_attention_backward as ob
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu

CASES = [
    # workload (shape, dtype, spectrum), eps_rel
    (wl.CONFIGS["c3"].with_(B=2, N=1000, M=8), 0.0),                # tensor-core path, ragged tail
    (wl.CONFIGS["c3"].with_(B=2, N=4096, M=8, r=27), 0.0),          # r not a multiple of 8
    (wl.CONFIGS["c3"].with_(B=1, N=20000, M=8, r=16), 1e-3),        # many row slices, stabilised F
    (wl.CONFIGS["c4"].with_(B=2, N=700, M=8), 0.0),                 # d = 128, r = 64
    (wl.CONFIGS["c2"].with_(B=3, N=100, M=8), 0.0),                 # N < 128: FFMA kernel
    (wl.CONFIGS["c1"], 0.0),                                        # fp32 storage, d = 32
]


def _run(w, inp, eps_rel, seed):
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    H = ph.to_device(inp["H"], w.dtype)
    B, N, d = H.shape
    ws = solar.alloc_workspace(B, w.M, N, d, w.r, tdt)
    S, V = solar.lowrank_factor(H, w.r, workspace=ws)
    g = torch.Generator().manual_seed(seed)
    dS = torch.randn(B, w.r, generator=g).cuda()
    dV = torch.randn(B, d, w.r, generator=g).cuda()
    out_buf = torch.full((B * N * d + 64,), float("nan"), dtype=tdt, device="cuda")
    dH = out_buf[: B * N * d].view(B, N, d)
    solar.svd_backward(H, S, V, dS, dV, dH, ws, eps_rel=eps_rel)
    torch.cuda.synchronize()
    assert torch.isnan(out_buf[B * N * d:].float()).all()           # nothing written past the end
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    return f64(S), f64(V), f64(dS), f64(dV), f64(dH)


@pytest.mark.parametrize("w,eps_rel", CASES, ids=[f"{c[0].name}_N{c[0].N}_r{c[0].r}" for c in CASES])
def test_svd_backward_matches_oracle(w, eps_rel):
    inp = wl.generate(w)
    S, V, dS, dV, dH = _run(w, inp, eps_rel, seed=w.N + w.r)
    assert np.isfinite(dH).all()
    for k in range(S.shape[0]):
        ref = ob.svd_backward(inp["H"][k].astype(np.float64), S[k], V[k], dS[k], dV[k], eps_rel)
        scale = np.abs(ref).max()
        # one rounding to the storage type plus fp32 arithmetic in the d x d matrix K
        tol = 2.0 ** -7 if w.dtype == "bf16" else 2e-4
        err = np.abs(dH[k] - ref).max() / scale
        assert err <= tol, (k, err)


def test_svd_backward_is_the_gradient_of_the_forward_pass():
    """r = d (nothing truncated, so Eq. 15 is the exact gradient): <dH, D> against central
    differences of the forward oracle along random directions D."""
    w = wl.Workload("fd", "f32", 1, 40, 32, 32, 6, "spectrum", rank=32, decay=0.5, seed_index=41)
    inp = wl.generate(w)
    H = inp["H"][0].astype(np.float64)
    C, Wq, Wk, Wv = (inp[k].astype(np.float64) for k in ("C", "Wq", "Wk", "Wv"))
    C = C[0]
    rng = np.random.default_rng(5)
    R = rng.standard_normal(C.shape)
    # dS, dV from the oracle's attention backward at the GPU's factors; dH from the CUDA path
    Hd = ph.to_device(inp["H"], "f32")
    ws = solar.alloc_workspace(1, w.M, w.N, w.d, w.r, torch.float32)
    S, V = solar.lowrank_factor(Hd, w.r, workspace=ws)
    s64, V64 = S[0].cpu().numpy().astype(np.float64), V[0].cpu().numpy().astype(np.float64)
    g = ob.svd_attention_backward(C, s64, V64, Wq, Wk, Wv, inp["scale"], R, True)
    dS = torch.from_numpy(g["ds"]).float().cuda()[None]
    dV = torch.from_numpy(g["dV"]).float().cuda()[None].contiguous()
    dH = torch.empty_like(Hd)
    solar.svd_backward(Hd, S, V, dS, dV, dH, ws)
    torch.cuda.synchronize()
    dH = dH[0].cpu().numpy().astype(np.float64)
    loss = lambda X: float((o.svd_attention(X, C, Wq, Wk, Wv, w.r, inp["scale"], True) * R).sum())
    for k in range(3):
        D = rng.standard_normal(H.shape)
        t = 1e-5
        fd = (loss(H + t * D) - loss(H - t * D)) / (2 * t)
        got = float((dH * D).sum())
        assert abs(got - fd) <= 2e-3 * max(abs(fd), np.abs(dH).max()), (k, got, fd)


def test_argument_checks():
    H = torch.zeros(1, 256, 64, dtype=torch.bfloat16, device="cuda")
    S = torch.ones(1, 8, device="cuda"); V = torch.zeros(1, 64, 8, device="cuda")
    dH = torch.empty_like(H)
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(solar.SolarError) as e:
        solar.svd_backward(H, S, V, S, V, dH, small)
    assert e.value.status == solar.ERR_WORKSPACE
    ws = solar.alloc_workspace(1, 1, 256, 64, 8, torch.bfloat16)
    with pytest.raises(solar.SolarError) as e:
        solar.svd_backward(H, S, V, S, V, dH, ws, eps_rel=-1.0)
    assert e.value.status == solar.ERR_INVALID_ARG
