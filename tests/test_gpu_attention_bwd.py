"""solar_svd_attention_bwd (chain rule through Eq. 11-12) against the CPU oracle on the
factors the CUDA factorization returns, element by element; the whole backward pass
(attention part, then Eq. 13-15) against the oracle's; reproducibility bit for bit."""
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
    # workload, flags
    (wl.CONFIGS["c1"], 0),                                           # fp32 storage, d = 32
    (wl.CONFIGS["c1"], solar.FLAG_NO_SOFTMAX),
    (wl.CONFIGS["c2"].with_(B=4, M=300), 0),                         # several chunks, ragged last batch
    (wl.CONFIGS["c2"].with_(B=3, M=5), 0),                           # fewer rows than one batch
    (wl.CONFIGS["c3"].with_(B=2, N=2048, M=700), 0),
    (wl.CONFIGS["c3"].with_(B=2, N=2048, M=257, r=27), solar.FLAG_NO_SOFTMAX),
    (wl.CONFIGS["c4"].with_(B=2, N=512, M=200), 0),                  # d = 128, r = 64
]


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _setup(w, seed):
    inp = wl.generate(w)
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    H = ph.to_device(inp["H"], w.dtype); C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    B, N, d = H.shape
    ws = solar.alloc_workspace(B, w.M, N, d, w.r, tdt)
    S, V = solar.lowrank_factor(H, w.r, workspace=ws)
    g = torch.Generator().manual_seed(seed)
    dO = torch.randn(B, w.M, d, generator=g).to(tdt).cuda()
    bws = solar.alloc_backward_workspace(B, w.M, N, d, w.r, tdt)
    return inp, H, C, Wq, Wk, Wv, S, V, dO, bws


def _rel(got, ref):
    return np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-300)


def _check_dC(got, ref, dtype):
    """dC against the oracle.  A row of dC = dS T^T is a difference of terms (dS = P o (dP - rowsum));
    where the softmax saturates the row nearly cancels, so the error is measured against the
    matrix's scale, and row by row only on the rows that carry weight."""
    tol = 2.0 ** -7 if dtype == "bf16" else 1e-4          # one rounding to the storage type
    assert _rel(got, ref) <= tol
    rows = np.abs(ref).max(axis=1) >= 1e-2 * np.abs(ref).max()
    assert rows.any()
    assert o.max_rel_err_rows(got[rows], ref[rows]) <= (2e-2 if dtype == "bf16" else 1e-4)


@pytest.mark.parametrize("w,flags", CASES, ids=[f"{c[0].name}_M{c[0].M}_r{c[0].r}_f{c[1]}" for c in CASES])
def test_attention_bwd_matches_oracle(w, flags):
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=w.M + w.r)
    bws.fill_(0xFF)
    dC, dWq, dWk, dWv, dS, dV = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws, flags=flags)
    torch.cuda.synchronize()
    S64, V64, dO64 = _f64(S), _f64(V), _f64(dO)
    B = S64.shape[0]
    sums = {k: 0.0 for k in ("dWq", "dWk", "dWv")}
    for k in range(B):
        g = ob.svd_attention_backward(inp["C"][k].astype(np.float64), S64[k], V64[k],
                                      *(inp[n].astype(np.float64) for n in ("Wq", "Wk", "Wv")),
                                      inp["scale"], dO64[k], softmax=not flags)
        _check_dC(_f64(dC[k]), g["dC"], w.dtype)
        assert _rel(_f64(dS[k]), g["ds"]) <= 1e-4
        assert _rel(_f64(dV[k]), g["dV"]) <= 1e-4
        for n in sums:
            sums[n] = sums[n] + g[n]
    for n, t in (("dWq", dWq), ("dWk", dWk), ("dWv", dWv)):
        assert _rel(_f64(t), sums[n]) <= 1e-4, n


def test_whole_backward_pass_matches_oracle():
    w = wl.CONFIGS["c3"].with_(B=2, N=1500, M=400)
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=11)
    dC, dWq, dWk, dWv, dS, dV = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws)
    dH = torch.empty_like(H)
    solar.svd_backward(H, S, V, dS, dV, dH, bws)
    torch.cuda.synchronize()
    S64, V64, dO64 = _f64(S), _f64(V), _f64(dO)
    for k in range(2):
        g = ob.svd_attention_backward_full(inp["H"][k].astype(np.float64), inp["C"][k].astype(np.float64),
                                           S64[k], V64[k], *(inp[n].astype(np.float64) for n in ("Wq", "Wk", "Wv")),
                                           inp["scale"], dO64[k])
        assert _rel(_f64(dH[k]), g["dH"]) <= 2.0 ** -7


@pytest.mark.parametrize("name,users", [("c3", (0, 15)), ("c4", (3,))])
def test_full_size_backward_sampled_users(name, users):
    """The headline shapes in the launch configuration the benchmark times: every gradient of the
    sampled users against the oracle (dW sums need all users: checked through per-user partial sums
    of the oracle over ALL users for c3 only, where that is cheap)."""
    w = wl.CONFIGS[name]
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=17)
    dC, dWq, dWk, dWv, dS, dV = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws)
    dH = torch.empty_like(H)
    solar.svd_backward(H, S, V, dS, dV, dH, bws, eps_rel=1e-4)
    torch.cuda.synchronize()
    S64, V64, dO64 = _f64(S), _f64(V), _f64(dO)
    W64 = [inp[n].astype(np.float64) for n in ("Wq", "Wk", "Wv")]
    sums = {k: 0.0 for k in ("dWq", "dWk", "dWv")}
    for k in (range(w.B) if name == "c3" else users):
        g = ob.svd_attention_backward(inp["C"][k].astype(np.float64), S64[k], V64[k], *W64, inp["scale"], dO64[k])
        for n in sums:
            sums[n] = sums[n] + g[n]
        if k not in users:
            continue
        _check_dC(_f64(dC[k]), g["dC"], w.dtype)
        assert _rel(_f64(dS[k]), g["ds"]) <= 1e-4
        assert _rel(_f64(dV[k]), g["dV"]) <= 1e-4
        ref = ob.svd_backward(inp["H"][k].astype(np.float64), S64[k], V64[k], _f64(dS[k]), _f64(dV[k]), 1e-4)
        assert _rel(_f64(dH[k]), ref) <= 2.0 ** -7
    if name == "c3":
        for n, t in (("dWq", dWq), ("dWk", dWk), ("dWv", dWv)):
            assert _rel(_f64(t), sums[n]) <= 1e-4, n


def test_attention_bwd_is_reproducible_bit_for_bit():
    w = wl.CONFIGS["c2"].with_(B=4, M=1000)
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=3)
    a = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws)
    torch.cuda.synchronize()
    bws2 = torch.zeros_like(bws)
    b = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws2)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))


def test_no_candidates_gives_zero_gradients():
    w = wl.CONFIGS["c2"].with_(B=2, M=1)
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=2)
    C0, dO0 = C[:, :0, :].contiguous(), dO[:, :0, :].contiguous()
    dC, dWq, dWk, dWv, dS, dV = solar.svd_attention_bwd(C0, S, V, Wq, Wk, Wv, inp["scale"], dO0, bws)
    torch.cuda.synchronize()
    for t in (dWq, dWk, dWv, dS, dV):
        assert torch.count_nonzero(t) == 0 and torch.isfinite(t).all()


def test_zero_history_has_zero_gradient_and_no_nan():
    """H = 0: every sigma is zero, so no direction has a U column and dH = 0 (no 0/0)."""
    B, N, d, r, M = 2, 300, 64, 8, 40
    H = torch.zeros(B, N, d, dtype=torch.bfloat16, device="cuda")
    g = torch.Generator().manual_seed(9)
    C = (torch.randn(B, M, d, generator=g) / 8).to(torch.bfloat16).cuda()
    dO = torch.randn(B, M, d, generator=g).to(torch.bfloat16).cuda()
    Wq, Wk, Wv = ((torch.randn(d, d, generator=g) / 8).to(torch.bfloat16).cuda() for _ in range(3))
    ws = solar.alloc_workspace(B, M, N, d, r, torch.bfloat16)
    S, V = solar.lowrank_factor(H, r, workspace=ws)
    bws = solar.alloc_backward_workspace(B, M, N, d, r, torch.bfloat16)
    out = solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, 0.125, dO, bws)
    dH = torch.full_like(H, float("nan"))
    solar.svd_backward(H, S, V, out[4], out[5], dH, bws)
    torch.cuda.synchronize()
    assert torch.count_nonzero(S) == 0
    for t in out:
        assert torch.isfinite(t.float()).all()
    assert torch.count_nonzero(dH) == 0
    # scores are all zero, so the probabilities are uniform and dC vanishes with T = 0
    assert torch.count_nonzero(out[0]) == 0


def test_attention_bwd_argument_checks():
    w = wl.CONFIGS["c1"]
    inp, H, C, Wq, Wk, Wv, S, V, dO, bws = _setup(w, seed=1)
    with pytest.raises(solar.SolarError) as e:
        solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws[:128])
    assert e.value.status == solar.ERR_WORKSPACE
    with pytest.raises(solar.SolarError) as e:
        solar.svd_attention_bwd(C, S, V, Wq, Wk, Wv, inp["scale"], dO, bws, flags=2)
    assert e.value.status == solar.ERR_UNSUPPORTED
