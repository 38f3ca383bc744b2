"""solar_factored_softmax_attention_fwd -- softmax over the N history positions evaluated
through the rank-r factors -- against the CPU oracle: its own step-by-step definition
(factored_exact_attention) and, on exactly rank-r histories, brute-force softmax attention
(Eq. 6-7), which it must then reproduce.  Tolerance: the bf16 bound of the parity tests
(max over rows of |dO|_inf / |O_ref|_inf <= 2e-2)."""
import numpy as np
import pytest
import torch

import oracle as o
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu


def _run(w, inp):
    H = ph.to_device(inp["H"], w.dtype); C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    B, N, d = H.shape
    US = torch.full((B, N, w.r), float("nan"), dtype=H.dtype, device="cuda")
    S, V = solar.lowrank_factor(H, w.r, US=US)
    O = torch.full_like(C, float("nan"))
    solar.factored_softmax_attention_fwd(C, US, V, Wq, Wk, Wv, inp["scale"], O=O)
    torch.cuda.synchronize()
    return O.float().cpu().numpy().astype(np.float64)


CASES = [
    # dtype, B, N, d, r, M, kind, rank
    ("bf16", 2, 700, 64, 32, 200, "product", 32),      # ragged N and M tails, exactly rank r
    ("bf16", 2, 128, 64, 16, 128, "product", 16),      # a single tile
    ("bf16", 1, 1300, 64, 64, 130, "product_noise", 64),
    ("bf16", 2, 515, 128, 32, 77, "product", 32),
    ("bf16", 1, 400, 128, 64, 300, "product_noise", 64),
    ("bf16", 3, 260, 128, 16, 5, "product", 16),
]


@pytest.mark.parametrize("dtype,B,N,d,r,M,kind,rank", CASES)
def test_matches_the_oracle(dtype, B, N, d, r, M, kind, rank):
    w = wl.Workload("fx", dtype, B, N, d, r, M, kind, rank=rank, noise_var=1e-2, seed_index=41)
    inp = wl.generate(w)
    got = _run(w, inp)
    assert np.isfinite(got).all()
    for k in range(B):
        H = inp["H"][k].astype(np.float64); C = inp["C"][k].astype(np.float64)
        ref = o.factored_exact_attention(H, C, inp["Wq"], inp["Wk"], inp["Wv"], r, inp["scale"])
        assert o.max_rel_err_rows(got[k], ref) <= ph.TOL["bf16"], (k, o.max_rel_err_rows(got[k], ref))
        if kind == "product":      # rank(H) = r: the factored form IS softmax attention over the N positions
            brute = o.softmax_attention(H, C, inp["Wq"], inp["Wk"], inp["Wv"], inp["scale"])
            assert o.max_rel_err_rows(got[k], brute) <= ph.TOL["bf16"]


def test_headline_shape_sampled_users():
    w = wl.CONFIGS["c3"].with_(B=3, M=600)
    inp = wl.generate(w)
    got = _run(w, inp)
    for k in (0, 2):
        H = inp["H"][k].astype(np.float64); C = inp["C"][k].astype(np.float64)
        brute = o.softmax_attention(H, C, inp["Wq"], inp["Wk"], inp["Wv"], inp["scale"])
        assert o.max_rel_err_rows(got[k], brute) <= ph.TOL["bf16"]


def test_unsupported_shapes_are_refused():
    C = torch.zeros(1, 8, 64, device="cuda", dtype=torch.bfloat16)
    W = torch.zeros(64, 64, device="cuda", dtype=torch.bfloat16)
    US = torch.zeros(1, 200, 24, device="cuda", dtype=torch.bfloat16)
    V = torch.zeros(1, 64, 24, device="cuda")
    with pytest.raises(solar.SolarError) as e:
        solar.factored_softmax_attention_fwd(C, US, V, W, W, W, 0.1)
    assert e.value.status == solar.ERR_UNSUPPORTED
