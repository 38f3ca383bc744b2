"""The two routes of the batched eigensolver (certified range finder of Algorithm 1 on the
Gram matrix; full d x d Jacobi) against each other and against the CPU oracle, and the
per-user choice between them."""
import numpy as np
import pytest
import torch

import oracle as o
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu


def _factor(w, inp, route):
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    H = ph.to_device(inp["H"], w.dtype)
    B = H.shape[0]
    ws = solar.alloc_workspace(B, w.M, w.N, w.d, w.r, tdt)
    S = torch.full((B, w.r), float("nan"), device="cuda")
    V = torch.full((B, w.d, w.r), float("nan"), device="cuda")
    info = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    taken = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    solar.gram_partials(H, ws)
    solar.eig_from_partials_ex(B, w.N, w.d, w.r, tdt, route, S, V, info, taken, ws)
    torch.cuda.synchronize()
    return (S.cpu().numpy().astype(np.float64), V.cpu().numpy().astype(np.float64),
            info.cpu().numpy(), taken.cpu().numpy())


def _oracle_check(w, inp, S, V, k):
    """s against the oracle's, and the subspace angle of every well-separated vector."""
    s, Vr, _ = o.truncated_svd(inp["H"][k].astype(np.float64), w.r)
    assert np.abs(S[k] - s).max() <= (1e-5 if w.dtype == "f32" else 1e-4) * s[0]
    ph.check_gauge_rule(V[k])
    gaps = np.minimum(np.abs(np.diff(s ** 2, prepend=np.inf)), np.abs(np.diff(s ** 2, append=0.0)))
    well = gaps > 1e-3 * s[0] ** 2
    dots = np.abs(np.sum(V[k] * Vr, axis=0))
    assert np.all(dots[well] > 1 - 1e-5), dots[well].min()
    assert np.abs(V[k].T @ V[k] - np.eye(w.r)).max() < 1e-4


CASES = [
    # (workload, users to check, route expected from AUTO: 1 subspace, 2 full, None = either)
    (wl.CONFIGS["c1"], [0], 1),
    (wl.CONFIGS["c2"].with_(B=8), [0, 7], 1),
    (wl.CONFIGS["c3"].with_(B=4, M=8), [0, 3], 1),
    # rank 27 kept out of 32 with sigma_i = 1/i: no gap at the cut, the range finder cannot be certified
    (wl.CONFIGS["c3"].with_(B=2, M=8, r=27, N=4096), [0], 2),
    # exactly rank 27 with r = 27: the oversampled directions deflate
    (wl.Workload("r27", "bf16", 3, 4000, 64, 27, 8, "spectrum", rank=27, decay=1.0, seed_index=31), [0, 2], 1),
    # r = d/2 of a full-rank power law (c4's structure at d = 64)
    (wl.Workload("pl", "bf16", 2, 3000, 64, 32, 8, "spectrum", rank=64, decay=1.5, seed_index=32), [0], 2),
    # r > d/2: only the full route applies
    (wl.Workload("wide", "f32", 2, 500, 32, 24, 8, "product_noise", rank=24, noise_var=1e-2, seed_index=33), [1], 2),
]


@pytest.mark.parametrize("w,users,expect", CASES, ids=[c[0].name + f"_r{c[0].r}" for c in CASES])
def test_auto_route_matches_full_route_and_oracle(w, users, expect):
    inp = wl.generate(w)
    Sa, Va, ia, ta = _factor(w, inp, solar.ROUTE_AUTO)
    Sf, Vf, if_, tf = _factor(w, inp, solar.ROUTE_FULL)
    assert np.all(ia == 0) and np.all(if_ == 0)
    assert np.all((tf & 0xFF) == 2)
    if expect is not None:
        assert np.all((ta & 0xFF) == expect), [hex(x) for x in ta]
    tol = 1e-5 if w.dtype == "f32" else 1e-4
    assert np.abs(Sa - Sf).max() <= tol * Sf.max()
    for k in users:
        _oracle_check(w, inp, Sa, Va, k)
        _oracle_check(w, inp, Sf, Vf, k)


def test_subspace_only_route_flags_what_it_cannot_certify():
    w = CASES[3][0]
    inp = wl.generate(w)
    S, V, info, taken = _factor(w, inp, solar.ROUTE_SUBSPACE)
    assert np.all((taken & 0xFF) == 1)
    assert np.all(info == solar.INFO_NOT_CERTIFIED)
    assert np.isfinite(S).all() and np.isfinite(V).all()


def test_routes_give_the_same_attention_output():
    w = wl.CONFIGS["c2"].with_(B=4, N=2000, M=300)
    inp = wl.generate(w)
    C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    outs = []
    for route in (solar.ROUTE_AUTO, solar.ROUTE_FULL):
        S, V, info, _ = _factor(w, inp, route)
        O = solar.svd_attention_fwd(C, torch.from_numpy(S).float().cuda(), torch.from_numpy(V).float().cuda(),
                                    Wq, Wk, Wv, inp["scale"])
        torch.cuda.synchronize()
        outs.append(O.float().cpu().numpy().astype(np.float64))
    assert o.max_rel_err_rows(outs[0], outs[1]) < 1e-2     # both are within 2e-2 of the oracle
