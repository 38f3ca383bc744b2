"""The routes of the batched eigensolver (tridiagonal reduction with Sturm multisection and
twisted factorisation; certified range finder of Algorithm 1 on the Gram matrix; full d x d
Jacobi) against each other and against the CPU oracle, and the per-user choice between them."""
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
    # (workload, users to check,
    #  does the range finder of Algorithm 1 certify its own result: True / False, None = no range
    #  finder for this shape (r > d/2),
    #  route AUTO ends with: 3 tridiagonal, 2 Jacobi (gaps between kept eigenvalues below what the
    #  tridiagonal route is trusted with), None = either)
    (wl.CONFIGS["c1"], [0], True, 3),
    (wl.CONFIGS["c2"].with_(B=8), [0, 7], True, 3),
    (wl.CONFIGS["c3"].with_(B=4, M=8), [0, 3], True, 3),
    # rank 27 kept out of 32 with sigma_i = 1/i: no gap at the cut, the range finder cannot be certified
    (wl.CONFIGS["c3"].with_(B=2, M=8, r=27, N=4096), [0], False, 3),
    # exactly rank 27 with r = 27: the oversampled directions deflate
    (wl.Workload("r27", "bf16", 3, 4000, 64, 27, 8, "spectrum", rank=27, decay=1.0, seed_index=31), [0, 2], True, 3),
    # r = d/2 of a full-rank power law (c4's structure at d = 64): lambda_i = i^-3, gaps of a few eps at i = 32
    (wl.Workload("pl", "bf16", 2, 3000, 64, 32, 8, "spectrum", rank=64, decay=1.5, seed_index=32), [0], False, 2),
    # r > d/2: no range finder
    (wl.Workload("wide", "f32", 2, 500, 32, 24, 8, "product_noise", rank=24, noise_var=1e-2, seed_index=33), [1], None, None),
    # c4's own structure (d = 128, r = 64 of a full-rank power law) and all 64 pairs of a 64 x 64 matrix
    (wl.CONFIGS["c4"].with_(B=2, N=2048, M=8), [0, 1], None, 2),
    (wl.Workload("all64", "bf16", 2, 2048, 64, 64, 8, "product_noise", rank=64, noise_var=1e-3, seed_index=34), [0], None, None),
    (wl.Workload("d128r20", "f32", 2, 700, 128, 20, 8, "product_noise", rank=20, noise_var=1e-3, seed_index=35), [1], True, 3),
]


@pytest.mark.parametrize("w,users,certifies,auto_route", CASES, ids=[c[0].name + f"_r{c[0].r}" for c in CASES])
def test_routes_match_each_other_and_the_oracle(w, users, certifies, auto_route):
    inp = wl.generate(w)
    Sa, Va, ia, ta = _factor(w, inp, solar.ROUTE_AUTO)
    Sf, Vf, if_, tf = _factor(w, inp, solar.ROUTE_FULL)
    assert np.all(ia == 0) and np.all(if_ == 0)
    assert np.all((tf & 0xFF) == 2)
    # the default route: tridiagonal reduction where it is certified, else the Jacobi solve
    assert np.all(((ta & 0xFF) == 3) | ((ta & 0xFF) == 2)), [hex(x) for x in ta]
    if auto_route is not None:
        assert np.all((ta & 0xFF) == auto_route), [hex(x) for x in ta]
    if auto_route == 2:
        assert np.all(((ta >> 24) & 0xFF) != 0), [hex(x) for x in ta]       # and it says why
    tol = 1e-5 if w.dtype == "f32" else 1e-4
    assert np.abs(Sa - Sf).max() <= tol * Sf.max()
    for k in users:
        _oracle_check(w, inp, Sa, Va, k)
        _oracle_check(w, inp, Sf, Vf, k)
    # Algorithm 1 on the Gram matrix, alone: certified where its bounds can hold
    Ss, Vs, is_, ts = _factor(w, inp, solar.ROUTE_SUBSPACE)
    if certifies is None:
        assert np.all((ts & 0xFF) == 2)
    else:
        assert np.all((ts & 0xFF) == 1), [hex(x) for x in ts]
        assert np.all(is_ == (0 if certifies else solar.INFO_NOT_CERTIFIED)), is_
        assert np.isfinite(Ss).all() and np.isfinite(Vs).all()
        if certifies:
            assert np.abs(Ss - Sf).max() <= tol * Sf.max()
            for k in users:
                _oracle_check(w, inp, Ss, Vs, k)


def _degenerate_histories(kind, B=3, N=400, d=64):
    """Histories whose Gram matrices have clusters the tridiagonal route cannot separate."""
    rng = np.random.default_rng(7)
    out = []
    for _ in range(B):
        if kind == "rank_deficient":                   # rank 10 < r = 16: six zero singular values
            H = rng.standard_normal((N, 10)) @ rng.standard_normal((10, d))
        else:                                          # sigma = 3, 3, 3, 2, 2, then 1/i: exact multiplicities
            Q, _ = np.linalg.qr(rng.standard_normal((N, 32)))
            P, _ = np.linalg.qr(rng.standard_normal((d, 32)))
            sv = np.array([3, 3, 3, 2, 2] + [1.0 / (i + 1) for i in range(27)])
            H = (Q * sv) @ P.T * 8.0
        out.append(H.astype(np.float32))
    return np.stack(out)


@pytest.mark.parametrize("kind,r", [("rank_deficient", 16), ("repeated", 8)])
def test_clustered_spectra_fall_back_to_the_jacobi_solve(kind, r):
    H = _degenerate_histories(kind)
    B, N, d = H.shape
    Hd = torch.from_numpy(H).cuda()
    ws = solar.alloc_workspace(B, 8, N, d, r, torch.float32)
    out = {}
    for route in (solar.ROUTE_AUTO, solar.ROUTE_TRIDIAG, solar.ROUTE_FULL):
        S = torch.full((B, r), float("nan"), device="cuda")
        V = torch.full((B, d, r), float("nan"), device="cuda")
        info = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        taken = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        solar.gram_partials(Hd, ws)
        solar.eig_from_partials_ex(B, N, d, r, torch.float32, route, S, V, info, taken, ws)
        torch.cuda.synchronize()
        out[route] = (S.cpu().numpy().astype(np.float64), V.cpu().numpy().astype(np.float64),
                      info.cpu().numpy(), taken.cpu().numpy())
    Sa, Va, ia, ta = out[solar.ROUTE_AUTO]
    St, Vt, it, tt = out[solar.ROUTE_TRIDIAG]
    Sf, Vf, if_, tf = out[solar.ROUTE_FULL]
    # AUTO: where the tridiagonal route's certificate fails (reason bits set) the Jacobi solve
    # answers; a cluster that rounding has split may still be certified after a few
    # orthogonalisation passes.  Zero singular values (a six-fold eigenvalue) never are.
    fell_back = (ta & 0xFF) == 2
    assert np.all(fell_back | ((ta & 0xFF) == 3)), [hex(x) for x in ta]
    assert np.all(((ta[fell_back] >> 24) & 0xFF) != 0), [hex(x) for x in ta]
    if kind == "rank_deficient":
        assert np.all(fell_back)
    assert np.all(ia == 0) and np.all(if_ == 0)
    # the tridiagonal route alone writes its result and says so where it is not certified
    assert np.all((tt & 0xFF) == 3)
    assert np.all((it == solar.INFO_NOT_CERTIFIED) == fell_back), (it, ta)
    assert np.isfinite(St).all()
    for k in range(B):
        sv = np.linalg.svd(H[k].astype(np.float64), compute_uv=False)[:r]
        nz = sv > 1e-5 * sv[0]
        # a zero singular value comes out of the Gram matrix as sqrt(rounding error of lambda_1)
        tol = np.where(nz, 2e-5, 1e-3) * sv[0]
        assert np.all(np.abs(Sa[k] - sv) <= tol)
        assert np.all(np.abs(St[k] - sv) <= tol)               # the eigenvalues themselves are fine
        assert np.abs(Va[k].T @ Va[k] - np.eye(r)).max() < 1e-4
        # the kept subspace of the non-zero singular values matches LAPACK's
        _, _, Vt_l = np.linalg.svd(H[k].astype(np.float64), full_matrices=False)
        Vl = Vt_l[:r].T
        Pa = Va[k][:, nz] @ Va[k][:, nz].T
        Pl = Vl[:, nz] @ Vl[:, nz].T
        assert np.abs(Pa - Pl).max() < 1e-4


def test_sweep_cap_reaches_the_caller():
    """A Jacobi solve cut short by a host-chosen sweep cap reports SOLAR_INFO_NOT_CONVERGED."""
    w = wl.CONFIGS["c2"].with_(B=3, N=512, M=8)
    inp = wl.generate(w)
    S, V, info, taken = _factor(w, inp, solar.route_with(solar.ROUTE_FULL, sweep_cap=1))
    assert np.all(info == solar.INFO_NOT_CONVERGED), info
    assert np.all((taken & 0xFF) == 2) and np.all(((taken >> 16) & 0xFF) == 1)
    assert np.isfinite(S).all() and np.isfinite(V).all()
    S, V, info, taken = _factor(w, inp, solar.ROUTE_FULL)
    assert np.all(info == 0)


def test_lost_gram_slice_reaches_the_caller():
    """A Gram CTA whose bounded wait ran out leaves its code in the slice's status word; the
    eigensolver then gives that user NaN factors and SOLAR_INFO_DEVICE_WAIT and leaves the
    other users alone.  The status word is overwritten from the host: no wait runs out here."""
    w = wl.CONFIGS["c2"].with_(B=4, N=2048, M=8)
    inp = wl.generate(w)
    tdt = torch.bfloat16
    H = ph.to_device(inp["H"], w.dtype)
    ws = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, tdt)
    parts = solar.gram_splits(w.B, w.N, w.d, tdt)          # partial matrices per user
    splits = solar.gram_slices(w.B, w.N, w.d, tdt)         # slices (CTAs, status words) per user
    solar.gram_partials(H, ws)
    torch.cuda.synchronize()
    off = (w.B * parts * w.d * w.d * 4 + 255) // 256 * 256
    status = ws[off: off + 4 * w.B * splits].view(torch.int32)
    assert torch.all(status == 0x600D)
    ref = {}
    for poisoned in (False, True):
        if poisoned:
            status[2 * splits + splits - 1] = 0x11          # user 2, last slice
        S = torch.full((w.B, w.r), 7.0, device="cuda")
        V = torch.full((w.B, w.d, w.r), 7.0, device="cuda")
        info = torch.full((w.B,), -1, dtype=torch.int32, device="cuda")
        solar.eig_from_partials_ex(w.B, w.N, w.d, w.r, tdt, solar.ROUTE_AUTO, S, V, info, None, ws)
        torch.cuda.synchronize()
        ref[poisoned] = (S.cpu(), V.cpu(), info.cpu())
    S0, V0, i0 = ref[False]
    S1, V1, i1 = ref[True]
    assert torch.all(i0 == 0)
    assert i1.tolist() == [0, 0, solar.INFO_DEVICE_WAIT, 0]
    assert torch.isnan(S1[2]).all() and torch.isnan(V1[2]).all()
    for k in (0, 1, 3):
        assert torch.equal(S0[k], S1[k]) and torch.equal(V0[k], V1[k])


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
