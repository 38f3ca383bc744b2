"""Pins for the CPU oracle: everything here is fixed by the paper or by mathematics
(closed forms, invariants, a LAPACK routine, brute force, a hand-worked case) and
none of it re-types the oracle's own formulae."""
import math
import os

import numpy as np
import pytest

import oracle as o

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rank_r(rng, N, d, r):
    return rng.standard_normal((N, r)) @ rng.standard_normal((r, d))


def _weights(rng, d):
    return [rng.standard_normal((d, d)) / math.sqrt(d) for _ in range(3)]


def _rel(a, b):
    return float(np.abs(a - b).max() / np.abs(b).max())


# ---- P1: factorization (Eq. 9: U^T U = I_r, H = U Sigma V^T) ---------------------
@pytest.mark.parametrize("N,d,r", [(40, 8, 3), (256, 32, 8), (300, 24, 24)])
def test_factors_orthonormal_and_reconstruct(N, d, r):
    rng = np.random.default_rng(1)
    H = _rank_r(rng, N, d, r)
    s, V, U = o.truncated_svd(H, r)
    assert np.abs(V.T @ V - np.eye(r)).max() < 1e-10
    assert np.abs(U.T @ U - np.eye(r)).max() < 1e-10
    assert np.linalg.norm(H - (U * s) @ V.T) < 1e-10 * np.linalg.norm(H)
    assert np.all(np.diff(s) <= 0) and np.all(s > 0)


def test_eckart_young_residual():
    rng = np.random.default_rng(2)
    H = rng.standard_normal((200, 16))
    sig_all, _, _, _ = o.hestenes_svd(H)
    for r in (1, 5, 15):
        s, V, _ = o.truncated_svd(H, r)
        res = np.linalg.norm(H - H @ V @ V.T) ** 2
        assert abs(res - (sig_all[r:] ** 2).sum()) < 1e-10 * (sig_all ** 2).sum()


# ---- P2: singular values known in closed form ------------------------------------
@pytest.mark.parametrize("decay", [1.0, 1.5])
def test_singular_values_closed_form(decay):
    rng = np.random.default_rng(3)
    N, d = 500, 32
    U0, _ = np.linalg.qr(rng.standard_normal((N, d)))
    V0, _ = np.linalg.qr(rng.standard_normal((d, d)))
    sig = 7.0 * np.arange(1, d + 1) ** (-decay)
    H = (U0 * sig) @ V0.T
    s, V, U = o.truncated_svd(H, 12)
    assert np.abs(s - sig[:12]).max() < 1e-12 * sig[0]
    # vectors equal the generating ones up to sign
    assert np.abs(np.abs(np.sum(V * V0[:, :12], axis=0)) - 1).max() < 1e-10


# ---- LAPACK as an independent library routine ------------------------------------
def test_against_lapack_svd():
    rng = np.random.default_rng(4)
    H = rng.standard_normal((300, 20)) * (np.arange(1, 21) ** -1.0)[None, :]
    s, V, U = o.truncated_svd(H, 7)
    _, sl, Vt = np.linalg.svd(H, full_matrices=False)
    assert np.abs(s - sl[:7]).max() < 1e-11 * sl[0]
    assert np.abs(np.abs(np.sum(V * Vt[:7].T, axis=0)) - 1).max() < 1e-9


# ---- sign gauge --------------------------------------------------------------------
def test_sign_gauge_rule():
    V = np.array([[0.1, -0.9, 0.5], [-0.8, 0.2, -0.5], [0.3, 0.3, 0.4]])
    Vg, flips = o.sign_gauge(V)
    assert list(flips) == [-1.0, -1.0, 1.0]       # third column: tie -> lowest index decides
    assert np.allclose(Vg, V * flips)
    rng = np.random.default_rng(5)
    s, V, _ = o.truncated_svd(rng.standard_normal((50, 6)), 4)
    lead = V[np.argmax(np.abs(V), axis=0), np.arange(4)]
    assert np.all(lead > 0)


# ---- P3: losslessness on rank-<=r matrices (Eq. 10) ------------------------------
@pytest.mark.parametrize("N,d,r,M", [(40, 8, 3, 5), (256, 32, 8, 16)])
def test_lossless_without_softmax(N, d, r, M):
    rng = np.random.default_rng(6)
    H = _rank_r(rng, N, d, r)
    C = rng.standard_normal((M, d)) / math.sqrt(d)
    Wq, Wk, Wv = _weights(rng, d)
    s, V, _ = o.truncated_svd(H, r)
    Key_r, Value_r = o.factor_tokens(s, V, Wk, Wv)
    KtV = (H @ Wk).T @ (H @ Wv)
    assert _rel(Key_r.T @ Value_r, KtV) < 1e-10
    scale = 1 / math.sqrt(d)
    a = o.svd_attention(H, C, Wq, Wk, Wv, r, scale, softmax=False)
    assert _rel(a, o.chain_attention(H, C, Wq, Wk, Wv, scale)) < 1e-10
    assert _rel(a, o.linear_attention(H, C, Wq, Wk, Wv, scale)) < 1e-10


# ---- P4: softmax over positions through the factors == brute force ----------------
def test_factored_exact_equals_full_softmax_attention():
    rng = np.random.default_rng(7)
    N, d, r, M = 256, 32, 8, 16
    H = _rank_r(rng, N, d, r) / math.sqrt(r)
    C = rng.standard_normal((M, d)) / math.sqrt(d)
    Wq, Wk, Wv = _weights(rng, d)
    scale = 1 / math.sqrt(d)
    a = o.factored_exact_attention(H, C, Wq, Wk, Wv, r, scale)
    b = o.softmax_attention(H, C, Wq, Wk, Wv, scale)
    assert _rel(a, b) < 1e-10


def test_softmax_attention_textbook_loops():
    """Brute-force comparator against explicit Python sums (Eq. 6-7)."""
    rng = np.random.default_rng(8)
    N, d, M = 5, 3, 2
    H = rng.standard_normal((N, d)); C = rng.standard_normal((M, d))
    Wq, Wk, Wv = _weights(rng, d)
    got = o.softmax_attention(H, C, Wq, Wk, Wv, 0.5)
    for m in range(M):
        q = [sum(C[m, k] * Wq[k, j] for k in range(d)) for j in range(d)]
        keys = [[sum(H[n, k] * Wk[k, j] for k in range(d)) for j in range(d)] for n in range(N)]
        vals = [[sum(H[n, k] * Wv[k, j] for k in range(d)) for j in range(d)] for n in range(N)]
        sc = [0.5 * sum(q[j] * keys[n][j] for j in range(d)) for n in range(N)]
        z = sum(math.exp(x) for x in sc)
        for j in range(d):
            want = sum(math.exp(sc[n]) / z * vals[n][j] for n in range(N))
            assert abs(got[m, j] - want) < 1e-12


# ---- P5: N = r with orthogonal rows  ==> textbook softmax attention over those tokens
def test_orthogonal_rows_reduce_to_softmax_attention():
    rng = np.random.default_rng(9)
    r, d, M = 6, 16, 9
    Q, _ = np.linalg.qr(rng.standard_normal((d, r)))
    rows = Q.T.copy()
    for i in range(r):                       # make the largest component positive
        if rows[i, np.argmax(np.abs(rows[i]))] < 0:
            rows[i] = -rows[i]
    H = rows * np.array([9.0, 7.0, 5.0, 3.0, 2.0, 1.0])[:, None]
    C = rng.standard_normal((M, d))
    Wq, Wk, Wv = _weights(rng, d)
    a = o.svd_attention(H, C, Wq, Wk, Wv, r, 0.3)
    b = o.softmax_attention(H, C, Wq, Wk, Wv, 0.3)
    assert np.abs(a - b).max() < 1e-12


# ---- P6: r = 1 closed form ---------------------------------------------------------
def test_rank_one_closed_form():
    rng = np.random.default_rng(10)
    N, d, M = 30, 8, 4
    H = rng.standard_normal((N, d))
    C = rng.standard_normal((M, d))
    Wq, Wk, Wv = _weights(rng, d)
    _, sl, Vt = np.linalg.svd(H, full_matrices=False)
    v1 = Vt[0] * (1 if Vt[0][np.argmax(np.abs(Vt[0]))] > 0 else -1)
    row = sl[0] * v1 @ Wv
    out = o.svd_attention(H, C, Wq, Wk, Wv, 1, 0.7)
    assert np.abs(out - row[None, :]).max() < 1e-10
    out2 = o.svd_attention(H, C, Wq, Wk, Wv, 1, 0.7, softmax=False)
    k1 = sl[0] * v1 @ Wk
    want = 0.7 * ((C @ Wq) @ k1)[:, None] * row[None, :]
    assert np.abs(out2 - want).max() < 1e-9


# ---- P7: the output depends on H only through H^T H -------------------------------
def test_invariances():
    rng = np.random.default_rng(11)
    N, d, r, M = 64, 12, 5, 7
    H = rng.standard_normal((N, d)) * (np.arange(1, d + 1) ** -1.0)[None, :]
    C = rng.standard_normal((M, d))
    Wq, Wk, Wv = _weights(rng, d)
    base = o.svd_attention(H, C, Wq, Wk, Wv, r, 0.4)
    perm = rng.permutation(N)
    assert np.abs(o.svd_attention(H[perm], C, Wq, Wk, Wv, r, 0.4) - base).max() < 1e-10
    Hz = np.vstack([H, np.zeros((9, d))])
    assert np.abs(o.svd_attention(Hz, C, Wq, Wk, Wv, r, 0.4) - base).max() < 1e-10
    Qo, _ = np.linalg.qr(rng.standard_normal((N, N)))
    assert np.abs(o.svd_attention(Qo @ H, C, Wq, Wk, Wv, r, 0.4) - base).max() < 1e-10
    R = np.linalg.qr(H, mode="r")
    assert np.abs(o.svd_attention(R, C, Wq, Wk, Wv, r, 0.4) - base).max() < 1e-10
    s1, V1, _ = o.truncated_svd(H, r)
    s2, V2, _ = o.truncated_svd(np.vstack([H, H]), r)
    assert np.abs(s2 - math.sqrt(2) * s1).max() < 1e-11 and np.abs(V1 - V2).max() < 1e-10


# ---- P8b: the power iteration of Algorithm 1 on a full-rank history -----------------------
def test_randomized_svd_power_steps_contract_the_subspace_error():
    """On a full-rank H with singular values sigma_i = 4 * 2^-i the range of H^T(H Omega) loses
    the discarded directions by (sigma_{r+1} / sigma_r)^2 = 1/4 per power step (subspace
    iteration with H^T H): the tangent of the largest principal angle between R and the true
    top-r right subspace (LAPACK) must fall by that factor from n_iter to n_iter + 1.  A power
    loop that does not run, or that applies anything but H^T H, leaves the band."""
    rng = np.random.default_rng(21)
    N, d, r = 80, 12, 4
    U0, _ = np.linalg.qr(rng.standard_normal((N, d)))
    V0, _ = np.linalg.qr(rng.standard_normal((d, d)))
    sig = 4.0 * 0.5 ** np.arange(d)
    H = (U0 * sig) @ V0.T
    Vt = np.linalg.svd(H, full_matrices=False)[2]
    Vtop, Vrest = Vt[:r].T, Vt[r:].T
    Omega = rng.standard_normal((d, r))
    tans = []
    for n_iter in (0, 1, 2, 3):
        _, R = o.randomized_svd(H, r, n_iter, Omega)
        Qr, _ = np.linalg.qr(R)                          # R is orthonormal already; this only guards the test
        # tan of the largest principal angle: largest singular value of (Vrest^T Q)(Vtop^T Q)^-1
        tans.append(np.linalg.svd((Vrest.T @ Qr) @ np.linalg.inv(Vtop.T @ Qr), compute_uv=False)[0])
    q2 = (sig[r] / sig[r - 1]) ** 2
    assert tans[0] > 1e-3                                # no power step: a visibly wrong subspace
    for a, b in zip(tans[:-1], tans[1:]):
        assert q2 / 2 <= b / a <= q2 * 2, (tans, q2)
    assert tans[1] < 0.6 * tans[0]                       # one step differs measurably from none


# ---- P8: Algorithm 1 reaches the same factors on rank-r input ----------------------
@pytest.mark.parametrize("n_iter", [0, 2])
def test_randomized_svd_matches_on_low_rank(n_iter):
    rng = np.random.default_rng(12)
    N, d, r, M = 120, 20, 6, 5
    H = _rank_r(rng, N, d, r) / math.sqrt(r)
    s, V, _ = o.truncated_svd(H, r)
    s2, R = o.randomized_svd(H, r, n_iter, rng.standard_normal((d, r)))
    assert np.abs(s - s2).max() < 1e-8 * s[0]
    assert np.abs(V - R).max() < 1e-8
    C = rng.standard_normal((M, d))
    Wq, Wk, Wv = _weights(rng, d)
    a = o.svd_attention_from_factors(C, s, V, Wq, Wk, Wv, 0.2)
    b = o.svd_attention_from_factors(C, s2, R, Wq, Wk, Wv, 0.2)
    assert _rel(a, b) < 1e-8


def test_householder_basis_is_orthonormal_and_spans():
    rng = np.random.default_rng(13)
    Y = rng.standard_normal((30, 5))
    Q = o.householder_qr_basis(Y)
    assert np.abs(Q.T @ Q - np.eye(5)).max() < 1e-13
    assert np.abs(Q @ (Q.T @ Y) - Y).max() < 1e-12


# ---- P9: tiny inputs against the 2x2 characteristic polynomial ---------------------
def test_tiny_two_by_two_brute_force():
    H = np.array([[1.0, 2.0], [0.5, -1.0], [3.0, 0.25], [-2.0, 1.0]])
    G = H.T @ H
    tr, det = G[0, 0] + G[1, 1], G[0, 0] * G[1, 1] - G[0, 1] ** 2
    lam1 = tr / 2 + math.sqrt(tr * tr / 4 - det)
    lam2 = tr / 2 - math.sqrt(tr * tr / 4 - det)
    v1 = np.array([G[0, 1], lam1 - G[0, 0]]); v1 /= np.linalg.norm(v1)
    if v1[np.argmax(np.abs(v1))] < 0:
        v1 = -v1
    s, V, _ = o.truncated_svd(H, 1)
    assert abs(s[0] - math.sqrt(lam1)) < 1e-13 and np.abs(V[:, 0] - v1).max() < 1e-13
    s2, V2, _ = o.truncated_svd(H, 2)
    assert abs(s2[1] - math.sqrt(lam2)) < 1e-13
    # r=2 attention by explicit sums
    v2 = np.array([-v1[1], v1[0]])
    if v2[np.argmax(np.abs(v2))] < 0:
        v2 = -v2
    Wq = np.array([[1.0, 0.5], [0.0, 1.0]]); Wk = np.array([[0.5, 0.0], [1.0, 1.0]])
    Wv = np.array([[1.0, -1.0], [2.0, 0.0]]); c = np.array([[0.3, -0.7]])
    q = c @ Wq
    toks = [math.sqrt(lam1) * v1, math.sqrt(lam2) * v2]
    sc = [0.9 * float(q[0] @ (t @ Wk)) for t in toks]
    w = [math.exp(x) / sum(math.exp(y) for y in sc) for x in sc]
    want = sum(wi * (t @ Wv) for wi, t in zip(w, toks))
    got = o.svd_attention(H, c, Wq, Wk, Wv, 2, 0.9)
    assert np.abs(got[0] - want).max() < 1e-12


# ---- hand-worked golden case -------------------------------------------------------
def test_golden_diagonal_case():
    rows = np.loadtxt(os.path.join(GOLD, "diag2x2_svd_attention.txt"))
    H = np.array([[2.0, 0.0], [0.0, 1.0]])
    I = np.eye(2)
    out = o.svd_attention(H, rows[:, :2], I, I, I, 2, 1.0)
    assert np.abs(out - rows[:, 2:]).max() < 1e-14


# ---- softmax is a genuine part of the operator: SVD-Attention != full attention ----
def test_softmax_over_tokens_differs_from_softmax_over_positions():
    rng = np.random.default_rng(14)
    H = _rank_r(rng, 40, 8, 3)
    C = rng.standard_normal((4, 8)); Wq, Wk, Wv = _weights(rng, 8)
    a = o.svd_attention(H, C, Wq, Wk, Wv, 3, 0.35)
    b = o.softmax_attention(H, C, Wq, Wk, Wv, 0.35)
    assert np.abs(a - b).max() > 1e-3
    P = o.row_softmax(rng.standard_normal((5, 7)))
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-15 and (P > 0).all()


def test_rank_deficient_input_gives_zero_tokens():
    """rank(H) < r: the surplus tokens have sigma = 0 and still take softmax weight exp(0 - max)."""
    rng = np.random.default_rng(15)
    H = _rank_r(rng, 50, 10, 2)
    s, V, _ = o.truncated_svd(H, 4)
    assert s[2] == 0.0 and s[3] == 0.0 and s[1] > 0
    C = rng.standard_normal((3, 10)); Wq, Wk, Wv = _weights(rng, 10)
    out = o.svd_attention(H, C, Wq, Wk, Wv, 4, 0.3)
    Key_r, Value_r = o.factor_tokens(s[:2], V[:, :2], Wk, Wv)
    S = 0.3 * (C @ Wq) @ Key_r.T
    Sfull = np.hstack([S, np.zeros((3, 2))])
    E = np.exp(Sfull - Sfull.max(axis=1, keepdims=True))
    want = (E / E.sum(axis=1, keepdims=True))[:, :2] @ Value_r
    assert np.abs(out - want).max() < 1e-10


def test_max_rel_err_rows():
    a = np.array([[1.0, 2.0], [0.0, 4.0]]); b = np.array([[1.0, 2.2], [0.0, 4.0]])
    assert abs(o.max_rel_err_rows(b, a) - 0.1) < 1e-12
