"""CPU oracle for the SVD-Attention forward pass (SOLAR, arxiv 2603.02561).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, double-precision
statement of what the hot path computes.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it; the CUDA library never does,
and nothing here imports the CUDA package.  No blocking, fusion or reordering
beyond what the cited passages state.

Notation (paper -> here): N_L -> N (history length), N_C -> M (candidates),
d (embedding width), r (rank).  One user at a time; batches are Python loops.

Pin status: every function below is pinned by tests/test_oracle_pins.py
(closed forms, invariants, a LAPACK SVD, brute force, a hand-computed golden
case).  Two conventions are this implementation's own and are "parity unpinned" against
the authors' unpublished system: the sign gauge of V (`sign_gauge`) and the
value of `scale` (an explicit argument; the paper prints no 1/sqrt(d)).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Step 1 -- rank-r truncated SVD, H = U Sigma V^T  (Section 4.1, Eq. 9)
# --------------------------------------------------------------------------
def hestenes_svd(H, tol=1e-15, max_sweeps=60):
    """Thin SVD of an N x d matrix by one-sided (Hestenes) Jacobi rotations.

    Returns (sigma[d] descending, V[d,d], U[N,d], sweeps).  Columns of U that
    belong to a zero singular value are left as zero vectors.

    Cyclic sweeps over all column pairs (p<q); a pair is rotated when
    |h_p.h_q| > tol*|h_p||h_q|, with the rotation that makes the two columns
    orthogonal.  Works on H itself (never on H^T H), so small singular values
    keep their relative accuracy.
    """
    H = np.asarray(H, dtype=F64)
    N, d = H.shape
    A = np.ascontiguousarray(H.T)          # A[j] is column j of the working matrix
    V = np.eye(d, dtype=F64)               # V[j] is column j of V (stored as rows)
    # Columns whose norm is below eps*|H|_F are rounding residue of a rank
    # deficient H: they are treated as exactly zero (sigma = 0).
    floor = (np.finfo(F64).eps ** 2) * float(np.einsum("ij,ij->", A, A))
    sweeps = 0
    for sweeps in range(1, max_sweeps + 1):
        rotated = False
        for p in range(d - 1):
            for q in range(p + 1, d):
                alpha = float(A[p] @ A[p])
                beta = float(A[q] @ A[q])
                gamma = float(A[p] @ A[q])
                if alpha <= floor or beta <= floor:
                    continue
                if abs(gamma) <= tol * np.sqrt(alpha * beta):
                    continue
                rotated = True
                zeta = (beta - alpha) / (2.0 * gamma)
                t = np.copysign(1.0, zeta) / (abs(zeta) + np.sqrt(1.0 + zeta * zeta))
                c = 1.0 / np.sqrt(1.0 + t * t)
                s = c * t
                ap = A[p].copy()
                A[p] = c * ap - s * A[q]
                A[q] = s * ap + c * A[q]
                vp = V[p].copy()
                V[p] = c * vp - s * V[q]
                V[q] = s * vp + c * V[q]
        if not rotated:
            break
    sq = np.einsum("ij,ij->i", A, A)
    sigma = np.sqrt(np.where(sq > floor, sq, 0.0))
    order = np.argsort(-sigma, kind="stable")
    sigma = sigma[order]
    A = A[order]
    V = V[order]
    U = np.zeros((N, d), dtype=F64)
    nz = sigma > 0.0
    U[:, nz] = (A[nz] / sigma[nz, None]).T
    return sigma, np.ascontiguousarray(V.T), U, sweeps


def sign_gauge(V):
    """Fix the sign of each right singular vector (column of V[d,r]).

    Convention of this implementation (the paper is silent and the softmax over the r
    factor-tokens is NOT invariant to v_i -> -v_i): the component of largest
    magnitude is made positive; ties go to the lowest index.  Returns
    (V_fixed, flips[r]) with flips in {+1,-1} such that V_fixed = V * flips.
    """
    V = np.asarray(V, dtype=F64)
    idx = np.argmax(np.abs(V), axis=0)          # first maximum = lowest index
    lead = V[idx, np.arange(V.shape[1])]
    flips = np.where(lead < 0.0, -1.0, 1.0)
    return V * flips[None, :], flips


def truncated_svd(H, r):
    """Rank-r truncated SVD (Eq. 9): s[r] descending, V[d,r] gauge-fixed, U[N,r].

    U's columns carry the same flips as V's, so H ~= U diag(s) V^T still holds.
    """
    sigma, V, U, _ = hestenes_svd(H)
    Vr, flips = sign_gauge(V[:, :r])
    return sigma[:r].copy(), Vr, U[:, :r] * flips[None, :]


# --------------------------------------------------------------------------
# Steps 2-6 -- SVD-Attention  (Eq. 11, Eq. 12)
# --------------------------------------------------------------------------
def factor_tokens(s, V, Wk, Wv):
    """Key_r = (V Sigma)^T W_K and Value_r = (V Sigma)^T W_V, both r x d (Eq. 11)."""
    VS = np.asarray(V, F64) * np.asarray(s, F64)[None, :]       # V Sigma, d x r
    return VS.T @ np.asarray(Wk, F64), VS.T @ np.asarray(Wv, F64)


def row_softmax(S):
    """Row-stochastic softmax with max subtraction."""
    S = S - S.max(axis=1, keepdims=True)
    E = np.exp(S)
    return E / E.sum(axis=1, keepdims=True)


def svd_attention_from_factors(C, s, V, Wq, Wk, Wv, scale, softmax=True):
    """Attn_SVD = MatMul(MatMul(Query, Key_r^T), Value_r)  (Eq. 12).

    Query = C W_Q (Eq. 11).  The softmax (kept by the method, Section 3 closing
    remark and Section 6) acts on the M x r matrix scale*Query*Key_r^T, row by
    row over the r factor-tokens.  softmax=False is the "SVD-Attn without
    Softmax" row of Table 4: scale*Query*Key_r^T*Value_r.
    """
    Query = np.asarray(C, F64) @ np.asarray(Wq, F64)
    Key_r, Value_r = factor_tokens(s, V, Wk, Wv)
    S = scale * (Query @ Key_r.T)
    P = row_softmax(S) if softmax else S
    return P @ Value_r


def svd_attention(H, C, Wq, Wk, Wv, r, scale, softmax=True, flips=None):
    """Whole forward for one user: truncated SVD of H, then Eq. 11-12.

    `flips[r]` (+1/-1), when given, is applied on top of the gauge: used by the
    parity harness where a vector's two largest components tie within rounding
    and either sign is a valid reading of the gauge.
    """
    s, V, _ = truncated_svd(H, r)
    if flips is not None:
        V = V * np.asarray(flips, F64)[None, :]
    return svd_attention_from_factors(C, s, V, Wq, Wk, Wv, scale, softmax)


# --------------------------------------------------------------------------
# Comparators
# --------------------------------------------------------------------------
def softmax_attention(H, C, Wq, Wk, Wv, scale):
    """Brute-force target attention, softmax over the N positions (Eq. 6-7)."""
    Query = np.asarray(C, F64) @ np.asarray(Wq, F64)
    Key = np.asarray(H, F64) @ np.asarray(Wk, F64)
    Value = np.asarray(H, F64) @ np.asarray(Wv, F64)
    return row_softmax(scale * (Query @ Key.T)) @ Value


def chain_attention(H, C, Wq, Wk, Wv, scale):
    """Softmax-free chain scale*(Query Key^T) Value in the order of Eq. 7."""
    Query = np.asarray(C, F64) @ np.asarray(Wq, F64)
    Key = np.asarray(H, F64) @ np.asarray(Wk, F64)
    Value = np.asarray(H, F64) @ np.asarray(Wv, F64)
    return (scale * (Query @ Key.T)) @ Value


def linear_attention(H, C, Wq, Wk, Wv, scale):
    """Attn_lin = MatMul(Query, MatMul(Key^T, Value)), times scale (Eq. 8)."""
    Query = np.asarray(C, F64) @ np.asarray(Wq, F64)
    Key = np.asarray(H, F64) @ np.asarray(Wk, F64)
    Value = np.asarray(H, F64) @ np.asarray(Wv, F64)
    return scale * (Query @ (Key.T @ Value))


def factored_exact_attention(H, C, Wq, Wk, Wv, r, scale):
    """Softmax over the N positions evaluated through the rank-r factors.

    NOT the paper's operator (which eliminates U, Eq. 10): scores are
    (C W_Q W_K^T V)(U Sigma)^T and values are (U Sigma)(V^T W_V).  On a matrix
    of rank <= r it equals `softmax_attention`; kept as the comparator for
    which "equal to full softmax attention on rank-r inputs" holds literally.
    """
    s, V, U = truncated_svd(H, r)
    US = U * s[None, :]
    Qp = (np.asarray(C, F64) @ np.asarray(Wq, F64)) @ (np.asarray(Wk, F64).T @ V)
    return (row_softmax(scale * (Qp @ US.T)) @ US) @ (V.T @ np.asarray(Wv, F64))


def householder_qr_basis(Y):
    """Orthonormal basis Q[N,k] of the columns of Y[N,k] by Householder QR."""
    Y = np.array(Y, dtype=F64)
    N, k = Y.shape
    vs = []
    for j in range(k):
        x = Y[j:, j].copy()
        nx = np.linalg.norm(x)
        v = x
        if nx > 0.0:
            v[0] += np.copysign(nx, x[0])
            v = v / np.linalg.norm(v)
            Y[j:, j:] -= 2.0 * np.outer(v, v @ Y[j:, j:])
        vs.append(v)
    Q = np.zeros((N, k), dtype=F64)
    Q[:k, :k] = np.eye(k)
    for j in reversed(range(k)):
        v = vs[j]
        Q[j:, :] -= 2.0 * np.outer(v, v @ Q[j:, :])
    return Q


def randomized_svd(H, r, n_iter, Omega):
    """Algorithm 1 (randomized SVD with power iteration), steps in its order.

    `Omega[d,r]` is the Gaussian test matrix, passed in (the method's random
    draw is an input).  Returns (s[r], R[d,r]); R is gauge-fixed like V.
    """
    H = np.asarray(H, F64)
    Om = np.asarray(Omega, F64).copy()
    for _ in range(n_iter):
        Om = H.T @ (H @ Om)                     # power iteration
    Q = householder_qr_basis(H @ Om)            # basis of H Omega
    Bm = Q.T @ H                                # r x d, = U_S S R^T
    # SVD of the transpose (d x r, tall): its left vectors are R, its right
    # vectors are U_S.
    sig, _U_S, R, _ = hestenes_svd(Bm.T)
    Rg, _ = sign_gauge(R[:, :r])
    return sig[:r].copy(), Rg


# --------------------------------------------------------------------------
# Error measure used by the parity tests
# --------------------------------------------------------------------------
def max_rel_err_rows(O, O_ref):
    """max over rows m of |O[m]-O_ref[m]|_inf / |O_ref[m]|_inf."""
    O = np.asarray(O, F64)
    O_ref = np.asarray(O_ref, F64)
    num = np.abs(O - O_ref).max(axis=-1)
    den = np.abs(O_ref).max(axis=-1)
    den = np.where(den > 0.0, den, 1.0)
    return float((num / den).max())
