"""CPU oracle for the backward pass of SVD-Attention (SOLAR, arxiv 2603.02561).

TEST INFRASTRUCTURE ONLY, like svd_attention.py: plain numpy in double precision, one
user at a time, imported by the tests, the smoke check and the benchmark's CPU legs and
by nothing else.

Two parts:
  * `svd_backward`: the gradient of the truncated SVD with U absent from the forward pass
    (Eq. 13-15 and the appendix that derives them), evaluated in the paper's order:
    U = H V Sigma^-1, the r x r matrix of Eq. 15, then U [.] V^T.
  * `svd_attention_backward`: the chain rule through Eq. 11-12 (projections, scores,
    softmax over the r factor tokens, weighted sum).  The paper prints no formulas for
    this part; it is the plain derivative of the forward definition.

Reading of Eq. 15 (the printed derivation is at odds with itself).  The appendix solves
    (Omega_V)_ij = (sigma_i dP_ij + sigma_j dP_ji) / (sigma_j^2 - sigma_i^2)
and then expands Tr(Vbar^T dV) = Tr((V^T Vbar)^T Omega_V) as sum_ij P_ji (Omega_V)_ij with
P = V^T Vbar.  The trace of A^T B is sum_ij A_ij B_ij, so the sum is over P_ij (Omega_V)_ij;
Omega_V being skew-symmetric, the printed index order flips the sign of the whole
off-diagonal term.  With the index order corrected the result is
    G_ij = sigma_i F_ij (P_ji - P_ij),   F_ij = 1 / (sigma_i^2 - sigma_j^2)   (Eq. 14 as printed),
that is Eq. 15 with the Hadamard factor Vbar^T V in place of V^T Vbar.  Finite differences
(tests/test_oracle_backward_pins.py) fix this sign: the printed one fails them.

Stabilisation of F (the paper gives none): F_ij = D / (D^2 + eps^2) with
D = sigma_i^2 - sigma_j^2 and eps = eps_rel * sigma_1^2; eps_rel = 0 is Eq. 14 itself
(and F_ij = 0 where D = 0).  This convention is this implementation's own: "parity unpinned"
against the authors' system for eps_rel > 0; for eps_rel = 0 everything here is pinned.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def svd_grad_F(s, eps_rel=0.0):
    """F of Eq. 14, r x r, zero diagonal, with the stabilisation described in the header."""
    s = np.asarray(s, F64)
    s2 = s * s
    D = s2[:, None] - s2[None, :]
    eps = eps_rel * (s2.max() if s2.size else 0.0)
    den = D * D + eps * eps
    F = np.where(den > 0.0, D / np.where(den > 0.0, den, 1.0), 0.0)
    np.fill_diagonal(F, 0.0)
    return F


def svd_grad_core(s, V, ds, dV, eps_rel=0.0):
    """The r x r matrix in the brackets of Eq. 15: diag(ds) + 2 Sigma sym(F o (Vbar^T V))."""
    s = np.asarray(s, F64)
    Pt = np.asarray(dV, F64).T @ np.asarray(V, F64)        # Vbar^T V  (see the header)
    X = svd_grad_F(s, eps_rel) * Pt
    return np.diag(np.asarray(ds, F64)) + s[:, None] * (X + X.T)


def left_factor(H, s, V):
    """U = H V Sigma^-1 (Eq. 9 solved for U); a column with sigma = 0 is a zero column."""
    s = np.asarray(s, F64)
    inv = np.where(s > 0.0, 1.0 / np.where(s > 0.0, s, 1.0), 0.0)
    return (np.asarray(H, F64) @ np.asarray(V, F64)) * inv[None, :]


def svd_backward(H, s, V, ds, dV, eps_rel=0.0):
    """dL/dH of Eq. 15 for one user: U [diag(ds) + 2 Sigma sym(F o (Vbar^T V))] V^T.

    H[N,d]; s[r], V[d,r] from the truncated SVD; ds[r] = dL/dSigma, dV[d,r] = dL/dV.
    """
    U = left_factor(H, s, V)
    return U @ svd_grad_core(s, V, ds, dV, eps_rel) @ np.asarray(V, F64).T


def svd_attention_backward(C, s, V, Wq, Wk, Wv, scale, dO, softmax=True):
    """Gradients of L through Eq. 11-12 given dO = dL/dO, for one user.

    Returns a dict: dC[M,d], dWq, dWk, dWv [d,d] (this user's contribution), ds[r], dV[d,r].
    """
    C = np.asarray(C, F64); s = np.asarray(s, F64); V = np.asarray(V, F64)
    Wq = np.asarray(Wq, F64); Wk = np.asarray(Wk, F64); Wv = np.asarray(Wv, F64)
    dO = np.asarray(dO, F64)
    A = (V * s[None, :]).T                     # (V Sigma)^T, r x d
    Key_r, Value_r = A @ Wk, A @ Wv            # Eq. 11
    Query = C @ Wq
    S = scale * (Query @ Key_r.T)
    if softmax:
        E = np.exp(S - S.max(axis=1, keepdims=True))
        P = E / E.sum(axis=1, keepdims=True)
    else:
        P = S
    # O = P Value_r
    dValue = P.T @ dO
    dP = dO @ Value_r.T
    dS = P * (dP - (P * dP).sum(axis=1, keepdims=True)) if softmax else dP
    # S = scale Query Key_r^T
    dQuery = scale * (dS @ Key_r)
    dKey = scale * (dS.T @ Query)
    # Query = C W_Q
    dC = dQuery @ Wq.T
    dWq = C.T @ dQuery
    # Key_r = A W_K, Value_r = A W_V
    dA = dKey @ Wk.T + dValue @ Wv.T
    dWk = A.T @ dKey
    dWv = A.T @ dValue
    # A = Sigma V^T
    ds = (dA * V.T).sum(axis=1)
    dV = dA.T * s[None, :]
    return {"dC": dC, "dWq": dWq, "dWk": dWk, "dWv": dWv, "ds": ds, "dV": dV}


def svd_attention_backward_full(H, C, s, V, Wq, Wk, Wv, scale, dO, softmax=True, eps_rel=0.0):
    """Both parts for one user: the dict of `svd_attention_backward` plus dH (Eq. 15)."""
    g = svd_attention_backward(C, s, V, Wq, Wk, Wv, scale, dO, softmax)
    g["dH"] = svd_backward(H, s, V, g["ds"], g["dV"], eps_rel)
    return g
