"""Pins of the backward oracle (oracle/svd_attention_backward.py) against what the
mathematics fixes: central finite differences of the forward oracle, textbook closed
forms (gradient of the nuclear norm and of the squared Frobenius norm of the rank-r
part), and directional derivatives inside the truncated subspace (the setting of
Eq. 13-15).  A wrong sign, a transposed factor, a dropped 2 or sigma_i for sigma_j in
Eq. 15 fails the finite-difference cases; the printed index order of the appendix is
shown to fail them."""
import numpy as np
import pytest

import oracle as o
from oracle import svd_attention_backward as ob


def _rng(seed):
    return np.random.default_rng(seed)


def _fd(f, x, h=1e-6):
    """Central finite differences of the scalar f at x, element by element."""
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        xp = x.copy(); xp[i] += h
        xm = x.copy(); xm[i] -= h
        g[i] = (f(xp) - f(xm)) / (2 * h)
    return g


def _problem(seed, N, d, r, M):
    g = _rng(seed)
    H = g.standard_normal((N, d))
    C = g.standard_normal((M, d)) / np.sqrt(d)
    Wq, Wk, Wv = (g.standard_normal((d, d)) / np.sqrt(d) for _ in range(3))
    R = g.standard_normal((M, d))
    return H, C, Wq, Wk, Wv, R, 1.0 / np.sqrt(d)


@pytest.mark.parametrize("softmax", [True, False])
def test_attention_part_matches_finite_differences(softmax):
    H, C, Wq, Wk, Wv, R, scale = _problem(1, 12, 5, 3, 6)
    s, V, _ = o.truncated_svd(H, 3)
    g = ob.svd_attention_backward(C, s, V, Wq, Wk, Wv, scale, R, softmax)
    loss = lambda **kw: float((o.svd_attention_from_factors(
        kw.get("C", C), kw.get("s", s), kw.get("V", V), kw.get("Wq", Wq), kw.get("Wk", Wk),
        kw.get("Wv", Wv), scale, softmax) * R).sum())
    for name, x in (("C", C), ("Wq", Wq), ("Wk", Wk), ("Wv", Wv), ("s", s), ("V", V)):
        fd = _fd(lambda z: loss(**{name: z}), x)
        got = g["d" + name]
        assert np.abs(got - fd).max() <= 1e-7 * max(1.0, np.abs(fd).max()), name


def test_singular_value_losses_have_their_textbook_gradients():
    g = _rng(2)
    H = g.standard_normal((10, 6))
    r = 4
    s, V, U = o.truncated_svd(H, r)
    zero = np.zeros_like(V)
    # d(sum of the kept singular values)/dH = U V^T
    assert np.abs(ob.svd_backward(H, s, V, np.ones(r), zero) - U @ V.T).max() < 1e-12
    # d(1/2 sum sigma_i^2)/dH = U Sigma V^T, the rank-r part of H
    assert np.abs(ob.svd_backward(H, s, V, s, zero) - (U * s) @ V.T).max() < 1e-12
    # and U = H V Sigma^-1 is the left factor of the SVD
    assert np.abs(ob.left_factor(H, s, V) - U).max() < 1e-12


@pytest.mark.parametrize("softmax", [True, False])
def test_full_gradient_matches_finite_differences_when_nothing_is_truncated(softmax):
    # r = d: the subspace of Eq. 13-15 is the whole space and the formula is the exact gradient
    N, d, M = 9, 4, 5
    H, C, Wq, Wk, Wv, R, scale = _problem(3, N, d, d, M)
    s, V, _ = o.truncated_svd(H, d)
    g = ob.svd_attention_backward_full(H, C, s, V, Wq, Wk, Wv, scale, R, softmax)
    loss = lambda X: float((o.svd_attention(X, C, Wq, Wk, Wv, d, scale, softmax) * R).sum())
    fd = _fd(loss, H)
    assert np.abs(g["dH"] - fd).max() <= 2e-6 * np.abs(fd).max()


def test_v_only_loss_matches_finite_differences():
    g = _rng(4)
    N, d = 8, 4
    H = g.standard_normal((N, d))
    R = g.standard_normal((d, d))
    s, V, _ = o.truncated_svd(H, d)
    loss = lambda X: float((o.truncated_svd(X, d)[1] * R).sum())
    fd = _fd(loss, H)
    got = ob.svd_backward(H, s, V, np.zeros(d), R)
    assert np.abs(got - fd).max() <= 2e-6 * np.abs(fd).max()
    # the appendix's printed index order (V^T Vbar in the Hadamard product) has the wrong sign
    U = ob.left_factor(H, s, V)
    X = ob.svd_grad_F(s) * (V.T @ R)
    printed = U @ (s[:, None] * (X + X.T)) @ V.T
    assert np.abs(printed + fd).max() <= 2e-6 * np.abs(fd).max()      # exactly the negative
    assert np.abs(printed - fd).max() > 0.5 * np.abs(fd).max()


def test_truncated_case_inside_the_subspace():
    # exactly rank-r history, d > r: perturbations U X V^T stay inside the truncated subspace,
    # where Eq. 15 is the gradient:  d/dt L(H + t U X V^T) = <core, X>
    N, d, r, M = 14, 6, 3, 5
    g = _rng(5)
    H = g.standard_normal((N, r)) @ g.standard_normal((r, d))
    _, C, Wq, Wk, Wv, R, scale = _problem(6, N, d, r, M)
    s, V, U = o.truncated_svd(H, r)
    grads = ob.svd_attention_backward(C, s, V, Wq, Wk, Wv, scale, R, True)
    core = ob.svd_grad_core(s, V, grads["ds"], grads["dV"])
    loss = lambda X: float((o.svd_attention(X, C, Wq, Wk, Wv, r, scale, True) * R).sum())
    for k in range(4):
        X = g.standard_normal((r, r))
        D = U @ X @ V.T
        t = 1e-6
        fd = (loss(H + t * D) - loss(H - t * D)) / (2 * t)
        assert abs(fd - float((core * X).sum())) <= 2e-6 * max(1.0, abs(fd)), k
    # and dH itself lies in that subspace: U U^T dH V V^T = dH
    dH = ob.svd_backward(H, s, V, grads["ds"], grads["dV"])
    assert np.abs(U @ (U.T @ dH @ V) @ V.T - dH).max() < 1e-12 * max(1.0, np.abs(dH).max())


def test_diagonal_2x2_against_first_order_perturbation_theory():
    """H = diag(a, b), a > b > 0: U = V = I.  Textbook perturbation of the eigenvectors of H^T H:
    adding eps at (1,2) turns v1 by +a eps/(a^2-b^2) towards e2 (and v2 by the opposite), adding
    eps at (2,1) turns it by +b eps/(a^2-b^2).  So for a loss with dL/dV = R and dL/dSigma = g:
      dL/dH = [[g1, a (R21 - R12)/(a^2-b^2)], [b (R21 - R12)/(a^2-b^2), g2]]."""
    a, b = 3.0, 2.0
    H = np.diag([a, b])
    s, V = np.array([a, b]), np.eye(2)
    R = np.array([[0.3, -1.1], [0.7, 0.4]])
    g = np.array([0.5, -0.25])
    k = (R[1, 0] - R[0, 1]) / (a * a - b * b)
    want = np.array([[g[0], a * k], [b * k, g[1]]])
    got = ob.svd_backward(H, s, V, g, R)
    assert np.abs(got - want).max() < 1e-14
    # the same numbers, worked by hand, in the golden file
    import os
    gold = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "diag2x2_svd_backward.txt"))
    assert np.abs(got - gold).max() < 1e-14


def test_F_and_its_stabilisation():
    s = np.array([3.0, 2.0, 1.0])
    F = ob.svd_grad_F(s)
    assert F[0, 1] == pytest.approx(1.0 / (9.0 - 4.0)) and F[1, 0] == pytest.approx(-0.2)
    assert F[0, 2] == pytest.approx(1.0 / 8.0) and np.all(np.diag(F) == 0.0)
    assert np.abs(F + F.T).max() == 0.0                       # skew-symmetric
    Fe = ob.svd_grad_F(s, eps_rel=0.1)                        # eps = 0.9
    assert Fe[0, 1] == pytest.approx(5.0 / (25.0 + 0.81))
    assert np.abs(Fe).max() <= 1.0 / (2 * 0.9) + 1e-15        # |D/(D^2+eps^2)| <= 1/(2 eps)
    # equal singular values: finite with eps, zero without
    t = np.array([2.0, 2.0, 1.0])
    assert ob.svd_grad_F(t)[0, 1] == 0.0 and np.isfinite(ob.svd_grad_F(t, 1e-3)).all()


def test_zero_singular_value_gives_no_gradient_through_its_direction():
    g = _rng(7)
    N, d, r = 10, 5, 3
    H = g.standard_normal((N, 2)) @ g.standard_normal((2, d))       # rank 2 < r
    s, V, _ = o.truncated_svd(H, r)
    assert s[2] < 1e-12
    s = s.copy(); s[2] = 0.0
    dH = ob.svd_backward(H, s, V, np.ones(r), g.standard_normal((d, r)), eps_rel=1e-6)
    assert np.isfinite(dH).all()
