"""The default eigensolver route on randomly drawn shapes and spectra (seeded): whatever route a
user ends up on -- tridiagonal, or the Jacobi solve after a failed certificate or a small gap --
the singular values, the orthonormality of V and the residual against H^T H must hold, and info
must be clean.  The reference is the oracle's one-sided Jacobi SVD of H itself (Eq. 9)."""
import numpy as np
import pytest
import torch

import oracle as o
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu

KINDS = ["lowrank", "lowrank_noise", "power", "geometric", "flat", "cluster", "deficient"]


def _spectrum(kind, k, r, d, rng):
    i = np.arange(1, k + 1, dtype=np.float64)
    if kind == "lowrank":
        return np.where(i <= r, 1.0 / i, 0.0)
    if kind == "lowrank_noise":
        return np.where(i <= r, 1.0 / i, 1e-3 / np.sqrt(d) * (1 + 0.1 * rng.random(k)))
    if kind == "power":
        return i ** -float(rng.uniform(0.5, 2.0))
    if kind == "geometric":
        return float(rng.uniform(0.7, 0.95)) ** i
    if kind == "flat":
        return np.sort(1.0 + 0.3 * rng.random(k))[::-1]
    if kind == "cluster":                    # three singular values equal to 1e-7: no unique vectors there
        s = 1.0 / i
        s[1:4] = s[1] * (1 + 1e-7 * np.arange(3))
        return np.sort(s)[::-1]
    rk = max(1, r // 2)                      # rank(H) < r
    return np.where(i <= rk, 1.0 / i, 0.0)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_and_spectra(seed):
    rng = np.random.default_rng(seed)
    seen = set()
    for case in range(24):
        d = int(rng.choice([32, 64, 64, 128]))
        dtype = "f32" if (d == 32 or rng.random() < 0.25) else "bf16"
        N = max(2, int(rng.integers(1, 6)) * int(rng.choice([7, 64, 128])) + int(rng.integers(0, 5)))
        r = int(rng.integers(1, min(d, 64, N) + 1))
        B = int(rng.integers(1, 4))
        kind = KINDS[int(rng.integers(len(KINDS)))]
        k = min(N, d)
        H = np.empty((B, N, d), np.float32)
        for b in range(B):
            U, _ = np.linalg.qr(rng.standard_normal((N, k)))
            Vq, _ = np.linalg.qr(rng.standard_normal((d, k)))
            H[b] = ((U * _spectrum(kind, k, r, d, rng)) @ Vq.T * np.sqrt(N)).astype(np.float32)
        if dtype == "bf16":
            H = wl.round_to_bf16(H)
        Hd = ph.to_device(H, dtype)
        info = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        rt = torch.zeros(B, dtype=torch.int32, device="cuda")
        ws = solar.alloc_workspace(B, 1, N, d, r, Hd.dtype)
        S = torch.full((B, r), float("nan"), device="cuda"); V = torch.full((B, d, r), float("nan"), device="cuda")
        solar.gram_partials(Hd, ws)
        solar.eig_from_partials_ex(B, N, d, r, Hd.dtype, solar.ROUTE_AUTO, S, V, info, rt, ws)
        torch.cuda.synchronize()
        S = S.cpu().numpy().astype(np.float64); V = V.cpu().numpy().astype(np.float64)
        for b in range(B):
            tag = (seed, case, b, kind, dtype, N, d, r, hex(int(rt[b]) & 0xffffffff))
            seen.add((kind, int(rt[b]) & 0xff))
            # a strongly graded 128 x 128 matrix can use up the sweep cap on eigenvalues at the
            # rounding level; the kept pairs are checked all the same
            allowed = (0, solar.INFO_NOT_CONVERGED) if (kind == "geometric" and d == 128) else (0,)
            assert int(info[b]) in allowed, tag
            s_ref, _, _ = o.truncated_svd(H[b].astype(np.float64), r)
            tol = 1e-5 if dtype == "f32" else 1e-4
            # through the Gram matrix a singular value far below sigma_1 carries eps sigma_1^2 / sigma_i
            lim = np.where(s_ref > 1e-2 * s_ref[0], tol, 1e-3)
            assert np.all(np.abs(S[b] - s_ref) <= lim * s_ref[0]), tag
            assert np.abs(V[b].T @ V[b] - np.eye(r)).max() <= 2e-5, tag
            G = H[b].astype(np.float64).T @ H[b].astype(np.float64)
            res = np.linalg.norm(G @ V[b] - V[b] * (S[b] ** 2), axis=0).max() / s_ref[0] ** 2
            assert res <= 2e-5, tag
    # the draw reaches both outcomes
    assert {rr for _, rr in seen} >= {2, 3}
