"""Seeded synthetic inputs for the SVD-Attention forward pass.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic (no SVD, no attention): it only draws the
history matrices H, the candidates C and the projection weights, shaped like
the paper's lifelong-sequence workloads (Table 3: ten-thousand-scale histories,
thousands of candidates; Figure 1: effective rank in the high twenties).

Every tensor is drawn in double precision from a counter-based generator keyed
by (seed, tensor id, user), then rounded ONCE to the storage type.  The arrays
returned are float32 whose values are exactly representable in the storage
type, so both sides start from identical numbers.

"N(0, x)" in the workload recipes means variance x.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import math

import numpy as np

BASE_SEED = 26030256100

_T_H, _T_C, _T_WQ, _T_WK, _T_WV, _T_AUX = 1, 2, 3, 4, 5, 6


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "f32" | "bf16"  (storage type; accumulation is fp32 or wider)
    B: int              # users in the batch
    N: int              # history length (paper: N_L)
    d: int              # embedding width
    r: int              # rank kept
    M: int              # candidates per user (paper: N_C)
    kind: str           # "product" | "product_noise" | "spectrum"
    rank: int = 0       # rank of the generating product / number of non-zero sigmas
    decay: float = 0.0  # sigma_i = i^-decay for kind == "spectrum"
    noise_var: float = 0.0
    seed_index: int = 0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.seed_index

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    @property
    def pairs(self) -> int:
        """Work units of the headline metric: candidates x sequence positions."""
        return self.B * self.M * self.N


CONFIGS = {
    # exact rank-8 product, fp32 storage
    "c1": Workload("c1", "f32", 1, 256, 32, 8, 16, "product", rank=8, seed_index=1),
    # rank-16 product + N(0,1e-3) noise
    "c2": Workload("c2", "bf16", 32, 1024, 64, 16, 256, "product_noise", rank=16,
                   noise_var=1e-3, seed_index=2),
    # headline: rank-32 factors, sigma_i = 1/i
    "c3": Workload("c3", "bf16", 16, 10240, 64, 32, 2048, "spectrum", rank=32,
                   decay=1.0, seed_index=3),
    # full-rank power-law spectrum sigma_i = i^-1.5 over all 128 directions
    "c4": Workload("c4", "bf16", 8, 16384, 128, 64, 4096, "spectrum", rank=128,
                   decay=1.5, seed_index=4),
    # online-serving shape of Table 3 (12,000 behaviours x 3000 candidates), rank ~ Figure 1
    "serve": Workload("serve", "bf16", 8, 12000, 64, 32, 3000, "spectrum", rank=32,
                      decay=1.0, seed_index=6),
    # the same shape at the rank Figure 1 reads off a user sequence (27: not a multiple of 8 or 16)
    "serve27": Workload("serve27", "bf16", 8, 12000, 64, 27, 3000, "spectrum", rank=27,
                        decay=1.0, seed_index=7),
    # offline evaluation shape of Table 3 (history 50, 120 candidates per request; many requests per
    # batch): N < d, so the history has at most 50 directions, kept at rank 16 and 27
    "offline16": Workload("offline16", "bf16", 128, 50, 64, 16, 120, "product_noise", rank=16,
                          noise_var=1e-3, seed_index=8),
    "offline27": Workload("offline27", "bf16", 128, 50, 64, 27, 120, "product_noise", rank=27,
                          noise_var=1e-3, seed_index=9),
}


def sweep_configs(B=64, d=64, M=1024,
                  ranks=(8, 16, 32, 64), lengths=(2048, 4096, 8192, 16384, 32768)):
    """The c5 sweep: rank-r products + N(0,1e-3) noise for every (N, r)."""
    out = []
    for N in lengths:
        for r in ranks:
            out.append(Workload(f"c5_N{N}_r{r}", "bf16", B, N, d, r, M, "product_noise",
                                rank=r, noise_var=1e-3, seed_index=5))
    return out


def lookup(name: str) -> Workload:
    """A named configuration: c1..c4, serve, or a point of the c5 sweep (c5_N<N>_r<r>)."""
    if name in CONFIGS:
        return CONFIGS[name]
    for w in sweep_configs():
        if w.name == name:
            return w
    raise KeyError(name)


# --------------------------------------------------------------------------
def _rng(seed: int, tensor: int, user: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), (tensor << 32) | user]))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) >> 16).astype(np.uint32) << 16
    return r.view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def _store(x64: np.ndarray, dtype: str) -> np.ndarray:
    x32 = x64.astype(np.float32)
    return round_to_bf16(x32) if dtype == "bf16" else x32


def _orthonormal(g: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    q, _ = np.linalg.qr(g.standard_normal((rows, cols)))
    return q


def spectrum(w: Workload) -> np.ndarray | None:
    """Closed-form singular values of each user's H before storage rounding."""
    if w.kind != "spectrum":
        return None
    i = np.arange(1, w.rank + 1, dtype=np.float64)
    sig = i ** (-w.decay)
    gamma = math.sqrt(w.N * w.d / float((sig ** 2).sum()))   # unit-variance entries
    return gamma * sig


def history(w: Workload, user: int, exact: bool = False) -> np.ndarray:
    """History matrix H[N,d] of one user; `exact` skips the storage rounding (float64)."""
    g = _rng(w.seed, _T_H, user)
    if w.kind in ("product", "product_noise"):
        std = (1.0 / math.sqrt(w.rank)) ** 0.5          # variance 1/sqrt(rank)
        A = g.standard_normal((w.N, w.rank)) * std
        Bm = g.standard_normal((w.d, w.rank)) * std
        H = A @ Bm.T
        if w.kind == "product_noise":
            H = H + g.standard_normal((w.N, w.d)) * math.sqrt(w.noise_var)
    elif w.kind == "spectrum":
        U0 = _orthonormal(g, w.N, w.rank)
        V0 = _orthonormal(g, w.d, w.rank)
        H = (U0 * spectrum(w)[None, :]) @ V0.T
    else:
        raise ValueError(w.kind)
    return H if exact else _store(H, w.dtype)


def candidates(w: Workload, user: int) -> np.ndarray:
    """Candidate item embeddings C[M,d], i.i.d. N(0, 1/d)."""
    g = _rng(w.seed, _T_C, user)
    return _store(g.standard_normal((w.M, w.d)) / math.sqrt(w.d), w.dtype)


def weights(w: Workload):
    """Random-init projections W_Q, W_K, W_V [d,d], i.i.d. N(0, 1/d), shared by users."""
    out = []
    for t in (_T_WQ, _T_WK, _T_WV):
        g = _rng(w.seed, t, 0)
        out.append(_store(g.standard_normal((w.d, w.d)) / math.sqrt(w.d), w.dtype))
    return tuple(out)


def generate(w: Workload, users=None) -> dict:
    """All inputs of a workload (or of the listed users) as float32 arrays."""
    users = list(range(w.B)) if users is None else list(users)
    H = np.stack([history(w, b) for b in users])
    C = np.stack([candidates(w, b) for b in users])
    Wq, Wk, Wv = weights(w)
    return {"H": H, "C": C, "Wq": Wq, "Wk": Wk, "Wv": Wv, "scale": w.scale, "users": users}
