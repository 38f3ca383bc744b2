"""US = H V (the left factor times Sigma, which Eq. 10 drops from the forward pass) against
the plain product in fp64, element by element: both kernels (tensor cores for bf16 with
d = 64 or 128 and N >= 128; FFMA otherwise), ragged tails, several row slices per user,
ranks that are not multiples of 8 or 16."""
import numpy as np
import pytest
import torch

from paper_2603_02561_b200 import solar

pytestmark = pytest.mark.gpu

CASES = [
    # (dtype, B, N, d, r)
    ("bf16", 2, 128, 64, 32),          # exactly one tile
    ("bf16", 3, 1000, 64, 32),         # ragged tail
    ("bf16", 2, 5000, 64, 27),         # rows of 54 bytes: the scalar store path
    ("bf16", 1, 40000, 64, 16),        # many slices for one user
    ("bf16", 2, 777, 64, 64),          # r = d
    ("bf16", 5, 900, 64, 8),
    ("bf16", 2, 1500, 128, 64),
    ("bf16", 2, 300, 128, 40),
    ("bf16", 2, 2000, 128, 1),
    ("bf16", 2, 100, 64, 16),          # N < 128: FFMA kernel
    ("bf16", 2, 500, 32, 16),          # d = 32: FFMA kernel
    ("f32", 2, 700, 64, 24),           # fp32 storage: FFMA kernel
]


@pytest.mark.parametrize("dtype,B,N,d,r", CASES, ids=[f"{c[0]}_B{c[1]}_N{c[2]}_d{c[3]}_r{c[4]}" for c in CASES])
def test_project_us_matches_plain_product(dtype, B, N, d, r):
    g = torch.Generator().manual_seed(1000 * N + 10 * d + r)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    H = torch.randn(B, N, d, generator=g).to(tdt)
    # orthonormal-like columns with mixed signs and magnitudes, as the eigensolver returns
    V = torch.linalg.qr(torch.randn(B, d, d, generator=g))[0][:, :, :r].contiguous()
    # a dense [B, N, r] output with guard elements behind it
    out_buf = torch.full((B * N * r + 64,), float("nan"), dtype=tdt).cuda()
    out = out_buf[: B * N * r].view(B, N, r)
    solar.project_us(H.cuda(), V.cuda(), out)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    ref = H.double().numpy() @ V.double().numpy()
    scale = np.abs(ref).max()
    # fp32 accumulation of exact products, then one rounding to the storage type
    tol = (2.0 ** -8 if dtype == "bf16" else 2e-6)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= tol * scale, np.abs(got - ref).max() / scale
    assert torch.isnan(out_buf[B * N * r:].float()).all()               # nothing written past the end


def test_project_us_is_deterministic_and_stream_ordered():
    B, N, d, r = 4, 3000, 64, 32
    g = torch.Generator().manual_seed(7)
    H = torch.randn(B, N, d, generator=g).to(torch.bfloat16).cuda()
    V = torch.linalg.qr(torch.randn(B, d, d, generator=g))[0][:, :, :r].contiguous().cuda()
    a = torch.empty(B, N, r, dtype=torch.bfloat16, device="cuda")
    b = torch.empty_like(a)
    solar.project_us(H, V, a)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        solar.project_us(H, V, b, stream=st)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
