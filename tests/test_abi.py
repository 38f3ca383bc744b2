"""The C-ABI library loads, exports everything include/solar.h declares, and rejects
bad arguments on the host before anything touches a GPU (no device is needed here)."""
import ctypes
import os
import re

import pytest
import torch

from paper_2603_02561_b200 import build as solar_build
from paper_2603_02561_b200 import solar

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    solar_build.build()
    return solar.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "solar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(solar_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(L):
    names = declared_symbols()
    assert "solar_lowrank_factor" in names and "solar_svd_attention_fwd" in names
    for n in names:
        assert hasattr(L, n), n
        assert n in solar.SIGNATURES, f"binding lacks {n}"
    assert sorted(solar.SIGNATURES) == names


def test_status_strings(L):
    assert L.solar_status_string(0) == b"ok"
    assert b"workspace" in L.solar_status_string(solar.ERR_WORKSPACE)


def test_workspace_bytes_and_splits(L):
    bf = torch.bfloat16
    assert solar.workspace_bytes(16, 2048, 10240, 64, 32, bf) >= 16 * solar.gram_splits(16, 10240, 64, bf) * 64 * 64 * 4
    assert solar.workspace_bytes(1, 16, 256, 32, 8, torch.float32) > 0
    assert solar.workspace_bytes(1, 16, 256, 48, 8, torch.float32) == 0      # unsupported d
    assert solar.workspace_bytes(1, 16, 256, 64, 65, torch.float32) == 0     # r > 64
    assert 1 <= solar.gram_splits(16, 10240, 64, bf) <= 64
    assert solar.gram_splits(1000, 128, 64, bf) == 1
    # slices (CTAs, status words) per user and partial matrices per user
    assert solar.gram_slices(16, 10240, 64, bf) == 9
    for (B, N) in [(1, 128), (3, 1000), (16, 10240), (64, 32768), (8, 12000), (1, 100000)]:
        sl, pa = solar.gram_slices(B, N, 64, bf), solar.gram_splits(B, N, 64, bf)
        assert sl % pa == 0 and sl // pa <= 8 and 1 <= sl <= 64


def _factor(L, B, M, N, d, r, dt, H=0x1000, S=0x1000, V=0x1000, ws=0x1000, wsb=1 << 40):
    vp = ctypes.c_void_p
    return L.solar_lowrank_factor(B, M, N, d, r, dt, vp(H), vp(S), vp(V), None, None, vp(ws), wsb, None)


def test_host_side_rejections_need_no_gpu(L):
    # all of these must return before any CUDA call (fake pointers are never dereferenced)
    assert _factor(L, 1, 1, 256, 48, 8, 0) == solar.ERR_UNSUPPORTED
    assert _factor(L, 1, 1, 256, 64, 65, 0) == solar.ERR_INVALID_ARG       # r > d
    assert _factor(L, 1, 1, 256, 128, 65, 0) == solar.ERR_UNSUPPORTED      # r > 64
    assert _factor(L, 1, 1, 4, 64, 8, 0) == solar.ERR_INVALID_ARG          # r > N
    assert _factor(L, -1, 1, 256, 64, 8, 0) == solar.ERR_INVALID_ARG
    assert _factor(L, 1, 1, 256, 64, 8, 7) == solar.ERR_UNSUPPORTED        # dtype
    assert _factor(L, 1, 1, 256, 64, 8, 0, H=0) == solar.ERR_INVALID_ARG   # NULL
    assert _factor(L, 1, 1, 256, 64, 8, 0, H=0x1004) == solar.ERR_INVALID_ARG   # misaligned
    assert _factor(L, 1, 1, 256, 64, 8, 0, wsb=16) == solar.ERR_WORKSPACE
    assert _factor(L, 1, 1, 256, 64, 8, 0, ws=0) == solar.ERR_WORKSPACE
    assert _factor(L, 0, 1, 256, 64, 8, 0) == solar.OK                     # empty batch: no-op
    vp = ctypes.c_void_p
    p = vp(0x1000)
    st = L.solar_svd_attention_fwd(1, 4, 256, 64, 8, 1, p, p, p, p, p, p, 0.125, 2, p, p, 1 << 40, None)
    assert st == solar.ERR_UNSUPPORTED                                     # unknown flag
    st = L.solar_svd_attention_fwd(1, 0, 256, 64, 8, 1, p, p, p, p, p, p, 0.125, 0, p, p, 1 << 40, None)
    assert st == solar.OK                                                  # no candidates: no-op
    st = L.solar_svd_attention_fwd(1, 4, 256, 64, 8, 1, p, p, p, p, p, p, 0.125, 0, p, p, 8, None)
    assert st == solar.ERR_WORKSPACE


def test_backward_calls_reject_bad_arguments_on_the_host(L):
    vp = ctypes.c_void_p
    p = vp(0x1000)
    bf = torch.bfloat16
    need = solar.backward_workspace_bytes(16, 2048, 10240, 64, 32, bf)
    # attention workspace, per-chunk partials [B][chunks][2][d][64] f32, dW [B][3][d][d] f32, operands
    assert need >= solar.workspace_bytes(16, 2048, 32, 64, 32, bf) // 2
    assert need >= 16 * 2 * 64 * 64 * 4 + 16 * 3 * 64 * 64 * 4
    assert need >= 16 * 64 * 64 * 4                                         # K_b of solar_svd_backward
    assert solar.backward_workspace_bytes(1, 16, 256, 48, 8, bf) == 0       # unsupported d

    def bwd(B=1, M=4, d=64, r=8, dt=1, flags=0, wsb=1 << 40, C=p):
        return L.solar_svd_attention_bwd(B, M, 256, d, r, dt, C, p, p, p, p, p, 0.125, flags, p,
                                         p, p, p, p, p, p, p, wsb, None)
    assert bwd(d=48) == solar.ERR_UNSUPPORTED
    assert bwd(r=65) == solar.ERR_INVALID_ARG
    assert bwd(flags=2) == solar.ERR_UNSUPPORTED
    assert bwd(wsb=64) == solar.ERR_WORKSPACE
    assert bwd(C=vp(0)) == solar.ERR_INVALID_ARG
    assert bwd(B=0) == solar.OK

    def svdb(B=1, N=256, d=64, r=8, eps=0.0, wsb=1 << 40, H=p):
        return L.solar_svd_backward(B, N, d, r, 1, H, p, p, p, p, eps, p, p, wsb, None)
    assert svdb(d=48) == solar.ERR_UNSUPPORTED
    assert svdb(N=4) == solar.ERR_INVALID_ARG                               # r > N
    assert svdb(eps=-1.0) == solar.ERR_INVALID_ARG
    assert svdb(eps=float("nan")) == solar.ERR_INVALID_ARG
    assert svdb(wsb=64) == solar.ERR_WORKSPACE
    assert svdb(H=vp(0x1002)) == solar.ERR_INVALID_ARG
    assert svdb(B=0) == solar.OK


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(solar, "_lib", None)
    monkeypatch.setattr(solar, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        solar.lib()


def test_slice_limit_is_a_host_side_setting():
    """solar_set_slice_limit needs no GPU: it returns the previous value, caps the slice count
    the planning calls report, and never makes a workspace larger."""
    from paper_2603_02561_b200 import solar
    L = solar.lib()
    args = (16, 2048, 10240, 64, 32, solar.BF16)
    old = L.solar_set_slice_limit(0)
    try:
        n0 = L.solar_gram_slices(16, 10240, 64, solar.BF16)
        b0 = L.solar_workspace_bytes(*args)
        assert n0 == 9
        assert L.solar_set_slice_limit(3) == 0
        assert L.solar_gram_slices(16, 10240, 64, solar.BF16) == 3
        assert L.solar_workspace_bytes(*args) <= b0
        assert L.solar_set_slice_limit(-5) == 3           # negative means no cap
        assert L.solar_gram_slices(16, 10240, 64, solar.BF16) == n0
    finally:
        L.solar_set_slice_limit(old)
