"""solar_svd_attention_fused (the whole forward pass in one call, the eigensolver CTAs ending
with the factor-token projections) against the two-call path, bit for bit, and against the
oracle; and the rule that a call may follow a kernel that writes its inputs on the same stream."""
import numpy as np
import pytest
import torch

from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu

SHAPES = [
    wl.CONFIGS["c1"],
    wl.CONFIGS["c2"].with_(B=5, N=1300, M=300),
    wl.CONFIGS["c3"].with_(B=3, N=2500, M=700),
    wl.CONFIGS["c4"].with_(B=2, N=1100, M=260),
    wl.Workload("all64", "bf16", 2, 900, 64, 64, 130, "product_noise", rank=64, noise_var=1e-3, seed_index=41),
    wl.Workload("f32d128", "f32", 2, 600, 128, 20, 50, "product_noise", rank=20, noise_var=1e-3, seed_index=42),
    wl.Workload("r1", "bf16", 2, 400, 64, 1, 9, "product_noise", rank=4, noise_var=1e-2, seed_index=43),
]


def _dev(w, inp):
    H = ph.to_device(inp["H"], w.dtype); C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    return H, C, Wq, Wk, Wv


@pytest.mark.parametrize("w", SHAPES, ids=[w.name for w in SHAPES])
@pytest.mark.parametrize("flags", [0, solar.FLAG_NO_SOFTMAX])
def test_fused_call_equals_the_two_calls_bit_for_bit(w, flags):
    inp = wl.generate(w)
    H, C, Wq, Wk, Wv = _dev(w, inp)
    ws2 = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype); ws2.fill_(0xFF)
    S2, V2 = solar.lowrank_factor(H, w.r, workspace=ws2, M=w.M)
    O2 = solar.svd_attention_fwd(C, S2, V2, Wq, Wk, Wv, inp["scale"], flags, workspace=ws2, N=w.N)
    wsf = solar.alloc_fused_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype); wsf.fill_(0xFF)
    info = torch.full((w.B,), -1, dtype=torch.int32, device="cuda")
    S = torch.full_like(S2, float("nan")); V = torch.full_like(V2, float("nan")); O = torch.full_like(O2, float("nan"))
    solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"], flags, S=S, V=V, O=O, info=info, workspace=wsf)
    torch.cuda.synchronize()
    assert torch.all(info == 0)
    assert torch.equal(S, S2) and torch.equal(V, V2)
    assert torch.equal(O.view(torch.uint8), O2.view(torch.uint8))


def test_fused_call_against_the_oracle():
    w = wl.CONFIGS["c2"].with_(B=4, N=900, M=200)
    inp = wl.generate(w)
    H, C, Wq, Wk, Wv = _dev(w, inp)
    O, S, V = solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"])
    torch.cuda.synchronize()
    got = {"S": S.cpu().numpy().astype(np.float64), "V": V.cpu().numpy().astype(np.float64),
           "O": O.float().cpu().numpy().astype(np.float64)}
    for k in range(w.B):
        res = ph.compare_user(w, inp, got, k)
        assert res["o_err"] <= ph.TOL[w.dtype], (k, res["o_err"])


def test_fused_call_rejects_a_small_workspace_on_the_host():
    w = wl.CONFIGS["c2"].with_(B=2, N=512, M=64)
    inp = wl.generate(w)
    H, C, Wq, Wk, Wv = _dev(w, inp)
    small = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype)      # the two-call size: too small
    assert small.numel() < solar.fused_workspace_bytes(w.B, w.M, w.N, w.d, w.r, H.dtype)
    with pytest.raises(solar.SolarError) as e:
        solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"], workspace=small)
    assert e.value.status == solar.ERR_WORKSPACE


@pytest.mark.parametrize("fused", [False, True])
def test_inputs_written_by_the_kernel_just_before_the_call(fused):
    """H, C and the weights are produced by kernels queued on the same stream right before the
    library call, with fresh data each round and no synchronisation in between: the first kernel
    of the call must wait for them.  Compared bit for bit with a run that synchronises first."""
    w = wl.CONFIGS["c3"].with_(B=8, N=4096, M=1024)
    inp = wl.generate(w)
    H0, C0, Wq0, Wk0, Wv0 = _dev(w, inp)
    H = torch.empty_like(H0); C = torch.empty_like(C0)
    Wq = torch.empty_like(Wq0); Wk = torch.empty_like(Wk0); Wv = torch.empty_like(Wv0)
    ws = (solar.alloc_fused_workspace if fused else solar.alloc_workspace)(w.B, w.M, w.N, w.d, w.r, H.dtype)
    S = torch.empty(w.B, w.r, device="cuda"); V = torch.empty(w.B, w.d, w.r, device="cuda"); O = torch.empty_like(C)

    def call():
        if fused:
            solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"], S=S, V=V, O=O, workspace=ws)
        else:
            solar.lowrank_factor(H, w.r, S=S, V=V, workspace=ws, M=w.M)
            solar.svd_attention_fwd(C, S, V, Wq, Wk, Wv, inp["scale"], O=O, workspace=ws, N=w.N)

    def produce(round_):
        # element-wise kernels on the current stream: a permutation of the users plus a scaling
        perm = torch.roll(torch.arange(w.B, device="cuda"), round_)
        g = 1.0 + 0.25 * round_
        torch.mul(H0[perm], g, out=H); torch.mul(C0[perm], 1.0, out=C)
        torch.mul(Wq0, g, out=Wq); torch.mul(Wk0, 1.0, out=Wk); torch.mul(Wv0, 1.0, out=Wv)

    for round_ in range(4):
        H.fill_(float("nan")); C.fill_(float("nan")); Wq.fill_(float("nan"))
        produce(round_)
        torch.cuda.synchronize()
        call()
        torch.cuda.synchronize()
        ref = (S.clone(), V.clone(), O.clone())
        for _ in range(3):
            H.fill_(float("nan")); C.fill_(float("nan")); Wq.fill_(float("nan"))   # stale contents are poison
            produce(round_)
            call()                                  # no synchronisation between producer and call
            torch.cuda.synchronize()
            assert torch.equal(S, ref[0]) and torch.equal(V, ref[1])
            assert torch.equal(O.view(torch.uint8), ref[2].view(torch.uint8))


def test_slice_limit_changes_the_slicing_not_the_result():
    """solar_set_slice_limit: fewer, longer row slices per user (the setting for throughput with many
    requests in flight).  The partial sums are grouped differently, so the factors agree to rounding
    and the output within the parity tolerance; the oracle is matched either way; a workspace sized
    under a cap is refused once the cap is lifted."""
    w = wl.CONFIGS["c3"].with_(B=3, N=5000, M=300)
    inp = wl.generate(w)
    H, C, Wq, Wk, Wv = _dev(w, inp)
    old = solar.set_slice_limit(0)
    try:
        n_default = solar.gram_slices(w.B, w.N, w.d, H.dtype)
        O0, S0, V0 = solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"])
        assert solar.set_slice_limit(2) == 0
        assert solar.gram_slices(w.B, w.N, w.d, H.dtype) == 2 < n_default
        small = solar.alloc_fused_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype)
        O2, S2, V2 = solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"], workspace=small)
        S2b, V2b = solar.lowrank_factor(H, w.r)                       # the two-call path follows the cap too
        torch.cuda.synchronize()
        assert torch.equal(S2, S2b) and torch.equal(V2, V2b)
        assert (S2 - S0).abs().max() <= 1e-5 * S0.max()
        got = {"S": S2.cpu().numpy().astype(np.float64), "V": V2.cpu().numpy().astype(np.float64),
               "O": O2.float().cpu().numpy().astype(np.float64)}
        for k in range(w.B):
            assert ph.compare_user(w, inp, got, k)["o_err"] <= ph.TOL[w.dtype]
        assert solar.set_slice_limit(0) == 2
        assert small.numel() < solar.fused_workspace_bytes(w.B, w.M, w.N, w.d, w.r, H.dtype)
        with pytest.raises(solar.SolarError) as e:
            solar.svd_attention_fused(H, C, Wq, Wk, Wv, w.r, inp["scale"], workspace=small)
        assert e.value.status == solar.ERR_WORKSPACE
    finally:
        solar.set_slice_limit(old)


@pytest.mark.parametrize("M,r,flags", [(2048, 32, 0), (1000, 27, 0), (3000, 16, 0), (515, 5, 0),
                                       (1300, 32, solar.FLAG_NO_SOFTMAX)])
def test_throughput_attention_kernel_gives_the_same_bits(M, r, flags):
    """Under a slice limit the candidate attention runs as long CTAs that overlap the candidate
    stream, the GEMMs and the softmax of consecutive tiles (bf16, d = 64, r <= 32, at least four
    tiles).  Same GEMMs in the same order, same softmax: the output must equal the
    one-tile-per-CTA kernel's bit for bit, ragged last tile included."""
    w = wl.CONFIGS["c3"].with_(B=3, N=1500, M=M, r=r)
    inp = wl.generate(w)
    H, C, Wq, Wk, Wv = _dev(w, inp)
    old = solar.set_slice_limit(0)
    try:
        ws = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype)
        S, V = solar.lowrank_factor(H, w.r, workspace=ws, M=w.M)
        O0 = torch.full_like(C, float("nan"))
        solar.svd_attention_fwd(C, S, V, Wq, Wk, Wv, inp["scale"], flags, O=O0, workspace=ws, N=w.N)
        solar.set_slice_limit(2)
        guard = torch.full((w.B, w.M + 128, w.d), 7.0, dtype=C.dtype, device="cuda")    # rows past M stay untouched
        O1 = guard[:, :w.M]
        O1c = torch.full_like(C, float("nan"))
        for _ in range(2):
            solar.svd_attention_fwd(C, S, V, Wq, Wk, Wv, inp["scale"], flags, O=O1c, workspace=ws, N=w.N)
        torch.cuda.synchronize()
        assert torch.equal(O1c.view(torch.uint8), O0.view(torch.uint8))
        assert not torch.isnan(O1c.float()).any()
        del O1, guard
    finally:
        solar.set_slice_limit(old)
