"""solar_lowrank_factor_static -- the factorization for hosts that may not allocate device
memory (a serving process whose buffers all come from an arena planned at start-up, a plug-in
that is given only its inputs and outputs).  Its scratch is a fixed array inside the library,
so the checks here are: it gives what solar_lowrank_factor gives, twice in a row (the array
keeps the previous call's contents), and it refuses sizes the array cannot hold.

Collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import ctypes

import gc

import numpy as np
import pytest
import torch

from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph


def test_oversized_request_is_refused_on_the_host():
    # B * splits * d*d*4 bytes far beyond the 16 MiB array; fake pointers are never used
    vp = ctypes.c_void_p
    p = vp(0x1000)
    L = solar.lib()
    assert solar.static_scratch_bytes() == 16 << 20
    st = L.solar_lowrank_factor_static(4096, 0, 4096, 128, 8, solar.BF16, p, p, p, None, None)
    assert st == solar.ERR_WORKSPACE
    st = L.solar_lowrank_factor_static(1, 0, 256, 48, 8, solar.BF16, p, p, p, None, None)
    assert st == solar.ERR_UNSUPPORTED


@pytest.mark.gpu
def test_static_scratch_variant_matches_workspace_variant_twice():
    cases = [wl.CONFIGS["c2"].with_(B=6, N=900, M=4),
             wl.Workload("na", "f32", 3, 500, 32, 8, 4, "product_noise", rank=8, noise_var=1e-2,
                         seed_index=21)]
    for rep in range(2):                       # second pass reuses the array left by the first
        for w in cases:
            inp = wl.generate(w)
            H = ph.to_device(inp["H"], w.dtype)
            S0, V0 = solar.lowrank_factor(H, w.r)
            S1 = torch.full((w.B, w.r), float("nan"), device="cuda")
            V1 = torch.full((w.B, w.d, w.r), float("nan"), device="cuda")
            info = torch.full((w.B,), -1, dtype=torch.int32, device="cuda")
            solar.lowrank_factor_static(H, w.r, S=S1, V=V1, info=info)
            torch.cuda.synchronize()
            assert (info == 0).all()
            s0, s1 = S0.cpu().numpy().astype(np.float64), S1.cpu().numpy().astype(np.float64)
            v0, v1 = V0.cpu().numpy().astype(np.float64), V1.cpu().numpy().astype(np.float64)
            tol = 1e-5 if w.dtype == "f32" else 1e-4      # the singular-value tolerance of the parity tests
            assert np.abs(s1 - s0).max() <= tol * s0.max(), (rep, w.name)
            assert np.abs(v1 - v0).max() <= tol, (rep, w.name)
            # the same kernels in the same order on the same numbers: the bits agree as well
            assert torch.equal(S0, S1) and torch.equal(V0, V1), (rep, w.name)


@pytest.mark.gpu
def test_static_scratch_variant_allocates_nothing():
    """After the first call on the device (which looks up the array's address), a call leaves
    both the caching allocator's books and the driver's free-memory figure where they were."""
    w = wl.CONFIGS["c2"].with_(B=4, N=700, M=4)
    inp = wl.generate(w)
    H = ph.to_device(inp["H"], w.dtype)
    S = torch.empty(w.B, w.r, device="cuda"); V = torch.empty(w.B, w.d, w.r, device="cuda")
    info = torch.empty(w.B, dtype=torch.int32, device="cuda")
    solar.lowrank_factor_static(H, w.r, S=S, V=V, info=info)          # first call: set-up
    torch.cuda.synchronize()
    # tensors left behind by earlier tests must not be freed inside the measured window
    gc.collect()
    gc.disable()
    try:
        before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
        for _ in range(3):
            solar.lowrank_factor_static(H, w.r, S=S, V=V, info=info)
        torch.cuda.synchronize()
        after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    finally:
        gc.enable()
    assert before == after, (before, after)
    assert (info == 0).all()
