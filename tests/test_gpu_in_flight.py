"""Many requests in flight on different streams, each on buffers of its own: every result must equal,
bit for bit, the result of the same call made alone.  The kernels of different requests share the
SMs and run at shifted paces, which is when a missing wait or a miscounted barrier arrival inside
a kernel shows (the bounded waits would turn it into NaN rows or a non-zero info word)."""
import numpy as np
import pytest
import torch

from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [0, 2])
def test_requests_in_flight_match_the_calls_made_alone(limit):
    w = wl.CONFIGS["c3"].with_(B=6, N=4096, M=2048)
    inp = wl.generate(w)
    H0 = ph.to_device(inp["H"], w.dtype); C0 = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    lanes, steps = 16, 6
    old = solar.set_slice_limit(limit)
    try:
        # distinct inputs per request: the users rotated
        Hs = [torch.roll(H0, i, 0).contiguous() for i in range(w.B)]
        Cs = [torch.roll(C0, i, 0).contiguous() for i in range(w.B)]
        ref = []
        for i in range(w.B):
            O, S, V = solar.svd_attention_fused(Hs[i], Cs[i], Wq, Wk, Wv, w.r, inp["scale"])
            torch.cuda.synchronize()
            ref.append((O.clone(), S.clone(), V.clone()))
        streams = [torch.cuda.Stream() for _ in range(lanes)]
        out = []
        for l in range(lanes):
            ws = solar.alloc_fused_workspace(w.B, w.M, w.N, w.d, w.r, H0.dtype)
            per_step = []
            for s in range(steps):
                per_step.append((torch.full_like(C0, float("nan")), torch.full((w.B, w.r), float("nan"), device="cuda"),
                                 torch.full((w.B, w.d, w.r), float("nan"), device="cuda"),
                                 torch.full((w.B,), -1, dtype=torch.int32, device="cuda")))
            out.append((ws, per_step))
        torch.cuda.synchronize()
        for s in range(steps):
            for l in range(lanes):
                k = (l + s) % w.B
                ws, per_step = out[l]
                O, S, V, info = per_step[s]
                solar.svd_attention_fused(Hs[k], Cs[k], Wq, Wk, Wv, w.r, inp["scale"], S=S, V=V, O=O, info=info,
                                          workspace=ws, stream=streams[l])
        torch.cuda.synchronize()
        for l in range(lanes):
            for s in range(steps):
                k = (l + s) % w.B
                O, S, V, info = out[l][1][s]
                assert torch.all(info == 0), (l, s)
                assert torch.equal(S, ref[k][1]) and torch.equal(V, ref[k][2]), (l, s)
                assert torch.equal(O.view(torch.uint8), ref[k][0].view(torch.uint8)), (l, s)
    finally:
        solar.set_slice_limit(old)
