"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element,
on the same seeded inputs.  Tolerances: see parity_harness.TOL (fp32 1e-4, bf16 2e-2,
max over rows of |dO|_inf / |O_ref|_inf)."""
import math

import numpy as np
import pytest
import torch

import oracle as o
from paper_2603_02561_b200 import solar
from paper_2603_02561_b200 import workloads as wl

import parity_harness as ph

pytestmark = pytest.mark.gpu


def _check(w, users_to_check, flags=0, want_us=False):
    inp = wl.generate(w)
    got = ph.run_gpu(w, inp, flags=flags, want_us=want_us)
    assert np.all(got["info"] == 0), got["info"]
    assert np.isfinite(got["O"]).all() and np.isfinite(got["V"]).all()
    worst = 0.0
    for k in users_to_check:
        res = ph.compare_user(w, inp, got, k, softmax=not (flags & solar.FLAG_NO_SOFTMAX))
        assert res["o_err"] <= ph.TOL[w.dtype], (w.name, k, res["o_err"])
        assert res["s_err"] <= (1e-5 if w.dtype == "f32" else 1e-4), (w.name, k, res["s_err"])
        worst = max(worst, res["o_err"])
        if want_us:
            us_ref = res["U"] * res["s"][None, :]
            tol = 1e-4 if w.dtype == "f32" else 2e-2
            err = np.abs(got["US"][k] - us_ref).max() / np.abs(us_ref).max()
            assert err <= tol, (w.name, k, err)
    return got, worst


# ---- the five named configurations ---------------------------------------------------
def test_c1_fp32_exact_rank8():
    _check(wl.CONFIGS["c1"], [0])


def test_c2_bf16_rank16_plus_noise():
    _check(wl.CONFIGS["c2"], [0, 7, 31])


def test_c3_headline_full_size_every_user():
    w = wl.CONFIGS["c3"]
    got, _ = _check(w, range(w.B))
    # closed-form singular values (storage rounding moves them by ~2^-9 relative at most)
    want = wl.spectrum(w)
    assert np.abs(got["S"] / want[None, :] - 1).max() < 5e-3


def test_c4_full_rank_power_law_full_size_every_user():
    w = wl.CONFIGS["c4"]
    inp = wl.generate(w)
    got = ph.run_gpu(w, inp)
    assert np.all(got["info"] == 0)
    for k in range(w.B):
        res = ph.compare_user(w, inp, got, k)
        assert res["o_err"] <= ph.TOL["bf16"], (k, res["o_err"])
        if k not in (0, 5):
            continue
        # truncation error against the full-rank operator is reported, not asserted
        H = inp["H"][k].astype(np.float64); C = inp["C"][k][:256].astype(np.float64)
        full = o.svd_attention(H, C, inp["Wq"], inp["Wk"], inp["Wv"], w.d, inp["scale"])
        trunc = o.max_rel_err_rows(res["O_ref"][:256], full)
        print(f"c4 user {k}: gpu-vs-oracle {res['o_err']:.3e}; rank-{w.r} vs rank-{w.d} operator {trunc:.3e}")


@pytest.mark.parametrize("N,r", [(2048, 8), (8192, 64), (32768, 8), (32768, 16), (32768, 32), (32768, 64)])
def test_c5_sweep_points(N, r):
    w = [x for x in wl.sweep_configs() if x.N == N and x.r == r][0]
    _check(w, [0, 63])


def test_serving_shape_12000_by_3000():
    _check(wl.CONFIGS["serve"], [3])


def test_serving_shape_at_rank_27():
    _check(wl.CONFIGS["serve27"], [0, 7])


@pytest.mark.parametrize("name", ["offline16", "offline27"])
def test_offline_shape_50_by_120(name):
    """Table 3's offline shape: a history shorter than the embedding is wide (N = 50 < d = 64)."""
    w = wl.CONFIGS[name]
    _check(w, [0, 1, 64, 127])


# ---- small shapes: several tiles, ragged tails, degenerate sizes -------------------------
SMALL = [
    ("f32", 3, 300, 32, 8, 65), ("f32", 2, 1000, 64, 64, 1), ("f32", 1, 257, 128, 33, 130),
    ("bf16", 3, 300, 32, 32, 65), ("bf16", 2, 1000, 64, 1, 7), ("bf16", 2, 515, 128, 64, 200),
    ("bf16", 5, 129, 64, 27, 64), ("f32", 2, 64, 64, 64, 3),
    # subspace dimensions 24 and 16 of the range-finder route (Ritz problems of every layout)
    ("bf16", 2, 700, 64, 20, 40), ("bf16", 2, 400, 128, 24, 50), ("f32", 2, 600, 128, 12, 33),
]


@pytest.mark.parametrize("dtype,B,N,d,r,M", SMALL)
def test_small_ragged_shapes(dtype, B, N, d, r, M):
    w = wl.Workload("small", dtype, B, N, d, r, M, "product_noise", rank=min(r + 3, d),
                    noise_var=1e-2, seed_index=11)
    _check(w, range(B), want_us=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_no_softmax_flag_matches_chain_on_low_rank(dtype):
    """Table 4 ablation: without the softmax the operator is the exact chain of Eq. 10."""
    w = wl.Workload("nosm", dtype, 2, 700, 64, 16, 90, "product", rank=16, seed_index=12)
    inp = wl.generate(w)
    got, _ = _check(w, [0, 1], flags=solar.FLAG_NO_SOFTMAX)
    for k in range(2):
        ref = o.chain_attention(inp["H"][k], inp["C"][k], inp["Wq"], inp["Wk"], inp["Wv"], inp["scale"])
        assert o.max_rel_err_rows(got["O"][k], ref) <= (3e-4 if dtype == "f32" else 2e-2)


def test_gram_partials_sum_to_HtH():
    for dtype, B, N, d in [("f32", 2, 777, 32), ("bf16", 3, 2500, 64), ("bf16", 2, 1300, 128)]:
        w = wl.Workload("g", dtype, B, N, d, 8, 4, "product_noise", rank=8, noise_var=1e-2, seed_index=13)
        inp = wl.generate(w)
        H = ph.to_device(inp["H"], dtype)
        ws = solar.alloc_workspace(B, 4, N, d, 8, H.dtype)
        ws.fill_(0xFF)
        solar.gram_partials(H, ws)
        torch.cuda.synchronize()
        S = solar.gram_splits(B, N, d, H.dtype)
        part = ws[: B * S * d * d * 4].view(torch.float32).view(B, S, d, d).cpu().numpy().astype(np.float64)
        G = part.sum(axis=1)
        H64 = inp["H"].astype(np.float64)
        ref = np.einsum("bni,bnj->bij", H64, H64)
        assert np.abs(G - ref).max() <= 2e-6 * np.abs(ref).max()


def test_stage_calls_compose_to_the_two_entry_points():
    w = wl.CONFIGS["c2"].with_(B=4, N=700, M=100)
    inp = wl.generate(w)
    got = ph.run_gpu(w, inp)
    H = ph.to_device(inp["H"], w.dtype); C = ph.to_device(inp["C"], w.dtype)
    Wq, Wk, Wv = (ph.to_device(inp[k], w.dtype) for k in ("Wq", "Wk", "Wv"))
    ws = solar.alloc_workspace(w.B, w.M, w.N, w.d, w.r, H.dtype)
    S = torch.empty(w.B, w.r, device="cuda"); V = torch.empty(w.B, w.d, w.r, device="cuda")
    info = torch.zeros(w.B, dtype=torch.int32, device="cuda"); O = torch.empty_like(C)
    solar.gram_partials(H, ws)
    solar.eig_from_partials(w.B, w.N, w.d, w.r, H.dtype, S, V, info, ws)
    solar.attn_prepare(S, V, Wq, Wk, Wv, inp["scale"], ws)
    solar.attn_apply(C, w.r, 0, O, ws)
    torch.cuda.synchronize()
    assert np.array_equal(S.cpu().numpy().astype(np.float64), got["S"])
    assert np.array_equal(V.cpu().numpy().astype(np.float64), got["V"])
    assert np.array_equal(O.float().cpu().numpy().astype(np.float64), got["O"])


# ---- degenerate inputs ------------------------------------------------------------------
def test_zero_history_gives_zero_output():
    w = wl.Workload("zero", "f32", 2, 200, 32, 4, 9, "product", rank=4, seed_index=14)
    inp = wl.generate(w)
    inp["H"][:] = 0
    got = ph.run_gpu(w, inp)
    assert np.all(got["info"] == 0) and np.all(got["S"] == 0) and np.all(got["O"] == 0)
    assert np.array_equal(got["V"][0], np.eye(32)[:, :4])


def test_rank_deficient_history_zero_tokens_take_softmax_weight():
    w = wl.Workload("rd", "f32", 2, 300, 32, 6, 20, "product", rank=3, seed_index=15)
    inp = wl.generate(w)
    got = ph.run_gpu(w, inp)
    assert np.all(got["info"] == 0)
    for k in range(2):
        s, V, _ = o.truncated_svd(inp["H"][k].astype(np.float64), 3)
        assert np.abs(got["S"][k][:3] - s).max() < 1e-5 * s[0]
        assert got["S"][k][3:].max() < 3e-3 * s[0]        # sqrt of fp32 rounding residue of G
        # oracle with the three real tokens plus three zero tokens
        ref = o.svd_attention(inp["H"][k].astype(np.float64), inp["C"][k], inp["Wq"], inp["Wk"],
                              inp["Wv"], 6, inp["scale"])
        assert o.max_rel_err_rows(got["O"][k], ref) < 5e-3


def test_nonfinite_input_is_reported_not_trapped():
    w = wl.Workload("nan", "bf16", 3, 400, 64, 8, 16, "product", rank=8, seed_index=16)
    inp = wl.generate(w)
    inp["H"][1, 17, 5] = np.nan
    got = ph.run_gpu(w, inp)
    assert got["info"][1] == solar.INFO_NONFINITE and got["info"][0] == 0 and got["info"][2] == 0
    assert np.isnan(got["S"][1]).all() and np.isnan(got["O"][1]).all()
    res = ph.compare_user(w, {**inp, "H": np.nan_to_num(inp["H"])}, got, 0)
    assert res["o_err"] <= ph.TOL["bf16"]


def test_empty_batch_and_no_candidates_are_noops():
    H = torch.zeros(0, 64, 64, device="cuda"); C = torch.zeros(0, 5, 64, device="cuda")
    S, V = solar.lowrank_factor(H, 8)
    assert S.shape == (0, 8)
    W = torch.zeros(64, 64, device="cuda")
    S = torch.ones(2, 8, device="cuda"); V = torch.zeros(2, 64, 8, device="cuda")
    C = torch.zeros(2, 0, 64, device="cuda")
    O = solar.svd_attention_fwd(C, S, V, W, W, W, 0.1)
    assert O.shape == (2, 0, 64)


def test_bad_arguments_raise():
    H = torch.zeros(1, 100, 48, device="cuda")
    with pytest.raises(solar.SolarError):
        solar.lowrank_factor(H, 8)
    H = torch.zeros(1, 100, 64, device="cuda")
    with pytest.raises(solar.SolarError):
        solar.lowrank_factor(H, 8, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
