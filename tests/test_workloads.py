"""The seeded input generators: determinism, storage rounding, stated structure."""
import numpy as np

from paper_2603_02561_b200 import workloads as wl


def test_bf16_rounding_is_nearest_even_and_idempotent():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.001953125, -3.14159, 1e-20, 65504.0], np.float32)
    r = wl.round_to_bf16(x)
    assert r[0] == 1.0
    assert r[1] == 1.0                      # 1 + 2^-8 is a tie -> even mantissa (1.0)
    assert r[2] == np.float32(1.0078125)    # 1 + 1.5*2^-8 -> up
    assert np.array_equal(wl.round_to_bf16(r), r)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)
    bits = wl.bf16_bits(r)
    assert bits.dtype == np.uint16
    assert np.array_equal((bits.astype(np.uint32) << 16).view(np.float32), r)


def test_generation_is_deterministic_and_per_user():
    w = wl.CONFIGS["c2"].with_(B=3, N=64, M=8)
    a = wl.generate(w)
    b = wl.generate(w)
    assert all(np.array_equal(a[k], b[k]) for k in ("H", "C", "Wq", "Wk", "Wv"))
    one = wl.generate(w, users=[2])
    assert np.array_equal(one["H"][0], a["H"][2]) and np.array_equal(one["C"][0], a["C"][2])
    assert not np.array_equal(a["H"][0], a["H"][1])
    assert np.array_equal(wl.round_to_bf16(a["H"]), a["H"])   # already storage-exact


def test_c1_is_exactly_rank_r_before_rounding():
    w = wl.CONFIGS["c1"]
    H = wl.history(w, 0, exact=True)
    sv = np.linalg.svd(H, compute_uv=False)
    assert sv[w.r - 1] > 1.0 and sv[w.r] < 1e-12 * sv[0]
    assert abs(H.var() - 1.0) < 0.35          # unit-variance entries (variance 1/sqrt(8) factors)


def test_spectrum_workload_has_the_stated_singular_values():
    w = wl.CONFIGS["c3"].with_(B=1, N=512, M=4)
    H = wl.history(w, 0, exact=True)
    sv = np.linalg.svd(H, compute_uv=False)
    want = wl.spectrum(w)
    assert np.abs(sv[:32] - want).max() < 1e-10 * want[0]
    assert sv[32] < 1e-12 * want[0]
    assert abs(want[0] / want[31] - 32.0) < 1e-12
    assert abs((H ** 2).mean() - 1.0) < 1e-12


def test_candidate_and_weight_variance():
    w = wl.CONFIGS["c3"].with_(B=1, N=64)
    C = wl.candidates(w, 0)
    assert abs(C.var() * w.d - 1.0) < 0.05
    for W in wl.weights(w):
        assert W.shape == (w.d, w.d) and abs(W.var() * w.d - 1.0) < 0.1


def test_sweep_grid():
    s = wl.sweep_configs()
    assert len(s) == 20 and {x.r for x in s} == {8, 16, 32, 64}
    assert all(x.B == 64 and x.M == 1024 and x.d == 64 for x in s)
