"""The seeded input recipes: determinism, structure of the Byzantine rows, bf16 rounding."""
import numpy as np
import torch

import synthetic_inputs as si


def test_generation_is_deterministic_and_thread_count_independent():
    w = si.WORKLOADS["cfg2"].scaled(3 * si.CHUNK // 2 + 17)
    a = si.generate(w, threads=1)
    b = si.generate(w, threads=4)
    assert a.dtype == np.float32 and a.shape == (w.p, w.n)
    assert np.array_equal(a, b)


def test_signflip_rows_are_identical_and_opposed_to_the_mean():
    w = si.WORKLOADS["cfg1"]
    G = si.generate(w)
    byz = si.byzantine_positions(w)
    assert len(byz) == 2 and np.array_equal(G[byz[0]], G[byz[1]])
    honest = np.delete(np.arange(w.p), byz)
    mu_hat = G[honest].astype(np.float64).mean(axis=0)
    cos = (G[byz[0]] @ mu_hat) / (np.linalg.norm(G[byz[0]]) * np.linalg.norm(mu_hat))
    assert cos < -0.95


def test_mixed_workload_has_a_zero_row_a_huge_row_and_a_flipped_row():
    w = si.WORKLOADS["cfg2"].scaled(50_001)
    G = si.generate(w).astype(np.float64)
    byz = si.byzantine_positions(w)
    norms = np.sum(G * G, axis=1) / w.n
    assert sorted(np.round(norms[byz], 0)) == [0.0, 100.0, 100.0] or (
        norms[byz].min() == 0.0 and np.all(np.sort(norms[byz])[1:] > 80))
    honest = np.delete(np.arange(w.p), byz)
    assert np.all(np.abs(norms[honest] - 1.09) < 0.05)


def test_lowrank_shift_rows_sit_50_from_the_honest_mean():
    w = si.WORKLOADS["cfg3"].scaled(40_000)
    G = si.generate(w).astype(np.float64)
    byz = si.byzantine_positions(w)
    honest = np.delete(np.arange(w.p), byz)
    mean_h = G[honest].mean(axis=0)
    dist = np.linalg.norm(G[byz] - mean_h[None, :], axis=1)
    assert np.allclose(dist, 50.0, rtol=1e-4)
    s = np.linalg.svd(G[honest], compute_uv=False)
    assert s[3] > 3 * s[4]                      # rank-4 component stands out of the noise


def test_heavytail_has_two_means_and_no_byzantine_rows():
    w = si.WORKLOADS["cfg4"].scaled(60_000)
    G = si.generate(w).astype(np.float64)
    assert len(si.byzantine_positions(w)) == 0
    perm = si.row_permutation(w)
    second = np.nonzero(perm >= w.p - 4)[0]
    first = np.nonzero(perm < w.p - 4)[0]
    gap = G[second].mean(axis=0) - G[first].mean(axis=0)
    # shift variance 0.5 plus the noise of the two row means (t3 noise scaled 0.5 has variance 0.75)
    assert abs(np.mean(gap * gap) - (0.5 + 0.75 / 4 + 0.75 / 11)) < 0.1
    assert np.abs(G).max() > 20                 # Student-t(3) tails


def test_alie_rows_are_identical_bf16_and_below_the_mean():
    w = si.WORKLOADS["cfg5"].scaled(30_000)
    G = si.generate(w)
    assert G.dtype == np.uint16
    byz = si.byzantine_positions(w)
    assert len(byz) == 15 and all(np.array_equal(G[byz[0]], G[b]) for b in byz)
    X = si.to_float64(G)
    honest = np.delete(np.arange(w.p), byz)
    shift = X[honest].mean(axis=0) - X[byz[0]]
    assert abs(shift.mean() - 1.5 * 0.3) < 0.02


def test_bf16_rounding_matches_round_to_nearest_even():
    x = np.random.default_rng(0).standard_normal(100_000).astype(np.float32) * 37.0
    x[:4] = [1.0, 1.00390625, 1.01171875, -0.0]          # exact, tie to even (down), tie to even (up), signed zero
    bits = si.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = si.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy())


def test_ladder_cases_have_the_advertised_structure():
    G = si.ladder_case(7, 33, 3, "dup_zero")
    assert np.array_equal(G[0], G[1]) and not G[6].any()
    B = si.ladder_case(5, 64, 3, "gauss", bf16=True)
    assert B.dtype == np.uint16 and B.shape == (5, 64)
