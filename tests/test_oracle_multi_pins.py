"""Pins for the several-gradients-per-worker oracle (oracle/fa_multi.py).

Each check reaches the pinned quantity by a route that is not the oracle's own: the already pinned
single-gradient oracle, the objective typed out with traces from the appendix restatement, a
brute-force search over directions, finite differences, closed forms.
"""
import numpy as np
import pytest

from oracle import fa_multi as fm
from oracle import fa_oracle as fo


def rng(seed):
    return np.random.default_rng(seed)


def typed_objective(G, counts, Y, lam, a=2.0):
    """sum_i (1 - tr(Y^T g_i g_i^T Y)/tr(g_i^T g_i))^(1/a) + lam/(p-1) sum_{i!=j} (...)^(1/a) on worker means,
    with g_i the n x k_i matrix of worker i (appendix restatement of Eq. (5)), typed with traces."""
    p = len(counts)
    val, r0, means = 0.0, 0, []
    for k in counts:
        gi = G[r0:r0 + k].T                              # n x k_i
        r0 += k
        means.append(gi.mean(axis=1))
        tr = np.trace(gi.T @ gi)
        if tr > 0:
            val += max(1.0 - np.trace(Y.T @ gi @ gi.T @ Y) / tr, 0.0) ** (1.0 / a)
    if lam > 0 and p > 1:
        for i in range(p):
            for j in range(p):
                x = means[i] - means[j]
                if i != j and x @ x > 0:
                    val += lam / (p - 1) * max(1.0 - (Y.T @ x) @ (Y.T @ x) / (x @ x), 0.0) ** (1.0 / a)
    return val


def workers(counts, n, seed, sigma=0.5, outliers=1):
    r = rng(seed)
    mu = r.standard_normal(n)
    rows = []
    for i, k in enumerate(counts):
        centre = mu + 0.3 * r.standard_normal(n)
        block = centre[None, :] + sigma * r.standard_normal((k, n))
        if i >= len(counts) - outliers:
            block = 4.0 * r.standard_normal((k, n))
        rows.append(block * 10.0 ** r.uniform(-1, 1))
    return np.concatenate(rows, axis=0)


@pytest.mark.parametrize("lam,a", [(0.0, 2.0), (0.3, 2.0), (0.2, 3.0)])
def test_one_gradient_per_worker_is_the_single_gradient_method(lam, a):
    G = workers([1] * 9, 40, 1, outliers=2)
    one = fo.fa_aggregate(G, 4, lam, iters=7, a=a)
    many = fm.fa_aggregate_multi(G, [1] * 9, 4, lam, iters=7, a=a)
    assert fo.principal_angles(one["Y"], many["Y"]).max() < 1e-9
    assert np.allclose(one["objective"], many["objective"], rtol=1e-10, atol=1e-12)
    assert np.allclose(one["w"], many["w"], rtol=1e-8)
    assert fo.rel_l2(many["d"], one["d"]) < 1e-9


@pytest.mark.parametrize("lam,a", [(0.0, 2.0), (0.4, 2.0), (0.4, 1.5)])
def test_objective_matches_the_trace_form(lam, a):
    counts = [3, 1, 2, 4, 1]
    G = workers(counts, 17, 2)
    Y, _ = np.linalg.qr(rng(3).standard_normal((17, 3)))
    assert abs(fm.objective(G, counts, Y, lam, a) - typed_objective(G, counts, Y, lam, a)) < 1e-12
    out = fm.fa_aggregate_multi(G, counts, 3, lam, iters=4, a=a)
    # the typed form cancels in 1 - v; a rounding of 1e-16 under a root moves it by up to 1e-8
    assert abs(out["objective"][-1] - typed_objective(G, counts, out["Y"], lam, a)) < 1e-7


@pytest.mark.parametrize("seed,outliers", [(4, 0), (5, 1), (7, 1)])
def test_a_worker_that_repeats_one_gradient_scores_like_that_gradient(seed, outliers):
    """g_i = [g, g, g]: tr(Y^T g_i g_i^T Y)/tr(g_i^T g_i) = ||Y^T g||^2/||g||^2 and the mean is g, so the
    objective equals the single-gradient one for every Y and every reweighted round is the same map;
    only the uniform first round differs, so on data with one basin the fixed points coincide."""
    single = workers([1] * 6, 15, seed, outliers=outliers)
    counts = [3, 1, 2, 1, 4, 1]
    G = np.concatenate([np.repeat(single[i:i + 1], k, axis=0) for i, k in enumerate(counts)], axis=0)
    for seed in range(3):
        Y, _ = np.linalg.qr(rng(seed).standard_normal((15, 2)))
        assert abs(fm.objective(G, counts, Y, 0.3) - fo.objective(single, Y, 0.3)) < 1e-12
    many = fm.fa_aggregate_multi(G, counts, 2, 0.3, iters=300)
    one = fo.fa_aggregate(single, 2, 0.3, iters=300)
    assert fo.principal_angles(one["Y"], many["Y"]).max() < 1e-6
    assert fo.rel_l2(many["d"], one["d"]) < 1e-6
    assert np.allclose(many["w"] * np.asarray(counts), one["w"], rtol=1e-5)


def test_mixing_a_workers_gradients_orthogonally_changes_nothing_without_regulariser():
    counts = [3, 2, 4, 1]
    G = workers(counts, 20, 5)
    H = G.copy()
    r0 = 0
    for k in counts:
        Q, _ = np.linalg.qr(rng(k).standard_normal((k, k)))
        H[r0:r0 + k] = Q @ G[r0:r0 + k]
        r0 += k
    a = fm.fa_aggregate_multi(G, counts, 3, 0.0, iters=6)
    b = fm.fa_aggregate_multi(H, counts, 3, 0.0, iters=6)
    assert fo.principal_angles(a["Y"], b["Y"]).max() < 1e-9
    assert np.allclose(a["objective"], b["objective"], rtol=1e-10)
    assert np.allclose(a["w"], b["w"], rtol=1e-8)


@pytest.mark.parametrize("lam,a,seed", [(0.0, 2.0, 6), (0.5, 2.0, 7), (3.0, 2.0, 8), (0.3, 3.0, 9)])
def test_monotone_descent(lam, a, seed):
    counts = [2, 3, 1, 4, 2, 1, 3]
    G = workers(counts, 30, seed, outliers=2)
    objs = fm.fa_aggregate_multi(G, counts, 4, lam, iters=25, a=a)["objective"]
    # round one is plain PCA; from then on every round minimises a majoriser of the objective
    assert all(objs[t + 1] <= objs[t] + 1e-10 for t in range(len(objs) - 1))
    assert objs[-1] < objs[0]


@pytest.mark.parametrize("lam,seed", [(0.0, 10), (0.4, 11)])
def test_fixed_point_is_a_local_minimum_of_the_trace_objective(lam, seed):
    counts = [2, 1, 3, 2, 1, 2]
    n, m = 12, 3
    G = workers(counts, n, seed, outliers=1)
    Y = fm.fa_aggregate_multi(G, counts, m, lam, iters=500)["Y"]
    base = typed_objective(G, counts, Y, lam)
    r = rng(seed + 50)
    worst = 0.0
    for _ in range(60):
        D = r.standard_normal((n, m))
        D -= Y @ (Y.T @ D)
        D /= np.linalg.norm(D)
        for t in (1e-2, 1e-3, 1e-4):
            Q, _ = np.linalg.qr(Y + t * D)
            worst = max(worst, (base - typed_objective(G, counts, Q, lam)) / t)
    assert worst < 1e-5
    # plain PCA of the same rows is not a minimiser: the probe finds descent there
    Ypca = fm.fa_aggregate_multi(G, counts, m, lam, iters=1)["Y"]
    b0 = typed_objective(G, counts, Ypca, lam)
    best = 0.0
    for _ in range(60):
        D = r.standard_normal((n, m))
        D -= Ypca @ (Ypca.T @ D)
        D /= np.linalg.norm(D)
        Q, _ = np.linalg.qr(Ypca + 1e-3 * D)
        best = max(best, (b0 - typed_objective(G, counts, Q, lam)) / 1e-3)
    assert best > 1e-3


@pytest.mark.parametrize("lam", [0.0, 0.3])
def test_brute_force_lines_in_the_plane(lam):
    counts = [2, 3, 1, 2, 2]
    r = rng(12)
    mu = r.standard_normal(2)
    G = np.concatenate([mu[None, :] * r.uniform(0.5, 2.0) + 0.2 * r.standard_normal((k, 2)) for k in counts])
    G[-2:] = 2.0 * r.standard_normal((2, 2))
    out = fm.fa_aggregate_multi(G, counts, 1, lam, iters=300)
    k = 6000
    ang = (np.arange(k) + 0.5) * np.pi / k
    values = [typed_objective(G, counts, np.array([[np.cos(t)], [np.sin(t)]]), lam) for t in ang]
    # the iteration stops at a local minimum: it must be one of the grid's local minima
    vals = np.asarray(values)
    is_min = (vals <= np.roll(vals, 1)) & (vals <= np.roll(vals, -1))
    p = len(counts)
    resolution = (np.pi / k) * (p + 2 * lam * p) + 1e-9
    assert np.min(np.abs(vals[is_min] - out["objective"][-1])) < resolution
    assert out["objective"][-1] <= vals.min() + 0.35 * (vals.max() - vals.min())


def test_mean_recovery_and_full_dimension():
    counts = [2, 3, 1]
    g = rng(13).standard_normal(9)
    G = np.repeat(g[None, :], 6, axis=0) * np.array([1, 2, 3, 0.5, 1, 4.0])[:, None]
    out = fm.fa_aggregate_multi(G, counts, 1, 0.2, iters=5)
    means = fm.worker_means(G, counts)
    assert fo.rel_l2(out["d"], means.mean(axis=0)) < 1e-12      # everything lies on one line
    H = workers(counts, 6, 14, outliers=0)
    full = fm.fa_aggregate_multi(H, counts, 6, 0.1, iters=5)
    assert fo.rel_l2(full["d"], fm.worker_means(H, counts).mean(axis=0)) < 1e-10
    assert max(abs(x) for x in full["objective"]) < 1e-6


def test_zero_worker_identical_means_and_argument_checks():
    counts = [2, 2, 2, 1]
    G = workers(counts, 10, 15, outliers=0)
    G[2:4] = 0.0                                   # worker 1 hands in nothing
    G[4:6] = G[0:2][::-1]                          # worker 2 has worker 0's gradients: same mean
    out = fm.fa_aggregate_multi(G, counts, 2, 0.5, iters=6)
    assert out["w"][1] == 0.0 and out["u"][1] == 0.0
    assert np.isfinite(out["d"]).all() and np.isfinite(out["objective"]).all()
    assert abs(out["objective"][-1] - typed_objective(G, counts, out["Y"], 0.5)) < 1e-7
    with pytest.raises(ValueError):
        fm.fa_aggregate_multi(G, [2, 2, 2], 2)
    with pytest.raises(ValueError):
        fm.fa_aggregate_multi(G, [7, 0], 2)
    zero = fm.fa_aggregate_multi(np.zeros((3, 5)), [2, 1], 1, 0.1, iters=2)
    assert not zero["d"].any() and zero["Y"].shape == (5, 0)
