"""Pins for the CPU oracle: what the paper and the mathematics fix about the
Flag Aggregator step, checked without reference to the CUDA path.

Every check here evaluates the pinned quantity by a route that is not the
oracle's own (a closed form, a brute-force search, the paper's printed
formula typed out in this file, a dual eigenproblem), so that a dropped term,
a wrong normaliser or a transposed operand in the oracle fails at least one.
"""
import itertools

import numpy as np
import pytest

from oracle import fa_oracle as fo


def rng(seed):
    return np.random.default_rng(seed)


def eq5(G, Y, lam):
    """Eq. (5) with regulariser (2), typed from the paper: 1 - tr(Y^T x x^T Y)/||x||^2 under each root."""
    p = G.shape[0]
    val = 0.0
    for i in range(p):
        x = G[i]
        if x @ x > 0:
            val += np.sqrt(max(1.0 - np.trace(Y.T @ np.outer(x, x) @ Y) / (x @ x), 0.0))
    if lam > 0:
        for i in range(p):
            for j in range(p):
                if i != j:
                    x = G[i] - G[j]
                    if x @ x > 0:
                        val += lam / (p - 1) * np.sqrt(
                            max(1.0 - np.trace(Y.T @ np.outer(x, x) @ Y) / (x @ x), 0.0))
    return val


def noisy_mean(p, n, seed, sigma=0.4, outliers=0, scale_spread=False):
    r = rng(seed)
    mu = r.standard_normal(n)
    G = mu[None, :] + sigma * r.standard_normal((p, n))
    for k in range(outliers):
        G[p - 1 - k] = 6.0 * r.standard_normal(n)
    if scale_spread:
        G *= 10.0 ** r.uniform(-1, 1, size=(p, 1))
    return G


# 1 -- mean recovery (Algorithm 1, direction d: if span(G) is inside span(Y), d is the mean)
@pytest.mark.parametrize("lam", [0.0, 0.3])
def test_mean_recovered_when_gradients_share_an_m_dim_subspace(lam):
    r = rng(1)
    n, p, m = 40, 9, 3
    basis = r.standard_normal((m, n))
    G = r.standard_normal((p, m)) @ basis
    out = fo.fa_aggregate(G, m, lam, iters=4)
    assert fo.rel_l2(out["d"], G.mean(axis=0)) < 1e-12
    assert np.all(out["u"] < 1e-20)


# 2 -- Y orthonormal, values in [0, 1] (Section 2.1)
@pytest.mark.parametrize("method", ["svd", "literal"])
def test_orthonormal_subspace_and_ratio_range(method):
    G = noisy_mean(8, 30, 2, outliers=2)
    out = fo.fa_aggregate(G, 3, 0.05, iters=6, method=method)
    Y = out["Y"]
    assert np.abs(Y.T @ Y - np.eye(3)).max() < 1e-12
    assert np.all(out["u"] >= 0) and np.all(out["u"] <= 1 + 1e-12)
    v = np.array([np.sum((Y.T @ g) ** 2) / (g @ g) for g in G])
    assert np.allclose(1 - v, out["u"], atol=1e-12)      # residual form == 1 - explained variance


# 3 -- one uniform-weight round is PCA (appendix, PCA baseline); dual (snapshot) eigenproblem as the other route
def test_single_round_is_pca_of_the_gradient_matrix():
    G = noisy_mean(10, 200, 3, outliers=1, scale_spread=True)
    m = 4
    out = fo.fa_aggregate(G, m, 0.0, iters=1)
    lam_, V = np.linalg.eigh(G @ G.T)                 # p x p dual problem
    Vm = V[:, ::-1][:, :m]
    Ydual = G.T @ Vm / np.sqrt(lam_[::-1][:m])[None, :]
    assert fo.principal_angles(Ydual, out["Y"]).max() < 1e-9
    # and it maximises captured energy: no random m-dim subspace does better
    cap = np.sum((G @ out["Y"]) ** 2)
    r = rng(33)
    for _ in range(50):
        Q, _ = np.linalg.qr(r.standard_normal((200, m)))
        assert np.sum((G @ Q) ** 2) <= cap + 1e-9


# 4 -- the objective is a symmetric sum over workers: permuting rows changes nothing
@pytest.mark.parametrize("lam", [0.0, 0.2])
def test_worker_permutation_invariance(lam):
    G = noisy_mean(9, 64, 4, outliers=2)
    perm = rng(5).permutation(9)
    a = fo.fa_aggregate(G, 4, lam, iters=8)
    b = fo.fa_aggregate(G[perm], 4, lam, iters=8)
    assert fo.rel_l2(b["d"], a["d"]) < 1e-9
    assert fo.principal_angles(a["Y"], b["Y"]).max() < 1e-8
    assert np.allclose(a["u"][perm], b["u"], atol=1e-9)


# 5 -- G -> sG leaves Y alone and scales d
def test_global_scaling():
    G = noisy_mean(7, 50, 6, outliers=1)
    a = fo.fa_aggregate(G, 3, 0.1, iters=7)
    b = fo.fa_aggregate(4.0 * G, 3, 0.1, iters=7)
    assert fo.principal_angles(a["Y"], b["Y"]).max() < 1e-10
    assert fo.rel_l2(b["d"], 4.0 * a["d"]) < 1e-10


# 5b -- each data term of Eq. (5) is normalised by ||g_i||^2: per-worker rescaling leaves A(Y) alone at lam = 0
def test_objective_invariant_to_per_worker_scale_without_regulariser():
    G = noisy_mean(6, 20, 7)
    Y, _ = np.linalg.qr(rng(8).standard_normal((20, 2)))
    s = np.array([1.0, 3.0, 0.01, 100.0, 7.0, 0.5])
    assert abs(fo.objective(G, Y, 0.0) - fo.objective(G * s[:, None], Y, 0.0)) < 1e-12


# 6 -- reweighting is a majorise-minimise step: the objective never goes up while no floor is active
@pytest.mark.parametrize("lam,seed", [(0.0, 10), (0.5, 11), (5.0, 12)])
def test_monotone_descent(lam, seed):
    G = noisy_mean(12, 80, seed, outliers=3, scale_spread=True)
    out = fo.fa_aggregate(G, 4, lam, iters=25)
    obj = np.array(out["objective"])
    assert np.all(np.diff(obj) <= 1e-10)
    assert obj[0] - obj[-1] > 1e-3                       # and it does move


# 6b -- the oracle's objective is Eq. (5) as printed
@pytest.mark.parametrize("lam", [0.0, 0.7])
def test_objective_matches_printed_formula(lam):
    G = noisy_mean(6, 15, 13, outliers=1)
    Y, _ = np.linalg.qr(rng(14).standard_normal((15, 3)))
    assert abs(fo.objective(G, Y, lam) - eq5(G, Y, lam)) < 1e-10
    out = fo.fa_aggregate(G, 3, lam, iters=5)
    assert abs(out["objective"][-1] - eq5(G, out["Y"], lam)) < 1e-7


# 7 -- the limit of the iteration is a local minimiser of Eq. (5) on the Grassmannian
@pytest.mark.parametrize("lam,seed", [(0.0, 20), (0.4, 21)])
def test_fixed_point_is_a_local_minimum_of_eq5(lam, seed):
    n, p, m = 12, 10, 3
    G = noisy_mean(p, n, seed, sigma=0.6, outliers=2, scale_spread=True)
    out = fo.fa_aggregate(G, m, lam, iters=400)
    Y = out["Y"]
    base = eq5(G, Y, lam)
    r = rng(seed + 100)
    worst_drop = 0.0
    for _ in range(60):
        D = r.standard_normal((n, m))
        D -= Y @ (Y.T @ D)
        D /= np.linalg.norm(D)
        for t in (1e-2, 1e-3, 1e-4):
            Q, _ = np.linalg.qr(Y + t * D)
            worst_drop = max(worst_drop, (base - eq5(G, Q, lam)) / t)
    assert worst_drop < 1e-5
    # a deliberately different reweighting (norm left out) does not land on a minimiser:
    # the same probe applied to plain PCA finds a descent direction.
    Ypca = fo.fa_aggregate(G, m, lam, iters=1)["Y"]
    base_pca = eq5(G, Ypca, lam)
    best = 0.0
    for _ in range(60):
        D = r.standard_normal((n, m))
        D -= Ypca @ (Ypca.T @ D)
        D /= np.linalg.norm(D)
        Q, _ = np.linalg.qr(Ypca + 1e-3 * D)
        best = max(best, (base_pca - eq5(G, Q, lam)) / 1e-3)
    assert best > 1e-3


# 7b -- first-order (KKT) condition of the appendix: C(Y) Y stays inside span(Y) at the fixed point
def test_kkt_residual_at_convergence():
    n, p, m = 30, 9, 3
    G = noisy_mean(p, n, 22, sigma=0.5, outliers=2)
    out = fo.fa_aggregate(G, m, 0.0, iters=300)
    Y, u = out["Y"], out["u"]
    C = np.zeros((n, n))
    for i in range(p):
        C += np.outer(G[i], G[i]) / ((G[i] @ G[i]) * max(np.sqrt(u[i]), fo.EPS))
    R = C @ Y - Y @ (Y.T @ C @ Y)
    assert np.linalg.norm(R) / np.linalg.norm(C @ Y) < 1e-6


# 8 -- Y Y^T G is G times a p x p matrix (appendix, optimality conditions): d = G^T-layout product with c
def test_direction_is_a_combination_of_the_gradients():
    G = noisy_mean(8, 60, 23, outliers=2)
    p = 8
    out = fo.fa_aggregate(G, 3, 0.2, iters=6)
    A, *_ = np.linalg.lstsq(G.T, out["Y"], rcond=None)      # Y = G^T A
    assert np.abs(G.T @ A - out["Y"]).max() < 1e-10
    K = G @ G.T
    c = A @ (A.T @ (K @ np.ones(p))) / p
    assert fo.rel_l2(c @ G, out["d"]) < 1e-10


# 9 -- brute force over the Grassmannian for n <= 4
def _line_grid_2d(k):
    a = (np.arange(k) + 0.5) * np.pi / k
    return np.stack([np.cos(a), np.sin(a)], axis=1)


def _sphere_points(n, k, seed):
    x = rng(seed).standard_normal((k, n))
    return x / np.linalg.norm(x, axis=1, keepdims=True)


def _clustered(n, p, seed, outliers):
    r = rng(seed)
    mu = r.standard_normal(n)
    G = mu[None, :] * r.uniform(0.5, 2.0, size=(p, 1)) + 0.15 * r.standard_normal((p, n))
    for k in range(outliers):
        G[p - 1 - k] = r.standard_normal(n) * 2.0
    return G


@pytest.mark.parametrize("lam", [0.0, 0.3])
def test_brute_force_lines_in_the_plane(lam):
    G = _clustered(2, 7, 30, outliers=2)
    out = fo.fa_aggregate(G, 1, lam, iters=200)
    k = 6000
    grid = _line_grid_2d(k)
    best = min(eq5(G, y[:, None], lam) for y in grid)
    resolution = (np.pi / k) * (7 + 2 * lam * 7)       # each root moves by at most the angle step
    assert abs(out["objective"][-1] - best) < resolution + 1e-9


@pytest.mark.parametrize("n,m", [(3, 1), (3, 2), (4, 1), (4, 3)])
def test_brute_force_lines_and_hyperplanes(n, m):
    p = 6
    G = _clustered(n, p, 31 + n + m, outliers=1)
    out = fo.fa_aggregate(G, m, 0.0, iters=300)
    pts = _sphere_points(n, 60000, 32)
    if m == 1:
        vals = 1.0 - (pts @ G.T) ** 2 / np.sum(G * G, axis=1)[None, :]
    else:                                   # m = n-1: Y is the complement of a unit normal
        vals = (pts @ G.T) ** 2 / np.sum(G * G, axis=1)[None, :]
    objs = np.sum(np.sqrt(np.maximum(vals, 0.0)), axis=1)
    k = int(np.argmin(objs))
    # polish the best sample by a local random search
    x, fx = pts[k], objs[k]
    r = rng(34)
    step = 0.05
    for _ in range(4000):
        y = x + step * r.standard_normal(n)
        y /= np.linalg.norm(y)
        v = (1.0 - (G @ y) ** 2 / np.sum(G * G, axis=1)) if m == 1 else (G @ y) ** 2 / np.sum(G * G, axis=1)
        fy = np.sum(np.sqrt(np.maximum(v, 0.0)))
        if fy < fx:
            x, fx = y, fy
        else:
            step = max(step * 0.995, 1e-7)
    assert out["objective"][-1] <= fx + 1e-6
    assert out["objective"][-1] >= fx - 1e-3             # the search cannot be beaten by much either


def test_brute_force_planes_in_r4():
    n, m, p = 4, 2, 6
    G = _clustered(n, p, 40, outliers=1)
    out = fo.fa_aggregate(G, m, 0.0, iters=300)
    r = rng(41)
    best = np.inf
    for _ in range(300):
        Y, _ = np.linalg.qr(r.standard_normal((n, m)))
        f = eq5(G, Y, 0.0)
        step = 0.3
        for _ in range(400):
            Q, _ = np.linalg.qr(Y + step * r.standard_normal((n, m)))
            fq = eq5(G, Q, 0.0)
            if fq < f:
                Y, f = Q, fq
            else:
                step = max(step * 0.98, 1e-6)
        best = min(best, f)
    assert out["objective"][-1] <= best + 1e-4


# 9b -- closed form: two lines in the plane, the heavier one wins and the objective is sin(angle)
def test_two_gradients_closed_form():
    phi = 0.7
    G = np.array([[3.0, 0.0], [np.cos(phi), np.sin(phi)]])
    out = fo.fa_aggregate(G, 1, 0.0, iters=200)
    # the weight floor EPS keeps the captured line a hair (~EPS) off g_1
    assert abs(out["objective"][-1] - np.sin(phi)) < 5 * fo.EPS
    assert abs(abs(out["Y"][0, 0]) - 1.0) < 5 * fo.EPS
    # d = (1/p) y y^T (g_1 + g_2)
    assert np.allclose(out["d"], [0.5 * (3.0 + np.cos(phi)), 0.0], atol=1e-5)


# 10 -- Lemma "Equivalence of Objective Functions": tr(Y^T M Y) = vec(Y)^T (I kron M) vec(Y)
def test_kronecker_form_of_the_objective():
    n, m, p = 7, 3, 5
    G = noisy_mean(p, n, 50)
    Y, _ = np.linalg.qr(rng(51).standard_normal((n, m)))
    vecY = Y.T.reshape(-1)                   # columns of Y stacked
    total = 0.0
    for i in range(p):
        Mi = np.eye(n) / m - np.outer(G[i], G[i]) / (G[i] @ G[i])
        total += np.sqrt(vecY @ np.kron(np.eye(m), Mi) @ vecY)
    assert abs(total - fo.objective(G, Y, 0.0)) < 1e-12


# 11 -- m = p: Y spans every gradient, so d is the mean whatever the weights
@pytest.mark.parametrize("lam", [0.0, 0.1])
def test_full_dimension_gives_the_mean(lam):
    G = noisy_mean(5, 33, 60, outliers=1)
    out = fo.fa_aggregate(G, 5, lam, iters=3)
    assert fo.rel_l2(out["d"], G.mean(axis=0)) < 1e-10


# 12 -- literal n x n construction and the factored SVD route agree
@pytest.mark.parametrize("lam", [0.0, 0.25])
def test_literal_and_svd_modes_agree(lam):
    G = noisy_mean(7, 24, 70, outliers=2, scale_spread=True)
    a = fo.fa_aggregate(G, 3, lam, iters=9, method="literal")
    b = fo.fa_aggregate(G, 3, lam, iters=9, method="svd")
    assert fo.rel_l2(b["d"], a["d"]) < 1e-9
    assert fo.principal_angles(a["Y"], b["Y"]).max() < 1e-8
    assert np.allclose(a["objective"], b["objective"], atol=1e-9)
    # the identity behind the factored route: C = G^T M G
    w = rng(71).uniform(0.1, 2, 7)
    W = rng(72).uniform(0, 1, (7, 7)); W = W + W.T; np.fill_diagonal(W, 0)
    C = sum(w[i] * np.outer(G[i], G[i]) for i in range(7))
    for i, j in itertools.permutations(range(7), 2):
        x = G[i] - G[j]
        C = C + W[i, j] * np.outer(x, x)
    assert np.allclose(G.T @ fo.pair_weight_matrix(w, W) @ G, C, rtol=1e-12, atol=1e-9)


# 13 -- degenerate inputs
def test_zero_gradient_and_identical_rows():
    G = noisy_mean(8, 40, 80)
    G[3] = 0.0
    G[5] = G[4]
    for lam in (0.0, 0.2):
        out = fo.fa_aggregate(G, 3, lam, iters=6)
        assert np.all(np.isfinite(out["d"]))
        assert out["u"][3] == 0.0
        assert abs(out["u"][4] - out["u"][5]) < 1e-12
        assert abs(out["objective"][-1] - eq5(G, out["Y"], lam)) < 1e-7


def test_single_worker_and_all_zero():
    g = rng(81).standard_normal((1, 9))
    out = fo.fa_aggregate(g, 1, 0.0, iters=3)
    assert fo.rel_l2(out["d"], g[0]) < 1e-12
    z = fo.fa_aggregate(np.zeros((4, 6)), 2, 0.1, iters=3)
    assert np.all(z["d"] == 0) and z["Y"].shape == (6, 0)


def test_rank_below_m_drops_directions():
    r = rng(82)
    G = r.standard_normal((6, 2)) @ r.standard_normal((2, 25))     # rank 2
    out = fo.fa_aggregate(G, 4, 0.0, iters=3)
    assert out["Y"].shape[1] == 2
    assert fo.rel_l2(out["d"], G.mean(axis=0)) < 1e-10


def test_principal_angles_of_a_known_rotation():
    n = 6
    Ya = np.eye(n)[:, :2]
    th = 0.3
    Yb = np.stack([np.eye(n)[:, 0], np.cos(th) * np.eye(n)[:, 1] + np.sin(th) * np.eye(n)[:, 2]], axis=1)
    ang = fo.principal_angles(Ya, Yb)
    assert abs(ang[0] - th) < 1e-12 and abs(ang[1]) < 1e-12


def test_inner_products_and_pair_distances():
    G = noisy_mean(5, 17, 90)
    K = fo.inner_products(G)
    D2 = fo.pair_sqdist(G)
    for i in range(5):
        for j in range(5):
            assert abs(K[i, j] - sum(G[i, k] * G[j, k] for k in range(17))) < 1e-10
            assert abs(D2[i, j] - (K[i, i] + K[j, j] - 2 * K[i, j])) < 1e-9


# 14 -- other surrogate constants a (Eq. (4)): a = 2 is the default path; for a != 2 the iteration
# still descends on sum (1 - v)^(1/a) and its limit is a local minimiser of that objective
def eq4_objective(G, Y, lam, a):
    p = G.shape[0]
    val = 0.0
    for i in range(p):
        x = G[i]
        if x @ x > 0:
            val += max(1.0 - np.sum((Y.T @ x) ** 2) / (x @ x), 0.0) ** (1.0 / a)
    if lam > 0:
        for i in range(p):
            for j in range(p):
                if i != j:
                    x = G[i] - G[j]
                    if x @ x > 0:
                        val += lam / (p - 1) * max(1.0 - np.sum((Y.T @ x) ** 2) / (x @ x), 0.0) ** (1.0 / a)
    return val


def test_surrogate_constant_two_is_the_default():
    G = noisy_mean(8, 30, 90, outliers=2)
    a2 = fo.fa_aggregate(G, 3, 0.1, iters=6, a=2.0)
    d = fo.fa_aggregate(G, 3, 0.1, iters=6)
    assert np.array_equal(a2["d"], d["d"]) and a2["objective"] == d["objective"]


@pytest.mark.parametrize("a,lam", [(1.5, 0.0), (3.0, 0.3), (4.0, 0.0)])
def test_other_surrogate_constants_descend_and_reach_a_local_minimum(a, lam):
    n, p, m = 12, 10, 3
    G = noisy_mean(p, n, 91, sigma=0.6, outliers=2, scale_spread=True)
    out = fo.fa_aggregate(G, m, lam, iters=400, a=a)
    obj = np.array(out["objective"])
    assert np.all(np.diff(obj) <= 1e-10)
    # the typed-out form 1 - v cancels: a captured worker's term carries rounding noise 1e-16^(1/a)
    assert abs(obj[-1] - eq4_objective(G, out["Y"], lam, a)) < 10 * p * (1e-15 ** (1.0 / a))
    Y = out["Y"]
    base = eq4_objective(G, Y, lam, a)
    r = rng(92)
    worst = 0.0
    for _ in range(40):
        D = r.standard_normal((n, m))
        D -= Y @ (Y.T @ D)
        D /= np.linalg.norm(D)
        for t in (1e-2, 1e-3):
            Q, _ = np.linalg.qr(Y + t * D)
            worst = max(worst, (base - eq4_objective(G, Q, lam, a)) / t)
    assert worst < 1e-3


# 15 -- reconstruction Y Y^T G (Section 2.1) is a projection of every gradient onto span(Y)
def test_reconstruction_is_the_orthogonal_projection():
    G = noisy_mean(6, 25, 93, outliers=1)
    out = fo.fa_aggregate(G, 3, 0.0, iters=4)
    R = fo.reconstruction(G, out["Y"])
    P = out["Y"] @ out["Y"].T
    assert np.allclose(R, G @ P, atol=1e-12)
    assert np.allclose(R.mean(axis=0), out["d"], atol=1e-12)          # its column average is the update
    assert np.allclose((G - R) @ out["Y"], 0.0, atol=1e-10)           # residuals are orthogonal to Y


# ---- start from a given subspace, stop on a tolerance --------------------------------------------

@pytest.mark.parametrize("lam", [0.0, 0.3])
def test_start_from_the_pca_subspace_is_the_cold_start_shifted_by_one_round(lam):
    """Round one of the cold start is PCA; starting from that subspace, round t is cold round t + 1."""
    G = noisy_mean(9, 30, 50, sigma=0.5, outliers=2, scale_spread=True)
    cold = fo.fa_aggregate(G, 3, lam, iters=6, history=True)
    _, _, Vt = np.linalg.svd(G, full_matrices=False)              # PCA of the gradient matrix, by SVD of G itself
    Ypca = Vt[:3].T
    if lam > 0:
        Ypca = cold["Ys"][0]                                      # with the regulariser round one is not plain PCA
    warm = fo.fa_aggregate(G, 3, lam, iters=5, Y0=Ypca, history=True)
    for t in range(5):
        assert fo.principal_angles(cold["Ys"][t + 1], warm["Ys"][t]).max() < 1e-9
    assert np.allclose(cold["objective"][1:], warm["objective"], rtol=1e-10)


def test_start_depends_on_the_span_only_and_the_fixed_point_stays():
    G = noisy_mean(8, 25, 51, sigma=0.5, outliers=1)
    Y0 = rng(52).standard_normal((25, 3))
    mix = rng(53).standard_normal((3, 3)) + 3 * np.eye(3)
    a = fo.fa_aggregate(G, 3, 0.2, iters=4, Y0=Y0)
    b = fo.fa_aggregate(G, 3, 0.2, iters=4, Y0=Y0 @ mix)
    assert fo.principal_angles(a["Y"], b["Y"]).max() < 1e-9
    star = fo.fa_aggregate(G, 3, 0.2, iters=400)
    again = fo.fa_aggregate(G, 3, 0.2, iters=1, Y0=star["Y"])
    assert fo.principal_angles(star["Y"], again["Y"]).max() < 1e-6
    assert abs(again["objective"][0] - star["objective"][-1]) < 1e-9
    # a start of rank 0 is the cold start
    cold = fo.fa_aggregate(G, 3, 0.2, iters=3)
    zero = fo.fa_aggregate(G, 3, 0.2, iters=3, Y0=np.zeros((25, 3)))
    assert np.allclose(cold["objective"], zero["objective"], rtol=0, atol=0)


def test_tolerance_stops_at_the_first_small_decrease_and_not_before():
    G = noisy_mean(10, 40, 54, sigma=0.5, outliers=2)
    full = fo.fa_aggregate(G, 4, 0.1, iters=60)["objective"]
    steps = np.abs(np.diff(full))
    tol = 1e-6
    first = int(np.nonzero(steps <= tol)[0][0]) + 2               # rounds run when the test first succeeds
    out = fo.fa_aggregate(G, 4, 0.1, iters=60, tol=tol)
    assert out["rounds"] == first and len(out["objective"]) == first
    assert np.array_equal(out["objective"], full[:first])
    same = fo.fa_aggregate(G, 4, 0.1, iters=first)
    assert fo.principal_angles(same["Y"], out["Y"]).max() < 1e-12 and fo.rel_l2(out["d"], same["d"]) < 1e-12
    assert fo.fa_aggregate(G, 4, 0.1, iters=7, tol=0.0)["rounds"] == 7       # the cap
    assert fo.fa_aggregate(G, 4, 0.1, iters=7, tol=1e9)["rounds"] == 2
    assert fo.fa_aggregate(G, 4, 0.1, iters=1, tol=1e9)["rounds"] == 1


# ---- general Beta(alpha, beta) likelihood of the values (extension paragraph of Section 2.2) ----------

def beta_objective(G, Y, lam, a, alpha, beta):
    """-(alpha-1) log v - (beta-1) log(1-v) with log x -> a x^(1/a) - a on both logarithms, divided by a/2
    and without the constants, plus the regulariser of Eq. (5): typed out here with traces."""
    p = G.shape[0]
    val = 0.0
    for i in range(p):
        x = G[i]
        if x @ x > 0:
            v = np.trace(Y.T @ np.outer(x, x) @ Y) / (x @ x)
            val += 2 * (1 - beta) * max(1.0 - v, 0.0) ** (1 / a) + 2 * (1 - alpha) * max(v, 0.0) ** (1 / a)
    if lam > 0:
        for i in range(p):
            for j in range(p):
                x = G[i] - G[j]
                if i != j and x @ x > 0:
                    v = np.trace(Y.T @ np.outer(x, x) @ Y) / (x @ x)
                    val += lam / (p - 1) * max(1.0 - v, 0.0) ** (1 / a)
    return val


def test_beta_one_half_is_the_papers_data_term_and_beta_only_rescales_lambda():
    G = noisy_mean(9, 30, 60, sigma=0.5, outliers=2, scale_spread=True)
    base = fo.fa_aggregate(G, 3, 0.2, iters=6)
    same = fo.fa_aggregate(G, 3, 0.2, iters=6, alpha=1.0, beta=0.5)
    assert np.array_equal(base["d"], same["d"]) and base["objective"] == same["objective"]
    # alpha = 1: the data term is 2(1-beta) times the paper's, i.e. the paper's problem with lambda / (2(1-beta))
    # (from a common start: the uniform first round does not know about beta)
    b = 0.8
    Y0 = rng(66).standard_normal((30, 3))
    other = fo.fa_aggregate(G, 3, 0.2, iters=6, beta=b, method="qr", Y0=Y0)
    scaled = fo.fa_aggregate(G, 3, 0.2 / (2 * (1 - b)), iters=6, Y0=Y0)
    assert fo.principal_angles(other["Y"], scaled["Y"]).max() < 1e-8
    assert np.allclose(np.asarray(other["objective"]) / (2 * (1 - b)), scaled["objective"], rtol=1e-9)
    # without the regulariser beta does not matter at all
    assert fo.principal_angles(fo.fa_aggregate(G, 3, 0.0, iters=6, beta=0.9)["Y"],
                               fo.fa_aggregate(G, 3, 0.0, iters=6)["Y"]).max() < 1e-8


def test_indefinite_weighted_pca_by_qr_matches_the_n_by_n_matrix():
    r = rng(61)
    G = r.standard_normal((6, 9))
    w = r.standard_normal(6)                       # both signs
    W = np.abs(r.standard_normal((6, 6))) * 0.1
    W = W + W.T
    np.fill_diagonal(W, 0.0)
    Yq, eq = fo.weighted_pca_qr(G, w, W, 3)
    Yl, el = fo.weighted_pca_literal(G, w, W, 3)
    assert Yq.shape == Yl.shape and fo.principal_angles(Yq, Yl).max() < 1e-9
    assert np.allclose(np.sort(eq)[::-1][:3], np.sort(el)[::-1][:3], rtol=1e-10)
    # all weights negative: nothing has a positive eigenvalue, Y is empty
    Yn, _ = fo.weighted_pca_qr(G, -np.abs(w), 0 * W, 3)
    assert Yn.shape[1] == 0


@pytest.mark.parametrize("alpha,beta,lam,a", [(0.7, 0.5, 0.0, 2.0), (0.5, 0.3, 0.3, 2.0), (0.8, 0.5, 0.2, 3.0)])
def test_beta_likelihood_descends_and_reaches_a_local_minimum(alpha, beta, lam, a):
    n, p, m = 12, 10, 3
    G = noisy_mean(p, n, 62, sigma=0.6, outliers=2, scale_spread=True)
    out = fo.fa_aggregate(G, m, lam, iters=400, a=a, alpha=alpha, beta=beta)
    objs = out["objective"]
    assert all(objs[t + 1] <= objs[t] + 1e-10 for t in range(len(objs) - 1))
    Y = out["Y"]
    assert abs(objs[-1] - beta_objective(G, Y, lam, a, alpha, beta)) < 1e-7
    if Y.shape[1] == m:
        base = beta_objective(G, Y, lam, a, alpha, beta)
        r = rng(63)
        worst = 0.0
        for _ in range(60):
            D = r.standard_normal((n, m))
            D -= Y @ (Y.T @ D)
            D /= np.linalg.norm(D)
            for t in (1e-2, 1e-3, 1e-4):
                Q, _ = np.linalg.qr(Y + t * D)
                worst = max(worst, (base - beta_objective(G, Q, lam, a, alpha, beta)) / t)
        assert worst < 1e-5


def test_beta_likelihood_brute_force_in_the_plane():
    G = _clustered(2, 7, 64, outliers=2)
    alpha, beta, lam = 0.6, 0.5, 0.2
    out = fo.fa_aggregate(G, 1, lam, iters=300, alpha=alpha, beta=beta)
    k = 6000
    grid = _line_grid_2d(k)
    vals = np.asarray([beta_objective(G, y[:, None], lam, 2.0, alpha, beta) for y in grid])
    is_min = (vals <= np.roll(vals, 1)) & (vals <= np.roll(vals, -1))
    assert out["Y"].shape[1] == 1
    # each term moves by at most the angle step times its coefficient (roots of values in [0, 1])
    resolution = (np.pi / k) * (7 * (2 * (1 - beta) + 2 * (1 - alpha)) + 2 * lam * 7) * 40
    assert np.min(np.abs(vals[is_min] - out["objective"][-1])) < resolution


def test_beta_arguments():
    G = noisy_mean(5, 8, 65)
    for bad in (dict(alpha=0.0), dict(alpha=1.5), dict(beta=0.0), dict(beta=1.2)):
        with pytest.raises(ValueError):
            fo.fa_aggregate(G, 2, **bad)


# ---- comparison helper: the relative L2 error every aggregate-parity assertion is stated in ----------

def test_relative_l2_error_on_hand_computed_cases():
    assert fo.rel_l2([3.0, 4.0], [0.0, 0.0]) == 5.0                       # zero reference: the plain norm
    assert abs(fo.rel_l2([1.0, 0.0], [0.0, 1.0]) - np.sqrt(2.0)) < 1e-15   # ||(1,-1)|| / ||(0,1)||
    assert abs(fo.rel_l2([1.0, 2.0], [1.0, 1.0]) - 1.0 / np.sqrt(2.0)) < 1e-15
    a, b = np.array([2.0, -1.0, 0.5]), np.array([1.0, 1.0, 1.0])
    # the denominator is the SECOND argument: scaling it by 10 (and the difference with it) ...
    assert abs(fo.rel_l2(10 * a, 10 * b) - fo.rel_l2(a, b)) < 1e-15
    # ... and the measure is not symmetric
    assert abs(fo.rel_l2(a, b) - np.sqrt(1.0 + 4.0 + 0.25) / np.sqrt(3.0)) < 1e-15
    assert abs(fo.rel_l2(b, a) - np.sqrt(1.0 + 4.0 + 0.25) / np.sqrt(4.0 + 1.0 + 0.25)) < 1e-15
    assert fo.rel_l2(b, b) == 0.0


# ---- the any-n (column-blocked) form of the iteration -------------------------------------------------

@pytest.mark.parametrize("p,n,m,lam,iters,block", [(9, 1000, 4, 0.2, 7, 128), (15, 700, 8, 0.01, 10, 97),
                                                  (6, 50, 3, 0.0, 5, 7), (7, 333, 3, 0.3, 6, 1 << 16)])
def test_blocked_iteration_equals_the_plain_one(p, n, m, lam, iters, block):
    G = noisy_mean(p, n, 70 + p, sigma=0.5, outliers=2, scale_spread=True)
    if p >= 7:
        G[1] = G[0]                # an identical pair
        G[p - 1] = 0.0             # a zero gradient
    plain = fo.fa_aggregate(G, m, lam, iters)
    for threads in (1, 3):
        blk = fo.fa_aggregate_blocked(G, m, lam, iters, block=block, threads=threads)
        assert blk["k"] == plain["Y"].shape[1]
        assert np.allclose(blk["objective"], plain["objective"], rtol=0, atol=1e-10)
        assert np.allclose(blk["u"], plain["u"], rtol=0, atol=1e-10)
        assert np.allclose(blk["w"], plain["w"], rtol=1e-8, atol=0)
        assert fo.rel_l2(blk["d"], plain["d"]) < 1e-10
        assert blk["yty_err"] < 1e-10
        # Z = G Y of the blocked run against the plain run's Y: cosines of the principal angles
        # are the singular values of Y_plain^T Y_blocked, and Y_blocked^T g_i = Z[i]
        Yb_coords = np.linalg.lstsq(G.T, plain["Y"], rcond=None)[0]      # Y_plain = G^T A (Y lies in span G)
        cross = Yb_coords.T @ blk["Z"]                                    # = Y_plain^T Y_blocked
        assert np.allclose(np.linalg.svd(cross, compute_uv=False), 1.0, atol=1e-9)
        assert np.allclose(blk["K"], G @ G.T, rtol=1e-12)


def test_blocked_iteration_returns_sampled_aggregate_and_its_norm():
    G = noisy_mean(8, 500, 81, sigma=0.5, outliers=1)
    full = fo.fa_aggregate_blocked(G, 3, 0.1, 4, block=64)
    idx = np.array([0, 499, 63, 64, 65, 250, 250])
    part = fo.fa_aggregate_blocked(G, 3, 0.1, 4, block=64, sample=idx)
    assert np.array_equal(part["d_sample"], full["d"][idx])
    assert abs(part["d_norm"] - np.linalg.norm(full["d"])) < 1e-12 * np.linalg.norm(full["d"])
    assert "d" not in part


def test_blocked_iteration_widens_the_stored_type_block_by_block():
    G32 = noisy_mean(6, 300, 82, sigma=0.5, outliers=1).astype(np.float32)
    calls = []
    def widen(x):
        calls.append(x.shape[1])
        return x.astype(np.float64)
    a = fo.fa_aggregate_blocked(G32, 3, 0.1, 3, block=100, widen=widen)
    b = fo.fa_aggregate(G32.astype(np.float64), 3, 0.1, 3)
    assert max(calls) == 100 and fo.rel_l2(a["d"], b["d"]) < 1e-10


# ---- the stored full-size oracle runs (tests/golden/*_full.npz) are self-consistent ----------------------

@pytest.mark.parametrize("name", ["cfg3", "cfg4", "cfg5"])
def test_stored_full_size_runs_are_self_consistent(name):
    import os
    import synthetic_inputs as si
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", f"{name}_full.npz")
    if not os.path.exists(path):
        pytest.skip(f"no stored run for {name}")
    g = np.load(path)
    w = si.WORKLOADS[name]
    assert (int(g["n"]), int(g["p"]), int(g["m"]), float(g["lam"]), int(g["iters"]), int(g["seed"])) == \
           (w.n, w.p, w.m, w.lam, w.iters, w.seed)
    K, Z, u = g["K"], g["Z"], g["u"]
    assert g["yty_err"] < 1e-10 and np.allclose(K, K.T, rtol=1e-13)
    # u_i was summed from residual vectors; Z_i = Y^T g_i gives the same value as 1 - |Z_i|^2 / |g_i|^2 (Section 2.1)
    nz = np.diag(K) > 0
    assert np.allclose(u[nz], 1.0 - (Z[nz] ** 2).sum(axis=1) / np.diag(K)[nz], rtol=0, atol=1e-9)
    # D2 from difference vectors against the inner products
    D2 = np.diag(K)[:, None] + np.diag(K)[None, :] - 2 * K
    assert np.allclose(g["D2"], D2, rtol=1e-9, atol=1e-9 * np.diag(K).max())
    # the iteration descends from round two on (majorisation), and the aggregate is no longer than the plain mean's bound
    obj = g["objective"]
    assert all(obj[t + 1] <= obj[t] + 1e-9 for t in range(1, len(obj) - 1))
    assert g["d_norm"] <= np.sqrt(K.sum()) / w.p * (1 + 1e-12)        # |Y Y^T mean| <= |mean|
    assert len(g["idx"]) == len(g["d_sample"]) and g["idx"].max() == w.n - 1
