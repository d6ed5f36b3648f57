"""CUDA path vs the CPU oracle, through the C ABI (python binding = argument marshalling only).

Tolerances (floating point): aggregate relative L2 <= 1e-4 and principal angles < 1e-3 rad for
fp32 gradients, 2e-3 and 1e-2 rad for bf16 gradients.  Inner products: |K - K_oracle| <=
5e-7 * sqrt(K_ii K_jj) (fp32 products, fp32 runs of <= 64 columns, fp64 above that); 2e-6 on the
tensor-core path (bf16, p > 16).
"""
import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import fa_multi as fm
from oracle import fa_oracle as fo

pytestmark = pytest.mark.gpu

TOL = {"f32": (1e-4, 1e-3), "bf16": (2e-3, 1e-2)}
GRAM_TOL = 5e-7
# bf16 with 16 < p <= 64 runs on the tensor cores: exact products, fp32 running sums over 256 columns
# (16 MMA steps) that the hardware rounds toward zero: up to about 16 * 2^-24 of relative bias
GRAM_TOL_TC = 2e-6


@pytest.fixture(scope="module")
def fa():
    import paper_2302_05865_b200 as mod
    return mod


def _gram_err(K, Kref):
    scale = np.sqrt(np.outer(np.diag(Kref), np.diag(Kref)))
    scale[scale == 0] = 1.0
    return float(np.max(np.abs(K - Kref) / scale))


LADDER = [
    # p, n, kind, bf16, misalign
    (1, 1, "gauss", False, 0), (2, 3, "gauss", False, 1), (3, 5, "noisy_mean", False, 0),
    (4, 31, "noisy_mean", False, 3), (7, 33, "dup_zero", False, 1), (8, 1023, "gauss", False, 2),
    (12, 4097, "noisy_mean", False, 0), (15, 65_537, "noisy_mean", False, 1), (15, 300_002, "dup_zero", False, 0),
    (16, 70_000, "gauss", False, 0), (17, 40_001, "noisy_mean", False, 0), (31, 50_000, "dup_zero", False, 2),
    (32, 9_999, "gauss", False, 1), (33, 20_000, "noisy_mean", False, 0), (63, 30_001, "noisy_mean", False, 0),
    (64, 12_345, "gauss", False, 3),
    (5, 7, "gauss", True, 1), (15, 100_003, "noisy_mean", True, 0), (16, 50_000, "dup_zero", True, 4),
    (31, 40_002, "noisy_mean", True, 2), (63, 66_000, "dup_zero", True, 0), (64, 8_191, "gauss", True, 5),
    # fp32, 16 < p <= 32, rows on 16-byte boundaries: the tensor-fed kernel with teams of four warps
    (31, 50_000, "dup_zero", False, 0), (17, 4_096, "gauss", False, 0), (32, 300_004, "noisy_mean", False, 0),
    (24, 1_000_000, "gauss", False, 4), (31, 4_100, "noisy_mean", False, 0),
    # fp32 rows on 8-byte but not all on 16-byte boundaries (n % 4 = 2 and / or a base that is 8 modulo 16):
    # the output pass reads 16-byte vectors and hands half of them to the neighbouring thread
    (15, 65_538, "noisy_mean", False, 2), (16, 10, "gauss", False, 0), (3, 8, "gauss", False, 2),
    (9, 130, "noisy_mean", False, 0), (33, 4_098, "dup_zero", False, 2), (64, 1_026, "gauss", False, 0),
    # fp32, 13 to 16 rows in the tensor-fed kernel, rows in one, two and four alignment classes (4-byte operand loads
    # of columns half a tile apart; the tile step is 256 or 252 columns)
    (13, 20_001, "noisy_mean", False, 0), (14, 30_002, "gauss", False, 0), (16, 50_003, "dup_zero", False, 0),
    (16, 40_002, "noisy_mean", False, 2), (13, 8_192, "gauss", False, 4),
    # fp32, 32 < p <= 64, rows on 16-byte boundaries: two triangle launches and the rectangle between the row blocks
    (48, 100_000, "noisy_mean", False, 0), (63, 40_004, "dup_zero", False, 0), (64, 8_192, "gauss", False, 0),
    (40, 4_096, "gauss", False, 4), (34, 300_000, "noisy_mean", False, 0), (57, 1_000_000, "gauss", False, 8),
    # bf16, p > 16, 16-byte aligned rows: the tensor-core kernel
    (17, 64, "gauss", True, 0), (33, 264, "noisy_mean", True, 0), (63, 4_096, "dup_zero", True, 0),
    (64, 65_536, "gauss", True, 0), (31, 1_000_000, "dup_zero", True, 8), (48, 300_008, "noisy_mean", True, 0),
]


@pytest.mark.parametrize("p,n,kind,bf16,mis", LADDER)
def test_gram_matches_plain_inner_products(fa, p, n, kind, bf16, mis):
    from tests.gpu_util import to_device, redzones_intact
    G_np = si.ladder_case(p, n, 11, kind, bf16=bf16)
    G, buf = to_device(G_np, misalign_elems=mis)
    K = fa.fa_gram(G)
    K2 = fa.fa_gram(G)
    torch.cuda.synchronize()
    assert torch.equal(K, K2)                                   # fixed reduction order
    Kref = fo.inner_products(si.to_float64(G_np))
    Kh = K.cpu().numpy()
    assert np.array_equal(Kh, Kh.T)
    assert _gram_err(Kh, Kref) < (GRAM_TOL_TC if (bf16 and p > 16) else GRAM_TOL)
    assert redzones_intact(buf, 64 + mis, p * n)
    if kind == "dup_zero" and p >= 3:                           # identical rows give identical entries
        assert Kh[0, 0] == Kh[0, 1] == Kh[1, 1]
        assert not Kh[p - 1].any()


@pytest.mark.parametrize("p,n,kind,bf16,mis", [c for c in LADDER if c[1] > 1])
def test_combine_matches_weighted_row_sum(fa, p, n, kind, bf16, mis):
    from tests.gpu_util import to_device
    G_np = si.ladder_case(p, n, 12, kind, bf16=bf16)
    G, _ = to_device(G_np, misalign_elems=mis)
    c = np.random.default_rng(p * 1000 + n).standard_normal(p).astype(np.float32)
    guard = torch.full((n + 128,), float("nan"), device="cuda")
    out = guard[64 + (mis % 4):64 + (mis % 4) + n]
    fa.fa_combine(G, torch.from_numpy(c).cuda(), out=out)
    torch.cuda.synchronize()
    ref = c.astype(np.float64) @ si.to_float64(G_np)
    scale = np.abs(c.astype(np.float64)) @ np.abs(si.to_float64(G_np)) + 1e-30
    assert np.max(np.abs(out.cpu().numpy() - ref) / scale) < 1e-5
    assert torch.isnan(guard[:64 + (mis % 4)]).all() and torch.isnan(guard[64 + (mis % 4) + n:]).all()


IRLS_CASES = [
    (1, 9, "noisy_mean", 1, 0.0, 3), (2, 5, "noisy_mean", 1, 0.3, 4), (3, 33, "dup_zero", 2, 0.2, 5),
    (7, 33, "dup_zero", 3, 0.0, 6), (15, 2000, "noisy_mean", 8, 0.01, 10), (16, 100, "gauss", 8, 0.1, 6),
    (17, 64, "noisy_mean", 9, 0.05, 6), (31, 3000, "noisy_mean", 12, 0.01, 12), (6, 3, "gauss", 4, 0.1, 5),
    (63, 200, "dup_zero", 16, 0.02, 8), (64, 300, "noisy_mean", 20, 0.01, 8),
]


@pytest.mark.parametrize("p,n,kind,m,lam,iters", IRLS_CASES)
def test_irls_rounds_match_oracle_from_exact_inner_products(fa, p, n, kind, m, lam, iters):
    """K comes from the oracle's plain definition; only the p-dimensional IRLS kernel is on trial."""
    G = si.ladder_case(p, n, 5, kind).astype(np.float64)
    ref = fo.fa_aggregate(G, m, lam, iters)
    K = torch.from_numpy(fo.inner_products(G)).cuda()
    A = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    w = torch.zeros(p, dtype=torch.float64, device="cuda")
    obj = torch.zeros(iters, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = fa.fa_irls(K, m, lam, iters, A_out=A, w_out=w, obj_out=obj, status=status)
    torch.cuda.synchronize()
    k = ref["Y"].shape[1]
    st = int(status.item())
    assert st & ~fa.ST_RANK_LT_M == 0 and bool(st & fa.ST_RANK_LT_M) == (k < m)
    Ah = A.cpu().numpy()
    assert not Ah[:, k:].any()
    Y = G.T @ Ah[:, :k]
    assert np.abs(Y.T @ Y - np.eye(k)).max() < 1e-9
    if k:
        assert fo.principal_angles(ref["Y"], Y).max() < 1e-7
    assert np.allclose(obj.cpu().numpy(), ref["objective"], rtol=0, atol=1e-9)
    assert np.allclose(w.cpu().numpy(), ref["w"], rtol=1e-6, atol=0)
    d = c.cpu().numpy().astype(np.float64) @ G
    assert fo.rel_l2(d, ref["d"]) < 1e-6

    # the single-round entry point, iterated, walks the same path
    A1 = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    o1 = torch.zeros(1, dtype=torch.float64, device="cuda")
    objs = []
    for t in range(iters):
        fa.fa_irls_step(K, m, lam, t == 0, A1, objective=o1)
        objs.append(float(o1.item()))
    assert np.allclose(objs, ref["objective"], rtol=0, atol=1e-9)
    if k:
        assert fo.principal_angles(ref["Y"], G.T @ A1.cpu().numpy()[:, :k]).max() < 1e-7


EX_CASES = [
    (1, 9, "noisy_mean", 1, 0.0, 1.5, 3), (3, 33, "dup_zero", 2, 0.2, 3.0, 5), (15, 2000, "noisy_mean", 8, 0.01, 1.5, 10),
    (15, 2000, "noisy_mean", 8, 0.01, 4.0, 10), (16, 100, "gauss", 8, 0.1, 3.0, 6), (31, 3000, "noisy_mean", 12, 0.01, 2.5, 12),
    (63, 200, "dup_zero", 16, 0.02, 1.25, 8), (64, 300, "noisy_mean", 20, 0.01, 2.0, 8),
]


@pytest.mark.parametrize("p,n,kind,m,lam,a,iters", EX_CASES)
def test_irls_with_another_surrogate_constant_and_the_selection_matrix(fa, p, n, kind, m, lam, a, iters):
    """Exponent 1/a of Eq. (4) with a != 2, and S with Y Y^T g_j = sum_i S[i][j] g_i."""
    G = si.ladder_case(p, n, 9, kind).astype(np.float64)
    ref = fo.fa_aggregate(G, m, lam, iters, a=a)
    K = torch.from_numpy(fo.inner_products(G)).cuda()
    A = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    S = torch.full((p, p), float("nan"), dtype=torch.float64, device="cuda")
    w = torch.zeros(p, dtype=torch.float64, device="cuda")
    obj = torch.zeros(iters, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = fa.fa_irls_ex(K, m, lam, a, iters, A_out=A, S_out=S, w_out=w, obj_out=obj, status=status)
    torch.cuda.synchronize()
    k = ref["Y"].shape[1]
    assert int(status.item()) & ~fa.ST_RANK_LT_M == 0
    Y = G.T @ A.cpu().numpy()[:, :k]
    if k:
        assert fo.principal_angles(ref["Y"], Y).max() < 1e-7
    assert np.allclose(obj.cpu().numpy(), ref["objective"], rtol=1e-9, atol=1e-9)
    assert np.allclose(w.cpu().numpy(), ref["w"], rtol=1e-6, atol=0)
    assert fo.rel_l2(c.cpu().numpy().astype(np.float64) @ G, ref["d"]) < 1e-6
    Sh = S.cpu().numpy()
    R = fo.reconstruction(G, ref["Y"])
    assert np.abs(Sh.T @ G - R).max() <= 1e-8 * max(1.0, np.abs(R).max())
    assert np.allclose(Sh.sum(axis=1) / p, c.cpu().numpy(), rtol=1e-5, atol=1e-7)


def test_aggregate_ex_equals_its_parts(fa):
    G_np = si.ladder_case(15, 70_001, 4, "noisy_mean")
    G = torch.from_numpy(G_np).cuda()
    S = torch.zeros((15, 15), dtype=torch.float64, device="cuda")
    out = fa.fa_aggregate_ex(G, 8, 0.01, 3.0, 7, S_out=S)
    ref = fo.fa_aggregate(G_np.astype(np.float64), 8, 0.01, 7, a=3.0)
    assert fo.rel_l2(out.cpu().numpy(), ref["d"]) < 1e-4
    R = fo.reconstruction(G_np.astype(np.float64), ref["Y"])
    assert fo.rel_l2(S.cpu().numpy().T @ G_np.astype(np.float64), R) < 1e-4
    assert torch.equal(fa.fa_aggregate_ex(G, 8, 0.01, 2.0, 7), fa.fa_aggregate(G, 8, 0.01, 7))
    with pytest.raises(fa.FaError):
        fa.fa_aggregate_ex(G, 8, 0.01, 1.0, 7)
    with pytest.raises(fa.FaError):
        fa.fa_irls_ex(torch.eye(3, dtype=torch.float64, device="cuda"), 2, 0.0, float("nan"), 3)


def _worker_rows(counts, n, seed, outliers, bf16=False):
    """Rows of workers with counts[i] gradients each: a common mean, a per-worker offset, per-gradient noise;
    the last `outliers` workers send large random gradients."""
    r = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, len(counts), n, 91])))
    mu = r.standard_normal(n).astype(np.float32)
    rows = []
    for i, k in enumerate(counts):
        if i >= len(counts) - outliers:
            block = np.float32(5.0) * r.standard_normal((k, n)).astype(np.float32)
        else:
            centre = mu + np.float32(0.2) * r.standard_normal(n).astype(np.float32)
            block = centre[None, :] + np.float32(0.5) * r.standard_normal((k, n)).astype(np.float32)
        rows.append(block)
    G = np.ascontiguousarray(np.concatenate(rows, axis=0), dtype=np.float32)
    return si.f32_to_bf16_bits(G) if bf16 else G


MULTI_IRLS = [
    ([1] * 9, 40, 4, 0.3, 2.0, 7, 2), ([3, 1, 2, 4, 1], 200, 3, 0.0, 2.0, 8, 1), ([3, 1, 2, 4, 1], 200, 5, 0.4, 2.0, 8, 1),
    ([2, 3, 1, 4, 2, 1, 3], 300, 6, 0.5, 3.0, 10, 2), ([4] * 16, 500, 20, 0.05, 2.0, 8, 3), ([1, 63], 100, 3, 0.2, 2.0, 5, 0),
    ([5], 50, 2, 0.3, 2.0, 4, 0), ([2] * 15, 1000, 8, 0.01, 2.0, 10, 3), ([8, 7, 8, 8], 400, 10, 0.1, 1.5, 6, 1),
]


@pytest.mark.parametrize("counts,n,m,lam,a,iters,outliers", MULTI_IRLS)
def test_irls_for_workers_with_several_gradients(fa, counts, n, m, lam, a, iters, outliers):
    G = _worker_rows(counts, n, 3, outliers).astype(np.float64)
    ref = fm.fa_aggregate_multi(G, counts, m, lam, iters, a=a)
    rows, nw = G.shape[0], len(counts)
    K = torch.from_numpy(fo.inner_products(G)).cuda()
    A = torch.zeros((rows, m), dtype=torch.float64, device="cuda")
    w = torch.full((nw + 2,), float("nan"), dtype=torch.float64, device="cuda")
    obj = torch.zeros(iters, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = fa.fa_irls_multi(K, counts, m, lam, iters, a=a, A_out=A, w_out=w, obj_out=obj, status=status)
    torch.cuda.synchronize()
    k = ref["Y"].shape[1]
    assert int(status.item()) & ~fa.ST_RANK_LT_M == 0
    assert torch.isnan(w[nw:]).all()                     # one weight per worker, nothing written beyond
    Y = G.T @ A.cpu().numpy()[:, :k]
    assert np.abs(Y.T @ Y - np.eye(k)).max() < 1e-9
    assert fo.principal_angles(ref["Y"], Y).max() < 1e-7
    assert np.allclose(obj.cpu().numpy(), ref["objective"], rtol=1e-9, atol=1e-9)
    assert np.allclose(w[:nw].cpu().numpy(), ref["w"], rtol=1e-6, atol=0)
    assert fo.rel_l2(c.cpu().numpy().astype(np.float64) @ G, ref["d"]) < 1e-6


MULTI_AGG = [
    ([3, 1, 2, 4, 1], 70_001, False, 4, 0.2, 2.0, 7, 1), ([2] * 15, 50_000, False, 8, 0.01, 2.0, 8, 3),
    ([4] * 16, 66_000, True, 16, 0.02, 2.0, 6, 3), ([1] * 15, 65_537, False, 8, 0.01, 3.0, 6, 2),
]


@pytest.mark.parametrize("counts,n,bf16,m,lam,a,iters,outliers", MULTI_AGG)
def test_aggregate_for_workers_with_several_gradients(fa, counts, n, bf16, m, lam, a, iters, outliers):
    from tests.gpu_util import to_device
    G_np = _worker_rows(counts, n, 8, outliers, bf16=bf16)
    G, _ = to_device(G_np)
    out = fa.fa_aggregate_multi(G, counts, m, lam, iters, a=a)
    torch.cuda.synchronize()
    ref = fm.fa_aggregate_multi(si.to_float64(G_np), counts, m, lam, iters, a=a)
    rel_tol, _ = TOL["bf16" if bf16 else "f32"]
    assert fo.rel_l2(out.cpu().numpy(), ref["d"]) < rel_tol
    if all(k == 1 for k in counts):
        assert torch.equal(out, fa.fa_aggregate_ex(G, m, lam, a, iters))
    for bad in ([1] * (len(counts) - 1), [0] + list(counts), list(counts) + [1]):
        with pytest.raises(fa.FaError):
            fa.fa_aggregate_multi(G, bad, m, lam, iters)


def _aggregate_and_compare(fa, G_np, m, lam, iters, dtype_key, mis=0):
    from tests.gpu_util import to_device, redzones_intact, subspace_from_A
    p, n = G_np.shape
    G, buf = to_device(G_np, misalign_elems=mis)
    A = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    guard = torch.full((n + 128,), float("nan"), device="cuda")
    out = guard[64:64 + n]
    fa.fa_aggregate(G, m, lam, iters, out=out, A_out=A, status=status)
    out2 = fa.fa_aggregate(G, m, lam, iters)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    assert redzones_intact(buf, 64 + mis, p * n)
    assert torch.isnan(guard[:64]).all() and torch.isnan(guard[64 + n:]).all()
    X = si.to_float64(G_np)
    ref = fo.fa_aggregate(X, m, lam, iters)
    k = ref["Y"].shape[1]
    st = int(status.item())
    assert st & ~fa.ST_RANK_LT_M == 0, f"device status {st}"
    rel_tol, ang_tol = TOL[dtype_key]
    rel = fo.rel_l2(out.cpu().numpy(), ref["d"])
    Y = subspace_from_A(G_np, A.cpu().numpy())
    assert Y.shape[1] == k
    ang = float(fo.principal_angles(ref["Y"], Y).max()) if k else 0.0
    assert rel < rel_tol, f"relative L2 {rel}"
    assert ang < ang_tol, f"principal angle {ang}"
    # element by element: a norm hides an error confined to a few columns (a ragged tail, one tile).
    # d_j = sum_i c_i G_ij with |c|_1 of order 1, so the error of one element is measured against
    # the mean magnitude of its column, with ten times the norm-wise tolerance
    scale = np.abs(X).mean(axis=0) + 1e-30 * float(np.abs(X).max() + 1.0)
    worst = float(np.max(np.abs(out.cpu().numpy().astype(np.float64) - ref["d"]) / scale))
    assert worst < 10 * rel_tol, f"largest element error over column scale {worst}"
    return rel, ang


AGG_LADDER = [
    (1, 17, "noisy_mean", False, 1, 0.0, 3, 0), (2, 3, "gauss", False, 1, 0.5, 4, 1),
    (3, 5, "noisy_mean", False, 2, 0.1, 5, 0), (7, 33, "dup_zero", False, 3, 0.2, 6, 1),
    (15, 65_537, "noisy_mean", False, 8, 0.01, 10, 1), (16, 70_000, "gauss", False, 8, 0.1, 6, 0),
    (17, 40_001, "noisy_mean", False, 9, 0.05, 6, 0), (31, 50_000, "dup_zero", False, 12, 0.01, 8, 2),
    (33, 20_000, "noisy_mean", False, 12, 0.0, 6, 0), (64, 12_345, "noisy_mean", False, 20, 0.01, 6, 3),
    (31, 50_000, "dup_zero", False, 12, 0.01, 8, 0), (24, 1_000_000, "noisy_mean", False, 10, 0.02, 6, 4),
    (15, 100_003, "noisy_mean", True, 8, 0.01, 8, 0), (31, 40_002, "noisy_mean", True, 12, 0.02, 8, 2),
    (63, 66_000, "dup_zero", True, 16, 0.01, 8, 0), (33, 264, "noisy_mean", True, 10, 0.02, 6, 0),
    (64, 65_536, "noisy_mean", True, 20, 0.01, 6, 0), (31, 1_000_000, "dup_zero", True, 12, 0.01, 8, 8),
    (48, 100_000, "noisy_mean", False, 16, 0.01, 6, 0), (63, 40_004, "dup_zero", False, 16, 0.02, 6, 4),
]


@pytest.mark.parametrize("p,n,kind,bf16,m,lam,iters,mis", AGG_LADDER)
def test_aggregate_matches_oracle_on_the_ladder(fa, p, n, kind, bf16, m, lam, iters, mis):
    G_np = si.ladder_case(p, n, 21, kind, bf16=bf16)
    _aggregate_and_compare(fa, G_np, m, lam, iters, "bf16" if bf16 else "f32", mis)


@pytest.mark.parametrize("name,n", [("cfg1", None), ("cfg2", 1_300_003), ("cfg3", 700_001),
                                    ("cfg4", 2_000_000), ("cfg5", 400_000)])
def test_aggregate_matches_oracle_on_the_workload_recipes(fa, name, n):
    w = si.WORKLOADS[name]
    if n is not None:
        w = w.scaled(n)
    G_np = si.generate(w)
    _aggregate_and_compare(fa, G_np, w.m, w.lam, w.iters, w.dtype)


def test_degenerate_inputs_report_status_and_stay_finite(fa):
    G = torch.zeros((5, 1000), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    A = torch.ones((5, 2), dtype=torch.float64, device="cuda")
    out = fa.fa_aggregate(G, 2, 0.1, 3, A_out=A, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == fa.ST_RANK0 and not out.any() and not A.any()
    G = torch.randn((5, 1000), device="cuda")
    G[2, 17] = float("inf")
    out = fa.fa_aggregate(G, 2, 0.1, 3, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == fa.ST_NONFINITE and not out.any()


def test_host_side_argument_checks(fa):
    G = torch.randn((4, 100), device="cuda")
    with pytest.raises(fa.FaError):
        fa.fa_aggregate(G, 5, 0.0, 3)                 # m > p
    with pytest.raises(fa.FaError):
        fa.fa_aggregate(G, 2, -1.0, 3)                # negative lambda
    with pytest.raises(fa.FaError):
        fa.fa_aggregate(G, 2, float("nan"), 3)
    with pytest.raises(fa.FaError):
        fa.fa_aggregate(G, 2, 0.0, 0)                 # no rounds
    with pytest.raises(fa.FaError):
        fa.fa_aggregate(G, 2, 0.0, 3, ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(fa.FaError):
        fa.fa_gram(torch.randn((65, 10), device="cuda"))


def test_host_buffer_entry_point_round_trips(fa):
    w = si.WORKLOADS["cfg1"]
    G_np = si.generate(w)
    Gh = torch.from_numpy(G_np).pin_memory()
    outh = torch.empty(w.n, dtype=torch.float32).pin_memory()
    sth = torch.zeros(1, dtype=torch.int32).pin_memory()
    Gd = torch.empty((w.p, w.n), device="cuda")
    outd = torch.empty(w.n, device="cuda")
    std = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = fa.new_workspace(Gd, w.m)
    fa.fa_aggregate_host(Gh, w.m, w.lam, w.iters, outh, Gd, outd, ws, sth, std)
    torch.cuda.synchronize()
    ref = fa.fa_aggregate(torch.from_numpy(G_np).cuda(), w.m, w.lam, w.iters)
    assert torch.equal(outh.cuda(), ref) and int(sth.item()) == 0


@pytest.mark.parametrize("p,n,bf16,world", [(15, 300_007, False, 3), (31, 200_000, True, 4), (15, 20, False, 8)])
def test_column_sharded_step_equals_the_whole_step(fa, p, n, bf16, world):
    """One GPU plays the ranks one after another (no rank waits on another): pass 1 takes every shard's
    partial inner products, pass 2 hands each rank the sum in place of the all-reduce."""
    from paper_2302_05865_b200 import sharded
    from tests.gpu_util import to_device
    m, lam, iters = min(8, p), 0.01, 8
    G_np = si.ladder_case(p, n, 31, "noisy_mean", bf16=bf16)
    G, _ = to_device(G_np)
    bounds = [sharded.shard_bounds(n, world, r) for r in range(world)]
    shards = [G[:, lo:hi].contiguous() for lo, hi in bounds]
    Ksum = torch.zeros((p, p), dtype=torch.float64, device="cuda")
    for sh in shards:
        if sh.shape[1]:
            Ksum += fa.fa_gram(sh)
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    for (lo, hi), sh in zip(bounds, shards):
        step = sharded.ShardedStep(m, lam, iters, reduce_fn=lambda K: K.copy_(Ksum))
        out[lo:hi] = step(sh)
    torch.cuda.synchronize()
    ref = fo.fa_aggregate(si.to_float64(G_np), m, lam, iters)
    rel_tol, _ = TOL["bf16" if bf16 else "f32"]
    assert fo.rel_l2(out.cpu().numpy(), ref["d"]) < rel_tol
    whole = fa.fa_aggregate(G, m, lam, iters)
    assert fo.rel_l2(out.cpu().numpy(), whole.cpu().numpy().astype(np.float64)) < rel_tol


WARM_CASES = [(15, 2000, "noisy_mean", 8, 0.01, 6), (7, 33, "dup_zero", 3, 0.2, 5), (31, 3000, "noisy_mean", 12, 0.01, 6),
              (64, 300, "noisy_mean", 20, 0.01, 5), (2, 5, "noisy_mean", 1, 0.3, 4)]


@pytest.mark.parametrize("p,n,kind,m,lam,iters", WARM_CASES)
def test_irls_from_a_given_subspace_and_with_a_tolerance(fa, p, n, kind, m, lam, iters):
    G = si.ladder_case(p, n, 9, kind).astype(np.float64)
    K = torch.from_numpy(fo.inner_products(G)).cuda()
    A0_np = np.random.default_rng(1).standard_normal((p, m))
    A = torch.from_numpy(A0_np).cuda()                          # started from and overwritten in place
    obj = torch.zeros(iters, dtype=torch.float64, device="cuda")
    rounds = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = fa.fa_irls_warm(K, m, lam, iters, A0=A, A_out=A, obj_out=obj, rounds_out=rounds)
    ref = fo.fa_aggregate(G, m, lam, iters, Y0=G.T @ A0_np)
    k = ref["Y"].shape[1]
    assert int(rounds.item()) == iters
    assert fo.principal_angles(ref["Y"], G.T @ A.cpu().numpy()[:, :k]).max() < 1e-7
    assert np.allclose(obj.cpu().numpy(), ref["objective"], rtol=1e-9, atol=1e-9)
    assert fo.rel_l2(c.cpu().numpy().astype(np.float64) @ G, ref["d"]) < 1e-6
    # a start without rank is the uniform first round
    cold = fa.fa_irls(K, m, lam, iters)
    zero = fa.fa_irls_warm(K, m, lam, iters, A0=torch.zeros((p, m), dtype=torch.float64, device="cuda"))
    assert torch.equal(cold, zero) and torch.equal(cold, fa.fa_irls_warm(K, m, lam, iters))
    # tolerance: same number of rounds as the oracle, same result, tail of the objective repeated
    cap, tol = 40, 1e-5
    ref = fo.fa_aggregate(G, m, lam, cap, tol=tol)
    obj = torch.full((cap,), float("nan"), dtype=torch.float64, device="cuda")
    c = fa.fa_irls_warm(K, m, lam, cap, tol=tol, obj_out=obj, rounds_out=rounds)
    r = int(rounds.item())
    oh = obj.cpu().numpy()
    assert r == ref["rounds"]
    assert np.allclose(oh[:r], ref["objective"], rtol=1e-9, atol=1e-9) and (oh[r:] == oh[r - 1]).all()
    assert fo.rel_l2(c.cpu().numpy().astype(np.float64) @ G, ref["d"]) < 1e-6


def test_aggregate_continues_from_the_previous_steps_subspace(fa):
    """Two training steps: the second starts from the first one's A and needs fewer rounds."""
    from tests.gpu_util import to_device
    p, n, m, lam = 15, 120_001, 8, 0.01
    G1_np = si.ladder_case(p, n, 41, "noisy_mean")
    noise = np.random.Generator(np.random.PCG64(42)).standard_normal((p, n)).astype(np.float32)
    G2_np = (G1_np + np.float32(0.05) * noise).astype(np.float32)          # the next step's gradients
    G1, _ = to_device(G1_np)
    G2, _ = to_device(G2_np)
    A = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    rounds = torch.zeros(1, dtype=torch.int32, device="cuda")
    fa.fa_aggregate_warm(G1, m, lam, 30, tol=1e-7, A_out=A, rounds_out=rounds)
    r_cold = int(rounds.item())
    A_prev = A.clone()
    out = fa.fa_aggregate_warm(G2, m, lam, 30, tol=1e-7, A0=A, A_out=A, rounds_out=rounds)
    r_warm = int(rounds.item())
    ref = fo.fa_aggregate(G2_np.astype(np.float64), m, lam, 30, tol=1e-7,
                          Y0=G2_np.astype(np.float64).T @ A_prev.cpu().numpy())
    assert r_warm == ref["rounds"] and r_warm <= r_cold
    assert fo.rel_l2(out.cpu().numpy(), ref["d"]) < 1e-4
    with pytest.raises(fa.FaError):
        fa.fa_aggregate_warm(G2, m, lam, 5, tol=float("nan"))


BETA_CASES = [
    (15, 2000, "noisy_mean", 8, 0.01, 2.0, 0.7, 0.5, 8), (7, 33, "dup_zero", 3, 0.2, 2.0, 0.5, 0.3, 6),
    (31, 3000, "noisy_mean", 12, 0.01, 3.0, 0.8, 0.5, 8), (64, 300, "noisy_mean", 20, 0.01, 2.0, 0.9, 0.6, 6),
    (15, 2000, "gauss", 8, 0.1, 2.0, 1.0, 0.8, 6),
    # weights of both signs, and all negative (nothing enters Y)
    (12, 400, "gauss", 6, 0.5, 2.0, 0.3, 0.8, 6), (15, 2000, "noisy_mean", 8, 0.5, 2.0, 0.4, 0.8, 6),
    (9, 100, "noisy_mean", 4, 1.0, 2.0, 0.5, 0.9, 6), (10, 50, "noisy_mean", 5, 0.0, 2.0, 0.3, 0.9, 6),
]


@pytest.mark.parametrize("p,n,kind,m,lam,a,alpha,beta,iters", BETA_CASES)
def test_irls_with_a_general_beta_likelihood(fa, p, n, kind, m, lam, a, alpha, beta, iters):
    G = si.ladder_case(p, n, 9, kind).astype(np.float64)
    ref = fo.fa_aggregate(G, m, lam, iters, a=a, alpha=alpha, beta=beta)
    K = torch.from_numpy(fo.inner_products(G)).cuda()
    A = torch.zeros((p, m), dtype=torch.float64, device="cuda")
    w = torch.zeros(p, dtype=torch.float64, device="cuda")
    obj = torch.zeros(iters, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = fa.fa_irls_beta(K, m, lam, iters, alpha, beta, a=a, A_out=A, w_out=w, obj_out=obj, status=status)
    torch.cuda.synchronize()
    k = ref["Y"].shape[1]
    st = int(status.item())
    assert st & ~fa.ST_RANK_LT_M == 0 and bool(st & fa.ST_RANK_LT_M) == (k < m)
    if k:
        assert fo.principal_angles(ref["Y"], G.T @ A.cpu().numpy()[:, :k]).max() < 1e-7
    assert not A.cpu().numpy()[:, k:].any()
    assert np.allclose(obj.cpu().numpy(), ref["objective"], rtol=1e-9, atol=1e-9)
    assert np.allclose(w.cpu().numpy(), ref["w"], rtol=1e-6, atol=1e-12 * np.abs(ref["w"]).max())
    assert fo.rel_l2(c.cpu().numpy().astype(np.float64) @ G, ref["d"]) < 1e-6 or not ref["d"].any()


def test_aggregate_with_a_general_beta_likelihood(fa):
    G_np = si.ladder_case(15, 90_001, 4, "noisy_mean")
    G = torch.from_numpy(G_np).cuda()
    out = fa.fa_aggregate_beta(G, 8, 0.05, 7, 0.6, 0.7)
    ref = fo.fa_aggregate(G_np.astype(np.float64), 8, 0.05, 7, alpha=0.6, beta=0.7)
    assert fo.rel_l2(out.cpu().numpy(), ref["d"]) < 1e-4
    assert torch.equal(fa.fa_aggregate_beta(G, 8, 0.05, 7, 1.0, 0.5), fa.fa_aggregate(G, 8, 0.05, 7))
    for alpha, beta in ((0.0, 0.5), (1.5, 0.5), (1.0, 0.0), (1.0, 1.5), (float("nan"), 0.5)):
        with pytest.raises(fa.FaError):
            fa.fa_aggregate_beta(G, 8, 0.05, 7, alpha, beta)
