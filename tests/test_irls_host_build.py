"""The p-dimensional IRLS of csrc/fa_irls_core.cuh, compiled for the host (one "thread"), against the
CPU oracle -- the kernel's arithmetic is checked on every CPU run, without a GPU.

K comes from the oracle's plain inner products, so only the IRLS code is on trial: the isometric
embedding, the weights and terms of Eq. (5), the eigensolver (Jacobi sweeps + refinement), the
selection vector.  Same cases and tolerances as the GPU test of the same kernel.
"""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import synthetic_inputs as si
from oracle import fa_multi as fm
from oracle import fa_oracle as fo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

IRLS_CASES = [
    (1, 9, "noisy_mean", 1, 0.0, 3), (2, 5, "noisy_mean", 1, 0.3, 4), (3, 33, "dup_zero", 2, 0.2, 5),
    (7, 33, "dup_zero", 3, 0.0, 6), (15, 2000, "noisy_mean", 8, 0.01, 10), (16, 100, "gauss", 8, 0.1, 6),
    (17, 64, "noisy_mean", 9, 0.05, 6), (31, 3000, "noisy_mean", 12, 0.01, 12), (6, 3, "gauss", 4, 0.1, 5),
    (63, 200, "dup_zero", 16, 0.02, 8), (64, 300, "noisy_mean", 20, 0.01, 8),
]


@pytest.fixture(scope="module")
def host(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("irls_host") / "libirls_host.so")
    src = os.path.join(ROOT, "tests", "irls_host_shim.cpp")
    r = subprocess.run(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-x", "c++", src, "-o", out],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    lib = ctypes.CDLL(out)
    vp, i, d = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
    lib.irls_host.argtypes = [vp, i, i, d, d, i, i, vp, d, vp, vp, vp, vp, vp, vp, i, vp, d, d, vp, vp, vp]
    lib.irls_host.restype = i
    return lib


def run_host(lib, K, m, lam, iters, a=2.0, A0=None, tol=-1.0, counts=None, cb=1.0, ca=0.0):
    p = K.shape[0]
    K = np.ascontiguousarray(K, dtype=np.float64)
    A = np.zeros((p, m))
    c = np.zeros(p, dtype=np.float32)
    nw = len(counts) if counts is not None else p
    w = np.zeros(nw)
    obj = np.zeros(iters)
    rounds = np.zeros(1, dtype=np.int32)
    work = np.zeros(3, dtype=np.int32)
    cnt = np.zeros(64, dtype=np.uint8)
    if counts is not None:
        cnt[:nw] = counts
    A0c = None if A0 is None else np.ascontiguousarray(A0, dtype=np.float64)
    st = lib.irls_host(K.ctypes.data, p, m, float(lam), float(a), iters, 0 if A0 is None else 2,
                       None if A0c is None else A0c.ctypes.data, float(tol), A.ctypes.data, c.ctypes.data,
                       w.ctypes.data, obj.ctypes.data, None, rounds.ctypes.data, 0 if counts is None else nw,
                       cnt.ctypes.data, cb, ca, work.ctypes.data, work.ctypes.data + 4, work.ctypes.data + 8)
    return dict(status=st, A=A, c=c, w=w, objective=obj, rounds=int(rounds[0]), sweeps=int(work[0]),
                refinements=int(work[1]), sweeps_f32=int(work[2]))


@pytest.mark.parametrize("p,n,kind,m,lam,iters", IRLS_CASES)
def test_host_build_of_the_irls_kernel_matches_the_oracle(host, p, n, kind, m, lam, iters):
    G = si.ladder_case(p, n, 5, kind).astype(np.float64)
    ref = fo.fa_aggregate(G, m, lam, iters)
    got = run_host(host, fo.inner_products(G), m, lam, iters)
    k = ref["Y"].shape[1]
    assert got["status"] & ~4 == 0 and bool(got["status"] & 4) == (k < m)      # 4 = fewer than m directions
    assert not got["A"][:, k:].any()
    Y = G.T @ got["A"][:, :k]
    assert np.abs(Y.T @ Y - np.eye(k)).max() < 1e-9
    if k:
        assert fo.principal_angles(ref["Y"], Y).max() < 1e-7
    assert np.allclose(got["objective"], ref["objective"], rtol=0, atol=1e-9)
    assert np.allclose(got["w"], ref["w"], rtol=1e-6, atol=0)
    assert fo.rel_l2(got["c"].astype(np.float64) @ G, ref["d"]) < 1e-6


@pytest.mark.parametrize("name,n", [("cfg1", None), ("cfg2", 150_000), ("cfg3", 60_000), ("cfg5", 30_000)])
def test_host_build_on_the_workload_recipes_and_the_work_it_takes(host, name, n):
    """The workloads' spectra (huge weights on captured outliers next to a tight cluster of noise
    directions) are where a matrix-product refinement could lose accuracy: objective per round and
    subspace against the n-space oracle.  Also: the refinement must take over most of the work."""
    w = si.WORKLOADS[name]
    if n is not None:
        w = w.scaled(n)
    G = si.to_float64(si.generate(w))
    ref = fo.fa_aggregate(G, w.m, w.lam, w.iters)
    got = run_host(host, fo.inner_products(G), w.m, w.lam, w.iters)
    k = ref["Y"].shape[1]
    assert got["status"] & ~4 == 0
    assert np.allclose(got["objective"], ref["objective"], rtol=0, atol=1e-9)
    assert fo.principal_angles(ref["Y"], G.T @ got["A"][:, :k]).max() < 1e-7
    assert fo.rel_l2(got["c"].astype(np.float64) @ G, ref["d"]) < 1e-6
    print(f"{w.name}: {got['sweeps_f32']} fp32 and {got['sweeps']} fp64 Jacobi sweeps, {got['refinements']} refinement "
          f"steps in {w.iters} rounds")
    assert got["sweeps"] + got["sweeps_f32"] <= 3 * w.iters and got["refinements"] >= w.iters
    assert (got["sweeps_f32"] > 0) == (w.p > 32)         # fp32 sweeps only where the rounds are bound by shared-memory traffic


def test_host_build_with_workers_that_hold_several_gradients(host):
    counts = [2, 3, 1, 4, 2, 1, 3]
    r = np.random.default_rng(3)
    G = r.standard_normal(300)[None, :] + 0.5 * r.standard_normal((sum(counts), 300))
    ref = fm.fa_aggregate_multi(G, counts, 6, 0.5, 10, a=3.0)
    got = run_host(host, fo.inner_products(G), 6, 0.5, 10, a=3.0, counts=counts)
    assert np.allclose(got["objective"], ref["objective"], rtol=1e-9, atol=1e-9)
    assert np.allclose(got["w"], ref["w"], rtol=1e-6, atol=0)
    assert fo.rel_l2(got["c"].astype(np.float64) @ G, ref["d"]) < 1e-6


@pytest.mark.parametrize("alpha,beta", [(0.7, 0.5), (0.3, 0.8)])
def test_host_build_with_weights_of_both_signs(host, alpha, beta):
    G = si.ladder_case(12, 400, 9, "gauss").astype(np.float64)
    ref = fo.fa_aggregate(G, 6, 0.5, 6, alpha=alpha, beta=beta)
    got = run_host(host, fo.inner_products(G), 6, 0.5, 6, cb=2 * (1 - beta), ca=2 * (1 - alpha))
    k = ref["Y"].shape[1]
    assert np.allclose(got["objective"], ref["objective"], rtol=1e-9, atol=1e-9)
    if k:
        assert fo.principal_angles(ref["Y"], G.T @ got["A"][:, :k]).max() < 1e-7


def test_host_build_from_a_given_subspace_and_with_a_tolerance(host):
    G = si.ladder_case(15, 2000, 9, "noisy_mean").astype(np.float64)
    A0 = np.random.default_rng(1).standard_normal((15, 8))
    ref = fo.fa_aggregate(G, 8, 0.01, 6, Y0=G.T @ A0)
    got = run_host(host, fo.inner_products(G), 8, 0.01, 6, A0=A0)
    assert np.allclose(got["objective"], ref["objective"], rtol=1e-9, atol=1e-9)
    ref = fo.fa_aggregate(G, 8, 0.01, 40, tol=1e-5)
    got = run_host(host, fo.inner_products(G), 8, 0.01, 40, tol=1e-5)
    assert got["rounds"] == ref["rounds"]
    assert np.allclose(got["objective"][:got["rounds"]], ref["objective"], rtol=1e-9, atol=1e-9)
