"""TEST INFRASTRUCTURE -- fp64 CPU statement of the Flag Aggregator with several gradients per worker.

Nothing in the product path may import this file (see oracle/fa_oracle.py).

What it computes (Flag Aggregator paper, arXiv 2302.05865): worker i hands in k_i gradients, the
columns of g_i in R^{n x k_i} (Section 2.1 "Advantages of Subspace based Aggregation", the
extension paragraph of Section 2.2, and the appendix restatement of the objective with
tr(Y^T g_i g_i^T Y) / tr(g_i^T g_i)).  Here the k_i gradients of worker i are k_i consecutive ROWS
of the row-major array G (sum_i k_i rows in all) and `counts` = (k_1, ..., k_p).

  value of worker i   v_i = tr(g_i^T Y Y^T g_i) / tr(g_i^T g_i)
  objective           A(Y) = sum_i (1 - v_i)^(1/a)
                           + lam/(p-1) sum_{i != j} (1 - ||Y^T (gbar_i-gbar_j)||^2 / ||gbar_i-gbar_j||^2)^(1/a)
  direction           d = (1/p) Y Y^T sum_i gbar_i

Readings (the paper gives the data term only; each is listed in the design notes):
  * gbar_i, the mean of worker i's gradients, stands for the worker in the pairwise regulariser
    and in the final average -- g_i - g_j has no meaning when k_i != k_j, and with k_i = 1 this is
    the single-gradient method of oracle/fa_oracle.py;
  * the reweighting of a term is the same as there: 1 / (normaliser * max(u^(1-1/a), EPS)), the
    weight of worker i multiplies all k_i of its outer products; round one is uniform (weight 1
    on every gradient, lam/(p-1) on every pair);
  * a worker whose gradients are all zero, and a pair of identical means, carry weight 0.

The eigenvectors of C = sum_i w_i g_i g_i^T + sum_{i != j} w_ij (gbar_i-gbar_j)(gbar_i-gbar_j)^T come
from the thin SVD of the matrix whose columns are the sqrt-weighted vectors themselves.

Parity pins (tests/test_oracle_multi_pins.py): k_i = 1 reduces to fa_oracle; a worker that repeats
one gradient scores like that gradient; rotation of a worker's gradients among themselves;
monotone descent; stationarity by finite differences; brute force over directions in the plane;
trace form against residual form; mean recovery.
"""
from __future__ import annotations

import numpy as np

from .fa_oracle import EPS, RANK_REL, SAME_PAIR_REL, ZERO_NORM_REL


def blocks(counts):
    """Row ranges [(start, stop)] of the workers."""
    out, r0 = [], 0
    for k in counts:
        k = int(k)
        if k < 1:
            raise ValueError("every worker needs at least one gradient")
        out.append((r0, r0 + k))
        r0 += k
    return out


def worker_means(G, counts):
    G = np.asarray(G, dtype=np.float64)
    return np.stack([G[s:e].mean(axis=0) for s, e in blocks(counts)])


def _setup(G, counts, lam):
    G = np.asarray(G, dtype=np.float64)
    bl = blocks(counts)
    if bl[-1][1] != G.shape[0]:
        raise ValueError("counts do not add up to the number of rows")
    p = len(bl)
    traces = np.array([float(np.sum(G[s:e] * G[s:e])) for s, e in bl])
    zero = traces <= ZERO_NORM_REL * traces.max() if p else np.zeros(0, dtype=bool)
    means = worker_means(G, counts)
    D2 = np.zeros((p, p))
    active = np.zeros((p, p), dtype=bool)
    if lam > 0 and p > 1:
        mn = np.einsum("ij,ij->i", means, means)
        for i in range(p):
            for j in range(i + 1, p):
                diff = means[i] - means[j]
                D2[i, j] = D2[j, i] = float(diff @ diff)
        active = D2 > SAME_PAIR_REL * (mn[:, None] + mn[None, :])
        np.fill_diagonal(active, False)
    return G, bl, traces, zero, means, D2, active


def term_values(G, counts, Y, lam, setup=None):
    """u_i = 1 - v_i and u_ij, both as relative squared residuals (no cancellation)."""
    G, bl, traces, zero, means, D2, active = setup if setup is not None else _setup(G, counts, lam)
    p = len(bl)
    R = G - (G @ Y) @ Y.T
    u = np.zeros(p)
    for i, (s, e) in enumerate(bl):
        if not zero[i]:
            u[i] = float(np.sum(R[s:e] * R[s:e])) / traces[i]
    U = np.zeros((p, p))
    if lam > 0 and p > 1:
        Rm = np.stack([R[s:e].mean(axis=0) for s, e in bl])
        for i in range(p):
            for j in range(i + 1, p):
                if active[i, j]:
                    diff = Rm[i] - Rm[j]
                    U[i, j] = U[j, i] = float(diff @ diff) / D2[i, j]
    return u, U


def objective(G, counts, Y, lam, a=2.0) -> float:
    p = len(counts)
    u, U = term_values(G, counts, Y, lam)
    val = float(np.sum(np.maximum(u, 0.0) ** (1.0 / a)))
    if lam > 0 and p > 1:
        val += lam / (p - 1) * float(np.sum(np.maximum(U, 0.0) ** (1.0 / a)))
    return val


def weighted_pca(G, bl, means, w, W, m):
    """m leading eigenvectors of C from the SVD of its sqrt-weighted generating vectors."""
    cols = []
    for i, (s, e) in enumerate(bl):
        if w[i] != 0.0:
            cols.append(np.sqrt(w[i]) * G[s:e])
    p = len(bl)
    for i in range(p):
        for j in range(p):
            if i != j and W[i, j] != 0.0:
                cols.append(np.sqrt(W[i, j]) * (means[i] - means[j])[None, :])
    B = np.concatenate(cols, axis=0).T                      # n x (number of vectors)
    Uleft, s, _ = np.linalg.svd(B, full_matrices=False)
    evals = s * s
    lim = min(m, B.shape[0])
    k = int(np.sum(evals[:lim] > RANK_REL * evals[0])) if evals.size and evals[0] > 0 else 0
    return Uleft[:, :k], evals


def fa_aggregate_multi(G, counts, m, lam=0.0, iters=5, a=2.0, eps=EPS, history=False):
    """`iters` IRLS rounds for workers with counts[i] gradients each.

    returns dict: d (n,), Y (n, k <= m), u (p,), w (p,) last worker weights, objective (per round).
    """
    setup = _setup(G, counts, lam)
    G, bl, traces, zero, means, D2, active = setup
    rows, n = G.shape
    p = len(bl)
    if not (1 <= m <= rows):
        raise ValueError("need 1 <= m <= number of gradients")
    if iters < 1 or lam < 0 or not (a > 1.0):
        raise ValueError("need iters >= 1, lam >= 0 and a > 1")
    coef = lam / (p - 1) if (lam > 0 and p > 1) else 0.0
    if np.all(zero):
        return dict(d=np.zeros(n), Y=np.zeros((n, 0)), u=np.zeros(p), w=np.zeros(p),
                    objective=[0.0] * iters, Ys=[])
    u = np.zeros(p)
    U = np.zeros((p, p))
    objs, Ys = [], []
    for t in range(1, iters + 1):
        w = np.zeros(p)
        W = np.zeros((p, p))
        if t == 1:
            w[~zero] = 1.0
            W[active] = coef
        else:
            r = np.maximum(u, 0.0) ** (1.0 - 1.0 / a)
            w[~zero] = 1.0 / (traces[~zero] * np.maximum(r[~zero], eps))
            if coef > 0:
                Rr = np.maximum(U, 0.0) ** (1.0 - 1.0 / a)
                W[active] = coef / (D2[active] * np.maximum(Rr[active], eps))
        Y, _ = weighted_pca(G, bl, means, w, W, m)
        u, U = term_values(G, counts, Y, lam, setup)
        obj = float(np.sum(np.maximum(u, 0.0) ** (1.0 / a)))
        if coef > 0:
            obj += coef * float(np.sum(np.maximum(U, 0.0) ** (1.0 / a)))
        objs.append(obj)
        if history:
            Ys.append(Y)
    d = Y @ (Y.T @ means.sum(axis=0)) / p
    return dict(d=d, Y=Y, u=u, w=w, objective=objs, Ys=Ys)
