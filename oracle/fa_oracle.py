"""TEST INFRASTRUCTURE -- plain fp64 CPU statement of the Flag Aggregator step.

Nothing in the product path may import this file: it exists so that tests, the
smoke check and the benchmark's CPU-baseline leg have something slow and
readable to compare the CUDA path against.  It shares no code with the CUDA
path and works directly on n-dimensional vectors.

What it computes (Flag Aggregator paper, arXiv 2302.05865):

  * gradients g_1..g_p in R^n, the rows of the worker-major array G (the
    paper's gradient matrix, Section 2.1, is its transpose);
  * the subspace Y (n x m, orthonormal columns) that the iteratively
    reweighted least-squares ("flag mean") procedure of Algorithm 1 reaches
    for the objective of Eq. (5) with the data-dependent regulariser (2) of
    Section 2.3,
        A(Y) = sum_i sqrt(1 - ||Y^T g_i||^2 / ||g_i||^2)
             + lam/(p-1) * sum_{i != j} sqrt(1 - ||Y^T (g_i-g_j)||^2 / D_ij^2),
    D_ij^2 = ||g_i - g_j||^2;
  * the update direction d = (1/p) Y Y^T G 1 of Algorithm 1.

How each round is taken (the paper names the procedure but prints no update
formula; this is the reading used, each item listed in the design notes):

  * the first round uses uniform weights, so it is PCA of the gradient matrix
    (appendix "Experiments with other Byzantine attacks or baselines");
  * later rounds reweight every square-root term of the objective by
    1 / (normaliser * sqrt(term's current value)) -- for the data terms this
    is -d_i of the appendix equation defining g-tilde_i -- and take the m
    leading eigenvectors of
        C = sum_i w_i g_i g_i^T + sum_{i != j} w_ij (g_i-g_j)(g_i-g_j)^T,
    i.e. one weighted PCA;
  * the value under each square root is evaluated as the relative squared
    residual ||x - Y Y^T x||^2 / ||x||^2, which equals 1 - ||Y^T x||^2/||x||^2
    for orthonormal Y (Section 2.1) and does not cancel;
  * sqrt(.) in a weight is floored at EPS; zero gradients and identical pairs
    carry weight 0 and contribute 0 to the objective; eigen-directions whose
    eigenvalue is <= RANK_REL * largest are left out of Y;
  * exactly `iters` rounds are run unless a tolerance is given (see fa_aggregate).

Two ways of getting the eigenvectors of C are provided and tested against
each other: "literal" builds the n x n matrix C term by term (small n only);
"svd" uses C = B B^T with B = G^T M^(1/2), M = diag(w) + sum w_ij (e_i-e_j)
(e_i-e_j)^T, and takes the left singular vectors of the n x p matrix B.

fa_aggregate_blocked is the "svd" iteration for gradient lengths whose fp64
copies do not fit in memory: the same rounds with every n-vector visited in
column blocks (the thin SVD of B through the triangular factor of a QR that
takes B one block of rows at a time).  It is pinned against fa_aggregate.

Parity pins (tests/test_oracle_pins.py): mean recovery, orthonormality and
ratio range, PCA special case, worker-permutation and scaling invariance,
monotone descent, first-order stationarity of Eq. (5) at the fixed point by
finite differences, the right-multiplication form of the appendix KKT section,
brute force over the Grassmannian for n <= 4, the Kronecker/trace identity of
Lemma "Equivalence of Objective Functions", m = p, literal vs svd.
"""
from __future__ import annotations

import numpy as np

EPS = 1e-6              # floor on sqrt(1 - v) inside a weight
ZERO_NORM_REL = 1e-30   # ||g_i||^2 <= this * max_k ||g_k||^2  => zero gradient
SAME_PAIR_REL = 1e-12   # D_ij^2 <= this * (||g_i||^2 + ||g_j||^2) => identical pair
RANK_REL = 1e-12        # eigenvalue <= this * largest => direction dropped from Y


# -- plain definitions -------------------------------------------------------

def inner_products(G: np.ndarray) -> np.ndarray:
    """K_ij = <g_i, g_j> (Section 2.1: ||g_i||^2 on the diagonal)."""
    G = np.asarray(G, dtype=np.float64)
    return G @ G.T


def pair_sqdist(G: np.ndarray) -> np.ndarray:
    """D_ij^2 = ||g_i - g_j||^2 from the difference vector (Section 2.3, item 2)."""
    G = np.asarray(G, dtype=np.float64)
    p = G.shape[0]
    D2 = np.zeros((p, p))
    for i in range(p):
        for j in range(i + 1, p):
            diff = G[i] - G[j]
            D2[i, j] = D2[j, i] = float(diff @ diff)
    return D2


def _classify(G):
    p = G.shape[0]
    norms = np.einsum("ij,ij->i", G, G)
    top = float(norms.max()) if p else 0.0
    zero = norms <= ZERO_NORM_REL * top
    return norms, zero


def _pairs(G, norms, lam):
    """D_ij^2 and the mask of pairs that take part (i != j, not identical)."""
    p = G.shape[0]
    if lam <= 0 or p < 2:
        return np.zeros((p, p)), np.zeros((p, p), dtype=bool)
    D2 = pair_sqdist(G)
    active = D2 > SAME_PAIR_REL * (norms[:, None] + norms[None, :])
    np.fill_diagonal(active, False)
    return D2, active


def residuals(G, Y):
    """Rows r_i = g_i - Y Y^T g_i (what the subspace does not reconstruct, Section 2.1)."""
    return G - (G @ Y) @ Y.T


def term_values(G, Y, lam, norms=None, zero=None, D2=None, active=None):
    """u_i and u_ij: the quantities under the square roots of Eq. (5).

    The projector is linear, so the residual of g_i - g_j is r_i - r_j.
    """
    G = np.asarray(G, dtype=np.float64)
    p = G.shape[0]
    if norms is None:
        norms, zero = _classify(G)
    if D2 is None:
        D2, active = _pairs(G, norms, lam)
    R = residuals(G, Y)
    u = np.zeros(p)
    for i in range(p):
        if not zero[i]:
            u[i] = float(R[i] @ R[i]) / norms[i]
    U = np.zeros((p, p))
    if lam > 0:
        for i in range(p):
            for j in range(i + 1, p):
                if active[i, j]:
                    diff = R[i] - R[j]
                    U[i, j] = U[j, i] = float(diff @ diff) / D2[i, j]
    return u, U


def objective(G, Y, lam, a=2.0) -> float:
    """A(Y) of Eq. (5) with regulariser (2); the pair sum runs over ordered pairs.

    a is the constant of the Taylor surrogate of Eq. (4): each term is (1 - v)^(1/a); a = 2 (the
    paper's choice, Section 2.3) gives the square roots of Eq. (5).  The constant factor a and
    the offset -a of Eq. (4) do not move the minimiser and are left out.
    """
    G = np.asarray(G, dtype=np.float64)
    p = G.shape[0]
    u, U = term_values(G, Y, lam)
    val = float(np.sum(np.maximum(u, 0.0) ** (1.0 / a)))
    if lam > 0 and p > 1:
        val += lam / (p - 1) * float(np.sum(np.maximum(U, 0.0) ** (1.0 / a)))
    return val


# -- one weighted PCA ----------------------------------------------------------

def _keep(evals_desc, m):
    if evals_desc.size == 0 or evals_desc[0] <= 0:
        return 0
    return int(np.sum(evals_desc[:m] > RANK_REL * evals_desc[0]))


def weighted_pca_literal(G, w, W, m):
    """Leading eigenvectors of C built term by term as an n x n matrix."""
    p, n = G.shape
    C = np.zeros((n, n))
    for i in range(p):
        if w[i] != 0.0:
            C += w[i] * np.outer(G[i], G[i])
    for i in range(p):
        for j in range(p):
            if i != j and W[i, j] != 0.0:
                x = G[i] - G[j]
                C += W[i, j] * np.outer(x, x)
    evals, evecs = np.linalg.eigh(C)
    evals, evecs = evals[::-1], evecs[:, ::-1]
    k = _keep(evals, min(m, n))
    return evecs[:, :k], evals


def pair_weight_matrix(w, W):
    """M with C = G^T M G for worker-major G: diag(w) + sum_{i != j} W_ij (e_i-e_j)(e_i-e_j)^T."""
    p = w.shape[0]
    M = np.diag(np.asarray(w, dtype=np.float64))
    for i in range(p):
        for j in range(p):
            if i != j and W[i, j] != 0.0:
                M[i, i] += W[i, j]
                M[j, j] += W[i, j]
                M[i, j] -= W[i, j]
                M[j, i] -= W[i, j]
    return M


def weighted_pca_qr(G, w, W, m):
    """Same subspace when some weights are negative (C indefinite): with the thin QR G^T = Q R,
    C = G^T M G = Q (R M R^T) Q^T, so the eigenvectors of C with non-zero eigenvalue are Q times
    those of the p x p matrix R M R^T."""
    M = pair_weight_matrix(w, W)
    Q, R = np.linalg.qr(G.T)
    S = R @ M @ R.T
    evals, V = np.linalg.eigh(0.5 * (S + S.T))
    evals, V = evals[::-1], V[:, ::-1]
    k = _keep(evals, min(m, G.shape[1]))
    return Q @ V[:, :k], evals


def weighted_pca_svd(G, w, W, m):
    """Same subspace from the thin SVD of B = G^T M^(1/2) (n x p)."""
    p, n = G.shape
    if np.any(W != 0.0):
        M = pair_weight_matrix(w, W)
        e, E = np.linalg.eigh(M)
        S = E * np.sqrt(np.maximum(e, 0.0))[None, :]      # S S^T = M
        B = G.T @ S
    else:
        B = G.T * np.sqrt(w)[None, :]
    Uleft, s, _ = np.linalg.svd(B, full_matrices=False)
    evals = s * s
    k = _keep(evals, min(m, n))
    return Uleft[:, :k], evals


# -- the iteration -------------------------------------------------------------

def fa_aggregate(G, m, lam=0.0, iters=5, method="svd", eps=EPS, history=False, a=2.0, Y0=None, tol=None,
                 alpha=1.0, beta=0.5):
    """Run `iters` IRLS rounds and return the aggregate.

    G      : (p, n) array, rows are worker gradients (converted to float64)
    a      : surrogate constant of Eq. (4), a > 1; terms are (1 - v)^(1/a) and the reweighting
             of a term with value u is 1 / (normaliser * max(u^(1 - 1/a), eps))  (a = 2: the paper's
             square roots)
    alpha, beta : shape parameters of the Beta likelihood of the values v_i (Eq. (1) uses alpha = 1,
             beta = 1/2).  The negative log-likelihood -(alpha-1) log v - (beta-1) log(1-v), with
             the surrogate log x ~ a x^(1/a) - a of Eq. (4) on both logarithms (the "two terms" of the
             extension paragraph of Section 2.2) and the scale in which alpha = 1, beta = 1/2 gives
             the data term of Eq. (5), is the data term
                 2 (1 - beta) (1 - v_i)^(1/a) + 2 (1 - alpha) v_i^(1/a).
             Both terms are concave in v_i for alpha <= 1, beta <= 1 (required here), so the tangent
             majoriser gives the weight
                 [2 (1 - beta) / max(u_i^(1-1/a), eps) - 2 (1 - alpha) / max(v_i^(1-1/a), eps)] / ||g_i||^2,
             which may be negative; C is then indefinite and only eigen-directions with positive
             eigenvalue enter Y.
    Y0     : optional (n, k) matrix of full column rank, a subspace to start from (the "smart
             initialization" Section 2.1 mentions): round one then reweights by the term values at
             span(Y0) instead of being uniform.  A Y0 of rank 0 (or None) is the cold start.
    tol    : optional; stop after round t >= 2 once |objective_{t-1} - objective_t| <= tol (the
             "small error" convergence criterion of the implementation details in Section 3,
             which the paper pairs with a cap on the rounds: `iters` is that cap)
    returns: dict with d (n,), Y (n, k<=m), u (p,), w (p,) last data weights,
             objective (list, one per round run), rounds, evals (last round, descending),
             and with history=True the list of Y per round.
    """
    G = np.asarray(G, dtype=np.float64)
    p, n = G.shape
    if not (1 <= m <= p):
        raise ValueError("need 1 <= m <= p")
    if iters < 1 or lam < 0 or not (a > 1.0):
        raise ValueError("need iters >= 1, lam >= 0 and a > 1")
    if not (0.0 < alpha <= 1.0 and 0.0 < beta <= 1.0):
        raise ValueError("need 0 < alpha <= 1 and 0 < beta <= 1")
    norms, zero = _classify(G)
    D2, active = _pairs(G, norms, lam)
    coef = lam / (p - 1) if (lam > 0 and p > 1) else 0.0
    cb, ca = 2.0 * (1.0 - beta), 2.0 * (1.0 - alpha)
    if method == "literal":
        pca = weighted_pca_literal
    elif ca != 0.0 or method == "qr":
        pca = weighted_pca_qr
    else:
        pca = weighted_pca_svd

    def explained(Y):
        """v_i = ||Y^T g_i||^2 / ||g_i||^2 (Section 2.1), 0 for a zero gradient."""
        Z = G @ Y
        v = np.zeros(p)
        v[~zero] = np.einsum("ij,ij->i", Z, Z)[~zero] / norms[~zero]
        return v

    def data_terms(u, v):
        t = np.maximum(u, 0.0) ** (1.0 / a) if cb == 1.0 else cb * np.maximum(u, 0.0) ** (1.0 / a)
        if ca != 0.0:
            t = t + ca * np.where(zero, 0.0, np.maximum(v, 0.0) ** (1.0 / a))
        return float(np.sum(t))

    if np.all(zero):                       # every gradient is zero: nothing to span
        return dict(d=np.zeros(n), Y=np.zeros((n, 0)), u=np.zeros(p), w=np.zeros(p),
                    objective=[0.0] * iters, rounds=iters, evals=np.zeros(p), Ys=[])

    u = np.zeros(p)
    v = np.zeros(p)
    U = np.zeros((p, p))
    warm = False
    if Y0 is not None and np.asarray(Y0).size:
        Q, R = np.linalg.qr(np.asarray(Y0, dtype=np.float64))
        diag = np.abs(np.diag(R))
        if diag.size and diag.min() > 1e-12 * diag.max():
            u, U = term_values(G, Q, lam, norms, zero, D2, active)
            v = explained(Q)
            warm = True
    objs, Ys = [], []
    for t in range(1, iters + 1):
        w = np.zeros(p)
        W = np.zeros((p, p))
        if t == 1 and not warm:
            w[~zero] = 1.0
            W[active] = coef
        else:
            r = np.maximum(u, 0.0) ** (1.0 - 1.0 / a)
            if cb == 1.0 and ca == 0.0:
                w[~zero] = 1.0 / (norms[~zero] * np.maximum(r[~zero], eps))
            else:
                rv = np.maximum(v, 0.0) ** (1.0 - 1.0 / a)
                w[~zero] = (cb / np.maximum(r[~zero], eps) - ca / np.maximum(rv[~zero], eps)) / norms[~zero]
            if coef > 0:
                R = np.maximum(U, 0.0) ** (1.0 - 1.0 / a)
                W[active] = coef / (D2[active] * np.maximum(R[active], eps))
        Y, evals = pca(G, w, W, m)
        u, U = term_values(G, Y, lam, norms, zero, D2, active)
        v = explained(Y)
        obj = data_terms(u, v)
        if coef > 0:
            obj += coef * float(np.sum(np.maximum(U, 0.0) ** (1.0 / a)))
        objs.append(obj)
        if history:
            Ys.append(Y)
        if tol is not None and t >= 2 and abs(objs[-2] - objs[-1]) <= tol:
            break
    d = Y @ (Y.T @ G.sum(axis=0)) / p
    return dict(d=d, Y=Y, u=u, w=w, objective=objs, rounds=len(objs), evals=evals, Ys=Ys)


# -- the same iteration for any n: every n-vector is visited in column blocks ----------------

def _blocks(n, block):
    return [(c0, min(c0 + block, n)) for c0 in range(0, n, block)]


def _for_blocks(fn, spans, threads):
    """fn(c0, c1) for every column block, results in block order (plain loop unless threads > 1)."""
    if threads <= 1:
        return [fn(c0, c1) for c0, c1 in spans]
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(threads) as ex:
        return list(ex.map(lambda s: fn(*s), spans))


def fa_aggregate_blocked(G, m, lam=0.0, iters=5, block=1 << 16, widen=None, eps=EPS, sample=None, threads=1):
    """fa_aggregate(..., method="svd") with a = 2 and the Beta(1, 1/2) likelihood of Eq. (1), for any n.

    The rounds, weights, term values and the final average are those of fa_aggregate; what changes
    is only how the n-dimensional objects are held.  G stays in its storage type and is widened
    to fp64 one column block at a time (`widen`, default: plain conversion), and Y (n x m) is never
    kept: per round
      1. the thin SVD of B = G^T M^(1/2) (n x p) is taken through a QR that sees B one block of
         rows at a time (R of [R_so_far; B_block]), then R = U S V^T, so that B = (Q U) S V^T and the
         left singular vectors are Y = B V S^-1, formed block by block;
      2. Z = G Y (p x k: the coordinates Y^T g_i of every gradient) is summed over the blocks;
      3. the residual rows r_i = g_i - Y Y^T g_i are formed block by block and their squared norms,
         and those of the explicit differences r_i - r_j of the active pairs, are summed.
    After the last round d = (1/p) Y (Y^T G 1) is formed block by block.

    sample  : optional integer array of column indices; d is then returned only there (d_sample),
              together with its full norm (d_norm), instead of as a full vector
    threads : column blocks of one pass may be worked on by this many threads (sums are still added
              in block order)
    returns : dict with objective (one per round), u, w, evals (last round), k, Z = G Y (p x k) of the
              last round, yty_err = max |Y^T Y - I| of the last round, K = G G^T, D2, d or
              (d_sample, d_norm).
    """
    p, n = G.shape
    if widen is None:
        widen = lambda x: np.asarray(x, dtype=np.float64)
    if not (1 <= m <= p) or iters < 1 or lam < 0:
        raise ValueError("need 1 <= m <= p, iters >= 1, lam >= 0")
    spans = _blocks(n, int(block))
    coef = lam / (p - 1) if (lam > 0 and p > 1) else 0.0

    # inner products, and D_ij^2 from the difference vectors
    def first_pass(c0, c1):
        X = widen(G[:, c0:c1])
        return X @ X.T, (pair_sqdist(X) if coef > 0 else None)
    K = np.zeros((p, p))
    D2 = np.zeros((p, p))
    for Kb, Db in _for_blocks(first_pass, spans, threads):
        K += Kb
        if Db is not None:
            D2 += Db
    norms = np.diag(K).copy()
    zero = norms <= ZERO_NORM_REL * float(norms.max())
    active = np.zeros((p, p), dtype=bool)
    if coef > 0:
        active = D2 > SAME_PAIR_REL * (norms[:, None] + norms[None, :])
        np.fill_diagonal(active, False)
    if np.all(zero):
        out = dict(objective=[0.0] * iters, u=np.zeros(p), w=np.zeros(p), evals=np.zeros(p), k=0,
                   Z=np.zeros((p, 0)), yty_err=0.0, K=K, D2=D2)
        if sample is None:
            out["d"] = np.zeros(n)
        else:
            out["d_sample"], out["d_norm"] = np.zeros(len(sample)), 0.0
        return out

    u = np.zeros(p)
    U = np.zeros((p, p))
    objs = []
    for t in range(1, iters + 1):
        w = np.zeros(p)
        W = np.zeros((p, p))
        if t == 1:
            w[~zero] = 1.0
            W[active] = coef
        else:
            w[~zero] = 1.0 / (norms[~zero] * np.maximum(np.sqrt(np.maximum(u[~zero], 0.0)), eps))
            if coef > 0:
                W[active] = coef / (D2[active] * np.maximum(np.sqrt(np.maximum(U[active], 0.0)), eps))
        # M^(1/2) as in weighted_pca_svd
        if np.any(W != 0.0):
            e, E = np.linalg.eigh(pair_weight_matrix(w, W))
            S = E * np.sqrt(np.maximum(e, 0.0))[None, :]
        else:
            S = np.diag(np.sqrt(w))
        # 1. triangular factor of B, one block of rows at a time
        Rfac = np.zeros((0, p))
        for B in _for_blocks(lambda c0, c1: np.linalg.qr(widen(G[:, c0:c1]).T @ S, mode="r"), spans, threads):
            Rfac = np.linalg.qr(np.vstack([Rfac, B]), mode="r")
        _, sv, Vt = np.linalg.svd(Rfac)
        evals = sv * sv
        k = _keep(evals, min(m, n))
        Ymap = S @ (Vt[:k].T / sv[:k][None, :])          # Y_block = G_block^T Ymap  (= B_block V S^-1)
        # 2. coordinates of every gradient, and Y^T Y as a check on the blocked SVD
        def second_pass(c0, c1):
            X = widen(G[:, c0:c1])
            Yb = X.T @ Ymap
            return X @ Yb, Yb.T @ Yb
        Z = np.zeros((p, k))
        YtY = np.zeros((k, k))
        for Zb, Yb2 in _for_blocks(second_pass, spans, threads):
            Z += Zb
            YtY += Yb2
        # 3. residual rows and the values under the roots of Eq. (5)
        def third_pass(c0, c1):
            X = widen(G[:, c0:c1])
            R = X - Z @ (X.T @ Ymap).T
            return np.einsum("ij,ij->i", R, R), (pair_sqdist(R) if coef > 0 else None)
        rr = np.zeros(p)
        RR = np.zeros((p, p))
        for rb, Rb in _for_blocks(third_pass, spans, threads):
            rr += rb
            if Rb is not None:
                RR += Rb
        u = np.zeros(p)
        u[~zero] = rr[~zero] / norms[~zero]
        U = np.zeros((p, p))
        U[active] = RR[active] / D2[active]
        obj = float(np.sum(np.sqrt(np.maximum(u, 0.0))))
        if coef > 0:
            obj += coef * float(np.sum(np.sqrt(np.maximum(U, 0.0))))
        objs.append(obj)

    # d = (1/p) Y (Y^T sum_i g_i); Y^T sum_i g_i = sum_i Z[i]
    zsum = Z.sum(axis=0) / p
    out = dict(objective=objs, u=u, w=w, evals=evals, k=k, Z=Z, K=K, D2=D2,
               yty_err=float(np.abs(YtY - np.eye(k)).max()) if k else 0.0)
    if sample is None:
        d = np.empty(n)
        for c0, c1 in spans:
            d[c0:c1] = (widen(G[:, c0:c1]).T @ Ymap) @ zsum
        out["d"] = d
    else:
        sample = np.asarray(sample, dtype=np.int64)
        d_sample = np.empty(sample.size)
        norm2 = 0.0
        for c0, c1 in spans:
            db = (widen(G[:, c0:c1]).T @ Ymap) @ zsum
            norm2 += float(db @ db)
            sel = (sample >= c0) & (sample < c1)
            d_sample[sel] = db[sample[sel] - c0]
        out["d_sample"], out["d_norm"] = d_sample, float(np.sqrt(norm2))
    return out


def reconstruction(G, Y):
    """Y Y^T g_i for every worker, as rows (the reconstruction Y Y^T G of Section 2.1, transposed)."""
    G = np.asarray(G, dtype=np.float64)
    return (G @ Y) @ Y.T


# -- comparison helpers ----------------------------------------------------------

def principal_angles(Ya, Yb) -> np.ndarray:
    """asin of the singular values of (I - Ya Ya^T) Yb, largest first (radians)."""
    Ya = np.asarray(Ya, dtype=np.float64)
    Yb = np.asarray(Yb, dtype=np.float64)
    if Ya.shape[1] == 0 or Yb.shape[1] == 0:
        return np.zeros(0)
    R = Yb - Ya @ (Ya.T @ Yb)
    s = np.linalg.svd(R, compute_uv=False)
    return np.arcsin(np.clip(s, 0.0, 1.0))


def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / den if den > 0 else float(np.linalg.norm(a))
