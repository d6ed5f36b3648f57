"""Write tests/golden/<workload>_full.npz: the CPU oracle's result for a workload at its full size.

Run from the repository root:  python tests/golden/make_fullsize_goldens.py cfg3 [cfg4 ...] [--threads T]

Imports only the oracle and the seeded input generators.  The oracle's any-n mode
(fa_aggregate_blocked) visits the gradients in column blocks, so that the fp64 copies of the
n-vectors never have to exist at once.  Stored per workload (everything a p-dimensional
comparison needs, nothing of size n):
  K, D2          inner products and squared pair distances (from the difference vectors)
  objective      Eq. (5) after every round
  u, w           values under the roots and data weights of the last round
  Z              G Y of the last round (p x k): Y^T g_i for every worker; with it the cosines of the
                 principal angles between the oracle's Y and any subspace G^T A are the singular
                 values of Z^T A (after orthonormalising G^T A through K)
  evals, k       spectrum of the last weighted PCA and the number of directions kept
  idx, d_sample  seeded column indices and the aggregate d there; d_norm its full Euclidean norm
  yty_err        max |Y^T Y - I| of the blocked SVD (a check on the oracle run itself)
"""
import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import synthetic_inputs as si            # noqa: E402
from oracle import fa_oracle as fo       # noqa: E402


def sample_indices(w):
    n = w.n
    edge = np.array([0, 1, n // 2, n - 2, n - 1], dtype=np.int64)
    return np.unique(np.concatenate([edge, np.random.default_rng(w.seed).integers(0, n, 8192)]))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("names", nargs="+")
    ap.add_argument("--threads", type=int, default=max(1, (os.cpu_count() or 2) // 2))
    ap.add_argument("--n", type=int, default=None, help="another gradient length (timing the script; not stored)")
    args = ap.parse_args()
    for name in args.names:
        w = si.WORKLOADS[name]
        if args.n:
            w = w.scaled(args.n)
        t0 = time.time()
        G = si.generate(w)
        t1 = time.time()
        idx = sample_indices(w)
        res = fo.fa_aggregate_blocked(G, w.m, w.lam, w.iters, widen=si.to_float64, sample=idx,
                                      threads=args.threads)
        t2 = time.time()
        print(f"{w.name}: generate {t1 - t0:.0f} s, oracle {t2 - t1:.0f} s, k={res['k']}, "
              f"yty_err={res['yty_err']:.2e}, objective {res['objective'][0]:.6f} -> {res['objective'][-1]:.6f}",
              flush=True)
        if args.n:
            continue
        np.savez(os.path.join(os.path.dirname(os.path.abspath(__file__)), f"{name}_full.npz"),
                 K=res["K"], D2=res["D2"], objective=np.asarray(res["objective"]), u=res["u"], w=res["w"],
                 Z=res["Z"], evals=res["evals"], k=np.int64(res["k"]), idx=idx, d_sample=res["d_sample"],
                 d_norm=np.float64(res["d_norm"]), yty_err=np.float64(res["yty_err"]),
                 n=np.int64(w.n), p=np.int64(w.p), m=np.int64(w.m), lam=np.float64(w.lam), iters=np.int64(w.iters),
                 seed=np.int64(w.seed))


if __name__ == "__main__":
    main()
