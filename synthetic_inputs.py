"""Seeded synthetic gradient sets for the Flag Aggregator hot path.

This module only draws random numbers and arranges them into worker-major
p x n gradient matrices.  It contains none of the aggregation arithmetic and
is the one piece of code that both the CPU oracle's tests and the CUDA
path's tests / benchmark import.

The five named workloads are shaped like the settings the paper trains in
(Section 3 "Setup" and the appendix experiments): p = 15 workers with f = 1..3
Byzantine ones on ResNet-18-sized gradients, ResNet-50-sized gradients, the
p = 60 scaling run, and the data-augmentation regime with dependent noise.
They stand in for gradients of those models, which need the datasets.

Recipe (identical on every machine, numpy only):
  * columns are generated in chunks of CHUNK = 2**20; chunk c of a data set
    with seed s uses numpy Generator(PCG64(SeedSequence([s, c]))) and draws,
    in this order, the shared mean chunk and then each logical row's noise;
  * quantities that are not per-column (mixing vectors, the row permutation)
    come from SeedSequence([s, 2**31 - 1]);
  * logical rows are "honest first, Byzantine after"; the stored matrix is a
    fixed seeded permutation of the logical rows;
  * Byzantine rows are computed in fp32 from the true mean unless stated;
  * bf16 storage is round-to-nearest-even of the fp32 value, returned as the
    uint16 bit pattern.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np

CHUNK = 1 << 20
BASE_SEED = 20230205


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str          # which row recipe below
    p: int             # workers
    f: int             # Byzantine workers among them
    n: int             # gradient length
    dtype: str         # "f32" | "bf16" (storage type of G)
    m: int             # subspace dimension
    lam: float         # regularisation weight lambda
    iters: int         # IRLS rounds
    seed: int

    def scaled(self, n: int) -> "Workload":
        """Same recipe at another gradient length (parity-test sizes)."""
        return replace(self, n=int(n), name=f"{self.name}@n={int(n)}")

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def algorithmic_bytes(self) -> int:
        """Two reads of G plus one fp32 write of the aggregate."""
        return 2 * self.p * self.n * self.itemsize + 4 * self.n


WORKLOADS = {
    "cfg1": Workload("cfg1", "signflip", 15, 2, 65_536, "f32", 5, 0.0, 10, BASE_SEED + 1),
    "cfg2": Workload("cfg2", "mixed", 15, 3, 11_173_962, "f32", 8, 1e-2, 10, BASE_SEED + 2),
    "cfg3": Workload("cfg3", "lowrank_shift", 31, 7, 25_557_032, "f32", 12, 1e-2, 20, BASE_SEED + 3),
    "cfg4": Workload("cfg4", "heavytail_two_means", 15, 0, 100_000_000, "f32", 10, 5e-2, 15, BASE_SEED + 4),
    "cfg5": Workload("cfg5", "alie", 63, 15, 124_439_808, "bf16", 16, 1e-2, 20, BASE_SEED + 5),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_float64(G: np.ndarray) -> np.ndarray:
    """Exact widening of a stored gradient matrix (fp32, or bf16 bit patterns)."""
    if G.dtype == np.uint16:
        return bf16_bits_to_f32(G).astype(np.float64)
    return G.astype(np.float64)


def _chunk_rng(seed: int, c: int, stream: int = 0) -> np.random.Generator:
    key = [seed, c] if stream == 0 else [seed, c, stream]
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(key)))


def _global_rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 2**31 - 1])))


def _randn(rng, L):
    return rng.standard_normal(L, dtype=np.float32)


def _n_threads(threads):
    if threads is not None:
        return max(1, int(threads))
    return max(1, min(16, os.cpu_count() or 1))


def row_permutation(w: Workload) -> np.ndarray:
    """perm[r] = logical row stored at position r."""
    g = _global_rng(w.seed)
    return g.permutation(w.p)


def byzantine_positions(w: Workload) -> np.ndarray:
    """Stored row indices that hold Byzantine rows."""
    perm = row_permutation(w)
    return np.nonzero(perm >= w.p - w.f)[0]


def generate(w: Workload, threads: int | None = None) -> np.ndarray:
    """Return G as a C-contiguous (p, n) array: float32, or uint16 bf16 bits."""
    p, f, n = w.p, w.f, w.n
    h = p - f
    g = _global_rng(w.seed)
    perm = g.permutation(p)                 # same first draw as row_permutation()
    inv = np.empty(p, dtype=np.int64)
    inv[perm] = np.arange(p)                # logical row l is stored at inv[l]
    out_dtype = np.float32 if w.dtype == "f32" else np.uint16
    G = np.empty((p, n), dtype=out_dtype)
    n_chunks = (n + CHUNK - 1) // CHUNK

    extra = {}
    if w.kind == "lowrank_shift":
        extra["z"] = g.standard_normal((h, 4)).astype(np.float32)
        # exact unit directions need the norms of the raw draws first
        def _norm2(c):
            L = min(CHUNK, n - c * CHUNK)
            r = _chunk_rng(w.seed, c, 1)
            return [float(np.sum(_randn(r, L).astype(np.float64) ** 2)) for _ in range(f)]
        with ThreadPoolExecutor(_n_threads(threads)) as ex:
            parts = list(ex.map(_norm2, range(n_chunks)))
        extra["unorm"] = np.sqrt(np.sum(np.asarray(parts, dtype=np.float64), axis=0))

    def store(c0, L, logical_row, values_f32):
        dst = G[inv[logical_row], c0:c0 + L]
        if out_dtype is np.float32:
            dst[:] = values_f32
        else:
            dst[:] = f32_to_bf16_bits(values_f32)

    def do_chunk(c):
        c0 = c * CHUNK
        L = min(CHUNK, n - c0)
        r = _chunk_rng(w.seed, c)
        kind = w.kind
        if kind == "signflip":            # honest mu + 0.5 N(0,I); Byzantine both -4 mu
            mu = _randn(r, L)
            for l in range(h):
                store(c0, L, l, mu + np.float32(0.5) * _randn(r, L))
            for l in range(h, p):
                store(c0, L, l, np.float32(-4.0) * mu)
        elif kind == "mixed":             # honest mu + 0.3 N; Byzantine 10 N(0,I), -10 mu, 0
            mu = _randn(r, L)
            for l in range(h):
                store(c0, L, l, mu + np.float32(0.3) * _randn(r, L))
            byz = [np.float32(10.0) * _randn(r, L), np.float32(-10.0) * mu,
                   np.zeros(L, dtype=np.float32)]
            for k, l in enumerate(range(h, p)):
                store(c0, L, l, byz[k % 3] if k < 3 else np.float32(10.0) * _randn(r, L))
        elif kind == "lowrank_shift":     # honest U z_i + 0.2 N; Byzantine honest mean + 50 u_b
            U = r.standard_normal((L, 4), dtype=np.float32)
            acc = np.zeros(L, dtype=np.float32)
            for l in range(h):
                row = U @ extra["z"][l] + np.float32(0.2) * _randn(r, L)
                acc += row
                store(c0, L, l, row)
            mean_h = acc / np.float32(h)
            rb = _chunk_rng(w.seed, c, 1)
            for k, l in enumerate(range(h, p)):
                u = _randn(rb, L) / np.float32(extra["unorm"][k])
                store(c0, L, l, mean_h + np.float32(50.0) * u)
        elif kind == "heavytail_two_means":   # Student-t(3) noise, 4 rows around a second mean
            mu = _randn(r, L)
            mu2 = mu + np.float32(np.sqrt(0.5)) * _randn(r, L)
            n_second = min(4, p)
            for l in range(p):
                t = r.standard_t(3.0, L).astype(np.float32)
                base = mu2 if l >= p - f - n_second and l < p - f else mu
                store(c0, L, l, base + np.float32(0.5) * t)
        elif kind == "alie":              # honest mu + 0.3 N; Byzantine mean_h - 1.5 std_h
            mu = _randn(r, L)
            H = np.empty((h, L), dtype=np.float32)
            for l in range(h):
                H[l] = mu + np.float32(0.3) * _randn(r, L)
                store(c0, L, l, H[l])
            mean_h = H.mean(axis=0, dtype=np.float32)
            std_h = H.std(axis=0, dtype=np.float32)
            b = mean_h - np.float32(1.5) * std_h
            for l in range(h, p):
                store(c0, L, l, b)
        else:
            raise ValueError(f"unknown workload kind {kind!r}")

    with ThreadPoolExecutor(_n_threads(threads)) as ex:
        list(ex.map(do_chunk, range(n_chunks)))
    return G


# ----------------------------------------------------------------------------
# Small structured cases for the correctness ladder (fp32 unless bf16=True).
# ----------------------------------------------------------------------------

def ladder_case(p: int, n: int, seed: int, kind: str = "noisy_mean", bf16: bool = False) -> np.ndarray:
    """Tiny / medium matrices with the same flavour as the workloads.

    kinds: "noisy_mean"  mu + 0.4 N(0,I), last max(1,p//5) rows (p>=4) large random outliers
           "gauss"       i.i.d. N(0,I) rows with row scales spread over 1e-2..1e2
           "dup_zero"    noisy_mean, then row 1 := row 0 and the last row := 0 (p>=3)
    """
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, p, n, 77])))
    if kind == "gauss":
        G = rng.standard_normal((p, n)).astype(np.float32)
        scales = np.float32(10.0) ** rng.uniform(-2, 2, size=(p, 1)).astype(np.float32)
        G = (G * scales).astype(np.float32)
    else:
        mu = rng.standard_normal(n).astype(np.float32)
        G = (mu[None, :] + np.float32(0.4) * rng.standard_normal((p, n)).astype(np.float32)).astype(np.float32)
        if p >= 4:
            k = max(1, p // 5)
            G[p - k:] = np.float32(5.0) * rng.standard_normal((k, n)).astype(np.float32)
        if kind == "dup_zero" and p >= 3:
            G[1] = G[0]
            G[p - 1] = 0
        elif kind not in ("noisy_mean", "dup_zero"):
            raise ValueError(kind)
    G = np.ascontiguousarray(G, dtype=np.float32)
    return f32_to_bf16_bits(G) if bf16 else G
