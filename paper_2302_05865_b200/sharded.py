"""The Flag Aggregator step on several GPUs, one process per GPU, gradients sharded along n.

The step depends on the gradients only through K = G G^T, and K is a sum over columns.  So rank r
keeps columns [lo_r, hi_r) of all p gradients, runs the Gram pass on them, the p x p partial sums
are added across ranks (ONE all-reduce of p*p doubles: 1.8 KB at p = 15), every rank runs the same
deterministic IRLS kernel on the same K, and the output pass writes the rank's slice of
d = (1/p) Y Y^T G 1 (Algorithm 1, last line of the server part).

When the gradients start out on their workers (rank i holds the whole of its own gradients: the
data-parallel situation of Algorithm 1, without the parameter server), `WorkerResidentStep` first
re-shards with one all-to-all -- each rank sends (N-1)/N of its gradient bytes, the volume of a
reduce-scatter -- and ends with an all-gather of the slices of d, together the wire traffic of the
ring all-reduce that plain averaging would use.  Received slices land in this GPU's own memory
first; the kernels never read a peer's memory.

Only orchestration lives here: the three kernels are the package's entry points (`ops` can be
replaced by stand-ins with the same call signatures, which is how the rank logic is exercised
on CPU processes).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

SHARD_ALIGN = 8     # columns per shard are a multiple of this: rows stay 16-byte aligned for bf16


def shard_size(n: int, world: int) -> int:
    """Columns per rank (the last non-empty rank may hold fewer, later ones none)."""
    per = (n + world - 1) // world
    return (per + SHARD_ALIGN - 1) // SHARD_ALIGN * SHARD_ALIGN


def shard_bounds(n: int, world: int, rank: int):
    per = shard_size(n, world)
    lo = min(n, rank * per)
    return lo, min(n, lo + per)


class ShardedStep:
    """fa_aggregate for a rank that holds columns [lo, hi) of every gradient.

    reduce_fn(K) must leave the sum of all ranks' K in K on every rank; the default is
    torch.distributed.all_reduce on `group`.  A rank whose shard is empty still takes part.
    """

    def __init__(self, m, lam, iters, group=None, ops=None, reduce_fn=None):
        if ops is None:
            import paper_2302_05865_b200 as ops       # the CUDA entry points; raises if not built
        self.ops, self.m, self.lam, self.iters, self.group = ops, m, lam, iters, group
        self.reduce_fn = reduce_fn if reduce_fn is not None else self._all_reduce
        self.K = self.c = self.ws = None          # per-shape buffers, allocated on first use

    def _all_reduce(self, K):
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1:
            dist.all_reduce(K, op=dist.ReduceOp.SUM, group=self.group)

    def coefficients(self, G_shard):
        """c (p,) with d = sum_i c_i g_i, from this rank's columns and the other ranks' partial sums."""
        p, cols = int(G_shard.shape[0]), int(G_shard.shape[1])
        key = (p, cols, G_shard.dtype, G_shard.device)
        if self.K is None or self._key != key:
            self._key = key
            self.K = torch.zeros((p, p), dtype=torch.float64, device=G_shard.device)
            self.c = torch.zeros(p, dtype=torch.float32, device=G_shard.device)
            make_ws = getattr(self.ops, "new_workspace", None)
            self.ws = make_ws(G_shard, self.m) if (make_ws and cols > 0) else None
        if cols > 0:
            self.ops.fa_gram(G_shard, K=self.K, ws=self.ws)
        else:
            self.K.zero_()
        self.reduce_fn(self.K)
        return self.ops.fa_irls(self.K, self.m, self.lam, self.iters, c_out=self.c)

    def __call__(self, G_shard, out=None):
        c = self.coefficients(G_shard)
        cols = int(G_shard.shape[1])
        if out is None:
            out = torch.empty(cols, dtype=torch.float32, device=G_shard.device)
        if cols > 0:
            self.ops.fa_combine(G_shard, c, out=out)
        return out


class WorkerResidentStep:
    """Every rank starts with the full-length gradients of its own workers (rows_local x n) and ends
    with the full aggregate d (n,).  counts_per_rank[r] = number of gradients rank r holds."""

    def __init__(self, n, counts_per_rank, m, lam, iters, group=None, ops=None):
        self.n, self.counts, self.group = int(n), [int(k) for k in counts_per_rank], group
        self.world = len(self.counts)
        self.per = shard_size(self.n, self.world)
        self.step = ShardedStep(m, lam, iters, group=group, ops=ops)

    def reshard(self, g_own):
        """all-to-all: returns this rank's column shard of ALL gradients, (p, hi - lo) row-major."""
        rank = dist.get_rank(self.group)
        k_own = self.counts[rank]
        assert g_own.shape == (k_own, self.n)
        bounds = [shard_bounds(self.n, self.world, r) for r in range(self.world)]
        lo, hi = bounds[rank]
        p = sum(self.counts)
        G_shard = torch.empty((p, hi - lo), dtype=g_own.dtype, device=g_own.device)
        if k_own == 1:                      # column slices of one row are contiguous: send in place
            send = g_own.reshape(-1)
        else:                               # pack (k_own x cols_r) blocks, destination by destination
            send = torch.cat([g_own[:, a:b].reshape(-1) for a, b in bounds])
        in_splits = [k_own * (b - a) for a, b in bounds]
        out_splits = [k * (hi - lo) for k in self.counts]
        dist.all_to_all_single(G_shard.view(-1), send, output_split_sizes=out_splits,
                               input_split_sizes=in_splits, group=self.group)
        return G_shard

    def __call__(self, g_own):
        rank = dist.get_rank(self.group)
        G_shard = self.reshard(g_own)
        lo, hi = shard_bounds(self.n, self.world, rank)
        gathered = torch.zeros(self.world * self.per, dtype=torch.float32, device=g_own.device)
        mine = gathered[rank * self.per: rank * self.per + self.per]
        self.step(G_shard, out=mine[: hi - lo])
        dist.all_gather_into_tensor(gathered, mine.clone(), group=self.group)
        return gathered[: self.n]
