"""Rank logic of the n-sharded step on CPU processes (gloo): shard bounds, the all-reduce of the partial
inner products, the all-to-all re-shard of worker-resident gradients and the all-gather of the output
slices.  The three kernels are replaced by CPU stand-ins with the same call signatures, built on the
oracle; what is on trial is the orchestration, compared with the oracle on the unsharded matrix."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleOps:
    """Stand-ins for fa_gram / fa_irls / fa_combine on CPU tensors."""

    @staticmethod
    def fa_gram(G, K=None, ws=None):
        import torch
        from oracle import fa_oracle as fo
        K.copy_(torch.from_numpy(fo.inner_products(G.numpy())))
        return K

    @staticmethod
    def fa_irls(K, m, lam, iters, c_out=None):
        """The step depends on the gradients only through K: any L with L L^T = K gives the same c."""
        import torch
        from oracle import fa_oracle as fo
        Kh = K.numpy()
        e, V = np.linalg.eigh(0.5 * (Kh + Kh.T))
        L = V * np.sqrt(np.maximum(e, 0.0))[None, :]             # rows l_i with <l_i, l_j> = K_ij
        ref = fo.fa_aggregate(L, m, lam, iters)
        c = ref["d"] @ np.linalg.pinv(L)                          # d_L = sum_i c_i l_i
        c_out.copy_(torch.from_numpy(c.astype(np.float32)))
        return c_out

    @staticmethod
    def fa_combine(G, c, out=None):
        import torch
        out.copy_((c.double() @ G.double()).float())
        return out


def _case(p, n, seed):
    r = np.random.default_rng(seed)
    mu = r.standard_normal(n)
    G = mu[None, :] + 0.4 * r.standard_normal((p, n))
    G[-2:] = 5.0 * r.standard_normal((2, n))
    return G.astype(np.float32)


def _rank_main(rank, world, port, q, n, counts):
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    from paper_2302_05865_b200 import sharded
    p = sum(counts)
    G = torch.from_numpy(_case(p, n, 5))
    # (1) column-sharded input
    lo, hi = sharded.shard_bounds(n, world, rank)
    step = sharded.ShardedStep(3, 0.1, 6, ops=OracleOps)
    out_slice = step(G[:, lo:hi].contiguous())
    # (2) worker-resident input
    r0 = sum(counts[:rank])
    wr = sharded.WorkerResidentStep(n, counts, 3, 0.1, 6, ops=OracleOps)
    d_full = wr(G[r0:r0 + counts[rank]].contiguous())
    q.put((rank, lo, hi, out_slice.numpy(), d_full.numpy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,n,counts", [(2, 1003, [3, 4]), (3, 50, [1, 1, 1]), (3, 21, [2, 1, 3]), (4, 17, [1, 2, 1, 1])])
def test_sharded_and_worker_resident_steps_match_the_unsharded_oracle(world, n, counts):
    import torch.multiprocessing as mp
    from oracle import fa_oracle as fo
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() * 7 + n) % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q, n, counts)) for r in range(world)]
    for pr in procs:
        pr.start()
    got = [q.get(timeout=180) for _ in procs]
    for pr in procs:
        pr.join(60)
    ref = fo.fa_aggregate(_case(sum(counts), n, 5).astype(np.float64), 3, 0.1, 6)["d"]
    covered = np.zeros(n, dtype=int)
    for rank, lo, hi, out_slice, d_full in got:
        covered[lo:hi] += 1
        assert out_slice.shape == (hi - lo,)
        if hi > lo:
            assert fo.rel_l2(out_slice, ref[lo:hi]) < 1e-5
        assert d_full.shape == (n,) and fo.rel_l2(d_full, ref) < 1e-5
    assert (covered == 1).all()                      # the shards tile [0, n) exactly once


def test_shard_bounds_are_aligned_and_cover():
    sys.path.insert(0, ROOT)
    from paper_2302_05865_b200 import sharded
    for n in (1, 7, 8, 9, 1000, 11_173_962, 124_439_808):
        for world in (1, 2, 3, 4, 8):
            b = [sharded.shard_bounds(n, world, r) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == n
            assert all(b[r][1] == b[r + 1][0] for r in range(world - 1))
            assert all(lo % sharded.SHARD_ALIGN == 0 or lo == n for lo, _ in b)
            assert max(hi - lo for lo, hi in b) == min(n, sharded.shard_size(n, world))


def _rank_with_a_missing_peer(rank, world, port, q):
    """Rank 1 never joins the all-reduce of the partial inner products; rank 0 must get an error from the
    collective within its time limit instead of waiting for ever."""
    import datetime
    import time
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=datetime.timedelta(seconds=5))
    sys.path.insert(0, ROOT)
    from paper_2302_05865_b200 import sharded
    if rank == 1:
        time.sleep(12)                       # alive, but absent from the collective
        q.put((rank, "absent"))
        return
    G = torch.from_numpy(_case(6, 64, 9))
    lo, hi = sharded.shard_bounds(64, world, rank)
    step = sharded.ShardedStep(3, 0.1, 4, ops=OracleOps)
    t0 = time.time()
    try:
        step(G[:, lo:hi].contiguous())
        q.put((rank, "returned"))
    except Exception as e:                   # gloo reports the time-out as a RuntimeError
        q.put((rank, f"error after {time.time() - t0:.1f} s: {type(e).__name__}"))


def test_a_rank_missing_at_the_all_reduce_ends_the_collective_with_an_error():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() + 977) % 2000
    procs = [ctx.Process(target=_rank_with_a_missing_peer, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(30)
        if p.is_alive():
            p.kill()
    assert got[0].startswith("error after"), got
    assert float(got[0].split()[2]) < 11.0, got
