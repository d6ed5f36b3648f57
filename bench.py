#!/usr/bin/env python
"""Benchmark of the Flag Aggregator step (Gram pass -> IRLS -> output pass) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2]

One step = one whole aggregation of a seeded synthetic gradient set (default: the p=15,
n=11,173,962 fp32 workload the headline metric is quoted on).  Prints ONE JSON line.

Timing: batches of `--steps` aggregations, each batch bracketed by a barrier + synchronize and
timed with CUDA events (max over ranks); batches are repeated until the timed region is at least
`--min-time` seconds long, and the median batch is what is reported (with the spread).

With N > 1 (under torchrun) the ONE workload is sharded along n over the ranks: local Gram pass,
one all-reduce of p x p doubles, the same IRLS on every rank, local slice of the output (strong
scaling; the value is aggregations/s of that one job).  `--worker-resident` adds the all-to-all of
gradients that start on their workers and the all-gather of the result; `--replicas` runs N
independent copies of the single-GPU step instead (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synthetic_inputs as si  # noqa: E402

METRIC = "aggregations/sec at p=15, n=11.2M (whole Flag Aggregator step)"
UNIT = "aggregations/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (file absent)"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples (read-only queries), time-stamped so that only the
    samples taken while the timed region ran are used."""
    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and the set of active slow-down reasons over [t_begin, t_end] (time.time()
        values); falls back to the samples closest to the window when none fell inside it."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        rows = []
        for line in self.file.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[2]), float(parts[3]), parts[6:10]))
            except ValueError:
                continue
        self.file.close()
        os.unlink(self.file.name)
        if not rows:
            return out
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        if not inside and t_begin is not None:
            mid = 0.5 * (t_begin + t_end)
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:2]
            out["note"] = "no sample fell inside the timed region; nearest samples used"
        if not inside:
            inside = rows
        reasons = set()
        for r in inside:
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                   reasons=sorted(reasons), samples=len(inside))
        return out


def whole_job_rate(elapsed_ms_max_over_ranks: float, steps: int, world: int) -> float:
    """Aggregations per second of the whole job: every rank ran `steps` independent aggregations and the
    job is as slow as its slowest rank."""
    return world * steps / (elapsed_ms_max_over_ranks * 1e-3)


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        nums = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        if nums:
            return max(nums)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(w: si.Workload, n_sample: int, repeats: int = 1):
    """Oracle, as it stands, on the same recipe at n_sample columns; returns seconds per sample run."""
    from oracle import fa_oracle as fo
    ws = w.scaled(n_sample)
    G = si.to_float64(si.generate(ws))
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        fo.fa_aggregate(G, w.m, w.lam, w.iters)
        times.append(time.perf_counter() - t0)
    return min(times)


def workload_config(w, n_total, nbuf, parallelism):
    return {"workload": w.name, "p": w.p, "f": w.f, "n": n_total, "m": w.m, "lambda": w.lam, "iters": w.iters,
            "storage": w.dtype, "l2": f"inputs larger than L2; {nbuf} device copies of G rotated between steps",
            "parallelism": parallelism}


def run_reference(args, w):
    """The CPU oracle as the reference arm: each step is the oracle on a bounded sample of the workload
    (its cost is linear in n), and the line's figures are that time scaled to the full gradient length."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import fa_oracle as fo
    n_sample = max(4096, min(w.n // 64, int(10.0 / (2.7e-9 * w.p * w.p * w.iters))))   # about 10 s of oracle time per step
    ws = w.scaled(n_sample)
    G = si.to_float64(si.generate(ws))
    for _ in range(args.warmup):
        fo.fa_aggregate(G, w.m, w.lam, w.iters)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        fo.fa_aggregate(G, w.m, w.lam, w.iters)
    dt = (time.perf_counter() - t0) / args.steps
    scale = w.n / n_sample
    value = 1.0 / (dt * scale)
    sample = f"{w.name} recipe at n={n_sample} (1/{scale:.1f} of the columns), cost scaled linearly in n"
    cfg = workload_config(w, w.n, args.buffers, "single GPU")      # the keys of the GPU arm's config
    cfg["l2"] = "host memory (CPU run)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * scale * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
        "extrapolated_from_n": n_sample, "steps_run": args.steps, "measured_ms_per_sample_step": dt * 1e3,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def multi_gpu_mode(world, replicas, worker_resident):
    """Which step `--gpus N` times: 'single' on one GPU; with more, the n-sharded step unless asked otherwise."""
    if world <= 1:
        return "single"
    if replicas:
        return "replicas"
    return "worker-resident" if worker_resident else "sharded"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(si.WORKLOADS))
    ap.add_argument("--n", type=int, default=None, help="override the gradient length (profiling small cases)")
    ap.add_argument("--buffers", type=int, default=3, help="independent copies of G rotated between steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--min-time", type=float, default=1.0, help="length of the timed region in seconds, at least")
    ap.add_argument("--kernel-reps", type=int, default=100, help="launches per kernel for the per-kernel medians "
                    "(fewer under a profiler)")
    ap.add_argument("--replicas", action="store_true",
                    help="N > 1: N independent copies of the single-GPU step (weak scaling) instead of the n-sharded step")
    ap.add_argument("--worker-resident", action="store_true",
                    help="N > 1: gradients start on their workers (rank r holds whole rows): all-to-all, sharded step, "
                         "all-gather of the result")
    ap.add_argument("--sharded", action="store_true", help="accepted for compatibility: the default with N > 1")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    w = si.WORKLOADS[args.workload]
    if args.n:
        w = w.scaled(args.n)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    import paper_2302_05865_b200 as fa

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the aggregation has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: generated once on the host, R copies on the device (addresses differ, so a
    # step never finds its gradients in L2 from the previous step); every copy is > L2 at cfg2
    G_np = si.generate(w)
    host = torch.from_numpy(G_np.view(np.int16)).view(torch.bfloat16) if w.dtype == "bf16" else torch.from_numpy(G_np)
    mode = multi_gpu_mode(world, args.replicas, args.worker_resident)
    n_total, w_full = w.n, w
    nbuf = max(1, args.buffers)
    stream = torch.cuda.current_stream()
    if mode in ("sharded", "worker-resident"):
        from paper_2302_05865_b200 import sharded
    if mode == "sharded":                  # this rank keeps its columns only; everything below sees the shard
        lo, hi = sharded.shard_bounds(w.n, world, rank)
        host = host[:, lo:hi].contiguous()
        w = w.scaled(hi - lo)
    if mode == "worker-resident":          # this rank keeps whole rows: the gradients of its own workers
        counts = [w.p // world + (1 if r < w.p % world else 0) for r in range(world)]
        first = sum(counts[:rank])
        host = host[first:first + counts[rank]].contiguous()
    Gs = [host.cuda() for _ in range(nbuf)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    if mode == "sharded":
        out = torch.empty(w.n, dtype=torch.float32, device="cuda")
        sharded_step = sharded.ShardedStep(w.m, w.lam, w.iters)

        def step(i):
            sharded_step(Gs[i % nbuf], out=out)
    elif mode == "worker-resident":
        resident_step = sharded.WorkerResidentStep(w.n, counts, w.m, w.lam, w.iters)

        def step(i):
            resident_step(Gs[i % nbuf])
    else:
        out = torch.empty(w.n, dtype=torch.float32, device="cuda")
        wsb = fa.new_workspace(Gs[0], w.m)

        def step(i):
            fa.fa_aggregate(Gs[i % nbuf], w.m, w.lam, w.iters, out=out, ws=wsb, status=status, stream=stream)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for i in range(args.warmup):
        step(i)

    # ---- timed region: batches of `steps` aggregations, each between a barrier + synchronize and timed
    # with CUDA events; as many batches as it takes to fill --min-time (decided from the first batch,
    # on rank 0, so that every rank runs the same number)
    def timed_batch():
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for i in range(args.steps):
            step(i)
        ev1.record(stream)
        barrier()
        return ev0.elapsed_time(ev1)

    t_begin = time.time()
    batch_ms = [timed_batch()]
    n_batches = torch.tensor([max(1, int(np.ceil(args.min_time * 1e3 / max(batch_ms[0], 1e-3))))], device="cuda")
    if world > 1:
        dist.broadcast(n_batches, src=0)
    for _ in range(int(n_batches.item()) - 1):
        batch_ms.append(timed_batch())
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} after the timed region")
    times = torch.tensor(batch_ms, device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)          # a batch is as slow as its slowest rank
    batch_ms = sorted(float(x) for x in times.tolist())
    elapsed_ms = statistics.median(batch_ms)
    ms_per_step = elapsed_ms / args.steps
    value = whole_job_rate(elapsed_ms, args.steps, world if mode == "replicas" else 1)

    # ---- per-kernel times, same buffers and stream, CUDA events around single launches (median)
    def time_call(fn, reps):
        e0 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
        e1 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
        for i in range(reps):
            e0[i].record(stream)
            fn(i)
            e1[i].record(stream)
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in zip(e0, e1))

    kernels, roofline, step_hbm = None, None, None
    peak, peak_src = measured_peaks()

    if mode != "worker-resident":
        reps = max(3, args.kernel_reps if w.p * w.n * w.itemsize < 4e9 else min(args.kernel_reps, 30))
        K = torch.empty((w.p, w.p), dtype=torch.float64, device="cuda")
        cvec = torch.full((w.p,), 1.0 / w.p, dtype=torch.float32, device="cuda")
        wsk = fa.new_workspace(Gs[0], w.m)
        fa.fa_gram(Gs[0], K=K, ws=wsk); fa.fa_combine(Gs[0], cvec, out=out)
        if mode == "sharded":
            dist.all_reduce(K)
        fa.fa_irls(K, w.m, w.lam, w.iters, c_out=cvec)
        torch.cuda.synchronize()
        t_gram = time_call(lambda i: fa.fa_gram(Gs[i % nbuf], K=K, ws=wsk, stream=stream), reps)
        t_comb = time_call(lambda i: fa.fa_combine(Gs[i % nbuf], cvec, out=out, stream=stream), reps)
        t_irls = time_call(lambda i: fa.fa_irls(K, w.m, w.lam, w.iters, c_out=cvec, stream=stream), reps)
        gram_bytes = w.p * w.n * w.itemsize
        comb_bytes = w.p * w.n * w.itemsize + 4 * w.n
        gram_gbs = gram_bytes / (t_gram * 1e-3) / 1e9
        comb_gbs = comb_bytes / (t_comb * 1e-3) / 1e9
        step_gbs = w_full.algorithmic_bytes / (ms_per_step * 1e-3) / 1e9
        # DRAM bytes of one Gram launch, from ncu captures of the kernels as they stand, on cases small enough to
        # capture: fp32 p = 15 at n = 4,000,002 (rows in two alignment classes, as in the full workload): 240.11 MB
        # read for 240.00 MB of gradients, 8.8 MB written; fp32 p = 31 at n = 2,000,000: 248.10 MB read for
        # 248.00 MB, 4.0 MB written.  The reads grow with n; the writes are per block and do not.
        traffic, traffic_source = None, None
        if w.p == 15 and w.dtype == "f32" and w.n >= 4096:
            traffic = int(240.110e6 * (w.n / 4_000_002) + 8.8e6)
            traffic_source = ("ncu capture of gramtm::gram_tri_tm_kernel<float,2,15> at n = 4,000,002 "
                              "(dram__bytes_read 240.11 MB, dram__bytes_write 8.8 MB); reads scaled by n, writes not")
        elif w.p == 31 and w.dtype == "f32" and w.n >= 4096:
            traffic = int(248.10e6 * (w.n / 2_000_000) + 4.0e6)
            traffic_source = ("ncu capture of gram_quad_tm_kernel at n = 2,000,000 "
                              "(dram__bytes_read 248.10 MB, dram__bytes_write 4.0 MB); reads scaled by n, writes not")
        roofline = {"kernel": "gram pass (K = G G^T)", "bound": "hbm", "achieved": gram_gbs, "peak": peak,
                    "unit": "GB/s", "frac": gram_gbs / peak, "frac_of_nominal_8TBs": gram_gbs / 8000.0,
                    "traffic": traffic, "traffic_source": traffic_source, "peak_source": peak_src,
                    "bytes_per_launch": int(gram_bytes), "ms_per_launch": t_gram}
        kernels = {"gram_ms": t_gram, "irls_ms": t_irls, "combine_ms": t_comb, "launches_timed": reps,
                   "combine_gbs": comb_gbs, "combine_frac": comb_gbs / peak, "combine_frac_of_nominal_8TBs": comb_gbs / 8000.0,
                   "two_passes_gbs": (gram_bytes + comb_bytes) / ((t_gram + t_comb) * 1e-3) / 1e9,
                   "two_passes_frac": (gram_bytes + comb_bytes) / ((t_gram + t_comb) * 1e-3) / 1e9 / peak}
        step_hbm = {"algorithmic_bytes": int(w_full.algorithmic_bytes), "achieved_gbs": step_gbs,
                    "frac_of_measured": step_gbs / peak, "frac_of_nominal_8TBs": step_gbs / 8000.0}

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    e2e = None
    if not args.no_e2e and mode in ("single", "replicas"):
        Gh = host.pin_memory()
        outh = torch.empty(w.n, dtype=torch.float32).pin_memory()
        sth = torch.zeros(1, dtype=torch.int32).pin_memory()
        k_e2e = max(3, min(args.steps, 10))
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(2):
            fa.fa_aggregate_host(Gh, w.m, w.lam, w.iters, outh, Gs[0], out, wsb, sth, status, stream=stream)
        barrier()
        ev0.record(stream)
        for i in range(k_e2e):
            fa.fa_aggregate_host(Gh, w.m, w.lam, w.iters, outh, Gs[i % nbuf], out, wsb, sth, status, stream=stream)
        ev1.record(stream)
        barrier()
        ms = ev0.elapsed_time(ev1)
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        e2e = {"value": world * 1e3 / (ms / k_e2e), "unit": UNIT,
               "h2d_bytes_per_step": int(w.p * w.n * w.itemsize), "d2h_bytes_per_step": int(4 * w.n + 4),
               "steps": k_e2e, "ms_per_step": ms / k_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        # about 20 s of oracle time: its cost grows like n * p^2 * rounds (2.7e-9 s per unit on this class of host)
        n_sample = max(4096, min(w.n // 8, int(20.0 / (2.7e-9 * w.p * w.p * w.iters))))
        t_s = time_oracle(w, n_sample)
        scale = w.n / n_sample
        cpu = {"value": 1.0 / (t_s * scale), "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": f"{w.name} recipe at n={n_sample} (1/{scale:.1f} of the columns), {t_s:.1f} s measured, "
                         f"cost scaled linearly in n"}

    parallelism = {"single": "single GPU", "replicas": f"replicas x{world}",
                   "sharded": f"n-sharded x{world}, one all-reduce of p*p fp64 per step; roofline and kernel times "
                              f"are rank 0's shard of {w.n} columns",
                   "worker-resident": f"worker-resident x{world}: all-to-all of the gradients, n-sharded step, "
                                      f"all-gather of the aggregate"}[mode]
    if clocks and clocks.get("sm_mhz"):
        clocks["ms_per_step_x_sm_mhz"] = ms_per_step * clocks["sm_mhz"]
    launches_per_step = 3 if mode != "worker-resident" else 3
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak" if mode in ("single", "replicas") else "strong",
        "vs_baseline": None, "dtype": "f32" if w.dtype == "f32" else "bf16", "data": "synthetic",
        "config": workload_config(w_full, n_total, nbuf, parallelism),
        "timing": {"batches": len(batch_ms), "steps_per_batch": args.steps, "timed_region_s": sum(batch_ms) * 1e-3,
                   "ms_per_step_min": batch_ms[0] / args.steps, "ms_per_step_median": ms_per_step,
                   "ms_per_step_max": batch_ms[-1] / args.steps},
        "roofline": roofline, "kernels": kernels, "step_hbm": step_hbm,
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps * len(batch_ms), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
