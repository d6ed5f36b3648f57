"""CPU-side checks: the shared library builds, loads and exports what include/fa.h declares;
host-side argument validation answers before anything is enqueued; bench.py's reference arm
and multi-rank timing reduction work without a GPU."""
import ctypes
import json
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as entry
    entry.build()
    import paper_2302_05865_b200 as fa
    return ctypes.CDLL(fa.LIB_PATH)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported(lib):
    names = declared_functions()
    assert {"fa_workspace_bytes", "fa_gram", "fa_irls_step", "fa_irls", "fa_combine", "fa_aggregate",
            "fa_aggregate_host", "fa_error_string"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/fa.h but not exported"


def test_workspace_query_and_error_codes_without_a_device(lib):
    size = ctypes.c_size_t(0)
    assert lib.fa_workspace_bytes(15, ctypes.c_longlong(11_173_962), 8, 0, ctypes.byref(size)) == 0
    assert 0 < size.value < 64 << 20
    assert lib.fa_workspace_bytes(65, ctypes.c_longlong(10), 1, 0, ctypes.byref(size)) == -1     # p > FA_MAX_P
    assert lib.fa_workspace_bytes(4, ctypes.c_longlong(0), 1, 0, ctypes.byref(size)) == -1      # n < 1
    assert lib.fa_workspace_bytes(4, ctypes.c_longlong(10), 1, 7, ctypes.byref(size)) == -1     # dtype
    lib.fa_error_string.restype = ctypes.c_char_p
    assert lib.fa_error_string(-3) == b"workspace too small"
    # null pointers are rejected on the host; nothing reaches a device
    lib.fa_aggregate.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong, ctypes.c_int,
                                 ctypes.c_double, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                 ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    assert lib.fa_aggregate(None, 0, 4, 10, 2, 0.0, 3, None, None, None, 0, None, None) == -1


def test_binding_rejects_wrong_buffers_before_any_launch(lib):
    """Every tensor handed to the binding is checked for element type and size on the host: a float32
    A_out or an obj_out shorter than `iters` would otherwise be an out-of-bounds write on the device.
    (Checked in this order: type, contiguity, size, device -- so CPU tensors reach the first three.)"""
    import torch
    import paper_2302_05865_b200 as fa
    ok = torch.zeros(15 * 8, dtype=torch.float64)
    for bad, what in ((torch.zeros(15 * 8, dtype=torch.float32), "dtype"), (torch.zeros(15 * 8 - 1, dtype=torch.float64), "at least"),
                      (torch.zeros((15, 16), dtype=torch.float64)[:, :8], "contiguous")):
        with pytest.raises(ValueError, match=what):
            fa._dev(bad, torch.float64, 15 * 8, "A_out")
    with pytest.raises(ValueError, match="CUDA"):
        fa._dev(ok, torch.float64, 15 * 8, "A_out")
    with pytest.raises(TypeError):
        fa._dev([0.0] * 120, torch.float64, 120, "A_out")
    # the sizes the IRLS entry points ask of their optional outputs: p*m, p, workers, iters, 1
    c = torch.zeros(15, dtype=torch.float32)
    cases = dict(A_out=torch.zeros(15 * 8 - 1, dtype=torch.float64), w_out=torch.zeros(14, dtype=torch.float64),
                 obj_out=torch.zeros(9, dtype=torch.float64), status=torch.zeros(1, dtype=torch.int64))
    for name, bad in cases.items():
        kw = dict(A_out=None, c_out=c, w_out=None, obj_out=None, status=None)
        kw[name] = bad
        with pytest.raises(ValueError, match=name):
            fa._irls_outputs(None, 15, 8, 10, 15, **kw)
    K = torch.zeros((15, 15), dtype=torch.float64)
    for call in (lambda: fa.fa_irls(K, 8, 0.0, 10), lambda: fa.fa_irls(K[:, :14], 8, 0.0, 10),
                 lambda: fa.fa_gram(torch.zeros((4, 10))), lambda: fa.fa_combine(torch.zeros((4, 10)), c)):
        with pytest.raises(ValueError):
            call()


def test_package_refuses_to_import_without_its_library(tmp_path):
    """There is no CPU fallback: without libfa_b200.so the import itself fails."""
    pkg = tmp_path / "paper_2302_05865_b200"
    pkg.mkdir()
    src = os.path.join(ROOT, "paper_2302_05865_b200", "__init__.py")
    (pkg / "__init__.py").write_text(open(src).read())
    r = subprocess.run([sys.executable, "-c", "import paper_2302_05865_b200"], cwd=tmp_path,
                       capture_output=True, text=True, env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert r.returncode != 0 and "libfa_b200.so is missing" in r.stderr


def test_product_sources_do_not_touch_the_oracle():
    for base, _, files in os.walk(os.path.join(ROOT, "paper_2302_05865_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(base, f)).read().lower(), f


def test_reference_arm_prints_one_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "cfg1"], capture_output=True, text=True, cwd=ROOT)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    # same config keys as the GPU arm's line, and the extrapolation is declared
    sys.path.insert(0, ROOT)
    import bench
    import synthetic_inputs as si
    assert set(line["config"]) == set(bench.workload_config(si.WORKLOADS["cfg1"], 65_536, 3, "single GPU"))
    assert line["steps_run"] == 1 and 0 < line["extrapolated_from_n"] <= 65_536


def test_which_step_the_gpu_count_selects():
    """`--gpus N` alone must time the n-sharded step (one job over N GPUs); replicas and the
    worker-resident variant are opt-in; one GPU has a single mode whatever the flags."""
    sys.path.insert(0, ROOT)
    import bench
    assert bench.multi_gpu_mode(1, False, False) == "single"
    assert bench.multi_gpu_mode(1, True, True) == "single"
    assert bench.multi_gpu_mode(2, False, False) == "sharded"
    assert bench.multi_gpu_mode(8, False, True) == "worker-resident"
    assert bench.multi_gpu_mode(8, True, False) == "replicas"


def _rank_main(rank, world, port, q):
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    # each rank measured a different time; the job's rate uses the slowest rank
    t = torch.tensor([10.0 + 5.0 * rank])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    q.put((rank, bench.whole_job_rate(float(t.item()), steps=5, world=world)))
    dist.destroy_process_group()


def test_two_rank_timing_reduction_over_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
    # 2 replicas, slowest rank took 15 ms for 5 steps -> 2 * 5 / 0.015 s
    assert got[0] == got[1] == pytest.approx(2 * 5 / 0.015)
