"""B200 Flag Aggregator step: thin Python binding over the C ABI in include/fa.h.

Every function here only marshals arguments (torch tensors -> device pointers,
the current CUDA stream) and calls the entry point of the same name in
libfa_b200.so; all arithmetic runs in the CUDA kernels.  There is no CPU
fallback: importing the package without the built library raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfa_b200.so")

FA_F32, FA_BF16 = 0, 1
FA_MAX_P = 64
ST_NONFINITE, ST_RANK0, ST_RANK_LT_M, ST_EIG_SWEEPS, ST_TIMEOUT = 1, 2, 4, 8, 16

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2302_05865_b200/build.py` "
        "(needs nvcc; there is no non-CUDA path)")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i, _ll, _d, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_double, ctypes.c_size_t
_lib.fa_error_string.restype = ctypes.c_char_p
_lib.fa_error_string.argtypes = [_i]
_lib.fa_workspace_bytes.argtypes = [_i, _ll, _i, _i, ctypes.POINTER(_sz)]
_lib.fa_gram.argtypes = [_vp, _i, _i, _ll, _vp, _vp, _sz, _vp]
_lib.fa_irls_step.argtypes = [_vp, _i, _i, _d, _i, _vp, _vp, _vp, _vp, _vp]
_lib.fa_irls.argtypes = [_vp, _i, _i, _d, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fa_irls_ex.argtypes = [_vp, _i, _i, _d, _d, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fa_aggregate_ex.argtypes = [_vp, _i, _i, _ll, _i, _d, _d, _i, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_irls_multi.argtypes = [_vp, _i, _vp, _i, _i, _d, _d, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fa_aggregate_multi.argtypes = [_vp, _i, _i, _ll, _vp, _i, _i, _d, _d, _i, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_irls_warm.argtypes = [_vp, _i, _i, _d, _d, _i, _d, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fa_aggregate_warm.argtypes = [_vp, _i, _i, _ll, _i, _d, _d, _i, _d, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_irls_beta.argtypes = [_vp, _i, _i, _d, _d, _d, _d, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fa_aggregate_beta.argtypes = [_vp, _i, _i, _ll, _i, _d, _d, _d, _d, _i, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_combine.argtypes = [_vp, _i, _i, _ll, _vp, _vp, _vp]
_lib.fa_aggregate.argtypes = [_vp, _i, _i, _ll, _i, _d, _i, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_aggregate_host.argtypes = [_vp, _i, _i, _ll, _i, _d, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.fa_gram_static.argtypes = [_vp, _i, _i, _ll, _vp, _vp]
_lib.fa_gram_static.restype = _i
for _name in ("fa_workspace_bytes", "fa_gram", "fa_irls_step", "fa_irls", "fa_irls_ex", "fa_aggregate_ex",
              "fa_irls_multi", "fa_aggregate_multi", "fa_irls_warm", "fa_aggregate_warm", "fa_irls_beta", "fa_aggregate_beta", "fa_combine", "fa_aggregate", "fa_aggregate_host"):
    getattr(_lib, _name).restype = _i


class FaError(RuntimeError):
    pass


def _check(code: int, what: str) -> None:
    if code != 0:
        raise FaError(f"{what}: {_lib.fa_error_string(code).decode()} ({code})")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return FA_F32
    if t.dtype == torch.bfloat16:
        return FA_BF16
    raise TypeError(f"G must be float32 or bfloat16, got {t.dtype}")


def _gradients(G: torch.Tensor):
    if not (G.is_cuda and G.dim() == 2 and G.is_contiguous()):
        raise ValueError("G must be a contiguous 2-D CUDA tensor of shape (p, n), one row per worker")
    return _dtype_code(G), int(G.shape[0]), int(G.shape[1])


def _dev(t, dtype, numel, name, device=None):
    """Pointer of a tensor the kernels will read or write `numel` elements of `dtype` through.

    Checked here, before anything is enqueued, because a buffer of the wrong type or size would
    otherwise become an out-of-bounds access on the device: element type, contiguity, size, then
    that it lives on the GPU the call runs on.
    """
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name} must be a torch tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if t.numel() < numel:
        raise ValueError(f"{name} must have at least {numel} elements, got {t.numel()}")
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if device is not None and t.device != device:
        raise ValueError(f"{name} is on {t.device}, the call runs on {device}")
    return t.data_ptr()


def _opt(t, dtype, numel, name, device=None):
    return None if t is None else _dev(t, dtype, numel, name, device)


def _ws(ws, device):
    if not (isinstance(ws, torch.Tensor) and ws.is_cuda and ws.is_contiguous() and ws.device == device):
        raise ValueError(f"ws must be a contiguous CUDA tensor on {device}")
    return ws.data_ptr(), ws.numel() * ws.element_size()


class _on:
    """Make `device` current for the duration of a call and hand out the stream to enqueue on.

    The library launches on the current device (its tensor maps, its SM count, the built-in scratch
    array of fa_gram_static all belong to it), so the call must run with the tensors' device current
    and on one of that device's streams.
    """

    def __init__(self, device, stream):
        self.guard = torch.cuda.device(device)
        self.device = device
        self.stream = stream

    def __enter__(self):
        self.guard.__enter__()
        s = torch.cuda.current_stream(self.device) if self.stream is None else self.stream
        if s.device != self.device:
            self.guard.__exit__(None, None, None)
            raise ValueError(f"stream belongs to {s.device}, the tensors are on {self.device}")
        return ctypes.c_void_p(s.cuda_stream)

    def __exit__(self, *exc):
        return self.guard.__exit__(*exc)


def _square(K, name="K"):
    if not (isinstance(K, torch.Tensor) and K.dim() == 2 and K.shape[0] == K.shape[1]):
        raise ValueError(f"{name} must be a square 2-D tensor")
    p = int(K.shape[0])
    return p, _dev(K, torch.float64, p * p, name)


def fa_workspace_bytes(p: int, n: int, m: int, dtype) -> int:
    code = dtype if isinstance(dtype, int) else (FA_F32 if dtype == torch.float32 else FA_BF16)
    out = _sz(0)
    _check(_lib.fa_workspace_bytes(p, n, m, code, ctypes.byref(out)), "fa_workspace_bytes")
    return int(out.value)


def new_workspace(G: torch.Tensor, m: int = 1) -> torch.Tensor:
    code, p, n = _gradients(G)
    return torch.empty(fa_workspace_bytes(p, n, m, code), dtype=torch.uint8, device=G.device)


def fa_gram(G, K=None, ws=None, stream=None):
    code, p, n = _gradients(G)
    dev = G.device
    K = torch.empty((p, p), dtype=torch.float64, device=dev) if K is None else K
    ws = new_workspace(G) if ws is None else ws
    Kp, (wp, wb) = _dev(K, torch.float64, p * p, "K", dev), _ws(ws, dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_gram(G.data_ptr(), code, p, n, Kp, wp, wb, st), "fa_gram")
    return K


def fa_gram_static(G, K=None, stream=None):
    """fa_gram for callers that cannot allocate: no workspace argument, the partial sums use an array
    built into the library (p <= 32).  Pass K to keep this wrapper from allocating the result too.
    Calls that may overlap on the GPU must not share a device: they race on that array."""
    code, p, n = _gradients(G)
    dev = G.device
    K = torch.empty((p, p), dtype=torch.float64, device=dev) if K is None else K
    Kp = _dev(K, torch.float64, p * p, "K", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_gram_static(G.data_ptr(), code, p, n, Kp, st), "fa_gram_static")
    return K


def fa_irls_step(K, m, lam, first, A, w=None, objective=None, status=None, stream=None):
    p, Kp = _square(K)
    dev = K.device
    w = torch.empty(p, dtype=torch.float64, device=dev) if w is None else w
    args = (Kp, p, m, float(lam), 1 if first else 0, _dev(A, torch.float64, p * max(m, 0), "A", dev),
            _dev(w, torch.float64, p, "w", dev), _opt(objective, torch.float64, 1, "objective", dev),
            _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_irls_step(*args, st), "fa_irls_step")
    return A, w


def _irls_outputs(dev, p, m, iters, nweights, A_out, c_out, w_out, obj_out, status):
    """Pointers of the outputs every IRLS entry point shares, sized as include/fa.h states."""
    Ap = _opt(A_out, torch.float64, p * max(m, 0), "A_out", dev)
    wp = _opt(w_out, torch.float64, nweights, "w_out", dev)
    op = _opt(obj_out, torch.float64, max(iters, 0), "obj_out", dev)
    sp = _opt(status, torch.int32, 1, "status", dev)
    return Ap, _dev(c_out, torch.float32, p, "c_out", dev), wp, op, sp


def fa_irls(K, m, lam, iters, A_out=None, c_out=None, w_out=None, obj_out=None, status=None, stream=None):
    p, Kp = _square(K)
    dev = K.device
    c_out = torch.empty(p, dtype=torch.float32, device=dev) if c_out is None else c_out
    Ap, cp, wp, op, sp = _irls_outputs(dev, p, m, iters, p, A_out, c_out, w_out, obj_out, status)
    with _on(dev, stream) as st:
        _check(_lib.fa_irls(Kp, p, m, float(lam), iters, Ap, cp, wp, op, sp, st), "fa_irls")
    return c_out


def fa_irls_ex(K, m, lam, a, iters, A_out=None, c_out=None, S_out=None, w_out=None, obj_out=None, status=None,
               stream=None):
    """fa_irls with the surrogate constant a (a = 2: the paper's) and the p x p selection matrix S_out."""
    p, Kp = _square(K)
    dev = K.device
    c_out = torch.empty(p, dtype=torch.float32, device=dev) if c_out is None else c_out
    Ap, cp, wp, op, sp = _irls_outputs(dev, p, m, iters, p, A_out, c_out, w_out, obj_out, status)
    Sp = _opt(S_out, torch.float64, p * p, "S_out", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_irls_ex(Kp, p, m, float(lam), float(a), iters, Ap, cp, Sp, wp, op, sp, st), "fa_irls_ex")
    return c_out


def fa_aggregate_ex(G, m, lam, a, iters, out=None, A_out=None, S_out=None, ws=None, status=None, stream=None):
    """fa_aggregate with the surrogate constant a and the selection matrix S_out."""
    code, p, n = _gradients(G)
    dev = G.device
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    args = (_dev(out, torch.float32, n, "out", dev), _opt(A_out, torch.float64, p * max(m, 0), "A_out", dev),
            _opt(S_out, torch.float64, p * p, "S_out", dev), *_ws(ws, dev), _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate_ex(G.data_ptr(), code, p, n, m, float(lam), float(a), iters, *args, st),
               "fa_aggregate_ex")
    return out


def fa_irls_warm(K, m, lam, iters, a=2.0, tol=-1.0, A0=None, A_out=None, c_out=None, w_out=None, obj_out=None,
                 rounds_out=None, status=None, stream=None):
    """IRLS from the subspace spanned by A0 (None: uniform first round), stopping once the objective moved by
    <= tol (tol < 0: all rounds)."""
    p, Kp = _square(K)
    dev = K.device
    c_out = torch.empty(p, dtype=torch.float32, device=dev) if c_out is None else c_out
    Ap, cp, wp, op, sp = _irls_outputs(dev, p, m, iters, p, A_out, c_out, w_out, obj_out, status)
    A0p = _opt(A0, torch.float64, p * max(m, 0), "A0", dev)
    rp = _opt(rounds_out, torch.int32, 1, "rounds_out", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_irls_warm(Kp, p, m, float(lam), float(a), iters, float(tol), A0p, Ap, cp, wp, op, rp, sp, st),
               "fa_irls_warm")
    return c_out


def fa_aggregate_warm(G, m, lam, iters, a=2.0, tol=-1.0, A0=None, out=None, A_out=None, rounds_out=None, ws=None,
                      status=None, stream=None):
    """The whole step, started from the subspace of A0 (e.g. the previous step's A_out) and/or stopped on tol."""
    code, p, n = _gradients(G)
    dev = G.device
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    args = (_opt(A0, torch.float64, p * max(m, 0), "A0", dev), _dev(out, torch.float32, n, "out", dev),
            _opt(A_out, torch.float64, p * max(m, 0), "A_out", dev), _opt(rounds_out, torch.int32, 1, "rounds_out", dev),
            *_ws(ws, dev), _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate_warm(G.data_ptr(), code, p, n, m, float(lam), float(a), iters, float(tol), *args, st),
               "fa_aggregate_warm")
    return out


def fa_irls_beta(K, m, lam, iters, alpha, beta, a=2.0, A_out=None, c_out=None, w_out=None, obj_out=None, status=None,
                 stream=None):
    """IRLS with a Beta(alpha, beta) likelihood of the workers' values (alpha = 1, beta = 1/2: fa_irls)."""
    p, Kp = _square(K)
    dev = K.device
    c_out = torch.empty(p, dtype=torch.float32, device=dev) if c_out is None else c_out
    Ap, cp, wp, op, sp = _irls_outputs(dev, p, m, iters, p, A_out, c_out, w_out, obj_out, status)
    with _on(dev, stream) as st:
        _check(_lib.fa_irls_beta(Kp, p, m, float(lam), float(a), float(alpha), float(beta), iters, Ap, cp, wp, op, sp,
                                 st), "fa_irls_beta")
    return c_out


def fa_aggregate_beta(G, m, lam, iters, alpha, beta, a=2.0, out=None, A_out=None, ws=None, status=None, stream=None):
    code, p, n = _gradients(G)
    dev = G.device
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    args = (_dev(out, torch.float32, n, "out", dev), _opt(A_out, torch.float64, p * max(m, 0), "A_out", dev),
            *_ws(ws, dev), _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate_beta(G.data_ptr(), code, p, n, m, float(lam), float(a), float(alpha), float(beta),
                                      iters, *args, st), "fa_aggregate_beta")
    return out


def _counts(counts):
    return (ctypes.c_int * len(counts))(*[int(k) for k in counts])


def fa_irls_multi(K, counts, m, lam, iters, a=2.0, A_out=None, c_out=None, S_out=None, w_out=None, obj_out=None,
                  status=None, stream=None):
    """IRLS rounds for workers that hold counts[i] consecutive rows of K each; returns c (one entry per row)."""
    rows, Kp = _square(K)
    dev = K.device
    arr = _counts(counts)
    c_out = torch.empty(rows, dtype=torch.float32, device=dev) if c_out is None else c_out
    Ap, cp, wp, op, sp = _irls_outputs(dev, rows, m, iters, len(counts), A_out, c_out, w_out, obj_out, status)
    Sp = _opt(S_out, torch.float64, rows * rows, "S_out", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_irls_multi(Kp, rows, arr, len(counts), m, float(lam), float(a), iters, Ap, cp, Sp, wp, op, sp,
                                  st), "fa_irls_multi")
    return c_out


def fa_aggregate_multi(G, counts, m, lam, iters, a=2.0, out=None, A_out=None, w_out=None, ws=None, status=None,
                       stream=None):
    """The whole step for workers with several gradients each (rows of one worker consecutive in G)."""
    code, rows, n = _gradients(G)
    dev = G.device
    arr = _counts(counts)
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    args = (_dev(out, torch.float32, n, "out", dev), _opt(A_out, torch.float64, rows * max(m, 0), "A_out", dev),
            _opt(w_out, torch.float64, len(counts), "w_out", dev), *_ws(ws, dev),
            _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate_multi(G.data_ptr(), code, rows, n, arr, len(counts), m, float(lam), float(a), iters,
                                       *args, st), "fa_aggregate_multi")
    return out


def fa_combine(G, c, out=None, stream=None):
    code, p, n = _gradients(G)
    dev = G.device
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    cp, op = _dev(c, torch.float32, p, "c", dev), _dev(out, torch.float32, n, "out", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_combine(G.data_ptr(), code, p, n, cp, op, st), "fa_combine")
    return out


def fa_aggregate(G, m, lam, iters, out=None, A_out=None, ws=None, status=None, stream=None):
    code, p, n = _gradients(G)
    dev = G.device
    out = torch.empty(n, dtype=torch.float32, device=dev) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    args = (_dev(out, torch.float32, n, "out", dev), _opt(A_out, torch.float64, p * max(m, 0), "A_out", dev),
            *_ws(ws, dev), _opt(status, torch.int32, 1, "status", dev))
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate(G.data_ptr(), code, p, n, m, float(lam), iters, *args, st), "fa_aggregate")
    return out


def _host(t, dtype, numel, name):
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise ValueError(f"{name} must be a CPU tensor (pinned for the copies to be asynchronous)")
    if (dtype is not None and t.dtype != dtype) or not t.is_contiguous() or t.numel() < numel:
        raise ValueError(f"{name} must be contiguous, of dtype {dtype or 'float32/bfloat16'}, with at least {numel} elements")
    return t.data_ptr()


def fa_aggregate_host(G_host, m, lam, iters, out_host, G_dev, out_dev, ws, status_host=None, status_dev=None,
                      stream=None):
    """Host-buffer variant: G_host (pinned CPU tensor, p x n) -> out_host (pinned CPU, n floats).

    G_dev / out_dev / ws / status_dev are caller-owned device staging buffers.  The copies and the
    three kernels are enqueued on the stream; the caller synchronises before reading out_host.
    """
    if not (isinstance(G_host, torch.Tensor) and G_host.dim() == 2):
        raise ValueError("G_host must be a 2-D CPU tensor of shape (p, n)")
    code, p, n = _dtype_code(G_host), int(G_host.shape[0]), int(G_host.shape[1])
    dev = G_dev.device if isinstance(G_dev, torch.Tensor) else None
    args_host = (_host(G_host, None, p * n, "G_host"), _host(out_host, torch.float32, n, "out_host"),
                 None if status_host is None else _host(status_host, torch.int32, 1, "status_host"))
    Gd = _dev(G_dev, G_host.dtype, p * n, "G_dev", dev)
    od = _dev(out_dev, torch.float32, n, "out_dev", dev)
    wp, wb = _ws(ws, dev)
    sd = _opt(status_dev, torch.int32, 1, "status_dev", dev)
    with _on(dev, stream) as st:
        _check(_lib.fa_aggregate_host(args_host[0], code, p, n, m, float(lam), iters, args_host[1], args_host[2],
                                      Gd, od, wp, wb, sd, st), "fa_aggregate_host")
    return out_host
