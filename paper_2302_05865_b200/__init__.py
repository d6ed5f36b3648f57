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


def _dev(t, dtype, numel, name):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous() and t.numel() >= numel):
        raise ValueError(f"{name} must be a contiguous CUDA tensor of {dtype} with at least {numel} elements")
    return t.data_ptr()


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


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
    K = torch.empty((p, p), dtype=torch.float64, device=G.device) if K is None else K
    ws = new_workspace(G) if ws is None else ws
    _check(_lib.fa_gram(G.data_ptr(), code, p, n, _dev(K, torch.float64, p * p, "K"), ws.data_ptr(),
                        ws.numel() * ws.element_size(), _stream(stream)), "fa_gram")
    return K


def fa_gram_static(G, K=None, stream=None):
    """fa_gram for callers that cannot allocate: no workspace argument, the partial sums use an array
    built into the library (p <= 32).  Pass K to keep this wrapper from allocating the result too.
    Calls that may overlap on the GPU must not share a device: they race on that array."""
    code, p, n = _gradients(G)
    K = torch.empty((p, p), dtype=torch.float64, device=G.device) if K is None else K
    _check(_lib.fa_gram_static(G.data_ptr(), code, p, n, _dev(K, torch.float64, p * p, "K"), _stream(stream)),
           "fa_gram_static")
    return K


def fa_irls_step(K, m, lam, first, A, w=None, objective=None, status=None, stream=None):
    p = int(K.shape[0])
    w = torch.empty(p, dtype=torch.float64, device=K.device) if w is None else w
    _check(_lib.fa_irls_step(_dev(K, torch.float64, p * p, "K"), p, m, float(lam), 1 if first else 0,
                             _dev(A, torch.float64, p * m, "A"), _dev(w, torch.float64, p, "w"),
                             _ptr(objective), _ptr(status), _stream(stream)), "fa_irls_step")
    return A, w


def fa_irls(K, m, lam, iters, A_out=None, c_out=None, w_out=None, obj_out=None, status=None, stream=None):
    p = int(K.shape[0])
    c_out = torch.empty(p, dtype=torch.float32, device=K.device) if c_out is None else c_out
    _check(_lib.fa_irls(_dev(K, torch.float64, p * p, "K"), p, m, float(lam), iters, _ptr(A_out),
                        _dev(c_out, torch.float32, p, "c_out"), _ptr(w_out), _ptr(obj_out), _ptr(status),
                        _stream(stream)), "fa_irls")
    return c_out


def fa_irls_ex(K, m, lam, a, iters, A_out=None, c_out=None, S_out=None, w_out=None, obj_out=None, status=None,
               stream=None):
    """fa_irls with the surrogate constant a (a = 2: the paper's) and the p x p selection matrix S_out."""
    p = int(K.shape[0])
    c_out = torch.empty(p, dtype=torch.float32, device=K.device) if c_out is None else c_out
    if S_out is not None:
        _dev(S_out, torch.float64, p * p, "S_out")
    _check(_lib.fa_irls_ex(_dev(K, torch.float64, p * p, "K"), p, m, float(lam), float(a), iters, _ptr(A_out),
                           _dev(c_out, torch.float32, p, "c_out"), _ptr(S_out), _ptr(w_out), _ptr(obj_out),
                           _ptr(status), _stream(stream)), "fa_irls_ex")
    return c_out


def fa_aggregate_ex(G, m, lam, a, iters, out=None, A_out=None, S_out=None, ws=None, status=None, stream=None):
    """fa_aggregate with the surrogate constant a and the selection matrix S_out."""
    code, p, n = _gradients(G)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    if A_out is not None:
        _dev(A_out, torch.float64, p * m, "A_out")
    if S_out is not None:
        _dev(S_out, torch.float64, p * p, "S_out")
    _check(_lib.fa_aggregate_ex(G.data_ptr(), code, p, n, m, float(lam), float(a), iters,
                                _dev(out, torch.float32, n, "out"), _ptr(A_out), _ptr(S_out), ws.data_ptr(),
                                ws.numel() * ws.element_size(), _ptr(status), _stream(stream)), "fa_aggregate_ex")
    return out


def fa_irls_warm(K, m, lam, iters, a=2.0, tol=-1.0, A0=None, A_out=None, c_out=None, w_out=None, obj_out=None,
                 rounds_out=None, status=None, stream=None):
    """IRLS from the subspace spanned by A0 (None: uniform first round), stopping once the objective moved by
    <= tol (tol < 0: all rounds)."""
    p = int(K.shape[0])
    c_out = torch.empty(p, dtype=torch.float32, device=K.device) if c_out is None else c_out
    if A0 is not None:
        _dev(A0, torch.float64, p * m, "A0")
    _check(_lib.fa_irls_warm(_dev(K, torch.float64, p * p, "K"), p, m, float(lam), float(a), iters, float(tol),
                             _ptr(A0), _ptr(A_out), _dev(c_out, torch.float32, p, "c_out"), _ptr(w_out),
                             _ptr(obj_out), _ptr(rounds_out), _ptr(status), _stream(stream)), "fa_irls_warm")
    return c_out


def fa_aggregate_warm(G, m, lam, iters, a=2.0, tol=-1.0, A0=None, out=None, A_out=None, rounds_out=None, ws=None,
                      status=None, stream=None):
    """The whole step, started from the subspace of A0 (e.g. the previous step's A_out) and/or stopped on tol."""
    code, p, n = _gradients(G)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    for t, name in ((A0, "A0"), (A_out, "A_out")):
        if t is not None:
            _dev(t, torch.float64, p * m, name)
    _check(_lib.fa_aggregate_warm(G.data_ptr(), code, p, n, m, float(lam), float(a), iters, float(tol), _ptr(A0),
                                  _dev(out, torch.float32, n, "out"), _ptr(A_out), _ptr(rounds_out), ws.data_ptr(),
                                  ws.numel() * ws.element_size(), _ptr(status), _stream(stream)),
           "fa_aggregate_warm")
    return out


def fa_irls_beta(K, m, lam, iters, alpha, beta, a=2.0, A_out=None, c_out=None, w_out=None, obj_out=None, status=None,
                 stream=None):
    """IRLS with a Beta(alpha, beta) likelihood of the workers' values (alpha = 1, beta = 1/2: fa_irls)."""
    p = int(K.shape[0])
    c_out = torch.empty(p, dtype=torch.float32, device=K.device) if c_out is None else c_out
    _check(_lib.fa_irls_beta(_dev(K, torch.float64, p * p, "K"), p, m, float(lam), float(a), float(alpha), float(beta),
                             iters, _ptr(A_out), _dev(c_out, torch.float32, p, "c_out"), _ptr(w_out), _ptr(obj_out),
                             _ptr(status), _stream(stream)), "fa_irls_beta")
    return c_out


def fa_aggregate_beta(G, m, lam, iters, alpha, beta, a=2.0, out=None, A_out=None, ws=None, status=None, stream=None):
    code, p, n = _gradients(G)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    _check(_lib.fa_aggregate_beta(G.data_ptr(), code, p, n, m, float(lam), float(a), float(alpha), float(beta), iters,
                                  _dev(out, torch.float32, n, "out"), _ptr(A_out), ws.data_ptr(),
                                  ws.numel() * ws.element_size(), _ptr(status), _stream(stream)),
           "fa_aggregate_beta")
    return out


def _counts(counts):
    return (ctypes.c_int * len(counts))(*[int(k) for k in counts])


def fa_irls_multi(K, counts, m, lam, iters, a=2.0, A_out=None, c_out=None, S_out=None, w_out=None, obj_out=None,
                  status=None, stream=None):
    """IRLS rounds for workers that hold counts[i] consecutive rows of K each; returns c (one entry per row)."""
    rows = int(K.shape[0])
    arr = _counts(counts)
    c_out = torch.empty(rows, dtype=torch.float32, device=K.device) if c_out is None else c_out
    if w_out is not None:
        _dev(w_out, torch.float64, len(counts), "w_out")
    _check(_lib.fa_irls_multi(_dev(K, torch.float64, rows * rows, "K"), rows, arr, len(counts), m, float(lam), float(a),
                              iters, _ptr(A_out), _dev(c_out, torch.float32, rows, "c_out"), _ptr(S_out), _ptr(w_out),
                              _ptr(obj_out), _ptr(status), _stream(stream)), "fa_irls_multi")
    return c_out


def fa_aggregate_multi(G, counts, m, lam, iters, a=2.0, out=None, A_out=None, w_out=None, ws=None, status=None,
                       stream=None):
    """The whole step for workers with several gradients each (rows of one worker consecutive in G)."""
    code, rows, n = _gradients(G)
    arr = _counts(counts)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    if A_out is not None:
        _dev(A_out, torch.float64, rows * m, "A_out")
    if w_out is not None:
        _dev(w_out, torch.float64, len(counts), "w_out")
    _check(_lib.fa_aggregate_multi(G.data_ptr(), code, rows, n, arr, len(counts), m, float(lam), float(a), iters,
                                   _dev(out, torch.float32, n, "out"), _ptr(A_out), _ptr(w_out), ws.data_ptr(),
                                   ws.numel() * ws.element_size(), _ptr(status), _stream(stream)),
           "fa_aggregate_multi")
    return out


def fa_combine(G, c, out=None, stream=None):
    code, p, n = _gradients(G)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    _check(_lib.fa_combine(G.data_ptr(), code, p, n, _dev(c, torch.float32, p, "c"),
                           _dev(out, torch.float32, n, "out"), _stream(stream)), "fa_combine")
    return out


def fa_aggregate(G, m, lam, iters, out=None, A_out=None, ws=None, status=None, stream=None):
    code, p, n = _gradients(G)
    out = torch.empty(n, dtype=torch.float32, device=G.device) if out is None else out
    ws = new_workspace(G, m) if ws is None else ws
    if A_out is not None:
        _dev(A_out, torch.float64, p * m, "A_out")
    _check(_lib.fa_aggregate(G.data_ptr(), code, p, n, m, float(lam), iters, _dev(out, torch.float32, n, "out"),
                             _ptr(A_out), ws.data_ptr(), ws.numel() * ws.element_size(), _ptr(status),
                             _stream(stream)), "fa_aggregate")
    return out


def fa_aggregate_host(G_host, m, lam, iters, out_host, G_dev, out_dev, ws, status_host=None, status_dev=None,
                      stream=None):
    """Host-buffer variant: G_host (pinned CPU tensor, p x n) -> out_host (pinned CPU, n floats).

    G_dev / out_dev / ws / status_dev are caller-owned device staging buffers.  The copies and the
    three kernels are enqueued on the stream; the caller synchronises before reading out_host.
    """
    code, p, n = _dtype_code(G_host), int(G_host.shape[0]), int(G_host.shape[1])
    if G_host.is_cuda or out_host.is_cuda or not G_host.is_contiguous():
        raise ValueError("G_host and out_host must be contiguous CPU tensors (pinned for async copies)")
    _check(_lib.fa_aggregate_host(G_host.data_ptr(), code, p, n, m, float(lam), iters, out_host.data_ptr(),
                                  _ptr(status_host), G_dev.data_ptr(), _dev(out_dev, torch.float32, n, "out_dev"),
                                  ws.data_ptr(), ws.numel() * ws.element_size(), _ptr(status_dev),
                                  _stream(stream)), "fa_aggregate_host")
    return out_host
