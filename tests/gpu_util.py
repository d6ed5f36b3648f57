"""Helpers shared by the GPU parity tests (imported only when a CUDA device is present)."""
import numpy as np
import torch

import synthetic_inputs as si


def to_device(G_np: np.ndarray, misalign_elems: int = 0, redzone: int = 64):
    """Upload a generated matrix.  The rows are placed inside a larger NaN-filled buffer
    (red zones on both sides) starting `misalign_elems` elements past a 256-byte boundary.
    Returns (G view (p, n), whole buffer)."""
    p, n = G_np.shape
    if G_np.dtype == np.uint16:
        host = torch.from_numpy(G_np.view(np.int16)).view(torch.bfloat16)
        fill = float("nan")
    else:
        host = torch.from_numpy(G_np)
        fill = float("nan")
    lead = redzone + misalign_elems
    buf = torch.full((lead + p * n + redzone,), fill, dtype=host.dtype, device="cuda")
    buf[lead:lead + p * n] = host.reshape(-1).cuda()
    return buf[lead:lead + p * n].view(p, n), buf


def redzones_intact(buf: torch.Tensor, lead: int, count: int) -> bool:
    head = buf[:lead]
    tail = buf[lead + count:]
    return bool(torch.isnan(head.float()).all().item() and torch.isnan(tail.float()).all().item())


def subspace_from_A(G_np: np.ndarray, A: np.ndarray) -> np.ndarray:
    """Y = G^T A in fp64 (n x m), dropping all-zero columns of A."""
    X = si.to_float64(G_np)
    keep = np.any(A != 0.0, axis=0)
    return X.T @ A[:, keep]
