"""A device-side wait that runs out must end the kernel, not hang it: the kernel lets its copies land,
reports FA_ST_TIMEOUT and returns; the results are marked invalid (non-finite K, zero aggregate) and the
next call works.

Nothing is made to fail here.  The launch is a correct one; a test hook of the library (exported, not
part of the C ABI in include/fa.h) shortens the limit of the waits for a tile to one cycle, so the first
wait of every warp gives up while its tile is still on the way.  The waits that let copies in flight
land before a block exits keep their long limit, so every copy completes and the kernel ends normally.
"""
import ctypes

import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import fa_oracle as fo

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("p,n,m", [(15, 300_002, 8), (31, 200_000, 12), (40, 100_000, 12)])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_works(p, n, m):
    import paper_2302_05865_b200 as fa
    lib = ctypes.CDLL(fa.LIB_PATH)
    lib.fa_test_set_gram_wait_cycles.argtypes = [ctypes.c_longlong]
    lib.fa_test_set_gram_wait_cycles.restype = None
    G_np = si.ladder_case(p, n, 3, "noisy_mean")
    G = torch.from_numpy(G_np).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((n,), float("nan"), device="cuda")
    A = torch.full((p, m), float("nan"), dtype=torch.float64, device="cuda")
    try:
        lib.fa_test_set_gram_wait_cycles(1)
        fa.fa_aggregate(G, m, 0.01, 6, out=out, A_out=A, status=status)
        K = fa.fa_gram(G)
        torch.cuda.synchronize()
    finally:
        lib.fa_test_set_gram_wait_cycles(0)            # back to the default limit
    st = int(status.item())
    assert st & fa.ST_TIMEOUT, f"status {st}"
    assert st & fa.ST_NONFINITE                         # the IRLS kernel refused the unfinished inner products
    assert not out.any() and not A.any()                # ... and the outputs are zero, not garbage
    assert torch.isnan(K).all()                         # a caller of the Gram pass alone sees it too
    # the context is intact: the same call with the default limit gives the right answer
    out2 = fa.fa_aggregate(G, m, 0.01, 6, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = fo.fa_aggregate(G_np.astype(np.float64), m, 0.01, 6)
    assert fo.rel_l2(out2.cpu().numpy(), ref["d"]) < 1e-4
