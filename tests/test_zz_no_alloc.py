"""fa_gram_static: the Gram pass for callers that cannot allocate device memory (no workspace
argument; the partial sums sit in an array built into the library).

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.  Checks, through the C ABI: same result as fa_gram, and as the CPU oracle's
plain inner products, on two calls in a row (the second call finds the first call's leftovers in
the shared array), a different shape in between, and a clear refusal beyond the array's size.
"""
import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import fa_oracle as fo

pytestmark = pytest.mark.gpu

GRAM_TOL = 5e-7     # same bound as the Gram parity tests, relative to sqrt(K_ii K_jj)


def _rel_err(K, Kref):
    scale = np.sqrt(np.outer(np.diag(Kref), np.diag(Kref)))
    scale[scale == 0] = 1.0
    return float(np.max(np.abs(K - Kref) / scale))


def test_static_scratch_gram_matches_workspace_gram_twice_in_a_row():
    import paper_2302_05865_b200 as fa
    big_np = si.ladder_case(15, 700_001, 31, "noisy_mean")
    small_np = si.ladder_case(32, 5_000, 32, "dup_zero")
    big, small = torch.from_numpy(big_np).cuda(), torch.from_numpy(small_np).cuda()
    exact, exact_small = fo.inner_products(si.to_float64(big_np)), fo.inner_products(si.to_float64(small_np))
    K = torch.empty((15, 15), dtype=torch.float64, device="cuda")
    ref = fa.fa_gram(big).cpu().numpy()
    first = fa.fa_gram_static(big, K=K).cpu().numpy()           # first call on this device: address lookup
    second = fa.fa_gram_static(big, K=K).cpu().numpy()          # array still holds the first call's sums
    assert _rel_err(first, ref) < GRAM_TOL and _rel_err(second, ref) < GRAM_TOL
    assert _rel_err(first, exact) < GRAM_TOL and _rel_err(second, exact) < GRAM_TOL and _rel_err(ref, exact) < GRAM_TOL
    # another shape (fewer blocks, wider slots) in between, then the first shape again
    ref_small = fa.fa_gram(small).cpu().numpy()
    got_small = fa.fa_gram_static(small).cpu().numpy()
    assert _rel_err(got_small, ref_small) < GRAM_TOL and _rel_err(got_small, exact_small) < GRAM_TOL
    third = fa.fa_gram_static(big, K=K).cpu().numpy()
    assert _rel_err(third, ref) < GRAM_TOL and _rel_err(third, exact) < GRAM_TOL


def test_static_scratch_gram_refuses_what_does_not_fit():
    import paper_2302_05865_b200 as fa
    G = torch.randn((33, 1000), device="cuda")
    with pytest.raises(fa.FaError, match="built-in scratch"):
        fa.fa_gram_static(G)
