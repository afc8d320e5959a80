"""anpd_gemm_static: the GEMM entry point that allocates nothing.

It is meant for callers that cannot let the library call cudaMalloc (a serving loop that must not be
stalled by an allocation's device-wide synchronisation; a process whose device memory belongs to
another allocator).  Its temporaries live in one fixed array inside the loaded library, shared by all
calls.  The test runs it twice in a row, the second time on a smaller problem with other values so
that anything left over from the first call would show, and compares each result with
anpd_debug_gemm, the allocating entry point for the same product.  This file sorts last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from helpers import require_gpu
from workloads.rng import normal_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def A():
    require_gpu()
    from paper_2404_08698_b200 import binding
    return binding


def one_call(A, N, K, rows, seed):
    w = normal_tensor(seed, 1, N * K, 0.05).view(N, K).to(torch.bfloat16)
    a = normal_tensor(seed, 2, rows * K, 1.0).view(rows, K)
    want = A.anpd_debug_gemm(w, a.numpy())                      # existing entry point (allocates)
    w_dev, a_dev = w.cuda(), a.cuda()
    out_dev = torch.full((rows, N), float("nan"), device="cuda")
    torch.cuda.synchronize()
    A.anpd_gemm_static(w_dev, a_dev, out_dev)
    got = out_dev.cpu().numpy()
    scale = float(np.abs(want).max()) + 1e-6
    err = float(np.abs(got - want).max())
    assert err <= 2e-5 * scale + 1e-6, (N, K, rows, err, scale)   # the tolerance of the GEMM tests
    return got, want


def test_two_calls_in_a_row_match_the_allocating_entry_point(A):
    got1, want1 = one_call(A, 1000, 512, 16, seed=41)             # 8 x 8 blocks, ragged N
    got2, want2 = one_call(A, 300, 200, 8, seed=42)               # smaller, ragged N and K: stale scratch would show
    # same kernel, same order of additions: the two entry points agree to the last bit
    assert np.array_equal(got1, want1) and np.array_equal(got2, want2)


def test_same_shape_other_weights_uses_the_new_weights(A):
    """Two calls of one shape with different weights: the second must see its own weight blocks in the
    shared scratch, not the first call's (the GEMM may not fetch them ahead of the kernel that writes them)."""
    got1, want1 = one_call(A, 640, 448, 8, seed=51)
    got2, want2 = one_call(A, 640, 448, 8, seed=52)
    assert np.array_equal(got1, want1) and np.array_equal(got2, want2)
    assert not np.array_equal(got1, got2)


def test_sizes_beyond_the_fixed_scratch_are_rejected(A):
    w = torch.zeros(4096, 4096, dtype=torch.bfloat16, device="cuda")   # 32 x 64 = 2048 blocks > 128
    a = torch.zeros(8, 4096, device="cuda")
    out = torch.zeros(8, 4096, device="cuda")
    with pytest.raises(A.AnpdError) as e:
        A.anpd_gemm_static(w, a, out)
    assert e.value.status == A.ERR_CAPACITY
    with pytest.raises(A.AnpdError) as e:
        A.anpd_gemm_static(w[:128, :64].contiguous(), torch.zeros(40, 64, device="cuda"), torch.zeros(40, 128, device="cuda"))
    assert e.value.status == A.ERR_CAPACITY                            # 40 rows > 32
