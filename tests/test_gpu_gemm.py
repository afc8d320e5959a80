"""The weight-streaming GEMM kernel alone, through its C-ABI test hook, against an fp64 product
of the same bf16 weights and fp32 activations (a library matmul as the plain definition)."""
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


SHAPES = [
    (128, 64, 8),        # one tile, one k-block
    (128, 256, 8),       # one tile, several k-blocks
    (384, 64, 8),        # several tiles
    (300, 200, 8),       # ragged N and K (TMA zero fill on both edges)
    (1376, 256, 8),      # C1 gate/up
    (256, 688, 8),       # C1 down: K tail of 48
    (4096, 256, 8),      # C1 LM head
    (4096, 4096, 8),     # 7B O projection: every tile cut into several segments
    (1000, 2048, 24),    # 3 sequences: MMA N = 32
    (640, 1024, 64),     # prefill width
    (512, 512, 128),     # widest batch
    (22016, 4096, 8),    # 7B gate/up: two MMA row tiles per CTA in the row-range kernel
    (4096, 11008, 8),    # 7B down: 28 features per CTA, four k-blocks per stage
    (30, 72, 8),         # fewer feature pairs than SMs, K tail of 8
    (301, 64, 8),        # odd N: the last feature pair is half empty
]


@pytest.mark.parametrize("N,K,rows", SHAPES)
def test_gemm_matches_fp64_product(A, N, K, rows):
    w = normal_tensor(N * 7 + K, 1, N * K, 0.05).view(N, K).to(torch.bfloat16)
    a = normal_tensor(N + K * 3, 2, rows * K, 1.0).view(rows, K)
    a[0, :] = 0.0                      # a zero row must give exact zeros
    a[1, 0] = 1000.0                   # mixed magnitudes exercise the hi + lo split
    want = a.double() @ w.double().T
    scale = float(want.abs().max()) + 1e-6
    for plain in ((1, 0, 2) if rows == 8 else (1, 0)):          # 2: the row-range kernel of single-sequence steps
        got = torch.from_numpy(A.anpd_debug_gemm(w, a.numpy(), plain=plain)).double()
        err = float((got - want).abs().max())
        # hi + lo carries about 16 mantissa bits: 2e-5.  The row-range kernel keeps ONE fp32 accumulator over the whole of
        # K (K / 16 tensor-core accumulation steps, each of which may drop the bits below the accumulator's last place),
        # where stream-K adds a few shorter segments: allow one unit in the last place (2^-23) per step beside it.
        tol = 2e-5 + (2.0 ** -23) * (K / 16) if plain == 2 else 2e-5
        assert err <= tol * scale + 1e-6, (plain, err, scale)
        assert float(got[0].abs().max()) == 0.0


def test_rows_do_not_influence_each_other(A):
    N, K = 1024, 1024
    w = normal_tensor(5, 1, N * K, 0.05).view(N, K).to(torch.bfloat16)
    a = normal_tensor(6, 2, 64 * K, 1.0).view(64, K).numpy()
    wide = A.anpd_debug_gemm(w, a)
    narrow = A.anpd_debug_gemm(w, a[:8])
    other = a.copy()
    other[8:] = 3.0
    mixed = A.anpd_debug_gemm(w, other[:16])
    assert np.array_equal(wide[:8], narrow) and np.array_equal(mixed[:8], narrow)


def test_row_range_kernel_rows_are_independent(A):
    """Single-sequence steps always carry 8 rows; a row's result must not depend on what the other rows hold."""
    N, K = 1536, 1024
    w = normal_tensor(15, 1, N * K, 0.05).view(N, K).to(torch.bfloat16)
    a = normal_tensor(16, 2, 8 * K, 1.0).view(8, K).numpy()
    full = A.anpd_debug_gemm(w, a, plain=2)
    other = a.copy()
    other[1:] = 0.0
    alone = A.anpd_debug_gemm(w, other, plain=2)
    assert np.array_equal(full[0], alone[0]) and float(np.abs(alone[1:]).max()) == 0.0
