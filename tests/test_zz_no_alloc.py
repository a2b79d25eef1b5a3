"""The allocation-free contraction entry point against the ordinary one.

Some callers of this library may not allocate GPU memory and may not let a library do so on
their behalf: a server that hands all device memory to its own pool at start-up, or a
plug-in that runs at a point where cudaMalloc would block or fail.  For them
mbd_gemm_bf16_noalloc keeps its partial sums in a fixed array built into the library.  This
file is collected last on purpose; it checks two calls in a row (the array is shared and keeps
the previous call's contents) against mbd_gemm_bf16, which takes its scratch from the caller.
"""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import to_dev, to_np

pytestmark = pytest.mark.gpu


def _operands(variant, M, N, K, seed):
    r = np.random.default_rng(seed)
    a_shape = (M, K) if variant < 2 else (K, M)
    b_shape = (N, K) if variant == 0 else (K, N)
    return (I.round_to_bf16(r.standard_normal(a_shape).astype(np.float32)),
            I.round_to_bf16(r.standard_normal(b_shape).astype(np.float32)))


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    import torch
    from paper_1712_04432_b200 import mbd
    # first call: larger problem, 4 partial sums; second: smaller and 3 partial sums, so stale
    # contents of the shared array from the first call would show up if they were read
    cases = [(2, 520, 392, 1024, 4), (1, 264, 328, 448, 3), (0, 136, 200, 72, 1)]
    for variant, M, N, K, S in cases:
        A, B = _operands(variant, M, N, K, seed=M + S)
        a, b = to_dev(A, True), to_dev(B, True)
        ref = mbd.gemm_bf16(variant, a, b, k_splits=S)
        out = torch.empty((M, N), dtype=torch.float32, device="cuda")
        got = mbd.gemm_bf16_noalloc(variant, a, b, k_splits=S, out=out)
        # same kernels, same split, same summation order: identical, hence also within the
        # 2e-5 relative tolerance the contraction tests use
        assert torch.equal(got, ref)
        exact = (A.astype(np.float64) @ B.astype(np.float64).T if variant == 0 else
                 A.astype(np.float64) @ B.astype(np.float64) if variant == 1 else
                 A.astype(np.float64).T @ B.astype(np.float64))
        assert np.linalg.norm(to_np(got) - exact) / np.linalg.norm(exact) < 2e-5


def test_rejects_problems_beyond_the_fixed_scratch():
    import torch
    from paper_1712_04432_b200 import mbd
    a = torch.zeros((2048, 256), dtype=torch.bfloat16, device="cuda")
    b = torch.zeros((2048, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mbd.MbdError) as e:
        mbd.gemm_bf16_noalloc(0, a, b, k_splits=2)        # 2 * 2048 * 2048 floats > 4 Mi
    assert e.value.status == mbd.E_TOO_LARGE
    assert "scratch" in str(e.value)
    mbd.gemm_bf16_noalloc(0, a, b, k_splits=1)            # without partial sums it fits
