"""The tensor-core contraction alone, against fp64 products of the same bf16 inputs:
each operand-major combination (forward, backward-data, backward-weight), one tile,
several tiles with ragged edges, and K cut into partial sums."""
import numpy as np
import pytest

from oracle import mbd_oracle as O
from paper_1712_04432_b200 import inputs as I
from tests.helpers import rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu

# bf16 inputs are exact, products exact in fp32, only the fp32 accumulation rounds
TOL = 2e-5


def operands(variant, M, N, K, seed):
    r = np.random.default_rng(seed)
    a_shape = (M, K) if variant < 2 else (K, M)
    b_shape = (N, K) if variant == 0 else (K, N)
    A = I.round_to_bf16(r.standard_normal(a_shape).astype(np.float32))
    B = I.round_to_bf16(r.standard_normal(b_shape).astype(np.float32))
    return A, B


def reference(variant, A, B):
    A = A.astype(np.float64)
    B = B.astype(np.float64)
    if variant == 0:
        return O.affine(A, B.T)            # A [M,K] (B [N,K])^T
    if variant == 1:
        return O.affine(A, B)              # A [M,K] B [K,N]
    return O.fc_dW(A.T, B.T)               # (A [K,M])^T B [K,N] = sum_k A[k,:]^T B[k,:]


SHAPES = [(128, 128, 64), (128, 256, 128), (128, 128, 1024), (256, 512, 192), (200, 328, 72),
          (392, 1000, 520), (64, 8, 40), (1024, 1024, 1024)]


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("shape", SHAPES)
def test_gemm_matches_fp64(variant, shape):
    from paper_1712_04432_b200 import mbd
    M, N, K = shape
    A, B = operands(variant, M, N, K, seed=100 * variant + M + N + K)
    D = mbd.gemm_bf16(variant, to_dev(A, True), to_dev(B, True))
    err = rel_fro(to_np(D), reference(variant, A, B))
    assert err < TOL, (variant, shape, err)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("S", [2, 3, 8])
def test_k_split_partials_and_their_sum(variant, S):
    from paper_1712_04432_b200 import mbd
    M, N, K = 264, 392, 1024
    A, B = operands(variant, M, N, K, seed=7 + S)
    D, parts = mbd.gemm_bf16(variant, to_dev(A, True), to_dev(B, True), k_splits=S, return_partials=True)
    ref = reference(variant, A, B)
    assert rel_fro(to_np(D), ref) < TOL
    # each partial is the product over its own K range (64-wide blocks, balanced)
    kb = (K + 63) // 64
    P = to_np(parts)
    for s in range(S):
        k0, k1 = 64 * ((s * kb) // S), min(K, 64 * (((s + 1) * kb) // S))
        if variant == 0:
            ref_s = reference(0, A[:, k0:k1], B[:, k0:k1])
        elif variant == 1:
            ref_s = reference(1, A[:, k0:k1], B[k0:k1, :])
        else:
            ref_s = reference(2, A[k0:k1, :], B[k0:k1, :])
        assert rel_fro(P[s], ref_s) < TOL, (variant, S, s)
    # fixed ascending order: the sum is reproducible bit for bit
    D2 = mbd.gemm_bf16(variant, to_dev(A, True), to_dev(B, True), k_splits=S)
    assert np.array_equal(to_np(D), to_np(D2))


def test_asymmetric_values_catch_transposition():
    # A = outer(row index, 1), B = outer(col index, 1) over K: D[m,n] = K * m * n exactly
    from paper_1712_04432_b200 import mbd
    M, N, K = 128, 136, 64
    A = np.repeat(np.arange(M, dtype=np.float32)[:, None] % 16, K, axis=1)
    B = np.repeat(np.arange(N, dtype=np.float32)[:, None] % 8, K, axis=1)
    D = to_np(mbd.gemm_bf16(0, to_dev(A, True), to_dev(B, True)))
    assert np.array_equal(D, K * np.outer(np.arange(M) % 16, np.arange(N) % 8))


MODES = {
    "tile128x128": {"MBD_TC_MH": "1", "MBD_TC_BN": "128", "MBD_TC_PAIR": "0"},
    "tile128x256": {"MBD_TC_MH": "1", "MBD_TC_BN": "256", "MBD_TC_PAIR": "0"},
    "tile256x256": {"MBD_TC_MH": "2", "MBD_TC_BN": "256", "MBD_TC_PAIR": "0"},
    "cta_pair": {"MBD_TC_PAIR": "1"},
    "cta_pair512x256": {"MBD_TC_PAIR": "2"},
}


@pytest.mark.parametrize("mode", sorted(MODES))
@pytest.mark.parametrize("variant", [0, 1, 2])
def test_every_tile_shape_and_the_cta_pair(monkeypatch, mode, variant):
    # the planner normally picks the tile shape; force each one (tuning knobs) on ragged sizes
    from paper_1712_04432_b200 import mbd
    for k, v in MODES[mode].items():
        monkeypatch.setenv(k, v)
    for (M, N, K, S) in [(648, 776, 328, 1), (392, 1000, 520, 3)]:
        A, B = operands(variant, M, N, K, seed=31 * variant + S)
        D = mbd.gemm_bf16(variant, to_dev(A, True), to_dev(B, True), k_splits=S)
        err = rel_fro(to_np(D), reference(variant, A, B))
        assert err < TOL, (mode, variant, M, N, K, S, err)


def test_random_shapes_sweep():
    # 24 seeded random problems: sizes are multiples of 8 (the 16-byte rule of TMA), any layout,
    # K cut into 1..5 pieces; whatever tile shape the planner picks must agree with fp64
    from paper_1712_04432_b200 import mbd
    r = np.random.default_rng(2024)
    for case in range(24):
        variant = int(r.integers(0, 3))
        M, N, K = (8 * int(r.integers(1, 150)) for _ in range(3))
        S = int(r.integers(1, 6))
        A, B = operands(variant, M, N, K, seed=1000 + case)
        D = mbd.gemm_bf16(variant, to_dev(A, True), to_dev(B, True), k_splits=S)
        err = rel_fro(to_np(D), reference(variant, A, B))
        assert err < TOL, (case, variant, M, N, K, S, err)
