"""The block operations of the C ABI (mbd_block_gemm_bf16, mbd_block_reduce, mbd_softmax_xent) on caller-owned
buffers, element by element against fp64: every tail operation, strided outputs and operands, both the
synchronous form and the enqueue-only form with a caller-owned status word."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu


def bf(a):
    return I.round_to_bf16(np.asarray(a, np.float32))


@pytest.mark.parametrize("enqueue_only", [False, True])
def test_block_products_with_every_tail(enqueue_only):
    import torch
    from paper_1712_04432_b200 import mbd
    r = np.random.default_rng(5)
    M, N, K = 72, 40, 136
    A, Bm = bf(r.standard_normal((M, K))), bf(r.standard_normal((N, K)))
    bias = r.standard_normal(N).astype(np.float32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda") if enqueue_only else None
    ref = A.astype(np.float64) @ Bm.astype(np.float64).T
    # variant 0, bias + ReLU, bf16 output written into a column slice of a wider buffer
    wide = torch.zeros((M, 2 * N), dtype=torch.bfloat16, device="cuda")
    mbd.block_gemm(0, to_dev(A, True), to_dev(Bm, True), wide[:, N:], mbd.TAIL_STORE, relu=True,
                   bias=torch.from_numpy(bias).cuda(), status=status)
    torch.cuda.synchronize()
    assert rel_fro(to_np(wide[:, N:]), np.maximum(ref + bias, 0)) < 5e-3 and not wide[:, :N].any()
    # variant 1 with a ReLU mask, float output; A is a column slice (row stride larger than K)
    Awide = to_dev(np.concatenate([A, A], axis=1), True)
    Bt = to_dev(np.ascontiguousarray(Bm.T), True)                       # [K, N]
    mask = bf(r.standard_normal((M, N)))
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    mbd.block_gemm(1, Awide[:, K:], Bt, out, mbd.TAIL_MASK, mask=torch.from_numpy(mask).cuda(), status=status)
    torch.cuda.synchronize()
    assert rel_fro(to_np(out), ref * (mask > 0)) < 2e-5
    # variant 2 with the update of Eq. 1 on bf16 weights
    At = to_dev(np.ascontiguousarray(A.T), True)                        # [K, M]
    W0 = bf(r.standard_normal((M, N)))
    W = to_dev(W0, True)
    mbd.block_gemm(2, At, Bt, W, mbd.TAIL_SGD, scale=-0.01, status=status)
    torch.cuda.synchronize()
    assert rel_fro(to_np(W), W0 - 0.01 * ref) < 5e-3
    if enqueue_only:
        assert int(status.item()) == 0


def test_block_reduce_and_softmax():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    r = np.random.default_rng(6)
    S, M, N = 3, 24, 40
    parts = r.standard_normal((S, M, N)).astype(np.float32)
    mask = bf(r.standard_normal((M, N)))
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    mbd.block_reduce(torch.from_numpy(parts).cuda(), out, mbd.TAIL_MASK, mask=to_dev(mask, True))
    want = ((parts[0] + parts[1]) + parts[2]) * (mask > 0)              # ascending order, fp32
    assert np.array_equal(to_np(out), bf(want).astype(np.float64))
    # one plane: the tail applied to a sum that is already complete
    W0 = r.standard_normal((M, N)).astype(np.float32)
    W = torch.from_numpy(W0.copy()).cuda()
    mbd.block_reduce(torch.from_numpy(parts[0]).cuda(), W, mbd.TAIL_SGD, scale=0.5)
    assert np.allclose(to_np(W), W0 + 0.5 * parts[0], rtol=0, atol=1e-6)
    # loss
    Bn, d = 12, 40
    logits = r.standard_normal((Bn, d)).astype(np.float32) * 3
    labels = r.integers(0, d, Bn).astype(np.int32)
    dY = torch.empty((Bn, d), dtype=torch.float32, device="cuda")
    per = torch.empty(Bn, dtype=torch.float32, device="cuda")
    mbd.softmax_xent(torch.from_numpy(logits).cuda(), torch.from_numpy(labels).cuda(), dY, per)
    J, per_ref, dY_ref = O.softmax_ce(logits.astype(np.float64).T, labels)
    assert rel_fro(to_np(per), per_ref) < 1e-5 and rel_fro(to_np(dY), dY_ref.T) < 1e-5


def test_views_at_odd_offsets_take_the_element_wise_kernels():
    # mbd_block_reduce and mbd_softmax_xent move 16 bytes per access only when every base is 16-byte aligned;
    # a view that starts 4 bytes into a buffer (leading dimension still a multiple of 8) gives the same values
    import torch
    from paper_1712_04432_b200 import mbd
    r = np.random.default_rng(8)
    S, M, N = 2, 16, 40
    parts = r.standard_normal((S, M, N)).astype(np.float32)
    mask = r.standard_normal((M, N)).astype(np.float32)
    buf = torch.zeros(M * N + 8, dtype=torch.float32, device="cuda")
    out = buf[1:1 + M * N].view(M, N)                                   # 4 bytes past a 16-byte boundary
    mbuf = torch.zeros(M * N + 8, dtype=torch.float32, device="cuda")
    mview = mbuf[3:3 + M * N].view(M, N)
    mview.copy_(torch.from_numpy(mask))
    mbd.block_reduce(torch.from_numpy(parts).cuda(), out, mbd.TAIL_MASK, mask=mview)
    assert np.array_equal(to_np(out), ((parts[0] + parts[1]) * (mask > 0)).astype(np.float64))
    assert float(buf[0]) == 0 and not buf[1 + M * N:].any()
    # softmax on a logits view at an odd offset, with one label out of range: NaN loss for that sample only
    Bn, d = 6, 40
    logits = r.standard_normal((Bn, d)).astype(np.float32)
    lbuf = torch.zeros(Bn * d + 8, dtype=torch.float32, device="cuda")
    lview = lbuf[1:1 + Bn * d].view(Bn, d)
    lview.copy_(torch.from_numpy(logits))
    labels = np.array([0, 5, 39, 40, -1, 7], np.int32)
    dY = torch.empty((Bn, d), dtype=torch.float32, device="cuda")
    per = torch.empty(Bn, dtype=torch.float32, device="cuda")
    mbd.softmax_xent(lview, torch.from_numpy(labels).cuda(), dY, per)
    p = np.exp(logits - logits.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    per_h = to_np(per)
    assert np.isnan(per_h[3]) and np.isnan(per_h[4]) and not np.isnan(per_h[[0, 1, 2, 5]]).any()
    for b in (0, 1, 2, 5):
        assert abs(per_h[b] + np.log(p[b, labels[b]])) < 1e-5
    assert np.allclose(to_np(dY)[3], p[3], atol=1e-6) and np.allclose(to_np(dY)[4], p[4], atol=1e-6)
