"""Host-side logic of the C ABI that needs no GPU: argument validation of mbd_net_create
(checked before any CUDA call), and the loud failure when no device is present."""
import ctypes as C

import pytest

from paper_1712_04432_b200 import mbd


def create(layers, B, P_r=1, P_c=1, dtype=mbd.BF16, loss=mbd.LOSS_SOFTMAX_CE, max_partials=0):
    h = C.c_void_p()
    st = mbd.lib().mbd_net_create(mbd._layer_array(layers), len(layers), B, P_r, P_c, dtype, loss, max_partials,
                                  None, C.byref(h))
    if st == mbd.OK:
        mbd.lib().mbd_net_destroy(h)
    return st


def test_grid_errors():
    fc = mbd.fc_layers((64, 32, 16))
    assert create(fc, 8, 0, 1) == mbd.E_GRID
    assert create(fc, 8, 1, 0) == mbd.E_GRID
    assert create(fc, 8, 1, 9) == mbd.E_GRID          # more batch blocks than samples
    assert create(fc, 8, 17, 1) == mbd.E_GRID         # more row blocks than neurons of the last layer
    conv = mbd.conv_layers(2, 64, 8, 16)
    assert create(conv, 4, 9, 1, loss=mbd.LOSS_HALF_SSQ) == mbd.E_GRID    # strips shorter than one row
    assert create(conv, 4, 2, 5, loss=mbd.LOSS_HALF_SSQ) == mbd.E_GRID    # more batch blocks than samples


def test_invalid_and_unsupported():
    fc = mbd.fc_layers((64, 32, 16))
    assert create(fc, 0) == mbd.E_INVALID
    assert create(fc, 8, dtype=5) == mbd.E_INVALID
    assert create(fc, 8, loss=9) == mbd.E_INVALID
    assert create(fc, 8, max_partials=-1) == mbd.E_INVALID
    assert create(mbd.fc_layers((64, 32)) + mbd.fc_layers((48, 16)), 8) == mbd.E_INVALID   # dims do not chain
    assert create(mbd.fc_layers((60, 30)), 8) == mbd.E_UNSUPPORTED                         # bf16 needs multiples of 8
    conv9 = mbd.conv_layers(1, 64, 8, 16)
    conv9[0].kh = conv9[0].kw = 13                                                         # kernels up to 11 x 11
    assert create(conv9, 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_UNSUPPORTED
    conv43 = mbd.conv_layers(1, 64, 8, 16)
    conv43[0].kh = 4                                                                       # even sizes have no centre tap
    assert create(conv43, 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_UNSUPPORTED
    assert create(mbd.conv_layers(1, 12, 8, 16), 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_UNSUPPORTED      # channels: multiples of 8
    assert create(mbd.conv_layers(2, 16, 8, 16, channels=(16, 32, 8))[:1] + mbd.conv_layers(1, 16, 8, 16), 4,
                  loss=mbd.LOSS_HALF_SSQ) == mbd.E_INVALID                                 # channel counts do not chain
    assert create(mbd.conv_layers(2, 16, 8, 16, k=[(5, 5), (1, 7)], channels=(16, 32, 8)), 4, loss=mbd.LOSS_HALF_SSQ) in (mbd.OK, mbd.E_CUDA)
    # strides: the image sizes must chain (H_{i+1} = H_i / s_i), divide by the stride, and the stride is at most 4
    assert create(mbd.conv_layers(2, 16, 16, 16, strides=(2, 1)), 4, loss=mbd.LOSS_HALF_SSQ) in (mbd.OK, mbd.E_CUDA)
    unchained = mbd.conv_layers(2, 16, 16, 16, strides=(2, 1))
    unchained[1].H = 16
    assert create(unchained, 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_INVALID
    odd = mbd.conv_layers(1, 16, 16, 16)
    odd[0].stride = 3                                                                      # 16 rows, stride 3
    assert create(odd, 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_INVALID
    far = mbd.conv_layers(1, 16, 40, 40)
    far[0].stride = 5
    assert create(far, 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_UNSUPPORTED
    assert create(mbd.conv_layers(1, 16, 16, 16, strides=(2,)), 4, 16, 1, loss=mbd.LOSS_HALF_SSQ) == mbd.E_GRID    # 8 output rows, 16 strips
    assert create(mbd.conv_layers(2, 64, 8, 16, k=[3, 1]), 4, loss=mbd.LOSS_HALF_SSQ) in (mbd.OK, mbd.E_CUDA)   # valid; E_CUDA only without a device
    assert create(mbd.conv_layers(1, 64, 8, 16), 4, loss=mbd.LOSS_SOFTMAX_CE) == mbd.E_UNSUPPORTED
    assert create(fc, 8, loss=mbd.LOSS_NONE) == mbd.E_UNSUPPORTED                          # "no loss" is for convolution stacks
    assert create(mbd.conv_layers(1, 64, 8, 16), 4, loss=mbd.LOSS_NONE) in (mbd.OK, mbd.E_CUDA)
    # convolutions first, fully connected layers after them
    conv = mbd.conv_layers(1, 64, 8, 16)
    assert create(mbd.fc_layers((64, 64 * 8 * 16)) + conv, 4) == mbd.E_UNSUPPORTED          # convolution above an FC layer
    assert create(conv + mbd.fc_layers((64 * 8 * 16 - 8, 16)), 4) == mbd.E_INVALID          # d_in is not C*H*W
    assert create(conv + mbd.fc_layers((64 * 8 * 16, 16)), 4, loss=mbd.LOSS_HALF_SSQ) == mbd.E_UNSUPPORTED
    assert create(conv + mbd.fc_layers((64 * 8 * 16, 16)), 4, dtype=mbd.F32) == mbd.E_UNSUPPORTED


def test_null_handles_are_rejected():
    L = mbd.lib()
    assert L.mbd_forward(None, None, None, None) == mbd.E_INVALID
    assert L.mbd_backward(None, 0.0) == mbd.E_INVALID
    assert L.mbd_sgd_step(None, 0.1) == mbd.E_INVALID
    assert L.mbd_poll_status(None) == mbd.E_INVALID
    assert L.mbd_enable_master_weights(None) == mbd.E_INVALID
    assert L.mbd_conv_stage_input(None, None) == mbd.E_INVALID
    assert L.mbd_conv_forward_layer(None, 0, None) == mbd.E_INVALID
    assert L.mbd_conv_backward_layer(None, 0, 0.0) == mbd.E_INVALID
    assert L.mbd_conv_outer_rows(None, 0, 0, 0, None, 0, 0) == mbd.E_INVALID
    assert L.mbd_launch_count(None) == -1
    assert L.mbd_net_destroy(None) == mbd.E_INVALID


def test_no_silent_fallback_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # valid arguments, but no device: the library reports a CUDA error instead of computing elsewhere
    assert create(mbd.fc_layers((64, 32, 16)), 8) == mbd.E_CUDA
    assert create(mbd.fc_layers((64, 32, 16)), 8, dtype=mbd.F32) == mbd.E_CUDA


def test_block_calls_reject_bad_arguments():
    import ctypes as C
    from paper_1712_04432_b200 import mbd
    L = mbd.lib()
    t = mbd.Tail(mbd.TAIL_STORE, 0, 0, 0, None, 8, None, None, 0, 0.0)          # no output buffer
    assert L.mbd_block_gemm_bf16(0, 8, 8, 8, None, 8, None, 8, C.byref(t), None, None) == mbd.E_INVALID
    assert L.mbd_block_reduce(None, 1, 8, 8, C.byref(t), 1, None) == mbd.E_INVALID
    assert L.mbd_softmax_xent(None, 1, 8, None, None, 0, None, 1, None) == mbd.E_INVALID


def test_misaligned_bases_are_rejected_before_anything_is_launched():
    # The contraction moves its operands by TMA and its results by 16-byte stores: a view that starts
    # at an odd offset (leading dimension still a multiple of 8) gets a return code, never a launch.
    # The addresses are made up and never dereferenced: the checks run before any CUDA call.
    L = mbd.lib()
    ok, odd = 0x7000000000, 0x7000000000 + 4
    args = lambda A, B, D: (0, 64, 64, 64, C.c_void_p(A), 64, C.c_void_p(B), 64, C.c_void_p(D), 64, 1)
    for A, B, D in [(odd, ok, ok), (ok, odd, ok), (ok, ok, odd)]:
        assert L.mbd_gemm_bf16(*args(A, B, D), None, None) == mbd.E_UNSUPPORTED
        assert L.mbd_gemm_bf16_noalloc(*args(A, B, D), None) == mbd.E_UNSUPPORTED
    for field in ("out", "mask", "bias"):
        t = mbd.Tail(mbd.TAIL_MASK, 1, 0, 0, odd if field == "out" else ok, 64, odd if field == "bias" else None,
                     odd if field == "mask" else None, 64, 0.0)
        assert L.mbd_block_gemm_bf16(0, 64, 64, 64, C.c_void_p(ok), 64, C.c_void_p(ok), 64, C.byref(t), None, None) == mbd.E_UNSUPPORTED


def test_plan_query_rejects_bad_arguments():
    p = mbd.Plan()
    assert mbd.lib().mbd_get_plan(None, 0, 0, C.byref(p)) == mbd.E_INVALID
