"""The strided general-convolution workload of the benchmark (conv5x5s2: 5 x 5 stride 2, 64 -> 128 channels on 224 x 224
inputs, then 3 x 3, 128 -> 128 on the 112 x 112 result, 32 images) at FULL size and in the launch configuration
`bench.py --workload conv5x5s2` times (2 strips, max_partials 2).

The oracle cannot run 32 such images in seconds, so it computes what can be computed piece by piece:
  * the step is independent per image except for the sums over the batch in dK: forward outputs and the
    back-propagated gradient of three sampled images from the oracle's own step on exactly those images (ReLU decisions
    of those images forced to the oracle's stored activations, as in the other parity tests);
  * J as the half sum of squares of the device's own stored last output (the loss reduction at this size);
  * the sums over the batch: dK of the second layer in full, and of the first (strided) layer for eight sampled output
    channels, from the oracle's weight-gradient functions fed with the operands the device itself stored; the fused
    update at a learning rate that makes the step as large as the weights, against Eq. 1 on those gradients.
"""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import bf16_store, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu

SEL = [0, 17, 31]
O_SEL = [0, 1, 31, 64, 65, 100, 126, 127]


def make_net(w, inp, mp=2):
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.conv_layers(w.n_layers, w.dims[0], w.dims[1], w.dims[2], k=[w.kshape(i) for i in range(w.n_layers)],
                                  channels=w.channels, strides=w.strides), w.B, 2, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, mp)
    for i in range(w.n_layers):
        net.set_weights(i, to_dev(inp.Ws[i], True))
    return net


def test_conv5x5s2_in_the_benchmarks_configuration():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.WORKLOADS["conv5x5s2"]
    assert w.grids[1] == (2, 1) and w.strides == (2, 1)
    inp = I.make_inputs(w, seed=0)
    layers = [O.Conv3x3(inp.Ws[i].astype(np.float64), relu=True, stride=w.stride(i)) for i in range(2)]
    o = O.train_step(layers, inp.X[SEL].astype(np.float64), None, "half_ssq", w.eta, store=bf16_store)
    X = to_dev(inp.X, True)
    net = make_net(w, inp)
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    net.forward(X, None, J)
    act0, act1 = net.get_tensor(mbd.T_ACT, 0), net.get_tensor(mbd.T_ACT, 1)
    assert tuple(act0.shape) == (32, 128, 112, 112) and tuple(act1.shape) == (32, 128, 112, 112)
    assert rel_fro(to_np(act0[SEL]), o["Xs"][1]) < 1e-2 and rel_fro(to_np(act1[SEL]), o["Ys"][1]) < 1e-2
    J_own = 0.5 * float((act1.double() ** 2).sum())
    assert abs(float(J.item()) - J_own) < 1e-4 * J_own
    # ReLU decisions of the sampled images on the oracle's stored activations
    act0[SEL] = to_dev(np.ascontiguousarray(o["Xs"][1], np.float32), True)
    net.set_tensor(mbd.T_ACT, 0, act0)
    net.backward(0.0)
    net.poll()
    dY0, dY1 = net.get_tensor(mbd.T_DY, 0), net.get_tensor(mbd.T_DY, 1)
    assert rel_fro(to_np(dY1[SEL]), o["dYs"][1]) < 1e-2 and rel_fro(to_np(dY0[SEL]), o["dYs"][0]) < 1e-2
    # the sums over the batch, from the device's own stored operands
    dK1_ref = O.conv3x3_dK(to_np(dY1), to_np(act0), (3, 3))
    dK1 = to_np(net.get_tensor(mbd.T_DW, 1))
    assert rel_fro(dK1, dK1_ref) < 1e-4, "dK of the 3 x 3 layer, all 32 images"
    dK0_ref = O.conv_strided_dK(to_np(dY0[:, O_SEL]), inp.X.astype(np.float64), (5, 5), 2)
    dK0 = to_np(net.get_tensor(mbd.T_DW, 0))
    assert rel_fro(dK0[O_SEL], dK0_ref) < 1e-4, "dK of the strided 5 x 5 layer, sampled output channels"
    net.sgd_step(0.0)
    # the fused update at a learning rate that moves the kernels by their own norm
    eta = w.B * max(np.linalg.norm(inp.Ws[0][O_SEL]) / np.linalg.norm(dK0_ref), np.linalg.norm(inp.Ws[1]) / np.linalg.norm(dK1_ref))
    net.forward(X, None, J)
    net.set_tensor(mbd.T_ACT, 0, act0)
    net.backward(float(eta))
    net.poll()
    for i, (ref, sel) in enumerate([(dK0_ref, O_SEL), (dK1_ref, slice(None))]):
        W0 = inp.Ws[i].astype(np.float64)[sel]
        want = O.sgd(W0, ref, eta, w.B)
        got = to_np(net.get_weights(i))[sel]
        step = np.linalg.norm(want - W0)
        assert step > 0.5 * np.linalg.norm(W0)
        assert np.linalg.norm((got - W0) - (want - W0)) < 5e-3 * step, f"K_new[{i}] - K_0[{i}]"
    net.close()
