"""The integrated workload with the layer shapes of Section 3's network (alexlike: 11 x 11 stride 4, 5 x 5 stride 2, three
3 x 3 layers, the last with stride 2, then three fully connected layers; 128 images of 8 x 192 x 192) at FULL size and in
the launch configuration `bench.py --workload alexlike` times (the workload's second grid, 2 partial sums, fused update).

The oracle cannot run 128 such images in seconds, so it computes what can be computed piece by piece:
  * the step is independent per image except for the sums over the batch in dW / dK / db: activations, per-sample
    losses and back-propagated gradients of three sampled images from the oracle's own step on exactly those images
    (ReLU decisions of those images forced to the oracle's stored activations, as in the other parity tests);
  * J as the sum of the device's own per-sample losses (the loss reduction at this size);
  * the sums over the batch from the oracle's weight-gradient functions fed with the operands the device itself
    stored: dW and db of every fully connected layer in full, dK of every convolution for eight sampled output
    channels; then the fused update at a learning rate that makes the step as large as the weights, against Eq. 1 on
    those gradients.
"""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import bf16_store, mixed_layers, oracle_kernel, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu

SEL = [0, 77, 127]


def o_sel(c_out):
    return sorted({0, 1, c_out // 3, c_out // 2, c_out // 2 + 1, c_out - 33, c_out - 2, c_out - 1})


def make_net(w, inp, grid, mp):
    import torch
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mixed_layers(w), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
    for i in range(w.L):
        if i < w.n_layers:
            net.set_weights(i, to_dev(inp.Ws[i], True))
        else:
            net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    return net


def test_alexlike_in_the_benchmarks_configuration():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.WORKLOADS["alexlike"]
    grid = w.grids[1]
    L, Lc, B = w.L, w.n_layers, w.B
    assert grid == (2, 8) and w.strides == (4, 2, 1, 1, 2) and B == 128
    inp = I.make_inputs(w, seed=0)
    layers = [O.Conv3x3(oracle_kernel(inp.Ws[i]), relu=True, stride=w.stride(i)) for i in range(Lc)]
    layers += [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64), relu=True) for i in range(Lc, L)]
    o = O.train_step(layers, inp.X[SEL].astype(np.float64), inp.labels[SEL], "softmax_ce", w.eta, store=bf16_store)

    def ref_layout(a, i):           # the oracle's tensor on the output side of layer i, in the device's layout, sampled images
        if i < Lc:
            return a if a.ndim == 4 else np.ascontiguousarray(a.T).reshape(len(SEL), w.chan(Lc), *w.out_hw(Lc - 1))
        return a.T

    X = to_dev(inp.X, True)
    labels = torch.from_numpy(inp.labels).cuda()
    net = make_net(w, inp, grid, 2)
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    net.forward(X, labels, J)
    acts = [net.get_tensor(mbd.T_ACT, i) for i in range(L)]
    for i in range(L):
        ref = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        assert rel_fro(to_np(acts[i][SEL]), ref_layout(ref, i)) < 1e-2, f"Y[{i}] of the sampled images"
    loss = to_np(net.get_tensor(mbd.T_LOSS))
    assert rel_fro(loss[SEL], o["per_sample"]) < 1e-2
    assert abs(float(J.item()) - loss.sum()) < 1e-4 * loss.sum()
    # ReLU decisions of the sampled images on the oracle's stored activations
    for i in range(L - 1):
        acts[i][SEL] = to_dev(np.ascontiguousarray(ref_layout(o["Xs"][i + 1], i), np.float32), True)
        net.set_tensor(mbd.T_ACT, i, acts[i])
    net.backward(0.0)
    net.poll()
    dYs = [net.get_tensor(mbd.T_DY, i) for i in range(L)]
    for i in range(L):
        assert rel_fro(to_np(dYs[i][SEL]), ref_layout(o["dYs"][i], i)) < 1e-2, f"dY[{i}] of the sampled images"
    # the sums over the batch, from the device's own stored operands
    refs, sels = [], []
    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_DW, i))
        if i < Lc:
            sel = o_sel(w.chan(i + 1))
            x_in = inp.X.astype(np.float64) if i == 0 else to_np(acts[i - 1])
            dy = to_np(dYs[i][:, sel])
            ref = O.conv_strided_dK(dy, x_in, w.kshape(i), w.stride(i)) if w.stride(i) > 1 else O.conv3x3_dK(dy, x_in, w.kshape(i))
            assert rel_fro(got[sel], ref) < 1e-4, f"dK[{i}], sampled output channels, all {B} images"
        else:
            sel = slice(None)
            x_in = to_np(acts[i - 1]).reshape(B, -1)
            dy = to_np(dYs[i])
            ref = O.fc_dW(dy.T, x_in.T)
            assert rel_fro(got, ref) < 1e-4, f"dW[{i}], all {B} samples"
            db = to_np(net.get_tensor(mbd.T_DB, i))
            assert rel_fro(db, dy.sum(axis=0)) < 1e-4, f"db[{i}]"
        refs.append(ref)
        sels.append(sel)
    net.sgd_step(0.0)
    # the fused update at a learning rate that moves every layer by at least its own norm
    eta = B * max(np.linalg.norm(inp.Ws[i].astype(np.float64)[sels[i]]) / np.linalg.norm(refs[i]) for i in range(L))
    net.forward(X, labels, J)
    for i in range(L - 1):
        net.set_tensor(mbd.T_ACT, i, acts[i])
    net.backward(float(eta))
    net.poll()
    for i in range(L):
        W0 = inp.Ws[i].astype(np.float64)[sels[i]]
        want = O.sgd(W0, refs[i], eta, B)
        got = to_np(net.get_weights(i))[sels[i]]
        step = np.linalg.norm(want - W0)
        assert step > 0.5 * np.linalg.norm(W0), i
        assert np.linalg.norm((got - W0) - (want - W0)) < 5e-3 * step, f"W_new[{i}] - W_0[{i}]"
    net.close()
