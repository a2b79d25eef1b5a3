"""The integrated stack of the benchmark (two convolutions on 256 images of 56 x 56, then
200704 -> 1024 -> 1024 -> 1000) at FULL size and in the benchmark's launch configuration.  The
oracle cannot run the whole step in seconds, so it computes what is independent per sample on a few
samples (forward activations, loss, back-propagated gradients), and every sum over the batch
(dW_i = dY_i X_i^T, the kernel gradients) from the device's own stored dY_i and X_i in fp64."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import bf16_store, mixed_layers, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu


def test_mixed_full_size_sampled_and_batch_sums():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.WORKLOADS["mixed"]
    inp = I.make_inputs(w, seed=0)
    L, Lc, B = w.L, w.n_layers, w.B
    C_, H, Wd = w.dims
    rows = np.array([0, 1, 2, 127, 128, 255])          # samples from several batch blocks

    net = mbd.Net(mixed_layers(w), B, 4, 4, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 0)
    for i in range(L):
        bias = None if i < Lc else torch.from_numpy(inp.bs[i]).cuda()
        net.set_weights(i, to_dev(inp.Ws[i], True), bias)
    X = to_dev(inp.X, True)
    labels = torch.from_numpy(inp.labels).cuda()
    net.forward(X, labels)

    layers = [O.Conv3x3(inp.Ws[i].astype(np.float64)) for i in range(Lc)]
    layers += [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64)) for i in range(Lc, L)]
    o = O.train_step(layers, inp.X[rows].astype(np.float64), inp.labels[rows], "softmax_ce", w.eta, store=bf16_store)

    def dev_layout(a, i):
        if i < Lc:
            return a if a.ndim == 4 else np.ascontiguousarray(a.T).reshape(len(rows), C_, H, Wd)
        return a.T

    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_ACT, i)[rows])
        ref = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        assert rel_fro(got, dev_layout(ref, i)) < 1e-2, f"Y[{i}]"
    assert rel_fro(to_np(net.get_tensor(mbd.T_LOSS)[rows]), o["per_sample"]) < 1e-2

    # ReLU decisions of the sampled images forced to the oracle's stored activations, then back-propagate
    for i in range(L - 1):
        act = net.get_tensor(mbd.T_ACT, i)
        act[rows] = to_dev(np.ascontiguousarray(dev_layout(o["Xs"][i + 1], i), np.float32), True)
        net.set_tensor(mbd.T_ACT, i, act)
    net.backward(0.0)
    net.poll()
    dY = [net.get_tensor(mbd.T_DY, i) for i in range(L)]
    for i in range(L):
        assert rel_fro(to_np(dY[i][rows]), dev_layout(o["dYs"][i], i)) < 1e-2, f"dY[{i}]"

    # sums over the whole batch, from the device's own stored operands
    acts = [X] + [net.get_tensor(mbd.T_ACT, i) for i in range(L - 1)]
    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_DW, i))
        if i < Lc:
            ref = O.conv3x3_dK(to_np(dY[i]), to_np(acts[i]))
        else:
            x_in = to_np(acts[i]).reshape(B, -1)                     # NCHW order for the first FC layer
            ref = O.fc_dW(to_np(dY[i]).T, x_in.T)
        assert rel_fro(got, ref) < 1e-2, f"dW[{i}]"
        if i >= Lc:
            assert rel_fro(to_np(net.get_tensor(mbd.T_DB, i)), to_np(dY[i]).sum(axis=0)) < 1e-2, f"db[{i}]"
    net.close()
