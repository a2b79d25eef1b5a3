"""The largest workload (8 layers of 8192 x 8192, batch 8192) at FULL size, in the launch
configuration of the benchmark: the oracle cannot run the whole step in seconds, so it computes
what can be computed sample by sample -- the step is independent per sample except for the sum
over the batch in dW -- and the paper's own block structure supplies the rest: with a 1 x 64 grid
and every partial materialised, partial c of dW_1 is the sum over the 128 samples of batch block
c (Appendix A.2), which the oracle forms from exactly those samples."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import bf16_store, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu


def test_cfg5_sampled_columns_and_one_batch_block():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.WORKLOADS["cfg5"]
    inp = I.make_inputs(w, seed=0)
    L, B, d = 8, w.B, 8192
    P_c, block = 64, 5                       # batch block 5 = samples 640..767
    rows = np.arange(block * (B // P_c), (block + 1) * (B // P_c))

    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), B, 1, P_c, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 64)
    for i in range(L):
        net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    X = to_dev(inp.X, True)
    labels = torch.from_numpy(inp.labels).cuda()
    net.forward(X, labels)

    # oracle on the 128 samples of the block (fp64, stored activations rounded like the device's)
    layers = [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64)) for i in range(L)]
    o = O.train_step(layers, inp.X[rows].astype(np.float64).T, inp.labels[rows], "softmax_ce", w.eta, store=bf16_store)

    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_ACT, i)[rows])
        ref = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        assert rel_fro(got, ref.T) < 1e-2, f"Y[{i}]"
    assert rel_fro(to_np(net.get_tensor(mbd.T_LOSS)[rows]), o["per_sample"]) < 1e-2

    # force the ReLU decisions of those samples to the oracle's stored activations, then back-propagate
    for i in range(L - 1):
        act = net.get_tensor(mbd.T_ACT, i)
        act[rows] = to_dev(np.ascontiguousarray(o["Xs"][i + 1].T, np.float32), True)
        net.set_tensor(mbd.T_ACT, i, act)
    net.backward(0.0)
    net.poll()
    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_DY, i)[rows])
        assert rel_fro(got, o["dYs"][i].T) < 1e-2, f"dY[{i}]"

    # the last reduction executed was dW_1: its 64 partials are still in the workspace
    n1 = d * d
    parts = net.get_tensor(mbd.T_PARTIALS, 0, numel=P_c * n1).view(P_c, d, d)
    assert rel_fro(to_np(parts[block]), o["dWs"][0]) < 1e-2           # oracle's dW over exactly this block
    dW = net.get_tensor(mbd.T_DW, 0)
    ref_sum = parts.double().sum(dim=0)
    assert float((dW.double() - ref_sum).norm() / ref_sum.norm()) < 1e-6   # reduction = sum of the partials
    net.close()
