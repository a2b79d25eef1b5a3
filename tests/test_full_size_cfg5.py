"""The largest workload (8 layers of 8192 x 8192, batch 8192) at FULL size, on every grid the
workload lists and in the launch configuration the benchmark times (16 x 16 with two partial
sums per reduction, update fused into the tail of the reduction).

The oracle cannot run the whole step in seconds, so it computes what can be computed sample by
sample -- the step is independent per sample except for the sums over the batch in dW and db:
  * forward outputs, per-sample loss and the back-propagated gradients dY_i of the 128 samples of
    one batch block, from the oracle's own step on exactly those samples (ReLU decisions of those
    samples forced to the oracle's stored activations, as in the other parity tests);
  * the sums over the batch, on sampled rows of W_i with the full K = 8192 range: the oracle's
    product dY_i X_i^T and its update (Eq. 1), fed with the operands the device itself stored
    (dY_i and X_i as bf16), compared with the step the device applied, W_new - W_0, at a
    learning rate that makes the step as large as the weights; the same for the biases;
  * the paper's own block structure for one materialised partial: with a 1 x 64 grid and every
    partial kept, partial c of dW_1 is the sum over the 128 samples of batch block c
    (Appendix A.2), which the oracle forms from exactly those samples.
"""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import bf16_store, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu

L, D, B = 8, 8192, 8192
BLOCK = 5                                    # batch block 5 of 64 = samples 640..767
ROWS = np.arange(BLOCK * 128, (BLOCK + 1) * 128)
# rows of W_i whose update is checked with full-K products: first and last rows of tiles of every height in
# use (128, 256, 512), a few in the middle, the last row
W_ROWS = np.array([0, 1, 127, 128, 255, 256, 511, 512, 1000, 2047, 2048, 4095, 4096, 4097, 5555, 6143, 6144, 7679, 7680,
                   8063, 8064, 8190, 8191])
CHECK_LAYERS = (0, 4, 7)                     # first (no backward-data below it), a middle one, the classifier


@pytest.fixture(scope="module")
def cfg5():
    import torch
    from oracle import mbd_oracle as O
    w = I.WORKLOADS["cfg5"]
    assert w.dims == (D,) * (L + 1) and w.B == B
    inp = I.make_inputs(w, seed=0)
    layers = [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64)) for i in range(L)]
    o = O.train_step(layers, inp.X[ROWS].astype(np.float64).T, inp.labels[ROWS], "softmax_ce", w.eta, store=bf16_store)
    dev = dict(W=[to_dev(inp.Ws[i], True) for i in range(L)], b=[torch.from_numpy(inp.bs[i]).cuda() for i in range(L)],
               X=to_dev(inp.X, True), labels=torch.from_numpy(inp.labels).cuda())
    return dict(w=w, inp=inp, o=o, dev=dev, eta=None)


def make_net(c, grid, mp):
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers(c["w"].dims, bias=True), B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
    for i in range(L):
        net.set_weights(i, c["dev"]["W"][i], c["dev"]["b"][i])
    return net


def forward_and_force(c, net):
    """Forward pass; the block's outputs against the oracle; then the ReLU decisions of the block's samples
    are set to the oracle's stored activations."""
    from paper_1712_04432_b200 import mbd
    o = c["o"]
    net.forward(c["dev"]["X"], c["dev"]["labels"])
    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_ACT, i)[ROWS])
        ref = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        assert rel_fro(got, ref.T) < 1e-2, f"Y[{i}]"
    assert rel_fro(to_np(net.get_tensor(mbd.T_LOSS)[ROWS]), o["per_sample"]) < 1e-2
    for i in range(L - 1):
        act = net.get_tensor(mbd.T_ACT, i)
        act[ROWS] = to_dev(np.ascontiguousarray(o["Xs"][i + 1].T, np.float32), True)
        net.set_tensor(mbd.T_ACT, i, act)


def layer_input(c, net, i):
    from paper_1712_04432_b200 import mbd
    return c["dev"]["X"] if i == 0 else net.get_tensor(mbd.T_ACT, i - 1)


def sized_eta(c):
    """A learning rate at which Eq. 1 moves every W_i by at least its own norm; the gradient norms come from an
    un-fused pass of the device (any eta would do for correctness: this one makes the comparison sharp)."""
    if c["eta"] is None:
        from paper_1712_04432_b200 import mbd
        net = make_net(c, (1, 1), 1)
        forward_and_force(c, net)
        net.backward(0.0)
        net.poll()
        ratio = max(float(c["dev"]["W"][i].float().norm() / net.get_tensor(mbd.T_DW, i).norm()) for i in range(L))
        c["eta"] = B * ratio
        # while the gradients are materialised: sampled rows of dW_i of a middle layer against the oracle's
        # product over the whole batch, from the device's stored operands
        from oracle import mbd_oracle as O
        i = 4
        dY = to_np(net.get_tensor(mbd.T_DY, i)[:, W_ROWS.tolist()])
        Xi = to_np(layer_input(c, net, i))
        ref = O.fc_dW(dY.T, Xi.T)
        assert rel_fro(to_np(net.get_tensor(mbd.T_DW, i)[W_ROWS.tolist()]), ref) < 1e-4, "dW[4], sampled rows, full K"
        net.close()
    return c["eta"]


@pytest.mark.parametrize("grid,mp,bench_plan,any_s", [((16, 16), 2, True, False), ((1, 1), 1, False, False), ((64, 4), 2, False, False),
                                                      ((4, 64), 2, False, False),
                                                      ((16, 16), 4, False, False),     # four planes and the reduction kernel
                                                      ((16, 16), 4, False, True)])     # four pieces as a running sum (tuning knob)
def test_cfg5_listed_grids_fused_step(monkeypatch, cfg5, grid, mp, bench_plan, any_s):
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    c, o = cfg5, cfg5["o"]
    eta = sized_eta(c)
    if any_s:
        monkeypatch.setenv("MBD_FIX_ANY_S", "1")
    net = make_net(c, grid, mp)
    if mp == 4:
        p = net.plan(3, 2)
        assert (p["k_pieces"], p["running_sum"]) == (4, 1 if any_s else 0), p
    if bench_plan:
        # what `bench.py` launches by default: unsplit forward products on 512 x 256 CTA-pair tiles, both backward
        # products cut in two pieces on 256 x 256 CTA-pair tiles, the pieces added as a running sum in the epilogue
        for i in range(L):
            p = net.plan(i, 0)
            assert (p["tile_m"], p["tile_n"], p["cta_pair"], p["k_pieces"], p["ctas"]) == (512, 256, 1, 1, 148)
            for product in ((1, 2) if i > 0 else (2,)):
                p = net.plan(i, product)
                assert (p["tile_m"], p["tile_n"], p["cta_pair"], p["k_pieces"], p["running_sum"]) == (256, 256, 1, 2, 1)
    forward_and_force(c, net)
    X_in = {i: layer_input(c, net, i).clone() for i in CHECK_LAYERS}
    net.backward(eta)                                    # fused update
    net.poll()
    for i in range(L):
        got = to_np(net.get_tensor(mbd.T_DY, i)[ROWS])
        assert rel_fro(got, o["dYs"][i].T) < 1e-2, f"dY[{i}]"
    for i in CHECK_LAYERS:
        dY_full = net.get_tensor(mbd.T_DY, i)
        W0 = c["inp"].Ws[i][W_ROWS].astype(np.float64)
        dW_rows = O.fc_dW(to_np(dY_full[:, W_ROWS.tolist()]).T, to_np(X_in[i]).T)          # full K = 8192, fp64
        want = O.sgd(W0, dW_rows, eta, B)
        got = to_np(net.get_weights(i)[W_ROWS.tolist()])
        step = np.linalg.norm(want - W0)
        assert step > 0.5 * np.linalg.norm(W0)                                   # the step is as large as the weights
        # the device's operands are the oracle's inputs here: what remains is fp32 accumulation and the one bf16
        # rounding of W_new (1.1e-3 of ||W_new||)
        assert np.linalg.norm((got - W0) - (want - W0)) < 5e-3 * step, f"W_new[{i}] - W_0[{i}]"
        db = to_np(dY_full).sum(axis=0)
        b_new = to_np(net.get_weights(i, with_bias=True)[1])
        assert rel_fro(b_new, O.sgd(c["inp"].bs[i].astype(np.float64), db, eta, B)) < 1e-4, f"b_new[{i}]"
    net.close()


def test_cfg5_one_materialised_batch_block_partial(cfg5):
    from paper_1712_04432_b200 import mbd
    c, o = cfg5, cfg5["o"]
    P_c = 64
    net = make_net(c, (1, P_c), 64)
    forward_and_force(c, net)
    net.backward(0.0)
    net.poll()
    # the last reduction executed was dW_1: its 64 partials are still in the workspace
    n1 = D * D
    parts = net.get_tensor(mbd.T_PARTIALS, 0, numel=P_c * n1).view(P_c, D, D)
    assert rel_fro(to_np(parts[BLOCK]), o["dWs"][0]) < 1e-2          # oracle's dW over exactly this block
    dW = net.get_tensor(mbd.T_DW, 0)
    ref_sum = parts.double().sum(dim=0)
    assert float((dW.double() - ref_sum).norm() / ref_sum.norm()) < 1e-6   # reduction = sum of the partials
    net.close()
