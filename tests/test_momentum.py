"""Heavy-ball momentum (mbd_enable_momentum): v <- mu v + dW / B, w <- w - eta v in place of Eq. 1 (Section 2: SGD
stands for any first-order method).  Checked (a) as a whole trajectory in the fp32 mode against the oracle's own
steps, (b) step by step on bf16 networks from the gradient the device itself materialised -- the update is a
function of (w, v, dW) alone, and the gradient's parity is the business of the other tests -- with and without
fp32 master weights, fused, un-fused and through the captured step, (c) on an integrated convolution + fully
connected stack."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import mixed_layers, rel_fro, to_dev, to_np

pytestmark = pytest.mark.gpu

MU = 0.9


def test_fp32_trajectory_follows_the_oracle():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((96, 64, 48, 10), 32, "fp32")
    inp = I.make_inputs(w, seed=5)
    eta, L = 0.05, len(inp.Ws)
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, 2, 2, mbd.F32, mbd.LOSS_SOFTMAX_CE, 2)
    net.enable_momentum(MU)
    for i in range(L):
        net.set_weights(i, torch.from_numpy(inp.Ws[i]).cuda(), torch.from_numpy(inp.bs[i]).cuda())
    X, labels = torch.from_numpy(inp.X).cuda(), torch.from_numpy(inp.labels).cuda()
    Ws = [a.astype(np.float64) for a in inp.Ws]
    bs = [a.astype(np.float64) for a in inp.bs]
    Vs, Vb = [np.zeros_like(a) for a in Ws], [np.zeros_like(a) for a in bs]
    for step in range(5):
        layers = [O.FC(Ws[i], bs[i], relu=(i < L - 1)) for i in range(L)]
        o = O.train_step(layers, inp.X.astype(np.float64).T, inp.labels, "softmax_ce", eta)
        for i in range(L):
            Ws[i], Vs[i] = O.sgd_momentum(Ws[i], Vs[i], o["dWs"][i], eta, w.B, MU)
            bs[i], Vb[i] = O.sgd_momentum(bs[i], Vb[i], o["dbs"][i], eta, w.B, MU)
        if step % 2 == 0:
            net.forward(X, labels); net.backward(eta)                       # update inside the backward call
        else:
            net.forward(X, labels); net.backward(0.0); net.sgd_step(eta)    # update as a call of its own
        net.poll()
        for i in range(L):
            Wg, bg = net.get_weights(i, with_bias=True)
            assert rel_fro(to_np(Wg), Ws[i]) < 1e-5 and rel_fro(to_np(bg), bs[i]) < 1e-5, (step, i)
            assert rel_fro(to_np(net.get_tensor(mbd.T_VELOCITY, i)), Vs[i]) < 1e-5, (step, i)
            assert rel_fro(to_np(net.get_tensor(mbd.T_VELOCITY_BIAS, i)), Vb[i]) < 1e-5, (step, i)
    # after five steps the velocity is no longer the last gradient: the history is in it
    assert rel_fro(Vs[0], o["dWs"][0] / w.B) > 0.5
    net.close()


def _bf16_net(w, inp, master, grid, mp):
    import torch
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
    for i in range(len(inp.Ws)):
        net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    if master:
        net.enable_master_weights()
    net.enable_momentum(MU)
    return net


@pytest.mark.parametrize("master", [True, False])
@pytest.mark.parametrize("grid,mp", [((1, 1), 0), ((2, 4), 2), ((1, 2), 2)])
def test_bf16_update_from_the_devices_own_gradient(master, grid, mp):
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 72, 40, 24), 32, "bf16")
    inp = I.make_inputs(w, seed=81)
    L = len(inp.Ws)
    X, labels = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    # a learning rate at which a step moves the weights by about a tenth of their norm: far above bf16 rounding
    probe = _bf16_net(w, inp, False, (1, 1), 0)
    probe.forward(X, labels); probe.backward(0.0)
    eta = 0.1 * w.B * min(float(np.linalg.norm(inp.Ws[i]) / probe.get_tensor(mbd.T_DW, i).norm()) for i in range(L))
    probe.sgd_step(0.0); probe.close()
    nets = {m: _bf16_net(w, inp, master, grid, mp) for m in ("unfused", "fused", "graph")}
    for step in range(3):
        u = nets["unfused"]
        W_old = [to_np(u.get_tensor(mbd.T_MASTER, i)) if master else to_np(u.get_weights(i)) for i in range(L)]
        b_old = [to_np(u.get_weights(i, with_bias=True)[1]) for i in range(L)]
        V_old = [to_np(u.get_tensor(mbd.T_VELOCITY, i)) for i in range(L)]
        Vb_old = [to_np(u.get_tensor(mbd.T_VELOCITY_BIAS, i)) for i in range(L)]
        u.forward(X, labels); u.backward(0.0)
        dW = [to_np(u.get_tensor(mbd.T_DW, i)) for i in range(L)]
        db = [to_np(u.get_tensor(mbd.T_DB, i)) for i in range(L)]
        u.sgd_step(eta)
        nets["fused"].forward(X, labels); nets["fused"].backward(eta)
        nets["graph"].train_step(X, labels, eta)
        for n in nets.values():
            n.poll()
        for i in range(L):
            W_want, V_want = O.sgd_momentum(W_old[i], V_old[i], dW[i], eta, w.B, MU)
            b_want, Vb_want = O.sgd_momentum(b_old[i], Vb_old[i], db[i], eta, w.B, MU)
            assert rel_fro(to_np(u.get_tensor(mbd.T_VELOCITY, i)), V_want) < 1e-6, (step, i)
            assert rel_fro(to_np(u.get_tensor(mbd.T_VELOCITY_BIAS, i)), Vb_want) < 1e-6, (step, i)
            assert rel_fro(to_np(u.get_weights(i, with_bias=True)[1]), b_want) < 1e-6, (step, i)
            Wb = u.get_weights(i)
            if master:
                Wm = u.get_tensor(mbd.T_MASTER, i)
                assert rel_fro(to_np(Wm), W_want) < 1e-6, (step, i)
                assert torch.equal(Wm.to(torch.bfloat16), Wb)               # working copy = rounded master
            else:
                # one rounding of the new weight to bf16: the applied step against the oracle's step
                assert rel_fro(to_np(Wb) - W_old[i], W_want - W_old[i]) < 3e-2, (step, i)
                assert rel_fro(to_np(Wb), W_want) < 3e-3, (step, i)
            if step > 0:
                assert rel_fro(V_want, dW[i] / w.B) > 0.3, (step, i)        # the velocity carries the earlier steps
            # the update inside the backward call and inside the captured step: the same kernel, the same bits
            for other in ("fused", "graph"):
                assert torch.equal(nets[other].get_weights(i), Wb), (step, i, other)
                assert torch.equal(nets[other].get_tensor(mbd.T_VELOCITY, i), u.get_tensor(mbd.T_VELOCITY, i)), (step, i, other)
    for n in nets.values():
        n.close()


def test_momentum_on_an_integrated_stack():
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    w = I.mixed_workload(64, 8, 40, 2, (128, 16), 6, name="mixed_momentum", ksizes=(3, 1))
    inp = I.make_inputs(w, seed=83)
    X, labels = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    eta = 0.05

    def make():
        net = mbd.Net(mixed_layers(w), w.B, 2, 3, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 4)
        net.enable_master_weights()
        net.enable_momentum(MU)
        for i in range(w.L):
            bias = None if i < w.n_layers else torch.from_numpy(inp.bs[i]).cuda()
            net.set_weights(i, to_dev(inp.Ws[i], True), bias)
        return net
    a, b = make(), make()
    for step in range(3):
        W_old = [to_np(a.get_tensor(mbd.T_MASTER, i)) for i in range(w.L)]
        V_old = [to_np(a.get_tensor(mbd.T_VELOCITY, i)) for i in range(w.L)]
        a.forward(X, labels); a.backward(0.0)
        dW = [to_np(a.get_tensor(mbd.T_DW, i)) for i in range(w.L)]
        a.sgd_step(eta)
        b.forward(X, labels); b.backward(eta)
        a.poll(); b.poll()
        for i in range(w.L):
            W_want, V_want = O.sgd_momentum(W_old[i], V_old[i], dW[i], eta, w.B, MU)
            assert rel_fro(to_np(a.get_tensor(mbd.T_VELOCITY, i)), V_want) < 1e-6, (step, i)
            assert rel_fro(to_np(a.get_tensor(mbd.T_MASTER, i)), W_want) < 1e-6, (step, i)
            assert torch.equal(a.get_tensor(mbd.T_MASTER, i), b.get_tensor(mbd.T_MASTER, i)), (step, i)
            assert torch.equal(a.get_weights(i), b.get_weights(i)), (step, i)
            assert torch.equal(a.get_tensor(mbd.T_MASTER, i).to(torch.bfloat16), a.get_weights(i)), (step, i)
    a.close(); b.close()


def test_momentum_arguments():
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers((64, 32, 16)), 8, 1, 1, mbd.F32, mbd.LOSS_SOFTMAX_CE, 0)
    for bad in (-0.1, 1.0, float("nan")):
        with pytest.raises(mbd.MbdError) as e:
            net.enable_momentum(bad)
        assert e.value.status == mbd.E_INVALID
    with pytest.raises(mbd.MbdError):
        net.get_tensor(mbd.T_VELOCITY, 0)              # no velocity before momentum is enabled
    net.enable_momentum(0.5)
    assert float(net.get_tensor(mbd.T_VELOCITY, 0).abs().max()) == 0.0
    net.close()
