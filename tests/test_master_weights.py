"""fp32 master weights (mbd_enable_master_weights): Eq. 1 applied to an fp32 copy of every weight, the bf16
weights the contractions read being the rounded master.  Checked against the fp64 oracle's updated weights,
which a bf16-only update can only match to bf16 rounding."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import (bf16_store, like_device, mixed_layers, oracle_fc_step, oracle_hidden_acts, oracle_mixed_acts,
                           oracle_mixed_step, rel_fro, to_dev, to_np)

pytestmark = pytest.mark.gpu


def fc_net(w, inp, master, grid=(1, 1), mp=0):
    import torch
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
    if master == "before":
        net.enable_master_weights()
    for i in range(len(inp.Ws)):
        net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    if master == "after":
        net.enable_master_weights()
    return net


@pytest.mark.parametrize("when", ["before", "after"])
@pytest.mark.parametrize("mode", ["fused", "unfused", "graph"])
@pytest.mark.parametrize("grid,mp", [((1, 1), 0), ((2, 4), 4)])
def test_master_update_matches_the_oracle_beyond_bf16(when, mode, grid, mp):
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 72, 40, 24), 32, "bf16")
    w.eta = 0.05
    inp = I.make_inputs(w, seed=81)
    o = oracle_fc_step(w, inp)
    L = len(inp.Ws)
    X, labels = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    errs = {}
    for master in (when, None):
        net = fc_net(w, inp, master, grid, mp)
        if mode == "graph":
            net.train_step(X, labels, w.eta)
        else:
            net.forward(X, labels)
            for i in range(L - 1):      # ReLU decisions on the oracle's stored activations, as in the parity tests
                net.set_tensor(mbd.T_ACT, i, to_dev(oracle_hidden_acts(o)[i], True))
            if mode == "fused":
                net.backward(w.eta)
            else:
                net.backward(0.0)
                net.sgd_step(w.eta)
        net.poll()
        Wb = [net.get_weights(i) for i in range(L)]
        if master:
            Wm = [net.get_tensor(mbd.T_MASTER, i) for i in range(L)]
            for i in range(L):
                assert torch.equal(Wm[i].to(torch.bfloat16), Wb[i])              # working copy = rounded master
            errs["master"] = max(rel_fro(to_np(Wm[i]), o["new_W"][i]) for i in range(L))
        else:
            errs["bf16"] = max(rel_fro(to_np(Wb[i]), o["new_W"][i]) for i in range(L))
        net.close()
    tol = 1e-3 if mode == "graph" else 1e-4        # the graph step takes its own ReLU decisions
    assert errs["master"] < tol, errs
    if mode != "graph":
        assert errs["bf16"] > 5 * errs["master"], errs


def test_small_updates_accumulate_in_the_master():
    """Steps far below half a bf16 ulp: bf16-only weights stay where they are, the master moves by the sum."""
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 72, 24), 16, "bf16")
    w.eta = 1e-5
    inp = I.make_inputs(w, seed=82)
    X, labels = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    steps = 6
    plain, mast = fc_net(w, inp, None), fc_net(w, inp, "after")
    plain.forward(X, labels); plain.backward(0.0)
    dW0 = [to_np(plain.get_tensor(mbd.T_DW, i)) for i in range(2)]
    plain.sgd_step(0.0)
    for _ in range(steps):
        for net in (plain, mast):
            net.forward(X, labels)
            net.backward(w.eta)
    plain.poll(); mast.poll()
    for i in range(2):
        W0 = inp.Ws[i].astype(np.float64)
        moved_plain = np.mean(to_np(plain.get_weights(i)) != W0)
        assert moved_plain < 0.02, moved_plain                                   # almost every update was rounded away
        delta = to_np(mast.get_tensor(mbd.T_MASTER, i)) - W0
        want = -steps * (w.eta / w.B) * dW0[i]
        assert rel_fro(delta, want) < 2e-2
    plain.close(); mast.close()


def test_master_weights_of_an_integrated_stack():
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.mixed_workload(64, 8, 40, 2, (128, 16), 6, name="mixed_master", ksizes=(3, 1))
    w.eta = 0.02
    inp = I.make_inputs(w, seed=83)
    o = oracle_mixed_step(w, inp)
    acts = oracle_mixed_acts(o, w)
    masters = []
    for fused in (True, False):
        net = mbd.Net(mixed_layers(w), w.B, 2, 3, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 4)
        net.enable_master_weights()
        for i in range(w.L):
            bias = None if i < w.n_layers else torch.from_numpy(inp.bs[i]).cuda()
            net.set_weights(i, to_dev(inp.Ws[i], True), bias)
        net.forward(to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda())
        for i in range(w.L - 1):
            net.set_tensor(mbd.T_ACT, i, to_dev(acts[i], True))
        if fused:
            net.backward(w.eta)
        else:
            net.backward(0.0)
            net.sgd_step(w.eta)
        net.poll()
        m = [net.get_tensor(mbd.T_MASTER, i) for i in range(w.L)]
        for i in range(w.L):
            got = to_np(m[i])
            W0 = inp.Ws[i].astype(np.float64)
            # the master holds the update itself to the gradient's tolerance (a bf16 weight cannot: its
            # rounding error is of the size of this update), hence the weights far beyond bf16 precision
            assert rel_fro(got - W0, like_device(o["new_W"][i], got) - W0) < 1e-2, i
            assert rel_fro(got, like_device(o["new_W"][i], got)) < 5e-4, i
            assert torch.equal(m[i].to(torch.bfloat16), net.get_weights(i))
        masters.append(m)
        net.close()
    for a, b in zip(*masters):
        assert torch.equal(a, b)                   # fused and un-fused updates are the same arithmetic


def test_master_weights_need_a_bf16_network():
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers((64, 32, 16)), 8, 1, 1, mbd.F32, mbd.LOSS_SOFTMAX_CE, 0)
    with pytest.raises(mbd.MbdError) as e:
        net.enable_master_weights()
    assert e.value.status == mbd.E_UNSUPPORTED
    net.close()
