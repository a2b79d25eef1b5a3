"""Edge cases on the GPU: call-order errors, smallest batch, one-layer nets, a batch block per
sample, bounded-wait time-out reporting, kernel-launch accounting."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import compare_fc_step, gpu_fc_step, oracle_fc_step, oracle_hidden_acts, to_dev

pytestmark = pytest.mark.gpu


def test_call_order_is_enforced():
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((64, 32, 16), 8, "bf16")
    inp = I.make_inputs(w, seed=1)
    net = mbd.Net(mbd.fc_layers(w.dims), w.B)
    with pytest.raises(mbd.MbdError) as e:
        net.backward(0.0)                                # no forward yet
    assert e.value.status == mbd.E_STATE
    X, lab = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    net.forward(X, lab)
    with pytest.raises(mbd.MbdError) as e:
        net.sgd_step(0.1)                                # no backward yet
    assert e.value.status == mbd.E_STATE
    net.backward(0.1)                                    # fused update
    with pytest.raises(mbd.MbdError) as e:
        net.sgd_step(0.1)                                # already applied
    assert e.value.status == mbd.E_STATE
    with pytest.raises(mbd.MbdError):
        net.backward(0.0)                                # needs a new forward
    net.poll()
    net.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_smallest_batch_and_one_block_per_sample(dtype):
    w = I.fc_workload((72, 40, 24), 8, dtype)
    inp = I.make_inputs(w, seed=2)
    o = oracle_fc_step(w, inp)
    tol = 1e-2 if dtype == "bf16" else 1e-5
    for grid in [(1, 8), (8, 1), (8, 8)]:                # P_c = B: one sample per process
        g = gpu_fc_step(w, inp, grid, max_partials=64, force_acts=oracle_hidden_acts(o))
        compare_fc_step(g, o, tol)
    w1 = I.fc_workload((72, 24), 1, dtype)               # a single sample, a single layer
    inp1 = I.make_inputs(w1, seed=3)
    compare_fc_step(gpu_fc_step(w1, inp1), oracle_fc_step(w1, inp1), tol)


def test_more_row_blocks_than_k_blocks():
    # P_r = 16 row blocks over d = 72 (2 k-blocks of 64): the tensor-core path caps the number of
    # partial sums at the number of 64-wide k-blocks; the result is unchanged
    w = I.fc_workload((136, 72, 72, 16), 24, "bf16")
    inp = I.make_inputs(w, seed=4)
    o = oracle_fc_step(w, inp)
    g = gpu_fc_step(w, inp, (16, 3), max_partials=64, force_acts=oracle_hidden_acts(o))
    compare_fc_step(g, o, 1e-2)


def test_bounded_wait_reports_timeout_and_context_survives():
    import torch
    from paper_1712_04432_b200 import mbd
    assert mbd.selftest_timeout(30) == mbd.E_TIMEOUT
    a = torch.ones((128, 64), dtype=torch.bfloat16, device="cuda")
    D = mbd.gemm_bf16(0, a, a)                            # the device still works
    assert float(D[0, 0]) == 64.0


def test_launch_accounting_and_profile():
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 136, 136), 128, "bf16")       # K = 136 and K = B = 128: two or more 64-wide k-blocks
    inp = I.make_inputs(w, seed=5)
    net = mbd.Net(mbd.fc_layers(w.dims), w.B, 2, 2, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 2)
    for i in range(2):
        net.set_weights(i, to_dev(inp.Ws[i], True))
    X, lab = to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda()
    J = torch.zeros(1, device="cuda")
    net.profile_enable(True)
    n0 = net.launch_count
    net.forward(X, lab, J)
    net.backward(0.01)
    # forward: 2 GEMMs + softmax + loss sum; backward: 2 x colsum (two stages) + dX GEMM + its reduction
    # + 2 x (dW GEMM + reduction with the fused update)
    assert net.launch_count - n0 == 4 + 4 + 2 + 4
    prof = net.profile_read()
    assert prof["gemm_fwd"]["launches"] == 2 and prof["gemm_bwd_weight"]["launches"] == 2
    assert prof["reduce_partials"]["launches"] == 3
    assert prof["gemm_fwd"]["work"] == 2.0 * 128 * (136 * 136 + 136 * 136)
    net.close()


def test_train_step_from_host_buffers():
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 72, 16), 16, "bf16")
    inp = I.make_inputs(w, seed=6)
    o = oracle_fc_step(w, inp)
    net = mbd.Net(mbd.fc_layers(w.dims), w.B)
    for i in range(2):
        net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    Xh = to_dev(inp.X, True).cpu().pin_memory()
    lh = torch.from_numpy(inp.labels).pin_memory()
    J = net.train_step_host(Xh, lh, w.eta)
    assert abs(J - o["J"]) < 1e-2 * abs(o["J"])
    for i in range(2):
        got = net.get_weights(i).float().cpu().numpy()
        assert np.linalg.norm(got - o["new_W"][i]) / np.linalg.norm(o["new_W"][i]) < 1e-2
    net.close()


def test_pipelined_host_steps_equal_synchronous_ones():
    # two steps in flight (copy of batch k+1 under the compute of batch k): same losses and
    # weights, bit for bit, as the synchronous entry point on the same sequence of batches
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((264, 136, 24), 40, "bf16")
    batches = [I.make_inputs(w, seed=20 + k) for k in range(5)]
    Xs = [to_dev(b.X, True).cpu().pin_memory() for b in batches]
    ls = [torch.from_numpy(b.labels).pin_memory() for b in batches]

    def fresh():
        net = mbd.Net(mbd.fc_layers(w.dims), w.B, 2, 2, stream=torch.cuda.Stream())
        for i in range(2):
            net.set_weights(i, to_dev(batches[0].Ws[i], True), torch.from_numpy(batches[0].bs[i]).cuda())
        return net

    net = fresh()
    J_sync = [net.train_step_host(Xs[k], ls[k], 0.05) for k in range(5)]
    W_sync = [net.get_weights(i).clone() for i in range(2)]
    torch.cuda.synchronize()
    net.close()

    net = fresh()
    with pytest.raises(mbd.MbdError) as e:
        net.train_step_host_end()                        # nothing in flight
    assert e.value.status == mbd.E_STATE
    J_pipe = []
    net.train_step_host_begin(Xs[0], ls[0], 0.05)
    for k in range(1, 5):
        net.train_step_host_begin(Xs[k], ls[k], 0.05)
        if k == 1:
            with pytest.raises(mbd.MbdError) as e:
                net.train_step_host_begin(Xs[k], ls[k], 0.05)    # a third step in flight
            assert e.value.status == mbd.E_STATE
        J_pipe.append(net.train_step_host_end())
    J_pipe.append(net.train_step_host_end())
    torch.cuda.synchronize()
    assert J_pipe == J_sync
    for i in range(2):
        assert torch.equal(net.get_weights(i), W_sync[i])
    assert len(set(J_sync)) == 5                         # the batches really differed
    net.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_graph_replayed_step_equals_direct_launches(dtype):
    import torch
    from paper_1712_04432_b200 import mbd
    w = I.fc_workload((136, 136, 72), 128, dtype)
    inp = I.make_inputs(w, seed=7)
    bf = dtype == "bf16"

    def make():
        net = mbd.Net(mbd.fc_layers(w.dims), w.B, 2, 2, mbd.BF16 if bf else mbd.F32, mbd.LOSS_SOFTMAX_CE, 2)
        for i in range(2):
            net.set_weights(i, to_dev(inp.Ws[i], bf), torch.from_numpy(inp.bs[i]).cuda())
        return net

    X, lab = to_dev(inp.X, bf), torch.from_numpy(inp.labels).cuda()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()                           # the default stream cannot be captured
    with torch.cuda.stream(side):
        a, b = make(), make()
        Ja, Jb = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
        for _ in range(3):                               # three steps: capture once, replay twice
            a.train_step(X, lab, w.eta, Ja)
            b.forward(X, lab, Jb)
            b.backward(w.eta)
        a.poll(); b.poll()
    assert a.launch_count == b.launch_count
    assert torch.equal(Ja, Jb)
    for i in range(2):
        assert torch.equal(a.get_weights(i), b.get_weights(i))
    a.close(); b.close()


def test_wide_classifier_uses_the_streaming_softmax():
    # more than 8192 classes: the row no longer fits the register-resident kernel
    w = I.fc_workload((72, 8264), 24, "bf16")
    inp = I.make_inputs(w, seed=8)
    compare_fc_step(gpu_fc_step(w, inp), oracle_fc_step(w, inp), 1e-2)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_layers_without_bias_and_without_relu(dtype):
    # a linear hidden layer (no ReLU, no bias): the mask and bias paths are switched off per layer
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    from tests.helpers import bf16_store, rel_fro, to_np
    bf = dtype == "bf16"
    w = I.fc_workload((136, 72, 40, 24), 32, dtype)
    inp = I.make_inputs(w, seed=9)
    flags = [(1, 0), (0, 1), (1, 1)]                    # (relu, bias) per layer
    layers = [mbd.Layer(kind=mbd.FC, split=mbd.SPLIT_MODEL, relu=r, bias=b, d_in=w.dims[i], d_out=w.dims[i + 1])
              for i, (r, b) in enumerate(flags)]
    net = mbd.Net(layers, w.B, 2, 2, mbd.BF16 if bf else mbd.F32, mbd.LOSS_SOFTMAX_CE, 4)
    for i in range(3):
        net.set_weights(i, to_dev(inp.Ws[i], bf), torch.from_numpy(inp.bs[i]).cuda() if flags[i][1] else None)
    X, lab = to_dev(inp.X, bf), torch.from_numpy(inp.labels).cuda()
    net.forward(X, lab)
    net.backward(0.0)
    net.poll()
    ol = [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64) if flags[i][1] else None, relu=bool(flags[i][0]))
          for i in range(3)]
    o = O.train_step(ol, inp.X.astype(np.float64).T, inp.labels, "softmax_ce", w.eta, store=bf16_store if bf else None)
    tol = 1e-2 if bf else 1e-5                            # free-running bf16 step (no forced ReLU decisions)
    for i in range(3):
        assert rel_fro(to_np(net.get_tensor(mbd.T_DW, i)), o["dWs"][i]) < tol
        assert rel_fro(to_np(net.get_tensor(mbd.T_DY, i)), o["dYs"][i].T) < tol
    assert rel_fro(to_np(net.get_tensor(mbd.T_DB, 1)), o["dbs"][1]) < tol
    net.close()
