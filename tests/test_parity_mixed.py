"""Parity of the integrated step of Section 2.4 (domain-parallel 3x3 convolutions first,
model-parallel fully connected layers after them, one P_r x P_c grid for both, Eq. 9) with
the fp64 oracle, through the C ABI; and of convolution stacks whose batch is split as well."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import (compare_conv_step, compare_mixed_step, gpu_conv_step, gpu_mixed_step, oracle_conv_step,
                           oracle_mixed_acts, oracle_mixed_step, oracle_with_eta, rel_fro, update_sized_eta)

pytestmark = pytest.mark.gpu
TOL = 1e-2
TOL_FREE = 1e-2      # free-running (ReLU decisions on the device's own stored activations): measured 3.2e-3 at worst


@pytest.fixture(scope="module")
def small():
    # 2 convolutions on 8 x 40 images (one ragged 40-pixel segment), then 20480 -> 256 -> 24
    w = I.mixed_workload(64, 8, 40, 2, (256, 24), 6, name="mixed_small")
    inp = I.make_inputs(w, seed=31)
    return w, inp, oracle_mixed_step(w, inp)


@pytest.mark.parametrize("grid", [(1, 1), (2, 1), (1, 3), (2, 3), (4, 2), (8, 6)])
def test_small_all_grids(small, grid):
    w, inp, o = small
    g = gpu_mixed_step(w, inp, grid, force_acts=oracle_mixed_acts(o, w))
    compare_mixed_step(g, o, w, TOL)
    g = gpu_mixed_step(w, inp, grid)
    compare_mixed_step(g, o, w, TOL, tol_below_relu=TOL_FREE)


@pytest.mark.parametrize("grid,max_partials", [((1, 1), 1), ((2, 2), 4), ((4, 2), 2)])
def test_small_fused_update(small, grid, max_partials):
    # at a learning rate that moves every kernel / matrix by at least its own norm, so that the comparison of the
    # applied update (W_new - W_0 against the oracle's step) is sharp on bf16 weights
    w, inp, o = small
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    g = gpu_mixed_step(w, inp, grid, max_partials, fused=True, force_acts=oracle_mixed_acts(o, w), eta=eta)
    compare_mixed_step(g, o, w, TOL, fused=True, init=inp, require_sized=True)
    u = gpu_mixed_step(w, inp, grid, max_partials, fused=False, force_acts=oracle_mixed_acts(o, w), eta=eta)
    for i in range(w.L):                                   # fully connected layers: fused = un-fused bit for bit
        if i >= w.n_layers:
            assert np.array_equal(g["new_W"][i], u["new_W"][i]) and np.array_equal(g["new_b"][i], u["new_b"][i])


def test_blocked_oracle_agrees(small):
    w, inp, _ = small
    ob = oracle_mixed_step(w, inp, blocked_grid=(4, 3))
    g = gpu_mixed_step(w, inp, (4, 3), 4, force_acts=oracle_mixed_acts(ob, w))
    compare_mixed_step(g, ob, w, TOL)


def test_one_convolution_three_fc_layers_ragged():
    # 28 rows (strips of 7), 130 pixels per row (two forward segments), 5 samples; FC 232960 -> 64 -> 32 -> 16
    w = I.mixed_workload(64, 28, 130, 1, (64, 32, 16), 5, name="mixed_ragged")
    inp = I.make_inputs(w, seed=32)
    o = oracle_mixed_step(w, inp)
    for grid in [(1, 1), (4, 5)]:
        g = gpu_mixed_step(w, inp, grid, force_acts=oracle_mixed_acts(o, w))
        compare_mixed_step(g, o, w, TOL)


def test_unequal_strips_under_fully_connected_layers():
    # 10 rows on 3 and 4 strips (heights 4, 3, 3 and 3, 2, 3, 2), batch split as well; then 25600 -> 64 -> 16
    w = I.mixed_workload(64, 10, 40, 2, (64, 16), 6, name="mixed_unequal")
    inp = I.make_inputs(w, seed=34)
    o = oracle_mixed_step(w, inp)
    for grid in [(3, 2), (4, 3)]:
        g = gpu_mixed_step(w, inp, grid, 4, force_acts=oracle_mixed_acts(o, w))
        compare_mixed_step(g, o, w, TOL)
        g = gpu_mixed_step(w, inp, grid, 4, fused=True, force_acts=oracle_mixed_acts(o, w))
        compare_mixed_step(g, o, w, TOL, fused=True)


@pytest.mark.parametrize("grid", [(2, 3), (3, 2), (6, 1)])
def test_batch_parallel_convolutions_under_model_parallel_layers(small, grid):
    """Section 3's improved case: the convolutions forced onto a 1 x P grid (pure batch parallelism: no strips, one
    weight-gradient partial per process), the fully connected layers on P_r x P_c.  Against the oracle that forms
    exactly those blocks; 6 samples on 6 processes is the limit (one sample per process), 12 processes are refused."""
    from paper_1712_04432_b200 import mbd
    w, inp, _ = small
    ob = oracle_mixed_step(w, inp, blocked_grid=grid, conv_split="batch")
    eta = update_sized_eta(ob, inp.Ws, w.B)
    ob = oracle_with_eta(ob, inp.Ws, inp.bs, w.B, eta)
    for fused in (False, True):
        g = gpu_mixed_step(w, inp, grid, 4, fused=fused, force_acts=oracle_mixed_acts(ob, w), eta=eta, conv_split="batch")
        compare_mixed_step(g, ob, w, TOL, fused=fused, init=inp, require_sized=True)
    from tests.helpers import mixed_layers
    with pytest.raises(mbd.MbdError) as e:
        mbd.Net(mixed_layers(w, "batch"), w.B, 4, 3, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 0)
    assert e.value.status == mbd.E_GRID


def test_train_step_graph_matches_separate_calls(small):
    """mbd_train_step (captured graph, fused update) leaves the same weights, bit for bit, as
    forward + backward(eta) issued one by one; and two steps change them twice."""
    import torch
    from paper_1712_04432_b200 import mbd
    from tests.helpers import mixed_layers, to_dev
    w, inp, _ = small
    outs = []
    for mode in ("calls", "graph"):
        net = mbd.Net(mixed_layers(w), w.B, 2, 3, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 0)
        for i in range(w.L):
            bias = None if i < w.n_layers else torch.from_numpy(inp.bs[i]).cuda()
            net.set_weights(i, to_dev(inp.Ws[i], True), bias)
        X = to_dev(inp.X, True)
        labels = torch.from_numpy(inp.labels).cuda()
        J = torch.zeros(1, dtype=torch.float32, device="cuda")
        losses = []
        for _ in range(2):
            if mode == "calls":
                net.forward(X, labels, J)
                net.backward(w.eta)
            else:
                net.train_step(X, labels, w.eta, J)
            net.poll()
            losses.append(float(J.item()))
        outs.append((losses, [net.get_weights(i).clone() for i in range(w.L)]))
        net.close()
    assert outs[0][0] == outs[1][0]
    for a, b in zip(outs[0][1], outs[1][1]):
        assert torch.equal(a, b)
    assert outs[0][0][1] != outs[0][0][0]


def test_host_step_of_a_mixed_stack(small):
    import torch
    from paper_1712_04432_b200 import mbd
    from tests.helpers import mixed_layers, to_dev
    w, inp, o = small
    net = mbd.Net(mixed_layers(w), w.B, 2, 2, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 0)
    for i in range(w.L):
        bias = None if i < w.n_layers else torch.from_numpy(inp.bs[i]).cuda()
        net.set_weights(i, to_dev(inp.Ws[i], True), bias)
    Xh = to_dev(inp.X, True).cpu().pin_memory()
    lh = torch.from_numpy(inp.labels).pin_memory()
    J = net.train_step_host(Xh, lh, w.eta)
    net.poll()
    assert abs(J - o["J"]) <= 1e-2 * abs(o["J"])
    for i in range(w.L):
        assert rel_fro(net.get_weights(i).float().cpu().numpy(), o["new_W"][i]) <= TOL
    net.close()


# ------------------------------------------------------------------ convolutions with a split batch
@pytest.mark.parametrize("grid", [(1, 2), (2, 3), (4, 2)])
def test_conv_stack_with_batch_blocks(grid):
    w = I.conv_workload(64, 8, 40, 6, name="conv_pc")
    inp = I.make_inputs(w, seed=33)
    o = oracle_conv_step(w, inp, grid=grid)
    hidden = [np.ascontiguousarray(x, np.float32) for x in o["Xs"][1:]]
    g = gpu_conv_step(w, inp, grid[0], P_c=grid[1], force_acts=hidden)
    compare_conv_step(g, o, TOL)


def test_one_by_one_convolution_below_fully_connected_layers():
    w = I.mixed_workload(64, 8, 40, 2, (128, 16), 6, name="mixed_1x1", ksizes=(3, 1))
    inp = I.make_inputs(w, seed=34)
    o = oracle_mixed_step(w, inp)
    for grid, fused in [((1, 1), False), ((4, 3), True)]:
        g = gpu_mixed_step(w, inp, grid, 4, fused=fused, force_acts=oracle_mixed_acts(o, w))
        compare_mixed_step(g, o, w, TOL, fused)


@pytest.mark.parametrize("case", range(8))
def test_seeded_random_integrated_stacks(case):
    """Depth of both groups, kernel sizes, image shape (from one pixel column groups of eight strips per tile
    to two segments per row), batch, grid, number of materialised partials and fused / un-fused update drawn
    from a seeded generator."""
    r = np.random.default_rng(5000 + case)
    n_conv = int(r.integers(1, 4))
    ksizes = tuple(int(k) for k in r.choice([1, 3], size=n_conv))
    H = int(r.choice([4, 6, 8, 12]))
    W = int(r.choice([int(r.integers(3, 15)), int(r.integers(15, 31)), int(r.integers(31, 63)), int(r.integers(63, 150))]))
    B = int(r.integers(1, 8))
    fc = tuple(8 * int(r.integers(1, 13)) for _ in range(int(r.integers(1, 4))))
    P_r = int(r.choice([p for p in range(1, H + 1) if H % p == 0 and p <= min(fc)]))
    P_c = int(r.integers(1, B + 1))
    mp = int(r.choice([1, 2, 4, 64]))
    fused = bool(r.integers(0, 2))
    w = I.mixed_workload(64, H, W, n_conv, fc, B, name=f"mixed_random{case}", ksizes=ksizes)
    inp = I.make_inputs(w, seed=200 + case)
    o = oracle_mixed_step(w, inp)
    g = gpu_mixed_step(w, inp, (P_r, P_c), mp, fused=fused, force_acts=oracle_mixed_acts(o, w))
    compare_mixed_step(g, o, w, TOL, fused)
