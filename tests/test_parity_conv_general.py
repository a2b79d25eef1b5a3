"""Convolution layers the 64-channel 3 x 3 / 1 x 1 kernels do not cover -- other odd kernel sizes (5 x 5, 1 x 7,
7 x 1, 9 x 9, 11 x 11, mixed in one network), strides 2 to 4, channel counts that change from layer to layer and are not multiples of 64 -- on row
strips with floor(k_h/2) halo rows (Section 2.2) and P_c batch blocks: forward outputs, J, the back-propagated
gradients, the kernel gradients and the applied update against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import (compare_conv_step, compare_mixed_step, gpu_conv_step, gpu_mixed_step, oracle_conv_step, oracle_mixed_acts,
                           oracle_mixed_step, oracle_with_eta, rel_fro, update_sized_eta)

pytestmark = pytest.mark.gpu
TOL = 1e-2

CASES = {
    # name: (channels C_0..C_L, kernel shapes, H, W, B)
    "five_by_five_then_three": ((16, 32, 24), ((5, 5), (3, 3)), 12, 20, 4),
    "wide_and_tall_kernels": ((8, 8, 8), ((1, 7), (7, 1)), 12, 18, 3),
    "channel_blocks_of_64": ((64, 128, 64), ((3, 3), (1, 1)), 16, 24, 4),
    "three_layers_7x7_first": ((8, 40, 72, 16), ((7, 7), (3, 5), (5, 3)), 18, 14, 2),
}


def stored_hidden(o):
    return [np.ascontiguousarray(x, np.float32) for x in o["Xs"][1:]]


@pytest.fixture(scope="module", params=sorted(CASES))
def case(request):
    ch, ks, H, W, B = CASES[request.param]
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name=request.param, ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=61)
    o = oracle_conv_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    return w, inp, oracle_with_eta(o, inp.Ws, [None] * w.n_layers, w.B, eta), eta


@pytest.mark.parametrize("P_r,P_c,mp", [(1, 1, 0), (2, 1, 0), (3, 2, 4), (1, 2, 1), (6, 1, 2)])
@pytest.mark.parametrize("fused", [False, True])
def test_general_layers_on_strips_and_batch_blocks(case, P_r, P_c, mp, fused):
    w, inp, o, eta = case
    H = w.dims[1]
    if P_c > w.B:
        pytest.skip("more batch blocks than samples")
    if P_r > 1 and H // P_r < max(w.kshape(i)[0] // 2 for i in range(w.n_layers)):
        pytest.skip("a strip shorter than its halo: refused by mbd_net_create (see the last test)")
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), P_c=P_c, eta=eta, max_partials=mp)
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)


def test_strip_formulation_of_the_oracle_agrees():
    ch, ks, H, W, B = CASES["five_by_five_then_three"]
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name="strips", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=62)
    ob = oracle_conv_step(w, inp, grid=(3, 2))             # strips with two halo rows, partials per process
    g = gpu_conv_step(w, inp, 3, P_c=2, force_acts=stored_hidden(ob))
    compare_conv_step(g, ob, TOL)


@pytest.mark.parametrize("name,grid", [("channel_blocks_of_64", (3, 2)), ("five_by_five_then_three", (5, 1)), ("three_layers_7x7_first", (4, 2))])
def test_strips_of_unequal_height_on_the_general_path(name, grid):
    # H mod P_r != 0: the balanced ranges of rows (16 rows on 3 strips: 5, 5, 6; 12 on 5: 2, 2, 2, 3, 3; 18 on 4: 4, 5, 4, 5);
    # every strip has ceil(H / P_r) row slots, the last slot of a shorter strip is a dead row that stays zero, and a
    # strip's lower halo rows follow its last OWN row.  Against the oracle's strip formulation on the same ranges.
    ch, ks, H, W, B = CASES[name]
    assert H % grid[0] != 0
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name="ragged_" + name, ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=64)
    ob = oracle_conv_step(w, inp, grid=grid)
    eta = update_sized_eta(ob, inp.Ws, w.B)
    ob = oracle_conv_step(w, inp, grid=grid, eta=eta)
    for fused in (False, True):
        g = gpu_conv_step(w, inp, grid[0], fused=fused, P_c=grid[1], force_acts=stored_hidden(ob), eta=eta, max_partials=2)
        compare_conv_step(g, ob, TOL, fused, init=inp, require_sized=True)


def test_listed_64_channel_layers_through_the_general_path(monkeypatch):
    # the layers that have kernels of their own, forced onto the contraction kernel: same oracle, same tolerance,
    # and the two device paths agree with each other far below it
    w = I.conv_workload(64, 16, 40, 3, name="conv_both_paths")
    inp = I.make_inputs(w, seed=63)
    o = oracle_conv_step(w, inp)
    own = gpu_conv_step(w, inp, 2, force_acts=stored_hidden(o))
    monkeypatch.setenv("MBD_CONV_GENERAL", "1")
    gen = gpu_conv_step(w, inp, 2, force_acts=stored_hidden(o))
    compare_conv_step(gen, o, TOL)
    for i in range(w.n_layers):
        assert rel_fro(gen["act"][i], own["act"][i]) < 5e-3 and rel_fro(gen["dW"][i], own["dW"][i]) < 1e-3, i
    assert abs(gen["J"] - own["J"]) < 1e-3 * abs(own["J"])


def test_free_running_step_and_reproducibility():
    ch, ks, H, W, B = CASES["channel_blocks_of_64"]
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name="free", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=64)
    o = oracle_conv_step(w, inp)
    a = gpu_conv_step(w, inp, 2, fused=True, P_c=2)
    compare_conv_step(a, o, TOL, fused=True, tol_below_relu=2e-2)
    b = gpu_conv_step(w, inp, 2, fused=True, P_c=2)
    for i in range(w.n_layers):
        assert np.array_equal(a["new_W"][i], b["new_W"][i]) and np.array_equal(a["dY"][i], b["dY"][i])


STRIDED = {
    # name: (channels, kernel shapes, strides, H, W, B)
    "stride2_3x3_between_unit_layers": ((16, 24, 32, 16), ((3, 3), (3, 3), (3, 3)), (1, 2, 1), 16, 24, 3),
    "stride2_5x5_first": ((8, 32, 16), ((5, 5), (3, 3)), (2, 1), 24, 16, 4),
    "stride2_7x7_then_stride2_1x1": ((8, 64, 72), ((7, 7), (1, 1)), (2, 2), 24, 32, 2),
    "stride3_3x3_and_stride4_5x3": ((16, 16, 8), ((3, 3), (5, 3)), (3, 4), 48, 24, 2),
    # the kernel sizes and strides of the network of Section 3 (its first layers: 11 x 11 stride 4, then 5 x 5, then 3 x 3)
    "stride4_11x11_then_5x5_then_3x3": ((8, 96, 64, 48), ((11, 11), (5, 5), (3, 3)), (4, 1, 1), 32, 48, 2),
    "unit_9x9_and_1x11": ((8, 16, 8), ((9, 9), (1, 11)), (1, 1), 12, 24, 2),
}


@pytest.fixture(scope="module", params=sorted(STRIDED))
def strided(request):
    ch, ks, st, H, W, B = STRIDED[request.param]
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name=request.param, ksizes=ks, channels=ch, strides=st)
    inp = I.make_inputs(w, seed=71)
    o = oracle_conv_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    return w, inp, oracle_with_eta(o, inp.Ws, [None] * w.n_layers, w.B, eta), eta


@pytest.mark.parametrize("P_r,P_c,mp", [(1, 1, 0), (2, 1, 0), (2, 2, 4), (4, 1, 2)])
@pytest.mark.parametrize("fused", [False, True])
def test_strided_layers(strided, P_r, P_c, mp, fused):
    # A stride-s layer keeps every s-th position of the stride-1 result (Section 2.2 speaks of the halo only; the halo a
    # strip needs is still floor(k_h/2) input rows).  The device never computes a position it does not keep: it reads
    # its input through s^2 phase planes, each a stride-1 shifted-view product again.
    w, inp, o, eta = strided
    H_last = w.out_hw(w.n_layers - 1)[0]
    halo = max(-(-(w.kshape(i)[0] // 2) // w.stride(i)) for i in range(w.n_layers))      # rows a strip needs from a neighbour
    if H_last % P_r or (P_r > 1 and H_last // P_r < halo):
        pytest.skip("strips of equal height, no shorter than the halo, at every resolution")
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), P_c=P_c, eta=eta, max_partials=mp)
    assert g["act"][-1].shape[2:] == w.out_hw(w.n_layers - 1)
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)


@pytest.mark.parametrize("grid,mp,fused", [((1, 1), 1, False), ((2, 3), 4, True), ((4, 2), 2, False)])
def test_integrated_stack_on_general_convolutions(grid, mp, fused):
    # Section 2.4 on layers of the general path: a 5 x 5 and a 3 x 3 convolution with 16 channels on 8 x 20 images, then
    # model-parallel fully connected layers 2560 -> 64 -> 16 on the same grid
    w = I.mixed_workload(16, 8, 20, 2, (64, 16), 6, name="mixed_general", ksizes=(5, 3))
    inp = I.make_inputs(w, seed=65)
    o = oracle_mixed_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    g = gpu_mixed_step(w, inp, grid, mp, fused=fused, force_acts=oracle_mixed_acts(o, w), eta=eta)
    compare_mixed_step(g, o, w, TOL, fused=fused, init=inp, require_sized=True)


@pytest.mark.parametrize("grid,mp,fused", [((1, 1), 1, True), ((2, 2), 2, False)])
def test_integrated_stack_with_a_strided_layer(grid, mp, fused):
    # 3 x 3 stride 2 (16 -> 32 channels, 16 x 24 -> 8 x 12), 3 x 3 stride 1, then FC 3072 -> 48 -> 16: the first fully
    # connected layer reads C_L * H_L * W_L values per sample
    w = I.mixed_workload(16, 16, 24, 2, (48, 16), 4, name="mixed_strided", ksizes=(3, 3), channels=(16, 32, 32), strides=(2, 1))
    assert w.fc_dims[0] == 32 * 8 * 12
    inp = I.make_inputs(w, seed=72)
    o = oracle_mixed_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    g = gpu_mixed_step(w, inp, grid, mp, fused=fused, force_acts=oracle_mixed_acts(o, w), eta=eta)
    compare_mixed_step(g, o, w, TOL, fused=fused, init=inp, require_sized=True)


@pytest.mark.parametrize("master,mu", [(True, None), (False, 0.9), (True, 0.9)])
def test_master_weights_and_momentum_on_general_layers(master, mu):
    # the update as a kernel of its own over the internal weight layout: from the gradient the device itself
    # materialised, three steps, mbd_backward(eta) and mbd_backward(0) + mbd_sgd_step(eta) bit for bit
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_dev, to_np
    ch, ks, st, H, W, B = (16, 24, 32), ((5, 5), (3, 3)), (1, 2), 16, 24, 3
    w = I.conv_workload(ch[0], H, W, B, n_layers=2, name="gen_update", ksizes=ks, channels=ch, strides=st)
    inp = I.make_inputs(w, seed=73)
    X = to_dev(inp.X, True)
    eta = 1e-3

    def make():
        net = mbd.Net(mbd.conv_layers(2, ch[0], H, W, k=list(ks), channels=ch, strides=st), B, 2, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 2)
        if master:
            net.enable_master_weights()
        for i in range(2):
            net.set_weights(i, to_dev(inp.Ws[i], True))
        if mu is not None:
            net.enable_momentum(mu)
        return net
    a, b = make(), make()
    for step in range(3):
        W_old = [to_np(a.get_tensor(mbd.T_MASTER, i)) if master else to_np(a.get_weights(i)) for i in range(2)]
        V_old = [to_np(a.get_tensor(mbd.T_VELOCITY, i)) if mu is not None else np.zeros_like(W_old[i]) for i in range(2)]
        a.forward(X); a.backward(0.0)
        dW = [to_np(a.get_tensor(mbd.T_DW, i)) for i in range(2)]
        a.sgd_step(eta)
        b.forward(X); b.backward(eta)
        a.poll(); b.poll()
        for i in range(2):
            W_want, V_want = O.sgd_momentum(W_old[i], V_old[i], dW[i], eta, B, mu if mu is not None else 0.0)
            if mu is not None:
                assert rel_fro(to_np(a.get_tensor(mbd.T_VELOCITY, i)), V_want) < 1e-6, (step, i)
            if master:
                assert rel_fro(to_np(a.get_tensor(mbd.T_MASTER, i)), W_want) < 1e-6, (step, i)
                assert torch.equal(a.get_tensor(mbd.T_MASTER, i).to(torch.bfloat16), a.get_weights(i))
                assert torch.equal(a.get_tensor(mbd.T_MASTER, i), b.get_tensor(mbd.T_MASTER, i)), (step, i)
            else:
                assert rel_fro(to_np(a.get_weights(i)), W_want) < 3e-3, (step, i)
            assert torch.equal(a.get_weights(i), b.get_weights(i)), (step, i)
            assert np.linalg.norm(dW[i]) > 0
    a.close(); b.close()


@pytest.mark.parametrize("grid,mp,fused", [((1, 1), 1, True), ((3, 2), 2, False), ((2, 2), 4, True)])
def test_layer_shapes_of_the_networks_of_section_3(grid, mp, fused):
    # the `alexlike` workload of the benchmark in miniature: 11 x 11 stride 4 (8 -> 96 channels), 5 x 5 stride 2 (96 -> 256),
    # 3 x 3 (256 -> 384 -> 384), 3 x 3 stride 2 (384 -> 256), then model-parallel fully connected layers, on 96 x 96 inputs
    w = I.mixed_workload(8, 96, 96, 5, (64, 32, 16), 4, name="alexlike_small", ksizes=((11, 11), (5, 5), (3, 3), (3, 3), (3, 3)),
                         channels=(8, 96, 256, 384, 384, 256), strides=(4, 2, 1, 1, 2))
    assert w.fc_dims[0] == 256 * 6 * 6 and [w.out_hw(i) for i in range(5)] == [(24, 24), (12, 12), (12, 12), (12, 12), (6, 6)]
    inp = I.make_inputs(w, seed=74)
    o = oracle_mixed_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    g = gpu_mixed_step(w, inp, grid, mp, fused=fused, force_acts=oracle_mixed_acts(o, w), eta=eta)
    compare_mixed_step(g, o, w, TOL, fused=fused, init=inp, require_sized=True)


@pytest.mark.parametrize("name,Cin,k,s,blocks_folded,blocks_plain", [
    ("3x3", 8, (3, 3), 1, 3, 9),              # a row of three taps of 8 channels fits one 64-wide block
    ("7x7", 16, (7, 7), 1, 14, 49),           # four taps of 16 channels per block: two blocks per kernel row
    ("11x11 stride 4", 8, (11, 11), 4, 44, 121),    # 16 phase planes, up to three taps of a row per plane
    ("5x5 stride 2", 32, (5, 5), 2, 15, 25)])
def test_first_layer_with_few_channels_folds_its_taps(monkeypatch, name, Cin, k, s, blocks_folded, blocks_plain):
    # The input is pixel-major, so the channels of consecutive pixels are contiguous: through a tensor map whose rows
    # overlap, one 64-element operand row holds 64 / C_in horizontally adjacent taps.  Fewer, fuller k-blocks, the
    # same sums: both forms against the oracle, and against each other far below the tolerance.
    from paper_1712_04432_b200 import mbd
    H, W, B = 8 * s * 2, 12 * s, 3
    w = I.conv_workload(Cin, H, W, B, n_layers=2, name="fold", ksizes=(k, (3, 3)), channels=(Cin, 40, 24), strides=(s, 1))
    inp = I.make_inputs(w, seed=75)
    o = oracle_conv_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    res = {}
    for fold in (True, False):
        if not fold:
            monkeypatch.setenv("MBD_CONV_NO_FOLD", "1")
        net = mbd.Net(mbd.conv_layers(2, Cin, H, W, k=[k, (3, 3)], channels=(Cin, 40, 24), strides=(s, 1)), B, 2, 1, mbd.BF16,
                      mbd.LOSS_HALF_SSQ, 2)
        want = blocks_folded if fold else blocks_plain
        assert net.plan(0, 0)["k_blocks"] == want, (name, net.plan(0, 0))
        assert net.plan(0, 2)["ctas"] > 0 and net.plan(1, 0)["k_blocks"] == 9           # 40 channels: one block per tap
        net.close()
        for fused in (False, True):
            g = gpu_conv_step(w, inp, 2, fused=fused, force_acts=stored_hidden(o), eta=eta, max_partials=2)
            compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)
            res[(fold, fused)] = g
    a, b = res[(True, False)], res[(False, False)]
    for i in range(2):
        assert rel_fro(a["act"][i], b["act"][i]) < 5e-3 and rel_fro(a["dW"][i], b["dW"][i]) < 1e-3, (name, i)


@pytest.mark.parametrize("ch,ks,st,H,W,B,P_r,P_c", [
    ((8, 8), ((7, 7),), (1,), 4, 4, 1, 1, 1),                # an image smaller than its kernel, one sample
    ((24, 16, 8), ((3, 5), (1, 1)), (1, 1), 5, 37, 5, 1, 5),  # odd width, one sample per batch block
    ((8, 72), ((9, 1),), (1,), 16, 3, 2, 2, 1),              # three pixels per row, a tall kernel, two strips of 8 rows
    ((16, 8), ((3, 3),), (4,), 8, 8, 3, 2, 1),               # stride 4 down to 2 x 2 outputs, strips of one row
    ((32, 40), ((5, 5),), (2,), 4, 6, 2, 1, 2)])             # stride 2 on a 4 x 6 image
def test_small_and_ragged_shapes(ch, ks, st, H, W, B, P_r, P_c):
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name="edge", ksizes=ks, channels=ch, strides=st)
    inp = I.make_inputs(w, seed=76)
    o = oracle_conv_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    for fused in (False, True):
        g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), P_c=P_c, eta=eta, max_partials=2)
        compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)


def test_unsupported_shapes_are_refused():
    from paper_1712_04432_b200 import mbd
    for kw in (dict(k=(4, 3)), dict(k=13), dict(channels=(12, 8, 8)), dict(channels=(8, 4, 8))):
        layers = mbd.conv_layers(2, 8, 12, 12, **{"k": 3, **kw}) if "channels" not in kw else \
            mbd.conv_layers(2, kw["channels"][0], 12, 12, channels=kw["channels"])
        with pytest.raises(mbd.MbdError) as e:
            mbd.Net(layers, 2, 1, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
        assert e.value.status == mbd.E_UNSUPPORTED, kw
    # a 7-row kernel needs three halo rows from the adjacent strip: strips of two rows cannot supply them
    with pytest.raises(mbd.MbdError) as e:
        mbd.Net(mbd.conv_layers(1, 8, 12, 12, k=7), 2, 6, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    assert e.value.status == mbd.E_GRID
    # strips of unequal height: not under a strided layer (its phase planes are cut per strip)
    with pytest.raises(mbd.MbdError) as e:
        mbd.Net(mbd.conv_layers(1, 8, 20, 12, k=5, strides=(2,)), 2, 3, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    assert e.value.status == mbd.E_UNSUPPORTED


MODEL_CASES = {
    # convolutions in L_M: channels C_0..C_L (every C_out a multiple of 64 P_r), kernel shapes, H, W, B
    "five_by_five_then_three_on_wide_layers": ((16, 128, 256), ((5, 5), (3, 3)), 12, 16, 4),
    "three_by_three_then_one_by_one": ((64, 256, 256), ((3, 3), (1, 1)), 10, 12, 6),
}


@pytest.mark.parametrize("name", sorted(MODEL_CASES))
@pytest.mark.parametrize("grid,mp", [((2, 1), 2), ((2, 2), 2), ((1, 2), 2), ((2, 2), 1), ((4, 2), 2), ((4, 1), 4)])
@pytest.mark.parametrize("fused", [False, True])
def test_model_parallel_convolutions(name, grid, mp, fused):
    # Eq. 8 for convolution layers: the P_r groups split the output channels, the P_c groups the batch; dX is the sum
    # over the groups' partial results (a cut of the backward-data product's K range over blocks of output channels),
    # dK a sum over the batch blocks.  Against the oracle's blocked step of the same grid.
    from paper_1712_04432_b200 import mbd
    ch, ks, H, W, B = MODEL_CASES[name]
    P_r, P_c = grid
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name=name, ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=81)
    if any(c % (64 * P_r) for c in ch[1:]):
        with pytest.raises(mbd.MbdError) as e:
            gpu_conv_step(w, inp, P_r, P_c=P_c, max_partials=mp, split=mbd.SPLIT_MODEL)
        assert e.value.status == mbd.E_UNSUPPORTED          # a group's channels must be whole 64-channel blocks
        return
    o = oracle_conv_step(w, inp, grid=grid, split="model")
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_conv_step(w, inp, grid=grid, split="model", eta=eta)
    plans = {(1, 1): None, (1, 2): None}
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), P_c=P_c, eta=eta, max_partials=mp, split=mbd.SPLIT_MODEL,
                      plans=plans)
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)
    assert plans[(1, 1)]["k_pieces"] == min(P_r, mp), plans              # dX: one partial sum per group (or per max_partials)
    assert plans[(1, 2)]["k_pieces"] % min(P_c, mp) == 0, plans          # dK: batch blocks first, then the planner's own cuts


def test_model_parallel_convolutions_equal_the_unsplit_layers_up_to_the_order_of_sums():
    from paper_1712_04432_b200 import mbd
    ch, ks, H, W, B = MODEL_CASES["five_by_five_then_three_on_wide_layers"]
    w = I.conv_workload(ch[0], H, W, B, n_layers=len(ks), name="model_vs_unsplit", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=82)
    a = gpu_conv_step(w, inp, 1, P_c=1)
    b = gpu_conv_step(w, inp, 2, P_c=2, max_partials=2, split=mbd.SPLIT_MODEL)
    for i in range(w.n_layers):
        assert np.array_equal(a["act"][i], b["act"][i]), i                 # forward: no sum is cut
        # (dY below the top is stored in bf16 after sums taken in another order: a few roundings differ)
        assert rel_fro(b["dW"][i], a["dW"][i]) < 1e-3 and rel_fro(b["dY"][i], a["dY"][i]) < 1e-2, i


@pytest.mark.parametrize("grid,mp,fused", [((2, 2), 2, True), ((2, 3), 1, False), ((1, 1), 1, True)])
def test_integrated_stack_with_model_parallel_convolutions(grid, mp, fused):
    # every layer in L_M: convolutions and fully connected layers alike split their outputs over P_r and the batch over
    # P_c (Eq. 8 for the whole network); 5 x 5 and 3 x 3 on 16 -> 128 -> 128 channels, then FC 12288 -> 64 -> 16
    w = I.mixed_workload(16, 8, 12, 2, (64, 16), 6, name="mixed_model_split", ksizes=((5, 5), (3, 3)), channels=(16, 128, 128))
    inp = I.make_inputs(w, seed=83)
    o = oracle_mixed_step(w, inp, blocked_grid=grid, conv_split="model")
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_mixed_step(w, inp, blocked_grid=grid, conv_split="model", eta=eta)
    g = gpu_mixed_step(w, inp, grid, mp, fused=fused, force_acts=oracle_mixed_acts(o, w), eta=eta, conv_split="model")
    compare_mixed_step(g, o, w, TOL, fused=fused, init=inp, require_sized=True)


SPLIT_OF = {"domain": 1, "batch": 2, "model": 0}          # mbd.SPLIT_DOMAIN, SPLIT_BATCH, SPLIT_MODEL


@pytest.mark.parametrize("kinds", [("domain", "domain", "model"), ("domain", "model", "model"), ("model", "domain", "batch"),
                                   ("batch", "model", "domain")])
@pytest.mark.parametrize("grid,mp", [((2, 2), 2), ((2, 1), 1), ((1, 3), 3)])
@pytest.mark.parametrize("fused", [False, True])
def test_each_convolution_in_the_set_of_its_own(kinds, grid, mp, fused):
    # Section 2.4: every layer is in L_M or L_D on its own.  Three convolutions (5 x 5, 3 x 3, 3 x 3 on 16 -> 128 -> 128 -> 128
    # channels) whose split kinds differ: runs of equal kind are stacks of their own, and between two runs the activation
    # (forward) and its gradient (backward) change their distribution.  Against the oracle's blocked step with the same
    # kinds on the same grid.
    assert SPLIT_OF == {"domain": 1, "batch": 2, "model": 0}
    ch, ks, H, W, B = (16, 128, 128, 128), ((5, 5), (3, 3), (3, 3)), 12, 16, 6
    w = I.conv_workload(ch[0], H, W, B, n_layers=3, name="mixed_kinds", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=84)
    o = oracle_conv_step(w, inp, grid=grid, split=kinds)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_conv_step(w, inp, grid=grid, split=kinds, eta=eta)
    g = gpu_conv_step(w, inp, grid[0], fused=fused, force_acts=stored_hidden(o), P_c=grid[1], eta=eta, max_partials=mp,
                      split=[SPLIT_OF[k] for k in kinds])
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)


def test_integrated_stack_with_convolutions_of_different_kinds():
    # domain-split 5 x 5, model-split 3 x 3, then model-split fully connected layers on one 2 x 2 grid
    from paper_1712_04432_b200 import mbd
    import torch
    from tests.helpers import to_dev, to_np
    from oracle import mbd_oracle as O
    from tests.helpers import bf16_store, oracle_kernel
    w = I.mixed_workload(16, 8, 12, 2, (64, 16), 6, name="mixed_kinds_fc", ksizes=((5, 5), (3, 3)), channels=(16, 128, 128))
    inp = I.make_inputs(w, seed=85)
    kinds = ("domain", "model")
    layers = [O.Conv3x3(oracle_kernel(inp.Ws[i]), relu=True, split=kinds[i]) for i in range(2)]
    layers += [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64), relu=True) for i in range(2, w.L)]
    o = O.train_step_blocked(layers, inp.X.astype(np.float64), inp.labels, "softmax_ce", w.eta, 2, 2, store=bf16_store)
    spec = mbd.conv_layers(2, 16, 8, 12, k=[(5, 5), (3, 3)], channels=(16, 128, 128), split=[mbd.SPLIT_DOMAIN, mbd.SPLIT_MODEL]) + \
        mbd.fc_layers(w.fc_dims, bias=True)
    net = mbd.Net(spec, w.B, 2, 2, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 2)
    for i in range(w.L):
        if i < 2:
            net.set_weights(i, to_dev(inp.Ws[i], True))
        else:
            net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    net.forward(to_dev(inp.X, True), torch.from_numpy(inp.labels).cuda(), J)
    acts = oracle_mixed_acts(o, w)
    for i in range(w.L - 1):
        assert rel_fro(to_np(net.get_tensor(mbd.T_ACT, i)), acts[i]) < TOL, i
        net.set_tensor(mbd.T_ACT, i, to_dev(acts[i], True))
    assert abs(float(J.item()) - o["J"]) < 1e-2 * abs(o["J"])
    net.backward(0.0)
    net.poll()
    for i in range(w.L):
        got = to_np(net.get_tensor(mbd.T_DW, i))
        assert rel_fro(got, o["dWs"][i].reshape(got.shape)) < TOL, f"dW[{i}]"
    net.close()


@pytest.mark.parametrize("master,mu", [(True, None), (False, 0.9)])
def test_masters_and_momentum_on_a_stack_of_different_kinds(master, mu):
    # the update kernels run per run of layers: mbd_backward(eta) and mbd_backward(0) + mbd_sgd_step(eta) bit for bit,
    # and the step itself against Eq. 1 / the heavy-ball form on the gradient the device materialised
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_dev, to_np
    ch, ks, H, W, B = (16, 128, 128), ((5, 5), (3, 3)), 8, 12, 4
    w = I.conv_workload(ch[0], H, W, B, n_layers=2, name="kinds_update", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=86)
    X = to_dev(inp.X, True)
    eta = 1e-3

    def make():
        net = mbd.Net(mbd.conv_layers(2, ch[0], H, W, k=list(ks), channels=ch, split=[mbd.SPLIT_DOMAIN, mbd.SPLIT_MODEL]), B, 2, 2, mbd.BF16,
                      mbd.LOSS_HALF_SSQ, 2)
        if master:
            net.enable_master_weights()
        for i in range(2):
            net.set_weights(i, to_dev(inp.Ws[i], True))
        if mu is not None:
            net.enable_momentum(mu)
        return net
    a, b = make(), make()
    for step in range(2):
        W_old = [to_np(a.get_tensor(mbd.T_MASTER, i)) if master else to_np(a.get_weights(i)) for i in range(2)]
        V_old = [to_np(a.get_tensor(mbd.T_VELOCITY, i)) if mu is not None else np.zeros_like(W_old[i]) for i in range(2)]
        a.forward(X); a.backward(0.0)
        dW = [to_np(a.get_tensor(mbd.T_DW, i)) for i in range(2)]
        a.sgd_step(eta)
        b.forward(X); b.backward(eta)
        a.poll(); b.poll()
        for i in range(2):
            W_want, _ = O.sgd_momentum(W_old[i], V_old[i], dW[i], eta, B, mu if mu is not None else 0.0)
            got = to_np(a.get_tensor(mbd.T_MASTER, i)) if master else to_np(a.get_weights(i))
            assert rel_fro(got, W_want) < (1e-6 if master else 3e-3), (step, i)
            assert torch.equal(a.get_weights(i), b.get_weights(i)), (step, i)
            assert np.linalg.norm(dW[i]) > 0
    a.close(); b.close()


def test_graph_replay_of_a_stack_of_different_kinds_equals_direct_launches():
    # mbd_train_step captures the step once and replays it: runs of layers, re-distributions and all
    import torch
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_dev
    ch, ks, H, W, B = (16, 128, 128, 128), ((5, 5), (3, 3), (1, 1)), 8, 12, 4
    w = I.conv_workload(ch[0], H, W, B, n_layers=3, name="kinds_graph", ksizes=ks, channels=ch)
    inp = I.make_inputs(w, seed=87)
    X = to_dev(inp.X, True)

    def make():
        net = mbd.Net(mbd.conv_layers(3, ch[0], H, W, k=list(ks), channels=ch, split=[mbd.SPLIT_DOMAIN, mbd.SPLIT_MODEL, mbd.SPLIT_BATCH]), B, 2, 2,
                      mbd.BF16, mbd.LOSS_HALF_SSQ, 2)
        for i in range(3):
            net.set_weights(i, to_dev(inp.Ws[i], True))
        return net
    a, b = make(), make()
    Ja, Jb = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
    for step in range(3):
        a.train_step(X, None, 1e-4, Ja)
        b.forward(X, None, Jb); b.backward(1e-4)
        a.poll(); b.poll()
        assert float(Ja.item()) == float(Jb.item()) and float(Ja.item()) > 0, step
        for i in range(3):
            assert torch.equal(a.get_weights(i), b.get_weights(i)), (step, i)
    a.close(); b.close()
