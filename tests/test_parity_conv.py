"""Parity of the domain-parallel 3x3 convolution step (strips + halo rows) with the fp64
oracle, through the C ABI: forward outputs, the back-propagated gradient, the kernel gradients
and the updated kernels, for every strip count."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import compare_conv_step, gpu_conv_step, oracle_conv_step, oracle_with_eta, rel_fro, update_sized_eta

pytestmark = pytest.mark.gpu
TOL = 1e-2
TOL_FREE = 1e-2      # free-running (ReLU decisions on the device's own stored activations): measured 1.9e-3 at worst, no flips


def stored_hidden(o):
    return [np.ascontiguousarray(x, np.float32) for x in o["Xs"][1:]]


@pytest.fixture(scope="module")
def tiny():
    w = I.conv_workload(64, 8, 40, 2, name="conv_tiny")
    inp = I.make_inputs(w, seed=21)
    return w, inp, oracle_conv_step(w, inp)


@pytest.mark.parametrize("P_r", [1, 2, 4, 8])
def test_tiny_all_strip_counts(tiny, P_r):
    w, inp, o = tiny
    g = gpu_conv_step(w, inp, P_r, force_acts=stored_hidden(o))
    compare_conv_step(g, o, TOL)
    g = gpu_conv_step(w, inp, P_r)
    compare_conv_step(g, o, TOL, tol_below_relu=TOL_FREE)


@pytest.fixture(scope="module")
def ragged():
    # two forward segments (126 + 4 pixels), three backward-weight segments (64 + 64 + 2),
    # 28 rows (row blocks of 14 or 7 or 4), three images
    w = I.conv_workload(64, 28, 130, 3, name="conv_ragged")
    inp = I.make_inputs(w, seed=22)
    return w, inp, oracle_conv_step(w, inp)


@pytest.mark.parametrize("P_r", [1, 2, 7])
@pytest.mark.parametrize("fused", [False, True])
def test_ragged_shapes(ragged, P_r, fused):
    w, inp, o = ragged
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o))
    compare_conv_step(g, o, TOL, fused)


def test_strip_oracle_agrees(ragged):
    w, inp, _ = ragged
    ob = oracle_conv_step(w, inp, strips=4)
    g = gpu_conv_step(w, inp, 4, force_acts=stored_hidden(ob))
    compare_conv_step(g, ob, TOL)


def test_three_layers_and_reproducibility():
    w = I.conv_workload(64, 12, 64, 2, n_layers=3, name="conv3")
    inp = I.make_inputs(w, seed=23)
    o = oracle_conv_step(w, inp)
    a = gpu_conv_step(w, inp, 3, fused=True, force_acts=stored_hidden(o))
    compare_conv_step(a, o, TOL, fused=True)
    b = gpu_conv_step(w, inp, 3, fused=True, force_acts=stored_hidden(o))
    for i in range(3):
        assert np.array_equal(a["new_W"][i], b["new_W"][i]) and np.array_equal(a["dY"][i], b["dY"][i])


@pytest.mark.parametrize("P_r", [1, 8])
def test_full_resolution_two_images(P_r):
    # the 224 x 224 geometry of the large workload (strips of 224 / 28 rows), two images
    w = I.conv_workload(64, 224, 224, 2, name="conv_224")
    inp = I.make_inputs(w, seed=24)
    o = oracle_conv_step(w, inp)
    g = gpu_conv_step(w, inp, P_r, force_acts=stored_hidden(o))
    compare_conv_step(g, o, TOL)


@pytest.fixture(scope="module")
def cfg4_full():
    w = I.WORKLOADS["cfg4"]
    inp = I.make_inputs(w, seed=0)
    o = oracle_conv_step(w, inp)
    # a learning rate at which Eq. 1 moves both kernels by at least their own norm (see helpers.update_checks)
    eta = update_sized_eta(o, inp.Ws, w.B)
    return w, inp, oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta), eta


@pytest.mark.parametrize("P_r,fused", [(1, False), (2, True), (4, True), (8, True)])
def test_full_workload_32_images_every_strip_count(cfg4_full, P_r, fused):
    # the whole workload -- 32 images of 64 x 224 x 224 -- on every strip count it lists; two strips with the fused
    # update is the benchmark's launch configuration
    w, inp, o, eta = cfg4_full
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), eta=eta)
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)


@pytest.mark.parametrize("H,W,B,P_r", [(8, 62, 3, 1), (8, 56, 4, 2), (8, 30, 5, 2), (6, 14, 3, 3), (8, 7, 2, 1),
                                       (4, 1, 9, 1), (8, 63, 2, 2)])
@pytest.mark.parametrize("fused", [False, True])
def test_narrow_images_share_tiles(H, W, B, P_r, fused):
    """Images of at most 62 / 30 / 14 pixels per row put 2 / 4 / 8 strips into one 128-pixel tile; strip
    counts that do not fill the last group, the widest image of each class, and the first width that
    does not pack."""
    w = I.conv_workload(64, H, W, B, name=f"conv_narrow_{W}")
    inp = I.make_inputs(w, seed=40 + W)
    o = oracle_conv_step(w, inp)
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o))
    compare_conv_step(g, o, TOL, fused)


@pytest.mark.parametrize("mode", ["fused", "unfused", "graph"])
def test_second_step_uses_the_updated_kernels(mode):
    """Two steps in a row against two oracle steps: the operand layouts the convolution kernels read are
    refreshed by whatever updates the weights (fused update, mbd_sgd_step), also under graph replay."""
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    from tests.helpers import bf16_store, to_dev, to_np
    w = I.conv_workload(64, 8, 40, 2, name="conv_two_steps")
    w.eta = 2e-5
    inp = I.make_inputs(w, seed=61)
    layers = [O.Conv3x3(k.astype(np.float64), relu=True) for k in inp.Ws]
    X = inp.X.astype(np.float64)
    o1 = O.train_step(layers, X, None, "half_ssq", w.eta, store=bf16_store)
    # the device keeps its weights in bf16: the second oracle step starts from the rounded update
    layers2 = [O.Conv3x3(bf16_store(k), relu=True) for k in o1["new_W"]]
    o2 = O.train_step(layers2, X, None, "half_ssq", w.eta, store=bf16_store)
    assert abs(o2["J"] - o1["J"]) > 1e-3 * abs(o1["J"])          # the step is large enough to be seen

    net = mbd.Net(mbd.conv_layers(2, 64, 8, 40), w.B, 2, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    for i in range(2):
        net.set_weights(i, to_dev(inp.Ws[i], True))
    Xd = to_dev(inp.X, True)
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    Js = []
    for _ in range(2):
        if mode == "graph":
            net.train_step(Xd, None, w.eta, J)
        else:
            net.forward(Xd, None, J)
            if mode == "fused":
                net.backward(w.eta)
            else:
                net.backward(0.0)
                net.sgd_step(w.eta)
        net.poll()
        Js.append(float(J.item()))
    assert abs(Js[0] - o1["J"]) <= 1e-2 * abs(o1["J"])
    assert abs(Js[1] - o2["J"]) <= 1e-2 * abs(o2["J"])
    assert abs(Js[1] - o2["J"]) < 0.2 * abs(o2["J"] - o1["J"])    # and it is the second step's loss, not the first's
    for i in range(2):
        assert rel_fro(to_np(net.get_weights(i)), o2["new_W"][i]) <= TOL
    net.close()


@pytest.mark.parametrize("ksizes", [(3, 1, 3), (1, 3), (1, 1), (3, 1)])
@pytest.mark.parametrize("P_r", [1, 4])
@pytest.mark.parametrize("fused", [False, True])
def test_one_by_one_layers(ksizes, P_r, fused):
    """1 x 1 convolutions (the layers that need no halo, remark after Eq. 7) between, below and above
    3 x 3 ones; weights, gradients and updates are [C_out, C_in, 1, 1] at the boundary."""
    w = I.conv_workload(64, 8, 130, 3, n_layers=len(ksizes), name="conv_1x1", ksizes=ksizes)
    inp = I.make_inputs(w, seed=70 + len(ksizes) + ksizes[0])
    assert [k.shape[-1] for k in inp.Ws] == list(ksizes)
    o = oracle_conv_step(w, inp)
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o))
    assert [a.shape[-1] for a in g["new_W"]] == list(ksizes)
    compare_conv_step(g, o, TOL, fused)


@pytest.mark.parametrize("H,W,B,P_r,ksizes", [(10, 40, 2, 3, (3, 3)), (7, 130, 3, 2, (3, 3, 3)), (9, 64, 2, 4, (3, 1, 3)), (28, 130, 2, 5, (3, 3)),
                                              (10, 30, 5, 3, (3, 3)), (11, 14, 3, 4, (1, 3)), (5, 224, 1, 5, (3, 3)), (13, 40, 2, 7, (3, 3))])
@pytest.mark.parametrize("fused", [False, True])
def test_strips_of_unequal_height(H, W, B, P_r, ksizes, fused):
    """H is not a multiple of P_r: the strips are the balanced ranges [floor(s H / P_r), floor((s + 1) H / P_r)), one row
    apart in height (heights 4, 3, 3 for 10 rows on 3 strips; down to single-row strips) -- on wide, ragged and
    tile-sharing narrow images, with 1 x 1 layers in between; against the whole-image oracle and the oracle that
    forms the same strips with their halo rows."""
    w = I.conv_workload(64, H, W, B, n_layers=len(ksizes), name="conv_unequal", ksizes=ksizes)
    inp = I.make_inputs(w, seed=90 + H + W)
    o = oracle_conv_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    o = oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta)
    g = gpu_conv_step(w, inp, P_r, fused=fused, force_acts=stored_hidden(o), eta=eta)
    compare_conv_step(g, o, TOL, fused, init=inp, require_sized=True)
    assert abs(g["J"] - o["J"]) <= 1e-3 * abs(o["J"])            # the dead row of a short strip is not counted in the loss
    if not fused:
        ob = oracle_with_eta(oracle_conv_step(w, inp, strips=P_r), inp.Ws, inp.bs, w.B, eta)
        compare_conv_step(g, ob, TOL)
        one = gpu_conv_step(w, inp, 1, force_acts=stored_hidden(o), eta=eta)      # one strip: the same sums in another order
        for i in range(len(ksizes)):
            assert np.array_equal(g["act"][i], one["act"][i]) and np.array_equal(g["dY"][i], one["dY"][i]), i


@pytest.mark.parametrize("H,W,B,P_r,ksizes", [(8, 130, 3, 2, (1, 3, 1)), (8, 30, 5, 2, (1, 1)), (6, 14, 3, 3, (3, 1)), (12, 224, 2, 3, (1,))])
def test_one_by_one_layers_have_a_path_of_their_own(monkeypatch, H, W, B, P_r, ksizes):
    """A 1 x 1 layer reads one input row per output row and forms one tap (remark after Eq. 7: the layer that needs no
    halo); run instead as a 3 x 3 layer whose outer taps are zero it adds exact zeros to the same sums in the same
    order, so the two ways must agree bit for bit -- on wide, ragged and tile-sharing narrow images."""
    w = I.conv_workload(64, H, W, B, n_layers=len(ksizes), name="conv_1x1_path", ksizes=ksizes)
    inp = I.make_inputs(w, seed=80 + W)
    o = oracle_conv_step(w, inp)
    a = gpu_conv_step(w, inp, P_r, force_acts=stored_hidden(o))
    compare_conv_step(a, o, TOL)
    monkeypatch.setenv("MBD_CONV_1X1_AS_3X3", "1")
    b = gpu_conv_step(w, inp, P_r, force_acts=stored_hidden(o))
    for i in range(len(ksizes)):
        assert np.array_equal(a["act"][i], b["act"][i]) and np.array_equal(a["dY"][i], b["dY"][i]), i
        assert np.array_equal(a["dW"][i], b["dW"][i]) and np.array_equal(a["new_W"][i], b["new_W"][i]), i


def test_step_piece_by_piece_equals_the_whole_step():
    """mbd_forward / mbd_backward are the stepped calls in a row: same loss and, bit for bit, the same updated
    kernels; and halo rows written from outside are what the next layer reads (a strip cut out of a taller image
    gives the rows the whole image gives)."""
    import torch
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_dev, to_np
    w = I.conv_workload(64, 12, 40, 3, name="conv_steps")
    inp = I.make_inputs(w, seed=62)
    X = to_dev(inp.X, True)
    res = []
    for stepped in (False, True):
        net = mbd.Net(mbd.conv_layers(2, 64, 12, 40), w.B, 3, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
        for i in range(2):
            net.set_weights(i, to_dev(inp.Ws[i], True))
        J = torch.zeros(1, dtype=torch.float32, device="cuda")
        if stepped:
            net.conv_stage_input(X)
            net.conv_forward_layer(0)
            net.conv_forward_layer(1, J)
            net.conv_backward_layer(1, 1e-5)
            net.conv_backward_layer(0, 1e-5)
        else:
            net.forward(X, None, J)
            net.backward(1e-5)
        net.poll()
        res.append((float(J.item()), [net.get_weights(i).clone() for i in range(2)], net.get_tensor(mbd.T_ACT, 0).clone()))
        net.close()
    assert res[0][0] == res[1][0]
    for a, b in zip(res[0][1], res[1][1]):
        assert torch.equal(a, b)
    # rows 4..7 of the 12-row images as a network of their own, with rows 3 and 8 supplied as halo rows
    sub = mbd.Net(mbd.conv_layers(1, 64, 4, 40), w.B, 1, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    sub.set_weights(0, to_dev(inp.Ws[0], True))
    sub.conv_stage_input(X[:, :, 4:8, :].contiguous())
    nhwc = X.permute(0, 2, 3, 1).contiguous()                                  # [B, H, W, C]
    sub.conv_outer_rows(mbd.T_ACT, -1, 0, rows=nhwc[:, 3].contiguous())
    sub.conv_outer_rows(mbd.T_ACT, -1, 1, rows=nhwc[:, 8].contiguous())
    assert torch.equal(sub.conv_outer_rows(mbd.T_ACT, -1, 0), nhwc[:, 4].contiguous())   # first own row read back
    sub.conv_forward_layer(0)
    sub.poll()
    y_sub = to_np(sub.get_tensor(mbd.T_ACT, 0))                                # raw output of the last layer
    ref = inp.Ws[0].astype(np.float64)
    from oracle import mbd_oracle as O
    y_ref = O.conv3x3(ref, inp.X.astype(np.float64))[:, :, 4:8, :]
    assert rel_fro(y_sub, y_ref) < TOL
    sub.close()


@pytest.mark.parametrize("H,ksizes", [(12, (3, 3, 3)), (3, (3, 3)), (2, (3, 3)), (1, (3, 3)), (9, (3, 1, 3)), (5, (1, 1))])
def test_interior_and_boundary_rows_equal_the_whole_layer(H, ksizes):
    """Section 2.2: the rows of a strip that read no halo row (2 .. H - 1) can be computed while the halo rows travel.
    Every layer run as INTERIOR rows, then BOUNDARY rows -- forward and backward -- must leave, bit for bit, what the
    whole-layer calls leave: outputs, propagated gradients, kernel gradients (and the same loss up to the order in
    which the squares are added).  Strips of 1, 2 and 3 rows have
    no or one interior row; a 1 x 1 layer is all interior."""
    import torch
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_dev
    L = len(ksizes)
    w = I.conv_workload(64, H, 130, 3, n_layers=L, name="conv_rows", ksizes=ksizes)
    inp = I.make_inputs(w, seed=63 + H)
    X = to_dev(inp.X, True)
    res = []
    for split in (False, True):
        net = mbd.Net(mbd.conv_layers(L, 64, H, 130, k=list(ksizes)), w.B, 1, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
        for i in range(L):
            net.set_weights(i, to_dev(inp.Ws[i], True))
        J = torch.zeros(1, dtype=torch.float32, device="cuda")
        net.conv_stage_input(X)
        for i in range(L):
            out = J if i == L - 1 else None
            if split:
                net.conv_forward_layer(i, None, rows=mbd.ROWS_INTERIOR)
                net.conv_forward_layer(i, out, rows=mbd.ROWS_BOUNDARY)
            else:
                net.conv_forward_layer(i, out)
        for i in range(L - 1, -1, -1):
            if split:
                net.conv_backward_layer(i, 0.0, rows=mbd.ROWS_INTERIOR)
                net.conv_backward_layer(i, 0.0, rows=mbd.ROWS_BOUNDARY)
            else:
                net.conv_backward_layer(i, 0.0)
        net.poll()
        res.append(dict(J=float(J.item()), act=[net.get_tensor(mbd.T_ACT, i).clone() for i in range(L)],
                        dY=[net.get_tensor(mbd.T_DY, i).clone() for i in range(L)],
                        dK=[net.get_tensor(mbd.T_DW, i).clone() for i in range(L)]))
        net.close()
    a, b = res
    assert a["J"] > 0 and abs(a["J"] - b["J"]) <= 1e-5 * a["J"]       # the same squares, added in another order
    for i in range(L):
        assert torch.equal(a["act"][i], b["act"][i]) and torch.equal(a["dY"][i], b["dY"][i]) and torch.equal(a["dK"][i], b["dK"][i]), i
    # more than one strip per network has no such split
    net = mbd.Net(mbd.conv_layers(1, 64, 8, 40), 2, 2, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    net.conv_stage_input(to_dev(np.zeros((2, 64, 8, 40), np.float32), True))
    with pytest.raises(mbd.MbdError) as e:
        net.conv_forward_layer(0, None, rows=mbd.ROWS_INTERIOR)
    assert e.value.status == mbd.E_UNSUPPORTED
    net.close()
