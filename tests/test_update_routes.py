"""Eq. 1 on bf16 weights, route by route.

The update w <- w - (eta/B) dW is applied in several places of the library, depending on how
the backward-weight product of a layer is launched: in the epilogue of the product (through
shared-memory boxes moved by TMA on 128-row tiles, or from registers on 256-row tiles and CTA
pairs), in the tail of the partial-sum reduction when the batch is cut into P_c blocks (a
general kernel and one for two large planes), or by a kernel of its own from the materialised
gradient; the biases are updated at the end of the column sums.  At the workloads' eta = 0.01 a
step moves a weight matrix by a few 1e-4 of its norm -- less than the bf16 rounding of the
weights themselves -- so comparing updated weights cannot tell a correct update from none.  Here
the learning rate is chosen so that the step is as large as the weights, the ReLU decisions are
forced to the oracle's, and the applied step W_new - W_0 is compared with the oracle's step to
1e-2 of the STEP's norm.  Each case asserts, through mbd_get_plan, that the route it names is the
one that ran.
"""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import (compare_fc_step, gpu_fc_step, oracle_fc_step, oracle_hidden_acts, oracle_with_eta,
                           to_dev, update_sized_eta)

pytestmark = pytest.mark.gpu

TOL = 1e-2

# name: (environment knobs, grid, max_partials, fused, expected plan of layer 0's backward-weight product)
ROUTES = {
    "epilogue_tma_128_row_tiles": ({"MBD_TC_MH": "1", "MBD_TC_PAIR": "0"}, (1, 1), 1, True,
                                   dict(tile_m=128, cta_pair=0, k_pieces=1, tma_epilogue=1)),
    "epilogue_tma_cta_pair_256": ({"MBD_TC_PAIR": "1"}, (1, 1), 1, True,
                                  dict(tile_m=256, cta_pair=1, k_pieces=1, tma_epilogue=1)),
    "epilogue_registers_128_row_tiles": ({"MBD_TC_MH": "1", "MBD_TC_PAIR": "0", "MBD_TC_NO_TE": "1"}, (1, 1), 1, True,
                                         dict(tile_m=128, cta_pair=0, k_pieces=1, tma_epilogue=0)),
    "epilogue_registers_256_row_tiles": ({"MBD_TC_MH": "2", "MBD_TC_PAIR": "0"}, (1, 1), 1, True,
                                         dict(tile_m=256, cta_pair=0, k_pieces=1, tma_epilogue=0)),
    "epilogue_registers_cta_pair_512": ({"MBD_TC_PAIR": "2"}, (1, 1), 1, True,
                                        dict(tile_m=512, cta_pair=1, k_pieces=1, tma_epilogue=0)),
    "reduction_tail_three_planes": ({}, (1, 3), 3, True, dict(k_pieces=3, running_sum=0)),
    "reduction_tail_two_large_planes": ({}, (2, 2), 2, True, dict(k_pieces=2, running_sum=0)),
    "update_kernel_from_materialised_gradient": ({}, (1, 1), 1, False, dict(k_pieces=1)),
    "update_kernel_after_a_reduction": ({}, (1, 2), 2, False, dict(k_pieces=2)),
}


@pytest.fixture(scope="module")
def net_case():
    # layer 1 holds 2048 x 1024 = 2 Mi weights: with two batch blocks its reduction is the two-plane kernel;
    # ragged tiles elsewhere (264, 1000), K = B = 328 has a tail that is not a multiple of 64
    w = I.fc_workload((1024, 2048, 264, 1000), 328, "bf16", "relu_normal", name="update_routes")
    inp = I.make_inputs(w, seed=21)
    o = oracle_fc_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    return w, inp, oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta), eta


def _plan_of(w, grid, mp):
    from paper_1712_04432_b200 import mbd
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
    plans = [net.plan(i, 2) for i in range(len(w.dims) - 1)]
    net.close()
    return plans


@pytest.mark.parametrize("route", sorted(ROUTES))
def test_applied_step_matches_the_oracle_on_every_route(monkeypatch, net_case, route):
    w, inp, o, eta = net_case
    env, grid, mp, fused, want = ROUTES[route]
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    plan = _plan_of(w, grid, mp)[0]
    for k, v in want.items():
        assert plan[k] == v, (route, plan)
    g = gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta)
    compare_fc_step(g, o, TOL, fused, init=inp, require_sized=True)
    # the step is as large as the weights: an update that did not happen cannot hide
    for i in range(3):
        assert np.linalg.norm(g["new_W"][i] - inp.Ws[i]) > 0.5 * np.linalg.norm(inp.Ws[i])
        assert np.abs(g["new_b"][i]).max() > 0


@pytest.mark.parametrize("env,grid,mp", [({}, (1, 1), 1), ({"MBD_TC_PAIR": "2"}, (1, 1), 1), ({"MBD_TC_MH": "2", "MBD_TC_PAIR": "0"}, (1, 1), 1),
                                         ({"MBD_TC_MH": "1", "MBD_TC_PAIR": "0"}, (1, 1), 1), ({}, (2, 2), 2), ({}, (3, 5), 8),
                                         ({}, (4, 4), 2)])
def test_fused_update_equals_unfused_update_bit_for_bit(monkeypatch, net_case, env, grid, mp):
    # Same accumulator, same fmaf(scale, acc, w), one rounding to bf16: whether Eq. 1 runs inside the
    # product's epilogue / the reduction's tail or as a kernel of its own must not change a single bit.
    w, inp, o, eta = net_case
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    a = gpu_fc_step(w, inp, grid, max_partials=mp, fused=True, eta=eta)
    b = gpu_fc_step(w, inp, grid, max_partials=mp, fused=False, eta=eta)
    for i in range(3):
        assert np.array_equal(a["new_W"][i], b["new_W"][i]), f"W[{i}]"
        assert np.array_equal(a["new_b"][i], b["new_b"][i]), f"b[{i}]"


def test_planes_stored_by_tma_equal_planes_stored_from_registers(monkeypatch, net_case):
    # Short pieces of a sum over K leave the product as fp32 planes through TMA stores (a 3-D map over
    # partials[S][M][N]: rows of a ragged last tile -- M = 1000 here -- must be clipped, not land in the next
    # plane); the same planes written by the epilogue's own stores must agree bit for bit, and so must
    # everything computed from them.
    w, inp, o, eta = net_case
    grid, mp = (2, 3), 3
    plans = _plan_of(w, grid, mp)
    assert [(q["k_pieces"], q["tma_epilogue"]) for q in plans] == [(3, 2)] * 3, plans
    a = gpu_fc_step(w, inp, grid, max_partials=mp, fused=False, force_acts=oracle_hidden_acts(o), eta=eta)
    monkeypatch.setenv("MBD_TC_NO_TE", "1")
    assert all(q["tma_epilogue"] == 0 for q in _plan_of(w, grid, mp))
    b = gpu_fc_step(w, inp, grid, max_partials=mp, fused=False, force_acts=oracle_hidden_acts(o), eta=eta)
    for i in range(3):
        assert np.array_equal(a["dW"][i], b["dW"][i]) and np.array_equal(a["dY"][i], b["dY"][i]), i
        assert np.array_equal(a["new_W"][i], b["new_W"][i]), i
    compare_fc_step(a, o, TOL, False, init=inp, require_sized=True)


def test_planes_stored_from_the_idle_ring_equal_planes_stored_from_registers(monkeypatch):
    # A product whose work units all run at once (one per CTA) has an idle operand ring once its accumulator is
    # complete: the staging boxes of the TMA stores lie there, so pieces of any length leave by TMA.  The batch-256
    # network's first forward product (256 x 4096 x 9216, cut in 4 by the planner: 36 k-blocks per piece, 128 CTAs) is
    # such a launch; the same planes stored by the epilogue's own stores must give every bit of the step.
    from paper_1712_04432_b200 import mbd
    w = I.WORKLOADS["cfg2"]
    inp = I.make_inputs(w, seed=5)

    def fwd_plan():
        net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, 1, 1, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 2)
        q = net.plan(0, 0)
        net.close()
        return q
    q = fwd_plan()
    assert q["k_pieces"] == 4 and q["k_blocks"] // q["k_pieces"] >= 32 and q["tma_epilogue"] == 2, q
    a = gpu_fc_step(w, inp, (1, 1), max_partials=2, fused=True)
    monkeypatch.setenv("MBD_TC_NO_TE_RING", "1")
    assert fwd_plan()["tma_epilogue"] == 0
    b = gpu_fc_step(w, inp, (1, 1), max_partials=2, fused=True)
    for i in range(len(inp.Ws)):
        assert np.array_equal(a["act"][i], b["act"][i]) and np.array_equal(a["dY"][i], b["dY"][i]), i
        assert np.array_equal(a["new_W"][i], b["new_W"][i]) and np.array_equal(a["new_b"][i], b["new_b"][i]), i
    assert a["J"] == b["J"]


@pytest.mark.parametrize("grid,mp", [((1, 4), 2), ((4, 8), 4), ((8, 1), 2), ((4, 4), 2)])
@pytest.mark.parametrize("fused", [True, False])
def test_pieces_joined_in_tensor_memory_equal_planes_and_reduction(monkeypatch, net_case, grid, mp, fused):
    # Fewer partial sums than blocks (1 < S < P) and short pieces: the S pieces of a tile are accumulators of their
    # own in tensor memory and the product's epilogue adds them in ascending order before its tail operation.
    # Same pieces, same order as S fp32 planes and the reduction kernel: every bit must agree.
    w, inp, o, eta = net_case
    if grid[1] > 1:
        plans = _plan_of(w, grid, mp)
        assert [(q["k_pieces"], q["running_sum"]) for q in plans] == [(mp, 2)] * 3, plans
    a = gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta)
    monkeypatch.setenv("MBD_NO_JOIN", "1")
    assert all(q["running_sum"] == 0 for q in _plan_of(w, grid, mp))
    b = gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta)
    for i in range(3):
        assert np.array_equal(a["dY"][i], b["dY"][i]) and np.array_equal(a["new_W"][i], b["new_W"][i]), i
        if not fused:
            assert np.array_equal(a["dW"][i], b["dW"][i]), i
    compare_fc_step(a, o, TOL, fused, init=inp, require_sized=True)


def test_stand_alone_update_kernels_against_the_definition():
    # mbd_block_reduce with the SGD tail on one complete plane is Eq. 1 applied to a given gradient: bf16 weights
    # through the 16-byte path and (with a width that is not a multiple of 8) the element-wise path
    import torch
    from oracle import mbd_oracle as O
    from paper_1712_04432_b200 import mbd
    from tests.helpers import to_np
    r = np.random.default_rng(9)
    for (M, N) in [(40, 72), (24, 20)]:
        W0 = I.round_to_bf16(r.standard_normal((M, N)).astype(np.float32))
        G = r.standard_normal((M, N)).astype(np.float32) * 64
        W = to_dev(W0, True)
        mbd.block_reduce(torch.from_numpy(G).cuda(), W, mbd.TAIL_SGD, scale=-1.0 / 64)
        want = O.sgd(W0, G, 1.0, 64)                               # eta = 1, B = 64
        got = to_np(W)
        assert np.linalg.norm((got - W0) - (want - W0)) <= 3e-3 * np.linalg.norm(want - W0)   # bf16 rounding of W_new


@pytest.fixture(scope="module")
def long_k_case():
    # batch 4096 and 4096-wide layers: with two pieces per sum every piece is 32 k-blocks long, and every product
    # has more output tiles than CTA pairs -- the conditions under which the pieces are added as a running sum
    w = I.fc_workload((2048, 4096, 4096, 1000), 4096, "bf16", "relu_normal", name="running_sum")
    inp = I.make_inputs(w, seed=33)
    o = oracle_fc_step(w, inp)
    eta = update_sized_eta(o, inp.Ws, w.B)
    return w, inp, oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta), eta


@pytest.mark.parametrize("grid,mp", [((4, 4), 2), ((2, 8), 2)])
@pytest.mark.parametrize("fused", [True, False])
def test_running_sum_equals_planes_and_reduction_bit_for_bit(monkeypatch, long_k_case, grid, mp, fused):
    # With fewer partial sums than blocks (1 < S < P) and long pieces, the pieces of a product are added inside its
    # own epilogue: piece s adds its accumulator to the sum of pieces 0..s-1 that another CTA left in one fp32 plane,
    # and the last piece applies the tail operation (ReLU mask for backward-data, Eq. 1 or a plain store for
    # backward-weight).  Same ascending order as the reduction kernel over S planes: every bit must agree.
    from paper_1712_04432_b200 import mbd
    w, inp, o, eta = long_k_case
    runs = []
    for off in (False, True):
        if off:
            monkeypatch.setenv("MBD_NO_FIXUP", "1")
        net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, mp)
        plans = [net.plan(0, 2), net.plan(1, 2), net.plan(2, 1)]       # dW_1, dW_2 (K = B), dX_3 (K = 4096... of layer 2's outputs)
        net.close()
        assert [p["k_pieces"] for p in plans[:2]] == [2, 2]
        assert [p["running_sum"] for p in plans[:2]] == ([0, 0] if off else [1, 1]), plans
        runs.append(gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta))
    a, b = runs
    for i in range(3):
        assert np.array_equal(a["new_W"][i], b["new_W"][i]) and np.array_equal(a["dY"][i], b["dY"][i]), i
        if not fused:
            assert np.array_equal(a["dW"][i], b["dW"][i]), i
    compare_fc_step(a, o, TOL, fused, init=inp, require_sized=True)


def test_running_sum_of_the_backward_data_product(monkeypatch, long_k_case):
    # the ReLU-mask tail on the last piece: layer 2's input gradient sums over two row blocks of W_2 (K = 4096)
    from paper_1712_04432_b200 import mbd
    w, inp, o, eta = long_k_case
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, 4, 1, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 2)
    p = net.plan(1, 1)
    net.close()
    assert p["k_pieces"] == 2 and p["running_sum"] == 1, p
    a = gpu_fc_step(w, inp, (4, 1), max_partials=2, fused=True, force_acts=oracle_hidden_acts(o), eta=eta)
    monkeypatch.setenv("MBD_NO_FIXUP", "1")
    b = gpu_fc_step(w, inp, (4, 1), max_partials=2, fused=True, force_acts=oracle_hidden_acts(o), eta=eta)
    for i in range(3):
        assert np.array_equal(a["dY"][i], b["dY"][i]) and np.array_equal(a["new_W"][i], b["new_W"][i]), i
    compare_fc_step(a, o, TOL, True, init=inp, require_sized=True)
