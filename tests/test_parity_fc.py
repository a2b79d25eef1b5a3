"""Parity of the fully connected training step with the fp64 oracle, element by
element, through the C ABI: every tensor of every layer, for the grids of the
workloads, materialised and chained partial sums, fused and un-fused update."""
import numpy as np
import pytest

from paper_1712_04432_b200 import inputs as I
from tests.helpers import (compare_fc_step, gpu_fc_step, oracle_fc_step, oracle_hidden_acts, oracle_with_eta, rel_fro,
                           update_sized_eta)

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5     # fp32 check mode
TOL_BF16 = 1e-2    # bf16 storage, fp32 accumulation
# Free-running bf16 step (the device takes its ReLU decisions on its own stored activations).  fp32 (device)
# and fp64 (oracle) sums round a few stored activations to neighbouring bf16 values, which moves a few
# pre-activations of the next layer across zero; a flipped mask element is wrong by its full size, so a
# fraction f of flips costs about sqrt(f).  Measured, worst tensor below a ReLU, every grid of each case:
# 2.6e-3 (small_bf16, no flips), 6.0e-3 (cfg2, f = 1.3e-5 in layer 2), 1.09e-2 (cfg3, K = 25088, f = 6.6e-5).
# So every case but cfg3 meets the plain 1e-2 free-running as well; cfg3 gets 1.5 x its measured error, and
# meets 1e-2 with the ReLU decisions forced to the oracle's stored activations.
TOL_BF16_FREE = 1e-2
TOL_BF16_FREE_CFG3 = 1.65e-2


@pytest.fixture(scope="module")
def cfg1():
    w = I.WORKLOADS["cfg1"]
    inp = I.make_inputs(w, seed=0)
    return w, inp, oracle_fc_step(w, inp)


@pytest.mark.parametrize("grid", [(1, 1), (2, 2), (4, 1), (1, 4)])
@pytest.mark.parametrize("fused", [False, True])
def test_cfg1_fp32_all_grids(cfg1, grid, fused):
    w, inp, o = cfg1
    g = gpu_fc_step(w, inp, grid, max_partials=64, fused=fused)   # every block's partial materialised
    compare_fc_step(g, o, TOL_F32, fused)
    if not fused:
        # the update itself, not just the updated weights
        for i in range(3):
            delta = (g["new_W"][i] - inp.Ws[i].astype(np.float64)) / (-w.eta / w.B)
            assert rel_fro(delta, o["dWs"][i]) < 2e-3


def test_cfg1_same_result_for_every_grid_and_chaining(cfg1):
    w, inp, o = cfg1
    ref = gpu_fc_step(w, inp, (1, 1))
    for grid, mp in [((2, 2), 1), ((4, 1), 2), ((1, 4), 4), ((4, 4), 64)]:
        g = gpu_fc_step(w, inp, grid, max_partials=mp)
        for i in range(3):
            assert rel_fro(g["dW"][i], ref["dW"][i]) < 1e-6
            assert rel_fro(g["new_W"][i], ref["new_W"][i]) < 1e-6


@pytest.fixture(scope="module")
def small_bf16():
    # several 128x256 tiles with ragged edges in every dimension, K tails that are not
    # multiples of 64, a 1000-wide classifier like the large workloads
    w = I.fc_workload((1160, 520, 392, 1000), 328, "bf16", "relu_normal", name="small_bf16")
    inp = I.make_inputs(w, seed=3)
    return w, inp, oracle_fc_step(w, inp)


def sized(w, inp, o):
    """The oracle's step at a learning rate that moves every weight matrix by at least its own norm, so
    that the comparison of the applied update is sharp on bf16 weights (see helpers.update_checks)."""
    eta = update_sized_eta(o, inp.Ws, w.B)
    return oracle_with_eta(o, inp.Ws, inp.bs, w.B, eta), eta


@pytest.mark.parametrize("grid,mp", [((1, 1), 0), ((8, 1), 8), ((1, 8), 8), ((2, 4), 4), ((4, 2), 1), ((16, 16), 2),
                                     ((3, 5), 8)])
@pytest.mark.parametrize("fused", [False, True])
def test_small_bf16_grids(small_bf16, grid, mp, fused):
    w, inp, o = small_bf16
    o, eta = sized(w, inp, o)
    g = gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, eta=eta)
    compare_fc_step(g, o, TOL_BF16, fused, tol_below_relu=TOL_BF16_FREE, init=inp)
    g = gpu_fc_step(w, inp, grid, max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta)
    compare_fc_step(g, o, TOL_BF16, fused, init=inp, require_sized=True)


def test_small_bf16_against_unrounded_oracle(small_bf16):
    # Against the oracle WITHOUT storage rounding the forward pass (continuous in its inputs)
    # still meets the tolerance.  The gradients below a ReLU do not have to: a bf16 rounding
    # of X_i moves a few Y_i across zero, each flip changes one element of the mask by its
    # full size, and a fraction f of flipped elements costs about sqrt(f) in Frobenius norm.
    w, inp, _ = small_bf16
    o = oracle_fc_step(w, inp, exact=True)
    g = gpu_fc_step(w, inp, (1, 1))
    for i in range(3):
        ref = o["Ys"][i] if i == 2 else o["Xs"][i + 1]
        assert rel_fro(g["act"][i], ref.T) < TOL_BF16
    assert rel_fro(g["dY"][2], o["dYs"][2].T) < TOL_BF16       # top gradient: no mask above it
    assert rel_fro(g["dW"][2], o["dWs"][2]) < TOL_BF16
    for i in range(2):
        assert rel_fro(g["dW"][i], o["dWs"][i]) < 5e-2      # measured 3.3e-2: the unrounded oracle decides many ReLUs differently


def test_small_bf16_against_blocked_oracle(small_bf16):
    # the oracle formed block by block over the same grid (Appendix A.2) agrees as well
    w, inp, _ = small_bf16
    ob = oracle_fc_step(w, inp, blocked_grid=(4, 2))
    g = gpu_fc_step(w, inp, (4, 2), max_partials=8)
    compare_fc_step(g, ob, TOL_BF16)


def test_fp32_mode_on_ragged_shapes():
    w = I.fc_workload((200, 136, 72, 24), 40, "f32", "normal", name="small_f32")
    inp = I.make_inputs(w, seed=5)
    o = oracle_fc_step(w, inp)
    for grid in [(1, 1), (3, 2), (8, 5)]:
        compare_fc_step(gpu_fc_step(w, inp, grid, max_partials=64), o, TOL_F32)


def test_run_to_run_bitwise_reproducible(small_bf16):
    w, inp, _ = small_bf16
    a = gpu_fc_step(w, inp, (4, 4), max_partials=4, fused=True)
    b = gpu_fc_step(w, inp, (4, 4), max_partials=4, fused=True)
    for i in range(3):
        assert np.array_equal(a["new_W"][i], b["new_W"][i])
        assert np.array_equal(a["dY"][i], b["dY"][i])


@pytest.mark.parametrize("name,grid,mp", [("cfg2", (1, 1), 0), ("cfg2", (2, 4), 4), ("cfg2", (4, 2), 2), ("cfg2", (8, 1), 8),
                                          ("cfg2", (1, 8), 8), ("cfg3", (1, 1), 0), ("cfg3", (4, 4), 4), ("cfg3", (16, 1), 2),
                                          ("cfg3", (1, 16), 16)])
def test_full_size_fc_workloads(name, grid, mp):
    w = I.WORKLOADS[name]
    inp = I.make_inputs(w, seed=0)
    o, eta = sized(w, inp, oracle_fc_step(w, inp))
    g = gpu_fc_step(w, inp, grid, max_partials=mp, eta=eta)
    free = TOL_BF16_FREE_CFG3 if name == "cfg3" else TOL_BF16_FREE
    compare_fc_step(g, o, TOL_BF16, tol_below_relu=free, init=inp)
    g = gpu_fc_step(w, inp, grid, max_partials=mp, force_acts=oracle_hidden_acts(o), eta=eta)
    compare_fc_step(g, o, TOL_BF16, init=inp, require_sized=True)
    gf = gpu_fc_step(w, inp, grid, max_partials=mp, fused=True, force_acts=oracle_hidden_acts(o), eta=eta)
    compare_fc_step(gf, o, TOL_BF16, fused=True, init=inp, require_sized=True)
    gf = gpu_fc_step(w, inp, grid, max_partials=mp, fused=True)                    # the workload's own eta, free-running
    compare_fc_step(gf, oracle_with_eta(o, inp.Ws, inp.bs, w.B, w.eta), TOL_BF16, fused=True, tol_below_relu=free)


@pytest.mark.parametrize("case", range(10))
def test_seeded_random_networks_and_grids(case):
    # depth, widths (multiples of 8, so the tensor-core path applies), batch, grid, number of
    # materialised partials and dtype drawn from a seeded generator
    r = np.random.default_rng(4242 + case)
    L = int(r.integers(1, 5))
    dims = tuple(8 * int(r.integers(2, 90)) for _ in range(L + 1))
    B = 8 * int(r.integers(1, 40))
    dtype = "bf16" if case % 3 else "f32"
    P_r = int(r.integers(1, min(dims[1:]) // 8 + 1))
    P_c = int(r.integers(1, min(B, 12) + 1))
    mp = int(r.choice([1, 2, 4, 64]))
    fused = bool(r.integers(0, 2))
    w = I.fc_workload(dims, B, dtype, "relu_normal" if case % 2 else "normal", name=f"random{case}")
    inp = I.make_inputs(w, seed=100 + case)
    o = oracle_fc_step(w, inp)
    if dtype == "f32":
        compare_fc_step(gpu_fc_step(w, inp, (P_r, P_c), max_partials=mp, fused=fused), o, TOL_F32, fused, init=inp, bf16=False)
    else:
        o, eta = sized(w, inp, o)
        g = gpu_fc_step(w, inp, (P_r, P_c), max_partials=mp, fused=fused, force_acts=oracle_hidden_acts(o), eta=eta)
        compare_fc_step(g, o, TOL_BF16, fused, init=inp, require_sized=True)
