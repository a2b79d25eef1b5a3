"""Pins of the communication-time oracle (alpha-beta model, Eq. 3-9, and the grid choice of
Section 3) against what the paper and arithmetic fix: the pure schemes typed from their own
equations, closed forms, the constants of Table 1, limits, and brute force."""
import itertools
import math
from fractions import Fraction

import pytest

from oracle import comm_words as CW
from oracle import time_model as T

A, Bt = T.CORI_KNL_ALPHA, T.CORI_KNL_BETA


def fc(*dims):
    return [dict(kind="fc", d_in=a, d_out=b) for a, b in zip(dims[:-1], dims[1:])]


def conv(n, C, H, W, split="domain"):
    return [dict(kind="conv", C_in=C, C_out=C, H=H, W=W, kh=3, kw=3, split=split) for _ in range(n)]


NETS = {
    "fc3": fc(9216, 4096, 4096, 1000),
    "mlp": fc(784, 512, 512, 10),
    "conv2": conv(2, 64, 224, 224),
    "mixed": conv(2, 16, 32, 32) + fc(16 * 32 * 32, 256, 10),
}


def test_table1_constants():
    # latency 2 us; bandwidth 6 GB/s with 4-byte words
    assert A == 2e-6
    assert math.isclose(1.0 / Bt, 1.5e9)          # words per second


def test_ceil_log2():
    for p in range(1, 600):
        k = T.ceil_log2(p)
        assert 2 ** k >= p and (k == 0 or 2 ** (k - 1) < p)


@pytest.mark.parametrize("name", sorted(NETS))
def test_alpha_zero_is_beta_times_the_word_counts(name):
    # the integer word counts are pinned on their own (closed forms and the golden table)
    layers = NETS[name]
    for pr, pc in [(1, 1), (1, 8), (8, 1), (2, 4), (4, 4)]:
        words = CW.layer_words(layers, 64, pr, pc)
        exact = T.layer_words_exact(layers, 64, pr, pc)
        times = T.layer_times(layers, 64, pr, pc, 0.0, 1.0)
        for w, e, t in zip(words, exact, times):
            for k in T.TERMS:
                assert w[k] == math.ceil(e[k])
                assert math.isclose(t[k], float(e[k]), rel_tol=1e-15, abs_tol=0.0)


def test_beta_zero_counts_messages_closed_form():
    # L model-split layers: L all-gathers, 2(L-1) halves of dX all-reduces, 2L of dW all-reduces
    for L, pr, pc in itertools.product([1, 3, 5], [1, 2, 3, 8, 12], [1, 2, 5, 16]):
        layers = fc(*([64] * (L + 1)))
        got = T.comm_time(layers, 1024, pr, pc, 1.0, 0.0)
        want = (L + 2 * (L - 1)) * T.ceil_log2(pr) + 2 * L * T.ceil_log2(pc)
        assert got == want
    # domain-split layers: two halo messages (none for one strip) and 2 ceil(log2 P) per layer
    layers = conv(3, 8, 32, 32)
    assert T.comm_time(layers, 8, 4, 2, 1.0, 0.0) == 3 * (2 + 2 * 3)
    assert T.comm_time(layers, 8, 1, 8, 1.0, 0.0) == 3 * (2 * 3)


@pytest.mark.parametrize("name", ["fc3", "mlp"])
def test_integrated_formula_contains_the_pure_schemes(name):
    layers = NETS[name]
    for P in [2, 4, 7, 16]:
        # P_c = 1: pure model parallelism (Eq. 3); P_r = 1: pure batch parallelism (Eq. 4)
        assert math.isclose(T.comm_time(layers, 64, P, 1, A, Bt), T.eq3_model_time(layers, 64, P, A, Bt), rel_tol=1e-13)
        assert math.isclose(T.comm_time(layers, 64, 1, P, A, Bt), T.eq4_batch_time(layers, P, A, Bt), rel_tol=1e-13)


def test_domain_layers_contain_pure_domain_parallelism():
    layers = NETS["conv2"]
    for P in [1, 2, 4, 8]:
        assert math.isclose(T.comm_time(layers, 32, P, 1, A, Bt), T.eq7_domain_time(layers, 32, P, A, Bt), rel_tol=1e-13,
                            abs_tol=0.0)
    # Section 3, scenario (a): with B >= P the domain split never beats the batch split,
    # because it pays the same all-reduce plus the halos
    for P in [2, 4, 8]:
        assert T.eq7_domain_time(layers, 32, P, A, Bt) > T.eq4_batch_time(layers, P, A, Bt)


def test_one_by_one_convolution_needs_no_halo_exchange():
    # remark after Eq. 7: for a 1 x 1 convolution no communication is needed beyond the all-reduce of dW
    l = dict(kind="conv", C_in=64, C_out=64, H=56, W=56, kh=1, kw=1, split="domain")
    row = T.layer_times([l], 32, 4, 1, A, Bt)[0]
    assert row["halo_fwd"] == 0.0 and row["halo_bwd"] == 0.0
    assert math.isclose(row["allreduce_dw"], 2 * (A * 2 + Bt * 3 / 4 * 64 * 64), rel_tol=1e-13)
    assert math.isclose(T.eq7_domain_time([l], 32, 4, A, Bt), row["allreduce_dw"], rel_tol=1e-13)
    # a 3 x 3 kernel on the same activations does pay two halo messages
    l3 = dict(l, kh=3, kw=3)
    assert T.layer_times([l3], 32, 4, 1, 1.0, 0.0)[0]["halo_fwd"] == 1.0


def test_hand_computed_example():
    # two layers 6 -> 4 -> 2, B = 12, grid 2 x 3, alpha = 1, beta = 1/10 (by hand):
    # layer 1: all-gather 1 msg + 12/3 * 1/2 * 4 = 8 words; dW 2*2 msgs + 2 * 2/3 * 24/2 = 16 words
    # layer 2: all-gather 1 + 4 words; dX 2 msgs + 2 * 4 * 1/2 * 4 = 16 words; dW 4 msgs + 2 * 2/3 * 8/2 = 16/3 words
    rows = T.layer_times(fc(6, 4, 2), 12, 2, 3, 1.0, 0.1)
    assert math.isclose(rows[0]["allgather_y"], 1 + 0.8)
    assert rows[0]["allreduce_dx"] == 0.0
    assert math.isclose(rows[0]["allreduce_dw"], 4 + 1.6)
    assert math.isclose(rows[1]["allgather_y"], 1 + 0.4)
    assert math.isclose(rows[1]["allreduce_dx"], 2 + 1.6)
    assert math.isclose(rows[1]["allreduce_dw"], 4 + 16.0 / 30.0)


def test_eq5_ratio_and_crossover():
    # one interior 3x3 layer on 13x13x384 activations: batch volume / model volume = 2|W| / (3 B d)
    l = dict(kind="conv", C_in=384, C_out=384, H=13, W=13, kh=3, kw=3, split="model")
    first = dict(l)
    for B in [4, 12, 14, 64]:
        for P in [2, 8, 64]:
            model = T.layer_times([first, l], B, P, 1, 0.0, 1.0)[1]
            batch = T.layer_times([first, l], B, 1, P, 0.0, 1.0)[1]
            ratio = sum(batch.values()) / sum(model.values())
            assert math.isclose(ratio, 2 * 9 * 384 / (3 * B * 13 * 13), rel_tol=1e-12)
    # the paper's remark: model parallelism moves less for B <= 12 on this layer
    assert 2 * 9 * 384 / (3 * 12 * 169) > 1 > 2 * 9 * 384 / (3 * 14 * 169)


def test_redistribution_is_a_third_of_the_model_parallel_step():
    # Eq. 6 and the sentence after it: for a square interior layer the model-parallel step
    # (all-gather + all-reduce of dX) costs three times the redistribution, latency included
    d, B = 4096, 256
    layers = fc(d, d, d)
    for P in [2, 8, 64]:
        row = T.layer_times(layers, B, P, 1, A, Bt)[1]
        step = row["allgather_y"] + row["allreduce_dx"]
        assert math.isclose(step, 3.0 * T.redistribute_time(B, P, 1, d, A, Bt), rel_tol=1e-13)
    # literal Eq. 6
    assert math.isclose(T.redistribute_time(B, 8, 1, d, A, Bt), A * 3 + Bt * B * 7 / 8 * d, rel_tol=1e-13)


def test_weight_allreduce_shrinks_by_P_r():
    # remark after Eq. 8: against Eq. 4 the all-reduce volume of dW drops by the factor P_r
    # (exactly P_r * [(P-1)/P] / [(P_c-1)/P_c])
    layers = NETS["fc3"]
    for pr, pc in [(2, 4), (4, 16), (16, 32)]:
        P = pr * pc
        pure = sum(r["allreduce_dw"] for r in T.layer_times(layers, 2048, 1, P, 0.0, 1.0))
        integ = sum(r["allreduce_dw"] for r in T.layer_times(layers, 2048, pr, pc, 0.0, 1.0))
        want = Fraction(pr) * Fraction(P - 1, P) / Fraction(pc - 1, pc)
        assert math.isclose(pure / integ, float(want), rel_tol=1e-12)


def test_epoch_scaling():
    assert math.isclose(T.epoch_time(0.25, 1_200_000, 2048), 0.25 * 1_200_000 / 2048)


def test_total_time_limits_and_overlap():
    assert T.total_time(3.0, 1.0, 2.0, False) == 6.0
    assert T.total_time(0.0, 1.0, 2.0, True) == 3.0            # nothing to hide behind
    assert T.total_time(3.0, 0.0, 0.0, True) == 3.0            # nothing to hide
    assert T.total_time(3.0, 1.0, 1.5, True) == 4.0            # backward traffic fully hidden under 2/3 * 3
    assert T.total_time(3.0, 1.0, 2.5, True) == 4.5


def test_grid_table_lists_every_feasible_factorisation():
    layers = NETS["mlp"]                      # narrowest layer: 10 outputs
    tab = T.grid_table(layers, 64, 64, A, Bt)
    assert [(r["P_r"], r["P_c"]) for r in tab] == [(1, 64), (2, 32), (4, 16), (8, 8)]      # P_r <= 10
    tab = T.grid_table(layers, 4, 16, A, Bt)
    assert [(r["P_r"], r["P_c"]) for r in tab] == [(4, 4), (8, 2)]                        # P_c <= B
    # a number of processes with odd factors
    assert [(r["P_r"], r["P_c"]) for r in T.grid_table(NETS["fc3"], 64, 12, A, Bt)] == [(1, 12), (2, 6), (3, 4), (4, 3), (6, 2), (12, 1)]


def test_choice_is_the_brute_force_minimum_and_ties_go_to_small_P_r():
    for name, B, P in [("fc3", 2048, 512), ("fc3", 256, 8), ("mlp", 64, 16), ("conv2", 32, 8), ("mixed", 64, 32)]:
        layers = NETS[name]
        tab = T.grid_table(layers, B, P, A, Bt, compute=1e-3)
        best = T.choose_grid(layers, B, P, A, Bt, compute=1e-3)
        assert best["total"] == min(r["total"] for r in tab)
        assert best["P_r"] == min(r["P_r"] for r in tab if r["total"] == best["total"])
    # no communication cost at all: every grid ties, the smallest P_r wins
    assert T.choose_grid(NETS["fc3"], 64, 8, 0.0, 0.0)["P_r"] == 1


def test_large_fc_layers_prefer_an_integrated_grid():
    # Section 3: with many processes the integrated grid beats pure batch parallelism on the
    # fully connected layers (weights dominate)
    layers = NETS["fc3"]
    best = T.choose_grid(layers, 2048, 512, A, Bt)
    assert best["P_r"] > 1 and best["P_c"] > 1
    pure = T.comm_time(layers, 2048, 1, 512, A, Bt)
    assert pure / best["comm"] > 5.0
    # convolutions put on the same grid as model-split layers (large activations, few weights)
    # turn this around: their all-gathers dominate and the pure batch grid 1 x P wins
    convnet = conv(3, 64, 56, 56, split="model")
    assert T.choose_grid(convnet, 2048, 8, A, Bt)["P_r"] == 1
    assert T.choose_grid(convnet + layers, 2048, 8, A, Bt)["P_r"] == 1


def test_conv_batch_policy():
    layers = NETS["mixed"]
    B, P = 64, 32
    tab = {(r["P_r"], r["P_c"]): r for r in T.grid_table(layers, B, P, A, Bt, policy="conv_batch")}
    # convolutions cost the pure batch all-reduce whatever the grid of the fully connected layers
    conv_part = T.eq4_batch_time(layers[:2], P, A, Bt)
    fc_layers = layers[2:]
    for (pr, pc), r in tab.items():
        fc_rows = T.layer_times([layers[1]] + fc_layers, B, pr, pc, A, Bt)[1:]     # keeps "not the first layer"
        want = conv_part + sum(sum(x.values()) for x in fc_rows)
        if pr > 1:
            want += T.redistribute_time(B, pr, pc, 16 * 32 * 32, A, Bt)
        assert math.isclose(r["comm"], want, rel_tol=1e-12)
    # pure batch everywhere is the row P_r = 1
    assert math.isclose(tab[(1, P)]["comm"], T.eq4_batch_time([dict(l, split="model") for l in layers], P, A, Bt), rel_tol=1e-12)
    # needs B >= P
    assert T.grid_table(layers, 16, 32, A, Bt, policy="conv_batch") == []
    # without the redistribution charge the integrated rows get cheaper by exactly Eq. 6
    tab0 = {(r["P_r"], r["P_c"]): r for r in T.grid_table(layers, B, P, A, Bt, policy="conv_batch", charge_redistribution=False)}
    assert math.isclose(tab[(4, 8)]["comm"] - tab0[(4, 8)]["comm"], T.redistribute_time(B, 4, 8, 16 * 32 * 32, A, Bt), rel_tol=1e-9)
