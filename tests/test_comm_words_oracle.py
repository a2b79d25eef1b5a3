"""Pins for the word-count oracle: hand arithmetic, the reductions between the
paper's formulas (Eq. 3, 4, 7, 8, 9) and the worked example under Eq. 5."""
from fractions import Fraction

import pytest

from oracle import comm_words as CW


def fc(dims):
    return [dict(kind="fc", split="model", d_in=dims[i - 1], d_out=dims[i]) for i in range(1, len(dims))]


def conv(C_in, C_out, H, W, k=3, split="domain"):
    return dict(kind="conv", split=split, C_in=C_in, C_out=C_out, H=H, W=W, kh=k, kw=k)


MLP = fc((784, 512, 512, 10))


def test_hand_worked_2x2_on_small_mlp():
    # Eq. 8 with B=64, P_r=P_c=2, written out by hand:
    #   all-gather   B/P_c (P_r-1)/P_r d_i        = 32 * 1/2 * {512, 512, 10}   = 8192, 8192, 160
    #   all-reduce dX 2 B/P_c (P_r-1)/P_r d_{i-1} = 2*32*1/2 * {-, 512, 512}    = 0, 16384, 16384
    #   all-reduce dW 2 (P_c-1)/P_c |W_i|/P_r     = 2*1/2*{401408,262144,5120}/2 = 200704, 131072, 2560
    rows = CW.layer_words(MLP, 64, 2, 2)
    assert [r["allgather_y"] for r in rows] == [8192, 8192, 160]
    assert [r["allreduce_dx"] for r in rows] == [0, 16384, 16384]
    assert [r["allreduce_dw"] for r in rows] == [200704, 131072, 2560]
    assert CW.total_words(MLP, 64, 2, 2) == 383648


def test_one_process_moves_nothing():
    for layers, B in ((MLP, 64), ([conv(64, 64, 224, 224)] * 2, 32)):
        assert CW.total_words(layers, B, 1, 1) == 0


@pytest.mark.parametrize("P", [2, 4, 8, 16])
def test_Pr_1_reduces_to_pure_batch_Eq4(P):
    layers = fc((9216, 4096, 4096, 1000))
    rows = CW.layer_words(layers, 256, 1, P)
    assert all(r["allgather_y"] == 0 and r["allreduce_dx"] == 0 for r in rows)
    assert CW.total_words(layers, 256, 1, P) == CW.eq4_batch_words(layers, P)
    # literal Eq. 4 for one layer: 2 (P-1)/P |W|
    assert rows[0]["allreduce_dw"] == Fraction(2 * (P - 1) * 9216 * 4096, P)


@pytest.mark.parametrize("P", [2, 4, 8, 16])
def test_Pc_1_reduces_to_pure_model_Eq3(P):
    layers = fc((9216, 4096, 4096, 1000))
    rows = CW.layer_words(layers, 256, P, 1)
    assert all(r["allreduce_dw"] == 0 for r in rows)
    assert CW.total_words(layers, 256, P, 1) == CW.eq3_model_words(layers, 256, P)
    assert rows[0]["allreduce_dx"] == 0                      # second sum of Eq. 3 starts at i=2


def test_allreduce_dw_shrinks_by_Pr():
    # the sentence after Eq. 8: the dW all-reduce volume drops by a factor P_r
    layers = fc((8192, 8192, 8192))
    for P_r, P_c in ((2, 4), (4, 4), (16, 16)):
        a = CW.layer_words(layers, 8192, P_r, P_c)
        b = CW.layer_words(layers, 8192, 1, P_c)
        for ra, rb in zip(a, b):
            assert ra["allreduce_dw"] * P_r == rb["allreduce_dw"]


def test_Eq9_with_empty_LD_is_Eq8_and_pure_domain_is_Eq7():
    # L_D empty: conv layers split by model behave like FC layers with Eq. 2's sizes
    c = conv(8, 16, 12, 12, split="model")
    as_fc = dict(kind="fc", split="model", d_in=12 * 12 * 8, d_out=12 * 12 * 16)
    r1 = CW.layer_words([c, c | dict(C_in=16, C_out=16)], 32, 4, 2)
    r2 = CW.layer_words([as_fc, as_fc | dict(d_in=12 * 12 * 16)], 32, 4, 2)
    assert [x["allgather_y"] for x in r1] == [x["allgather_y"] for x in r2]
    assert [x["allreduce_dx"] for x in r1] == [x["allreduce_dx"] for x in r2]
    assert r1[0]["allreduce_dw"] == 2 * 1 * (9 * 8 * 16) // (2 * 4)
    # all layers in L_D with P_c = 1: Eq. 9 collapses to Eq. 7
    layers = [conv(64, 64, 224, 224)] * 2
    for P in (2, 4, 8):
        assert CW.total_words(layers, 32, P, 1) == CW.eq7_domain_words(layers, 32, P)


def test_domain_terms_hand_values():
    # B X_W X_C floor(k/2) = 32 * 224 * 64 * 1 = 458752 ; 2 (P-1)/P |W| with |W| = 9*64*64 = 36864
    rows = CW.layer_words([conv(64, 64, 224, 224)] * 2, 32, 4, 1)
    for r in rows:
        assert r["halo_fwd"] == 458752 and r["halo_bwd"] == 458752
        assert r["allreduce_dw"] == 55296 and r["allgather_y"] == 0 and r["allreduce_dx"] == 0
    # a 1x1 convolution needs no halo (remark after Eq. 7)
    r = CW.layer_words([conv(64, 64, 56, 56, k=1)], 32, 4, 1)[0]
    assert r["halo_fwd"] == 0 and r["halo_bwd"] == 0


def test_Eq5_worked_example_threshold():
    # 3x3 filters on 13x13x384 activations: batch volume 2|W| vs model volume 3 B d.
    # ratio = 2 k_h k_w X_C / (3 B Y_H Y_W); the paper states model wins for B <= 12.
    thr = Fraction(2 * 9 * 384, 3 * 169)
    assert 13 < thr < 14
    Y_C = 384
    layer = [conv(384, Y_C, 13, 13, split="model")]
    W = CW.n_weights(layer[0])
    d = CW.d_out(layer[0])
    assert W == 9 * 384 * Y_C and d == 169 * Y_C
    for B in range(1, 40):
        batch, model = 2 * W, 3 * B * d
        assert (model < batch) == (B <= 13)
    assert 3 * 12 * d < 2 * W          # B = 12: model parallelism moves fewer words
    assert 3 * 14 * d > 2 * W          # B = 14: batch parallelism does
    # large-P limit of the library-style counts agrees: per interior layer the model
    # terms are B(P-1)/P (d_i + 2 d_{i-1}) = 3 B d (P-1)/P and the batch term 2 (P-1)/P |W|
    P = 64                                      # divides 12 * d = 12 * 169 * 384
    two = [layer[0], layer[0]]
    m = CW.layer_words(two, 12, P, 1)[1]
    b = CW.layer_words(two, 12, 1, 12)[1]      # P_c cannot exceed B; ratio (P-1)/P differs only
    assert m["allgather_y"] + m["allreduce_dx"] == Fraction(3 * 12 * d * (P - 1), P)
    assert b["allreduce_dw"] == Fraction(2 * 11 * W, 12)


def test_non_integral_terms_round_up():
    # d_L = 10 over P_r = 4 with B/P_c = 16: 16 * 3/4 * 10 = 120 exactly; 3 samples: 3*3*10/4 = 22.5 -> 23
    assert CW.layer_words(fc((8, 10)), 3, 4, 1)[0]["allgather_y"] == 23
    assert CW.layer_words(fc((8, 10)), 64, 4, 1)[0]["allgather_y"] == 480


def test_pure_schemes_bracket_the_mixed_grids_at_small_batch():
    layers = fc((9216, 4096, 4096, 1000))
    t = {g: CW.total_words(layers, 256, *g) for g in [(8, 1), (1, 8), (2, 4), (4, 2)]}
    assert t[(8, 1)] < t[(4, 2)] < t[(2, 4)] < t[(1, 8)]
    assert t[(8, 1)] == 5729024 and t[(1, 8)] == 102588416


def test_batch_split_layers_move_what_Eq4_moves_on_all_processes():
    # Section 3's improved case ("we force P_r = 1, P_c = P for the convolutional layers"): whatever the grid
    # of the other layers, a batch-split layer contributes Eq. 4's term for P = P_r P_c processes and no other:
    # by hand for |W| = 9*64*64 = 36864 on 4 x 2: 2 * 7/8 * 36864 = 64512
    conv = dict(kind="conv", split="batch", C_in=64, C_out=64, H=56, W=56, kh=3, kw=3)
    row = CW.layer_words([conv], 32, 4, 2)[0]
    assert row == dict(allgather_y=0, allreduce_dx=0, allreduce_dw=64512, halo_fwd=0, halo_bwd=0)
    for P_r, P_c in [(1, 8), (8, 1), (2, 4), (16, 2)]:
        rows = CW.layer_words([conv, conv], 64, P_r, P_c)
        assert sum(sum(r.values()) for r in rows) == CW.eq4_batch_words([conv, conv], P_r * P_c)
        # the same layer on a 1 x P grid as a model-split layer: Eq. 8 with P_r = 1 leaves that one term as well
        as_model = CW.layer_words([dict(conv, split="model")] * 2, 64, 1, P_r * P_c)
        assert rows == as_model
