"""The launch planner of the tensor-core products (host logic, no GPU): mbd_plan_product runs the cost model that
mbd_net_create runs for every product of Section 1 -- tile shape, CTA pairs, cuts of the reduction length K, and how the
partial sums over K (Appendix A.2) are added -- and reports it as mbd_get_plan does for a network."""
import random

import pytest

from paper_1712_04432_b200 import mbd

X, I, BF = mbd.PLAN_EXTRA_CUTS, mbd.PLAN_INTERMEDIATE, mbd.PLAN_BF16_RESULT
SMS = 148


def units(p, M, N):
    """work units of a plan: output tiles x pieces that are launched as work of their own"""
    tiles = -(-M // p["tile_m"]) * -(-N // p["tile_n"])
    return tiles * (1 if p["running_sum"] == 2 else p["k_pieces"])


def test_plans_of_the_benchmarked_products():
    # the 8192^3 products of the default benchmark on 16 x 16 with two partial sums
    p = mbd.plan_product(0, 8192, 8192, 8192, 1, X | I | BF, SMS)
    assert (p["tile_m"], p["tile_n"], p["cta_pair"], p["k_pieces"], p["ctas"]) == (512, 256, 1, 1, 148)
    for variant in (1, 2):
        p = mbd.plan_product(variant, 8192, 8192, 8192, 2, I | BF, SMS)
        assert (p["tile_m"], p["tile_n"], p["cta_pair"], p["k_pieces"], p["running_sum"]) == (256, 256, 1, 2, 1), p
    # every block's partial sum kept as a plane of its own: no running sum, 16 planes and a reduction launch
    p = mbd.plan_product(2, 8192, 8192, 8192, 16, BF, SMS)
    assert p["k_pieces"] == 16 and p["running_sum"] == 0
    # the batch-512 weight gradient 4096 x 25088 x 512: unsplit with the fused update behind TMA boxes; two short pieces
    # that are only intermediate stay in tensor memory; two pieces that must be kept leave as planes by TMA
    p = mbd.plan_product(2, 4096, 25088, 512, 1, I | BF, SMS)
    assert (p["tile_m"], p["cta_pair"], p["k_pieces"], p["tma_epilogue"], p["k_blocks"]) == (256, 1, 1, 1, 8)
    p = mbd.plan_product(2, 4096, 25088, 512, 2, I | BF, SMS)
    assert (p["k_pieces"], p["running_sum"], p["tma_epilogue"]) == (2, 2, 1)
    p = mbd.plan_product(2, 4096, 25088, 512, 2, BF, SMS)
    assert (p["k_pieces"], p["running_sum"], p["tma_epilogue"], p["tile_m"]) == (2, 0, 2, 128)
    # small batches: the planner cuts K by itself so that the few output tiles fill the SMs
    p = mbd.plan_product(0, 512, 4096, 25088, 1, X | I | BF, SMS)
    assert p["k_pieces"] == 2 and p["ctas"] == 128
    p = mbd.plan_product(0, 256, 4096, 9216, 1, X | I | BF, SMS)
    assert p["k_pieces"] == 4 and p["ctas"] == 128


@pytest.mark.parametrize("M,N,K,pieces", [(128, 1600, 430592, 21), (128, 1152, 430592, 29)])
def test_cuts_of_a_long_reduction_fill_the_sms(M, N, K, pieces):
    # weight gradients of general convolutions: C_out x (taps x channels) outputs, K = all pixels of the batch.  The cut
    # is any integer, not a power of two: 7 x 21 = 147 and 5 x 29 = 145 work units on 148 SMs (16 pieces would leave
    # 112 resp. 80 of them busy)
    p = mbd.plan_product(2, M, N, K, 1, X, SMS)
    assert p["k_pieces"] == pieces and 140 <= units(p, M, N) <= SMS and p["ctas"] == units(p, M, N)
    # without the permission the caller's pieces stand
    assert mbd.plan_product(2, M, N, K, 1, 0, SMS)["k_pieces"] == 1
    assert mbd.plan_product(2, M, N, K, 2, 0, SMS)["k_pieces"] == 2


def test_plan_invariants_over_random_products():
    rng = random.Random(1712)
    dims = [8, 64, 100, 128, 200, 256, 512, 1000, 1024, 4096, 8192, 25088, 36864]
    for _ in range(600):
        variant = rng.randrange(3)
        M, N, K = rng.choice(dims), rng.choice(dims), rng.choice(dims + [16, 40, 430592])
        k_req = rng.choice([1, 1, 2, 2, 4, 8, 16])
        flags = rng.randrange(8)
        sms = rng.choice([8, 132, 148])
        p = mbd.plan_product(variant, M, N, K, k_req, flags, sms)
        assert p == mbd.plan_product(variant, M, N, K, k_req, flags, sms), "deterministic"
        what = (variant, M, N, K, k_req, flags, sms, p)
        kb = -(-K // 64)
        assert p["k_blocks"] == kb
        assert p["tile_m"] in (128, 256, 512) and p["tile_n"] in (128, 256), what
        rows_per_cta = p["tile_m"] // (2 if p["cta_pair"] else 1)
        assert rows_per_cta in (128, 256), what
        if p["cta_pair"]:
            assert p["tile_n"] == 256 and p["ctas"] % 2 == 0, what
        assert 1 <= p["ctas"] <= sms, what
        assert p["ctas"] <= units(p, M, N) * (2 if p["cta_pair"] else 1), what
        asked = min(k_req, kb)
        assert 1 <= p["k_pieces"] <= kb and p["k_pieces"] % asked == 0, what
        if not flags & X:
            assert p["k_pieces"] == asked, what
        if not flags & I:
            assert p["running_sum"] == 0, what
        if p["running_sum"] == 1:                   # running sum through one plane: two long pieces on CTA pairs
            assert p["cta_pair"] and p["k_pieces"] == 2 and kb // 2 >= 32, what
        if p["running_sum"] == 2:                   # pieces as accumulators of their own: they must fit tensor memory
            assert p["k_pieces"] in (2, 4) and p["k_pieces"] * (rows_per_cta // 128) * p["tile_n"] <= 512, what
        if p["tma_epilogue"] == 1:                  # bf16 result through TMA boxes: 128 rows per CTA, nothing left for a reduction
            assert flags & BF and rows_per_cta == 128 and (p["k_pieces"] == 1 or p["running_sum"] == 2), what
        if p["tma_epilogue"] == 2:                  # planes stored by TMA: kept pieces that are short, or one work unit per CTA
            slots = sms // 2 if p["cta_pair"] else sms
            assert p["k_pieces"] > 1 and p["running_sum"] == 0 and rows_per_cta == 128, what
            assert kb // p["k_pieces"] < 32 or units(p, M, N) <= slots, what


def test_plan_query_rejects_bad_arguments():
    for args in [(3, 128, 128, 128, 1, 0, SMS), (-1, 128, 128, 128, 1, 0, SMS), (0, 0, 128, 128, 1, 0, SMS),
                 (0, 128, 0, 128, 1, 0, SMS), (0, 128, 128, 0, 1, 0, SMS), (0, 128, 128, 128, 0, 0, SMS),
                 (0, 128, 128, 128, 1, 8, SMS), (0, 128, 128, 128, 1, 0, 1)]:
        with pytest.raises(mbd.MbdError) as e:
            mbd.plan_product(*args)
        assert e.value.status == mbd.E_INVALID, args
    with pytest.raises(mbd.MbdError) as e:
        mbd.plan_product(0, 1 << 31, 128, 128, 1, 0, SMS)
    assert e.value.status == mbd.E_UNSUPPORTED


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_host_plan_is_the_plan_a_network_runs(name):
    # what mbd_plan_product computes without a device is what mbd_net_create plans for the products of a network on
    # the 1 x 1 grid: forward and backward-data may be cut further by the planner, every piece is intermediate, hidden
    # results are bf16
    import torch
    from paper_1712_04432_b200 import inputs
    w = inputs.WORKLOADS[name]
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, 1, 1, mbd.BF16, mbd.LOSS_SOFTMAX_CE, 2)
    L = len(w.dims) - 1
    for i in range(L):
        d_in, d_out = w.dims[i], w.dims[i + 1]
        if i < L - 1:                                             # (the last layer's logits are fp32: no TMA epilogue)
            assert net.plan(i, 0) == mbd.plan_product(0, w.B, d_out, d_in, 1, X | I | BF, sms), (i, "forward")
        if i > 0:
            assert net.plan(i, 1) == mbd.plan_product(1, w.B, d_in, d_out, 1, X | I | BF, sms), (i, "backward-data")
        assert net.plan(i, 2) == mbd.plan_product(2, d_out, d_in, w.B, 1, I | BF, sms), (i, "backward-weight")
    net.close()
