"""The library's communication-time model and grid choice (host only, no GPU) against the
oracle, term by term, on seeded random networks and grids; argument checking."""
import math
import random

import pytest

from oracle import time_model as T
from paper_1712_04432_b200 import mbd
from tests.test_abi import _as_layers

REL = 1e-12
MACHINES = [mbd.MACHINE_CORI_KNL, mbd.MACHINE_B200_NVLINK5, (0.0, 1.0), (1.0, 0.0)]


def random_net(r: random.Random, kind: str):
    if kind == "fc":
        dims = [r.choice([10, 64, 784, 1000, 4096, 9216]) for _ in range(r.randint(2, 6))]
        return [dict(kind="fc", d_in=a, d_out=b) for a, b in zip(dims[:-1], dims[1:])]
    convs = []
    for _ in range(r.randint(1, 4)):
        c = r.choice([3, 16, 64, 384])
        k = r.choice([1, 3, 3, 5])
        convs.append(dict(kind="conv", C_in=c, C_out=r.choice([16, 64, 256]), H=r.choice([13, 32, 224]), W=r.choice([13, 32, 224]),
                          kh=k, kw=k, split="domain" if kind == "conv_domain" else "model"))
    if kind == "mixed":
        convs += [dict(kind="fc", d_in=convs[-1]["C_out"] * convs[-1]["H"] * convs[-1]["W"], d_out=256), dict(kind="fc", d_in=256, d_out=10)]
    return convs


def close(a, b):
    return math.isclose(a, b, rel_tol=REL, abs_tol=1e-300)


@pytest.mark.parametrize("kind", ["fc", "conv_domain", "conv_model", "mixed"])
def test_comm_time_matches_oracle_term_by_term(kind):
    r = random.Random({"fc": 1, "conv_domain": 2, "conv_model": 3, "mixed": 4}[kind])
    for _ in range(40):
        rows = random_net(r, kind)
        B = r.choice([1, 12, 64, 328, 2048])
        P_r, P_c = r.choice([1, 2, 3, 4, 8, 16, 30]), r.choice([1, 2, 4, 5, 16])
        if P_c > B:
            continue
        a, b = r.choice(MACHINES)
        got = mbd.comm_time(_as_layers(rows), B, P_r, P_c, (a, b))
        want = T.layer_times(rows, B, P_r, P_c, a, b)
        for g, w in zip(got, want):
            for k in T.TERMS:
                assert close(g[k], w[k]), (rows, B, P_r, P_c, k, g[k], w[k])


def test_batch_parallel_convolutions_equal_their_own_1xP_grid():
    # Section 3's improved case, two ways: the layer marked batch-split on the network's P_r x P_c grid, and the same
    # layer as a model-split layer on a grid of its own, 1 x P (the oracle's per-layer form, written separately)
    r = random.Random(7)
    for _ in range(40):
        rows = random_net(r, "mixed")
        B = r.choice([64, 328, 2048])
        P_r, P_c = r.choice([1, 2, 4, 8]), r.choice([1, 2, 4, 8])
        a, b = r.choice(MACHINES)
        batch = [dict(l, split="batch") if l["kind"] == "conv" else l for l in rows]
        got = mbd.comm_time(_as_layers(batch), B, P_r, P_c, (a, b))
        grids = [(1, P_r * P_c) if l["kind"] == "conv" else (P_r, P_c) for l in rows]
        want = T.per_layer_times(rows, B, grids, a, b)
        same = T.layer_times(batch, B, P_r, P_c, a, b)
        for g, w, s in zip(got, want, same):
            for k in T.TERMS:
                assert close(g[k], w[k]) and close(s[k], w[k]), (rows, B, P_r, P_c, k, g[k], w[k], s[k])


def test_redistribution_and_total_time():
    for B, pr, pc, d in [(256, 8, 1, 4096), (2048, 16, 32, 9216), (64, 1, 64, 100), (30, 3, 5, 7)]:
        for a, b in MACHINES:
            assert close(mbd.redistribute_time(B, pr, pc, d, (a, b)), T.redistribute_time(B, pr, pc, d, a, b))
    for args in [(3.0, 1.0, 2.0, False), (0.0, 1.0, 2.0, True), (3.0, 1.0, 1.5, True), (3.0, 1.0, 2.5, True), (1e-3, 2e-4, 9e-4, True)]:
        assert close(mbd.total_time(*args), T.total_time(*args))


@pytest.mark.parametrize("policy", ["uniform", "conv_batch"])
def test_grid_table_and_choice_match_oracle(policy):
    r = random.Random(7 if policy == "uniform" else 11)
    pol = mbd.GRID_UNIFORM if policy == "uniform" else mbd.GRID_CONV_BATCH
    n_rows = 0
    for _ in range(40):
        kind = r.choice(["fc", "conv_model", "mixed"] if policy == "uniform" else ["fc", "mixed", "mixed"])
        rows = random_net(r, kind)
        B = r.choice([8, 64, 256, 2048])
        P = r.choice([1, 2, 6, 8, 12, 64, 512])
        a, b = r.choice(MACHINES[:2])
        compute = r.choice([0.0, 1e-3, 0.2])
        overlap = r.random() < 0.5
        charge = r.random() < 0.7
        want = T.grid_table(rows, B, P, a, b, policy=policy, compute=compute, overlap=overlap, charge_redistribution=charge)
        got = mbd.grid_table(_as_layers(rows), B, P, (a, b), pol, compute, overlap, charge)
        assert [(g["P_r"], g["P_c"]) for g in got] == [(w["P_r"], w["P_c"]) for w in want]
        for g, w in zip(got, want):
            for k in ("comm_fwd", "comm_bwd", "comm", "total"):
                assert close(g[k], w[k]), (rows, B, P, k)
        n_rows += len(want)
        best = T.choose_grid(rows, B, P, a, b, policy=policy, compute=compute, overlap=overlap, charge_redistribution=charge)
        if best is None:
            with pytest.raises(mbd.MbdError) as e:
                mbd.choose_grid(_as_layers(rows), B, P, (a, b), pol, compute, overlap, charge)
            assert e.value.status == mbd.E_GRID
        else:
            g = mbd.choose_grid(_as_layers(rows), B, P, (a, b), pol, compute, overlap, charge)
            # equal totals up to rounding may order differently; the chosen total must be the minimum
            assert close(g["total"], best["total"])
            if (g["P_r"], g["P_c"]) != (best["P_r"], best["P_c"]):
                other = next(w for w in want if w["P_r"] == g["P_r"])
                assert close(other["total"], best["total"])
    assert n_rows > 100


def test_paper_setting_picks_an_integrated_grid_for_the_classifier():
    # Table 1 machine, B = 2048 on 512 processes: the fully connected stack wants P_r > 1
    layers = mbd.fc_layers([9216, 4096, 4096, 1000])
    best = mbd.choose_grid(layers, 2048, 512, mbd.MACHINE_CORI_KNL)
    assert (best["P_r"], best["P_c"]) == (32, 16)
    table = {r["P_r"]: r for r in mbd.grid_table(layers, 2048, 512, mbd.MACHINE_CORI_KNL)}
    assert table[1]["comm"] / best["comm"] > 17.0


def test_argument_checks():
    layers = mbd.fc_layers([64, 32, 10])
    m = mbd.MACHINE_CORI_KNL
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_time(layers, 4, 1, 8, m)                   # more batch blocks than samples
    assert e.value.status == mbd.E_GRID
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_time(layers, 4, 1, 1, (-1.0, 1.0))          # negative latency
    assert e.value.status == mbd.E_INVALID
    with pytest.raises(mbd.MbdError) as e:
        mbd.grid_table(layers, 4, 0, m)
    assert e.value.status == mbd.E_INVALID
    with pytest.raises(mbd.MbdError) as e:
        mbd.grid_table(layers, 4, 8, m, policy=5)
    assert e.value.status == mbd.E_INVALID
    with pytest.raises(mbd.MbdError) as e:
        mbd.choose_grid(layers, 2, 64, m)                    # 64 processes, batch 2, narrowest layer 10: no grid
    assert e.value.status == mbd.E_GRID
    bad = [mbd.Layer(kind=mbd.FC, split=mbd.SPLIT_DOMAIN, relu=1, bias=1, d_in=8, d_out=8)]
    with pytest.raises(mbd.MbdError):
        mbd.comm_time(bad, 4, 2, 1, m)                       # an FC layer has no halo
    # the table call reports the count even when the caller's buffer is too small
    import ctypes as C
    n = C.c_int()
    mm = mbd.Machine(*m)
    rows = (mbd.GridRow * 1)()
    st = mbd.lib().mbd_grid_table(mbd._layer_array(layers), 2, 64, 8, C.byref(mm), 0, 0.0, 0, 1, rows, 1, C.byref(n))
    assert st == mbd.E_INVALID and n.value == 4
