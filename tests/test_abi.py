"""CPU-side checks of the C ABI: the library loads, exports every symbol the header
declares, rejects bad arguments, and mbd_comm_words matches the oracle's closed forms and
the stored integers bit for bit.  No GPU is touched."""
import json
import os
import re

import pytest

from oracle import comm_words as CW
from paper_1712_04432_b200 import mbd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mbd.h")).read()
    declared = set(re.findall(r"MBD_API\s+[\w\s\*]+?\b(mbd_\w+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(mbd.EXPORTS)
    L = mbd.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_strerror():
    assert mbd.strerror(mbd.OK) == "ok"
    assert "grid" in mbd.strerror(mbd.E_GRID)


def _as_layers(rows):
    out = []
    for l in rows:
        if l["kind"] == "fc":
            out.append(mbd.Layer(kind=mbd.FC, split=mbd.SPLIT_MODEL, relu=1, bias=1, d_in=l["d_in"], d_out=l["d_out"]))
        else:
            out.append(mbd.Layer(kind=mbd.CONV3X3, split={"domain": mbd.SPLIT_DOMAIN, "batch": mbd.SPLIT_BATCH}.get(l["split"], mbd.SPLIT_MODEL),
                                 relu=1, bias=0, d_in=l["C_in"] * l["H"] * l["W"], d_out=l["C_out"] * l["H"] * l["W"],
                                 C_in=l["C_in"], C_out=l["C_out"], H=l["H"], W=l["W"], kh=l["kh"], kw=l["kw"], stride=l.get("stride", 0)))
    return out


def test_comm_words_match_stored_integers_exactly():
    gold = json.load(open(os.path.join(ROOT, "tests", "golden", "comm_words.json")))
    assert len(gold["cases"]) == 21
    for c in gold["cases"]:
        got = mbd.comm_words(_as_layers(c["layers"]), c["B"], c["P_r"], c["P_c"])
        assert got == c["rows"], (c["workload"], c["P_r"], c["P_c"])
        assert sum(sum(r.values()) for r in got) == c["total"]


@pytest.mark.parametrize("P_r,P_c", [(1, 1), (3, 5), (7, 2), (16, 16), (5, 1), (1, 9)])
def test_comm_words_match_oracle_on_odd_grids(P_r, P_c):
    dims = (1160, 520, 392, 1000)
    rows = [dict(kind="fc", split="model", d_in=dims[i - 1], d_out=dims[i]) for i in range(1, 4)]
    assert mbd.comm_words(_as_layers(rows), 328, P_r, P_c) == CW.layer_words(rows, 328, P_r, P_c)
    conv = [dict(kind="conv", split="domain", C_in=64, C_out=64, H=56, W=40, kh=3, kw=3)] * 2
    assert mbd.comm_words(_as_layers(conv), 30, P_r, P_c) == CW.layer_words(conv, 30, P_r, P_c)
    convm = [dict(kind="conv", split="model", C_in=8, C_out=24, H=13, W=13, kh=3, kw=3)] * 2
    assert mbd.comm_words(_as_layers(convm), 30, P_r, P_c) == CW.layer_words(convm, 30, P_r, P_c)


@pytest.mark.parametrize("P_r,P_c", [(1, 1), (4, 4), (2, 8), (16, 1), (3, 5)])
def test_comm_words_of_batch_parallel_convolutions(P_r, P_c):
    # Section 3's improved case: the convolutions forced onto 1 x P, the fully connected layers on P_r x P_c
    net = [dict(kind="conv", split="batch", C_in=64, C_out=64, H=56, W=56, kh=3, kw=3),
           dict(kind="conv", split="batch", C_in=64, C_out=64, H=56, W=56, kh=1, kw=1),
           dict(kind="fc", split="model", d_in=64 * 56 * 56, d_out=1024), dict(kind="fc", split="model", d_in=1024, d_out=1000)]
    got = mbd.comm_words(_as_layers(net), 256, P_r, P_c)
    assert got == CW.layer_words(net, 256, P_r, P_c)
    # the convolutions move what Eq. 4 moves on P processes, and nothing else
    assert sum(sum(r.values()) for r in got[:2]) == CW.eq4_batch_words(net[:2], P_r * P_c)
    assert all(r["halo_fwd"] == r["halo_bwd"] == r["allgather_y"] == r["allreduce_dx"] == 0 for r in got[:2])
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_words(_as_layers(net), 12, 4, 4)            # 16 processes, 12 samples
    assert e.value.status == mbd.E_GRID


@pytest.mark.parametrize("P_r,P_c", [(1, 1), (2, 3), (4, 1), (1, 6)])
def test_comm_words_of_strided_and_wide_kernels(P_r, P_c):
    # a 7 x 7 stride-2 layer: halo rows floor(7/2) = 3; the forward halo is X_W X_C wide (input), the backward one
    # Y_W Y_C (the output is half as wide); a model-split strided layer gathers an output of a quarter of the positions
    dom = [dict(kind="conv", split="domain", C_in=8, C_out=64, H=48, W=32, kh=7, kw=7, stride=2),
           dict(kind="conv", split="domain", C_in=64, C_out=64, H=24, W=16, kh=5, kw=3)]
    got = mbd.comm_words(_as_layers(dom), 12, P_r, P_c)
    assert got == CW.layer_words(dom, 12, P_r, P_c)
    if P_r > 1:
        assert got[0]["halo_fwd"] == -(-12 * 32 * 8 * 3 // P_c) and got[0]["halo_bwd"] == -(-12 * 16 * 64 * 3 // P_c)
        assert got[1]["halo_fwd"] == got[1]["halo_bwd"] == -(-12 * 16 * 64 * 2 // P_c)
    mod = [dict(kind="conv", split="model", C_in=8, C_out=24, H=12, W=12, kh=3, kw=3, stride=2)] * 1
    got = mbd.comm_words(_as_layers(mod), 12, P_r, P_c)
    assert got == CW.layer_words(mod, 12, P_r, P_c)
    assert got[0]["allgather_y"] == -(-12 * (P_r - 1) * 24 * 6 * 6 // (P_r * P_c))
    bad = _as_layers([dict(kind="conv", split="domain", C_in=8, C_out=8, H=9, W=12, kh=3, kw=3, stride=2)])
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_words(bad, 12, 1, 1)                # 9 rows do not divide by the stride
    assert e.value.status == mbd.E_INVALID


def test_comm_words_rejects_bad_arguments():
    layers = mbd.fc_layers((16, 8))
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_words(layers, 4, 1, 8)              # more batch blocks than samples
    assert e.value.status == mbd.E_GRID
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_words(layers, 4, 0, 1)
    assert e.value.status == mbd.E_GRID
    bad = [mbd.Layer(kind=mbd.FC, split=mbd.SPLIT_DOMAIN, d_in=8, d_out=8)]
    with pytest.raises(mbd.MbdError) as e:
        mbd.comm_words(bad, 4, 2, 1)                 # an FC layer has no halo
    assert e.value.status == mbd.E_INVALID


def test_comm_words_large_values_stay_exact():
    # products beyond 2^32 (and 2^53 for doubles): exact integer arithmetic required
    layers = mbd.fc_layers((1 << 20, 1 << 20, 1 << 20), bias=False)
    rows = [dict(kind="fc", split="model", d_in=1 << 20, d_out=1 << 20)] * 2
    B = (1 << 22) + 3
    assert mbd.comm_words(layers, B, 7, 3) == CW.layer_words(rows, B, 7, 3)
