"""Bandwidth (beta) terms of the paper's communication-cost formulas, as exact
integers of matrix elements ("words").

TEST INFRASTRUCTURE.  Each function restates one equation of the paper with
Python integers / Fractions; latency (alpha) terms are not part of the word
counts.

Readings taken (the paper leaves these open):
  * every sum runs over the layers that own a weight matrix, i = 1..L (the
    paper's lower limits i=0 in Eq. 4, 7, 8 have no W_0 to refer to);
  * a term is evaluated as ONE exact fraction (multiply first, divide last)
    and rounded up if it is not integral;
  * the halo terms are zero for a single strip (no neighbour), and both use
    floor(k_h/2) rows because the strips cut the height;
  * the all-reduce of dX is absent for the first layer (Section 2.2);
  * |W_i| excludes biases (Eq. 2 and the sentence after it).
"""
from __future__ import annotations

from fractions import Fraction
from math import ceil
from typing import Dict, List, Sequence


def n_weights(layer: Dict) -> int:
    """|W_i| of Eq. 2: k_h k_w X_C Y_C for a convolution, d_i d_{i-1} for FC."""
    if layer["kind"] == "conv":
        return layer["kh"] * layer["kw"] * layer["C_in"] * layer["C_out"]
    return layer["d_out"] * layer["d_in"]


def d_in(layer: Dict) -> int:
    if layer["kind"] == "conv":
        return layer["H"] * layer["W"] * layer["C_in"]          # Eq. 2, stride 1 padded
    return layer["d_in"]


def out_hw(layer: Dict):
    """Output image size of a convolution: a stride-s layer keeps every s-th position of its H x W input."""
    s = max(1, layer.get("stride", 1))
    return layer["H"] // s, layer["W"] // s


def d_out(layer: Dict) -> int:
    if layer["kind"] == "conv":
        return out_hw(layer)[0] * out_hw(layer)[1] * layer["C_out"]
    return layer["d_out"]


def _int(fr: Fraction) -> int:
    return int(ceil(fr))


def eq3_model_words(layers: Sequence[Dict], B: int, P: int) -> int:
    """Pure model parallelism: sum_{i=1..L} B (P-1)/P d_i + 2 sum_{i=2..L} B (P-1)/P d_{i-1}."""
    tot = 0
    for i, l in enumerate(layers):
        tot += _int(Fraction(B * (P - 1) * d_out(l), P))
        if i >= 1:
            tot += 2 * _int(Fraction(B * (P - 1) * d_in(l), P))
    return tot


def eq4_batch_words(layers: Sequence[Dict], P: int) -> int:
    """Pure batch parallelism: 2 sum_i (P-1)/P |W_i|."""
    return sum(_int(Fraction(2 * (P - 1) * n_weights(l), P)) for l in layers)


def eq7_domain_words(layers: Sequence[Dict], B: int, P: int) -> int:
    """Pure domain parallelism: halo rows forward and backward plus the
    weight-gradient all-reduce over all P processes."""
    tot = 0
    for l in layers:
        if P > 1:
            tot += B * l["W"] * l["C_in"] * (l["kh"] // 2)
            tot += B * out_hw(l)[1] * l["C_out"] * (l["kh"] // 2)          # Y_W Y_C floor(k_h/2) (Eq. 7)
        tot += _int(Fraction(2 * (P - 1) * n_weights(l), P))
    return tot


def layer_words(layers: Sequence[Dict], B: int, P_r: int, P_c: int) -> List[Dict[str, int]]:
    """Per-layer terms of Eq. 9 (which contains Eq. 8 as the case L_D empty).

    Layers with split == "model" (set L_M) contribute the all-gather of Y, the
    all-reduce of dX and the all-reduce of dW over P_c; layers with
    split == "domain" (set L_D) contribute the two halo exchanges and the
    all-reduce of dW over all P = P_r P_c processes; layers with
    split == "batch" are forced onto a 1 x P grid (Section 3: "we force P_r = 1,
    P_c = P for the convolutional layers") and contribute Eq. 4's all-reduce."""
    P = P_r * P_c
    rows = []
    for i, l in enumerate(layers):
        row = dict(allgather_y=0, allreduce_dx=0, allreduce_dw=0, halo_fwd=0, halo_bwd=0)
        if l.get("split", "model") == "batch":
            # Section 3, improved case: the layer runs on a 1 x P grid (pure batch parallelism): Eq. 4's term
            row["allreduce_dw"] = _int(Fraction(2 * (P - 1) * n_weights(l), P))
        elif l.get("split", "model") == "model":
            row["allgather_y"] = _int(Fraction(B * (P_r - 1) * d_out(l), P_r * P_c))
            if i >= 1:
                row["allreduce_dx"] = _int(Fraction(2 * B * (P_r - 1) * d_in(l), P_r * P_c))
            row["allreduce_dw"] = _int(Fraction(2 * (P_c - 1) * n_weights(l), P_c * P_r))
        else:
            if P_r > 1:
                row["halo_fwd"] = _int(Fraction(B * l["W"] * l["C_in"] * (l["kh"] // 2), P_c))
                row["halo_bwd"] = _int(Fraction(B * out_hw(l)[1] * l["C_out"] * (l["kh"] // 2), P_c))
            row["allreduce_dw"] = _int(Fraction(2 * (P - 1) * n_weights(l), P))
        rows.append(row)
    return rows


def total_words(layers: Sequence[Dict], B: int, P_r: int, P_c: int) -> int:
    return sum(sum(r.values()) for r in layer_words(layers, B, P_r, P_c))
