"""Communication TIME model of the paper: the alpha-beta cost formulas Eq. 3, 4, 6, 7, 8, 9
with their latency terms, the per-epoch scaling of Section 3, and the choice of the process
grid P_r x P_c by evaluating the formula for every factorisation of P.

TEST INFRASTRUCTURE.  Plain Python: exact Fractions for the word counts, one float
multiplication per term for the times.  Shares nothing with the library's C++.

A time is  alpha * (number of messages) + beta * (number of words)  per collective:
  * all-gather of Y_i over the P_r group (Bruck): ceil(log2 P_r) messages, (B/P_c)(P_r-1)/P_r d_i words;
  * all-reduce of dX_i over the P_r group (ring, hence the factor 2 on BOTH terms), layers
    i >= 2 only: 2 ceil(log2 P_r) messages, 2 (B/P_c)(P_r-1)/P_r d_{i-1} words;
  * all-reduce of dW_i over the P_c group: 2 ceil(log2 P_c) messages, 2 (P_c-1)/P_c |W_i|/P_r words;
  * domain-split layers: one message per halo exchange (forward: input rows; backward: rows
    of the gradient of the output), (B/P_c) W C floor(k_h/2) words each, and the all-reduce
    of dW over all P processes: 2 ceil(log2 P) messages, 2 (P-1)/P |W_i| words.

Readings taken (the paper leaves these open):
  * logarithms are base 2, and ceil(log2 1) = 0: a group of one process sends nothing;
  * the word counts are NOT rounded here (the time formulas are over the reals); they
    coincide with the integer word counts whenever those are integral;
  * "d_{i-1}" is the size of the layer's own input (they differ when a pooling layer sits
    between two weighted layers);
  * the halo terms, latency included, vanish for a single strip (P_r = 1) and for a 1 x 1
    convolution (floor(k_h/2) = 0: "no communication is needed", remark after Eq. 7);
  * sums run over the layers that own a weight matrix;
  * overlap (Section 3, the variant with communication hidden behind back-propagation): the
    two all-reduces (two thirds of the products' communication) run behind the backward
    compute, taken as two thirds of the compute time (two of the three products per layer):
        T = T_comp + T_comm,fwd + max(0, T_comm,bwd - (2/3) T_comp).
    The paper gives no formula for this variant; this function is PARITY UNPINNED beyond its
    limits (no communication -> T_comp; no compute -> T_comm).
  * the speed-ups the paper quotes for AlexNet (2.1x / 5.0x / 2.5x / 9.7x / 2.0x) need its
    per-layer table and measured single-node times, which the paper does not print:
    PARITY UNPINNED for those numbers.
"""
from __future__ import annotations

from fractions import Fraction
from typing import Dict, List, Optional, Sequence, Tuple

from .comm_words import d_in, d_out, n_weights, out_hw

TERMS = ("allgather_y", "allreduce_dx", "allreduce_dw", "halo_fwd", "halo_bwd")

# Table 1: latency 2 microseconds, bandwidth 6 GB/s; a word is one fp32 element there.
CORI_KNL_ALPHA = 2e-6
CORI_KNL_BETA = 4.0 / 6e9


def ceil_log2(p: int) -> int:
    """Smallest k with 2**k >= p (0 for p = 1), in integers."""
    k = 0
    while (1 << k) < p:
        k += 1
    return k


def layer_messages(layers: Sequence[Dict], P_r: int, P_c: int) -> List[Dict[str, int]]:
    """Latency terms of Eq. 9 per layer, as message counts."""
    P = P_r * P_c
    rows = []
    for i, l in enumerate(layers):
        row = dict.fromkeys(TERMS, 0)
        if l.get("split", "model") == "batch":      # forced onto 1 x P (Section 3's improved case): Eq. 4's all-reduce alone
            row["allreduce_dw"] = 2 * ceil_log2(P)
        elif l.get("split", "model") == "model":
            row["allgather_y"] = ceil_log2(P_r)
            if i >= 1:
                row["allreduce_dx"] = 2 * ceil_log2(P_r)
            row["allreduce_dw"] = 2 * ceil_log2(P_c)
        else:
            if P_r > 1 and l["kh"] // 2 > 0:      # a 1 x 1 convolution exchanges nothing (remark after Eq. 7)
                row["halo_fwd"] = 1
                row["halo_bwd"] = 1
            row["allreduce_dw"] = 2 * ceil_log2(P)
        rows.append(row)
    return rows


def layer_words_exact(layers: Sequence[Dict], B: int, P_r: int, P_c: int) -> List[Dict[str, Fraction]]:
    """Bandwidth terms of Eq. 9 per layer, as exact fractions of words."""
    P = P_r * P_c
    rows = []
    for i, l in enumerate(layers):
        row = dict.fromkeys(TERMS, Fraction(0))
        if l.get("split", "model") == "batch":
            row["allreduce_dw"] = 2 * Fraction(P - 1, P) * n_weights(l)
        elif l.get("split", "model") == "model":
            row["allgather_y"] = Fraction(B, P_c) * Fraction(P_r - 1, P_r) * d_out(l)
            if i >= 1:
                row["allreduce_dx"] = 2 * Fraction(B, P_c) * Fraction(P_r - 1, P_r) * d_in(l)
            row["allreduce_dw"] = 2 * Fraction(P_c - 1, P_c) * Fraction(n_weights(l), P_r)
        else:
            if P_r > 1:
                row["halo_fwd"] = Fraction(B, P_c) * l["W"] * l["C_in"] * (l["kh"] // 2)
                row["halo_bwd"] = Fraction(B, P_c) * out_hw(l)[1] * l["C_out"] * (l["kh"] // 2)
            row["allreduce_dw"] = 2 * Fraction(P - 1, P) * n_weights(l)
        rows.append(row)
    return rows


def layer_times(layers: Sequence[Dict], B: int, P_r: int, P_c: int, alpha: float, beta: float) -> List[Dict[str, float]]:
    """Eq. 9 (Eq. 8 when no layer is domain-split), term by term and layer by layer, in seconds."""
    msgs = layer_messages(layers, P_r, P_c)
    words = layer_words_exact(layers, B, P_r, P_c)
    return [{t: alpha * m[t] + beta * float(w[t]) for t in TERMS} for m, w in zip(msgs, words)]


def comm_time(layers: Sequence[Dict], B: int, P_r: int, P_c: int, alpha: float, beta: float) -> float:
    return sum(sum(r.values()) for r in layer_times(layers, B, P_r, P_c, alpha, beta))


# ---- the pure schemes, typed from their own equations (used to pin the integrated formula) -----------

def eq3_model_time(layers: Sequence[Dict], B: int, P: int, alpha: float, beta: float) -> float:
    t = 0.0
    lg = ceil_log2(P)
    for i, l in enumerate(layers):
        t += alpha * lg + beta * float(Fraction(B * (P - 1) * d_out(l), P))
        if i >= 1:
            t += 2.0 * (alpha * lg + beta * float(Fraction(B * (P - 1) * d_in(l), P)))
    return t


def eq4_batch_time(layers: Sequence[Dict], P: int, alpha: float, beta: float) -> float:
    lg = ceil_log2(P)
    return sum(2.0 * (alpha * lg + beta * float(Fraction((P - 1) * n_weights(l), P))) for l in layers)


def eq7_domain_time(layers: Sequence[Dict], B: int, P: int, alpha: float, beta: float) -> float:
    t = 0.0
    lg = ceil_log2(P)
    for l in layers:
        if P > 1 and l["kh"] // 2 > 0:
            t += alpha + beta * B * l["W"] * l["C_in"] * (l["kh"] // 2)
            t += alpha + beta * B * out_hw(l)[1] * l["C_out"] * (l["kh"] // 2)
        t += 2.0 * (alpha * lg + beta * float(Fraction((P - 1) * n_weights(l), P)))
    return t


def redistribute_time(B: int, P_r: int, P_c: int, d: int, alpha: float, beta: float) -> float:
    """Eq. 6, stated for a grid: the all-gather that replicates the (B/P_c) x d block of
    activations over the P_r processes of a group when a batch-parallel layer is followed
    by a layer on a P_r x P_c grid.  With P_c = 1 this is Eq. 6 literally."""
    return alpha * ceil_log2(P_r) + beta * float(Fraction(B, P_c) * Fraction(P_r - 1, P_r) * d)


def epoch_time(iteration_time: float, N: int, B: int) -> float:
    """Section 3: an epoch over N samples takes N/B iterations."""
    return iteration_time * N / B


# ---- total time and the choice of the grid (Section 3) ------------------------------------------------

def comm_split_fwd_bwd(times: Sequence[Dict[str, float]]) -> Tuple[float, float]:
    """Forward-pass communication (all-gathers, forward halos) and backward-pass
    communication (all-reduces, backward halos) of a list of per-layer rows."""
    fwd = sum(r["allgather_y"] + r["halo_fwd"] for r in times)
    bwd = sum(r["allreduce_dx"] + r["allreduce_dw"] + r["halo_bwd"] for r in times)
    return fwd, bwd


def total_time(compute: float, comm_fwd: float, comm_bwd: float, overlap: bool) -> float:
    if not overlap:
        return compute + comm_fwd + comm_bwd
    return compute + comm_fwd + max(0.0, comm_bwd - 2.0 * compute / 3.0)


def divisors(P: int) -> List[int]:
    return [p for p in range(1, P + 1) if P % p == 0]


def grid_feasible(layers: Sequence[Dict], B: int, P_r: int, P_c: int) -> bool:
    """One sample per process at most along the batch; a model-split layer cannot be cut
    into more row blocks than it has outputs, a domain-split layer not into more strips
    than it has rows."""
    if P_c > B:
        return False
    for l in layers:
        if l.get("split", "model") == "model":
            if P_r > d_out(l):
                return False
        elif l.get("split") == "batch":
            if P_r * P_c > B:
                return False
        elif P_r > l["H"]:
            return False
    return True


def per_layer_times(layers: Sequence[Dict], B: int, grids: Sequence[Tuple[int, int]], alpha: float, beta: float
                    ) -> List[Dict[str, float]]:
    """Eq. 9 with a grid of its own for every layer (Section 3 uses 1 x P for the
    convolutions and P_r x P_c for the fully connected layers)."""
    rows = []
    for i, (l, (pr, pc)) in enumerate(zip(layers, grids)):
        # evaluate the layer in place so that "first layer" keeps its meaning
        rows.append(layer_times(layers[: i + 1], B, pr, pc, alpha, beta)[i])
    return rows


def grid_table(layers: Sequence[Dict], B: int, P: int, alpha: float, beta: float, policy: str = "uniform",
               compute: float = 0.0, overlap: bool = False, charge_redistribution: bool = True
               ) -> List[Dict]:
    """One row per feasible factorisation P = P_r * P_c, in ascending P_r."""
    table = []
    for pr in divisors(P):
        pc = P // pr
        if policy == "uniform":
            if not grid_feasible(layers, B, pr, pc):
                continue
            rows = layer_times(layers, B, pr, pc, alpha, beta)
            extra = 0.0
        elif policy == "conv_batch":
            fc = [l for l in layers if l["kind"] == "fc"]
            if P > B or not grid_feasible(fc, B, pr, pc):
                continue
            grids = [(1, P) if l["kind"] == "conv" else (pr, pc) for l in layers]
            # a batch-parallel convolution keeps all its weights: it is a model-split layer on a 1 x P grid
            as_model = [dict(l, split="model") if l["kind"] == "conv" else l for l in layers]
            rows = per_layer_times(as_model, B, grids, alpha, beta)
            extra = 0.0
            if charge_redistribution and pr > 1:
                first_fc = next((i for i, l in enumerate(layers) if l["kind"] == "fc"), None)
                if first_fc is not None and first_fc > 0:
                    extra = redistribute_time(B, pr, pc, d_in(layers[first_fc]), alpha, beta)
        else:
            raise ValueError(policy)
        fwd, bwd = comm_split_fwd_bwd(rows)
        fwd += extra
        table.append(dict(P_r=pr, P_c=pc, comm=fwd + bwd, comm_fwd=fwd, comm_bwd=bwd,
                          total=total_time(compute, fwd, bwd, overlap)))
    return table


def choose_grid(layers: Sequence[Dict], B: int, P: int, alpha: float, beta: float, **kw) -> Optional[Dict]:
    """The factorisation with the least total time; ties go to the smaller P_r."""
    table = grid_table(layers, B, P, alpha, beta, **kw)
    best = None
    for row in table:
        if best is None or row["total"] < best["total"]:
            best = row
    return best
