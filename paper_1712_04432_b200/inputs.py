"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds NO arithmetic of the method: it only draws random numbers
(numpy Philox, counter based), rounds them to the storage type and describes
the five workloads.  Both the CUDA path and the CPU oracle are fed from the
arrays made here, so neither depends on the other.

The workloads stand in for the paper's AlexNet / ImageNet setting (Section 3):
fully connected stacks with classifier-head shapes, post-ReLU-like inputs and
uniform class labels, and a two-layer 3x3 convolution on 224x224 images.

Drawing order for one workload: X, then W_1..W_L, then the labels.
Layout: X is [B, d_0] row-major (row = sample, i.e. the paper's column of
X_1), W_i is [d_i, d_{i-1}] row-major, convolution input is NCHW and its
kernel [C_out, C_in, 3, 3].
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); the result
    is float32 holding exactly representable bf16 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-exact."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """float32 values of bf16 bit patterns."""
    return (np.ascontiguousarray(bits).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    name: str
    kind: str                      # "fc", "conv" or "mixed" (convolutions, then fully connected layers)
    dims: Tuple[int, ...]          # fc: d_0..d_L ; conv, mixed: (C, H, W) with C_in == C_out
    B: int
    dtype: str                     # "f32" or "bf16"
    x_dist: str                    # "normal" or "relu_normal"
    loss: str                      # "softmax_ce" or "half_ssq"
    eta: float = 0.01
    n_layers: int = 0
    grids: List[Tuple[int, int]] = field(default_factory=list)
    fc_dims: Tuple[int, ...] = ()  # mixed: C*H*W -> ... -> classes above the n_layers convolutions
    ksizes: Tuple = ()             # conv, mixed: kernel size per convolution, k or (k_h, k_w); empty = all 3 x 3
    channels: Tuple[int, ...] = () # conv: C_0 .. C_L (layer i maps C_{i-1} -> C_i); empty = dims[0] everywhere
    strides: Tuple[int, ...] = ()  # conv: stride per layer; empty = 1 everywhere

    def ksize(self, i: int) -> int:
        k = self.ksizes[i] if self.ksizes else 3
        assert isinstance(k, int)
        return k

    def kshape(self, i: int) -> Tuple[int, int]:
        k = self.ksizes[i] if self.ksizes else 3
        return (k, k) if isinstance(k, int) else (int(k[0]), int(k[1]))

    def stride(self, i: int) -> int:
        return self.strides[i] if self.strides else 1

    def out_hw(self, i: int) -> Tuple[int, int]:
        """Output image size of convolution layer i (dims[1:] is the network input's)."""
        H, W = self.dims[1], self.dims[2]
        for j in range(i + 1):
            H, W = H // self.stride(j), W // self.stride(j)
        return H, W

    def chan(self, i: int) -> int:
        """Channels of tensor i (0 = the input)."""
        return self.channels[i] if self.channels else self.dims[0]

    @property
    def L(self) -> int:
        if self.kind == "mixed":
            return self.n_layers + len(self.fc_dims) - 1
        return self.n_layers if self.kind == "conv" else len(self.dims) - 1


WORKLOADS = {
    "cfg1": Workload("cfg1", "fc", (784, 512, 512, 10), 64, "f32", "normal", "softmax_ce",
                     grids=[(1, 1), (2, 2), (4, 1), (1, 4)]),
    "cfg2": Workload("cfg2", "fc", (9216, 4096, 4096, 1000), 256, "bf16", "relu_normal",
                     "softmax_ce", grids=[(1, 1), (8, 1), (1, 8), (2, 4), (4, 2)]),
    "cfg3": Workload("cfg3", "fc", (25088, 4096, 4096, 1000), 512, "bf16", "relu_normal",
                     "softmax_ce", grids=[(1, 1), (4, 4), (16, 1), (1, 16)]),
    # eta: the half-sum-of-squares loss runs over 1e8 outputs; 1e-7 keeps repeated steps finite
    "cfg4": Workload("cfg4", "conv", (64, 224, 224), 32, "bf16", "normal", "half_ssq", eta=1e-7,
                     n_layers=2, grids=[(1, 1), (2, 1), (4, 1), (8, 1)]),
    "cfg5": Workload("cfg5", "fc", (8192,) * 9, 8192, "bf16", "normal", "softmax_ce",
                     grids=[(1, 1), (16, 16), (64, 4), (4, 64)]),
}
# Not a listed configuration: convolution layers the 64-channel kernels do not cover (5 x 5 and 3 x 3 kernels,
# 64 -> 128 -> 128 channels, 112 x 112 images), for measuring the general convolution path.
WORKLOADS["conv5x5"] = Workload("conv5x5", "conv", (64, 112, 112), 32, "bf16", "normal", "half_ssq", eta=1e-7, n_layers=2,
                                grids=[(1, 1), (2, 1), (4, 1), (8, 1)], ksizes=((5, 5), (3, 3)), channels=(64, 128, 128))
# The same two layers on 224 x 224 inputs, the first with stride 2 (its output is the 112 x 112 image of conv5x5).
WORKLOADS["conv5x5s2"] = Workload("conv5x5s2", "conv", (64, 224, 224), 32, "bf16", "normal", "half_ssq", eta=1e-7, n_layers=2,
                                  grids=[(1, 1), (2, 1), (4, 1), (8, 1)], ksizes=((5, 5), (3, 3)), channels=(64, 128, 128),
                                  strides=(2, 1))


def mixed_workload(C, H, W, n_conv, fc_dims, B, name="custom_mixed", grids=(), ksizes=(), channels=(), strides=()) -> "Workload":
    """n_conv convolutions (3x3, C -> C unless ksizes / channels / strides say otherwise) on H x W images, then a fully
    connected stack C_L*H_L*W_L -> fc_dims[0] -> ... -> fc_dims[-1] with softmax cross-entropy."""
    w = Workload(name, "mixed", (int(C), int(H), int(W)), int(B), "bf16", "normal", "softmax_ce",
                 n_layers=int(n_conv), grids=list(grids), ksizes=tuple(ksizes), channels=tuple(int(c) for c in channels),
                 strides=tuple(int(s) for s in strides))
    Ho, Wo = w.out_hw(int(n_conv) - 1)
    w.fc_dims = (w.chan(int(n_conv)) * Ho * Wo,) + tuple(int(x) for x in fc_dims)
    return w


# Beyond the five configurations: the integrated network of Section 2.4 in miniature (convolutions on
# row strips, a classifier head on row blocks of its matrices, one grid for both).
WORKLOADS["mixed"] = mixed_workload(64, 56, 56, 2, (1024, 1024, 1000), 256, name="mixed",
                                    grids=[(1, 1), (4, 4), (8, 1), (2, 8)])


# Not a listed configuration: the layer shapes of the network of the paper's Section 3 (five convolutions: 11 x 11 stride 4,
# 5 x 5, three 3 x 3; then a three-layer classifier), with what this library has in place of what it lacks: the three
# input channels padded to 8, no channel groups, no normalisation, and the two later pooling stages as strides of the
# second and fifth convolution (192 x 192 inputs: 48 x 48 after the first layer, 24 x 24, 12 x 12 at the classifier).
WORKLOADS["alexlike"] = mixed_workload(8, 192, 192, 5, (4096, 4096, 1000), 128, name="alexlike",
                                       grids=[(1, 1), (2, 8), (4, 4), (1, 16)],
                                       ksizes=((11, 11), (5, 5), (3, 3), (3, 3), (3, 3)), channels=(8, 96, 256, 384, 384, 256),
                                       strides=(4, 2, 1, 1, 2))


# The layers the paper singles out as needing no halo exchange (remark after Eq. 7): cfg4's stack with 1 x 1 kernels.
WORKLOADS["conv1x1"] = Workload("conv1x1", "conv", (64, 224, 224), 32, "bf16", "normal", "half_ssq", eta=1e-7,
                                n_layers=2, grids=[(1, 1), (2, 1), (4, 1), (8, 1)], ksizes=(1, 1))


def fc_workload(dims, B, dtype="bf16", x_dist="normal", name="custom") -> Workload:
    return Workload(name, "fc", tuple(int(d) for d in dims), int(B), dtype, x_dist, "softmax_ce")


def conv_workload(C, H, W, B, n_layers=2, dtype="bf16", name="custom_conv", ksizes=(), channels=(), strides=()) -> Workload:
    """`channels` = (C_0, .., C_L) for layers that change the channel count (then C = C_0)."""
    if channels:
        assert len(channels) == n_layers + 1 and channels[0] == C
    return Workload(name, "conv", (int(C), int(H), int(W)), int(B), dtype, "normal",
                    "half_ssq", n_layers=n_layers, ksizes=tuple(ksizes), channels=tuple(int(c) for c in channels),
                    strides=tuple(int(s) for s in strides))


@dataclass
class Inputs:
    X: np.ndarray                    # fc: [B, d_0] ; conv, mixed: [B, C, H, W]   (float32 values)
    Ws: List[np.ndarray]             # fc: [d_i, d_{i-1}] ; conv: [C_out, C_in, 3, 3] ; mixed: the kernels, then the matrices
    bs: List[Optional[np.ndarray]]   # zeros (fc layers) or None (conv layers)
    labels: Optional[np.ndarray]     # int32 [B] or None


def make_inputs(w: Workload, seed: int = 0) -> Inputs:
    """Draw one workload's tensors.  Values are float32; for dtype "bf16" they
    are already rounded to bf16 so that both paths start from identical data."""
    rng = np.random.Generator(np.random.Philox(key=seed))
    rnd = round_to_bf16 if w.dtype == "bf16" else (lambda a: np.ascontiguousarray(a, np.float32))
    if w.kind == "fc":
        d = w.dims
        X = rng.standard_normal((w.B, d[0]), dtype=np.float32)
        if w.x_dist == "relu_normal":
            np.maximum(X, 0.0, out=X)
        X = rnd(X)
        Ws, bs = [], []
        for i in range(1, len(d)):
            Wi = rng.standard_normal((d[i], d[i - 1]), dtype=np.float32)
            Wi *= np.float32(1.0 / np.sqrt(d[i - 1]))            # N(0, 1/fan_in)
            Ws.append(rnd(Wi))
            bs.append(np.zeros(d[i], np.float32))
        labels = rng.integers(0, d[-1], size=w.B, dtype=np.int64).astype(np.int32)
        return Inputs(X, Ws, bs, labels)
    C, H, Wd = w.dims
    X = rnd(rng.standard_normal((w.B, C, H, Wd), dtype=np.float32))
    Ws = []
    for i in range(w.n_layers):
        kh, kw = w.kshape(i)
        K = rng.standard_normal((w.chan(i + 1), w.chan(i), kh, kw), dtype=np.float32)
        K *= np.float32(np.sqrt(2.0 / (kh * kw * w.chan(i))))              # N(0, 2/(k_h k_w C_in))
        Ws.append(rnd(K))
    bs: List[Optional[np.ndarray]] = [None] * w.n_layers
    if w.kind != "mixed":
        return Inputs(X, Ws, bs, None)
    d = w.fc_dims
    for i in range(1, len(d)):
        Wi = rng.standard_normal((d[i], d[i - 1]), dtype=np.float32)
        Wi *= np.float32(1.0 / np.sqrt(d[i - 1]))
        Ws.append(rnd(Wi))
        bs.append(np.zeros(d[i], np.float32))
    labels = rng.integers(0, d[-1], size=w.B, dtype=np.int64).astype(np.int32)
    return Inputs(X, Ws, bs, labels)


def step_flops(w: Workload) -> int:
    """2 x MACs of the dense contractions one step needs: forward and
    backward-weight for every layer, backward-data for layers 2..L (layer 1 is the
    first layer of the whole network)."""
    if w.kind == "fc":
        d = w.dims
        macs = 0
        for i in range(1, len(d)):
            per = w.B * d[i] * d[i - 1]
            macs += (3 if i >= 2 else 2) * per
        return 2 * macs
    C, H, Wd = w.dims
    macs = 0
    for i in range(w.n_layers):
        per = w.B * w.out_hw(i)[0] * w.out_hw(i)[1] * w.chan(i) * w.chan(i + 1) * w.kshape(i)[0] * w.kshape(i)[1]
        macs += (3 if i >= 1 else 2) * per
    if w.kind == "mixed":
        d = w.fc_dims
        macs += sum(3 * w.B * d[i] * d[i - 1] for i in range(1, len(d)))
    return 2 * macs
