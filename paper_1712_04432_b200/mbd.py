"""Thin ctypes binding of libmbd.so: argument marshalling only.

Every step of the training path runs inside the CUDA library; torch is used
here for device memory and streams.  Loading fails loudly when the library has
not been built (`python -m paper_1712_04432_b200.build`); there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmbd.so")

OK, E_INVALID, E_GRID, E_ALLOC, E_CUDA, E_STATE, E_TIMEOUT, E_UNSUPPORTED, E_TOO_LARGE = range(9)
FC, CONV3X3 = 0, 1
SPLIT_MODEL, SPLIT_DOMAIN, SPLIT_BATCH = 0, 1, 2
F32, BF16 = 0, 1
LOSS_SOFTMAX_CE, LOSS_HALF_SSQ, LOSS_NONE = 0, 1, 2
T_ACT, T_DY, T_DW, T_DB, T_LOSS, T_PARTIALS, T_MASTER, T_VELOCITY, T_VELOCITY_BIAS = range(9)
ROWS_ALL, ROWS_INTERIOR, ROWS_BOUNDARY = range(3)

KERNEL_CLASSES = ["gemm_fwd", "gemm_bwd_data", "gemm_bwd_weight", "reduce_partials", "softmax_xent", "colsum",
                  "sgd_update", "halo_stage", "conv_fwd", "conv_bwd_data", "conv_bwd_weight", "other"]

EXPORTS = ["mbd_net_create", "mbd_net_destroy", "mbd_set_weights", "mbd_get_weights", "mbd_forward",
           "mbd_backward", "mbd_sgd_step", "mbd_train_step", "mbd_train_step_host", "mbd_comm_words", "mbd_get_tensor",
           "mbd_set_tensor", "mbd_poll_status", "mbd_profile_enable", "mbd_profile_read", "mbd_launch_count", "mbd_gemm_bf16", "mbd_gemm_bf16_noalloc", "mbd_selftest_timeout", "mbd_strerror",
           "mbd_train_step_host_begin", "mbd_train_step_host_end",
           "mbd_comm_time", "mbd_redistribute_time", "mbd_total_time", "mbd_grid_table", "mbd_choose_grid",
           "mbd_enable_master_weights", "mbd_enable_momentum", "mbd_block_gemm_bf16", "mbd_block_reduce", "mbd_softmax_xent",
           "mbd_conv_stage_input", "mbd_conv_forward_layer", "mbd_conv_backward_layer", "mbd_conv_outer_rows",
           "mbd_get_plan", "mbd_plan_product", "mbd_conv_forward_layer_rows", "mbd_conv_backward_layer_rows"]


class MbdError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({strerror(status)})")


class Layer(C.Structure):
    _fields_ = [("kind", C.c_int32), ("split", C.c_int32), ("relu", C.c_int32), ("bias", C.c_int32),
                ("d_in", C.c_int64), ("d_out", C.c_int64),
                ("C_in", C.c_int32), ("C_out", C.c_int32), ("H", C.c_int32), ("W", C.c_int32),
                ("kh", C.c_int32), ("kw", C.c_int32), ("stride", C.c_int32), ("reserved", C.c_int32)]


TAIL_STORE, TAIL_MASK, TAIL_SGD = range(3)


class Tail(C.Structure):
    """mbd_tail: the operation applied to a finished fp32 block (see include/mbd.h)."""
    _fields_ = [("op", C.c_int32), ("out_bf16", C.c_int32), ("relu", C.c_int32), ("reserved", C.c_int32),
                ("out_dev", C.c_void_p), ("ldo", C.c_int64), ("bias_dev", C.c_void_p), ("mask_dev", C.c_void_p),
                ("ldmask", C.c_int64), ("scale", C.c_float)]


class Plan(C.Structure):
    """mbd_plan: how one product of a layer is launched (see include/mbd.h)."""
    _fields_ = [("tile_m", C.c_int32), ("tile_n", C.c_int32), ("cta_pair", C.c_int32), ("k_pieces", C.c_int32),
                ("tma_epilogue", C.c_int32), ("ctas", C.c_int32), ("running_sum", C.c_int32), ("k_blocks", C.c_int32)]


class Words(C.Structure):
    _fields_ = [("allgather_y", C.c_int64), ("allreduce_dx", C.c_int64), ("allreduce_dw", C.c_int64),
                ("halo_fwd", C.c_int64), ("halo_bwd", C.c_int64)]


class Machine(C.Structure):
    """alpha: seconds per message; beta: seconds per word (one matrix element)."""
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double)]


class Times(C.Structure):
    _fields_ = [("allgather_y", C.c_double), ("allreduce_dx", C.c_double), ("allreduce_dw", C.c_double),
                ("halo_fwd", C.c_double), ("halo_bwd", C.c_double)]


class GridRow(C.Structure):
    _fields_ = [("P_r", C.c_int32), ("P_c", C.c_int32), ("comm_fwd", C.c_double), ("comm_bwd", C.c_double),
                ("comm", C.c_double), ("total", C.c_double)]


GRID_UNIFORM, GRID_CONV_BATCH = 0, 1
# Table 1 of the paper: 2 microseconds, 6 GB/s, 4-byte words
MACHINE_CORI_KNL = (2e-6, 4.0 / 6e9)
# One B200 on NVLink 5: measured peer copy 770 GB/s per direction, 2-byte words; the latency is a
# nominal few microseconds per collective step, not a measurement
MACHINE_B200_NVLINK5 = (5e-6, 2.0 / 770e9)

_lib = None


def lib():
    """The loaded library; raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1712_04432_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
        L.mbd_net_create.argtypes = [C.POINTER(Layer), i32, i64, i32, i32, i32, i32, i32, vp, C.POINTER(vp)]
        L.mbd_net_destroy.argtypes = [vp]
        L.mbd_set_weights.argtypes = [vp, i32, vp, vp]
        L.mbd_get_weights.argtypes = [vp, i32, vp, vp]
        L.mbd_forward.argtypes = [vp, vp, vp, vp]
        L.mbd_backward.argtypes = [vp, f32]
        L.mbd_sgd_step.argtypes = [vp, f32]
        L.mbd_train_step.argtypes = [vp, vp, vp, f32, vp]
        L.mbd_train_step_host.argtypes = [vp, vp, vp, f32, C.POINTER(f32)]
        L.mbd_train_step_host_begin.argtypes = [vp, vp, vp, f32]
        L.mbd_train_step_host_end.argtypes = [vp, C.POINTER(f32)]
        L.mbd_comm_words.argtypes = [C.POINTER(Layer), i32, i64, i32, i32, C.POINTER(Words)]
        f64 = C.c_double
        L.mbd_comm_time.argtypes = [C.POINTER(Layer), i32, i64, i32, i32, C.POINTER(Machine), C.POINTER(Times)]
        L.mbd_redistribute_time.argtypes = [i64, i32, i32, i64, C.POINTER(Machine), C.POINTER(f64)]
        L.mbd_total_time.argtypes = [f64, f64, f64, i32, C.POINTER(f64)]
        L.mbd_grid_table.argtypes = [C.POINTER(Layer), i32, i64, i32, C.POINTER(Machine), i32, f64, i32, i32,
                                     C.POINTER(GridRow), i32, C.POINTER(i32)]
        L.mbd_choose_grid.argtypes = [C.POINTER(Layer), i32, i64, i32, C.POINTER(Machine), i32, f64, i32, i32,
                                      C.POINTER(GridRow)]
        L.mbd_get_tensor.argtypes = [vp, i32, i32, vp, C.c_size_t]
        L.mbd_set_tensor.argtypes = [vp, i32, i32, vp, C.c_size_t]
        L.mbd_poll_status.argtypes = [vp]
        L.mbd_enable_master_weights.argtypes = [vp]
        L.mbd_enable_momentum.argtypes = [vp, C.c_float]
        L.mbd_block_gemm_bf16.argtypes = [i32, i64, i64, i64, vp, i64, vp, i64, C.POINTER(Tail), vp, vp]
        L.mbd_block_reduce.argtypes = [vp, i32, i64, i64, C.POINTER(Tail), i32, vp]
        L.mbd_softmax_xent.argtypes = [vp, i64, i64, vp, vp, i32, vp, i32, vp]
        L.mbd_conv_stage_input.argtypes = [vp, vp]
        L.mbd_conv_forward_layer.argtypes = [vp, i32, vp]
        L.mbd_conv_backward_layer.argtypes = [vp, i32, f32]
        L.mbd_conv_forward_layer_rows.argtypes = [vp, i32, i32, vp]
        L.mbd_conv_backward_layer_rows.argtypes = [vp, i32, i32, f32]
        L.mbd_conv_outer_rows.argtypes = [vp, i32, i32, i32, vp, C.c_size_t, i32]
        L.mbd_profile_enable.argtypes = [vp, i32]
        L.mbd_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(C.c_double)]
        L.mbd_launch_count.argtypes = [vp]
        L.mbd_launch_count.restype = i64
        L.mbd_get_plan.argtypes = [vp, i32, i32, C.POINTER(Plan)]
        L.mbd_plan_product.argtypes = [i32, i64, i64, i64, i32, i32, i32, C.POINTER(Plan)]
        L.mbd_gemm_bf16.argtypes = [i32, i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp, vp]
        L.mbd_gemm_bf16_noalloc.argtypes = [i32, i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
        L.mbd_selftest_timeout.argtypes = [i32, vp]
        L.mbd_strerror.argtypes = [i32]
        L.mbd_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().mbd_strerror(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        raise MbdError(status, what)


def fc_layers(dims: Sequence[int], bias: bool = True, relu: bool = True) -> List[Layer]:
    """Layer table of a fully connected stack d_0 -> ... -> d_L (model-split)."""
    return [Layer(kind=FC, split=SPLIT_MODEL, relu=int(relu), bias=int(bias), d_in=int(dims[i - 1]),
                  d_out=int(dims[i])) for i in range(1, len(dims))]


def conv_layers(n: int, C_: int, H: int, W: int, relu: bool = True, k=3, split: int = SPLIT_DOMAIN, channels=(),
                strides=()) -> List[Layer]:
    """n convolution layers on H x W input images, domain-split (row strips) or, with split=SPLIT_BATCH,
    batch-parallel on 1 x P (Section 3's improved case) or, with split=SPLIT_MODEL, model-parallel like a fully
    connected layer (output channels over P_r, batch over P_c: Eq. 8); `k` is the kernel size, k or (k_h, k_w), one value for all
    layers or one per layer; `channels` = (C_0, .., C_n) when the layers change the channel count (else C -> C);
    `strides` = one stride per layer (default 1): layer i then maps H_i x W_i images to H_i/s x W_i/s ones."""
    ks = [k] * n if isinstance(k, (int, tuple)) else list(k)
    assert len(ks) == n
    ks = [(q, q) if isinstance(q, int) else (int(q[0]), int(q[1])) for q in ks]
    ch = list(channels) if channels else [C_] * (n + 1)
    st = list(strides) if strides else [1] * n
    sp = [split] * n if isinstance(split, int) else [int(q) for q in split]      # one split kind for all layers, or one per layer
    assert len(ch) == n + 1 and len(st) == n and len(sp) == n
    out = []
    for i in range(n):
        assert H % st[i] == 0 and W % st[i] == 0
        Ho, Wo = H // st[i], W // st[i]
        out.append(Layer(kind=CONV3X3, split=sp[i], relu=int(relu), bias=0, d_in=ch[i] * H * W, d_out=ch[i + 1] * Ho * Wo,
                         C_in=ch[i], C_out=ch[i + 1], H=H, W=W, kh=ks[i][0], kw=ks[i][1], stride=st[i]))
        H, W = Ho, Wo
    return out


def _layer_array(layers: Sequence[Layer]):
    arr = (Layer * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = l
    return arr


def comm_words(layers: Sequence[Layer], B: int, P_r: int, P_c: int) -> List[Dict[str, int]]:
    """mbd_comm_words: per-layer word counts of Eq. 8 / Eq. 9 (host only, no GPU)."""
    out = (Words * len(layers))()
    _check(lib().mbd_comm_words(_layer_array(layers), len(layers), int(B), int(P_r), int(P_c), out), "mbd_comm_words")
    return [{k: int(getattr(w, k)) for k, _ in Words._fields_} for w in out]


def _machine(machine) -> Machine:
    return machine if isinstance(machine, Machine) else Machine(float(machine[0]), float(machine[1]))


def _row(r: GridRow) -> Dict[str, float]:
    return {k: (int(getattr(r, k)) if k in ("P_r", "P_c") else float(getattr(r, k))) for k, _ in GridRow._fields_}


def comm_time(layers: Sequence[Layer], B: int, P_r: int, P_c: int, machine) -> List[Dict[str, float]]:
    """mbd_comm_time: per-layer terms of Eq. 8 / Eq. 9 in seconds, latency terms included (host only)."""
    out = (Times * len(layers))()
    m = _machine(machine)
    _check(lib().mbd_comm_time(_layer_array(layers), len(layers), int(B), int(P_r), int(P_c), C.byref(m), out), "mbd_comm_time")
    return [{k: float(getattr(t, k)) for k, _ in Times._fields_} for t in out]


def redistribute_time(B: int, P_r: int, P_c: int, d: int, machine) -> float:
    """mbd_redistribute_time: Eq. 6 for a grid."""
    out = C.c_double()
    m = _machine(machine)
    _check(lib().mbd_redistribute_time(int(B), int(P_r), int(P_c), int(d), C.byref(m), C.byref(out)), "mbd_redistribute_time")
    return out.value


def total_time(compute: float, comm_fwd: float, comm_bwd: float, overlap: bool = False) -> float:
    out = C.c_double()
    _check(lib().mbd_total_time(float(compute), float(comm_fwd), float(comm_bwd), int(overlap), C.byref(out)), "mbd_total_time")
    return out.value


def grid_table(layers: Sequence[Layer], B: int, P: int, machine, policy: int = GRID_UNIFORM, compute: float = 0.0,
               overlap: bool = False, charge_redistribution: bool = True) -> List[Dict[str, float]]:
    """mbd_grid_table: one row per feasible factorisation P = P_r * P_c (Section 3)."""
    m = _machine(machine)
    arr = _layer_array(layers)
    n = C.c_int()
    args = (arr, len(layers), int(B), int(P), C.byref(m), int(policy), float(compute), int(overlap), int(charge_redistribution))
    _check(lib().mbd_grid_table(*args, None, 0, C.byref(n)), "mbd_grid_table")
    rows = (GridRow * max(n.value, 1))()
    _check(lib().mbd_grid_table(*args, rows, n.value, C.byref(n)), "mbd_grid_table")
    return [_row(rows[i]) for i in range(n.value)]


def choose_grid(layers: Sequence[Layer], B: int, P: int, machine, policy: int = GRID_UNIFORM, compute: float = 0.0,
                overlap: bool = False, charge_redistribution: bool = True) -> Dict[str, float]:
    """mbd_choose_grid: the factorisation with the least total time."""
    m = _machine(machine)
    best = GridRow()
    _check(lib().mbd_choose_grid(_layer_array(layers), len(layers), int(B), int(P), C.byref(m), int(policy), float(compute),
                                 int(overlap), int(charge_redistribution), C.byref(best)), "mbd_choose_grid")
    return _row(best)


def _ptr(t) -> Optional[int]:
    return None if t is None else C.c_void_p(t.data_ptr())


class Net:
    """One network on the current CUDA device (see include/mbd.h for semantics)."""

    def __init__(self, layers: Sequence[Layer], B: int, P_r: int = 1, P_c: int = 1, dtype: int = BF16,
                 loss: int = LOSS_SOFTMAX_CE, max_partials: int = 0, stream=None):
        import torch
        self._torch = torch
        self.layers = list(layers)
        self.L, self.B, self.P_r, self.P_c, self.dtype, self.loss = len(layers), int(B), P_r, P_c, dtype, loss
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self._h = C.c_void_p()
        self._keep = []
        _check(lib().mbd_net_create(_layer_array(layers), self.L, self.B, P_r, P_c, dtype, loss, max_partials,
                                    C.c_void_p(self.stream.cuda_stream), C.byref(self._h)), "mbd_net_create")

    # -- helpers
    @property
    def act_dtype(self):
        return self._torch.bfloat16 if self.dtype == BF16 else self._torch.float32

    def _wshape(self, i):
        l = self.layers[i]
        return (l.C_out, l.C_in, l.kh, l.kw) if l.kind == CONV3X3 else (l.d_out, l.d_in)

    def close(self):
        if self._h:
            lib().mbd_net_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI calls
    def set_weights(self, i: int, W, bias=None):
        assert W.is_cuda and W.is_contiguous() and W.dtype == self.act_dtype and tuple(W.shape) == self._wshape(i)
        if bias is not None:
            assert bias.is_cuda and bias.dtype == self._torch.float32 and bias.is_contiguous()
        _check(lib().mbd_set_weights(self._h, i, _ptr(W), _ptr(bias)), "mbd_set_weights")

    def get_weights(self, i: int, with_bias: bool = False):
        t = self._torch
        W = t.empty(self._wshape(i), dtype=self.act_dtype, device="cuda")
        b = t.empty(self.layers[i].d_out, dtype=t.float32, device="cuda") if with_bias else None
        _check(lib().mbd_get_weights(self._h, i, _ptr(W), _ptr(b)), "mbd_get_weights")
        return (W, b) if with_bias else W

    def forward(self, X, labels=None, loss_out=None):
        assert X.is_cuda and X.is_contiguous() and X.dtype == self.act_dtype
        if labels is not None:
            assert labels.is_cuda and labels.dtype == self._torch.int32 and labels.is_contiguous()
        self._keep = [X, labels, loss_out]      # the library reads X again during backward
        _check(lib().mbd_forward(self._h, _ptr(X), _ptr(labels), _ptr(loss_out)), "mbd_forward")

    # -- the convolution step piece by piece (see include/mbd.h)
    def conv_stage_input(self, X):
        assert X.is_cuda and X.is_contiguous() and X.dtype == self.act_dtype
        self._keep = [X]
        _check(lib().mbd_conv_stage_input(self._h, _ptr(X)), "mbd_conv_stage_input")

    def conv_forward_layer(self, layer: int, loss_out=None, rows: int = ROWS_ALL):
        """rows: ROWS_ALL, or ROWS_INTERIOR (the rows that read no halo row) / ROWS_BOUNDARY (the rest), see include/mbd.h"""
        _check(lib().mbd_conv_forward_layer_rows(self._h, layer, rows, _ptr(loss_out)), "mbd_conv_forward_layer_rows")

    def conv_backward_layer(self, layer: int, fused_eta: float = 0.0, rows: int = ROWS_ALL):
        _check(lib().mbd_conv_backward_layer_rows(self._h, layer, rows, float(fused_eta)), "mbd_conv_backward_layer_rows")

    def conv_outer_rows(self, which: int, layer: int, side: int, rows=None):
        """rows None: returns the first (side 0) / last (side 1) own row of every image, [B, W, C] bf16;
        otherwise writes `rows` into the upper / lower halo row."""
        t = self._torch
        l = self.layers[0]
        get = rows is None
        if get:
            rows = t.empty((self.B, l.W, l.C_out), dtype=t.bfloat16, device="cuda")
        assert rows.is_cuda and rows.is_contiguous() and rows.dtype == t.bfloat16
        _check(lib().mbd_conv_outer_rows(self._h, which, layer, side, _ptr(rows), rows.numel() * 2, int(not get)),
               "mbd_conv_outer_rows")
        return rows

    def enable_master_weights(self):
        """fp32 master copies of all weights from now on (see include/mbd.h)."""
        _check(lib().mbd_enable_master_weights(self._h), "mbd_enable_master_weights")

    def enable_momentum(self, mu: float):
        """Heavy-ball momentum from now on, velocities zero (see include/mbd.h)."""
        _check(lib().mbd_enable_momentum(self._h, float(mu)), "mbd_enable_momentum")

    def backward(self, fused_eta: float = 0.0):
        _check(lib().mbd_backward(self._h, float(fused_eta)), "mbd_backward")

    def sgd_step(self, eta: float):
        _check(lib().mbd_sgd_step(self._h, float(eta)), "mbd_sgd_step")

    def train_step(self, X, labels, eta: float, loss_out=None):
        """One fused step on device tensors, replayed from a CUDA graph after the first call."""
        assert X.is_cuda and X.is_contiguous() and X.dtype == self.act_dtype
        self._keep = [X, labels, loss_out]
        _check(lib().mbd_train_step(self._h, _ptr(X), _ptr(labels), float(eta), _ptr(loss_out)), "mbd_train_step")

    def train_step_host(self, X_host, labels_host, eta: float) -> float:
        """One step from host (ideally pinned) tensors; returns J."""
        assert not X_host.is_cuda and X_host.is_contiguous()
        out = C.c_float(0.0)
        _check(lib().mbd_train_step_host(self._h, _ptr(X_host), _ptr(labels_host), float(eta), C.byref(out)),
               "mbd_train_step_host")
        return out.value

    def train_step_host_begin(self, X_host, labels_host, eta: float):
        """Enqueue one step from host tensors (copy on the library's copy stream); at most two in flight.
        The host tensors must stay unchanged until the matching train_step_host_end()."""
        assert not X_host.is_cuda and X_host.is_contiguous()
        _check(lib().mbd_train_step_host_begin(self._h, _ptr(X_host), _ptr(labels_host), float(eta)), "mbd_train_step_host_begin")

    def train_step_host_end(self) -> float:
        """Wait for the oldest step begun; returns its J."""
        out = C.c_float(0.0)
        _check(lib().mbd_train_step_host_end(self._h, C.byref(out)), "mbd_train_step_host_end")
        return out.value

    def get_tensor(self, which: int, layer: int = 0, numel: Optional[int] = None):
        t = self._torch
        l = self.layers[min(layer, self.L - 1)]
        last = layer == self.L - 1
        conv = l.kind == CONV3X3
        if which == T_ACT:
            shape, dt = ((self.B, l.C_out, l.H // max(1, l.stride), l.W // max(1, l.stride)) if conv else (self.B, l.d_out)), \
                (t.float32 if (last and not conv) else self.act_dtype)
        elif which == T_DY:
            shape, dt = ((self.B, l.C_out, l.H // max(1, l.stride), l.W // max(1, l.stride)) if conv else (self.B, l.d_out)), self.act_dtype
        elif which in (T_DW, T_MASTER, T_VELOCITY):
            shape, dt = self._wshape(layer), t.float32
        elif which in (T_DB, T_VELOCITY_BIAS):
            shape, dt = (l.d_out,), t.float32
        elif which == T_LOSS:
            shape, dt = (self.B,), t.float32
        elif which == T_PARTIALS:
            shape, dt = (int(numel),), t.float32
        else:
            raise ValueError(which)
        out = t.empty(shape, dtype=dt, device="cuda")
        _check(lib().mbd_get_tensor(self._h, which, layer, _ptr(out), out.numel() * out.element_size()), "mbd_get_tensor")
        return out

    def set_tensor(self, which: int, layer: int, src):
        assert src.is_cuda and src.is_contiguous()
        _check(lib().mbd_set_tensor(self._h, which, layer, _ptr(src), src.numel() * src.element_size()), "mbd_set_tensor")

    def poll(self):
        _check(lib().mbd_poll_status(self._h), "mbd_poll_status")

    def profile_enable(self, on: bool = True):
        _check(lib().mbd_profile_enable(self._h, int(on)), "mbd_profile_enable")

    def profile_read(self) -> Dict[str, Dict[str, float]]:
        """Per kernel class: summed ms, launches, summed algorithmic work (flops or bytes)."""
        out = {}
        for k, name in enumerate(KERNEL_CLASSES):
            ms, n, w = C.c_double(0), C.c_int64(0), C.c_double(0)
            _check(lib().mbd_profile_read(self._h, k, C.byref(ms), C.byref(n), C.byref(w)), "mbd_profile_read")
            if n.value:
                out[name] = dict(ms=ms.value, launches=int(n.value), work=w.value)
        return out

    @property
    def launch_count(self) -> int:
        return int(lib().mbd_launch_count(self._h))

    def plan(self, layer: int, product: int) -> Dict[str, int]:
        """mbd_get_plan: tile shape, CTA pair, pieces of K, TMA epilogue, CTAs of product 0 / 1 / 2 of a layer."""
        p = Plan()
        _check(lib().mbd_get_plan(self._h, layer, product, C.byref(p)), "mbd_get_plan")
        return {k: int(getattr(p, k)) for k, _ in Plan._fields_}


PLAN_EXTRA_CUTS, PLAN_INTERMEDIATE, PLAN_BF16_RESULT = 1, 2, 4


def plan_product(variant: int, M: int, N: int, K: int, k_pieces: int = 1, flags: int = 0, num_sms: int = 148) -> Dict[str, int]:
    """mbd_plan_product: the launch plan of a stand-alone bf16 product, computed on the host (no device needed)."""
    p = Plan()
    _check(lib().mbd_plan_product(int(variant), C.c_int64(M), C.c_int64(N), C.c_int64(K), int(k_pieces), int(flags),
                                  int(num_sms), C.byref(p)), "mbd_plan_product")
    return {k: int(getattr(p, k)) for k, _ in Plan._fields_}


def gemm_bf16(variant: int, A, B, k_splits: int = 1, return_partials: bool = False):
    """mbd_gemm_bf16 on torch bf16 CUDA tensors.
    variant 0: A[M,K], B[N,K];  1: A[M,K], B[K,N];  2: A[K,M], B[K,N].  Returns float D[M,N]."""
    import torch
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1
    if variant == 0:
        M, K = A.shape; N = B.shape[0]; assert B.shape[1] == K
    elif variant == 1:
        M, K = A.shape; N = B.shape[1]; assert B.shape[0] == K
    else:
        K, M = A.shape; N = B.shape[1]; assert B.shape[0] == K
    D = torch.empty((M, N), dtype=torch.float32, device="cuda")
    parts = torch.empty((k_splits, M, N), dtype=torch.float32, device="cuda") if k_splits > 1 else None
    st = lib().mbd_gemm_bf16(variant, M, N, K, _ptr(A), A.stride(0), _ptr(B), B.stride(0), _ptr(D), D.stride(0),
                             k_splits, _ptr(parts), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    _check(st, "mbd_gemm_bf16")
    return (D, parts) if return_partials else D


def _tail(op: int, out, relu: bool = False, bias=None, mask=None, scale: float = 0.0) -> Tail:
    import torch
    assert out.is_cuda and out.stride(-1) == 1 and out.dtype in (torch.bfloat16, torch.float32)
    if mask is not None:
        assert mask.dtype == out.dtype and mask.stride(-1) == 1
    return Tail(op, int(out.dtype == torch.bfloat16), int(relu), 0, out.data_ptr(), out.stride(0),
                None if bias is None else bias.data_ptr(), None if mask is None else mask.data_ptr(),
                0 if mask is None else mask.stride(0), float(scale))


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def block_gemm(variant: int, A, B, out, op: int = TAIL_STORE, relu: bool = False, bias=None, mask=None, scale: float = 0.0,
               status=None):
    """mbd_block_gemm_bf16: one block product into `out` ([M, N] view, bf16 or float, row stride free) with the
    tail operation fused.  variant 0: A[M,K], B[N,K];  1: A[M,K], B[K,N];  2: A[K,M], B[K,N] (row strides free).
    `status` (int32 CUDA tensor of one zero): enqueue only; otherwise the call waits for the stream."""
    import torch
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1
    if variant == 0:
        M, K = A.shape; N = B.shape[0]; assert B.shape[1] == K
    elif variant == 1:
        M, K = A.shape; N = B.shape[1]; assert B.shape[0] == K
    else:
        K, M = A.shape; N = B.shape[1]; assert B.shape[0] == K
    assert tuple(out.shape) == (M, N)
    t = _tail(op, out, relu, bias, mask, scale)
    _check(lib().mbd_block_gemm_bf16(variant, M, N, K, _ptr(A), A.stride(0), _ptr(B), B.stride(0), C.byref(t),
                                     _ptr(status), _stream()), "mbd_block_gemm_bf16")
    return out


def block_reduce(parts, out, op: int = TAIL_STORE, relu: bool = False, bias=None, mask=None, scale: float = 0.0,
                 sync: bool = True):
    """mbd_block_reduce: sum of the S dense float planes parts[S, M, N] (or one plane [M, N]) in ascending
    order, then the tail operation into `out`."""
    import torch
    assert parts.is_cuda and parts.dtype == torch.float32 and parts.is_contiguous()
    if parts.dim() == 2:
        parts = parts.unsqueeze(0)
    S, M, N = parts.shape
    assert tuple(out.shape) == (M, N)
    t = _tail(op, out, relu, bias, mask, scale)
    _check(lib().mbd_block_reduce(_ptr(parts), S, M, N, C.byref(t), int(sync), _stream()), "mbd_block_reduce")
    return out


def softmax_xent(logits, labels, dY, per_sample, sync: bool = True):
    """mbd_softmax_xent: per-sample loss and dY = softmax - onehot of float logits [B, d]."""
    import torch
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    assert labels.dtype == torch.int32 and labels.is_cuda and dY.is_contiguous() and per_sample.dtype == torch.float32
    Bn, d = logits.shape
    _check(lib().mbd_softmax_xent(_ptr(logits), Bn, d, _ptr(labels), _ptr(dY), int(dY.dtype == torch.bfloat16),
                                  _ptr(per_sample), int(sync), _stream()), "mbd_softmax_xent")


def selftest_timeout(limit_ms: int = 50) -> int:
    """mbd_selftest_timeout: returns the status (E_TIMEOUT when the bounded wait fired)."""
    import torch
    return int(lib().mbd_selftest_timeout(int(limit_ms), C.c_void_p(torch.cuda.current_stream().cuda_stream)))


def gemm_bf16_noalloc(variant: int, A, B, k_splits: int = 1, out=None):
    """mbd_gemm_bf16_noalloc: as gemm_bf16, for callers that may not allocate device memory.
    The partial sums live in a fixed array inside the library (at most 4 Mi floats for
    k_splits * M * N); the library allocates nothing.  Pass `out` (float32 [M, N], CUDA) to
    keep this wrapper from allocating the result as well."""
    import torch
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1
    if variant == 0:
        M, K = A.shape; N = B.shape[0]
    elif variant == 1:
        M, K = A.shape; N = B.shape[1]
    else:
        K, M = A.shape; N = B.shape[1]
    D = out if out is not None else torch.empty((M, N), dtype=torch.float32, device="cuda")
    assert D.dtype == torch.float32 and tuple(D.shape) == (M, N) and D.stride(1) == 1
    st = lib().mbd_gemm_bf16_noalloc(variant, M, N, K, _ptr(A), A.stride(0), _ptr(B), B.stride(0), _ptr(D),
                                     D.stride(0), k_splits, C.c_void_p(torch.cuda.current_stream().cuda_stream))
    _check(st, "mbd_gemm_bf16_noalloc")
    return D
