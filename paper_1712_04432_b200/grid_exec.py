"""One training step of a fully connected stack executed for real over a P_r x P_c grid of PROCESSES
(Section 2.3, Fig. 5; Appendix A.1 / A.2): process (r, c) owns the row block W_i(r, :) of every weight
matrix and the batch block c of the samples.

    forward    Y_i(r, c) = W_i(r, :) X_i(:, c)                   block product, ReLU fused
               all-gather over the P_r group                     -> X_{i+1}(:, c)              Eq. 8, term 1
    backward   dX_i partial = W_i(r, :)^T dY_i(r, c)             block product, fp32
               all-reduce over the P_r group, ReLU mask          -> dY_{i-1}(:, c)             Eq. 8, term 2
               dW_i(r, :) partial = dY_i(r, c) X_i(:, c)^T       block product, fp32
               all-reduce over the P_c group, Eq. 1              -> W_i(r, :) updated          Eq. 8, term 3

Every arithmetic step runs in the library's kernels (mbd_block_gemm_bf16, mbd_block_reduce,
mbd_softmax_xent, all enqueue-only here: one status word is read at the end of the step);
torch.distributed only moves the blocks.  With the "nccl" backend the collectives run
on the device buffers; with "gloo" (tests: several processes sharing one GPU) they go through host copies.
The words every collective moves per process are counted from the buffers actually exchanged, so that
they can be compared with mbd_comm_words.

Rank layout: rank = c * P_r + r.

GridConv runs stacks of convolutions the same way under domain + batch parallelism (Section 2.2): one
process per row strip, halo rows exchanged with the neighbouring processes before every 3 x 3 layer,
weight gradients summed over all processes.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

from . import mbd


def grid_coords(rank: int, P_r: int, P_c: int):
    assert 0 <= rank < P_r * P_c
    return rank % P_r, rank // P_r


class GridComm:
    """The two process groups of one rank and the collectives of the step, with word accounting.

    Words per process follow the bandwidth-optimal algorithms the paper assumes: an all-gather over p
    processes of n words each receives (p - 1) n; an all-reduce of n words moves 2 (p - 1) / p * n."""

    def __init__(self, P_r: int, P_c: int, via_host: bool = False):
        import torch.distributed as dist
        self.dist = dist
        self.P_r, self.P_c = P_r, P_c
        assert dist.get_world_size() == P_r * P_c
        self.rank = dist.get_rank()
        self.r, self.c = grid_coords(self.rank, P_r, P_c)
        self.via_host = via_host
        # every process must create every group, in the same order
        self.row_group = self.col_group = None
        for c in range(P_c):
            g = dist.new_group([c * P_r + r for r in range(P_r)])
            if c == self.c:
                self.row_group = g
        for r in range(P_r):
            g = dist.new_group([c * P_r + r for c in range(P_c)])
            if r == self.r:
                self.col_group = g
        self.words: Dict[str, float] = {"allgather_y": 0.0, "allreduce_dx": 0.0, "allreduce_dw": 0.0}

    def all_gather_cols(self, block, out, kind="allgather_y", scratch=None):
        """out[:, r' * n : (r' + 1) * n] = block of process r' of the P_r group, for every r'.

        One collective into one buffer [P_r, m, n] (`scratch`, allocated here if not given) and one strided
        copy that puts block r' into its columns of `out` [m, P_r n]."""
        import torch
        p, (m, n) = self.P_r, block.shape
        assert out.shape[1] == p * n and out.shape[0] == m and out.is_contiguous()
        if p == 1:
            out.copy_(block)
            return out
        src = block.contiguous()
        if self.via_host:
            src = src.cpu()
            buf = torch.empty((p, m, n), dtype=src.dtype)
        else:
            buf = scratch if scratch is not None else torch.empty((p, m, n), dtype=src.dtype, device=src.device)
        assert tuple(buf.shape) == (p, m, n) and buf.is_contiguous()
        self.dist.all_gather_into_tensor(buf.view(p * m, n), src, group=self.row_group)
        out.view(m, p, n).copy_(buf.permute(1, 0, 2))
        self.words[kind] += (p - 1) * block.numel()
        return out

    def all_reduce_(self, t, over: str, kind: str):
        """In-place sum of a contiguous float tensor over the P_r ("rows") or the P_c ("cols") group."""
        p, g = (self.P_r, self.row_group) if over == "rows" else (self.P_c, self.col_group)
        if p == 1:
            return t
        assert t.is_contiguous()
        if self.via_host:
            h = t.cpu()
            self.dist.all_reduce(h, group=g)
            t.copy_(h)
        else:
            self.dist.all_reduce(t, group=g)
        self.words[kind] += 2.0 * (p - 1) / p * t.numel()
        return t

    def all_reduce_start(self, t, over: str, kind: str):
        """Starts the in-place sum of `t` and returns a handle for all_reduce_finish; what is enqueued or
        computed in between runs beside the exchange (Section 3: the all-reduce of dW_i can hide behind the
        products of the layers below)."""
        p, g = (self.P_r, self.row_group) if over == "rows" else (self.P_c, self.col_group)
        if p == 1:
            return (t, None, None)
        assert t.is_contiguous()
        self.words[kind] += 2.0 * (p - 1) / p * t.numel()
        if self.via_host:
            h = t.cpu()
            return (t, h, self.dist.all_reduce(h, group=g, async_op=True))
        return (t, None, self.dist.all_reduce(t, group=g, async_op=True))

    def all_reduce_finish(self, handle):
        t, h, work = handle
        if work is not None:
            work.wait()                  # nccl: the current stream waits; gloo: the host waits
            if h is not None:
                t.copy_(h)
        return t


class GridFC:
    """One process's share of a fully connected stack d_0 -> ... -> d_L (ReLU between layers, softmax
    cross-entropy on top, no bias): W_i(r, :) in bf16, and the step over its batch block."""

    def __init__(self, dims: Sequence[int], B: int, comm: GridComm, device="cuda"):
        import torch
        self.t = torch
        self.dims = [int(d) for d in dims]
        self.L = len(self.dims) - 1
        self.B = int(B)
        self.comm = comm
        P_r, P_c = comm.P_r, comm.P_c
        if self.B % P_c:
            raise ValueError("the batch must divide into P_c equal blocks")
        for d in self.dims[1:]:
            if d % P_r or (d // P_r) % 8:
                raise ValueError("every d_i must divide into P_r row blocks whose height is a multiple of 8")
        if self.dims[0] % 8:
            raise ValueError("d_0 must be a multiple of 8")
        self.m = self.B // P_c
        self.device = device
        self.W: List = [torch.zeros((self.dims[i + 1] // P_r, self.dims[i]), dtype=torch.bfloat16, device=device)
                        for i in range(self.L)]
        self.dW: List = [None] * self.L            # summed fp32 gradients of the last step (kept for inspection)
        # Every buffer of a step is allocated once, here: per layer the block product's output, the landing buffer
        # of the all-gather, the gathered activation, the fp32 summand of dX and of dW, the masked gradient.
        m, L, d = self.m, self.L, self.dims
        f32, bf = torch.float32, torch.bfloat16

        def buf(shape, dtype):
            return torch.empty(shape, dtype=dtype, device=device)

        self._blk = [buf((m, d[i + 1] // P_r), f32 if i == L - 1 else bf) for i in range(L)]
        self._gat = [buf((P_r, m, d[i + 1] // P_r), f32 if i == L - 1 else bf) if P_r > 1 else None for i in range(L)]
        self._act = [None] + [buf((m, d[i + 1]), f32 if i == L - 1 else bf) for i in range(L)]
        self._part = [buf((m, d[i]), f32) for i in range(L)]
        self._dYprev = [buf((m, d[i]), bf) for i in range(L)]
        self._g = [buf((d[i + 1] // P_r, d[i]), f32) for i in range(L)]
        self._dYtop = buf((m, d[L]), bf)
        self._per = buf((m,), f32)
        # word 0: bounded-wait status of the block products; word 1: the bits of this block's loss sum.  Read
        # back together, once, at the end of a step.
        self._tail = torch.zeros(2, dtype=torch.int32, device=device)
        self.status = self._tail[0:1]
        self._loss = self._tail[1:2].view(torch.float32)

    def _update(self, pending, scale: float):
        """Waits for the all-reduce of dW_i started earlier and applies Eq. 1 to the owned rows."""
        i, handle = pending
        g = self.comm.all_reduce_finish(handle)
        self.dW[i] = g
        mbd.block_reduce(g, self.W[i], mbd.TAIL_SGD, scale=scale, sync=False)

    def rows(self, i: int):
        """Row range of W_i (0-based layer i) this process owns."""
        h = self.dims[i + 1] // self.comm.P_r
        return self.comm.r * h, (self.comm.r + 1) * h

    def set_weights(self, i: int, W_full):
        """Takes this process's row block out of the full matrix [d_{i+1}, d_i] (bf16, any device)."""
        a, b = self.rows(i)
        self.W[i].copy_(W_full[a:b])

    def step(self, X_c, labels_c, eta: float, input_is_relu_output: bool = False):
        """One step on the batch block X_c [B / P_c, d_0] (bf16), labels_c int32.  Returns the sum of the
        losses of this block; the logits are kept in self.logits.  `input_is_relu_output`: the stack sits on
        top of other layers whose ReLU output X_c is -- the gradient with respect to X_c is then formed as
        well (masked by [X_c > 0]) and kept in self.dX0."""
        t, comm = self.t, self.comm
        m, L = self.m, self.L
        assert tuple(X_c.shape) == (m, self.dims[0]) and X_c.dtype == t.bfloat16
        acts = self._act
        acts[0] = X_c.contiguous()
        # ---- forward: block product, then the all-gather over the P_r group (Appendix A.1)
        for i in range(L):
            last = i == L - 1
            mbd.block_gemm(0, acts[i], self.W[i], self._blk[i], mbd.TAIL_STORE, relu=not last, status=self.status)
            comm.all_gather_cols(self._blk[i], acts[i + 1], scratch=self._gat[i])
        self.logits = acts[L]
        # ---- loss and top gradient (every process of a P_r group holds the full logits of its samples); the
        # block's losses are added, in sample order, by the library's reduction (S = m planes of one element)
        dY = self._dYtop
        mbd.softmax_xent(self.logits, labels_c, dY, self._per, sync=False)
        mbd.block_reduce(self._per.view(m, 1, 1), self._loss.view(1, 1), mbd.TAIL_STORE, sync=False)
        # ---- backward (Appendix A.2)
        scale = -float(eta) / self.B
        pending = None                                                  # the all-reduce of dW of the layer above, in flight
        for i in range(L - 1, -1, -1):
            a, b = self.rows(i)
            dY_r = dY[:, a:b]                                           # dY_i(r, c): this process's rows of layer i's output
            need_dx = i > 0 or input_is_relu_output
            hx = None
            if need_dx:
                part = self._part[i]
                mbd.block_gemm(1, dY_r, self.W[i], part, mbd.TAIL_STORE, status=self.status)       # W_i(r, :)^T dY_i(r, c), one summand
                hx = comm.all_reduce_start(part, "rows", "allreduce_dx")          # in flight beside the dW product below
            g = self._g[i]
            mbd.block_gemm(2, dY_r, acts[i], g, mbd.TAIL_STORE, status=self.status)                # dY_i(r, c) X_i(:, c)^T, one summand
            handle = comm.all_reduce_start(g, "cols", "allreduce_dw")          # runs beside the products of layer i - 1
            if pending is not None:
                self._update(pending, scale)
            pending = (i, handle)
            dY_prev = None
            if need_dx:
                part = comm.all_reduce_finish(hx)
                dY_prev = self._dYprev[i]
                mbd.block_reduce(part, dY_prev, mbd.TAIL_MASK, mask=acts[i], sync=False)   # ReLU derivative from the stored X_i
            dY = dY_prev
        self.dX0 = dY                                                   # None unless input_is_relu_output
        self._update(pending, scale)
        tail = self._tail.cpu()                      # (synchronises) status word and loss in one copy
        if int(tail[0]) != 0:                        # a bounded wait inside a product gave up
            self._tail.zero_()
            raise mbd.MbdError(mbd.E_TIMEOUT, "grid step")
        return float(tail[1:2].view(t.float32).item())


class GridConv:
    """One process's share of a stack of 64-channel convolutions under domain + batch parallelism
    (Section 2.2, Eq. 7 / Eq. 9): strip r (H / P_r rows) of the images of batch block c, held as a network of
    its own.  Before every 3 x 3 layer the strips' outer rows are exchanged with the processes above and
    below (a 1 x 1 layer needs none); the weight gradients are summed over all P processes.  Loss: half the
    sum of squares of the last layer's output."""

    def __init__(self, ksizes: Sequence[int], C_: int, H: int, W: int, B: int, comm: GridComm,
                 loss: int = mbd.LOSS_HALF_SSQ):
        import torch
        self.t = torch
        self.comm = comm
        self.loss = loss
        P_r, P_c = comm.P_r, comm.P_c
        if B % P_c or P_r > H:
            raise ValueError("the batch must divide into P_c blocks and every strip needs a row")
        self.ksizes = [int(k) for k in ksizes]
        self.L = len(self.ksizes)
        # strip r of the image: the balanced range of rows [floor(r H / P_r), floor((r + 1) H / P_r))
        self.h0, self.h1 = (comm.r * H) // P_r, ((comm.r + 1) * H) // P_r
        self.C, self.Hs, self.W, self.m = int(C_), self.h1 - self.h0, int(W), B // P_c
        self.net = mbd.Net(mbd.conv_layers(self.L, C_, self.Hs, W, k=self.ksizes), self.m, 1, 1, mbd.BF16, loss, 0)
        comm.words.setdefault("halo_fwd", 0.0)
        comm.words.setdefault("halo_bwd", 0.0)
        self.dK: List = [None] * self.L

    def set_weights(self, i: int, K):
        self.net.set_weights(i, K)

    def _exchange_start(self, which: int, layer: int, kind: str):
        """First own rows go to the process above, last own rows to the process below (started here, not waited
        for).  Counted as the paper counts it: one boundary of (B / P_c) W C words."""
        comm, dist, t = self.comm, self.comm.dist, self.t
        if comm.P_r == 1:
            return None
        up = comm.rank - 1 if comm.r > 0 else None
        down = comm.rank + 1 if comm.r < comm.P_r - 1 else None
        ops, got = [], {}
        for side, peer in ((0, up), (1, down)):
            if peer is None:
                continue
            out = self.net.conv_outer_rows(which, layer, side)
            if comm.via_host:
                out = out.cpu()
            inc = t.empty_like(out)
            got[side] = inc
            ops.append(dist.P2POp(dist.isend, out, peer))
            ops.append(dist.P2POp(dist.irecv, inc, peer))
        comm.words[kind] += self.m * self.W * self.C
        return (dist.batch_isend_irecv(ops), got, which, layer)

    def _exchange_finish(self, handle):
        """What arrived becomes this strip's halo rows."""
        if handle is None:
            return
        reqs, got, which, layer = handle
        for req in reqs:
            req.wait()
        for side, inc in got.items():
            self.net.conv_outer_rows(which, layer, side, rows=inc.cuda() if self.comm.via_host else inc)

    def step(self, X_local, eta: float):
        """One step on this process's strip X_local [B / P_c, C, H / P_r, W] (bf16).  Returns its share of J."""
        J = self.forward(X_local)
        self.backward(eta)
        return J

    def forward(self, X_local):
        t, net, L = self.t, self.net, self.L
        J = t.zeros(1, dtype=t.float32, device="cuda")
        net.conv_stage_input(X_local)
        for i in range(L):
            loss_out = J if i == L - 1 else None
            if self.ksizes[i] == 3 and self.comm.P_r > 1:
                # halo rows of the layer's input (Eq. 7, term 1) travel while the rows that need none are computed
                # (Section 2.2: "the halo exchange can be overlapped with the interior computation")
                h = self._exchange_start(mbd.T_ACT, i - 1, "halo_fwd")
                net.conv_forward_layer(i, None, rows=mbd.ROWS_INTERIOR)
                self._exchange_finish(h)
                net.conv_forward_layer(i, loss_out, rows=mbd.ROWS_BOUNDARY)
            else:
                net.conv_forward_layer(i, loss_out)
        return float(J.item()) if self.loss == mbd.LOSS_HALF_SSQ else 0.0

    def backward(self, eta: float):
        """Backward pass and update.  With LOSS_NONE the gradient of the last layer's output must have been
        set before (net.set_tensor(T_DY, L - 1, ...))."""
        t, net, comm, L = self.t, self.net, self.comm, self.L
        for i in range(L - 1, -1, -1):
            if i > 0 and self.ksizes[i] == 3 and comm.P_r > 1:
                h = self._exchange_start(mbd.T_DY, i, "halo_bwd")   # halo rows of dY_i (Eq. 7, term 2), in flight beside
                net.conv_backward_layer(i, 0.0, rows=mbd.ROWS_INTERIOR)     # the interior rows of the input gradient
                self._exchange_finish(h)
                net.conv_backward_layer(i, 0.0, rows=mbd.ROWS_BOUNDARY)     # its boundary rows, then the weight gradient
            else:
                net.conv_backward_layer(i, 0.0)
        P = comm.P_r * comm.P_c
        for i in range(L):                                            # all-reduce over all P processes (Eq. 7, term 3)
            g = net.get_tensor(mbd.T_DW, i)
            if P > 1:
                if comm.via_host:
                    h = g.cpu()
                    comm.dist.all_reduce(h)
                    g.copy_(h)
                else:
                    comm.dist.all_reduce(g)
                comm.words["allreduce_dw"] += 2.0 * (P - 1) / P * g.numel()
                net.set_tensor(mbd.T_DW, i, g)
            self.dK[i] = g
        net.sgd_step(eta / comm.P_c)          # the library divides by its own batch B / P_c: eta / B in total
        net.poll()


class GridMixed:
    """The integrated network of Section 2.4 over processes: convolutions with the P_r groups splitting the
    domain (GridConv), then fully connected layers with the same groups splitting the model (GridFC), one
    P_r x P_c grid (Eq. 9).  Between the two the strips of the last convolution's output are all-gathered
    over the P_r group into the [B / P_c, C H W] input every process of the group needs (the re-distribution
    of Section 2.1, Eq. 6), and the gradient of that input goes back to the strips' owners without
    communication: after the all-reduce of the first fully connected layer every process holds all of it."""

    def __init__(self, ksizes: Sequence[int], C_: int, H: int, W: int, fc_dims: Sequence[int], B: int, comm: GridComm):
        self.comm = comm
        self.C, self.H, self.W = int(C_), int(H), int(W)
        if H % comm.P_r:
            raise ValueError("the all-gather between the convolutions and the fully connected layers wants equal strips")
        self.conv = GridConv(ksizes, C_, H, W, B, comm, loss=mbd.LOSS_NONE)
        self.fc = GridFC([C_ * H * W] + [int(d) for d in fc_dims], B, comm)
        comm.words.setdefault("redistribute", 0.0)

    def step(self, X_local, labels_c, eta: float):
        import torch
        comm, conv = self.comm, self.conv
        m, Hs, L = conv.m, conv.Hs, conv.L
        conv.forward(X_local)
        strip = conv.net.get_tensor(mbd.T_ACT, L - 1)                       # [m, C, Hs, W], after the ReLU
        # all-gather of the strips over the P_r group; strip r' lands in rows r' Hs .. of every channel
        gathered = torch.empty((m, comm.P_r, self.C * Hs * self.W), dtype=strip.dtype, device=strip.device)
        comm.all_gather_cols(strip.view(m, -1), gathered.view(m, -1), kind="redistribute")
        X_fc = gathered.view(m, comm.P_r, self.C, Hs, self.W).permute(0, 2, 1, 3, 4).reshape(m, -1).contiguous()
        loss = self.fc.step(X_fc, labels_c, eta, input_is_relu_output=True)
        dX = self.fc.dX0.view(m, self.C, self.H, self.W)[:, :, comm.r * Hs:(comm.r + 1) * Hs, :].contiguous()
        conv.net.set_tensor(mbd.T_DY, L - 1, dX)
        conv.backward(eta)
        return loss


def expected_conv_words(ksizes: Sequence[int], C_: int, H: int, W: int, B: int, P_r: int, P_c: int) -> Dict[str, int]:
    """Per-process totals of mbd_comm_words (Eq. 9 with all layers in L_D).  The backward halo term is summed
    over the layers above the first: the formula counts it for every layer, the first layer needs no dX."""
    rows = mbd.comm_words(mbd.conv_layers(len(ksizes), C_, H, W, k=list(ksizes)), B, P_r, P_c)
    return {"halo_fwd": sum(r["halo_fwd"] for r in rows), "halo_bwd": sum(r["halo_bwd"] for r in rows[1:]),
            "allreduce_dw": sum(r["allreduce_dw"] for r in rows)}


def expected_mixed_words(ksizes: Sequence[int], C_: int, H: int, W: int, fc_dims: Sequence[int], B: int, P_r: int,
                         P_c: int) -> Dict[str, int]:
    """Per-process totals of mbd_comm_words for the integrated stack (Eq. 9), plus the re-distribution between
    the two groups of layers (Eq. 6 on the grid: (B / P_c) (P_r - 1) / P_r d words), which Eq. 9 leaves out."""
    layers = mbd.conv_layers(len(ksizes), C_, H, W, k=list(ksizes)) + mbd.fc_layers([C_ * H * W] + list(fc_dims), bias=False)
    rows = mbd.comm_words(layers, B, P_r, P_c)
    n = len(ksizes)
    return {"halo_fwd": sum(r["halo_fwd"] for r in rows), "halo_bwd": sum(r["halo_bwd"] for r in rows[1:]),
            "allgather_y": sum(r["allgather_y"] for r in rows), "allreduce_dx": sum(r["allreduce_dx"] for r in rows),
            "allreduce_dw": sum(r["allreduce_dw"] for r in rows),
            "redistribute": (B // P_c) * (P_r - 1) * (C_ * H * W // P_r)}


def expected_words(dims: Sequence[int], B: int, P_r: int, P_c: int) -> Dict[str, int]:
    """Per-process totals of mbd_comm_words for the stack (Eq. 8)."""
    rows = mbd.comm_words(mbd.fc_layers(dims, bias=False), B, P_r, P_c)
    return {k: sum(r[k] for r in rows) for k in ("allgather_y", "allreduce_dx", "allreduce_dw")}


def main(argv=None):
    """Runs a few steps of a fully connected stack over a P_r x P_c grid of processes (launch with torchrun,
    one process per grid position) and prints one JSON line from rank 0: time per step (slowest rank), the
    words each process moved against Eq. 8, and what the alpha-beta model predicts for them.

        python -m torch.distributed.run --nproc-per-node 4 --master-addr 127.0.0.1 \\
            -m paper_1712_04432_b200.grid_exec --grid 2x2 --dims 1024,1024,512 --batch 256 --backend nccl
    """
    import argparse
    import json
    import os
    import time

    import torch
    import torch.distributed as dist

    from . import inputs as I

    ap = argparse.ArgumentParser()
    ap.add_argument("--grid", default="2x1", help="P_r x P_c")
    ap.add_argument("--dims", default="1024,1024,512")
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--eta", type=float, default=0.01)
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="gloo: collectives through host copies (several processes may then share one GPU)")
    a = ap.parse_args(argv)
    P_r, P_c = (int(x) for x in a.grid.lower().split("x"))
    dims = [int(d) for d in a.dims.split(",")]
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local % torch.cuda.device_count())
    dist.init_process_group(a.backend)
    comm = GridComm(P_r, P_c, via_host=a.backend == "gloo")
    w = I.fc_workload(dims, a.batch, "bf16", "relu_normal")
    inp = I.make_inputs(w, seed=0)

    def dev(x):
        return torch.from_numpy(I.bf16_bits(x).view("int16")).cuda().view(torch.bfloat16)

    net = GridFC(dims, a.batch, comm)
    for i in range(len(dims) - 1):
        net.set_weights(i, dev(inp.Ws[i]))
    m = a.batch // P_c
    X_c = dev(inp.X[comm.c * m:(comm.c + 1) * m])
    labels_c = torch.from_numpy(inp.labels[comm.c * m:(comm.c + 1) * m]).cuda()
    net.step(X_c, labels_c, a.eta)                                   # warm-up
    for k in comm.words:
        comm.words[k] = 0.0
    dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    loss = 0.0
    for _ in range(a.steps):
        loss = net.step(X_c, labels_c, a.eta)
    torch.cuda.synchronize()
    dt = torch.tensor([(time.perf_counter() - t0) / a.steps], dtype=torch.float64)
    if a.backend == "nccl":
        dt = dt.cuda()
    dist.all_reduce(dt, op=dist.ReduceOp.MAX)
    if dist.get_rank() == 0:
        layers = mbd.fc_layers(dims, bias=False)
        model = mbd.comm_time(layers, a.batch, P_r, P_c, mbd.MACHINE_B200_NVLINK5)
        print(json.dumps({
            "grid": f"{P_r}x{P_c}", "dims": dims, "batch": a.batch, "backend": a.backend, "steps": a.steps,
            "ms_per_step": float(dt.item()) * 1e3, "loss_block_0": loss,
            "words_per_process_per_step": {k: v / a.steps for k, v in comm.words.items()},
            "eq8_words_per_process": expected_words(dims, a.batch, P_r, P_c),
            "alpha_beta_seconds_nvlink5": sum(sum(t.values()) for t in model)}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
