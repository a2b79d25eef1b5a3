"""Plain fp64 statement of one minibatch-SGD training step in matrix form.

TEST INFRASTRUCTURE: imported only by tests, the smoke check and the
CPU-baseline leg of the benchmark.  Shares no code with the CUDA path.

Notation follows the paper (Section 1): activations are matrices with one
COLUMN per sample, X_i in R^{d_{i-1} x B}, Y_i in R^{d_i x B}, and
W_i in R^{d_i x d_{i-1}}.  Convolution layers carry NCHW tensors
[B, C, H, W] instead (Section 2.1/2.2).  Everything is numpy float64; the
only library primitive used as a step is the dense matrix product `@`
(and `einsum` for the channel contraction inside the convolution).

    forward    Y_i = W_i X_i (+ b_i 1^T),  X_{i+1} = f(Y_i)      Section 1
    backward   dX_i = W_i^T dY_i,  dW_i = dY_i X_i^T             Section 1, Appendix A.2
    update     w <- w - eta (1/B) sum_{i in Batch} grad f_i      Eq. 1

Readings taken where the paper is silent: f = ReLU with derivative 0 at 0,
none after the last layer; gradients are SUMS over the batch and the 1/B of
Eq. 1 is applied once, in the update; softmax cross-entropy with natural log
(sum over samples) or half sum of squares as the loss; dX_1 is not formed
(Section 2.2: nothing is back-propagated beyond the first layer);
convolution is cross-correlation with zero padding.  Where a fully connected
layer follows a convolution (the integrated network of Section 2.4, Eq. 9:
domain-parallel layers first, model-parallel layers after them), the
activation [B, C, H, W] becomes the matrix with row index c*H*W + h*W + w
(NCHW order, the layout of Section 2.2; a fully connected layer is the
convolution whose kernel covers the whole input, end of Section 2.4).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# layers
# --------------------------------------------------------------------------
@dataclass
class FC:
    """Fully connected layer: W is d_i x d_{i-1}, b is d_i or None."""
    W: np.ndarray
    b: Optional[np.ndarray] = None
    relu: bool = True


@dataclass
class Conv3x3:
    """k_h x k_w (both odd; 3 x 3 in the listed workloads), stride 1, zero-pad floor(k/2) convolution:
    K is [C_out, C_in, k_h, k_w].
    split (used by the blocked step only): "domain" = row strips over the P_r groups (Section 2.2 / 2.4);
    "batch" = the layer forced onto a 1 x P grid, P = P_r P_c (Section 3's improved case: pure batch
    parallelism in the convolutional layers, P_r x P_c grids in the fully connected ones);
    "model" = the layer in L_M (Section 2.3 / 2.4, Eq. 8 with |W| = k_h k_w C_in C_out): the P_r groups split the
    output channels (the rows of the layer's weight matrix), the P_c groups the batch, no strips."""
    K: np.ndarray
    relu: bool = True
    split: str = "domain"
    stride: int = 1      # s > 1: the layer keeps the positions (s h', s w') of the stride-1 result (un-blocked step only)


def balanced_ranges(n: int, P: int):
    """Index ranges [floor(p n / P), floor((p+1) n / P)) for p = 0..P-1."""
    return [((p * n) // P, ((p + 1) * n) // P) for p in range(P)]


def flatten_nchw(T):
    """[B, C, H, W] -> the d x B matrix X with X[c*H*W + h*W + w, b] = T[b, c, h, w]:
    the input of a fully connected layer that follows a convolution
    (a fully connected layer = a convolution with k_h = X_H, k_w = X_W, Section 2.4)."""
    T = np.asarray(T, F64)
    return np.ascontiguousarray(T.reshape(T.shape[0], -1).T)


def unflatten_nchw(M, shape):
    """Inverse of `flatten_nchw`: d x B -> [B, C, H, W]."""
    return np.ascontiguousarray(np.asarray(M, F64).T).reshape(shape)


def _kept(A, lay, nxt, store):
    """What is kept of Y_i as the input of the next layer: f(Y_i), storage-rounded,
    flattened when a fully connected layer follows a convolution."""
    A = _stored(relu(A) if lay.relu else A, store)
    if A.ndim == 4 and isinstance(nxt, FC):
        A = flatten_nchw(A)
    return A


def _below(dX, Y_prev):
    """dX_i brought to the shape of the output of the layer below."""
    return unflatten_nchw(dX, Y_prev.shape) if dX.ndim == 2 and Y_prev.ndim == 4 else dX


# --------------------------------------------------------------------------
# single operations (un-blocked definitions)
# --------------------------------------------------------------------------
def affine(W, X, b=None):
    """Y = W X (+ b 1^T)   -- Section 1."""
    Y = np.asarray(W, F64) @ np.asarray(X, F64)
    if b is not None:
        Y = Y + np.asarray(b, F64)[:, None]
    return Y


def relu(Y):
    return np.maximum(Y, 0.0)


def fc_dX(W, dY):
    """dX = W^T dY   -- Section 1, Appendix A.2."""
    return np.asarray(W, F64).T @ np.asarray(dY, F64)


def fc_dW(dY, X):
    """dW = dY X^T = sum_b dY[:, b] X[:, b]^T   -- Appendix A.2."""
    return np.asarray(dY, F64) @ np.asarray(X, F64).T


def _pads(K):
    """Rows / columns of zero padding per side of a k_h x k_w kernel (odd sizes): floor(k/2), which is also the
    number of halo rows a strip needs from each neighbour (Section 2.2)."""
    kh, kw = K.shape[2], K.shape[3]
    assert kh % 2 == 1 and kw % 2 == 1
    return kh // 2, kw // 2


def conv3x3(K, X):
    """Y[b,o,h,w] = sum_{c,u,v} K[o,c,u,v] X[b,c,h+u-p_h,w+v-p_w], zero outside; p = floor(k/2)
    (for the 3 x 3 kernels of the listed workloads: h+u-1, w+v-1)."""
    K = np.asarray(K, F64)
    X = np.asarray(X, F64)
    ph, pw = _pads(K)
    B, C, H, W = X.shape
    Xp = np.zeros((B, C, H + 2 * ph, W + 2 * pw), F64)
    Xp[:, :, ph:H + ph, pw:W + pw] = X
    Y = np.zeros((B, K.shape[0], H, W), F64)
    for u in range(K.shape[2]):
        for v in range(K.shape[3]):
            Y += np.einsum("oc,bchw->bohw", K[:, :, u, v], Xp[:, :, u:u + H, v:v + W], optimize=True)
    return Y


def conv3x3_dX(K, dY):
    """dX[b,c,h,w] = sum_{o,u,v} K[o,c,u,v] dY[b,o,h-u+p_h,w-v+p_w], zero outside."""
    K = np.asarray(K, F64)
    dY = np.asarray(dY, F64)
    ph, pw = _pads(K)
    B, O, H, W = dY.shape
    dYp = np.zeros((B, O, H + 2 * ph, W + 2 * pw), F64)
    dYp[:, :, ph:H + ph, pw:W + pw] = dY
    dX = np.zeros((B, K.shape[1], H, W), F64)
    for u in range(K.shape[2]):
        for v in range(K.shape[3]):
            # index h-u+p_h in dY  ==  (h-u+2 p_h) in the padded array
            dX += np.einsum("oc,bohw->bchw", K[:, :, u, v],
                            dYp[:, :, 2 * ph - u:2 * ph - u + H, 2 * pw - v:2 * pw - v + W], optimize=True)
    return dX


def conv3x3_dK(dY, X, ksize=(3, 3)):
    """dK[o,c,u,v] = sum_{b,h,w} dY[b,o,h,w] X[b,c,h+u-p_h,w+v-p_w]; ksize = (k_h, k_w), both odd."""
    dY = np.asarray(dY, F64)
    X = np.asarray(X, F64)
    kh, kw = ksize
    ph, pw = kh // 2, kw // 2
    B, C, H, W = X.shape
    Xp = np.zeros((B, C, H + 2 * ph, W + 2 * pw), F64)
    Xp[:, :, ph:H + ph, pw:W + pw] = X
    dK = np.zeros((dY.shape[1], C, kh, kw), F64)
    for u in range(kh):
        for v in range(kw):
            dK[:, :, u, v] = np.einsum("bohw,bchw->oc", dY, Xp[:, :, u:u + H, v:v + W], optimize=True)
    return dK


def conv_strided(K, X, s):
    """A stride-s convolution is the stride-1 correlation kept at every s-th position in both directions:
    Y[b,o,h',w'] = conv3x3(K, X)[b,o,s h',s w'] (H and W multiples of s)."""
    assert X.shape[2] % s == 0 and X.shape[3] % s == 0
    return conv3x3(K, X)[:, :, ::s, ::s]


def _zero_stuffed(dY, s):
    """The gradient of a stride-s layer's output, put back at the positions (s h', s w') of the stride-1 result,
    zero elsewhere: what the kept positions' adjoint is."""
    dY = np.asarray(dY, F64)
    B, O, Ho, Wo = dY.shape
    full = np.zeros((B, O, Ho * s, Wo * s), F64)
    full[:, :, ::s, ::s] = dY
    return full


def conv_strided_dX(K, dY, s):
    return conv3x3_dX(K, _zero_stuffed(dY, s))


def conv_strided_dK(dY, X, ksize, s):
    return conv3x3_dK(_zero_stuffed(dY, s), X, ksize)


def softmax_ce(Y_L, labels):
    """J = sum_b [logsumexp_k Y[k,b] - Y[y_b,b]];  dY[:,b] = softmax(Y[:,b]) - e_{y_b}.

    Y_L is d_L x B (one column per sample).  Returns (J, per-sample loss, dY).
    """
    Y = np.asarray(Y_L, F64)
    labels = np.asarray(labels).astype(np.int64)
    d, B = Y.shape
    m = Y.max(axis=0)
    E = np.exp(Y - m[None, :])
    Z = E.sum(axis=0)
    lse = m + np.log(Z)
    cols = np.arange(B)
    per = lse - Y[labels, cols]
    dY = E / Z[None, :]
    dY[labels, cols] -= 1.0
    return float(per.sum()), per, dY


def half_ssq(Y_L):
    """J = 1/2 sum Y^2,  dY = Y."""
    Y = np.asarray(Y_L, F64)
    return float(0.5 * np.sum(Y * Y)), Y.copy()


def sgd(w, dw, eta, B):
    """Eq. 1 with dw = sum over the batch of per-sample gradients."""
    return np.asarray(w, F64) - (eta / B) * np.asarray(dw, F64)


def sgd_momentum(w, v, dw, eta, B, mu):
    """Heavy-ball momentum, the first-order method beside Eq. 1 (Section 2: the paper writes SGD for any
    of them).  v <- mu v + dw / B, w <- w - eta v; returns (w_new, v_new).  mu = 0 is Eq. 1."""
    v_new = mu * np.asarray(v, F64) + np.asarray(dw, F64) / B
    return np.asarray(w, F64) - eta * v_new, v_new


# --------------------------------------------------------------------------
# one training step, un-blocked
# --------------------------------------------------------------------------
def _batch_of(X):
    return X.shape[1] if X.ndim == 2 else X.shape[0]


def _stored(A, store):
    return A if store is None else np.asarray(store(A), F64)


def forward(layers: Sequence, X1, store=None):
    """Returns (Xs, Ys): Xs[i] is the input of layer i (0-based), Ys[i] its
    affine output before the nonlinearity.

    `store`, if given, is applied to every activation X_{i+1} = f(Y_i) that is
    kept for the next layer.  It models the storage type of the activations
    (e.g. rounding to bfloat16): the ReLU decision [Y_i > 0] of the layers
    above is a discrete decision, so it has to be taken on the same stored
    values on both sides of a comparison.  The arithmetic stays fp64."""
    Xs: List[np.ndarray] = [np.asarray(X1, F64)]
    Ys: List[np.ndarray] = []
    for i, lay in enumerate(layers):
        if isinstance(lay, FC):
            Y = affine(lay.W, Xs[i], lay.b)
        elif lay.stride > 1:
            Y = conv_strided(lay.K, Xs[i], lay.stride)
        else:
            Y = conv3x3(lay.K, Xs[i])
        Ys.append(Y)
        if i + 1 < len(layers):
            Xs.append(_kept(Y, lay, layers[i + 1], store))
    return Xs, Ys


def loss_and_top_grad(Y_L, loss: str, labels=None):
    if loss == "softmax_ce":
        J, per, dY = softmax_ce(Y_L, labels)
        return J, per, dY
    if loss == "half_ssq":
        J, dY = half_ssq(Y_L)
        return J, None, dY
    raise ValueError(loss)


def train_step(layers: Sequence, X1, labels, loss: str, eta: float, store=None):
    """One full step (`store`: see `forward`).  Returns a dict with
       Xs, Ys, J, per_sample, dYs (dJ/dY_i), dXs (dJ/dX_i, None for i=0),
       dWs, dbs, new_W, new_b   (lists indexed by layer, 0-based)."""
    L = len(layers)
    Xs, Ys = forward(layers, X1, store)
    B = _batch_of(Xs[0])
    J, per, dY_top = loss_and_top_grad(Ys[-1], loss, labels)
    dYs = [None] * L
    dXs = [None] * L
    dWs = [None] * L
    dbs = [None] * L
    dYs[L - 1] = dY_top
    for i in range(L - 1, -1, -1):
        lay = layers[i]
        if isinstance(lay, FC):
            dWs[i] = fc_dW(dYs[i], Xs[i])
            dbs[i] = dYs[i].sum(axis=1) if lay.b is not None else None
        elif lay.stride > 1:
            dWs[i] = conv_strided_dK(dYs[i], Xs[i], lay.K.shape[2:], lay.stride)
        else:
            dWs[i] = conv3x3_dK(dYs[i], Xs[i], lay.K.shape[2:])
        if i > 0:
            if isinstance(lay, FC):
                dXs[i] = fc_dX(lay.W, dYs[i])
            elif lay.stride > 1:
                dXs[i] = conv_strided_dX(lay.K, dYs[i], lay.stride)
            else:
                dXs[i] = conv3x3_dX(lay.K, dYs[i])
            dXs[i] = _below(dXs[i], Ys[i - 1])
            prev = layers[i - 1]
            dYs[i - 1] = dXs[i] * (Ys[i - 1] > 0.0) if prev.relu else dXs[i]
    new_W, new_b = [], []
    for i, lay in enumerate(layers):
        w = lay.W if isinstance(lay, FC) else lay.K
        new_W.append(sgd(w, dWs[i], eta, B))
        if isinstance(lay, FC) and lay.b is not None:
            new_b.append(sgd(lay.b, dbs[i], eta, B))
        else:
            new_b.append(None)
    return dict(Xs=Xs, Ys=Ys, J=J, per_sample=per, dYs=dYs, dXs=dXs, dWs=dWs,
                dbs=dbs, new_W=new_W, new_b=new_b)


# --------------------------------------------------------------------------
# the same step over a logical P_r x P_c grid (Section 2.3; Appendix A.1/A.2)
# --------------------------------------------------------------------------
def fc_forward_blocked(W, X, b, P_r, P_c):
    """Block (r,c) forms Y(r,c) = W(r,:) X(:,c); the all-gather over P_r only
    concatenates the row blocks (Appendix A.1)."""
    W = np.asarray(W, F64)
    X = np.asarray(X, F64)
    d, B = W.shape[0], X.shape[1]
    Y = np.empty((d, B), F64)
    for (r0, r1) in balanced_ranges(d, P_r):
        for (c0, c1) in balanced_ranges(B, P_c):
            blk = W[r0:r1, :] @ X[:, c0:c1]
            if b is not None:
                blk = blk + np.asarray(b, F64)[r0:r1, None]
            Y[r0:r1, c0:c1] = blk
    return Y


def fc_dX_blocked(W, dY, P_r, P_c):
    """Process row r holds W(r,:) and forms the partial W(r,:)^T dY(r,c); the
    all-reduce over the P_r group adds the partials (Appendix A.2).  Added in
    ascending r.  Returns (dX, partials[r])."""
    W = np.asarray(W, F64)
    dY = np.asarray(dY, F64)
    d_out, d_in = W.shape
    B = dY.shape[1]
    parts = []
    for (r0, r1) in balanced_ranges(d_out, P_r):
        part = np.zeros((d_in, B), F64)
        for (c0, c1) in balanced_ranges(B, P_c):
            part[:, c0:c1] = W[r0:r1, :].T @ dY[r0:r1, c0:c1]
        parts.append(part)
    dX = np.zeros((d_in, B), F64)
    for part in parts:
        dX = dX + part
    return dX, parts


def fc_dW_blocked(dY, X, P_r, P_c):
    """Process column c holds B/P_c samples and forms the partial
    sum_{b in c} dY_b X_b^T; the all-reduce over the P_c group adds them
    (Appendix A.2).  Added in ascending c.  Returns (dW, partials[c])."""
    dY = np.asarray(dY, F64)
    X = np.asarray(X, F64)
    d_out, B = dY.shape
    d_in = X.shape[0]
    parts = []
    for (c0, c1) in balanced_ranges(B, P_c):
        part = np.zeros((d_out, d_in), F64)
        for (r0, r1) in balanced_ranges(d_out, P_r):
            part[r0:r1, :] = dY[r0:r1, c0:c1] @ X[:, c0:c1].T
        parts.append(part)
    dW = np.zeros((d_out, d_in), F64)
    for part in parts:
        dW = dW + part
    return dW, parts


def strip_with_halo(T, h0, h1, halo=1):
    """Rows [h0-halo, h1+halo) of an NCHW tensor as a strip owner sees them after the halo exchange
    (Section 2.2): its own rows plus `halo` = floor(k_h/2) boundary rows copied from the strips above and
    below; zero rows where the image ends."""
    B, C, H, W = T.shape
    S = np.zeros((B, C, h1 - h0 + 2 * halo, W), F64)
    S[:, :, halo:halo + (h1 - h0), :] = T[:, :, h0:h1, :]
    for j in range(1, halo + 1):
        if h0 - j >= 0:
            S[:, :, halo - j, :] = T[:, :, h0 - j, :]              # row j above the strip: a neighbour's
        if h1 - 1 + j < H:
            S[:, :, halo + (h1 - h0) - 1 + j, :] = T[:, :, h1 - 1 + j, :]      # row j below it
    return S


def _conv_rows_valid(K, S):
    """Correlate a haloed strip S [B,C,hs+2 p_h,W]: zero padding in W only, the
    halo rows supply the H neighbours.  Output [B,O,hs,W]."""
    ph, pw = _pads(K)
    B, C, Hh, W = S.shape
    hs = Hh - 2 * ph
    Sp = np.zeros((B, C, Hh, W + 2 * pw), F64)
    Sp[:, :, :, pw:W + pw] = S
    Y = np.zeros((B, K.shape[0], hs, W), F64)
    for u in range(K.shape[2]):
        for v in range(K.shape[3]):
            Y += np.einsum("oc,bchw->bohw", K[:, :, u, v], Sp[:, :, u:u + hs, v:v + W], optimize=True)
    return Y


def conv3x3_strips(K, X, P_r):
    """Domain-parallel forward: each of P_r strips correlates its own rows
    after receiving floor(k_h/2) halo rows per neighbour (Section 2.2, Eq. 7)."""
    K = np.asarray(K, F64)
    X = np.asarray(X, F64)
    B, C, H, W = X.shape
    Y = np.empty((B, K.shape[0], H, W), F64)
    for (h0, h1) in balanced_ranges(H, P_r):
        Y[:, :, h0:h1, :] = _conv_rows_valid(K, strip_with_halo(X, h0, h1, _pads(K)[0]))
    return Y


def conv3x3_dX_strips(K, dY, P_r):
    """Domain-parallel backward-data: needs the dY halo rows (second term of
    Eq. 7); the transposed correlation flips the taps and swaps channels."""
    K = np.asarray(K, F64)
    dY = np.asarray(dY, F64)
    Kt = np.ascontiguousarray(K[:, :, ::-1, ::-1].transpose(1, 0, 2, 3))
    B, O, H, W = dY.shape
    dX = np.empty((B, K.shape[1], H, W), F64)
    for (h0, h1) in balanced_ranges(H, P_r):
        dX[:, :, h0:h1, :] = _conv_rows_valid(Kt, strip_with_halo(dY, h0, h1, _pads(K)[0]))
    return dX


def conv3x3_dK_strips(dY, X, P_r, ksize=(3, 3)):
    """Each strip forms a partial dK from its own output rows and its haloed
    input; the all-reduce over the strips adds them in ascending order
    (third term of Eq. 7).  Returns (dK, partials)."""
    dY = np.asarray(dY, F64)
    X = np.asarray(X, F64)
    kh, kw = ksize
    ph, pw = kh // 2, kw // 2
    B, C, H, W = X.shape
    parts = []
    for (h0, h1) in balanced_ranges(H, P_r):
        S = strip_with_halo(X, h0, h1, ph)
        hs = h1 - h0
        Sp = np.zeros((B, C, hs + 2 * ph, W + 2 * pw), F64)
        Sp[:, :, :, pw:W + pw] = S
        part = np.zeros((dY.shape[1], C, kh, kw), F64)
        for u in range(kh):
            for v in range(kw):
                part[:, :, u, v] = np.einsum("bohw,bchw->oc", dY[:, :, h0:h1, :],
                                             Sp[:, :, u:u + hs, v:v + W], optimize=True)
        parts.append(part)
    dK = np.zeros_like(parts[0])
    for part in parts:
        dK = dK + part
    return dK, parts


def conv3x3_dK_grid(dY, X, P_r, P_c, ksize=(3, 3)):
    """Weight gradient of a domain-parallel layer on a P_r x P_c grid: process
    (r, c) owns strip r of the samples of batch block c and forms one partial;
    the all-reduce over all P = P_r P_c processes (last term of Eq. 9) adds them,
    here in ascending c, then r.  Returns (dK, partials)."""
    dY = np.asarray(dY, F64)
    X = np.asarray(X, F64)
    parts = []
    for (c0, c1) in balanced_ranges(X.shape[0], P_c):
        _, strip_parts = conv3x3_dK_strips(dY[c0:c1], X[c0:c1], P_r, ksize)
        parts.extend(strip_parts)
    dK = np.zeros_like(parts[0])
    for part in parts:
        dK = dK + part
    return dK, parts


def conv3x3_model_blocked(K, X, P_r):
    """Forward of a model-parallel convolution: process group r computes the output channels of its block of
    filters, [o0, o1) = balanced range r of C_out, from the whole input; the blocks are concatenated (the
    all-gather of Appendix A.1).  No sum is formed, so the result is conv3x3(K, X) itself."""
    K = np.asarray(K, F64)
    return np.concatenate([conv3x3(K[o0:o1], X) for (o0, o1) in balanced_ranges(K.shape[0], P_r)], axis=1)


def conv3x3_dX_model_blocked(K, dY, P_r):
    """Backward-data of a model-parallel convolution (Appendix A.2: dX = sum over the P_r groups of W_r^T dY_r):
    group r back-propagates the gradient of its own output channels through its own filters; the P_r partial
    results are added in ascending r (the all-reduce of Eq. 8's second term).  Returns (sum, partials)."""
    K = np.asarray(K, F64)
    dY = np.asarray(dY, F64)
    parts = [conv3x3_dX(K[o0:o1], dY[:, o0:o1]) for (o0, o1) in balanced_ranges(K.shape[0], P_r)]
    total = np.zeros_like(parts[0])
    for p in parts:
        total = total + p
    return total, parts


def train_step_blocked(layers: Sequence, X1, labels, loss: str, eta: float,
                       P_r: int, P_c: int, store=None):
    """The step of `train_step`, every contraction formed block by block over
    the P_r x P_c grid and every cross-block sum taken as P separate partials
    added in ascending block index.  FC layers split the model over P_r and the
    batch over P_c; convolution layers split the image into P_r row strips and
    the batch over P_c (Eq. 9: their weight gradient is summed over all
    P = P_r P_c processes); convolution layers with split == "batch" are cut into
    P_r P_c batch blocks and no strips (Section 3's improved case); convolution layers with split == "model"
    split their output channels over P_r and the batch over P_c, like an FC layer."""
    L = len(layers)
    Xs = [np.asarray(X1, F64)]
    Ys = []
    for i, lay in enumerate(layers):
        if isinstance(lay, FC):
            Y = fc_forward_blocked(lay.W, Xs[i], lay.b, P_r, P_c)
        elif lay.split == "model":
            Y = conv3x3_model_blocked(lay.K, Xs[i], P_r)
        else:
            Y = conv3x3_strips(lay.K, Xs[i], 1 if lay.split == "batch" else P_r)
        Ys.append(Y)
        if i + 1 < L:
            Xs.append(_kept(Y, lay, layers[i + 1], store))
    B = _batch_of(Xs[0])
    J, per, dY_top = loss_and_top_grad(Ys[-1], loss, labels)
    dYs = [None] * L
    dXs = [None] * L
    dWs = [None] * L
    dbs = [None] * L
    dYs[L - 1] = dY_top
    for i in range(L - 1, -1, -1):
        lay = layers[i]
        if isinstance(lay, FC):
            dWs[i], _ = fc_dW_blocked(dYs[i], Xs[i], P_r, P_c)
            if lay.b is not None:
                db = np.zeros(lay.W.shape[0], F64)
                for (c0, c1) in balanced_ranges(B, P_c):
                    db = db + dYs[i][:, c0:c1].sum(axis=1)
                dbs[i] = db
        elif lay.split == "model":
            dWs[i], _ = conv3x3_dK_grid(dYs[i], Xs[i], 1, P_c, lay.K.shape[2:])            # rows of dK are independent: one partial per batch block
        elif lay.split == "batch":
            dWs[i], _ = conv3x3_dK_grid(dYs[i], Xs[i], 1, P_r * P_c, lay.K.shape[2:])      # one partial per process of the 1 x P grid
        else:
            dWs[i], _ = conv3x3_dK_grid(dYs[i], Xs[i], P_r, P_c, lay.K.shape[2:])
        if i > 0:
            if isinstance(lay, FC):
                dXs[i], _ = fc_dX_blocked(lay.W, dYs[i], P_r, P_c)
            elif lay.split == "model":
                dXs[i], _ = conv3x3_dX_model_blocked(lay.K, dYs[i], P_r)
            else:
                dXs[i] = conv3x3_dX_strips(lay.K, dYs[i], 1 if lay.split == "batch" else P_r)
            dXs[i] = _below(dXs[i], Ys[i - 1])
            prev = layers[i - 1]
            dYs[i - 1] = dXs[i] * (Ys[i - 1] > 0.0) if prev.relu else dXs[i]
    new_W, new_b = [], []
    for i, lay in enumerate(layers):
        w = lay.W if isinstance(lay, FC) else lay.K
        new_W.append(sgd(w, dWs[i], eta, B))
        if isinstance(lay, FC) and lay.b is not None:
            new_b.append(sgd(lay.b, dbs[i], eta, B))
        else:
            new_b.append(None)
    return dict(Xs=Xs, Ys=Ys, J=J, per_sample=per, dYs=dYs, dXs=dXs, dWs=dWs,
                dbs=dbs, new_W=new_W, new_b=new_b)


def total_loss(layers: Sequence, X1, labels, loss: str) -> float:
    """J alone (used by the finite-difference pins)."""
    _, Ys = forward(layers, X1)
    return loss_and_top_grad(Ys[-1], loss, labels)[0]
