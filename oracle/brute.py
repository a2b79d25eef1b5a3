"""Scalar loop nests of the same definitions, for tiny shapes only.

TEST INFRASTRUCTURE.  These pin `mbd_oracle` (which leans on numpy's matrix
product and einsum): every sum is written index by index, in Python floats
(fp64), so a transposed operand or a shifted index in the fast version shows.
"""
from __future__ import annotations

import math


def matmul_WX(W, X):
    """Y[j][b] = sum_k W[j][k] X[k][b]   (Y = W X, Section 1)."""
    d_out, d_in, B = len(W), len(W[0]), len(X[0])
    return [[sum(W[j][k] * X[k][b] for k in range(d_in)) for b in range(B)]
            for j in range(d_out)]


def dX_WtdY(W, dY):
    """dX[k][b] = sum_j W[j][k] dY[j][b]   (dX = W^T dY)."""
    d_out, d_in, B = len(W), len(W[0]), len(dY[0])
    return [[sum(W[j][k] * dY[j][b] for j in range(d_out)) for b in range(B)]
            for k in range(d_in)]


def dW_outer_sum(dY, X):
    """dW = sum_{b=1..B} dY[:,b] X[:,b]^T, one outer product per sample
    (Appendix A.2)."""
    d_out, d_in, B = len(dY), len(X), len(X[0])
    dW = [[0.0] * d_in for _ in range(d_out)]
    for b in range(B):
        for j in range(d_out):
            for k in range(d_in):
                dW[j][k] += dY[j][b] * X[k][b]
    return dW


def conv3x3(K, X):
    """Y[b][o][h][w] = sum_{c,u,v} K[o][c][u][v] X[b][c][h+u-p_h][w+v-p_w], p = floor(k/2) (k_h, k_w odd)."""
    KH, KW = len(K[0][0]), len(K[0][0][0])
    B, C, H, W = len(X), len(X[0]), len(X[0][0]), len(X[0][0][0])
    O = len(K)
    Y = [[[[0.0] * W for _ in range(H)] for _ in range(O)] for _ in range(B)]
    for b in range(B):
        for o in range(O):
            for h in range(H):
                for w in range(W):
                    s = 0.0
                    for c in range(C):
                        for u in range(KH):
                            for v in range(KW):
                                hh, ww = h + u - KH // 2, w + v - KW // 2
                                if 0 <= hh < H and 0 <= ww < W:
                                    s += K[o][c][u][v] * X[b][c][hh][ww]
                    Y[b][o][h][w] = s
    return Y


def conv3x3_dX(K, dY):
    """Scatter form of the adjoint: every product K*dY is added to the input
    position it came from."""
    B, O, H, W = len(dY), len(dY[0]), len(dY[0][0]), len(dY[0][0][0])
    C = len(K[0])
    KH, KW = len(K[0][0]), len(K[0][0][0])
    dX = [[[[0.0] * W for _ in range(H)] for _ in range(C)] for _ in range(B)]
    for b in range(B):
        for o in range(O):
            for h in range(H):
                for w in range(W):
                    g = dY[b][o][h][w]
                    for c in range(C):
                        for u in range(KH):
                            for v in range(KW):
                                hh, ww = h + u - KH // 2, w + v - KW // 2
                                if 0 <= hh < H and 0 <= ww < W:
                                    dX[b][c][hh][ww] += K[o][c][u][v] * g
    return dX


def conv3x3_dK(dY, X, ksize=(3, 3)):
    KH, KW = ksize
    B, C, H, W = len(X), len(X[0]), len(X[0][0]), len(X[0][0][0])
    O = len(dY[0])
    dK = [[[[0.0] * KW for _ in range(KH)] for _ in range(C)] for _ in range(O)]
    for b in range(B):
        for o in range(O):
            for h in range(H):
                for w in range(W):
                    g = dY[b][o][h][w]
                    for c in range(C):
                        for u in range(KH):
                            for v in range(KW):
                                hh, ww = h + u - KH // 2, w + v - KW // 2
                                if 0 <= hh < H and 0 <= ww < W:
                                    dK[o][c][u][v] += g * X[b][c][hh][ww]
    return dK


def conv_strided(K, X, s):
    """Y[b][o][h'][w'] = sum_{c,u,v} K[o][c][u][v] X[b][c][s h'+u-p_h][s w'+v-p_w], p = floor(k/2)."""
    KH, KW = len(K[0][0]), len(K[0][0][0])
    B, C, H, W = len(X), len(X[0]), len(X[0][0]), len(X[0][0][0])
    O = len(K)
    Y = [[[[0.0] * (W // s) for _ in range(H // s)] for _ in range(O)] for _ in range(B)]
    for b in range(B):
        for o in range(O):
            for h in range(H // s):
                for w in range(W // s):
                    acc = 0.0
                    for c in range(C):
                        for u in range(KH):
                            for v in range(KW):
                                hh, ww = s * h + u - KH // 2, s * w + v - KW // 2
                                if 0 <= hh < H and 0 <= ww < W:
                                    acc += K[o][c][u][v] * X[b][c][hh][ww]
                    Y[b][o][h][w] = acc
    return Y


def softmax_ce_column(y, label):
    """Loss and gradient for one sample, without the max-subtraction trick
    (safe for the small logits the tests use)."""
    e = [math.exp(v) for v in y]
    Z = sum(e)
    loss = math.log(Z) - y[label]
    g = [v / Z for v in e]
    g[label] -= 1.0
    return loss, g
