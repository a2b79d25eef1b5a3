"""Pins for the fp64 oracle: things the paper and the mathematics fix,
independent of the oracle's own code (CPU only)."""
import math

import numpy as np
import pytest

from oracle import brute
from oracle import mbd_oracle as O


def rng(seed=0):
    return np.random.default_rng(seed)


def relerr(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def tiny_mlp(seed=1, dims=(5, 7, 6, 3), B=4, bias=True):
    r = rng(seed)
    layers = []
    for i in range(1, len(dims)):
        W = r.standard_normal((dims[i], dims[i - 1])) / math.sqrt(dims[i - 1])
        b = 0.1 * r.standard_normal(dims[i]) if bias else None
        layers.append(O.FC(W, b, relu=True))
    X = r.standard_normal((dims[0], B))
    labels = r.integers(0, dims[-1], B)
    return layers, X, labels


# ---------------------------------------------------------------- forward
def test_fc_forward_matches_scalar_loops():
    layers, X, _ = tiny_mlp(bias=False)
    W = layers[0].W
    Y = O.affine(W, X)
    Yb = np.array(brute.matmul_WX(W.tolist(), X.tolist()))
    assert relerr(Y, Yb) < 1e-14
    # asymmetric shapes: a transposed operand cannot even multiply
    assert Y.shape == (7, 4)


def test_identity_weights_copy_input():
    X = rng(2).standard_normal((6, 3))
    assert np.array_equal(O.affine(np.eye(6), X), X)


def test_bias_added_per_neuron():
    X = np.zeros((4, 3))
    b = np.array([1.0, 2.0, 3.0])
    Y = O.affine(np.ones((3, 4)), X, b)
    assert np.array_equal(Y, np.repeat(b[:, None], 3, axis=1))


def test_forward_chain_hand_example():
    # 2 -> 2 -> 1, one sample, numbers worked by hand:
    # Y1 = [[1,-1],[2,0]] [1,2]^T = [-1, 2]; X2 = [0, 2]; Y2 = [3, 4].[0,2] = 8
    layers = [O.FC(np.array([[1.0, -1.0], [2.0, 0.0]])), O.FC(np.array([[3.0, 4.0]]), relu=False)]
    Xs, Ys = O.forward(layers, np.array([[1.0], [2.0]]))
    assert Ys[0].ravel().tolist() == [-1.0, 2.0]
    assert Xs[1].ravel().tolist() == [0.0, 2.0]
    assert Ys[1].ravel().tolist() == [8.0]


# ---------------------------------------------------------------- softmax-CE
def test_softmax_zero_logits_closed_form():
    d, B = 10, 6
    labels = np.arange(B) % d
    J, per, dY = O.softmax_ce(np.zeros((d, B)), labels)
    assert abs(J - B * math.log(d)) < 1e-12
    expect = np.full((d, B), 1.0 / d)
    expect[labels, np.arange(B)] -= 1.0
    assert np.allclose(dY, expect, atol=1e-15)


def test_softmax_columns_sum_to_zero_and_shift_invariance():
    r = rng(3)
    Y = 3 * r.standard_normal((7, 5))
    labels = r.integers(0, 7, 5)
    J, per, dY = O.softmax_ce(Y, labels)
    assert np.abs(dY.sum(axis=0)).max() < 1e-14
    J2, per2, dY2 = O.softmax_ce(Y + 1000.0 * np.arange(5)[None, :], labels)
    assert abs(J - J2) < 1e-9 and np.allclose(dY, dY2, atol=1e-12)


def test_softmax_matches_naive_per_sample():
    r = rng(4)
    Y = r.standard_normal((6, 4))
    labels = r.integers(0, 6, 4)
    J, per, dY = O.softmax_ce(Y, labels)
    for b in range(4):
        lb, g = brute.softmax_ce_column(Y[:, b].tolist(), int(labels[b]))
        assert abs(lb - per[b]) < 1e-13
        assert np.allclose(g, dY[:, b], atol=1e-14)
    assert abs(J - per.sum()) < 1e-13


def test_softmax_two_class_hand_value():
    # logits (0, ln 3): p = (1/4, 3/4); label 0: loss = ln 4, grad = (-3/4, 3/4)
    J, per, dY = O.softmax_ce(np.array([[0.0], [math.log(3.0)]]), np.array([0]))
    assert abs(J - math.log(4.0)) < 1e-14
    assert np.allclose(dY.ravel(), [-0.75, 0.75], atol=1e-15)


# ---------------------------------------------------------------- gradients
def _fd_check(layers, X, labels, loss, get, set_, idxs, eps=1e-6):
    res = O.train_step(layers, X, labels, loss, 0.0)
    out = []
    for (li, idx) in idxs:
        w = get(layers[li])
        old = w[idx]
        w[idx] = old + eps
        Jp = O.total_loss(layers, X, labels, loss)
        w[idx] = old - eps
        Jm = O.total_loss(layers, X, labels, loss)
        w[idx] = old
        out.append(((Jp - Jm) / (2 * eps), li, idx))
    return res, out


def _no_kink(layers, X, margin=1e-3):
    _, Ys = O.forward(layers, X)
    return all(np.abs(Y).min() > margin for Y in Ys[:-1])


def test_dW_and_db_by_central_differences_mlp():
    seed = 10
    while True:
        layers, X, labels = tiny_mlp(seed=seed)
        if _no_kink(layers, X):
            break
        seed += 1
    r = rng(5)
    idxs = []
    for li, lay in enumerate(layers):
        for _ in range(6):
            idxs.append((li, (int(r.integers(lay.W.shape[0])), int(r.integers(lay.W.shape[1])))))
    res, fd = _fd_check(layers, X, labels, "softmax_ce", lambda l: l.W, None, idxs)
    for g, li, idx in fd:
        assert abs(g - res["dWs"][li][idx]) < 1e-7 * max(1.0, abs(g)), (li, idx)
    # biases
    idxs = [(li, (int(r.integers(lay.b.shape[0])),)) for li, lay in enumerate(layers) for _ in range(3)]
    res, fd = _fd_check(layers, X, labels, "softmax_ce", lambda l: l.b, None, idxs)
    for g, li, idx in fd:
        assert abs(g - res["dbs"][li][idx]) < 1e-7 * max(1.0, abs(g)), (li, idx)


def test_dX_by_central_differences():
    layers, X, labels = tiny_mlp(seed=20)
    # differentiate J with respect to the INPUT OF LAYER 2 through layers 2..L
    Xs, Ys = O.forward(layers, X)
    sub = layers[1:]
    X2 = Xs[1].copy() + 0.05          # move off the ReLU's zeros
    res = O.train_step([O.FC(np.eye(X2.shape[0]), None, relu=False)] + list(sub), X2, labels,
                       "softmax_ce", 0.0)
    dX = res["dXs"][1]                # gradient w.r.t. the input of `sub[0]`
    eps = 1e-6
    for (k, b) in [(0, 0), (3, 2), (6, 3)]:
        Xp = X2.copy(); Xp[k, b] += eps
        Xm = X2.copy(); Xm[k, b] -= eps
        g = (O.total_loss(sub, Xp, labels, "softmax_ce") - O.total_loss(sub, Xm, labels, "softmax_ce")) / (2 * eps)
        assert abs(g - dX[k, b]) < 1e-7 * max(1.0, abs(g))


def test_dW_is_sum_of_per_sample_outer_products():
    r = rng(6)
    dY = r.standard_normal((4, 5))
    X = r.standard_normal((3, 5))
    assert relerr(O.fc_dW(dY, X), np.array(brute.dW_outer_sum(dY.tolist(), X.tolist()))) < 1e-14
    W = r.standard_normal((4, 3))
    assert relerr(O.fc_dX(W, dY), np.array(brute.dX_WtdY(W.tolist(), dY.tolist()))) < 1e-14


def test_adjoint_identity_fc():
    r = rng(7)
    W = r.standard_normal((6, 5)); X = r.standard_normal((5, 4)); Z = r.standard_normal((6, 4))
    assert abs(np.sum(O.affine(W, X) * Z) - np.sum(X * O.fc_dX(W, Z))) < 1e-12
    # <W X, Z> = <W, Z X^T>
    assert abs(np.sum(O.affine(W, X) * Z) - np.sum(W * O.fc_dW(Z, X))) < 1e-12


def test_relu_mask_zero_at_zero_and_no_dX1():
    layers = [O.FC(np.array([[1.0], [-1.0], [0.0]])), O.FC(np.ones((2, 3)), relu=False)]
    res = O.train_step(layers, np.array([[2.0]]), np.array([0]), "softmax_ce", 0.0)
    # Y1 = (2,-2,0): only the first neuron passes gradient
    assert res["dYs"][0][1, 0] == 0.0 and res["dYs"][0][2, 0] == 0.0
    assert res["dXs"][0] is None


# ---------------------------------------------------------------- SGD (Eq. 1)
def test_sgd_update_is_eta_over_B_times_sum():
    layers, X, labels = tiny_mlp(seed=30)
    eta = 0.05
    res = O.train_step(layers, X, labels, "softmax_ce", eta)
    B = X.shape[1]
    for i, lay in enumerate(layers):
        assert np.allclose(res["new_W"][i] - lay.W, -(eta / B) * res["dWs"][i], atol=1e-16)
        assert np.allclose(res["new_b"][i] - lay.b, -(eta / B) * res["dbs"][i], atol=1e-16)
    res0 = O.train_step(layers, X, labels, "softmax_ce", 0.0)
    for i, lay in enumerate(layers):
        assert np.array_equal(res0["new_W"][i], lay.W)


def test_minibatch_gradient_is_mean_of_single_sample_gradients():
    # Eq. 1: the step with batch B equals w - eta * mean of the B one-sample gradients
    layers, X, labels = tiny_mlp(seed=31)
    eta = 0.1
    B = X.shape[1]
    full = O.train_step(layers, X, labels, "softmax_ce", eta)
    acc = [np.zeros_like(l.W) for l in layers]
    for b in range(B):
        one = O.train_step(layers, X[:, b:b + 1], labels[b:b + 1], "softmax_ce", eta)
        for i in range(len(layers)):
            acc[i] += one["dWs"][i]                # B=1: the sum is the single gradient
    for i, lay in enumerate(layers):
        assert np.allclose(full["new_W"][i], lay.W - eta * acc[i] / B, atol=1e-15)


def test_sgd_descends():
    layers, X, labels = tiny_mlp(seed=32)
    J0 = O.total_loss(layers, X, labels, "softmax_ce")
    res = O.train_step(layers, X, labels, "softmax_ce", 0.05)
    new_layers = [O.FC(res["new_W"][i], res["new_b"][i], l.relu) for i, l in enumerate(layers)]
    assert O.total_loss(new_layers, X, labels, "softmax_ce") < J0


# ---------------------------------------------------------------- momentum (the first-order method beside Eq. 1)
def test_momentum_with_mu_zero_is_eq1_and_constant_gradient_sums_a_geometric_series():
    r = rng(33)
    w, g = r.standard_normal((4, 3)), r.standard_normal((4, 3))
    w1, v1 = O.sgd_momentum(w, np.zeros_like(w), g, 0.1, 8, 0.0)
    assert np.array_equal(w1, O.sgd(w, g, 0.1, 8)) and np.array_equal(v1, g / 8)
    # the same gradient k times: v_k = (1 + mu + ... + mu^(k-1)) g / B = (1 - mu^k) / (1 - mu) g / B
    mu, eta, B = 0.9, 0.05, 8
    wk, vk = w, np.zeros_like(w)
    total = np.zeros_like(w)
    for k in range(1, 7):
        wk, vk = O.sgd_momentum(wk, vk, g, eta, B, mu)
        assert np.allclose(vk, (1 - mu ** k) / (1 - mu) * g / B, atol=1e-15)
        total += vk
        assert np.allclose(wk, w - eta * total, atol=1e-15)


def test_momentum_on_a_quadratic_follows_the_two_term_recurrence():
    # J(w) = a w^2 / 2 with "batch" 1: w_{k+1} = (1 + mu - eta a) w_k - mu w_{k-1}, whose solution is a combination
    # of the powers of the roots of z^2 - (1 + mu - eta a) z + mu = 0 (complex here: a damped oscillation of
    # modulus sqrt(mu) per step)
    a, eta, mu = 2.0, 0.3, 0.64
    w, v = np.array([1.0]), np.array([0.0])
    traj = [w.copy()]
    for _ in range(12):
        w, v = O.sgd_momentum(w, v, a * w, eta, 1, mu)
        traj.append(w.copy())
    t = np.array(traj)[:, 0]
    c = 1 + mu - eta * a
    for k in range(1, 12):
        assert abs(t[k + 1] - (c * t[k] - mu * t[k - 1])) < 1e-14
    z = np.roots([1.0, -c, mu])
    assert np.iscomplex(z[0]) and abs(abs(z[0]) - np.sqrt(mu)) < 1e-12
    # w_0 = 1, w_1 = 1 - eta a: fit the two coefficients, check the closed form at every later step
    A = np.linalg.solve(np.array([[1, 1], [z[0], z[1]]]), np.array([t[0], t[1]], complex))
    for k in range(13):
        assert abs((A[0] * z[0] ** k + A[1] * z[1] ** k).real - t[k]) < 1e-12


# ---------------------------------------------------------------- grid invariance
@pytest.mark.parametrize("grid", [(1, 1), (2, 2), (4, 1), (1, 4), (3, 5), (8, 1), (1, 8), (2, 4)])
def test_blocked_step_equals_unblocked(grid):
    P_r, P_c = grid
    r = rng(40)
    dims = (23, 17, 19, 10)
    B = 16
    layers = [O.FC(r.standard_normal((dims[i], dims[i - 1])) / 4, 0.1 * r.standard_normal(dims[i]))
              for i in range(1, 4)]
    X = r.standard_normal((dims[0], B))
    labels = r.integers(0, 10, B)
    a = O.train_step(layers, X, labels, "softmax_ce", 0.01)
    b = O.train_step_blocked(layers, X, labels, "softmax_ce", 0.01, P_r, P_c)
    assert abs(a["J"] - b["J"]) < 1e-12 * abs(a["J"])
    for i in range(3):
        assert relerr(b["Ys"][i], a["Ys"][i]) < 1e-12
        assert relerr(b["dWs"][i], a["dWs"][i]) < 1e-12
        assert relerr(b["dbs"][i], a["dbs"][i]) < 1e-12
        assert relerr(b["new_W"][i], a["new_W"][i]) < 1e-12
        if i > 0:
            assert relerr(b["dXs"][i], a["dXs"][i]) < 1e-12


def test_partials_are_per_block_sums():
    r = rng(41)
    dY = r.standard_normal((6, 8)); X = r.standard_normal((5, 8)); W = r.standard_normal((6, 5))
    dW, parts = O.fc_dW_blocked(dY, X, 2, 4)
    assert len(parts) == 4
    assert relerr(parts[1], dY[:, 2:4] @ X[:, 2:4].T) < 1e-14
    dX, parts = O.fc_dX_blocked(W, dY, 3, 2)
    assert len(parts) == 3
    assert relerr(parts[2], W[4:6].T @ dY[4:6]) < 1e-14


# ---------------------------------------------------------------- convolution
def conv_case(seed=50, B=2, C=3, O_=4, H=5, W=6):
    r = rng(seed)
    return r.standard_normal((O_, C, 3, 3)), r.standard_normal((B, C, H, W)), r.standard_normal((B, O_, H, W))


def test_conv_matches_scalar_loops():
    K, X, dY = conv_case()
    assert relerr(O.conv3x3(K, X), np.array(brute.conv3x3(K.tolist(), X.tolist()))) < 1e-14
    assert relerr(O.conv3x3_dX(K, dY), np.array(brute.conv3x3_dX(K.tolist(), dY.tolist()))) < 1e-14
    assert relerr(O.conv3x3_dK(dY, X), np.array(brute.conv3x3_dK(dY.tolist(), X.tolist()))) < 1e-14


@pytest.mark.parametrize("ksize", [(5, 5), (1, 7), (7, 3), (1, 1)])
def test_conv_of_other_odd_kernel_sizes(ksize):
    # k_h x k_w kernels with floor(k/2) rows / columns of zero padding: scalar loops, the adjoint identities
    # <Y, conv(K, X)> = <conv_dX(K, Y), X> = <conv_dK(Y, X), K>, a 3 x 3 kernel embedded in the centre of the larger
    # one gives the 3 x 3 result, and strips with floor(k_h/2) halo rows (Section 2.2) reproduce the whole image
    kh, kw = ksize
    r = rng(58)
    K, X, dY = r.standard_normal((4, 3, kh, kw)), r.standard_normal((2, 3, 9, 8)), r.standard_normal((2, 4, 9, 8))
    Y = O.conv3x3(K, X)
    assert relerr(Y, np.array(brute.conv3x3(K.tolist(), X.tolist()))) < 1e-14
    assert relerr(O.conv3x3_dX(K, dY), np.array(brute.conv3x3_dX(K.tolist(), dY.tolist()))) < 1e-14
    assert relerr(O.conv3x3_dK(dY, X, ksize), np.array(brute.conv3x3_dK(dY.tolist(), X.tolist(), ksize))) < 1e-14
    lhs = float(np.sum(dY * Y))
    assert abs(lhs - float(np.sum(O.conv3x3_dX(K, dY) * X))) < 1e-11 * abs(lhs)
    assert abs(lhs - float(np.sum(O.conv3x3_dK(dY, X, ksize) * K))) < 1e-11 * abs(lhs)
    if kh >= 3 and kw >= 3:
        K3 = r.standard_normal((4, 3, 3, 3))
        Kbig = np.zeros((4, 3, kh, kw)); Kbig[:, :, kh // 2 - 1:kh // 2 + 2, kw // 2 - 1:kw // 2 + 2] = K3
        assert relerr(O.conv3x3(Kbig, X), O.conv3x3(K3, X)) < 1e-14
    for P_r in (1, 2, 3, 4):
        assert relerr(O.conv3x3_strips(K, X, P_r), Y) < 1e-14
        assert relerr(O.conv3x3_dX_strips(K, dY, P_r), O.conv3x3_dX(K, dY)) < 1e-14
        dK, parts = O.conv3x3_dK_grid(dY, X, P_r, 2, ksize)
        assert len(parts) == 2 * P_r and relerr(dK, O.conv3x3_dK(dY, X, ksize)) < 1e-13
    # a strip's halo holds exactly floor(k_h/2) rows of each neighbour
    S = O.strip_with_halo(X, 3, 6, kh // 2)
    assert S.shape[2] == 3 + 2 * (kh // 2)
    assert np.array_equal(S[:, :, 0], X[:, :, 3 - kh // 2]) and np.array_equal(S[:, :, -1], X[:, :, 5 + kh // 2])


def test_wide_kernel_tap_direction_and_finite_differences():
    # tap (u, v) = (0, 0) of a 5 x 5 kernel reads the input two rows up and two columns left of the output position
    X = np.zeros((1, 1, 5, 5)); X[0, 0, 2, 2] = 1.0
    K = np.zeros((1, 1, 5, 5)); K[0, 0, 0, 0] = 3.0
    Y = O.conv3x3(K, X)
    assert Y[0, 0, 4, 4] == 3.0 and np.count_nonzero(Y) == 1
    # the gradients of J = sum(Y^2)/2 through a 5 x 3 layer by central differences
    r = rng(59)
    K, X = r.standard_normal((2, 2, 5, 3)) / 3, r.standard_normal((1, 2, 6, 5))
    J = lambda K_, X_: 0.5 * float(np.sum(O.conv3x3(K_, X_) ** 2))
    Y = O.conv3x3(K, X)
    dK, dX = O.conv3x3_dK(Y, X, (5, 3)), O.conv3x3_dX(K, Y)
    eps = 1e-6
    for idx in [(0, 1, 0, 0), (1, 0, 4, 2), (1, 1, 2, 1)]:
        Kp, Km = K.copy(), K.copy(); Kp[idx] += eps; Km[idx] -= eps
        assert abs((J(Kp, X) - J(Km, X)) / (2 * eps) - dK[idx]) < 1e-6 * max(1.0, abs(dK[idx]))
    for idx in [(0, 0, 0, 0), (0, 1, 5, 4), (0, 1, 3, 2)]:
        Xp, Xm = X.copy(), X.copy(); Xp[idx] += eps; Xm[idx] -= eps
        assert abs((J(K, Xp) - J(K, Xm)) / (2 * eps) - dX[idx]) < 1e-6 * max(1.0, abs(dX[idx]))


@pytest.mark.parametrize("ksize,s", [((3, 3), 2), ((5, 5), 2), ((7, 7), 2), ((3, 3), 3), ((1, 1), 2), ((5, 3), 4), ((11, 11), 4)])
def test_strided_convolution(ksize, s):
    # scalar loops over the strided index, the adjoint identities of the three strided functions, central differences
    # of J = sum(Y^2)/2, and stride 1 as the un-strided functions
    kh, kw = ksize
    r = rng(66)
    H, W = 12, 24
    K, X = r.standard_normal((3, 2, kh, kw)) / 3, r.standard_normal((2, 2, H, W))
    Y = O.conv_strided(K, X, s)
    assert Y.shape == (2, 3, H // s, W // s)
    assert relerr(Y, np.array(brute.conv_strided(K.tolist(), X.tolist(), s))) < 1e-14
    dY = r.standard_normal(Y.shape)
    lhs = float(np.sum(dY * Y))
    assert abs(lhs - float(np.sum(O.conv_strided_dX(K, dY, s) * X))) < 1e-11 * abs(lhs)
    assert abs(lhs - float(np.sum(O.conv_strided_dK(dY, X, ksize, s) * K))) < 1e-11 * abs(lhs)
    assert np.array_equal(O.conv_strided(K, X, 1), O.conv3x3(K, X))
    J = lambda K_, X_: 0.5 * float(np.sum(O.conv_strided(K_, X_, s) ** 2))
    dK, dX = O.conv_strided_dK(Y, X, ksize, s), O.conv_strided_dX(K, Y, s)
    eps = 1e-6
    for idx in [(0, 0, 0, 0), (2, 1, kh - 1, kw // 2)]:
        Kp, Km = K.copy(), K.copy(); Kp[idx] += eps; Km[idx] -= eps
        assert abs((J(Kp, X) - J(Km, X)) / (2 * eps) - dK[idx]) < 1e-6 * max(1.0, abs(dK[idx]))
    for idx in [(0, 0, 0, 0), (1, 1, 5, 7), (0, 1, H - 1, W - 1)]:
        Xp, Xm = X.copy(), X.copy(); Xp[idx] += eps; Xm[idx] -= eps
        assert abs((J(K, Xp) - J(K, Xm)) / (2 * eps) - dX[idx]) < 1e-6 * max(1.0, abs(dX[idx]))


def test_strided_layer_inside_a_training_step():
    # a stride-2 layer between two stride-1 layers: the step's gradients against central differences of its loss
    r = rng(67)
    layers = [O.Conv3x3(r.standard_normal((3, 2, 3, 3)) / 3), O.Conv3x3(r.standard_normal((4, 3, 5, 5)) / 5, stride=2),
              O.Conv3x3(r.standard_normal((2, 4, 3, 3)) / 4)]
    X = r.standard_normal((2, 2, 8, 12))
    res = O.train_step(layers, X, None, "half_ssq", 0.0)
    assert res["Ys"][1].shape == (2, 4, 4, 6) and res["Ys"][2].shape == (2, 2, 4, 6)
    eps = 1e-6
    for li, idx in [(0, (1, 0, 2, 1)), (1, (3, 2, 0, 4)), (2, (0, 3, 1, 1))]:
        def J(delta):
            ls = [O.Conv3x3(l.K.copy(), l.relu, l.split, l.stride) for l in layers]
            ls[li].K[idx] += delta
            return O.total_loss(ls, X, None, "half_ssq")
        fd = (J(eps) - J(-eps)) / (2 * eps)
        assert abs(fd - res["dWs"][li][idx]) < 1e-5 * max(1.0, abs(fd)), (li, fd, res["dWs"][li][idx])


def test_conv_centre_tap_is_per_pixel_fc():
    # a kernel with only its centre tap is the 1x1 convolution: Y[:, :, h, w] = M X[:, :, h, w]
    K, X, _ = conv_case(seed=51)
    M = K[:, :, 1, 1].copy()
    K0 = np.zeros_like(K); K0[:, :, 1, 1] = M
    Y = O.conv3x3(K0, X)
    assert relerr(Y, np.einsum("oc,bchw->bohw", M, X)) < 1e-14


def test_conv_is_correlation_not_flipped():
    # single input pixel at the centre; tap (u,v)=(0,0) must land at output (h+1, w+1)
    X = np.zeros((1, 1, 3, 3)); X[0, 0, 1, 1] = 1.0
    K = np.zeros((1, 1, 3, 3)); K[0, 0, 0, 0] = 5.0
    Y = O.conv3x3(K, X)
    assert Y[0, 0, 2, 2] == 5.0 and np.count_nonzero(Y) == 1


def test_conv_covering_whole_input_is_fc():
    # on a 3x3 image the centre output pixel sees the whole input: an FC layer (Section 2.4)
    r = rng(52)
    K = r.standard_normal((4, 2, 3, 3)); X = r.standard_normal((3, 2, 3, 3))
    Y = O.conv3x3(K, X)
    fc = K.reshape(4, -1) @ X.reshape(3, -1).T
    assert relerr(Y[:, :, 1, 1].T, fc) < 1e-14


def test_conv_adjoint_identities():
    K, X, Z = conv_case(seed=53)
    lhs = np.sum(O.conv3x3(K, X) * Z)
    assert abs(lhs - np.sum(X * O.conv3x3_dX(K, Z))) < 1e-11
    assert abs(lhs - np.sum(K * O.conv3x3_dK(Z, X))) < 1e-11


def test_conv_grads_by_central_differences():
    r = rng(54)
    layers = [O.Conv3x3(r.standard_normal((3, 3, 3, 3)) / 3, relu=True),
              O.Conv3x3(r.standard_normal((3, 3, 3, 3)) / 3, relu=False)]
    X = r.standard_normal((2, 3, 4, 5))
    assert _no_kink(layers, X, 1e-4)
    res = O.train_step(layers, X, None, "half_ssq", 0.0)
    eps = 1e-6
    for li, idx in [(0, (1, 2, 0, 1)), (0, (0, 0, 2, 2)), (1, (2, 1, 1, 0)), (1, (0, 2, 0, 2))]:
        Kw = layers[li].K
        old = Kw[idx]
        Kw[idx] = old + eps; Jp = O.total_loss(layers, X, None, "half_ssq")
        Kw[idx] = old - eps; Jm = O.total_loss(layers, X, None, "half_ssq")
        Kw[idx] = old
        g = (Jp - Jm) / (2 * eps)
        assert abs(g - res["dWs"][li][idx]) < 1e-6 * max(1.0, abs(g))


@pytest.mark.parametrize("P_r", [1, 2, 3, 4, 8])
def test_strip_conv_equals_whole_image(P_r):
    r = rng(55)
    K = r.standard_normal((4, 3, 3, 3)); X = r.standard_normal((2, 3, 16, 7)); dY = r.standard_normal((2, 4, 16, 7))
    assert relerr(O.conv3x3_strips(K, X, P_r), O.conv3x3(K, X)) < 1e-13
    assert relerr(O.conv3x3_dX_strips(K, dY, P_r), O.conv3x3_dX(K, dY)) < 1e-13
    dK, parts = O.conv3x3_dK_strips(dY, X, P_r)
    assert len(parts) == P_r and relerr(dK, O.conv3x3_dK(dY, X)) < 1e-13


def test_halo_rows_are_neighbour_copies():
    T = np.arange(2 * 1 * 8 * 3, dtype=np.float64).reshape(2, 1, 8, 3)
    S = O.strip_with_halo(T, 2, 4)
    assert np.array_equal(S[:, :, 0], T[:, :, 1]) and np.array_equal(S[:, :, -1], T[:, :, 4])
    S = O.strip_with_halo(T, 0, 4)
    assert not S[:, :, 0].any()


def test_conv_blocked_step_equals_unblocked():
    r = rng(56)
    layers = [O.Conv3x3(r.standard_normal((4, 4, 3, 3)) / 4, relu=True),
              O.Conv3x3(r.standard_normal((4, 4, 3, 3)) / 4, relu=False)]
    X = r.standard_normal((2, 4, 8, 6))
    a = O.train_step(layers, X, None, "half_ssq", 0.01)
    for P_r in (2, 4, 8):
        b = O.train_step_blocked(layers, X, None, "half_ssq", 0.01, P_r, 1)
        for i in range(2):
            assert relerr(b["Ys"][i], a["Ys"][i]) < 1e-12
            assert relerr(b["new_W"][i], a["new_W"][i]) < 1e-12
        assert relerr(b["dXs"][1], a["dXs"][1]) < 1e-12


def test_half_ssq():
    Y = np.array([[1.0, -2.0], [3.0, 0.5]])
    J, dY = O.half_ssq(Y)
    assert J == 0.5 * (1 + 4 + 9 + 0.25) and np.array_equal(dY, Y)


def test_storage_rounding_only_touches_kept_activations():
    # `store` models the activation storage type: identity leaves the step unchanged, and a
    # coarse rounding changes exactly what the next layer reads (X_{i+1}), not Y_i itself
    layers, X, labels = tiny_mlp(seed=60)
    a = O.train_step(layers, X, labels, "softmax_ce", 0.01)
    b = O.train_step(layers, X, labels, "softmax_ce", 0.01, store=lambda A: A)
    assert all(np.array_equal(x, y) for x, y in zip(a["dWs"], b["dWs"]))
    q = lambda A: np.round(A * 8) / 8
    c = O.train_step(layers, X, labels, "softmax_ce", 0.01, store=q)
    assert np.array_equal(c["Ys"][0], a["Ys"][0])
    assert np.array_equal(c["Xs"][1], q(np.maximum(a["Ys"][0], 0)))
    assert np.array_equal(c["Ys"][1], O.affine(layers[1].W, c["Xs"][1], layers[1].b))
    d = O.train_step_blocked(layers, X, labels, "softmax_ce", 0.01, 2, 2, store=q)
    assert all(relerr(x, y) < 1e-12 for x, y in zip(c["dWs"], d["dWs"]))


# ---------------------------------------------------------------- convolutions followed by fully connected layers
def mixed_case(seed=70, B=3, C=2, H=4, W=3, hidden=5, classes=4, relu_conv=True):
    r = rng(seed)
    layers = [O.Conv3x3(r.standard_normal((C, C, 3, 3)) / 3, relu=True),
              O.Conv3x3(r.standard_normal((C, C, 3, 3)) / 3, relu=relu_conv),
              O.FC(r.standard_normal((hidden, C * H * W)) / math.sqrt(C * H * W), 0.1 * r.standard_normal(hidden), relu=True),
              O.FC(r.standard_normal((classes, hidden)) / math.sqrt(hidden), None, relu=False)]
    X = r.standard_normal((B, C, H, W))
    labels = r.integers(0, classes, B)
    return layers, X, labels


def test_flatten_is_nchw_order():
    """Row c*H*W + h*W + w of the fully connected input is pixel (c, h, w): width runs
    fastest, then height, then channels (Section 2.2)."""
    B, C, H, W = 2, 3, 4, 5
    T = rng(71).standard_normal((B, C, H, W))
    M = O.flatten_nchw(T)
    assert M.shape == (C * H * W, B)
    for b in range(B):
        for c in range(C):
            for h in range(H):
                for w in range(W):
                    assert M[c * H * W + h * W + w, b] == T[b, c, h, w]
    assert np.array_equal(O.unflatten_nchw(M, T.shape), T)


def test_fc_after_conv_is_conv_covering_whole_input():
    """A fully connected layer on the flattened activation equals the convolution whose kernel
    covers the whole input (end of Section 2.4), evaluated with scalar loops."""
    B, C, H, W, D = 2, 2, 3, 4, 3
    r = rng(72)
    T = r.standard_normal((B, C, H, W))
    Wm = r.standard_normal((D, C * H * W))
    Y = O.affine(Wm, O.flatten_nchw(T))
    Kfull = Wm.reshape(D, C, H, W)
    for b in range(B):
        for o in range(D):
            acc = 0.0
            for c in range(C):
                for h in range(H):
                    for w in range(W):
                        acc += Kfull[o, c, h, w] * T[b, c, h, w]
            assert abs(acc - Y[o, b]) < 1e-12


def test_mixed_stack_grads_by_central_differences():
    seed = 70
    while True:
        layers, X, labels = mixed_case(seed)
        if _no_kink(layers, X, 1e-4):
            break
        seed += 1
    res = O.train_step(layers, X, labels, "softmax_ce", 0.0)
    eps = 1e-6
    checks = [(0, "K", (1, 0, 2, 1)), (0, "K", (0, 1, 0, 0)), (1, "K", (1, 1, 1, 2)), (1, "K", (0, 0, 2, 2)),
              (2, "W", (3, 7)), (2, "W", (0, 23)), (3, "W", (2, 4)), (2, "b", (1,))]
    for li, name, idx in checks:
        arr = getattr(layers[li], name)
        old = arr[idx]
        arr[idx] = old + eps; Jp = O.total_loss(layers, X, labels, "softmax_ce")
        arr[idx] = old - eps; Jm = O.total_loss(layers, X, labels, "softmax_ce")
        arr[idx] = old
        g = (Jp - Jm) / (2 * eps)
        got = res["dbs"][li][idx] if name == "b" else res["dWs"][li][idx]
        assert abs(g - got) < 1e-6 * max(1.0, abs(g)), (li, name, idx, g, got)
    # dX of the first fully connected layer comes back in NCHW shape and feeds the convolution below it
    assert res["dXs"][2].shape == X.shape and res["dYs"][1].shape == X.shape


def test_mixed_stack_input_gradient_shape_and_mask():
    layers, X, labels = mixed_case(73)
    res = O.train_step(layers, X, labels, "softmax_ce", 0.0)
    dX_fc = O.fc_dX(layers[2].W, res["dYs"][2])                      # d x B
    assert np.array_equal(res["dXs"][2], O.unflatten_nchw(dX_fc, X.shape))
    assert np.array_equal(res["dYs"][1], res["dXs"][2] * (res["Ys"][1] > 0))


@pytest.mark.parametrize("grid", [(1, 1), (2, 1), (1, 3), (2, 3), (4, 2)])
def test_mixed_blocked_step_equals_unblocked(grid):
    layers, X, labels = mixed_case(74, B=6, H=8)
    a = O.train_step(layers, X, labels, "softmax_ce", 0.01)
    b = O.train_step_blocked(layers, X, labels, "softmax_ce", 0.01, *grid)
    assert abs(a["J"] - b["J"]) < 1e-12 * abs(a["J"])
    for i in range(4):
        assert relerr(b["Ys"][i], a["Ys"][i]) < 1e-12
        assert relerr(b["new_W"][i], a["new_W"][i]) < 1e-12
        assert relerr(b["dWs"][i], a["dWs"][i]) < 1e-12
    for i in range(1, 4):
        assert relerr(b["dXs"][i], a["dXs"][i]) < 1e-12


@pytest.mark.parametrize("grid", [(2, 3), (3, 2), (6, 1), (1, 6)])
def test_batch_split_convolutions_in_the_blocked_step(grid):
    """Section 3's improved case: convolutions on 1 x P, fully connected layers on P_r x P_c.  Re-blocking changes no
    sum (the step equals the un-blocked one), and the convolutions' weight gradient is formed from P = P_r P_c
    per-process partials over batch blocks of whole images -- what a 1 x P grid of the domain-split form gives."""
    import dataclasses
    layers, X, labels = mixed_case(77, B=6, H=8)
    batch = [dataclasses.replace(l, split="batch") if isinstance(l, O.Conv3x3) else l for l in layers]
    a = O.train_step(layers, X, labels, "softmax_ce", 0.01)
    b = O.train_step_blocked(batch, X, labels, "softmax_ce", 0.01, *grid)
    assert abs(a["J"] - b["J"]) < 1e-12 * abs(a["J"])
    for i in range(4):
        assert relerr(b["Ys"][i], a["Ys"][i]) < 1e-12 and relerr(b["dWs"][i], a["dWs"][i]) < 1e-12
        assert relerr(b["new_W"][i], a["new_W"][i]) < 1e-12
    P = grid[0] * grid[1]
    c = O.train_step_blocked(layers[:2], X, None, "half_ssq", 0.01, 1, P)      # the two convolutions alone, domain form on 1 x P
    d = O.train_step_blocked(batch[:2], X, None, "half_ssq", 0.01, *grid)      # ... and batch-split on the P_r x P_c grid
    for i in range(2):
        assert np.array_equal(c["dWs"][i], d["dWs"][i]) and np.array_equal(c["Ys"][i], d["Ys"][i])


@pytest.mark.parametrize("grid", [(2, 3), (4, 1), (3, 2), (1, 6)])
def test_model_split_convolutions_in_the_blocked_step(grid):
    """Convolutions in L_M (Section 2.3 / 2.4): output channels over the P_r groups, batch over P_c.  Re-blocking changes no
    sum (the step equals the un-blocked one); a group's partial of dX is the back-propagation of ITS output channels alone
    (brute force with the other filters zeroed), and the forward blocks are the un-blocked output's channels."""
    import dataclasses
    layers, X, labels = mixed_case(78, B=6, H=8)
    model = [dataclasses.replace(l, split="model") if isinstance(l, O.Conv3x3) else l for l in layers]
    a = O.train_step(layers, X, labels, "softmax_ce", 0.01)
    b = O.train_step_blocked(model, X, labels, "softmax_ce", 0.01, *grid)
    assert abs(a["J"] - b["J"]) < 1e-12 * abs(a["J"])
    for i in range(4):
        assert relerr(b["Ys"][i], a["Ys"][i]) < 1e-12 and relerr(b["dWs"][i], a["dWs"][i]) < 1e-12
        assert relerr(b["new_W"][i], a["new_W"][i]) < 1e-12
    for i in range(1, 4):
        assert relerr(b["dXs"][i], a["dXs"][i]) < 1e-12
    K, Xc, dY = conv_case(seed=79)
    P_r = grid[0]
    assert relerr(O.conv3x3_model_blocked(K, Xc, P_r), O.conv3x3(K, Xc)) < 1e-13        # (no sum is formed: library blocking only)
    total, parts = O.conv3x3_dX_model_blocked(K, dY, P_r)
    assert len(parts) == P_r and relerr(total, O.conv3x3_dX(K, dY)) < 1e-13
    r = P_r - 1
    o0, o1 = O.balanced_ranges(K.shape[0], P_r)[r]
    Kz = np.zeros_like(K); Kz[o0:o1] = K[o0:o1]
    assert relerr(parts[r], brute.conv3x3_dX(Kz, dY)) < 1e-12 if o1 > o0 else np.all(parts[r] == 0)


def test_conv_weight_gradient_partials_over_the_whole_grid():
    """P_r x P_c partials, one per process, whose sum is the un-blocked gradient (last term of Eq. 9)."""
    r = rng(75)
    X = r.standard_normal((6, 3, 8, 5)); dY = r.standard_normal((6, 4, 8, 5))
    for P_r, P_c in [(2, 3), (4, 2), (1, 6), (8, 1)]:
        dK, parts = O.conv3x3_dK_grid(dY, X, P_r, P_c)
        assert len(parts) == P_r * P_c
        assert relerr(dK, O.conv3x3_dK(dY, X)) < 1e-13
    # the partial of process (r=1, c=0) of a 2 x 3 grid: strip 1 of samples 0, 1
    _, parts = O.conv3x3_dK_grid(dY, X, 2, 3)
    Xz = X[0:2].copy(); dYz = dY[0:2].copy(); dYz[:, :, 0:4, :] = 0.0          # only output rows 4..7 contribute
    assert relerr(parts[1], O.conv3x3_dK(dYz, Xz)) < 1e-13


def test_centre_tap_gradient_is_the_per_pixel_outer_product_sum():
    """The gradient of the centre tap is the fully connected weight gradient with every pixel as a sample
    (the 1 x 1 convolution singled out after Eq. 7): sum over b, h, w of dY[b, o, h, w] X[b, c, h, w]."""
    K, X, dY = conv_case(seed=76)
    dK = O.conv3x3_dK(dY, X)
    B, C_, H, W = X.shape
    for o_ in range(dY.shape[1]):
        for c in range(C_):
            acc = 0.0
            for b in range(B):
                for h in range(H):
                    for w in range(W):
                        acc += dY[b, o_, h, w] * X[b, c, h, w]
            assert abs(acc - dK[o_, c, 1, 1]) < 1e-11
