"""Shared helpers for the parity tests: conversions between the oracle's fp64
numpy arrays and device tensors, and the error metric."""
import numpy as np

from paper_1712_04432_b200 import inputs as I


def rel_fro(got, ref):
    """||got - ref||_F / ||ref||_F in fp64."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (den if den > 0 else 1.0))


def to_dev(a, bf16):
    """numpy float32 (bf16-exact when bf16) -> CUDA tensor of the network dtype."""
    import torch
    a = np.ascontiguousarray(a, np.float32)
    if bf16:
        bits = I.bf16_bits(a).view(np.int16)
        return torch.from_numpy(bits).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_np(t):
    """CUDA tensor (bf16 or f32) -> numpy float64."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


# ---------------------------------------------------------------------------
# one training step on both sides
# ---------------------------------------------------------------------------
def bf16_store(A):
    """Storage rounding handed to the oracle for bf16 workloads: the kept activations
    are bfloat16 on the device, and the ReLU decisions above them must see the same
    stored values on both sides."""
    return I.round_to_bf16(np.asarray(A, np.float32)).astype(np.float64)


def oracle_fc_step(w, inp, blocked_grid=None, exact=False, eta=None):
    """fp64 oracle step for a fully connected workload (paper orientation: d x B).
    bf16 workloads round the STORED activations to bf16 unless `exact`."""
    from oracle import mbd_oracle as O
    store = bf16_store if (w.dtype == "bf16" and not exact) else None
    eta = w.eta if eta is None else eta
    L = len(inp.Ws)
    layers = [O.FC(inp.Ws[i].astype(np.float64), None if inp.bs[i] is None else inp.bs[i].astype(np.float64),
                   relu=True) for i in range(L)]
    X1 = inp.X.astype(np.float64).T
    if blocked_grid is None:
        return O.train_step(layers, X1, inp.labels, "softmax_ce", eta, store=store)
    return O.train_step_blocked(layers, X1, inp.labels, "softmax_ce", eta, *blocked_grid, store=store)


def update_sized_eta(o, Ws, B, ratio=1.0):
    """A learning rate at which Eq. 1 moves every weight matrix by at least `ratio` of its own norm:
    eta = ratio * B * max_i ||W_i|| / ||dW_i||.  At the workloads' eta = 0.01 a step moves the weights by
    1e-4 .. 5e-4 of their norm, less than one bf16 rounding of the weights themselves (1e-3), so a
    comparison of updated bf16 weights cannot tell an update from no update; at this eta it can."""
    worst = max(np.linalg.norm(_oracle_shape(Ws[i])) / np.linalg.norm(o["dWs"][i]) for i in range(len(Ws)))
    return float(ratio * B * worst)


def _oracle_shape(W):
    """A weight array as the oracle holds it (a 1 x 1 kernel is the centre tap of a 3 x 3 one)."""
    W = np.asarray(W, np.float64)
    return oracle_kernel(W) if W.ndim == 4 else W


def oracle_with_eta(o, Ws, bs, B, eta):
    """The oracle's result for another learning rate: only Eq. 1 depends on eta, so the updated weights
    are re-formed from the oracle's own gradients with the oracle's own update."""
    from oracle import mbd_oracle as O
    o2 = dict(o)
    o2["new_W"] = [O.sgd(_oracle_shape(Ws[i]), o["dWs"][i], eta, B) for i in range(len(Ws))]
    o2["new_b"] = [None if (bs[i] is None or o["dbs"][i] is None) else O.sgd(np.asarray(bs[i], np.float64), o["dbs"][i], eta, B)
                   for i in range(len(Ws))]
    return o2


def gpu_fc_step(w, inp, grid=(1, 1), max_partials=0, fused=False, force_acts=None, eta=None):
    """The same step through the C ABI.  Returns numpy fp64 arrays in the GPU's
    [B, d] / [d_out, d_in] layouts.  `force_acts` (list of [B, d_i] arrays for the hidden
    layers, bf16-exact) overwrites the stored activations after the forward pass, so that
    the backward pass takes the ReLU decisions on exactly those values."""
    import torch
    from paper_1712_04432_b200 import mbd
    bf = w.dtype == "bf16"
    L = len(inp.Ws)
    eta = w.eta if eta is None else eta
    net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16 if bf else mbd.F32,
                  mbd.LOSS_SOFTMAX_CE, max_partials)
    for i in range(L):
        net.set_weights(i, to_dev(inp.Ws[i], bf), torch.from_numpy(inp.bs[i]).cuda())
    X = to_dev(inp.X, bf)
    labels = torch.from_numpy(inp.labels).cuda()
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = {}
    net.forward(X, labels, J)
    out["act"] = [to_np(net.get_tensor(mbd.T_ACT, i)) for i in range(L)]
    if force_acts is not None:
        for i in range(L - 1):
            net.set_tensor(mbd.T_ACT, i, to_dev(force_acts[i], bf))
    if fused:
        net.backward(eta)
    else:
        net.backward(0.0)
        out["dW"] = [to_np(net.get_tensor(mbd.T_DW, i)) for i in range(L)]
        out["db"] = [to_np(net.get_tensor(mbd.T_DB, i)) for i in range(L)]
        net.sgd_step(eta)
    net.poll()
    out["J"] = float(J.item())
    out["loss"] = to_np(net.get_tensor(mbd.T_LOSS))
    out["dY"] = [to_np(net.get_tensor(mbd.T_DY, i)) for i in range(L)]
    nw = [net.get_weights(i, with_bias=True) for i in range(L)]
    out["new_W"] = [to_np(a) for a, _ in nw]
    out["new_b"] = [to_np(b) for _, b in nw]
    out["launches"] = net.launch_count
    net.close()
    return out


def oracle_hidden_acts(o):
    """The oracle's stored hidden activations X_2..X_L as [B, d] float32 arrays."""
    return [np.ascontiguousarray(x.T, np.float32) for x in o["Xs"][1:]]


BF16_ROUNDING_RMS = 2.0 ** -9 / np.sqrt(3.0)     # rms relative error of one round-to-nearest to bfloat16
FP32_ROUNDING_RMS = 2.0 ** -24 / np.sqrt(3.0)


def update_checks(chk, g, o, init_W, init_b, tols, bf16, require_sized):
    """Eq. 1 itself: the step that was applied, W_new - W_0 (and b_new - b_0), against the oracle's, relative
    to the size of the STEP, not of the weights.  Stored weights carry the rounding of W_new, which is
    BF16_ROUNDING_RMS (or FP32_ROUNDING_RMS) * ||W_new|| whatever the step was; it is added to the tolerance,
    so the check is sharp exactly when the step is comparable to the weights (`require_sized` demands that)."""
    for i in range(len(init_W)):
        w0 = np.asarray(init_W[i], np.float64)
        step_o = np.asarray(o["new_W"][i], np.float64) - w0
        rms = BF16_ROUNDING_RMS if bf16 else FP32_ROUNDING_RMS
        noise = 1.5 * rms * np.linalg.norm(o["new_W"][i]) / max(np.linalg.norm(step_o), 1e-300)
        if require_sized:
            assert noise <= 0.5 * tols[i], f"layer {i}: the step is too small against the weights for a sharp check"
        chk(f"W_new[{i}] - W_0[{i}]", g["new_W"][i] - w0, step_o, tols[i] + noise)
        if init_b is not None and init_b[i] is not None and o["new_b"][i] is not None:
            b0 = np.asarray(init_b[i], np.float64)
            if np.linalg.norm(o["new_b"][i] - b0) > 0:
                chk(f"b_new[{i}] - b_0[{i}]", g["new_b"][i] - b0, o["new_b"][i] - b0, tols[i])


def compare_fc_step(g, o, tol, fused=False, tol_below_relu=None, init=None, bf16=True, require_sized=False, errors=None):
    """Element-by-element comparison, tensor by tensor; returns the worst relative
    Frobenius error.  `tol_below_relu` (default `tol`) applies to the gradients that sit
    below a ReLU decision: dY_i, dW_i, db_i of every layer but the last.  `init` (the Inputs the
    step started from) adds the comparison of the applied update itself (see `update_checks`).
    `errors` (a dict) receives every measured error by tensor name."""
    L = len(o["Ys"])
    worst = 0.0
    report = []
    bad = []
    if tol_below_relu is None:
        tol_below_relu = tol

    def chk(name, got, ref, t=None):
        nonlocal worst
        e = rel_fro(got, ref)
        worst = max(worst, e)
        if errors is not None:
            errors[name] = e
        report.append(f"{name}: {e:.3e}")
        if e > (tol if t is None else t):
            bad.append(name)

    assert abs(g["J"] - o["J"]) <= max(tol, 1e-4) * abs(o["J"]), (g["J"], o["J"])
    chk("per-sample loss", g["loss"], o["per_sample"])
    for i in range(L):
        ref_act = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        chk(f"Y[{i}]", g["act"][i], ref_act.T)
        tg = tol if i == L - 1 else tol_below_relu
        chk(f"dY[{i}]", g["dY"][i], o["dYs"][i].T, tg)    # for i < L-1 this is dX_{i+1} after the mask
        if not fused:
            chk(f"dW[{i}]", g["dW"][i], o["dWs"][i], tg)
            chk(f"db[{i}]", g["db"][i], o["dbs"][i], tg)
        chk(f"W_new[{i}]", g["new_W"][i], o["new_W"][i], tg)
        ref_b = o["new_b"][i]
        assert np.abs(g["new_b"][i] - ref_b).max() <= tg * max(1.0, np.abs(ref_b).max()), f"b_new[{i}]"
    if init is not None:
        update_checks(chk, g, o, init.Ws, init.bs, [tol if i == L - 1 else tol_below_relu for i in range(L)], bf16,
                      require_sized)
    assert not bad, "rel. Frobenius error too large for %s: %s" % (bad, "; ".join(report))
    return worst


# ---------------------------------------------------------------------------
# convolution workloads
# ---------------------------------------------------------------------------
def oracle_kernel(K):
    """The oracle's 3 x 3 layer for a device kernel: a 1 x 1 kernel [O, C, 1, 1] is the 3 x 3 kernel whose
    centre tap holds it and whose other taps are zero (the same correlation)."""
    K = np.asarray(K, np.float64)
    if K.shape[2:] != (1, 1):
        return K
    K3 = np.zeros(K.shape[:2] + (3, 3), np.float64)
    K3[:, :, 1, 1] = K[:, :, 0, 0]
    return K3


def like_device(ref, got):
    """Oracle weight / gradient of a convolution in the device's shape: the centre tap for a 1 x 1 layer."""
    ref = np.asarray(ref)
    return ref[:, :, 1:2, 1:2] if (ref.ndim == 4 and got.shape[-1] == 1 and ref.shape[-1] == 3) else ref

def oracle_conv_step(w, inp, strips=None, grid=None, eta=None, split="domain"):
    """fp64 oracle step for a domain-parallel conv workload (NCHW); stored activations are
    rounded to bf16 like the device's.  `strips` = P_r (or `grid` = (P_r, P_c)) runs the
    strip / halo formulation."""
    from oracle import mbd_oracle as O
    splits = [split] * len(inp.Ws) if isinstance(split, str) else list(split)
    layers = [O.Conv3x3(oracle_kernel(k), relu=True, stride=w.stride(i), split=splits[i]) for i, k in enumerate(inp.Ws)]
    X = inp.X.astype(np.float64)
    eta = w.eta if eta is None else eta
    if strips is None and grid is None:
        return O.train_step(layers, X, None, "half_ssq", eta, store=bf16_store)
    P_r, P_c = grid if grid is not None else (strips, 1)
    return O.train_step_blocked(layers, X, None, "half_ssq", eta, P_r, P_c, store=bf16_store)


def gpu_conv_step(w, inp, P_r=1, fused=False, force_acts=None, P_c=1, eta=None, max_partials=0, split=None, plans=None):
    import torch
    from paper_1712_04432_b200 import mbd
    C_, H, Wd = w.dims
    L = w.n_layers
    eta = w.eta if eta is None else eta
    kw = {} if split is None else dict(split=split)
    net = mbd.Net(mbd.conv_layers(L, C_, H, Wd, k=[w.kshape(i) for i in range(L)], channels=w.channels, strides=w.strides, **kw), w.B, P_r, P_c, mbd.BF16,
                  mbd.LOSS_HALF_SSQ, max_partials)
    for i in range(L):
        net.set_weights(i, to_dev(inp.Ws[i], True))
    X = to_dev(inp.X, True)
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = {}
    net.forward(X, None, J)
    out["act"] = [to_np(net.get_tensor(mbd.T_ACT, i)) for i in range(L)]
    if force_acts is not None:
        for i in range(L - 1):
            net.set_tensor(mbd.T_ACT, i, to_dev(force_acts[i], True))
    if fused:
        net.backward(eta)
    else:
        net.backward(0.0)
        out["dW"] = [to_np(net.get_tensor(mbd.T_DW, i)) for i in range(L)]
        net.sgd_step(eta)
    net.poll()
    out["J"] = float(J.item())
    out["dY"] = [to_np(net.get_tensor(mbd.T_DY, i)) for i in range(L)]
    out["new_W"] = [to_np(net.get_weights(i)) for i in range(L)]
    out["launches"] = net.launch_count
    if plans is not None:                      # (layer, product) -> mbd_get_plan, for the caller's assertions
        for key in list(plans):
            plans[key] = net.plan(*key)
    net.close()
    return out


def compare_conv_step(g, o, tol, fused=False, tol_below_relu=None, init=None, require_sized=False):
    L = len(o["Ys"])
    report, bad = [], []
    if tol_below_relu is None:
        tol_below_relu = tol

    def chk(name, got, ref, t):
        e = rel_fro(got, ref)
        report.append(f"{name}: {e:.3e}")
        if e > t:
            bad.append(name)

    assert abs(g["J"] - o["J"]) <= tol * abs(o["J"]), (g["J"], o["J"])
    for i in range(L):
        chk(f"Y[{i}]", g["act"][i], o["Ys"][i] if i == L - 1 else o["Xs"][i + 1], tol)
        tg = tol if i == L - 1 else tol_below_relu
        chk(f"dY[{i}]", g["dY"][i], o["dYs"][i], tg)
        if not fused:
            chk(f"dK[{i}]", g["dW"][i], like_device(o["dWs"][i], g["dW"][i]), tg)
        chk(f"K_new[{i}]", g["new_W"][i], like_device(o["new_W"][i], g["new_W"][i]), tg)
    if init is not None:
        od = dict(o)
        od["new_W"] = [like_device(o["new_W"][i], g["new_W"][i]) for i in range(L)]
        od["new_b"] = [None] * L
        update_checks(chk, g, od, init.Ws, None, [tol if i == L - 1 else tol_below_relu for i in range(L)], True,
                      require_sized)
    assert not bad, "rel. Frobenius error too large for %s: %s" % (bad, "; ".join(report))
    return report


# ---------------------------------------------------------------------------
# convolutions followed by fully connected layers (Section 2.4)
# ---------------------------------------------------------------------------
def oracle_mixed_step(w, inp, blocked_grid=None, eta=None, conv_split="domain"):
    """fp64 oracle step of a mixed workload: Conv3x3 layers on NCHW, then FC layers on the
    flattened activation; stored activations rounded to bf16 like the device's."""
    from oracle import mbd_oracle as O
    Lc = w.n_layers
    layers = [O.Conv3x3(oracle_kernel(inp.Ws[i]), relu=True, split=conv_split, stride=w.stride(i)) for i in range(Lc)]
    for i in range(Lc, w.L):
        layers.append(O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64), relu=True))
    X = inp.X.astype(np.float64)
    eta = w.eta if eta is None else eta
    if blocked_grid is None:
        return O.train_step(layers, X, inp.labels, "softmax_ce", eta, store=bf16_store)
    return O.train_step_blocked(layers, X, inp.labels, "softmax_ce", eta, *blocked_grid, store=bf16_store)


def mixed_layers(w, conv_split=None):
    from paper_1712_04432_b200 import mbd
    C_, H, Wd = w.dims
    split = {None: mbd.SPLIT_DOMAIN, "domain": mbd.SPLIT_DOMAIN, "batch": mbd.SPLIT_BATCH, "model": mbd.SPLIT_MODEL}[conv_split]
    return mbd.conv_layers(w.n_layers, C_, H, Wd, k=[w.kshape(i) for i in range(w.n_layers)], split=split, channels=w.channels,
                           strides=w.strides) + mbd.fc_layers(w.fc_dims, bias=True)


def oracle_mixed_acts(o, w):
    """The oracle's stored hidden activations in the device's layouts: NCHW for the outputs of
    the convolutions, [B, d] for the outputs of the hidden fully connected layers."""
    C_, H, Wd = w.dims
    out = []
    for i in range(w.L - 1):
        x = o["Xs"][i + 1]
        if i < w.n_layers:
            x = x if x.ndim == 4 else np.ascontiguousarray(x.T).reshape(w.B, w.chan(i + 1), *w.out_hw(i))
        else:
            x = x.T
        out.append(np.ascontiguousarray(x, np.float32))
    return out


def gpu_mixed_step(w, inp, grid=(1, 1), max_partials=0, fused=False, force_acts=None, eta=None, conv_split=None):
    """The same step through the C ABI; conv tensors come back NCHW, FC tensors [B, d]."""
    import torch
    from paper_1712_04432_b200 import mbd
    L, Lc = w.L, w.n_layers
    eta = w.eta if eta is None else eta
    net = mbd.Net(mixed_layers(w, conv_split), w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_SOFTMAX_CE, max_partials)
    for i in range(L):
        if i < Lc:
            net.set_weights(i, to_dev(inp.Ws[i], True))
        else:
            net.set_weights(i, to_dev(inp.Ws[i], True), torch.from_numpy(inp.bs[i]).cuda())
    X = to_dev(inp.X, True)
    labels = torch.from_numpy(inp.labels).cuda()
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = {}
    net.forward(X, labels, J)
    out["act"] = [to_np(net.get_tensor(mbd.T_ACT, i)) for i in range(L)]
    if force_acts is not None:
        for i in range(L - 1):
            net.set_tensor(mbd.T_ACT, i, to_dev(force_acts[i], True))
    if fused:
        net.backward(eta)
    else:
        net.backward(0.0)
        out["dW"] = [to_np(net.get_tensor(mbd.T_DW, i)) for i in range(L)]
        out["db"] = [to_np(net.get_tensor(mbd.T_DB, i)) if i >= Lc else None for i in range(L)]
        net.sgd_step(eta)
    net.poll()
    out["J"] = float(J.item())
    out["loss"] = to_np(net.get_tensor(mbd.T_LOSS))
    out["dY"] = [to_np(net.get_tensor(mbd.T_DY, i)) for i in range(L)]
    out["new_W"], out["new_b"] = [], []
    for i in range(L):
        if i < Lc:
            out["new_W"].append(to_np(net.get_weights(i))); out["new_b"].append(None)
        else:
            a, b = net.get_weights(i, with_bias=True)
            out["new_W"].append(to_np(a)); out["new_b"].append(to_np(b))
    out["launches"] = net.launch_count
    net.close()
    return out


def compare_mixed_step(g, o, w, tol, fused=False, tol_below_relu=None, init=None, require_sized=False):
    L, Lc = w.L, w.n_layers
    C_, H, Wd = w.dims
    report, bad = [], []
    if tol_below_relu is None:
        tol_below_relu = tol

    def chk(name, got, ref, t):
        e = rel_fro(got, ref)
        report.append(f"{name}: {e:.3e}")
        if e > t:
            bad.append(name)

    def dev_layout(a, i):
        """oracle tensor of layer i's output side -> the device's layout"""
        if i < Lc:
            return a if a.ndim == 4 else np.ascontiguousarray(a.T).reshape(w.B, w.chan(w.n_layers), *w.out_hw(w.n_layers - 1))
        return a.T

    assert abs(g["J"] - o["J"]) <= max(tol, 1e-4) * abs(o["J"]), (g["J"], o["J"])
    chk("per-sample loss", g["loss"], o["per_sample"], tol)
    for i in range(L):
        ref_act = o["Ys"][i] if i == L - 1 else o["Xs"][i + 1]
        chk(f"Y[{i}]", g["act"][i], dev_layout(ref_act, i), tol)
        tg = tol if i == L - 1 else tol_below_relu
        chk(f"dY[{i}]", g["dY"][i], dev_layout(o["dYs"][i], i), tg)
        if not fused:
            chk(f"dW[{i}]", g["dW"][i], like_device(o["dWs"][i], g["dW"][i]), tg)
            if i >= Lc:
                chk(f"db[{i}]", g["db"][i], o["dbs"][i], tg)
        chk(f"W_new[{i}]", g["new_W"][i], like_device(o["new_W"][i], g["new_W"][i]), tg)
        if i >= Lc:
            ref_b = o["new_b"][i]
            assert np.abs(g["new_b"][i] - ref_b).max() <= tg * max(1.0, np.abs(ref_b).max()), f"b_new[{i}]"
    if init is not None:
        od = dict(o)
        od["new_W"] = [like_device(o["new_W"][i], g["new_W"][i]) for i in range(L)]
        update_checks(chk, g, od, init.Ws, init.bs, [tol if i == L - 1 else tol_below_relu for i in range(L)], True,
                      require_sized)
    assert not bad, "rel. Frobenius error too large for %s: %s" % (bad, "; ".join(report))
    return report
