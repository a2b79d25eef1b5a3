"""Runs a few launches of ONE kernel of the training step on synthetic data, for use under
a profiler (small, self-terminating):

    python -m paper_1712_04432_b200.profile_case gemm_fwd --size 8192 --launches 3
    python -m paper_1712_04432_b200.profile_case gemm_bwd_weight --size 4096
    python -m paper_1712_04432_b200.profile_case reduce --size 8192 --splits 2
    python -m paper_1712_04432_b200.profile_case conv --batch 4 --strips 4
    python -m paper_1712_04432_b200.profile_case conv --batch 64 --strips 2 --image 56
    python -m paper_1712_04432_b200.profile_case fc --batch 8192 --dims 1024,8192
    python -m paper_1712_04432_b200.profile_case fc --batch 8192 --dims 8192,8192,8192 --grid 16x16 --max-partials 2

gemm_*: one tensor-core contraction of size^3 in the operand layout of that product.
reduce: a split contraction followed by the partial-sum reduction (the reduction reads
`splits` fp32 planes of size^2 and writes one).
fc:     `launches` training steps of a small fully connected net (softmax, bias-gradient and
        update kernels at a size where their DRAM figures mean something); with --grid / --max-partials
        the products are launched as a workload on that logical grid launches them (two layers of
        8192 x 8192 at batch 8192 on 16x16 with 2 partials: the benchmark's three products, one of each
        per step plus a second forward and backward-weight product).
conv:   `launches` training steps of a two-layer convolution stack on `batch` images of
C_0 x image x image (default 64 x 224 x 224, 3 x 3 kernels), cut into `strips` row strips; --ksizes / --channels
select other odd kernel sizes and channel counts (the general convolution path), e.g.
    python -m paper_1712_04432_b200.profile_case conv --batch 16 --strips 2 --image 112 --ksizes 5,3 --channels 64,128,128
"""
import argparse

import torch

from . import mbd


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["gemm_fwd", "gemm_bwd_data", "gemm_bwd_weight", "reduce", "conv", "fc"])
    ap.add_argument("--dims", default="1024,8192")
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--strips", type=int, default=4)
    ap.add_argument("--image", type=int, default=224)
    ap.add_argument("--ksizes", default="3,3", help="conv: kernel size of each of the two layers (odd, up to 7)")
    ap.add_argument("--channels", default="64,64,64", help="conv: channels C_0,C_1,C_2 of the two layers (multiples of 8)")
    ap.add_argument("--strides", default="1,1", help="conv: stride of each of the two layers (1 to 4)")
    ap.add_argument("--size", type=int, default=8192)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--splits", type=int, default=2)
    ap.add_argument("--grid", default="1x1", help="fc: logical grid P_r x P_c")
    ap.add_argument("--max-partials", type=int, default=0, help="fc: as mbd_net_create")
    a = ap.parse_args()
    if a.case == "conv":
        return conv_case(a)
    if a.case == "fc":
        return fc_case(a)
    g = torch.Generator(device="cuda").manual_seed(0)
    n = a.size
    A = torch.randn((n, n), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    B = torch.randn((n, n), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    variant = {"gemm_fwd": 0, "gemm_bwd_data": 1, "gemm_bwd_weight": 2, "reduce": 2}[a.case]
    splits = a.splits if a.case == "reduce" else 1
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(a.launches):
        D = mbd.gemm_bf16(variant, A, B, k_splits=splits)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / a.launches
    print(f"{a.case} size={n} splits={splits}: {ms:.3f} ms per call, {2 * n ** 3 / ms / 1e9:.1f} TFLOP/s, "
          f"checksum {float(D.double().sum()):.6e}")


def fc_case(a):
    g = torch.Generator(device="cuda").manual_seed(0)
    dims = [int(d) for d in a.dims.split(",")]
    P_r, P_c = (int(x) for x in a.grid.lower().split("x"))
    net = mbd.Net(mbd.fc_layers(dims), a.batch, P_r, P_c, mbd.BF16, mbd.LOSS_SOFTMAX_CE, a.max_partials)
    for i in range(len(dims) - 1):
        for product in ((0, 2) if i == 0 else (0, 1, 2)):
            print(f"layer {i} product {product}: {net.plan(i, product)}")
    for i in range(len(dims) - 1):
        W = (torch.randn((dims[i + 1], dims[i]), generator=g, device="cuda") / dims[i] ** 0.5).to(torch.bfloat16)
        net.set_weights(i, W)
    X = torch.randn((a.batch, dims[0]), generator=g, device="cuda").to(torch.bfloat16)
    labels = torch.randint(0, dims[-1], (a.batch,), generator=g, device="cuda", dtype=torch.int32)
    J = torch.zeros(1, device="cuda")
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(a.launches):
        net.forward(X, labels, J)
        net.backward(0.01)
    ev1.record()
    torch.cuda.synchronize()
    net.poll()
    print(f"fc dims={dims} batch={a.batch} grid={a.grid} max_partials={a.max_partials}: "
          f"{ev0.elapsed_time(ev1) / a.launches:.3f} ms per step, J = {J.item():.4e}")


def conv_case(a):
    g = torch.Generator(device="cuda").manual_seed(0)
    ks = [int(k) for k in a.ksizes.split(",")]
    ch = [int(c) for c in a.channels.split(",")]
    st = [int(x) for x in a.strides.split(",")]
    net = mbd.Net(mbd.conv_layers(2, ch[0], a.image, a.image, k=ks, channels=ch, strides=st), a.batch, a.strips, 1, mbd.BF16, mbd.LOSS_HALF_SSQ, 0)
    for i in range(2):
        K = (torch.randn((ch[i + 1], ch[i], ks[i], ks[i]), generator=g, device="cuda") * (2.0 / (ch[i] * ks[i] ** 2)) ** 0.5).to(torch.bfloat16)
        net.set_weights(i, K)
    X = torch.randn((a.batch, ch[0], a.image, a.image), generator=g, device="cuda").to(torch.bfloat16)
    J = torch.zeros(1, device="cuda")
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(a.launches):
        net.forward(X, None, J)
        net.backward(1e-7)
    ev1.record()
    torch.cuda.synchronize()
    net.poll()
    print(f"conv batch={a.batch} image={a.image} strips={a.strips} kernels={ks} channels={ch} strides={st}: {ev0.elapsed_time(ev1) / a.launches:.3f} ms per step, J = {J.item():.4e}")


if __name__ == "__main__":
    main()
