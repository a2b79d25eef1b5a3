#!/usr/bin/env python
"""Training-step throughput of the matrix-form minibatch-SGD step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--grid 16x16]
                    [--max-partials 2] [--impl ours|reference]

One step = forward + loss + backward over the logical P_r x P_c grid + fused SGD update
on one batch of synthetic input.  `value` is timed with inputs resident in HBM; `e2e` goes
through mbd_train_step_host_begin / _end (two steps in flight) with pinned host buffers (H2D of the batch and D2H of the loss
inside the timed region).  With N > 1 (torchrun) every rank runs an independent replica
(weak scaling, no data-path collective); time is the max over ranks.  `--impl reference`
times the fp64 CPU oracle on a bounded sample of the same workload.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1712_04432_b200 import inputs as I  # noqa: E402

METRIC = "training-step TFLOP/s (fwd+bwd+update)"
SMI_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg5", choices=sorted(I.WORKLOADS))
    ap.add_argument("--momentum", type=float, default=None,
                    help="heavy-ball momentum with this mu (the update becomes a kernel of its own); not the default")
    ap.add_argument("--master-weights", action="store_true",
                    help="keep fp32 master weights (the update leaves the contraction's epilogue); not the default")
    ap.add_argument("--grid", default=None, help="P_r x P_c, e.g. 16x16 (default: the workload's second grid)")
    ap.add_argument("--max-partials", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="logical", choices=["logical", "grid"],
                    help="logical (default): the P_r x P_c grid as logical blocks on every GPU (replicas for N > 1).  "
                         "grid: one PROCESS per grid position (P_r * P_c = N, --grid required for N > 1), collectives "
                         "over NCCL; fully connected workloads only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks / throttle reasons of one GPU, sampled every 200 ms while running."""

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={SMI_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def pick_grid(w, arg):
    if arg:
        a, b = arg.lower().split("x")
        return int(a), int(b)
    return w.grids[1] if len(w.grids) > 1 else w.grids[0]


def workload_config(w, grid, max_partials):
    if w.kind == "fc":
        desc = f"{w.name}: FC stack {'-'.join(str(d) for d in w.dims)}, B={w.B}, ReLU, softmax-CE, {w.dtype}"
    elif w.kind == "mixed":
        if w.channels or w.strides or w.ksizes:
            lay = ", ".join(f"{w.kshape(i)[0]}x{w.kshape(i)[1]}{'/' + str(w.stride(i)) if w.stride(i) > 1 else ''} {w.chan(i)}->{w.chan(i + 1)}"
                            for i in range(w.n_layers))
            desc = (f"{w.name}: conv layers {lay} on {w.dims[1]}x{w.dims[2]}, then FC "
                    f"{'-'.join(str(d) for d in w.fc_dims)}, B={w.B}, ReLU, softmax-CE, {w.dtype}")
        else:
            desc = (f"{w.name}: {w.n_layers}x conv3x3 {w.dims[0]}ch on {w.dims[1]}x{w.dims[2]}, then FC "
                    f"{'-'.join(str(d) for d in w.fc_dims)}, B={w.B}, ReLU, softmax-CE, {w.dtype}")
    else:
        if w.channels or w.strides or any(w.kshape(i) != w.kshape(0) for i in range(w.n_layers)):
            lay = ", ".join(f"{w.kshape(i)[0]}x{w.kshape(i)[1]}{'/' + str(w.stride(i)) if w.stride(i) > 1 else ''} {w.chan(i)}->{w.chan(i + 1)}"
                            for i in range(w.n_layers))
            desc = f"{w.name}: conv layers {lay} on {w.dims[1]}x{w.dims[2]}, B={w.B}, half-SSQ, {w.dtype}"
        else:
            ks = "x".join(str(w.ksize(0)) * 2)
            desc = f"{w.name}: {w.n_layers}x conv{ks} {w.dims[0]}ch on {w.dims[1]}x{w.dims[2]}, B={w.B}, half-SSQ, {w.dtype}"
    return dict(workload=desc, grid=f"{grid[0]}x{grid[1]}", max_partials=max_partials, batch=w.B,
                l2="weights + activations per step exceed the 126 MB L2 (no flush needed)"
                if I.step_flops(w) > 1e12 else "L2 flushed by a 256 MB write between steps")


# ------------------------------------------------------------------------------ oracle timing
def oracle_sample(w, inp):
    """Time the fp64 oracle, as it stands, on a bounded sample of the workload: the whole
    network on the first `Bs` samples of the batch.  Returns (flops, seconds, description)."""
    from oracle import mbd_oracle as O
    if w.kind == "fc":
        flops_per_sample = I.step_flops(w) / w.B
        # aim at roughly 1.5 TFLOP of fp64 work at most
        Bs = int(max(1, min(w.B, 1.5e12 // flops_per_sample)))
        layers = [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64)) for i in range(len(inp.Ws))]
        X = inp.X[:Bs].astype(np.float64).T
        labels = inp.labels[:Bs]
        t0 = time.perf_counter()
        O.train_step(layers, X, labels, "softmax_ce", w.eta)
        dt = time.perf_counter() - t0
        return flops_per_sample * Bs, dt, f"whole {len(layers)}-layer network, first {Bs} of {w.B} samples, fp64 numpy"
    if w.kind == "mixed":
        Bs = min(w.B, 4)
        layers = [O.Conv3x3(inp.Ws[i].astype(np.float64), stride=w.stride(i)) for i in range(w.n_layers)]
        layers += [O.FC(inp.Ws[i].astype(np.float64), inp.bs[i].astype(np.float64)) for i in range(w.n_layers, w.L)]
        X = inp.X[:Bs].astype(np.float64)
        t0 = time.perf_counter()
        O.train_step(layers, X, inp.labels[:Bs], "softmax_ce", w.eta)
        dt = time.perf_counter() - t0
        return I.step_flops(w) / w.B * Bs, dt, f"whole {w.L}-layer network, first {Bs} of {w.B} samples, fp64 numpy"
    C, H, Wd = w.dims
    Bs, Hs = 1, min(H, 56)
    def as3x3(k):          # the oracle's layer is 3 x 3: a 1 x 1 kernel is its centre tap
        k = k.astype(np.float64)
        if k.shape[2:] != (1, 1):
            return k
        k3 = np.zeros(k.shape[:2] + (3, 3))
        k3[:, :, 1, 1] = k[:, :, 0, 0]
        return k3

    layers = [O.Conv3x3(as3x3(k), stride=w.stride(i)) for i, k in enumerate(inp.Ws)]
    X = inp.X[:Bs, :, :Hs, :].astype(np.float64)
    t0 = time.perf_counter()
    O.train_step(layers, X, None, "half_ssq", w.eta)
    dt = time.perf_counter() - t0
    flops = I.step_flops(w) / w.B / H * Bs * Hs          # the method's flops for these rows (1 x 1 layers: one tap)
    return flops, dt, f"{w.n_layers} conv layers on {Bs} image(s), first {Hs} rows, fp64 numpy"


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info()]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def small_inputs_for_oracle(w):
    """Inputs for the oracle sample without drawing the whole batch when it is huge."""
    if w.kind == "fc" and w.B > 1024:
        ws = I.Workload(w.name, w.kind, w.dims, 1024, w.dtype, w.x_dist, w.loss, w.eta)
        inp = I.make_inputs(ws, seed=0)
        return inp
    return I.make_inputs(w, seed=0)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = I.WORKLOADS[args.workload]
    grid = pick_grid(w, args.grid)
    inp = small_inputs_for_oracle(w)
    times, flops, desc = [], 0.0, ""
    for i in range(args.warmup + args.steps):
        flops, dt, desc = oracle_sample(w, inp)
        if i >= args.warmup:
            times.append(dt)
        if sum(times) > 150.0:      # keep the whole run within a few minutes
            break
    dt = sum(times) / len(times)
    val = flops / dt / 1e12
    cores = host_threads()
    line = dict(impl="reference", metric=METRIC, value=val, unit="TFLOP/s", n_gpus=args.gpus, steps=len(times),
                warmup=args.warmup, ms_per_step=dt * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", config=workload_config(w, grid, args.max_partials),
                cpu_baseline=dict(value=val, unit="TFLOP/s", cores=cores, kind="oracle", sample=desc),
                e2e=dict(value=val, unit="TFLOP/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ our arm
def max_over_ranks(x: float, world: int, device="cuda") -> float:
    """The slowest rank decides a multi-GPU time."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flops_per_replica: float, world: int, ms: float) -> float:
    """Whole-job throughput: every rank runs one replica of the step (weak scaling)."""
    return flops_per_replica * world / (ms * 1e-3) / 1e12


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1712_04432_b200 import mbd

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    torch.cuda.set_stream(torch.cuda.Stream())       # a capturable stream for everything below
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = I.WORKLOADS[args.workload]
    grid = pick_grid(w, args.grid)
    bf = w.dtype == "bf16"
    inp = I.make_inputs(w, seed=rank)          # every replica draws its own batch and weights
    flops = float(I.step_flops(w))

    def dev(a):
        a = np.ascontiguousarray(a, np.float32)
        if bf:
            return torch.from_numpy(I.bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    if w.kind == "fc":
        net = mbd.Net(mbd.fc_layers(w.dims, bias=True), w.B, grid[0], grid[1], mbd.BF16 if bf else mbd.F32,
                      mbd.LOSS_SOFTMAX_CE, args.max_partials)
        for i, Wi in enumerate(inp.Ws):
            net.set_weights(i, dev(Wi), torch.from_numpy(inp.bs[i]).cuda())
        labels = torch.from_numpy(inp.labels).cuda()
        labels_host = torch.from_numpy(inp.labels).pin_memory()
    elif w.kind == "mixed":
        C_, H, Wd = w.dims
        net = mbd.Net(mbd.conv_layers(w.n_layers, C_, H, Wd, k=[w.kshape(i) for i in range(w.n_layers)], channels=w.channels,
                                      strides=w.strides) + mbd.fc_layers(w.fc_dims, bias=True), w.B, grid[0], grid[1],
                      mbd.BF16, mbd.LOSS_SOFTMAX_CE, args.max_partials)
        for i, Wi in enumerate(inp.Ws):
            net.set_weights(i, dev(Wi), None if inp.bs[i] is None else torch.from_numpy(inp.bs[i]).cuda())
        labels = torch.from_numpy(inp.labels).cuda()
        labels_host = torch.from_numpy(inp.labels).pin_memory()
    else:
        C_, H, Wd = w.dims
        net = mbd.Net(mbd.conv_layers(w.n_layers, C_, H, Wd, k=[w.kshape(i) for i in range(w.n_layers)], channels=w.channels,
                                      strides=w.strides),
                      w.B, grid[0], grid[1], mbd.BF16, mbd.LOSS_HALF_SSQ, args.max_partials)
        for i, Ki in enumerate(inp.Ws):
            net.set_weights(i, dev(Ki))
        labels = labels_host = None
    if args.master_weights:
        net.enable_master_weights()
    if args.momentum is not None:
        net.enable_momentum(args.momentum)
    X = dev(inp.X)
    X_host = X.cpu().pin_memory()
    J = torch.zeros(1, dtype=torch.float32, device="cuda")
    flush = None
    if flops < 1e12:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    # Small workloads are dominated by launch cost: their timed steps replay the CUDA graph the
    # library captures (mbd_train_step); the per-kernel events then come from a second, directly
    # launched pass.  The large fully connected workload launches directly with the events inside the timed region
    # (23 long kernels per step); a convolution stack has dozens of short launches whatever its size.
    use_graph = flops < 1e12 or w.kind != "fc"

    def step():
        if flush is not None:
            flush.fill_(1)
        if use_graph:
            net.train_step(X, labels, w.eta, J)
        else:
            net.forward(X, labels, J)
            net.backward(w.eta)

    for _ in range(max(args.warmup, 3)):
        step()
    net.poll()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    if not use_graph:
        net.profile_enable(True)
    launches0 = net.launch_count
    barrier()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for k in range(args.steps):
        if flush is not None:
            flush.fill_(1)
        evs[k][0].record()
        if use_graph:
            net.train_step(X, labels, w.eta, J)
        else:
            net.forward(X, labels, J)
            net.backward(w.eta)
        evs[k][1].record()
    torch.cuda.synchronize()
    barrier()
    launches = net.launch_count - launches0
    per_step = [a.elapsed_time(b) for a, b in evs]
    ms = sum(per_step) / len(per_step)               # flush time excluded
    ms = max_over_ranks(ms, world)
    prof_ms = ms
    if use_graph:
        net.profile_enable(True)
        pe = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for k in range(args.steps):
            if flush is not None:
                flush.fill_(1)
            pe[k][0].record()
            net.forward(X, labels, J)
            net.backward(w.eta)
            pe[k][1].record()
        torch.cuda.synchronize()
        prof_ms = sum(a.elapsed_time(b) for a, b in pe) / args.steps
    prof = net.profile_read()
    net.profile_enable(False)
    net.poll()
    loss_last = float(J.item())

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        # Two steps in flight: the host-to-device copy of batch k+1 (library's copy stream) runs under
        # the compute of batch k; every step's batch is copied from pinned host memory and every
        # step's loss is read back on the host inside the timed region.
        for _ in range(2):
            net.train_step_host(X_host, labels_host, w.eta)
        barrier()
        t0 = time.perf_counter()
        net.train_step_host_begin(X_host, labels_host, w.eta)
        for _ in range(args.steps - 1):
            net.train_step_host_begin(X_host, labels_host, w.eta)
            net.train_step_host_end()                              # loss of the older step, on the host
        net.train_step_host_end()
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.steps
        dt = max_over_ranks(dt, world)
        h2d = X_host.numel() * X_host.element_size() + (labels_host.numel() * 4 if labels_host is not None else 0)
        e2e = dict(value=aggregate_tflops(flops, world, dt * 1e3), unit="TFLOP/s", h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=4,
                   ms_per_step=dt * 1e3)
    # ---- the partial-sum reduction kernel on its own (outside the timed region): with few partial sums per
    # reduction the step adds them inside the products' epilogues and never launches it, so its HBM rate is
    # measured here, on two fp32 planes of the workload's largest weight matrix with the update of Eq. 1 as tail
    reduce_probe = None
    if rank == 0 and bf and w.kind == "fc":
        d_out, d_in = max(((w.dims[i + 1], w.dims[i]) for i in range(len(w.dims) - 1)), key=lambda t: t[0] * t[1])
        parts = torch.randn((2, d_out, d_in), dtype=torch.float32, device="cuda")
        Wp = torch.randn((d_out, d_in), dtype=torch.float32, device="cuda").to(torch.bfloat16)
        reps = 5
        for _ in range(2):
            mbd.block_reduce(parts, Wp, mbd.TAIL_SGD, scale=-1e-6, sync=False)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a_, b_ in ev:
            if flush is not None:
                flush.fill_(1)
            a_.record()
            mbd.block_reduce(parts, Wp, mbd.TAIL_SGD, scale=-1e-6, sync=False)
            b_.record()
        torch.cuda.synchronize()
        r_ms = sum(a_.elapsed_time(b_) for a_, b_ in ev) / reps
        r_bytes = d_out * d_in * (2 * 4 + 2 + 2)          # two fp32 planes read, bf16 weights read and written
        peaks_ = measured_peaks()
        reduce_probe = dict(kernel="reduce_partials_vec8_two_planes + Eq. 1 tail" if d_out * d_in >= (2 << 20) else "reduce_partials_vec8 + Eq. 1 tail",
                            shape=[2, d_out, d_in], ms=r_ms, algorithmic_bytes=r_bytes, achieved=r_bytes / (r_ms * 1e-3) / 1e9,
                            peak=peaks_["hbm_gbs"], unit="GB/s", frac=r_bytes / (r_ms * 1e-3) / 1e9 / peaks_["hbm_gbs"],
                            peak_kind=f"{peaks_['source']} copy bandwidth")
        del parts, Wp
    clocks = sampler.stop() if rank == 0 else None
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # dominant kernel class by device time
    dom = max(prof.items(), key=lambda kv: kv[1]["ms"])[0] if prof else None
    gemm = {k: v for k, v in prof.items() if k.startswith("gemm") or k.startswith("conv")}
    roofline = None
    if gemm:
        g_ms = sum(v["ms"] for v in gemm.values())
        g_fl = sum(v["work"] for v in gemm.values())
        g_n = sum(v["launches"] for v in gemm.values())
        ach = g_fl / (g_ms * 1e-3) / 1e12
        # fp32 check mode runs on the FMA pipes: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
        peak = peaks["bf16_tflops_sustained"] if bf else 148 * 128 * 2 * 1.965e9 / 1e12
        if w.kind == "conv":
            kname = "conv_fwd_kernel (forward, backward-data) + conv_wgrad_kernel"
        elif w.kind == "mixed":
            kname = ("gemm_tc_kernel (convolutions as shifted-view products, fully connected layers)" if (w.channels or w.strides) else
                     "conv_fwd_kernel + conv_wgrad_kernel (convolutions), gemm_tc_kernel (fully connected layers)")
        elif bf:
            kname = "gemm_tc_kernel (all three operand layouts)"
        else:
            kname = "simt_gemm_kernel (fp32 check mode)"
        roofline = dict(bound="tensor" if bf else "alu", kernel=kname,
                        achieved=ach, peak=peak, unit="TFLOP/s", frac=(ach / peak) if peak else None,
                        peak_kind=(f"{peaks['source']} sustained bf16 (kernel timed inside a long step); "
                                   f"burst {peaks['bf16_tflops']}") if bf else
                                  "derived fp32 FMA peak: 148 SMs x 128 lanes x 2 flop x 1965 MHz",
                        frac_of_burst=ach / peaks["bf16_tflops"] if bf else None,
                        launches=g_n, avg_launch_ms=g_ms / g_n, flops_per_launch=g_fl / g_n,
                        share_of_step=g_ms / (prof_ms * args.steps),
                        traffic=(traffic_for(w, grid, args.max_partials) or {}).get("per_launch_mean"),
                        traffic_detail=traffic_for(w, grid, args.max_partials),
                        note="with few partial sums per reduction the backward products add their K pieces in their own "
                             "epilogue: the flops counted here are the products' alone, the time includes that reduction"
                             if bf and w.kind == "fc" else None,
                        timed_in="second pass, direct launches" if use_graph else "the timed region")
    kernels = {k: dict(ms_per_step=v["ms"] / args.steps, launches_per_step=v["launches"] / args.steps,
                       rate=(v["work"] / (v["ms"] * 1e-3) / (1e12 if (k.startswith("gemm") or k.startswith("conv_")) else 1e9))
                       if v["ms"] > 0 else None,
                       rate_unit="TFLOP/s" if (k.startswith("gemm") or k.startswith("conv_")) else "GB/s")
               for k, v in prof.items()}
    if "colsum" in kernels:
        kernels["colsum"]["note"] = "side stream, beside the products: the events span the co-running time, off the critical path"

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        inp_o = small_inputs_for_oracle(w)
        fl, dt, desc = oracle_sample(w, inp_o)
        cpu = dict(value=fl / dt / 1e12, unit="TFLOP/s", cores=host_threads(), kind="oracle", sample=desc,
                   seconds=dt)

    line = dict(metric=METRIC, value=aggregate_tflops(flops, world, ms), unit="TFLOP/s", n_gpus=world,
                steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype=w.dtype, data="synthetic",
                config=dict(workload_config(w, grid, args.max_partials), **({"master_weights": True} if args.master_weights else {}),
                            **({"momentum": args.momentum} if args.momentum is not None else {})),
                clocks=clocks, e2e=e2e,
                gpu_launches=int(launches) * world, roofline=roofline, cpu_baseline=cpu,
                frac_of_burst_peak=flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"] if bf else None,
                kernels=kernels, reduce_partials_probe=reduce_probe, dominant_kernel_class=dom, loss_last=loss_last,
                launch_mode="CUDA graph replay (mbd_train_step)" if use_graph else "direct launches",
                ms_per_step_direct=prof_ms if use_graph else None,
                ms_per_step_median=float(np.median(per_step)), ms_per_step_min=float(min(per_step)),
                ms_per_step_max=float(max(per_step)))
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ the grid over processes
def run_grid(args):
    """Section 2.3 for real: rank (r, c) of a P_r x P_c grid of processes owns W_i(r, :) and batch block c; block
    products with their tail operations in the library's kernels, all-gather / all-reduce over NCCL.  Strong
    scaling: the workload is fixed, the grid divides it.  Prints ms per step (slowest rank, CUDA events), the
    words every process moved per step against mbd_comm_words (Eq. 8), and the alpha-beta model's time for them."""
    import torch
    import torch.distributed as dist
    from paper_1712_04432_b200 import mbd
    from paper_1712_04432_b200.grid_exec import GridComm, GridFC, expected_words

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    os.environ.setdefault("RANK", "0")
    os.environ.setdefault("WORLD_SIZE", "1")
    torch.cuda.set_device(local)
    dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    w = I.WORKLOADS[args.workload]
    if w.kind != "fc" or w.dtype != "bf16":
        raise SystemExit("--mode grid runs the bf16 fully connected workloads (cfg2, cfg3, cfg5)")
    P_r, P_c = (int(x) for x in args.grid.lower().split("x")) if args.grid else (world, 1)
    if P_r * P_c != world:
        raise SystemExit(f"--grid {P_r}x{P_c} needs {P_r * P_c} processes, got {world}")
    comm = GridComm(P_r, P_c)
    net = GridFC(w.dims, w.B, comm)
    inp = I.make_inputs(w, seed=0)             # every process draws the same tensors and keeps its blocks

    def dev(a):
        return torch.from_numpy(I.bf16_bits(np.ascontiguousarray(a, np.float32)).view(np.int16)).cuda().view(torch.bfloat16)

    for i in range(len(w.dims) - 1):
        a, b = net.rows(i)
        net.W[i].copy_(dev(inp.Ws[i][a:b]))
    m = w.B // P_c
    X_c = dev(inp.X[comm.c * m:(comm.c + 1) * m])
    labels_c = torch.from_numpy(inp.labels[comm.c * m:(comm.c + 1) * m]).cuda()
    del inp
    for _ in range(max(args.warmup, 3)):
        net.step(X_c, labels_c, w.eta)
    for k in comm.words:
        comm.words[k] = 0.0
    dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    loss = 0.0
    for _ in range(args.steps):
        loss = net.step(X_c, labels_c, w.eta)
    ev1.record()
    torch.cuda.synchronize()
    dist.barrier()
    ms = max_over_ranks(ev0.elapsed_time(ev1) / args.steps, world)
    if rank == 0:
        flops = float(I.step_flops(w))
        model = mbd.comm_time(mbd.fc_layers(w.dims, bias=False), w.B, P_r, P_c, mbd.MACHINE_B200_NVLINK5)
        line = dict(metric=METRIC, value=flops / (ms * 1e-3) / 1e12, unit="TFLOP/s", n_gpus=world, steps=args.steps,
                    warmup=max(args.warmup, 3), ms_per_step=ms, higher_is_better=True, scaling="strong", vs_baseline=None,
                    dtype=w.dtype, data="synthetic",
                    config=dict(workload=workload_config(w, (P_r, P_c), 0)["workload"], grid=f"{P_r}x{P_c}",
                                mode="one process per grid position, NCCL collectives", batch=w.B),
                    words_per_process_per_step={k: v / args.steps for k, v in comm.words.items()},
                    eq8_words_per_process=expected_words(w.dims, w.B, P_r, P_c),
                    alpha_beta_seconds_nvlink5=sum(sum(t.values()) for t in model), loss_block_0=loss)
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of
# the same three products in the same plan: profiles/gemm_tc_kernel_8192_step_products.md).  gemm_tc_kernel is
# launched 23 times per step of cfg5 on 16x16 with 2 partials: 8 forward products (0.944 GB each), 7 backward-data
# (1.604 GB) and 8 backward-weight products (1.585 GB) whose two K pieces are added as a running sum in the
# epilogue (one fp32 plane written and read back inside the launch).  Other plans have no capture: null.
TRAFFIC_CFG5_16X16_2 = dict(per_launch_mean=(8 * 0.944e9 + 7 * 1.604e9 + 8 * 1.585e9) / 23,
                            forward=0.944e9, backward_data=1.604e9, backward_weight=1.585e9,
                            algorithmic=dict(forward=384e6, backward_data=384e6 + 134e6, backward_weight=384e6 + 134e6),
                            source="profiles/gemm_tc_kernel_8192_step_products.md")


def traffic_for(w, grid, max_partials):
    if w.name == "cfg5" and tuple(grid) == (16, 16) and max_partials == 2 and not os.environ.get("MBD_NO_FIXUP"):
        return TRAFFIC_CFG5_16X16_2
    return None


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.mode == "grid":
        run_grid(a)
    else:
        run_ours(a)
