"""The step of Section 2.3 executed over a P_r x P_c grid of processes (paper_1712_04432_b200.grid_exec).

CPU part (gloo, 4 processes): the two process groups, the placement of the gathered blocks, the sums, and
the per-process word counts of the collectives against mbd_comm_words (Eq. 8).
GPU part: the same 2 or 4 processes share one GPU (their kernels never wait on one another; the collectives
go through host copies over gloo) and run the whole step; the gathered result is compared with the fp64
oracle, block by block, and the counted words again with mbd_comm_words."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
_PORTS = iter(range(29541, 29700))          # a fresh rendezvous port for every launch

COMM_WORKER = r'''
import json, sys
sys.path.insert(0, %(root)r)
import torch, torch.distributed as dist
from paper_1712_04432_b200.grid_exec import GridComm, grid_coords, expected_words
dist.init_process_group("gloo")
P_r, P_c = %(P_r)d, %(P_c)d
comm = GridComm(P_r, P_c)
rank = dist.get_rank()
r, c = grid_coords(rank, P_r, P_c)
assert (comm.r, comm.c) == (r, c) and rank == c * P_r + r
dims, B = %(dims)r, %(B)d
m = B // P_c
ok = True
for i in range(1, len(dims)):
    h = dims[i] // P_r
    # forward: block (r, c) holds the value 1000 c + r in every element; after the gather column block r' holds 1000 c + r'
    blk = torch.full((m, h), float(1000 * c + r))
    full = torch.empty((m, dims[i]))
    comm.all_gather_cols(blk, full)
    for rr in range(P_r):
        ok = ok and bool((full[:, rr * h:(rr + 1) * h] == 1000 * c + rr).all())
    if i > 1:
        part = torch.full((m, dims[i - 1]), float(r + 1))
        comm.all_reduce_(part, "rows", "allreduce_dx")
        ok = ok and bool((part == P_r * (P_r + 1) / 2).all())                  # summed over the P_r group only
    g = torch.full((h, dims[i - 1]), float(c + 1))
    comm.all_reduce_(g, "cols", "allreduce_dw")
    ok = ok and bool((g == P_c * (P_c + 1) / 2).all())                          # summed over the P_c group only
want = expected_words(dims, B, P_r, P_c)
got = {k: int(round(v)) for k, v in comm.words.items()}
ok = ok and got == want
outs = [None] * dist.get_world_size()
dist.all_gather_object(outs, (ok, got, want))
if rank == 0:
    print(json.dumps({"ok": all(o[0] for o in outs), "got": outs[0][1], "want": outs[0][2]}))
dist.destroy_process_group()
'''

STEP_WORKER = r'''
import json, os, sys
sys.path.insert(0, %(root)r)
import numpy as np
import torch, torch.distributed as dist
from paper_1712_04432_b200 import inputs as I
from paper_1712_04432_b200.grid_exec import GridComm, GridFC, expected_words
from tests.helpers import to_dev
torch.cuda.set_device(0)
dist.init_process_group("gloo")
P_r, P_c = %(P_r)d, %(P_c)d
dims, B, eta, out_dir = %(dims)r, %(B)d, %(eta)r, %(out)r
comm = GridComm(P_r, P_c, via_host=True)
w = I.fc_workload(dims, B, "bf16", "relu_normal")
inp = I.make_inputs(w, seed=%(seed)d)                      # every process draws the same tensors and takes its blocks
net = GridFC(dims, B, comm)
for i in range(len(dims) - 1):
    net.set_weights(i, to_dev(inp.Ws[i], True))
m = B // P_c
rows = slice(comm.c * m, (comm.c + 1) * m)
X_c = to_dev(inp.X[rows], True)
labels_c = torch.from_numpy(inp.labels[rows]).cuda()
loss = net.step(X_c, labels_c, eta)
torch.cuda.synchronize()
np.savez(os.path.join(out_dir, "rank%%d.npz" %% dist.get_rank()), r=comm.r, c=comm.c, loss=loss,
         logits=net.logits.float().cpu().numpy(),
         **{"W%%d" %% i: net.W[i].float().cpu().numpy() for i in range(net.L)},
         **{"dW%%d" %% i: net.dW[i].cpu().numpy() for i in range(net.L)},
         words=json.dumps({k: int(round(v)) for k, v in comm.words.items()}),
         want=json.dumps(expected_words(dims, B, P_r, P_c)))
dist.barrier()
dist.destroy_process_group()
'''


def _torchrun(script, nproc, port, timeout=600):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(nproc), "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script)]
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


@pytest.mark.parametrize("P_r,P_c", [(2, 2), (4, 1), (1, 2)])
def test_groups_placement_sums_and_word_counts(tmp_path, P_r, P_c):
    script = tmp_path / "comm_worker.py"
    script.write_text(COMM_WORKER % {"root": ROOT, "P_r": P_r, "P_c": P_c, "dims": [64, 32, 48, 16], "B": 12})
    r = _torchrun(script, P_r * P_c, next(_PORTS))
    assert r.returncode == 0, r.stderr[-3000:]
    d = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert d["ok"], d
    assert d["got"] == d["want"]


@pytest.mark.gpu
@pytest.mark.parametrize("P_r,P_c", [(2, 2), (1, 2), (2, 1), (4, 1)])
def test_step_over_a_grid_of_processes_matches_the_oracle(tmp_path, P_r, P_c):
    from paper_1712_04432_b200 import inputs as I
    from tests.helpers import oracle_fc_step, rel_fro
    dims, B, eta, seed = [136, 96, 64, 32], 24, 0.05, 91
    script = tmp_path / "step_worker.py"
    script.write_text(STEP_WORKER % {"root": ROOT, "P_r": P_r, "P_c": P_c, "dims": dims, "B": B, "eta": eta,
                                     "out": str(tmp_path), "seed": seed})
    r = _torchrun(script, P_r * P_c, next(_PORTS))
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])

    w = I.fc_workload(dims, B, "bf16", "relu_normal")
    w.eta = eta
    inp = I.make_inputs(w, seed=seed)
    for i in range(len(inp.bs)):
        inp.bs[i] = None                                     # the grid runner has no bias
    o = oracle_fc_step(w, inp)
    L, m = len(dims) - 1, B // P_c
    loss = 0.0
    for rank in range(P_r * P_c):
        z = np.load(tmp_path / f"rank{rank}.npz")
        rr, cc = int(z["r"]), int(z["c"])
        assert rank == cc * P_r + rr
        if rr == 0:
            loss += float(z["loss"])
        # the logits of this batch block, identical in every process of the P_r group
        assert rel_fro(z["logits"], o["Ys"][L - 1].T[cc * m:(cc + 1) * m]) < 1e-2
        for i in range(L):
            h = dims[i + 1] // P_r
            rows = slice(rr * h, (rr + 1) * h)
            assert rel_fro(z[f"dW{i}"], o["dWs"][i][rows]) < 1e-2, (rank, i)
            assert rel_fro(z[f"W{i}"], o["new_W"][i][rows]) < 1e-2, (rank, i)
        assert json.loads(str(z["words"])) == json.loads(str(z["want"]))          # Eq. 8, per process
    assert abs(loss - o["J"]) < 1e-2 * abs(o["J"])


CONV_WORKER = r'''
import json, os, sys
sys.path.insert(0, %(root)r)
import numpy as np
import torch, torch.distributed as dist
from paper_1712_04432_b200 import inputs as I, mbd
from paper_1712_04432_b200.grid_exec import GridComm, GridConv, expected_conv_words
from tests.helpers import to_dev
torch.cuda.set_device(0)
dist.init_process_group("gloo")
P_r, P_c = %(P_r)d, %(P_c)d
ksizes, H, W, B, eta, out_dir = %(ksizes)r, %(H)d, %(W)d, %(B)d, %(eta)r, %(out)r
comm = GridComm(P_r, P_c, via_host=True)
w = I.conv_workload(64, H, W, B, n_layers=len(ksizes), ksizes=ksizes)
inp = I.make_inputs(w, seed=%(seed)d)                      # every process draws the same tensors and takes its block
net = GridConv(ksizes, 64, H, W, B, comm)
for i in range(len(ksizes)):
    net.set_weights(i, to_dev(inp.Ws[i], True))
m = B // P_c
X_local = to_dev(np.ascontiguousarray(inp.X[comm.c * m:(comm.c + 1) * m, :, net.h0:net.h1, :]), True)
loss = net.step(X_local, eta)
torch.cuda.synchronize()
L = len(ksizes)
np.savez(os.path.join(out_dir, "rank%%d.npz" %% dist.get_rank()), r=comm.r, c=comm.c, loss=loss,
         Y=net.net.get_tensor(mbd.T_ACT, L - 1).float().cpu().numpy(),
         dY0=net.net.get_tensor(mbd.T_DY, 0).float().cpu().numpy(),
         **{"K%%d" %% i: net.net.get_weights(i).float().cpu().numpy() for i in range(L)},
         **{"dK%%d" %% i: net.dK[i].cpu().numpy() for i in range(L)},
         words=json.dumps({k: int(round(v)) for k, v in comm.words.items() if k in ("halo_fwd", "halo_bwd", "allreduce_dw")}),
         want=json.dumps(expected_conv_words(ksizes, 64, H, W, B, P_r, P_c)))
dist.barrier()
dist.destroy_process_group()
'''


@pytest.mark.gpu
@pytest.mark.parametrize("P_r,P_c,ksizes,H", [(2, 1, (3, 3), 16), (2, 2, (3, 1, 3), 16), (4, 1, (3, 3, 3), 16), (1, 2, (3, 3), 16),
                                              (3, 1, (3, 3), 10)])       # 10 rows on 3 processes: strips of 3, 3 and 4 rows
def test_convolution_step_over_a_grid_of_processes_matches_the_oracle(tmp_path, P_r, P_c, ksizes, H):
    from paper_1712_04432_b200 import inputs as I
    from tests.helpers import like_device, oracle_conv_step, rel_fro
    W, B, eta, seed = 40, 4, 2e-5, 92
    script = tmp_path / "conv_worker.py"
    script.write_text(CONV_WORKER % {"root": ROOT, "P_r": P_r, "P_c": P_c, "ksizes": list(ksizes), "H": H, "W": W, "B": B,
                                     "eta": eta, "out": str(tmp_path), "seed": seed})
    r = _torchrun(script, P_r * P_c, next(_PORTS))
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])

    w = I.conv_workload(64, H, W, B, n_layers=len(ksizes), ksizes=ksizes)
    w.eta = eta
    inp = I.make_inputs(w, seed=seed)
    o = oracle_conv_step(w, inp)
    L, m = len(ksizes), B // P_c
    loss = 0.0
    for rank in range(P_r * P_c):
        z = np.load(tmp_path / f"rank{rank}.npz")
        rr, cc = int(z["r"]), int(z["c"])
        loss += float(z["loss"])
        own = (slice(cc * m, (cc + 1) * m), slice(None), slice((rr * H) // P_r, ((rr + 1) * H) // P_r), slice(None))
        assert rel_fro(z["Y"], o["Ys"][L - 1][own]) < 1e-2, rank                 # this strip of the last layer's output
        assert rel_fro(z["dY0"], o["dYs"][0][own]) < 1e-2, rank                  # ... and of the gradient that reached layer 1
        for i in range(L):
            assert rel_fro(z[f"dK{i}"], like_device(o["dWs"][i], z[f"dK{i}"])) < 1e-2, (rank, i)
            assert rel_fro(z[f"K{i}"], like_device(o["new_W"][i], z[f"K{i}"])) < 1e-2, (rank, i)
        assert json.loads(str(z["words"])) == json.loads(str(z["want"]))        # Eq. 9's terms for domain layers, per process
    assert abs(loss - o["J"]) < 1e-2 * abs(o["J"])


MIXED_WORKER = r'''
import json, os, sys
sys.path.insert(0, %(root)r)
import numpy as np
import torch, torch.distributed as dist
from paper_1712_04432_b200 import inputs as I, mbd
from paper_1712_04432_b200.grid_exec import GridComm, GridMixed, expected_mixed_words
from tests.helpers import to_dev
torch.cuda.set_device(0)
dist.init_process_group("gloo")
P_r, P_c = %(P_r)d, %(P_c)d
ksizes, H, W, fc, B, eta, out_dir = %(ksizes)r, %(H)d, %(W)d, %(fc)r, %(B)d, %(eta)r, %(out)r
comm = GridComm(P_r, P_c, via_host=True)
w = I.mixed_workload(64, H, W, len(ksizes), fc, B, ksizes=ksizes)
inp = I.make_inputs(w, seed=%(seed)d)
net = GridMixed(ksizes, 64, H, W, fc, B, comm)
Lc = len(ksizes)
for i in range(Lc):
    net.conv.set_weights(i, to_dev(inp.Ws[i], True))
for i in range(len(fc)):
    net.fc.set_weights(i, to_dev(inp.Ws[Lc + i], True))
m, Hs = B // P_c, H // P_r
X_local = to_dev(np.ascontiguousarray(inp.X[comm.c * m:(comm.c + 1) * m, :, comm.r * Hs:(comm.r + 1) * Hs, :]), True)
labels_c = torch.from_numpy(inp.labels[comm.c * m:(comm.c + 1) * m]).cuda()
loss = net.step(X_local, labels_c, eta)
torch.cuda.synchronize()
np.savez(os.path.join(out_dir, "rank%%d.npz" %% dist.get_rank()), r=comm.r, c=comm.c, loss=loss,
         logits=net.fc.logits.float().cpu().numpy(),
         **{"K%%d" %% i: net.conv.net.get_weights(i).float().cpu().numpy() for i in range(Lc)},
         **{"dK%%d" %% i: net.conv.dK[i].cpu().numpy() for i in range(Lc)},
         **{"W%%d" %% i: net.fc.W[i].float().cpu().numpy() for i in range(len(fc))},
         **{"dW%%d" %% i: net.fc.dW[i].cpu().numpy() for i in range(len(fc))},
         words=json.dumps({k: int(round(v)) for k, v in comm.words.items()}),
         want=json.dumps(expected_mixed_words(ksizes, 64, H, W, fc, B, P_r, P_c)))
dist.barrier()
dist.destroy_process_group()
'''


@pytest.mark.gpu
@pytest.mark.parametrize("P_r,P_c,ksizes", [(2, 2, (3, 3)), (4, 1, (3, 1)), (1, 2, (3,)), (2, 1, (1, 3))])
def test_integrated_step_over_a_grid_of_processes_matches_the_oracle(tmp_path, P_r, P_c, ksizes):
    """Eq. 9 executed: domain-split convolutions, the re-distribution of Eq. 6, model-split fully connected layers."""
    from paper_1712_04432_b200 import inputs as I
    from tests.helpers import like_device, oracle_mixed_step, rel_fro
    H, W, fc, B, eta, seed = 8, 40, [64, 32], 4, 0.02, 93
    script = tmp_path / "mixed_worker.py"
    script.write_text(MIXED_WORKER % {"root": ROOT, "P_r": P_r, "P_c": P_c, "ksizes": list(ksizes), "H": H, "W": W, "fc": fc,
                                      "B": B, "eta": eta, "out": str(tmp_path), "seed": seed})
    r = _torchrun(script, P_r * P_c, next(_PORTS))
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])

    w = I.mixed_workload(64, H, W, len(ksizes), fc, B, ksizes=ksizes)
    w.eta = eta
    inp = I.make_inputs(w, seed=seed)
    o = oracle_mixed_step(w, inp)
    Lc, Lf, m = len(ksizes), len(fc), B // P_c
    dims = [64 * H * W] + fc
    loss = 0.0
    for rank in range(P_r * P_c):
        z = np.load(tmp_path / f"rank{rank}.npz")
        rr, cc = int(z["r"]), int(z["c"])
        if rr == 0:
            loss += float(z["loss"])
        assert rel_fro(z["logits"], o["Ys"][-1].T[cc * m:(cc + 1) * m]) < 1e-2, rank
        for i in range(Lc):
            assert rel_fro(z[f"dK{i}"], like_device(o["dWs"][i], z[f"dK{i}"])) < 1e-2, (rank, i)
            assert rel_fro(z[f"K{i}"], like_device(o["new_W"][i], z[f"K{i}"])) < 1e-2, (rank, i)
        for i in range(Lf):
            h = dims[i + 1] // P_r
            rows = slice(rr * h, (rr + 1) * h)
            assert rel_fro(z[f"dW{i}"], o["dWs"][Lc + i][rows]) < 1e-2, (rank, i)
            assert rel_fro(z[f"W{i}"], o["new_W"][Lc + i][rows]) < 1e-2, (rank, i)
        assert json.loads(str(z["words"])) == json.loads(str(z["want"]))
    assert abs(loss - o["J"]) < 1e-2 * abs(o["J"])


@pytest.mark.gpu
def test_command_line_driver_prints_words_equal_to_eq8():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(next(_PORTS)), "-m", "paper_1712_04432_b200.grid_exec", "--grid", "2x1", "--dims", "256,128,64",
           "--batch", "32", "--steps", "2", "--backend", "gloo"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    d = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert {k: int(round(v)) for k, v in d["words_per_process_per_step"].items()} == d["eq8_words_per_process"]
    assert d["ms_per_step"] > 0 and d["alpha_beta_seconds_nvlink5"] > 0
