"""The column-sharded product path under two live ranks (two processes, one process group).

Only one GPU is available to the tests, so both ranks use cuda:0 and the process group is gloo: the ranks' kernels
never wait on one another (the one exchange step, the sum of the partial SVM margins, goes through the host), so they
may share a device.  What runs per rank is the product: hop_step, or hop_step_begin -> all-reduce -> hop_step_end."""
import dataclasses
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from oracle import protocol as op, update as up
from paper_1902_01064_b200 import inputs

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TOL_RUN = 1e-4


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _start(w, x0, lo, hi):
    """Context, ring and data of one column shard [lo, hi) on cuda:0."""
    from paper_1902_01064_b200 import hop
    dev = "cuda:0"
    ws = dataclasses.replace(w, P=hi - lo, svm=(w.svm.column_shard(lo, hi) if w.svm is not None else None), _p0=None)
    X = torch.zeros((w.N, w.s + 1, ws.P), dtype=torch.float32, device=dev)
    M = torch.zeros((w.N, ws.P), dtype=torch.float32, device=dev) if w.momentum else None
    G = None if w.grad_mode == inputs.GRAD_SVM_CSR else torch.zeros((w.N, ws.P), dtype=torch.float32, device=dev)
    h = hop.from_workload(ws)
    h.set_option(hop.OPT_COL_OFFSET, lo)
    h.bind_buffers(X, M, G, torch.cuda.current_stream().cuda_stream)
    keep = [X, M, G]
    if w.grad_mode == inputs.GRAD_SVM_DENSE:
        keep += [torch.from_numpy(ws.svm.dense).to(dev), torch.from_numpy(ws.svm.y).to(dev)]
        h.bind_svm_dense(keep[-2], keep[-1], ws.svm.rows_per_worker, ws.svm.batch)
    elif w.grad_mode == inputs.GRAD_SVM_CSR:
        keep += [torch.from_numpy(a).to(dev) for a in (ws.svm.row_ptr, ws.svm.col, ws.svm.val, ws.svm.y)]
        h.bind_svm_csr(*keep[-4:], ws.svm.rows_per_worker, ws.svm.batch)
    h.load_trace(h.sim_run(w.ticks, w.iters))
    for i in range(w.N):
        h.write_params(i, 0, np.ascontiguousarray(x0[i, lo:hi]))
    return h, keep


def _rank_main(rank, world, port, cfg, P, iters, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1902_01064_b200 import hop
    torch.cuda.set_device(0)
    w = inputs.make_workload(cfg, P=P, iters=iters)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    lo, hi = bench.shard_columns(P, world, rank)
    h, keep = _start(w, x0, lo, hi)
    for k in range(iters):
        if w.svm is not None:
            ptr, n = h.step_begin()
            part = torch.as_tensor(hop.DeviceSpan(ptr, n), device="cuda:0")
            host = part.cpu()                               # the stream is synchronised by the copy
            dist.all_reduce(host)                           # sum of the partial margins over the column shards
            part.copy_(host.to("cuda:0"))
            h.step_end()
        else:
            h.step()
    assert h.read_status() == 0
    mine = np.stack([h.read_params(i) for i in range(w.N)])
    newest = [h.newest_version(i) for i in range(w.N)]
    parts = [None] * world
    dist.all_gather_object(parts, (lo, mine, newest))
    dist.barrier()
    if rank == 0:
        assert all(p[2] == newest for p in parts)
        np.save(out, np.concatenate([p[1] for p in sorted(parts, key=lambda p: p[0])], axis=1))
    h.close()
    dist.destroy_process_group()


@pytest.mark.parametrize("cfg,P,iters", [(4, 5120, 20), (2, 4096, 24), (1, 1000, 20)])
def test_two_ranks_on_one_gpu_match_the_oracle(tmp_path, cfg, P, iters):
    out = str(tmp_path / "ranks.npy")
    mp.spawn(_rank_main, args=(2, _free_port(), cfg, P, iters, out), nprocs=2, join=True)
    got = np.load(out)
    w = inputs.make_workload(cfg, P=P, iters=iters)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    tr = op.simulate(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode,
                     stale_reduce=w.stale_reduce).to_arrays()
    if w.grad_mode == inputs.GRAD_SYNTHETIC:
        grad = up.GradSynthetic(w.grad_seed, w.sigma, np.arange(P))
    elif w.grad_mode == inputs.GRAD_SVM_DENSE:
        grad = up.GradSvmDense(w.svm.dense, w.svm.y, w.svm.batch, "hinge")
    else:
        grad = up.GradSvmCsr(w.svm.row_ptr, w.svm.col, w.svm.val, w.svm.y, w.svm.rows_per_worker, w.svm.batch, "hinge")
    X, newest = up.run_updates(tr, w.N, w.lr, w.momentum, x0.astype(np.float64), grad, levels=iters, s=w.s)
    want = np.stack([X[(i, newest[i])] for i in range(w.N)])
    scale = np.abs(want).max()
    worst = np.abs(got - want).max()
    assert worst <= TOL_RUN * scale, (worst, scale)
    if cfg == 4:                                   # no exchange step: the shards equal the unsharded GPU run bit for bit
        h, keep = _start(w, x0, 0, P)
        for k in range(iters):
            h.step()
        assert h.read_status() == 0
        full = np.stack([h.read_params(i) for i in range(w.N)])
        h.close()
        assert np.array_equal(got, full)


@pytest.mark.parametrize("cfg,P", [(4, 5120), (2, 4096)])
def test_bench_rank_launcher_runs_under_torch_distributed_run(cfg, P):
    """bench.py --gpus 2 as the driver launches it (one process per rank), process group on gloo, both ranks on cuda:0."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo",
           "--config", str(cfg), "--P", str(P), "--steps", "12", "--warmup", "3", "--no-cpu-baseline"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["value"] > 0 and d["steps"] == 12 and d["scaling"] == "strong"
    assert d["config"]["P"] == P and d["run"]["P_per_gpu"] == P // 2
    assert d["gpu_launches"] > 0 and d["roofline"]["launches"] == 12
