"""Multi-rank host logic of the column-sharded run (world size 2, gloo, CPU): shard boundaries, the
max-over-ranks timing reduction, and the fact that the path is separable by column, so that ranks
working on their own column ranges with the replicated trace reproduce the unsharded result."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from oracle import protocol as op, update as up
from paper_1902_01064_b200 import inputs


def test_shard_columns_partition():
    for P in (1, 4, 127, 128, 129, 1000, 25_600_000, 8_000_000, 1_200_000):
        for n in (1, 2, 3, 4, 8):
            spans = [bench.shard_columns(P, n, r) for r in range(n)]
            assert spans[0][0] == 0 and spans[-1][1] == P
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c and a <= b
            assert all(a % 128 == 0 for a, _ in spans)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, P, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.make_workload(3, P=P, iters=12)
    lo, hi = bench.shard_columns(P, world, rank)
    tr = op.simulate(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode,
                           stale_reduce=w.stale_reduce).to_arrays()   # replicated
    cols = np.arange(lo, hi)
    x0 = np.tile(w.p0()[cols].astype(np.float64), (w.N, 1))
    X, newest = up.run_updates(tr, w.N, w.lr, w.momentum, x0, up.GradSynthetic(w.grad_seed, w.sigma, cols), s=w.s)
    mine = np.stack([X[(i, newest[i])] for i in range(w.N)])
    # the timing reduction bench.py uses: max over ranks
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, mine))
    dist.barrier()
    if rank == 0:
        full = np.concatenate([p[2] for p in sorted(parts, key=lambda p: p[0])], axis=1)
        np.save(out, full)
        assert float(t.item()) == 10.0 + world - 1
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_run(tmp_path):
    P = 1000
    out = str(tmp_path / "sharded.npy")
    mp.spawn(_rank_main, args=(2, _free_port(), P, out), nprocs=2, join=True)
    got = np.load(out)
    w = inputs.make_workload(3, P=P, iters=12)
    tr = op.simulate(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode,
                           stale_reduce=w.stale_reduce).to_arrays()
    x0 = np.tile(w.p0().astype(np.float64), (w.N, 1))
    X, newest = up.run_updates(tr, w.N, w.lr, w.momentum, x0, up.GradSynthetic(w.grad_seed, w.sigma, np.arange(P)), s=w.s)
    want = np.stack([X[(i, newest[i])] for i in range(w.N)])
    assert np.array_equal(got, want)


def _dense_rows(svm, P):
    """Every worker's rows as one dense [N*R][P] float64 matrix, whichever layout the data has."""
    if svm.dense is not None:
        return svm.dense.reshape(-1, P).astype(np.float64)
    A = np.zeros((len(svm.row_ptr) - 1, P))
    for r in range(len(svm.row_ptr) - 1):
        a, b = svm.row_ptr[r], svm.row_ptr[r + 1]
        np.add.at(A[r], svm.col[a:b], svm.val[a:b])
    return A


@pytest.mark.parametrize("cfg,P", [(1, 1000), (2, 2048)])
def test_feature_column_shards_partition_the_data(cfg, P):
    w = inputs.make_workload(cfg, P=P, iters=4)
    full = _dense_rows(w.svm, P)
    edges = (0, 128, 896, P)
    parts = [_dense_rows(w.svm.column_shard(lo, hi), hi - lo) for lo, hi in zip(edges, edges[1:])]
    assert np.array_equal(np.concatenate(parts, axis=1), full)


def _margin_rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    P = 2048
    w = inputs.make_workload(2, P=P, iters=4)
    lo, hi = bench.shard_columns(P, world, rank)
    x = w.p0().astype(np.float64)[lo:hi]
    part = torch.from_numpy(_dense_rows(w.svm.column_shard(lo, hi), hi - lo) @ x)     # this rank's partial margins
    dist.all_reduce(part)                                                             # the one exchange step of an SVM level
    if rank == 0:
        np.save(out, part.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_partial_margins_summed_over_two_ranks_equal_the_full_margins(tmp_path):
    out = str(tmp_path / "margins.npy")
    mp.spawn(_margin_rank, args=(2, _free_port(), out), nprocs=2, join=True)
    w = inputs.make_workload(2, P=2048, iters=4)
    want = _dense_rows(w.svm, 2048) @ w.p0().astype(np.float64)
    assert np.allclose(np.load(out), want, rtol=1e-12, atol=1e-12)
