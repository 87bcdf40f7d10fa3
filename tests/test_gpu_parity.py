"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

The configurations run under both readings of the bounded-staleness Reduce set (only updates that arrived since the worker's previous Recv, the
default, as Eq. 2 and Fig. alg3 print it; or every update still inside the bound): `reduce` below.

Tolerances (float32 path against a float64 oracle): max|delta| <= 1e-6 * max|x| after one level,
<= 1e-4 * max|x| after a full run; traces are compared bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import philox, protocol as op, update as up
from paper_1902_01064_b200 import hop, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL_STEP, TOL_RUN = 1e-6, 1e-4
KEYS = ("op", "ptr", "nbr", "ver", "num", "den")


class GpuRun:
    """Device buffers (torch, plumbing only) + a configured context for a workload."""

    def __init__(self, w, mix_kernel=hop.MIX_AUTO, x0=None, external_G=None, variant=None):
        self.w = w
        self.variant = variant or {}
        S = w.s + 1
        self.X = torch.zeros((w.N, S, w.P), dtype=torch.float32, device=DEV)
        self.M = torch.zeros((w.N, w.P), dtype=torch.float32, device=DEV) if w.momentum else None
        self.G = None if w.grad_mode == inputs.GRAD_SVM_CSR else torch.zeros((w.N, w.P), dtype=torch.float32, device=DEV)
        self.h = hop.from_workload(w, mix_kernel)
        if external_G is not None:
            self.h.set_option(hop.OPT_GRAD_MODE, hop.GRAD_EXTERNAL)
        self.h.set_option(hop.OPT_LOSS, hop.LOSS_LOG if self.variant.get("loss") == "log" else hop.LOSS_HINGE)
        self.h.set_option(hop.OPT_WEIGHT_DECAY, self.variant.get("weight_decay", 0.0))
        self.h.set_option(hop.OPT_APPROACH, hop.APPROACH_SERIAL if self.variant.get("serial") else hop.APPROACH_PARALLEL)
        self.external_G = external_G
        self.h.bind_buffers(self.X, self.M, self.G, torch.cuda.current_stream().cuda_stream)
        if w.grad_mode == inputs.GRAD_SVM_DENSE:
            self.A = torch.from_numpy(w.svm.dense).to(DEV)
            self.y = torch.from_numpy(w.svm.y).to(DEV)
            self.h.bind_svm_dense(self.A, self.y, w.svm.rows_per_worker, w.svm.batch)
        elif w.grad_mode == inputs.GRAD_SVM_CSR:
            self.rp = torch.from_numpy(w.svm.row_ptr).to(DEV)
            self.col = torch.from_numpy(w.svm.col).to(DEV)
            self.val = torch.from_numpy(w.svm.val).to(DEV)
            self.y = torch.from_numpy(w.svm.y).to(DEV)
            self.h.bind_svm_csr(self.rp, self.col, self.val, self.y, w.svm.rows_per_worker, w.svm.batch)
        self.trace = self.h.sim_run(w.ticks, w.iters)
        self.h.load_trace(self.trace)
        self.x0 = np.tile(w.p0(), (w.N, 1)) if x0 is None else x0
        for i in range(w.N):
            self.h.write_params(i, 0, self.x0[i])

    def run(self, levels):
        for k in range(levels):
            if self.external_G is not None:
                self.G.copy_(torch.from_numpy(self.external_G[k]))
            self.h.step()
        assert self.h.read_status() == 0
        return [self.h.read_params(i) for i in range(self.w.N)]


def oracle_grad_fn(w, cols=None, external_G=None, loss="hinge"):
    if external_G is not None:
        return up.GradExternal(external_G if cols is None else external_G[:, :, cols])
    if w.grad_mode == inputs.GRAD_SYNTHETIC:
        return up.GradSynthetic(w.grad_seed, w.sigma, np.arange(w.P) if cols is None else cols)
    if w.grad_mode == inputs.GRAD_SVM_DENSE:
        return up.GradSvmDense(w.svm.dense, w.svm.y, w.svm.batch, loss)
    return up.GradSvmCsr(w.svm.row_ptr, w.svm.col, w.svm.val, w.svm.y, w.svm.rows_per_worker, w.svm.batch, loss)


def oracle_run(w, x0, levels, cols=None, external_G=None, variant=None):
    variant = variant or {}
    tr = op.simulate(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode,
                     stale_reduce=w.stale_reduce, serial=bool(variant.get("trace_serial", variant.get("serial")))).to_arrays()
    xs = x0.astype(np.float64) if cols is None else x0[:, cols].astype(np.float64)
    X, newest = up.run_updates(tr, w.N, w.lr, w.momentum, xs, oracle_grad_fn(w, cols, external_G, variant.get("loss", "hinge")),
                               levels=levels, s=w.s, weight_decay=variant.get("weight_decay", 0.0),
                               serial=bool(variant.get("serial")))
    return tr, [X[(i, newest[i])] for i in range(w.N)], newest


def check(w, levels, tol, mix_kernel=hop.MIX_AUTO, perturb=False, cols=None, external_G=None, variant=None):
    x0 = np.tile(w.p0(), (w.N, 1))
    if perturb:
        x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    g = GpuRun(w, mix_kernel, x0, external_G, variant)
    got = g.run(levels)
    tr, want, newest = oracle_run(w, x0, levels, cols, external_G, variant)
    gt = g.trace.to_arrays()
    for k in KEYS:
        assert np.array_equal(gt[k], tr[k]), k                                  # traces bit-exact
    scale = max(1e-30, max(np.abs(x).max() for x in want))
    worst = 0.0
    for i in range(w.N):
        assert g.h.newest_version(i) == newest[i]
        a = got[i].astype(np.float64) if cols is None else got[i][cols].astype(np.float64)
        worst = max(worst, np.abs(a - want[i]).max())
    assert worst <= tol * scale, f"max|delta| / max|x| = {worst / scale:.3e} > {tol:g}"
    g.h.close()
    return worst / scale


KERNELS = [hop.MIX_STAGED, hop.MIX_BULK]
REDUCE = [op.NEW_ONLY, op.REUSE]


def workload(cfg, reduce=op.NEW_ONLY, **kw):
    return dataclasses.replace(inputs.make_workload(cfg, **kw), stale_reduce=reduce)


# ------------------------------------------------------------------ configuration 1: dense SVM, 4 workers
@pytest.mark.parametrize("kernel", KERNELS)
def test_cfg1_full_run_and_one_step(kernel):
    w = inputs.make_workload(1)
    check(w, w.iters, TOL_RUN, kernel)
    check(w, 1, TOL_STEP, kernel, perturb=True)
    check(w, 5, TOL_RUN, kernel, perturb=True)


# ------------------------------------------------------------------ configuration 2: CSR SVM, 16 workers
@pytest.mark.parametrize("reduce", REDUCE)
@pytest.mark.parametrize("kernel", KERNELS)
def test_cfg2_reduced_full_run(kernel, reduce):
    w = workload(2, reduce, P=8192)
    check(w, w.iters, TOL_RUN, kernel)
    check(w, 1, TOL_STEP, kernel, perturb=True)


def test_cfg2_full_size_whole_run():
    # P = 2^20, all 200 levels: the acceptance bound of the full run at the size bench.py times
    w = inputs.make_workload(2)
    one = check(w, 1, TOL_STEP, perturb=True)
    full = check(w, w.iters, TOL_RUN)
    print(f"config 2 at full size: max|delta|/max|x| = {one:.2e} after one level, {full:.2e} after {w.iters} levels")


# ------------------------------------------------------------------ configuration 3: momentum + skipping
@pytest.mark.parametrize("reduce", REDUCE)
@pytest.mark.parametrize("kernel,P", [(hop.MIX_STAGED, 5000), (hop.MIX_BULK, 5000), (hop.MIX_STAGED, 4999), (hop.MIX_BULK, 4999),
                                      (hop.MIX_BULK, 132), (hop.MIX_STAGED, 3), (hop.MIX_BULK, 3), (hop.MIX_BULK, 4097),
                                      (hop.MIX_BULK, 130), (hop.MIX_BULK, 1023)])
def test_cfg3_reduced_full_run(kernel, P, reduce):
    w = workload(3, reduce, P=P)
    check(w, w.iters, TOL_RUN, kernel)
    check(w, 1, TOL_STEP, kernel, perturb=True)


def test_cfg3_full_size_sampled_columns():
    w = inputs.make_workload(3)
    g = GpuRun(w)
    tile = g.h.level_stats(0)["tile_w"]
    cols = np.unique(np.concatenate([np.arange(0, w.P, 997), np.arange(tile - 2, w.P, 50 * tile),
                                     np.arange(tile, w.P, 50 * tile), [w.P - 1, w.P - 2, w.P - 5]]))
    g.h.close()
    check(w, w.iters, TOL_RUN, cols=cols)


# ------------------------------------------------------------------ configuration 4: 64 workers, s=4, b=2
@pytest.mark.parametrize("reduce", REDUCE)
@pytest.mark.parametrize("kernel", KERNELS)
def test_cfg4_reduced_full_run(kernel, reduce):
    w = workload(4, reduce, P=3000)
    check(w, w.iters, TOL_RUN, kernel)
    check(w, 1, TOL_STEP, kernel, perturb=True)


def test_cfg4_full_size_sampled_columns():
    w = inputs.make_workload(4)
    free, _ = torch.cuda.mem_get_info()
    if free < 50 * 2 ** 30:
        pytest.skip("needs ~42 GB of device memory")
    cols = np.unique(np.concatenate([np.arange(0, w.P, 25013), np.arange(127, w.P, 128 * 4001),
                                     np.arange(128, w.P, 128 * 4001), [w.P - 1, w.P - 4]]))
    check(w, w.iters, TOL_RUN, cols=cols)


# ------------------------------------------------------------------ configuration 5: complete graph, 128 workers
@pytest.mark.parametrize("reduce", REDUCE)
@pytest.mark.parametrize("kernel", KERNELS + [hop.MIX_TENSOR])
def test_cfg5_reduced_full_run(kernel, reduce):
    w = workload(5, reduce, P=1536)
    g = GpuRun(w, kernel)
    assert g.h.level_stats(3)["kernel"] == kernel                      # the requested kernel is the one that runs
    g.h.close()
    check(w, w.iters, TOL_RUN, kernel)
    check(w, 1, TOL_STEP, kernel, perturb=True)


def test_cfg5_tensor_path_many_tiles_and_consensus_start():
    # more tiles than thread blocks (pipeline wrap-around, accumulator hand-over), and the workload's own
    # start where all replicas are equal (largest accumulators, every product of equal sign)
    w = inputs.make_workload(5, P=128 * 700, iters=6)
    check(w, 1, TOL_STEP, hop.MIX_TENSOR)
    check(w, w.iters, TOL_RUN, hop.MIX_TENSOR)
    check(w, 1, TOL_STEP, hop.MIX_TENSOR, perturb=True)


def test_tensor_path_with_idle_and_jumping_workers_and_fewer_than_128_workers():
    # not every worker is active in every level (skipping) and N < 128: rows leave one by one instead of as a box
    N, P, iters, s = 96, 128 * 9, 16, 3
    ptr, idx = inputs.graph_to_csr(inputs.complete(N))
    ticks = np.ones((N, iters), np.uint64)
    ticks[5, :] = 9
    w = inputs.Workload(0, "dense-skip", N, P, iters, s=s, b=6, max_skip=3, max_ig=4, lr=0.05, momentum=0.0,
                        weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                        ticks=ticks, grad_seed=4242)
    w._p0 = np.random.default_rng(3).standard_normal(P).astype(np.float32)
    g = GpuRun(w, hop.MIX_TENSOR)
    tr = g.trace.to_arrays()
    assert (tr["op"] == op.JUMP).sum() > 0 and (tr["op"] == op.IDLE).sum() > 0
    assert all(g.h.level_stats(k)["kernel"] == hop.MIX_TENSOR for k in range(iters))
    g.h.close()
    check(w, iters, TOL_RUN, hop.MIX_TENSOR, perturb=True)
    check(w, 1, TOL_STEP, hop.MIX_TENSOR, perturb=True)


def test_cfg5_full_size_sampled_columns_whole_run():
    # P = 8M, all 30 levels, on a strided column sample plus both edge columns of the first and the last 128-column tile
    # that each of the 148 persistent blocks owns
    w = inputs.make_workload(5)
    tiles, blocks = w.P // 128, 148
    edge_tiles = np.unique(np.concatenate([[b, b + blocks * ((tiles - 1 - b) // blocks)] for b in range(blocks)]))
    cols = np.unique(np.concatenate([np.arange(0, w.P, 40009), edge_tiles * 128, edge_tiles * 128 + 127,
                                     [w.P - 1, w.P - 3, 127, 128, 255, 256]]))
    g = GpuRun(w)
    assert all(g.h.level_stats(k)["kernel"] == hop.MIX_TENSOR for k in range(w.iters))   # what bench.py times for config 5
    g.h.close()
    full = check(w, w.iters, TOL_RUN, cols=cols)
    one = check(w, 1, TOL_STEP, cols=cols, perturb=True)
    print(f"config 5 at full size ({cols.size} columns): max|delta|/max|x| = {one:.2e} after one level, {full:.2e} after {w.iters} levels")


# ------------------------------------------------------------------ kernels in isolation / edge cases
def test_synthetic_gradient_kernel_matches_philox_box_muller():
    w = inputs.make_workload(3, P=10007)
    g = GpuRun(w, hop.MIX_STAGED)
    g.h.step()
    torch.cuda.synchronize()
    G = g.G.cpu().numpy()
    tr = g.trace.to_arrays()
    for i in range(w.N):
        if tr["op"][0, i] == op.NORMAL:
            want = philox.synthetic_gradient(w.grad_seed, i, 0, np.arange(w.P), w.sigma)
            assert np.abs(G[i] - want).max() <= 2e-6 * w.sigma * 6
    g.h.close()


def test_external_gradients_and_tiny_shapes():
    rng = np.random.default_rng(0)
    for (N, P, s) in [(1, 1, 0), (2, 4, 0), (3, 7, 1), (5, 33, 2), (6, 260, 0)]:
        n_in = inputs.complete(N) if N < 4 else inputs.ring(N)
        ptr, idx = inputs.graph_to_csr(n_in)
        iters = 6
        w = inputs.Workload(0, "tiny", N, P, iters, s=s, b=0, max_skip=0, max_ig=max(1, s), lr=0.25, momentum=0.5,
                            weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_EXTERNAL, in_ptr=ptr, in_idx=idx,
                            ticks=rng.integers(1, 9, size=(N, iters)).astype(np.uint64))
        w._p0 = rng.standard_normal(P).astype(np.float32)
        G = rng.standard_normal((iters, N, P)).astype(np.float32)
        for kernel in (hop.MIX_STAGED, hop.MIX_BULK):          # the bulk-copy kernel takes any P (unaligned rows included)
            check(w, iters, TOL_RUN, kernel, perturb=True, external_G=G)


def test_in_place_ring_hazard_single_slot_and_stale_reads():
    # s = 0: one slot per worker, every level overwrites what the neighbours read in that level.
    rng = np.random.default_rng(1)
    for s, P in [(0, 1000), (1, 1000), (3, 1000), (0, 20000)]:
        n_in = inputs.ring_chords(12, 5)
        ptr, idx = inputs.graph_to_csr(n_in)
        iters = 12
        ticks = rng.choice([1, 1, 7], size=(12, iters)).astype(np.uint64)     # stragglers -> oldest versions consumed
        w = inputs.Workload(0, "hazard", 12, P, iters, s=s, b=0, max_skip=0, max_ig=max(1, s), lr=0.1, momentum=0.0,
                            weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                            ticks=ticks, grad_seed=77)
        w._p0 = rng.standard_normal(P).astype(np.float32)
        for reduce in (REDUCE if s > 0 else REDUCE[:1]):
            w.stale_reduce = reduce
            tr = op.simulate(w.n_in, ticks, iters, s, 0, w.max_ig, 0, w.weight_mode, stale_reduce=reduce)
            if s > 0:
                oldest = sum(1 for (k, i), rec in tr.rec.items() for (j, v, _) in rec if j != i and v == k - s)
                assert oldest > 0, "no slot is read in the level that overwrites it: test is vacuous"
            for kernel in KERNELS:
                check(w, iters, TOL_RUN, kernel, perturb=True)


@pytest.mark.parametrize("cfg,P,iters", [(3, 2048, 40), (5, 1536, 8)])
def test_streaming_levels_equal_preloaded_trace_bitwise(cfg, P, iters):
    # configuration 5 goes through the tensor-core kernel in both modes
    w = inputs.make_workload(cfg, P=P, iters=iters)
    a = GpuRun(w)
    ref = a.run(w.iters)
    b = GpuRun(w)
    tr = b.trace.to_arrays()
    b.h.set_level(0)
    probe = np.zeros(16, np.float32)
    N = w.N
    for k in range(w.iters):
        lo, hi = tr["ptr"][k * N], tr["ptr"][(k + 1) * N]
        ptr = (tr["ptr"][k * N:(k + 1) * N + 1] - lo).astype(np.int64)
        b.h.step_host(np.ascontiguousarray(tr["op"][k]), ptr, np.ascontiguousarray(tr["nbr"][lo:hi]),
                      np.ascontiguousarray(tr["ver"][lo:hi]), np.ascontiguousarray(tr["num"][lo:hi]),
                      np.ascontiguousarray(tr["den"][k]), probe)
    for i in range(N):
        assert np.array_equal(ref[i], b.h.read_params(i))
    assert np.array_equal(probe, ref[0][:16])
    a.h.close()
    b.h.close()


def test_checkpoint_resume_is_bitwise():
    w = inputs.make_workload(3, P=1024, iters=30)
    a = GpuRun(w)
    a.h.set_option(hop.OPT_NVTX, 1)                 # host-side trace ranges change nothing on the device
    ref = a.run(w.iters)
    b = GpuRun(w)
    b.run(17)
    torch.cuda.synchronize()
    ringX, ringM = b.X.clone(), b.M.clone()
    c = GpuRun(w)
    c.X.copy_(ringX)
    c.M.copy_(ringM)
    c.h.set_level(17)
    for k in range(17, w.iters):
        c.h.step()
    for i in range(w.N):
        assert np.array_equal(ref[i], c.h.read_params(i))
    for x in (a, b, c):
        x.h.close()


def test_malformed_traces_are_rejected_on_the_host():
    w = inputs.make_workload(4, P=64, iters=8)
    g = GpuRun(w)
    good = g.trace.to_arrays()

    def load(mut):
        t = {k: good[k].copy() for k in KEYS}
        mut(t)
        with pytest.raises(hop.HopError) as e:
            g.h.load_trace(hop.Trace.from_arrays(*[t[k] for k in KEYS]))
        assert e.value.code == hop.E_TRACE
    load(lambda t: t["ver"].__setitem__(5, t["ver"][5] - 9))                  # older than the staleness window
    load(lambda t: t["nbr"].__setitem__(1, (t["nbr"][1] + 1) % 64))           # likely not an in-neighbour / duplicate
    load(lambda t: t["den"].__setitem__((3, 3), t["den"][3, 3] + 1))          # weights do not sum up
    load(lambda t: t["op"].__setitem__((2, 0), 7))                            # unknown op
    g.h.load_trace(g.trace)
    g.h.close()
    # a trace that reduces an update again is valid only under HOP_STALE_REUSE
    g = GpuRun(dataclasses.replace(w, stale_reduce=op.REUSE))
    reused = g.trace
    assert reused.dims()[2] > good["nbr"].size
    g.h.set_option(hop.OPT_STALE_REDUCE, hop.STALE_NEW_ONLY)
    with pytest.raises(hop.HopError) as e:
        g.h.load_trace(reused)
    assert e.value.code == hop.E_TRACE and "consumed before" in str(e.value)
    g.h.close()


def test_column_shards_equal_the_full_run_bitwise():
    # what `bench.py --gpus N` does per rank: a contiguous column range with HOP_OPT_COL_OFFSET
    import bench
    P = 5120
    w = inputs.make_workload(4, P=P, iters=20)
    full = GpuRun(w).run(w.iters)
    for world in (2, 3):
        for r in range(world):
            lo, hi = bench.shard_columns(P, world, r)
            ws = inputs.make_workload(4, P=P, iters=20)
            p0 = ws.p0()[lo:hi].copy()
            ws.P, ws._p0 = hi - lo, p0
            g = GpuRun(ws)
            g.h.set_option(hop.OPT_COL_OFFSET, lo)
            got = g.run(ws.iters)
            for i in range(w.N):
                assert np.array_equal(got[i], full[i][lo:hi])
            g.h.close()


@pytest.mark.parametrize("cfg,P,iters", [(1, None, 20), (3, 2048, 40), (5, 1536, 8), (2, 4096, 24)])
def test_graph_replay_of_level_ranges_equals_step_by_step(cfg, P, iters):
    # hop_run on a side stream captures the levels into a CUDA graph and replays it; same kernels, same arguments
    w = inputs.make_workload(cfg, P=P, iters=iters)
    ref = GpuRun(w).run(w.iters)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = GpuRun(w)                       # binds the side stream
        g.h.run(7)
        g.h.run(w.iters - 7)
        side.synchronize()
        # replay from the cache after a rewind: identical again
        first = [g.h.read_params(i) for i in range(w.N)]
        for i in range(w.N):
            g.h.write_params(i, 0, g.x0[i])
        if g.M is not None:
            g.M.zero_()
        g.h.set_level(0)
        g.h.run(7)
        g.h.run(w.iters - 7)
        second = [g.h.read_params(i) for i in range(w.N)]
        assert g.h.read_status() == 0
    exact = w.grad_mode != inputs.GRAD_SVM_CSR          # the sparse apply uses float atomics: order may differ
    for i in range(w.N):
        if exact:
            assert np.array_equal(first[i], ref[i]) and np.array_equal(second[i], ref[i])
        else:
            scale = np.abs(ref[i]).max() + 1e-30
            assert np.abs(first[i] - ref[i]).max() <= 1e-5 * scale and np.abs(second[i] - ref[i]).max() <= 1e-5 * scale
    g.h.close()


# ------------------------------------------------------------------ loss / regulariser / operation order variants
VARIANTS = [dict(loss="log"), dict(weight_decay=0.05), dict(loss="log", weight_decay=0.02, serial=True), dict(serial=True)]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("kernel", KERNELS)
def test_dense_svm_with_log_loss_weight_decay_momentum_and_serial_order(kernel, variant):
    # the paper's SVM runs: log loss, momentum 0.9, weight decay (Section 7.2)
    w = inputs.make_workload(1)
    w.momentum = 0.9
    check(w, w.iters, TOL_RUN, kernel, variant=variant)
    check(w, 1, TOL_STEP, kernel, perturb=True, variant=variant)


@pytest.mark.parametrize("variant", [dict(loss="log"), dict(weight_decay=0.05), dict(loss="log", serial=True)])
def test_csr_svm_variants(variant):
    w = inputs.make_workload(2, P=8192, iters=60)
    check(w, w.iters, TOL_RUN, variant=variant)
    check(w, 1, TOL_STEP, perturb=True, variant=variant)


@pytest.mark.parametrize("variant", [dict(serial=True), dict(weight_decay=0.01), dict(serial=True, weight_decay=0.01)])
def test_synthetic_gradient_variants_with_momentum_and_jumps(variant):
    w = inputs.make_workload(3, P=5000, iters=60)
    for kernel in KERNELS:
        check(w, w.iters, TOL_RUN, kernel, variant=variant)
        check(w, 1, TOL_STEP, kernel, perturb=True, variant=variant)


def test_tensor_path_in_serial_order():
    w = inputs.make_workload(5, P=1536, iters=10)
    g = GpuRun(w, hop.MIX_TENSOR, variant=dict(serial=True))
    assert g.h.level_stats(2)["kernel"] == hop.MIX_TENSOR
    g.h.close()
    check(w, w.iters, TOL_RUN, hop.MIX_TENSOR, variant=dict(serial=True))
    check(w, 1, TOL_STEP, hop.MIX_TENSOR, perturb=True, variant=dict(serial=True))


def test_unsupported_combinations_are_refused():
    w = inputs.make_workload(2, P=4096, iters=4)
    g = GpuRun(w, variant=dict(serial=True, weight_decay=0.1))
    with pytest.raises(hop.HopError) as e:
        g.h.step()
    assert e.value.code == hop.E_UNSUPPORTED
    g.h.close()


def test_tensor_path_with_more_than_eight_ring_slots_and_few_workers():
    # s + 1 = 10 slots: no output tensor map per slot is kept, rows leave by bulk copies; N = 24 < 32 workers
    N, P, iters, s = 24, 128 * 5, 14, 9
    ptr, idx = inputs.graph_to_csr(inputs.complete(N))
    rng = np.random.default_rng(9)
    w = inputs.Workload(0, "dense-deep-ring", N, P, iters, s=s, b=3, max_skip=0, max_ig=9, lr=0.05, momentum=0.0,
                        weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                        ticks=rng.choice([1, 2, 9], size=(N, iters)).astype(np.uint64), grad_seed=99)
    w._p0 = rng.standard_normal(P).astype(np.float32)
    g = GpuRun(w, hop.MIX_TENSOR)
    assert all(g.h.level_stats(k)["kernel"] == hop.MIX_TENSOR for k in range(iters))
    assert max(g.h.level_stats(k)["U"] for k in range(iters)) > N          # stale versions really are consumed
    g.h.close()
    check(w, iters, TOL_RUN, hop.MIX_TENSOR, perturb=True)


def test_tensor_path_with_a_ragged_last_quarter_of_workers():
    # N = 40: the second quarter of the gradient / result tile holds 8 real workers; the copy engine zero-fills the
    # rows past N on the way in and drops them on the way out
    N, P, iters, s = 40, 128 * 7, 10, 1
    ptr, idx = inputs.graph_to_csr(inputs.complete(N))
    rng = np.random.default_rng(11)
    w = inputs.Workload(0, "dense-40", N, P, iters, s=s, b=4, max_skip=0, max_ig=1, lr=0.05, momentum=0.0,
                        weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                        ticks=rng.choice([1, 2, 5], size=(N, iters)).astype(np.uint64), grad_seed=77)
    w._p0 = rng.standard_normal(P).astype(np.float32)
    g = GpuRun(w, hop.MIX_TENSOR)
    assert all(g.h.level_stats(k)["kernel"] == hop.MIX_TENSOR for k in range(iters))
    g.h.close()
    check(w, iters, TOL_RUN, hop.MIX_TENSOR, perturb=True)
    check(w, 1, TOL_STEP, hop.MIX_TENSOR, perturb=True)


@pytest.mark.parametrize("N,s,b", [(40, 8, 4), (72, 4, 6)])
def test_tensor_path_with_two_result_buffers(N, s, b):
    # enough distinct consumed slices (K >= 224) that the weight matrix leaves room for only two of the four
    # gradient / result buffers: each buffer then serves two quarters of the tile in turn.  N = 40: two quarters in one
    # buffer, 9 ring slots so the rows leave by bulk copies; N = 72: three quarters, box stores.
    P, iters = 128 * 6, 16
    ptr, idx = inputs.graph_to_csr(inputs.complete(N))
    rng = np.random.default_rng(31)
    w = inputs.Workload(0, "dense-stale", N, P, iters, s=s, b=b, max_skip=0, max_ig=s, lr=0.05, momentum=0.0,
                        weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                        ticks=rng.choice([1, 2, 9], size=(N, iters)).astype(np.uint64), grad_seed=5,
                        stale_reduce=op.REUSE)        # every update inside the bound is reduced: the widest contractions
    w._p0 = rng.standard_normal(P).astype(np.float32)
    g = GpuRun(w, hop.MIX_TENSOR)
    st = [g.h.level_stats(k) for k in range(iters)]
    assert all(x["kernel"] == hop.MIX_TENSOR for x in st)
    assert max(x["k_padded"] for x in st) >= 224
    g.h.close()
    check(w, iters, TOL_RUN, hop.MIX_TENSOR, perturb=True)


def test_streaming_rejects_bad_records_and_run_checks_its_range():
    w = inputs.make_workload(4, P=256, iters=6)
    g = GpuRun(w)
    tr = g.trace.to_arrays()
    N = w.N
    a, b = tr["ptr"][0], tr["ptr"][N]
    good = [np.ascontiguousarray(tr["op"][0]), (tr["ptr"][:N + 1] - a).astype(np.int64), np.ascontiguousarray(tr["nbr"][a:b]),
            np.ascontiguousarray(tr["ver"][a:b]), np.ascontiguousarray(tr["num"][a:b]), np.ascontiguousarray(tr["den"][0])]
    bad = [x.copy() for x in good]
    bad[3][2] = 5                                      # a version from the future
    g.h.set_level(0)
    with pytest.raises(hop.HopError) as e:
        g.h.step_host(*bad)
    assert e.value.code == hop.E_TRACE
    g.h.step_host(*good)                               # the rejected call left the context usable
    g.h.set_level(0)
    g.h.run(0)
    with pytest.raises(hop.HopError) as e:
        g.h.run(w.iters + 1)
    assert e.value.code == hop.E_STATE
    g.h.run(w.iters)
    with pytest.raises(hop.HopError):
        g.h.step()
    assert g.h.read_status() == 0
    g.h.close()


# ------------------------------------------------------------------ column-sharded SVM: split-phase stepping
@pytest.mark.parametrize("cfg,P,iters,edges", [(1, 1000, 40, (0, 384, 1000)), (2, 4096, 24, (0, 1024, 2560, 4096))])
def test_column_sharded_svm_with_summed_margins_equals_the_oracle(cfg, P, iters, edges):
    """Each shard owns a column range (its own context, ring and feature slice); the partial margins are summed
    between hop_step_begin and hop_step_end, as an all-reduce would between ranks.  Shards run one after the other
    on one stream, so nothing waits on anything."""
    import dataclasses
    w = inputs.make_workload(cfg, P=P, iters=iters)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    shards = []
    for lo, hi in zip(edges, edges[1:]):
        ws = dataclasses.replace(w, P=hi - lo, svm=w.svm.column_shard(lo, hi), _p0=None)
        shards.append(GpuRun(ws, x0=np.ascontiguousarray(x0[:, lo:hi])))
    for k in range(iters):
        views = []
        for g in shards:
            ptr, n = g.h.step_begin()
            assert n == w.N * w.svm.batch and ptr
            views.append((ptr, n))
        # plumbing: wrap the context-owned buffers and sum them in place (what dist.all_reduce does across ranks)
        bufs = [_as_f64_tensor(ptr, n) for ptr, n in views]
        total = torch.stack(bufs).sum(0)
        for b in bufs:
            b.copy_(total)
        for g in shards:
            g.h.step_end()
    tr, want, newest = oracle_run(w, x0, iters)
    scale = max(np.abs(x).max() for x in want)
    worst = 0.0
    for g, lo, hi in zip(shards, edges, edges[1:]):
        assert g.h.read_status() == 0
        for i in range(w.N):
            assert g.h.newest_version(i) == newest[i]
            worst = max(worst, np.abs(g.h.read_params(i).astype(np.float64) - want[i][lo:hi]).max())
        g.h.close()
    assert worst <= TOL_RUN * scale, (worst, scale)


def _as_f64_tensor(ptr, n):
    return torch.as_tensor(hop.DeviceSpan(ptr, n), device=DEV)


def test_split_phase_calls_must_alternate():
    w = inputs.make_workload(1, P=256, iters=8)
    g = GpuRun(w)
    with pytest.raises(hop.HopError):
        g.h.step_end()
    g.h.step_begin()
    for call in (g.h.step_begin, g.h.step, lambda: g.h.run(1)):
        with pytest.raises(hop.HopError):
            call()
    g.h.step_end()
    g.h.step()
    assert g.h.read_status() == 0
    g.h.close()


# ------------------------------------------------------------------ options and data changed after the trace was loaded
def _oracle_state(w, x0, levels, variant=None):
    tr, want, newest = oracle_run(w, x0, levels, variant=variant)
    return want, max(np.abs(x).max() for x in want)


def test_options_set_after_load_trace_plan_the_levels_again():
    # momentum switched on and off after the load: the staged rows and the tile width depend on it
    w = workload(3, P=2048, iters=30)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    for late_mu in (0.9, 0.0):
        g = GpuRun(w, x0=x0)                                   # planned with momentum 0.9, buffer bound
        g.h.set_option(hop.OPT_MOMENTUM, 0.9 - late_mu)       # planned again with the other setting ...
        g.h.set_option(hop.OPT_MOMENTUM, late_mu)             # ... and once more with the one that runs
        got = g.run(w.iters)
        want, scale = _oracle_state(dataclasses.replace(w, momentum=late_mu), x0, w.iters)
        assert max(np.abs(got[i] - want[i]).max() for i in range(w.N)) <= TOL_RUN * scale
        g.h.close()
    # tensor path: serial order and weight decay chosen after the load (the dense path bakes its gradient rows in)
    w = workload(5, P=1536, iters=8)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    g = GpuRun(w, hop.MIX_TENSOR, x0=x0)
    assert g.h.level_stats(2)["kernel"] == hop.MIX_TENSOR
    g.h.set_option(hop.OPT_APPROACH, hop.APPROACH_SERIAL)
    assert g.h.level_stats(2)["kernel"] == hop.MIX_TENSOR
    got = g.run(w.iters)
    # the trace was simulated before the switch (updates sent on entering an iteration); only the update rule changed
    want, scale = _oracle_state(w, x0, w.iters, variant=dict(serial=True, trace_serial=False))
    assert max(np.abs(got[i] - want[i]).max() for i in range(w.N)) <= TOL_RUN * scale
    g.h.close()
    g = GpuRun(w, hop.MIX_TENSOR, x0=x0)
    g.h.set_option(hop.OPT_WEIGHT_DECAY, 0.05)                 # the dense path then forms the update direction in a pre-pass
    assert g.h.level_stats(2)["kernel"] == hop.MIX_TENSOR
    got = g.run(w.iters)
    want, scale = _oracle_state(w, x0, w.iters, variant=dict(weight_decay=0.05))
    assert max(np.abs(got[i] - want[i]).max() for i in range(w.N)) <= TOL_RUN * scale
    # a value the loaded trace cannot be planned with is refused and leaves the context as it was
    g.h.close()
    # a parameter count that is not a multiple of 4: the general kernel first, the bulk-copy kernel chosen after the load
    w = workload(3, P=4999, iters=12)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    g = GpuRun(w, hop.MIX_STAGED, x0=x0)
    assert g.h.level_stats(1)["kernel"] == hop.MIX_STAGED
    g.h.set_option(hop.OPT_MIX_KERNEL, hop.MIX_BULK)
    assert g.h.level_stats(1)["kernel"] == hop.MIX_BULK
    got = g.run(w.iters)
    want, scale = _oracle_state(w, x0, w.iters)
    assert max(np.abs(got[i] - want[i]).max() for i in range(w.N)) <= TOL_RUN * scale
    with pytest.raises(hop.HopError):
        g.h.set_option(hop.OPT_MIX_KERNEL, 9)                  # refused; the context stays as it was
    assert g.h.level_stats(1)["kernel"] == hop.MIX_BULK
    g.h.close()


def test_option_change_in_the_middle_of_a_run_keeps_the_position():
    w = workload(3, op.REUSE, P=1024, iters=20)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    ref = GpuRun(w, x0=x0).run(w.iters)
    g = GpuRun(w, x0=x0)
    g.run(9)
    g.h.set_option(hop.OPT_STALE_REDUCE, hop.STALE_NEW_ONLY)  # a protocol option: acts on traces simulated or loaded later,
    g.h.set_option(hop.OPT_MIX_KERNEL, hop.MIX_STAGED)        # not on the loaded one, which is planned again at level 9
    assert g.h.level_stats(12)["kernel"] == hop.MIX_STAGED
    got = g.run(w.iters - 9)
    for i in range(w.N):
        assert g.h.newest_version(i) in (w.iters, w.iters - 1, w.iters - 2)
        assert np.abs(got[i] - ref[i]).max() <= 1e-6 * np.abs(ref[i]).max()
    g.h.close()


@pytest.mark.parametrize("cfg,P,iters", [(1, None, 20), (2, 4096, 16)])
def test_svm_rebind_between_graph_replays_uses_the_new_buffers(cfg, P, iters):
    # hop_run caches CUDA graphs whose kernels hold the SVM data and scratch pointers: binding other buffers must
    # drop them.  The old buffers are zeroed after the rebind, so a stale graph would show.
    w = workload(cfg, P=P, iters=iters)
    ref = GpuRun(w).run(w.iters)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = GpuRun(w)
        g.h.run(w.iters)
        side.synchronize()
        if cfg == 1:
            A2, y2 = g.A.clone(), g.y.clone()
            g.h.bind_svm_dense(A2, y2, w.svm.rows_per_worker, w.svm.batch)
            g.A.zero_(); g.y.zero_()
        else:
            new = [t.clone() for t in (g.rp, g.col, g.val, g.y)]
            g.h.bind_svm_csr(*new, w.svm.rows_per_worker, w.svm.batch)
            g.val.zero_(); g.y.zero_()
        for i in range(w.N):
            g.h.write_params(i, 0, g.x0[i])
        g.h.set_level(0)
        g.h.run(w.iters)
        got = [g.h.read_params(i) for i in range(w.N)]
        assert g.h.read_status() == 0
    for i in range(w.N):
        scale = np.abs(ref[i]).max() + 1e-30
        assert np.abs(got[i] - ref[i]).max() <= 1e-5 * scale
    g.h.close()


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    # a bounded wait that nothing satisfies returns by itself; the host sees HOP_E_DEVICE with the code and the detail
    w = workload(3, P=1024, iters=6)
    g = GpuRun(w)
    ref = GpuRun(w).run(w.iters)
    assert g.h.read_status_word() == (hop.OK, 0)
    g.h.selftest_bounded_wait(polls=200, detail=4242)
    rc, word = g.h.read_status_word()
    assert rc == hop.E_DEVICE and word >> 24 == 1 and word & 0xffffff == 4242
    with pytest.raises(hop.HopError) as e:
        g.h.read_status()
    assert e.value.code == hop.E_DEVICE and "copies did not arrive" in str(e.value) and "4242" in str(e.value)
    g.h.selftest_bounded_wait(polls=50, detail=7)              # the first event is the one that is kept
    assert g.h.read_status_word()[1] & 0xffffff == 4242
    g.h.clear_status()
    assert g.h.read_status_word() == (hop.OK, 0)
    got = g.run(w.iters)                                       # the context and the device are still good
    for i in range(w.N):
        assert np.array_equal(got[i], ref[i])
    g.h.close()


def test_level_with_only_jump_records_between_normal_levels():
    # A level whose active workers all jump has no gradient kernel in front of its mix-update launch, so that launch
    # must not start early; the levels around it do.  Hand-made trace (two workers, s = 1, every update inside the
    # bound reduced), run step by step and as one replayed graph, against the oracle's update rules on the same trace.
    P, N, s = 4096, 2, 1
    ptr, idx = inputs.graph_to_csr(inputs.complete(2))
    w = inputs.Workload(0, "jump-only-level", N, P, 4, s=s, b=0, max_skip=1, max_ig=1, lr=0.1, momentum=0.9,
                        weight_mode=inputs.STALE_LINEAR, grad_mode=inputs.GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx,
                        ticks=np.ones((N, 4), np.uint64), grad_seed=5, stale_reduce=op.REUSE)
    w._p0 = np.random.default_rng(2).standard_normal(P).astype(np.float32)
    NORMAL, JUMP = op.NORMAL, op.JUMP
    ops = np.array([[NORMAL, NORMAL], [JUMP, JUMP], [NORMAL, NORMAL], [NORMAL, NORMAL]], np.int32)
    recs = {(0, 0): [(0, 0), (1, 0)], (0, 1): [(0, 0), (1, 0)],
            (1, 0): [(0, 1), (1, 0)], (1, 1): [(0, 0), (1, 1)],           # own current parameters + the other's last sent update
            (2, 0): [(0, 2), (1, 2)], (2, 1): [(0, 2), (1, 2)],           # iteration 1 was skipped by both: nothing of it was sent
            (3, 0): [(0, 3), (1, 2)], (3, 1): [(0, 3), (1, 3)]}
    t_ptr, nbr, ver, num = [0], [], [], []
    den = np.zeros((4, N), np.int32)
    for k in range(4):
        for i in range(N):
            for (j, v) in recs[(k, i)]:
                nbr.append(j); ver.append(v); num.append(v - (k - s) + 1 if not (ops[k, i] == JUMP and j == i) else s + 1)
            den[k, i] = sum(num[t_ptr[-1]:])
            t_ptr.append(len(nbr))
    tr = dict(op=ops, ptr=np.asarray(t_ptr, np.int64), nbr=np.asarray(nbr, np.int32), ver=np.asarray(ver, np.int32),
              num=np.asarray(num, np.int32), den=den)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(N)])
    X, newest = up.run_updates(tr, N, w.lr, w.momentum, x0.astype(np.float64), up.GradSynthetic(w.grad_seed, w.sigma, np.arange(P)), s=s)
    want = [X[(i, newest[i])] for i in range(N)]
    scale = max(np.abs(x).max() for x in want)
    side = torch.cuda.Stream()
    for graph in (False, True):
        with torch.cuda.stream(side):
            g = GpuRun(w, x0=x0)
            g.h.load_trace(hop.Trace.from_arrays(*[tr[k] for k in KEYS]))
            assert [g.h.level_stats(k)["normal"] for k in range(4)] == [2, 0, 2, 2] and g.h.level_stats(1)["jump"] == 2
            if graph:
                g.h.run(4)
            else:
                for _ in range(4):
                    g.h.step()
            assert g.h.read_status() == 0
            for i in range(N):
                assert np.abs(g.h.read_params(i) - want[i]).max() <= TOL_RUN * scale
            g.h.close()


@pytest.mark.parametrize("P", [4999, 10001, 10002, 10003])
def test_bulk_kernel_with_unaligned_rows_equals_the_general_kernel_bitwise(P):
    # P % 4 = 3, 1, 2, 3: every row of the ring starts at a different distance from a 16-byte boundary; the last row of
    # each buffer ends 1-3 floats short of one (the plain-load tail).  Same multiply-adds in the same order as the
    # general kernel, so the results agree bit for bit; momentum, a jumping straggler and weight decay are on.
    w = workload(3, P=P, iters=30)
    x0 = np.stack([w.p0() + w.perturbation(i) for i in range(w.N)])
    for variant in (None, dict(weight_decay=0.01)):
        a = GpuRun(w, hop.MIX_STAGED, x0=x0, variant=variant)
        b = GpuRun(w, hop.MIX_BULK, x0=x0, variant=variant)
        assert a.h.level_stats(3)["kernel"] == hop.MIX_STAGED and b.h.level_stats(3)["kernel"] == hop.MIX_BULK
        ra, rb = a.run(w.iters), b.run(w.iters)
        for i in range(w.N):
            assert np.array_equal(ra[i], rb[i])
        assert torch.equal(a.M, b.M)
        a.h.close()
        b.h.close()


def test_a_level_with_more_distinct_slices_than_shared_memory_can_stage_is_refused():
    # 128 workers on a complete graph, 64 versions each in the ring: at level 63 every worker takes a different version
    # from every neighbour, 8192 distinct slices in one level.  No tile width fits: hop_load_trace says so (and nothing
    # is launched); a smaller trace then loads into the same context.
    N, s, P, L = 128, 63, 16, 64
    ptr, idx = inputs.graph_to_csr(inputs.complete(N))
    h = hop.Hop(ptr, idx, N, P, s, N - 1, 0)                       # one usable in-neighbour (the own update) suffices
    h.set_option(hop.OPT_WEIGHT_MODE, hop.W_STALE_LINEAR)
    h.set_option(hop.OPT_GRAD_MODE, hop.GRAD_SYNTHETIC)
    X = torch.zeros((N, s + 1, P), dtype=torch.float32, device=DEV)
    G = torch.zeros((N, P), dtype=torch.float32, device=DEV)
    h.bind_buffers(X, None, G, torch.cuda.current_stream().cuda_stream)
    ops = np.full((L, N), op.NORMAL, np.int32)
    t_ptr, nbr, ver, num = [0], [], [], []
    den = np.zeros((L, N), np.int32)
    for k in range(L):
        for i in range(N):
            rec = [(i, k)] if k < L - 1 else [(j, k if j == i else k - ((i + j) % 64)) for j in range(N)]
            for (j, v) in rec:
                nbr.append(j); ver.append(v); num.append(v - (k - s) + 1)
            den[k, i] = sum(num[t_ptr[-1]:])
            t_ptr.append(len(nbr))
    big = hop.Trace.from_arrays(ops, np.asarray(t_ptr, np.int64), nbr, ver, num, den)
    with pytest.raises(hop.HopError) as e:
        h.load_trace(big)
    assert e.value.code == hop.E_UNSUPPORTED and "distinct slices" in str(e.value)
    with pytest.raises(hop.HopError) as e:
        h.step()                                                   # nothing is loaded
    assert e.value.code == hop.E_STATE
    small = hop.Trace.from_arrays(ops[:3], np.asarray(t_ptr[:3 * N + 1], np.int64), nbr[:3 * N], ver[:3 * N], num[:3 * N], den[:3])
    h.load_trace(small)
    for _ in range(3):
        h.step()
    assert h.read_status() == 0
    h.close()


def test_reduce_set_study_runs_and_trains():
    from paper_1902_01064_b200 import study
    rows = study.reduce_set_study(P=2048, iters=200)
    assert len(rows) == 4
    start = 1.0                                        # hinge loss at p_0 = 0
    for reduce_name, weights, loss, spread, entries in rows:
        assert np.isfinite(loss) and loss < start and spread < 1.0
    by = {(r[0], r[1]): r for r in rows}
    assert by[("since previous Recv", "Eq. 2")][4] < by[("all inside the bound", "Eq. 2")][4]     # fewer terms per Reduce


@pytest.mark.parametrize("cfg,P,kernel", [(3, 5000, hop.MIX_BULK), (3, 4999, hop.MIX_BULK), (3, 4999, hop.MIX_STAGED),
                                          (4, 3001, hop.MIX_BULK), (5, 1536, hop.MIX_TENSOR), (2, 4098, hop.MIX_AUTO)])
def test_no_kernel_writes_outside_the_bound_buffers(cfg, P, kernel):
    # X, M and G are carved out of larger allocations whose margins hold a sentinel; after a full run (unaligned row
    # lengths, ragged last tiles, momentum, jumps, the tensor path, the sparse apply) every margin is untouched.
    w = workload(cfg, P=P, iters=12)
    S, guard, sentinel = w.s + 1, 4096, -12345.5
    def carve(n):
        if n == 0:
            return None, None
        whole = torch.full((guard + n + guard,), sentinel, dtype=torch.float32, device=DEV)
        return whole, whole[guard:guard + n]
    wx, X = carve(w.N * S * P)
    wm, M = carve(w.N * P if w.momentum else 0)
    wg, G = carve(0 if w.grad_mode == inputs.GRAD_SVM_CSR else w.N * P)
    X.zero_()
    if M is not None:
        M.zero_()
    if G is not None:
        G.zero_()
    h = hop.from_workload(w, kernel)
    h.bind_buffers(X, M, G, torch.cuda.current_stream().cuda_stream)
    keep = []
    if w.grad_mode == inputs.GRAD_SVM_CSR:
        keep = [torch.from_numpy(a).to(DEV) for a in (w.svm.row_ptr, w.svm.col, w.svm.val, w.svm.y)]
        h.bind_svm_csr(*keep, w.svm.rows_per_worker, w.svm.batch)
    h.load_trace(h.sim_run(w.ticks, w.iters))
    if kernel != hop.MIX_AUTO:
        assert h.level_stats(2)["kernel"] == kernel
    h.write_params(-1, 0, w.p0())
    for _ in range(w.iters):
        h.step()
    assert h.read_status() == 0
    torch.cuda.synchronize()
    for whole in (wx, wm, wg):
        if whole is not None:
            assert bool((whole[:guard] == sentinel).all()) and bool((whole[-guard:] == sentinel).all())
    assert bool(torch.isfinite(X).all())
    h.close()


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_full_size_graph_replay_equals_step_by_step(cfg):
    # bench.py times configurations 1-3 through hop_run (one replayed CUDA graph per pass of the trace, with the
    # dependent launches inside it); at full size that path must give what the step-by-step path gives, which the
    # full-size tests above compare with the oracle
    w = inputs.make_workload(cfg)
    ref = GpuRun(w).run(w.iters)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = GpuRun(w)
        g.h.run(w.iters)
        got = [g.h.read_params(i) for i in range(w.N)]
        assert g.h.read_status() == 0
        g.h.close()
    for i in range(w.N):
        if cfg == 2:                                   # float atomics in the sparse apply: order may differ
            assert np.abs(got[i] - ref[i]).max() <= 1e-5 * (np.abs(ref[i]).max() + 1e-30)
        else:
            assert np.array_equal(got[i], ref[i])


@pytest.mark.parametrize("momentum,variant", [(0.9, None), (0.0, dict(weight_decay=0.02)), (0.9, dict(weight_decay=0.02))])
def test_tensor_path_with_momentum_and_weight_decay(momentum, variant):
    # the dense path's epilogue applies -lr * G only: a pre-pass forms the update direction in G (momentum buffer, decay)
    w = workload(5, P=1536, iters=10)
    w.momentum = momentum
    g = GpuRun(w, hop.MIX_TENSOR, variant=variant)
    assert all(g.h.level_stats(k)["kernel"] == hop.MIX_TENSOR for k in range(w.iters))
    g.h.close()
    check(w, w.iters, TOL_RUN, hop.MIX_TENSOR, variant=variant)
    check(w, 1, TOL_STEP, hop.MIX_TENSOR, perturb=True, variant=variant)
    # and the general kernel gives the same within the run tolerance (both against the oracle)
    check(w, w.iters, TOL_RUN, hop.MIX_BULK, perturb=True, variant=variant)
