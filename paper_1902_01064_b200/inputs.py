"""Seeded synthetic workloads for the Hop hot path.

This module only *draws inputs*: communication graphs, per-(worker, iteration)
compute-time tables, SVM data shards, labels and initial parameters.  It contains
none of the method's arithmetic (no queue protocol, no mixing, no gradients) and
imports neither the CUDA binding nor the CPU oracle, so both of them can be fed
from it.

The five workloads take the shape of the paper's experiments (Section 7: SVM on
a very high-dimensional sparse data set with batch 128, CNN-sized parameter
vectors, ring-family graphs, random and deterministic slowdowns); the real data
sets are replaced by seeded draws.

Random source: numpy's Philox bit generator keyed by (base_seed + cfg, stream).
Streams: 0 graph, 1 compute time, 2 w*, 3 features, 4 label flips, 5 p_0,
7 test-only perturbations.  Stream 6 (synthetic gradients) is never drawn here:
the gradient of worker i at iteration k for parameter p is a pure function of
(seed, i, k, p) that the GPU path and the oracle each implement on their own.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

BASE_SEED = 190201064 * 100
TICKS_PER_UNIT = 1 << 20

UNIFORM = 0
STALE_LINEAR = 1

GRAD_EXTERNAL = 0
GRAD_SYNTHETIC = 1
GRAD_SVM_DENSE = 2
GRAD_SVM_CSR = 3


def _rng(cfg: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[BASE_SEED + cfg, stream]))


def to_ticks(tau: np.ndarray) -> np.ndarray:
    """Continuous durations -> integer ticks, never below one tick."""
    return np.maximum(1, np.rint(tau * TICKS_PER_UNIT)).astype(np.uint64)


def graph_to_csr(n_in: list[list[int]]):
    """In-neighbour lists (self included) -> (in_ptr[N+1], in_idx[nnz]) int32, ids ascending."""
    ptr = [0]
    idx: list[int] = []
    for nb in n_in:
        nb = sorted(set(int(j) for j in nb))
        idx.extend(nb)
        ptr.append(len(idx))
    return np.asarray(ptr, np.int32), np.asarray(idx, np.int32)


def csr_to_lists(in_ptr, in_idx) -> list[list[int]]:
    return [[int(j) for j in in_idx[in_ptr[i]:in_ptr[i + 1]]] for i in range(len(in_ptr) - 1)]


# ---------------------------------------------------------------- graph constructors
# Every constructor returns in-neighbour lists (self included) in ascending id order: that is the
# order in which trace records list the consumed neighbours.
def _canon(n_in):
    return [sorted(set(nb)) for nb in n_in]


def ring(n: int) -> list[list[int]]:
    """Bidirectional ring: N_in(i) = {i, i-1, i+1}."""
    return _canon([[i, (i - 1) % n, (i + 1) % n] for i in range(n)])


def ring_chords(n: int, chord: int) -> list[list[int]]:
    """Ring plus +-chord links: N_in(i) = {i, i+-1, i+-chord}."""
    return _canon([[i, (i - 1) % n, (i + 1) % n, (i - chord) % n, (i + chord) % n] for i in range(n)])


def torus(nx: int, ny: int) -> list[list[int]]:
    """2-D torus, worker id = y*nx + x, neighbours one step in each dimension."""
    out = []
    for y in range(ny):
        for x in range(nx):
            out.append([y * nx + x,
                        y * nx + (x - 1) % nx, y * nx + (x + 1) % nx,
                        ((y - 1) % ny) * nx + x, ((y + 1) % ny) * nx + x])
    return _canon(out)


def complete(n: int) -> list[list[int]]:
    return [list(range(n)) for _ in range(n)]


def directed_cycle(n: int) -> list[list[int]]:
    """i receives from i-1 only (plus itself)."""
    return _canon([[i, (i - 1) % n] for i in range(n)])


def ring_based(n: int) -> list[list[int]]:
    """Ring where every node is also linked to the most distant node (paper Fig. 'Graphs used in experiments' (2))."""
    return _canon([[i, (i - 1) % n, (i + 1) % n, (i + n // 2) % n] for i in range(n)])


def double_ring(n: int) -> list[list[int]]:
    """Two ring-based graphs of n/2 nodes joined node to node (paper Fig. 'Graphs used in experiments' (3))."""
    h = n // 2
    base = ring_based(h)
    out = []
    for g in range(2):
        for i in range(h):
            out.append([g * h + j for j in base[i]] + [(1 - g) * h + i])
    return _canon(out)


def _strongly_connected(n_in: list[list[int]]) -> bool:
    n = len(n_in)
    n_out = [[] for _ in range(n)]
    for i, nb in enumerate(n_in):
        for j in nb:
            n_out[j].append(i)
    for adj in (n_in, n_out):
        seen = {0}
        stack = [0]
        while stack:
            u = stack.pop()
            for v in adj[u]:
                if v not in seen:
                    seen.add(v)
                    stack.append(v)
        if len(seen) != n:
            return False
    return True


def random_regular_digraph(n: int, deg: int, rng: np.random.Generator) -> list[list[int]]:
    """Union of `deg` random permutations, each redrawn until it has no fixed point and repeats
    no edge of the earlier ones (so every node has deg distinct in- and out-neighbours); the
    whole graph is redrawn until strongly connected; self-loop added."""
    ident = np.arange(n)
    while True:
        perms = []
        while len(perms) < deg:
            p = rng.permutation(n)
            if np.any(p == ident) or any(np.any(p == q) for q in perms):
                continue
            perms.append(p)
        n_in = [[i] + [int(p[i]) for p in perms] for i in range(n)]
        if _strongly_connected(n_in):
            return _canon(n_in)


# ---------------------------------------------------------------- workload container
@dataclass
class SvmData:
    rows_per_worker: int
    batch: int
    y: np.ndarray                          # [N][R] float32, +-1
    dense: Optional[np.ndarray] = None     # [N][R][d] float32
    row_ptr: Optional[np.ndarray] = None   # [N*R+1] int64 (global offsets over all workers' rows)
    col: Optional[np.ndarray] = None       # [nnz] int32
    val: Optional[np.ndarray] = None       # [nnz] float32

    def column_shard(self, lo: int, hi: int) -> "SvmData":
        """The features with index in [lo, hi), renumbered from 0: what one rank of a column-sharded run binds."""
        if self.dense is not None:
            return SvmData(self.rows_per_worker, self.batch, self.y, dense=np.ascontiguousarray(self.dense[..., lo:hi]))
        keep = (self.col >= lo) & (self.col < hi)
        kept_before = np.concatenate([[0], np.cumsum(keep, dtype=np.int64)])
        return SvmData(self.rows_per_worker, self.batch, self.y, row_ptr=kept_before[self.row_ptr],
                       col=(self.col[keep] - lo).astype(np.int32), val=self.val[keep])


@dataclass
class Workload:
    cfg: int
    name: str
    N: int
    P: int
    iters: int
    s: int
    b: int
    max_skip: int
    max_ig: int
    lr: float
    momentum: float
    weight_mode: int
    grad_mode: int
    in_ptr: np.ndarray
    in_idx: np.ndarray
    ticks: np.ndarray                      # [N][iters] uint64
    grad_seed: int = 0
    sigma: float = 1e-3
    svm: Optional[SvmData] = None
    p0_zero: bool = False
    stale_reduce: int = 0                  # 0: only updates that arrived since the previous Recv are reduced (Eq. 2 as printed); 1: reuse
    _p0: Optional[np.ndarray] = field(default=None, repr=False)

    @property
    def n_in(self) -> list[list[int]]:
        return csr_to_lists(self.in_ptr, self.in_idx)

    def p0(self) -> np.ndarray:
        """Initial parameters p_0 (float32 [P]), common to all workers (paper Fig. alg1)."""
        if self._p0 is None:
            if self.p0_zero:
                self._p0 = np.zeros(self.P, np.float32)
            else:
                self._p0 = _rng(self.cfg, 5).standard_normal(self.P, dtype=np.float32)
        return self._p0

    def perturbation(self, worker: int, scale: float = 1.0) -> np.ndarray:
        """Test-only per-worker offset eps_i ~ N(0, scale^2) so that replicas differ at iteration 0."""
        g = np.random.Generator(np.random.Philox(key=[BASE_SEED + self.cfg, 7 + 16 * (worker + 1)]))
        return (scale * g.standard_normal(self.P, dtype=np.float32)).astype(np.float32)


def default_max_ig(s: int) -> int:
    return max(1, s)


def _labels(margin: np.ndarray, flips: np.ndarray) -> np.ndarray:
    y = np.where(margin >= 0, 1.0, -1.0).astype(np.float32)
    return np.where(flips, -y, y).astype(np.float32)


def make_workload(cfg: int, P: Optional[int] = None, iters: Optional[int] = None) -> Workload:
    """Build workload `cfg` (1..5).  `P` / `iters` override the size for reduced test cases;
    graph, protocol knobs and the compute-time model stay those of the configuration."""
    if cfg == 1:
        N, d, R, B = 4, 64 if P is None else P, 256, 32
        iters = 20 if iters is None else iters
        n_in = ring(N)
        tau = _rng(cfg, 1).exponential(1.0, size=(N, iters))
        wstar = _rng(cfg, 2).standard_normal(d)
        A = _rng(cfg, 3).standard_normal((N, R, d)).astype(np.float32)
        flips = _rng(cfg, 4).random((N, R)) < 0.05
        y = _labels(A.astype(np.float64) @ wstar, flips)
        ptr, idx = graph_to_csr(n_in)
        return Workload(cfg, "svm-dense-ring4", N, d, iters, s=1, b=0, max_skip=0, max_ig=default_max_ig(1),
                        lr=0.01, momentum=0.0, weight_mode=UNIFORM, grad_mode=GRAD_SVM_DENSE,
                        in_ptr=ptr, in_idx=idx, ticks=to_ticks(tau),
                        svm=SvmData(R, B, y, dense=A), p0_zero=True)
    if cfg == 2:
        N, d, B, nnz_row = 16, (1 << 20) if P is None else P, 128, 100
        R = 4096 if P is None else 512
        iters = 200 if iters is None else iters
        nnz_row = min(nnz_row, d)
        n_in = ring_chords(N, 4)
        slow = _rng(cfg, 1).random((N, iters)) < 0.1
        tau = np.where(slow, 5.0, 1.0)
        wstar = _rng(cfg, 2).standard_normal(d)
        g = _rng(cfg, 3)
        rows = N * R
        # distinct uniform-random columns per row: draw with replacement, redraw rows with repeats
        col = g.integers(0, d, size=(rows, nnz_row), dtype=np.int64)
        col.sort(axis=1)
        bad = np.nonzero((np.diff(col, axis=1) == 0).any(axis=1))[0]
        while bad.size:
            for r in bad:
                col[r] = np.sort(g.choice(d, size=nnz_row, replace=False))
            bad = np.nonzero((np.diff(col, axis=1) == 0).any(axis=1))[0]
        val = g.lognormal(0.0, 1.0, size=(rows, nnz_row))
        val /= np.sqrt((val * val).sum(axis=1, keepdims=True))
        val = val.astype(np.float32)
        margin = (val.astype(np.float64) * wstar[col]).sum(axis=1)
        flips = _rng(cfg, 4).random(rows) < 0.05
        y = _labels(margin, flips).reshape(N, R)
        row_ptr = (np.arange(rows + 1, dtype=np.int64) * nnz_row)
        ptr, idx = graph_to_csr(n_in)
        return Workload(cfg, "svm-csr-ring16-chords", N, d, iters, s=2, b=1, max_skip=0, max_ig=default_max_ig(2),
                        lr=0.05, momentum=0.0, weight_mode=STALE_LINEAR, grad_mode=GRAD_SVM_CSR,
                        in_ptr=ptr, in_idx=idx, ticks=to_ticks(tau),
                        svm=SvmData(R, B, y, row_ptr=row_ptr, col=col.reshape(-1).astype(np.int32),
                                    val=val.reshape(-1)), p0_zero=True)
    if cfg == 3:
        N = 32
        P = 1_200_000 if P is None else P
        iters = 100 if iters is None else iters
        n_in = torus(4, 8)
        tau = np.ones((N, iters))
        tau[0, :] = 4.0
        tau[17, :] = 4.0
        ptr, idx = graph_to_csr(n_in)
        return Workload(cfg, "synthetic-torus8x4-momentum-skip", N, P, iters, s=3, b=0, max_skip=2,
                        max_ig=default_max_ig(3), lr=0.1, momentum=0.9, weight_mode=STALE_LINEAR,
                        grad_mode=GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx, ticks=to_ticks(tau),
                        grad_seed=BASE_SEED + cfg)
    if cfg == 4:
        N = 64
        P = 25_600_000 if P is None else P
        iters = 50 if iters is None else iters
        g0 = _rng(cfg, 0)
        n_in = random_regular_digraph(N, 6, g0)
        g1 = _rng(cfg, 1)
        tau = g1.lognormal(0.0, 0.5, size=(N, iters))
        slow_worker = int(g1.integers(0, N))
        tau[slow_worker, :] *= 3.0
        ptr, idx = graph_to_csr(n_in)
        return Workload(cfg, "synthetic-random6regular64", N, P, iters, s=4, b=2, max_skip=0,
                        max_ig=default_max_ig(4), lr=0.1, momentum=0.0, weight_mode=STALE_LINEAR,
                        grad_mode=GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx, ticks=to_ticks(tau),
                        grad_seed=BASE_SEED + cfg)
    if cfg == 5:
        N = 128
        P = 8_000_000 if P is None else P
        iters = 30 if iters is None else iters
        n_in = complete(N)
        tau = _rng(cfg, 1).exponential(1.0, size=(N, iters))
        ptr, idx = graph_to_csr(n_in)
        return Workload(cfg, "synthetic-complete128-dense", N, P, iters, s=1, b=8, max_skip=0,
                        max_ig=default_max_ig(1), lr=0.05, momentum=0.0, weight_mode=STALE_LINEAR,
                        grad_mode=GRAD_SYNTHETIC, in_ptr=ptr, in_idx=idx, ticks=to_ticks(tau),
                        grad_seed=BASE_SEED + cfg)
    raise ValueError(f"unknown configuration {cfg}")


def small_cases():
    """Tiny graphs for exhaustive protocol enumeration: (name, in-neighbour lists)."""
    return [("complete3", complete(3)), ("cycle3", directed_cycle(3)),
            ("ring4", ring(4)), ("complete4", complete(4))]
