"""Production protocol simulator (C++, queue-free formulation) against the oracle (Python, literal
queues): traces must be bit-identical.  CPU only: hop_sim_run touches no GPU."""
import itertools

import numpy as np
import pytest

from oracle import protocol as op
from paper_1902_01064_b200 import hop, inputs

KEYS = ("op", "ptr", "nbr", "ver", "num", "den")


def both(n_in, ticks, iters, s, b, max_ig, max_skip, mode, exact=False, notify_ack=False, reduce=op.NEW_ONLY, serial=False):
    ptr, idx = inputs.graph_to_csr(n_in)
    n_in = inputs.csr_to_lists(ptr, idx)                 # records list neighbours in ascending id order
    h = hop.Hop(ptr, idx, len(n_in), 8, s, b, max_skip)
    h.set_option(hop.OPT_MAX_IG, 0 if max_ig is None else max_ig)
    h.set_option(hop.OPT_WEIGHT_MODE, mode)
    h.set_option(hop.OPT_BACKUP_MODE, hop.BACKUP_EXACT if exact else hop.BACKUP_AT_LEAST)
    h.set_option(hop.OPT_NOTIFY_ACK, 1 if notify_ack else 0)
    assert (hop.STALE_NEW_ONLY, hop.STALE_REUSE) == (op.NEW_ONLY, op.REUSE)
    h.set_option(hop.OPT_STALE_REDUCE, reduce)
    h.set_option(hop.OPT_APPROACH, hop.APPROACH_SERIAL if serial else hop.APPROACH_PARALLEL)
    got = h.sim_run(ticks, iters).to_arrays()
    want_tr = op.simulate(n_in, ticks, iters, s, b, None if notify_ack else max_ig, max_skip, mode, backup_exact=exact,
                          notify_ack=notify_ack, stale_reduce=reduce, serial=serial)
    want = want_tr.to_arrays()
    h.close()
    return got, want, want_tr.makespan


def assert_same(got, want, makespan, ctx=""):
    for k in KEYS:
        assert np.array_equal(got[k], want[k]), (k, ctx)
    assert got["makespan"] == makespan, ctx


@pytest.mark.parametrize("reduce", [op.NEW_ONLY, op.REUSE])
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_configs_bit_exact(cfg, reduce):
    w = inputs.make_workload(cfg, P=64 if cfg == 1 else 256)
    got, want, mk = both(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode, reduce=reduce)
    assert_same(got, want, mk, cfg)
    assert (got["op"] != op.IDLE).sum() > 0
    if reduce == op.NEW_ONLY:      # every configuration has stalled neighbours: the two readings must differ
        other = both(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode, reduce=op.REUSE)[0]
        assert np.array_equal(other["op"], got["op"]) and other["makespan"] == got["makespan"]
        assert other["ptr"][-1] > got["ptr"][-1]


def _enumerate(name, n_in, iters, values, combos):
    N = len(n_in)
    count = 0
    for flat in itertools.product(values, repeat=N * iters):
        ticks = np.asarray(flat, np.uint64).reshape(N, iters)
        for (s, b, max_skip) in combos:
            if any(b >= len(nb) for nb in n_in) or max_skip > s + 1:
                continue
            max_ig = max(1, s)
            for reduce in ((op.NEW_ONLY, op.REUSE) if s > 0 else (op.NEW_ONLY,)):    # the readings coincide at s = 0
                got, want, mk = both(n_in, ticks, iters, s, b, max_ig, max_skip, op.STALE_LINEAR, reduce=reduce)
                assert_same(got, want, mk, (name, flat, s, b, max_skip, reduce))
            count += 1
    return count


ALL_COMBOS = [(s, b, k) for s in (0, 1, 2) for b in (0, 1) for k in (0, 1, 2)]


def test_exhaustive_three_workers_two_iterations():
    for name, n_in in inputs.small_cases()[:2]:
        assert _enumerate(name, n_in, 2, (1, 2, 3), ALL_COMBOS) > 5000


def test_exhaustive_three_workers_three_iterations():
    # 2^9 tick tables x all protocol settings, two tick alphabets
    for name, n_in in inputs.small_cases()[:2]:
        _enumerate(name, n_in, 3, (1, 2), ALL_COMBOS)
        _enumerate(name, n_in, 3, (1, 3), [(1, 1, 2), (2, 0, 2), (0, 1, 1)])


def test_exhaustive_four_workers():
    for name, n_in in inputs.small_cases()[2:]:
        _enumerate(name, n_in, 2, (1, 2), ALL_COMBOS)
        _enumerate(name, n_in, 3, (1, 2), [(1, 1, 2), (2, 0, 1)])


def test_random_graphs_long_runs_with_ties_and_skips():
    rng = np.random.default_rng(42)
    for trial in range(60):
        N = int(rng.integers(3, 12))
        n_in = [{i, (i - 1) % N} for i in range(N)]
        for _ in range(int(rng.integers(0, 3 * N))):
            a, c = rng.integers(0, N, 2)
            n_in[int(a)].add(int(c))
        n_in = [sorted(x) for x in n_in]
        s = int(rng.integers(0, 4))
        b = int(rng.integers(0, min(len(x) for x in n_in)))
        max_skip = int(rng.integers(0, s + 2))
        max_ig = int(rng.integers(1, 5))
        iters = 25
        ticks = rng.choice([1, 1, 1, 2, 5], size=(N, iters)).astype(np.uint64)
        if trial % 3 == 0:
            ticks[int(rng.integers(0, N)), :] *= 4          # deterministic straggler
        mode = int(rng.integers(0, 2))
        try:
            want_tr = op.simulate(n_in, ticks, iters, s, b, max_ig, max_skip, mode)
        except op.Deadlock:
            ptr, idx = inputs.graph_to_csr(n_in)
            h = hop.Hop(ptr, idx, N, 8, s, b, max_skip)
            h.set_option(hop.OPT_MAX_IG, max_ig)
            with pytest.raises(hop.HopError) as e:
                h.sim_run(ticks, iters)
            assert e.value.code == hop.E_DEADLOCK
            continue
        for reduce in (op.NEW_ONLY, op.REUSE):
            got, want, mk = both(n_in, ticks, iters, s, b, max_ig, max_skip, mode, reduce=reduce)
            assert_same(got, want, mk, (trial, reduce))


def test_unbounded_gap_without_tokens():
    n_in = inputs.complete(3)
    ticks = np.ones((3, 12), np.uint64)
    ticks[0, 0] = 10 ** 12
    got, want, mk = both(n_in, ticks, 12, 0, 1, None, 0, op.UNIFORM)
    assert_same(got, want, mk)


def test_exact_backup_mode_bit_exact_and_exactly_d_minus_b():
    rng = np.random.default_rng(77)
    for trial in range(40):
        N = int(rng.integers(4, 12))
        n_in = [{i, (i - 1) % N, (i + 1) % N} for i in range(N)]
        for _ in range(int(rng.integers(N, 4 * N))):
            a, c = rng.integers(0, N, 2)
            n_in[int(a)].add(int(c))
        n_in = [sorted(x) for x in n_in]
        s = int(rng.integers(0, 3))
        b = int(rng.integers(1, min(len(x) for x in n_in)))
        max_skip = int(rng.integers(0, s + 2)) if trial % 2 else 0
        iters = 20
        ticks = rng.choice([1, 2, 3, 9], size=(N, iters)).astype(np.uint64)
        for reduce in (op.REUSE, op.NEW_ONLY):
            try:
                got, want, mk = both(n_in, ticks, iters, s, b, 3, max_skip, op.STALE_LINEAR, exact=True, reduce=reduce)
            except op.Deadlock:
                continue
            assert_same(got, want, mk, (trial, reduce))
            cnt = np.diff(got["ptr"]).reshape(iters, N)
            for i in range(N):
                active = got["op"][:, i] != op.IDLE
                if reduce == op.REUSE or s == 0:
                    assert (cnt[active, i] == len(n_in[i]) - b).all()      # exactly in-degree - b consumed
                else:
                    assert (cnt[active, i] >= 1).all() and (cnt[active, i] <= len(n_in[i]) - b).all()
    for name, n_in in inputs.small_cases():
        if name.endswith("3"):
            continue
        for flat in itertools.product((1, 2, 3), repeat=8):
            ticks = np.asarray(flat, np.uint64).reshape(4, 2)
            for reduce in (op.REUSE, op.NEW_ONLY):
                got, want, mk = both(n_in, ticks, 2, 1, 1, 1, 0, op.UNIFORM, exact=True, reduce=reduce)
                assert_same(got, want, mk, (name, flat, reduce))


@pytest.mark.parametrize("reduce", [op.REUSE, op.NEW_ONLY])
@pytest.mark.parametrize("cfg", [2, 4, 5])
def test_configs_bit_exact_in_exact_backup_mode(cfg, reduce):
    w = inputs.make_workload(cfg, P=256)
    got, want, mk = both(w.n_in, w.ticks, w.iters, w.s, w.b, w.max_ig, w.max_skip, w.weight_mode, exact=True, reduce=reduce)
    assert_same(got, want, mk, cfg)
    d = np.diff(w.in_ptr)
    cnt = np.diff(got["ptr"]).reshape(w.iters, w.N)
    if reduce == op.REUSE:
        assert (cnt == (d - w.b)[None, :]).all()
    else:
        assert (cnt >= 1).all() and (cnt <= (d - w.b)[None, :]).all() and (cnt < (d - w.b)[None, :]).any()


def test_notify_ack_bit_exact():
    rng = np.random.default_rng(5)
    for trial in range(30):
        N = int(rng.integers(3, 10))
        n_in = [{i, (i - 1) % N} for i in range(N)]
        for _ in range(int(rng.integers(0, 3 * N))):
            a, c = rng.integers(0, N, 2)
            n_in[int(a)].add(int(c))
        n_in = [sorted(x) for x in n_in]
        s = int(rng.integers(0, 3))
        b = int(rng.integers(0, min(len(x) for x in n_in)))
        ticks = rng.choice([1, 1, 2, 6], size=(N, 15)).astype(np.uint64)
        got, want, mk = both(n_in, ticks, 15, s, b, 1, 0, op.UNIFORM, notify_ack=True)
        assert_same(got, want, mk, trial)
    for name, n_in in inputs.small_cases()[:2]:
        for flat in itertools.product((1, 2, 3), repeat=9):
            got, want, mk = both(n_in, np.asarray(flat, np.uint64).reshape(3, 3), 3, 0, 0, 1, 0, op.UNIFORM, notify_ack=True)
            assert_same(got, want, mk, (name, flat))


def test_serial_approach_bit_exact():
    """Serial approach (Section 3.2): updates leave at the end of Compute.  Random graphs with ties, stragglers, backup
    workers, both Reduce sets, EXACT backup and skipping; plus an exhaustive sweep on the small graphs."""
    rng = np.random.default_rng(314)
    differs = 0
    for trial in range(40):
        N = int(rng.integers(3, 11))
        n_in = [{i, (i - 1) % N} for i in range(N)]
        for _ in range(int(rng.integers(0, 3 * N))):
            a, c = rng.integers(0, N, 2)
            n_in[int(a)].add(int(c))
        n_in = [sorted(x) for x in n_in]
        s = int(rng.integers(0, 4))
        b = int(rng.integers(0, min(len(x) for x in n_in)))
        max_skip = int(rng.integers(0, s + 2)) if trial % 2 else 0
        max_ig = int(rng.integers(1, 5))
        ticks = rng.choice([1, 1, 2, 5], size=(N, 20)).astype(np.uint64)
        kw = dict(exact=bool(trial % 3 == 0), reduce=op.REUSE if trial % 4 == 0 else op.NEW_ONLY)
        try:
            got, want, mk = both(n_in, ticks, 20, s, b, max_ig, max_skip, op.STALE_LINEAR, serial=True, **kw)
        except op.Deadlock:
            continue
        assert_same(got, want, mk, trial)
        try:
            par = both(n_in, ticks, 20, s, b, max_ig, max_skip, op.STALE_LINEAR, **kw)[0]
            differs += par["makespan"] != got["makespan"] or not np.array_equal(par["ver"], got["ver"])
        except op.Deadlock:
            pass
    assert differs > 10
    for name, n_in in inputs.small_cases():
        N = len(n_in)
        for flat in itertools.product((1, 2), repeat=N * 2):
            ticks = np.asarray(flat, np.uint64).reshape(N, 2)
            for (s, b, max_skip) in [(0, 0, 0), (1, 0, 0), (1, 1, 0), (2, 0, 2), (1, 1, 1)]:
                if any(b >= len(nb) for nb in n_in):
                    continue
                got, want, mk = both(n_in, ticks, 2, s, b, max(1, s), max_skip, op.STALE_LINEAR, serial=True)
                assert_same(got, want, mk, (name, flat, s, b, max_skip))
