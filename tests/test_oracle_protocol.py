"""Pins for the protocol oracle against what the paper and mathematics fix (CPU only)."""
import os

import numpy as np
import pytest

from oracle import protocol as op
from paper_1902_01064_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_examples.txt")
STUCK = 10 ** 15


def golden():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


def rand_ticks(rng, N, iters, lo=1, hi=6):
    return rng.integers(lo, hi, size=(N, iters)).astype(np.uint64)


GRAPHS = [("ring6", inputs.ring(6)), ("cycle5", inputs.directed_cycle(5)), ("torus", inputs.torus(3, 3)),
          ("complete4", inputs.complete(4)), ("ringbased8", inputs.ring_based(8))]


# ------------------------------------------------------------------ Theorem 1
@pytest.mark.parametrize("name,n_in", GRAPHS)
def test_theorem1_gap_bounded_by_shortest_path(name, n_in):
    rng = np.random.default_rng(1)
    N = len(n_in)
    dist = op.shortest_paths(n_in)
    for trial in range(10):
        seen = []

        def chk(p):
            for i in range(N):
                for j in range(N):
                    assert p.Iter[i] - p.Iter[j] <= dist[j][i]
            seen.append(max(p.Iter) - min(p.Iter))
        op.simulate(n_in, rand_ticks(rng, N, 12, 1, 9), 12, on_round=chk)
        assert seen


def test_theorem1_bound_is_reached_on_a_chain():
    # Chain 0 -> 1 -> 2 -> 3 with a slow head: the worker at distance d from worker 0 gets exactly
    # d iterations ahead of it, so the bound of Theorem 1 is tight.
    n_in = [[0], [0, 1], [1, 2], [2, 3]]
    ticks = np.ones((4, 8), np.uint64)
    ticks[0, :] = 100
    best = [0] * 4

    def chk(p):
        for i in range(4):
            best[i] = max(best[i], p.Iter[i] - p.Iter[0])
    op.simulate(n_in, ticks, 8, on_round=chk)
    assert best == [0, 1, 2, 3]


# ------------------------------------------------------------------ closed form (max-plus recurrence)
def recurrence(n_in, T, iters, s, max_ig, serial=False):
    """start/finish times for b = 0, no skipping: a worker finishes Recv(k) once its compute is over
    and every in-neighbour has sent iteration k - s -- on entering it (parallel approach) or at the end
    of its Compute (serial approach, Section 3.2); it enters k+1 once every out-neighbour has entered
    k + 1 - max_ig.  Returns (start, finish, sent)."""
    N = len(n_in)
    n_out = [[i for i in range(N) if j in n_in[i] and i != j] for j in range(N)]
    start = np.zeros((N, iters + 1), np.int64)
    fin = np.zeros((N, iters), np.int64)
    sent = np.zeros((N, iters), np.int64)
    for k in range(iters):
        for i in range(N):
            sent[i, k] = start[i, k] + (int(T[i][k]) if serial else 0)
        for i in range(N):
            f = start[i, k] + int(T[i][k])
            for j in n_in[i]:
                if j != i:
                    f = max(f, sent[j, max(k - s, 0)])
            fin[i, k] = f
        for i in range(N):
            st = fin[i, k]
            if max_ig is not None and k + 1 - max_ig >= 0:
                for j in n_out[i]:
                    st = max(st, start[j, k + 1 - max_ig])
            start[i, k + 1] = st
    return start, fin, sent


@pytest.mark.parametrize("serial", [False, True])
@pytest.mark.parametrize("s,max_ig", [(0, None), (0, 1), (0, 3), (2, None), (2, 2), (3, 1)])
def test_times_and_versions_match_maxplus_recurrence(s, max_ig, serial):
    rng = np.random.default_rng(7 + s)
    for name, n_in in GRAPHS:
        N = len(n_in)
        iters = 9
        T = rng.integers(10 ** 6, 3 * 10 ** 6, size=(N, iters)).astype(np.uint64)
        if max_ig is not None and max_ig < 1:
            continue
        starts = {}

        def chk(p):
            for i in range(N):
                starts.setdefault((i, p.Iter[i]), p.now)
        tr = op.simulate(n_in, T, iters, s=s, b=0, max_ig=max_ig, weight_mode=op.STALE_LINEAR, on_round=chk,
                         stale_reduce=op.REUSE, serial=serial)
        # in the parallel approach every wait looks at a lower or equal level whose start time is already final; in
        # the serial approach the level's own send times only need its start times: one sweep per level either way
        st, fin, sent = recurrence(n_in, T, iters, s, max_ig, serial)
        for i in range(N):
            for k in range(1, iters):
                assert starts[(i, k)] == st[i, k], (name, i, k)
        assert tr.makespan == fin[:, iters - 1].max()
        # generic position: consumed version = newest v <= k sent before Recv(k) finished
        for i in range(N):
            for k in range(iters):
                assert sorted(j for j, _, _ in tr.rec[(k, i)]) == sorted(n_in[i])
                for (j, v, w) in tr.rec[(k, i)]:
                    if j == i:
                        assert v == k
                        continue
                    cand = [u for u in range(0, k + 1) if sent[j, u] < fin[i, k]]
                    ties = [u for u in range(0, k + 1) if sent[j, u] == fin[i, k]]
                    if not ties:
                        assert v == max(cand), (name, i, k, j)
                    assert k - s <= v <= k
                    assert w == v - (k - s) + 1


def test_serial_approach_with_s0_waits_for_the_neighbours_compute():
    """Section 3.2: in the serial approach the update of iteration k leaves after Compute(k), so with s = 0 a worker's
    Recv(k) ends with the slowest in-neighbour's Compute(k); in the parallel approach that update was sent on entering k,
    and only the worker's own Compute counts."""
    n_in = [[0, 1], [1]]                                    # worker 0 listens to worker 1
    T = np.array([[1, 1, 1], [5, 5, 5]], np.uint64)
    par = op.simulate(n_in, T, 3, s=0, max_ig=None)
    ser = op.simulate(n_in, T, 3, s=0, max_ig=None, serial=True)
    assert (par.makespan, ser.makespan) == (15, 15)         # worker 1 alone sets the makespan
    done = {}

    def chk(p):
        done.setdefault((p.serial, p.Iter[0]), p.now)
    op.simulate(n_in, T, 3, s=0, max_ig=None, on_round=chk)
    op.simulate(n_in, T, 3, s=0, max_ig=None, serial=True, on_round=chk)
    assert done[(False, 1)] == 1 and done[(True, 1)] == 5   # tick at which worker 0 enters iteration 1


# ------------------------------------------------------------------ tokens
@pytest.mark.parametrize("max_ig", [1, 2, 3])
@pytest.mark.parametrize("name,n_in", GRAPHS)
def test_token_identity_theorem2_and_capacity(name, n_in, max_ig):
    rng = np.random.default_rng(3)
    N = len(n_in)
    dist = op.shortest_paths(n_in)
    for trial in range(6):
        def chk(p):
            assert op.token_identity_holds(p)                    # Section 4.2 proof
            for i in range(N):
                for j in range(N):
                    if i != j:
                        assert p.Iter[i] - p.Iter[j] <= min(dist[j][i], max_ig * dist[i][j])   # Theorem 2
            for (a, c), q in p.token_q.items():                  # TokenQ(a -> c): capacity bound
                assert len(q) <= max_ig * (dist[a][c] + 1)
        op.simulate(n_in, rand_ticks(rng, N, 10, 1, 12), 10, max_ig=max_ig, on_round=chk)


def test_token_prose_example_sender_stops_at_max_ig():
    g = golden()
    max_ig = int(g["token_example.max_ig"])
    # B (=1) sends to A (=0); A never finishes its first Compute.
    n_in = [[0, 1], [1]]
    ticks = np.ones((2, 10), np.uint64)
    ticks[0, 0] = STUCK
    top = [0]

    def chk(p):
        if p.Iter[0] == 0 and p.now < STUCK:
            top[0] = max(top[0], p.Iter[1])
    op.simulate(n_in, ticks, 10, max_ig=max_ig, on_round=chk)
    assert top[0] == int(g["token_example.sender_final_iter"])
    # without token queues nothing stops the sender (Theorem 1 only bounds the receiver)
    top[0] = 0
    op.simulate(n_in, ticks, 10, max_ig=None, on_round=chk)
    assert top[0] == 9


# ------------------------------------------------------------------ bounded staleness
@pytest.mark.parametrize("s", [1, 2, 4])
@pytest.mark.parametrize("name,n_in", GRAPHS)
def test_staleness_window_and_gap(name, n_in, s):
    rng = np.random.default_rng(11)
    N = len(n_in)
    dist = op.shortest_paths(n_in)
    for trial in range(5):
        def chk(p):
            for i in range(N):
                for j in range(N):
                    if i != j:
                        assert p.Iter[i] - p.Iter[j] <= (s + 1) * dist[j][i]      # Table 1, row 2
        T = rand_ticks(rng, N, 12, 1, 30)
        for mode in (op.NEW_ONLY, op.REUSE):
            tr = op.simulate(n_in, T, 12, s=s, weight_mode=op.STALE_LINEAR, on_round=chk, stale_reduce=mode)
            for (k, i), rec in tr.rec.items():
                if mode == op.REUSE:
                    assert sorted(j for j, _, _ in rec) == sorted(n_in[i])       # b = 0: everyone, every level
                else:
                    assert (i, k, s + 1) in rec                                  # the own update is always new
                    assert set(j for j, _, _ in rec) <= set(n_in[i])
                for (j, v, w) in rec:
                    assert k - s <= v <= k                                       # never older than s
                    assert 1 <= w == v - (k - s) + 1 <= s + 1                    # Eq. 2 numerator
                assert tr.den[(k, i)] == sum(w for _, _, w in rec)


def _pairs(text):
    return [tuple(int(x) for x in item.split(":")) for item in text.split(",")]


def test_stale_reduce_hand_worked_example():
    """Section 4.4 / Eq. 2 worked by hand (tests/golden): one neighbour stalls, its last update stays inside the
    bound for two more iterations.  NEW_ONLY (Eq. 2's index set, Fig. alg3's `if`) leaves it out of those Reduces,
    REUSE counts it again with a lower weight; both block and resume at the same tick."""
    g = golden()
    s = int(g["stale_example.s"])
    ticks = np.ones((3, 6), np.uint64)
    ticks[0, 1] = int(g["stale_example.slow_ticks"])
    want = {op.NEW_ONLY: ("den_new_only", "consumed_new_only_iter2"), op.REUSE: ("den_reuse", "consumed_reuse_iter2")}
    for mode, (kd, kc) in want.items():
        entered = {}

        def chk(p):
            entered.setdefault((1, p.Iter[1]), p.now)
        tr = op.simulate(inputs.complete(3), ticks, 6, s=s, b=0, max_ig=None, weight_mode=op.STALE_LINEAR,
                         stale_reduce=mode, on_round=chk)
        assert [tr.den[(k, 1)] for k in range(5)] == [int(x) for x in g["stale_example." + kd].split(",")]
        assert [(j, v) for j, v, _ in tr.rec[(2, 1)]] == _pairs(g["stale_example." + kc])
        assert entered[(1, 5)] == int(g["stale_example.release_tick_iter4"])    # Recv(4) completes, iteration 5 entered


@pytest.mark.parametrize("s,b,max_ig,max_skip", [(1, 0, None, 0), (2, 0, 2, 0), (3, 1, 3, 0), (2, 1, 2, 2), (4, 2, 4, 0)])
def test_new_only_is_reuse_minus_what_the_previous_recv_already_took(s, b, max_ig, max_skip):
    """The two readings differ only in the Reduce set, never in when a Recv completes: same ops, same makespan, and a
    NEW_ONLY record is the REUSE record without the (neighbour, iteration) pairs that the worker's previous Recv had
    already returned.  (Derived here from the REUSE trace alone, independently of the oracle's bookkeeping.)"""
    rng = np.random.default_rng(100 + s)
    dropped = 0
    for name, n_in in GRAPHS:
        if any(b >= len(nb) for nb in n_in):
            continue
        N = len(n_in)
        T = rand_ticks(rng, N, 14, 1, 25)
        kw = dict(s=s, b=b, max_ig=max_ig, max_skip=max_skip, weight_mode=op.STALE_LINEAR)
        new = op.simulate(n_in, T, 14, stale_reduce=op.NEW_ONLY, **kw)
        old = op.simulate(n_in, T, 14, stale_reduce=op.REUSE, **kw)
        assert np.array_equal(new.op, old.op) and new.makespan == old.makespan
        for i in range(N):
            prev = set()
            for k in range(14):
                if (k, i) not in old.rec:
                    continue
                full = [(j, v) for j, v, _ in old.rec[(k, i)]]
                expect = [(j, v) for (j, v) in full if j == i or (j, v) not in prev]
                assert [(j, v) for j, v, _ in new.rec[(k, i)]] == expect, (name, i, k)
                nums, den = op.reduce_weights([k if j == i else v for j, v in expect], k, s, op.STALE_LINEAR)
                assert [w for _, _, w in new.rec[(k, i)]] == nums and new.den[(k, i)] == den
                dropped += len(full) - len(expect)
                prev = set(full)
    assert dropped > 0, "no neighbour ever stalled: the test is vacuous"


def test_new_only_equals_reuse_when_nothing_is_stale():
    """s = 0 (Figs. alg1 / alg4): an update of iteration k is first dequeued by Recv(k), so both readings coincide."""
    rng = np.random.default_rng(17)
    for name, n_in in GRAPHS:
        for b in (0, 1):
            if any(b >= len(nb) for nb in n_in):
                continue
            T = rand_ticks(rng, len(n_in), 10, 1, 20)
            a = op.simulate(n_in, T, 10, s=0, b=b, max_ig=2, stale_reduce=op.NEW_ONLY).to_arrays()
            c = op.simulate(n_in, T, 10, s=0, b=b, max_ig=2, stale_reduce=op.REUSE).to_arrays()
            assert all(np.array_equal(a[k], c[k]) for k in a)


def test_staleness_stuck_neighbour_reaches_s_plus_one():
    g = golden()
    s = int(g["staleness_example.s"])
    n_in = inputs.complete(3)
    ticks = np.ones((3, 12), np.uint64)
    ticks[0, 0] = STUCK
    lead = [0, 0, 0]

    def chk(p):
        if p.now < STUCK:
            for i in range(3):
                lead[i] = max(lead[i], p.Iter[i] - p.Iter[0])
    op.simulate(n_in, ticks, 12, s=s, on_round=chk)
    assert lead[1] == lead[2] == int(g["staleness_example.max_lead"]) == s + 1


# ------------------------------------------------------------------ backup workers
def test_backup_counts_and_versions():
    rng = np.random.default_rng(5)
    for name, n_in in GRAPHS:
        N = len(n_in)
        for b in (1, 2):
            if any(b >= len(nb) for nb in n_in):
                continue
            tr = op.simulate(n_in, rand_ticks(rng, N, 10, 1, 40), 10, s=0, b=b, max_ig=2)
            short = 0
            for (k, i), rec in tr.rec.items():
                d = len(n_in[i])
                assert d - b <= len(rec) <= d                                     # Fig. alg4: needed + extras
                assert all(v == k for _, v, _ in rec)                             # only iteration k
                assert (i, k, 1) in rec                                           # own update, plain mean
                assert tr.den[(k, i)] == len(rec)
                short += len(rec) < d
            assert short > 0, "backup never used: test is vacuous"


def test_backup_prose_example_three_workers():
    g = golden()
    assert int(g["backup_example.workers"]) == 3
    b = 2 - int(g["backup_example.needed_neighbour_updates"])                    # two neighbours, one needed
    n_in = inputs.complete(3)
    ticks = np.ones((3, 15), np.uint64)
    ticks[0, 0] = STUCK
    top = [0, 0, 0]

    def chk(p):
        if p.now < STUCK:
            for i in range(3):
                top[i] = max(top[i], p.Iter[i])
    # no token queues: B and C run to the end relying on one another
    op.simulate(n_in, ticks, 15, s=0, b=b, max_ig=None, on_round=chk)
    assert top == [0, 14, 14]
    # without backup they are dragged down: one iteration ahead at most (Theorem 1)
    top[:] = [0, 0, 0]
    op.simulate(n_in, ticks, 15, s=0, b=0, max_ig=None, on_round=chk)
    assert top == [0, 1, 1]
    # with token queues the unbounded gap is cut at max_ig (Section 4.3)
    for max_ig in (1, 2, 4):
        top[:] = [0, 0, 0]
        op.simulate(n_in, ticks, 15, s=0, b=b, max_ig=max_ig, on_round=chk)
        assert top == [0, max_ig, max_ig]


@pytest.mark.parametrize("s,b", [(0, 1), (2, 0), (2, 1), (1, 2)])
def test_table1_last_row_with_tokens(s, b):
    rng = np.random.default_rng(13)
    for name, n_in in GRAPHS:
        if any(b >= len(nb) for nb in n_in):
            continue
        N = len(n_in)
        dist = op.shortest_paths(n_in)
        b0 = 10 ** 9 if b > 0 else s + 1
        for max_ig in (1, 3):
            def chk(p):
                assert op.token_identity_holds(p)
                for i in range(N):
                    for j in range(N):
                        if i != j:
                            assert p.Iter[i] - p.Iter[j] <= min(b0 * dist[j][i], max_ig * dist[i][j])
            T = rand_ticks(rng, N, 10, 1, 25)
            for mode in (op.NEW_ONLY, op.REUSE):
                tr = op.simulate(n_in, T, 10, s=s, b=b, max_ig=max_ig, weight_mode=op.STALE_LINEAR, on_round=chk,
                                 stale_reduce=mode)
                for (k, i), rec in tr.rec.items():
                    # the count rule of Fig. alg4 is about what is usable; NEW_ONLY may reduce fewer when s > 0
                    assert len(rec) >= (len(n_in[i]) - b if (mode == op.REUSE or s == 0) else 1)
                    assert all(k - s <= v <= k for _, v, _ in rec)


# ------------------------------------------------------------------ skipping iterations
def test_skipping_invariants_and_progress():
    n_in = inputs.ring_based(8)
    N, iters, s, max_ig = 8, 40, 3, 3
    ticks = np.ones((N, iters), np.uint64)
    ticks[2, :] = 4                                                # deterministic straggler (Section 7.3.5)
    for max_skip in (1, 2, 4):
        planned = []

        def chk(p):
            assert op.token_identity_holds(p)                      # (k - k0) tokens moved each way
            for i in range(N):
                if p.phase[i] == op._JUMPRECV:
                    outs = [j for j in p.n_out[i] if j != i]
                    # never jump past the slowest out-neighbour (Section 5: max_jump - max_ig)
                    assert p.jump_to[i] <= min(p.Iter[j] for j in outs)
                    assert 2 <= p.jump_to[i] - p.Iter[i] <= max_skip + 1
                    planned.append((i, p.Iter[i], p.jump_to[i]))
        tr = op.simulate(n_in, ticks, iters, s=s, max_ig=max_ig, max_skip=max_skip,
                         weight_mode=op.STALE_LINEAR, on_round=chk)
        base = op.simulate(n_in, ticks, iters, s=s, max_ig=max_ig, max_skip=0, weight_mode=op.STALE_LINEAR)
        assert planned and all(i == 2 for i, _, _ in planned)      # only the straggler identifies itself
        assert tr.makespan < base.makespan                         # others advance faster
        A = tr.to_arrays()
        for (i, k0, k) in set(planned):
            assert A["op"][k - 1, i] == op.JUMP
            assert all(A["op"][lv, i] == op.IDLE for lv in range(k0 + 1, k - 1))
            rec = tr.rec[(k - 1, i)]
            own = [r for r in rec if r[0] == i]
            assert own == [(i, k0 + 1, s + 1)]                     # own parameters, weighted as iteration k-1
            assert all((k - 1) - s <= v <= k - 1 for j, v, _ in rec if j != i)
        # skipped iterations are never consumed by anyone
        skipped = {(i, v) for (i, k0, k) in planned for v in range(k0 + 1, k)}
        for (k, i), rec in tr.rec.items():
            for (j, v, _) in rec:
                if j != i:
                    assert (j, v) not in skipped


def test_skipping_needs_token_queues_and_stays_off_by_default():
    n_in = inputs.ring(4)
    ticks = np.ones((4, 6), np.uint64)
    ticks[1, :] = 5
    with pytest.raises(ValueError):
        op.simulate(n_in, ticks, 6, s=1, max_ig=None, max_skip=1)
    tr = op.simulate(n_in, ticks, 6, s=1, max_ig=1)
    assert (tr.op == op.NORMAL).all()


# ------------------------------------------------------------------ reductions to the standard algorithm
def test_equal_speeds_reduce_to_standard_algorithm():
    for name, n_in in GRAPHS:
        N = len(n_in)
        for (s, b, max_ig) in [(0, 0, None), (2, 0, 2), (0, 1, 1), (1, 1, 3)]:
            if any(b >= len(nb) for nb in n_in):
                continue
            tr = op.simulate(n_in, np.full((N, 5), 3, np.uint64), 5, s=s, b=b, max_ig=max_ig,
                             weight_mode=op.STALE_LINEAR)
            for (k, i), rec in tr.rec.items():
                assert [(j, v) for j, v, _ in rec] == [(j, k) for j in n_in[i]]   # Fig. alg0: all of iteration k
                assert len(set(w for _, _, w in rec)) == 1                         # Eq. 2 == Eq. 1 here
            assert tr.makespan == 15


def test_weights_closed_forms():
    nums, den = op.reduce_weights([7, 7, 7], 7, 3, op.UNIFORM)
    assert (nums, den) == ([1, 1, 1], 3)                                           # Eq. 1: 1/|N_in|
    nums, den = op.reduce_weights([7, 6, 4, 5], 7, 3, op.STALE_LINEAR)
    assert (nums, den) == ([4, 3, 1, 2], 10)                                       # Eq. 2, k - s = 4
    for s in range(5):
        nums, den = op.reduce_weights([9] * 4, 9, s, op.STALE_LINEAR)
        assert all(n * 4 == den for n in nums)                                     # all fresh -> uniform


def test_rejects_bad_graphs():
    with pytest.raises(ValueError):
        op.simulate([[1], [0, 1]], np.ones((2, 2), np.uint64), 2)
    with pytest.raises(ValueError):
        op.simulate(inputs.ring(4), np.ones((4, 2), np.uint64), 2, b=3)


def test_deadlock_is_reported():
    class NoTokens(op.HopProtocol):
        def _tokens_available(self, i, n):
            return False
    with pytest.raises(op.Deadlock):
        NoTokens(inputs.ring(4), np.ones((4, 3), np.uint64), 3, max_ig=1).run()


def test_exact_backup_keeps_own_update_and_earliest_senders():
    # worker 0 listens to 1, 2, 3 (and itself), b = 2: it keeps its own update and ONE neighbour, the one whose
    # update of the iteration arrived first in its queue.  Senders enter iteration 1 at ticks 2, 5, 3.
    n_in = [[0, 1, 2, 3], [1], [2], [3]]
    ticks = np.array([[9, 1], [2, 1], [5, 1], [3, 1]], np.uint64)
    tr = op.simulate(n_in, ticks, 2, s=0, b=[2, 0, 0, 0], max_ig=None, backup_exact=True)
    assert [(j, v) for j, v, _ in tr.rec[(0, 0)]] == [(0, 0), (1, 0)]           # all sent iteration 0 at tick 0: ties by id
    assert [(j, v) for j, v, _ in tr.rec[(1, 0)]] == [(0, 1), (1, 1)]           # worker 1 entered iteration 1 first
    assert tr.den[(1, 0)] == 2
    loose = op.simulate(n_in, ticks, 2, s=0, b=[2, 0, 0, 0], max_ig=None)
    assert [j for j, _, _ in loose.rec[(1, 0)]] == [0, 1, 2, 3]                 # Fig. alg4 takes every available one
    # with staleness the kept neighbour's *newest* update is consumed, but the order is that of the first usable one
    tr = op.simulate(n_in, np.array([[9, 9], [2, 1], [1, 30], [3, 1]], np.uint64), 2, s=1, b=[2, 0, 0, 0], max_ig=None, backup_exact=True)
    assert [(j, v) for j, v, _ in tr.rec[(1, 0)]] == [(0, 1), (1, 1)]


@pytest.mark.parametrize("name,n_in", GRAPHS)
def test_notify_ack_gap_bounds_of_table1(name, n_in):
    # Table 1, row "Using NOTIFY-ACK": 1 towards in-neighbours, 2 towards out-neighbours,
    # min(dist(j->i), 2 dist(i->j)) for arbitrary pairs
    rng = np.random.default_rng(21)
    N = len(n_in)
    dist = op.shortest_paths(n_in)
    worst = [0]
    for trial in range(8):
        def chk(p):
            for i in range(N):
                for j in range(N):
                    if i != j:
                        assert p.Iter[i] - p.Iter[j] <= min(dist[j][i], 2 * dist[i][j])
                        if dist[i][j] == 1:
                            worst[0] = max(worst[0], p.Iter[i] - p.Iter[j])
        op.simulate(n_in, rand_ticks(rng, N, 12, 1, 30), 12, notify_ack=True, on_round=chk)
    if name == "cycle5":
        assert worst[0] == 2                                        # the bound of 2 is reached on a one-way edge


def test_notify_ack_prose_example_and_no_room_for_backup_workers():
    # Section 3.4: with NOTIFY-ACK, B and C are stuck in iteration 1 waiting for ACK(0) from A even though one
    # update would do (backup workers); with token queues they advance to max_ig.
    n_in = inputs.complete(3)
    ticks = np.ones((3, 10), np.uint64)
    ticks[0, 0] = STUCK
    top = [0, 0, 0]

    def chk(p):
        if p.now < STUCK:
            for i in range(3):
                top[i] = max(top[i], p.Iter[i])
    op.simulate(n_in, ticks, 10, s=0, b=1, notify_ack=True, on_round=chk)
    assert top == [0, 1, 1]
    top[:] = [0, 0, 0]
    op.simulate(n_in, ticks, 10, s=0, b=1, max_ig=4, on_round=chk)
    assert top == [0, 4, 4]


def test_notify_ack_chain_reaches_both_bounds_of_table1_exactly():
    # Section 3.3 / Table 1, row NOTIFY-ACK, on a chain 0 -> 1 -> 2 whose last worker never finishes its first Compute:
    # worker 1 reduces iterations 0 and 1 (ACKs both to worker 0) but cannot enter iteration 2 without ACK(0) from
    # worker 2; worker 0 enters 2 on ACK(0), 3 on ACK(1), and stops there: a sender exactly 2 ahead of its receiver,
    # a receiver exactly 1 ahead of its sender.
    n_in = [[0], [0, 1], [1, 2]]
    ticks = np.ones((3, 8), np.uint64)
    ticks[2, 0] = STUCK
    top = [0, 0, 0]

    def chk(p):
        if p.now < STUCK:
            for i in range(3):
                top[i] = max(top[i], p.Iter[i])
    op.simulate(n_in, ticks, 8, notify_ack=True, on_round=chk)
    assert top == [3, 1, 0]


@pytest.mark.parametrize("case,s,b,max_ig", [("a", 4, 0, 4), ("b", 4, 1, 5)])
def test_skipping_prose_examples_lead_then_as_much_again_after_the_jump(case, s, b, max_ig):
    """Section 5, the two examples of the skipping figure: three workers, A (worker 0) always slow.  Without skipping B and C
    get `lead` iterations ahead and wait; when A jumps to their iteration they run on for as many iterations again
    before A's next progress.  (a) the lead comes from the token queues of a staleness run (max_ig = s = 4);
    (b) from max_ig = 5 with one backup worker."""
    g = golden()
    lead, more = int(g[f"skip_example.{case}.lead"]), int(g[f"skip_example.{case}.more_after_jump"])
    if case == "b":
        assert max_ig == int(g["skip_example.b.max_ig"])
    slow = 1000
    ticks = np.ones((3, 40), np.uint64)
    ticks[0, :] = slow
    tops = {}

    def chk(p):
        w = int(p.now // slow)                      # which of A's computes is running
        tops[w] = max(tops.get(w, 0), p.Iter[1], p.Iter[2])
    no_skip = {}
    op.simulate(inputs.complete(3), ticks[:, :12], 12, s=s, b=b, max_ig=max_ig, max_skip=0, weight_mode=op.STALE_LINEAR,
                on_round=lambda p: no_skip.__setitem__(int(p.now // slow), max(no_skip.get(int(p.now // slow), 0), p.Iter[1])))
    assert no_skip[0] == lead and no_skip[1] == lead + 1      # dragged along: one more iteration per step of A
    tr = op.simulate(inputs.complete(3), ticks, 40, s=s, b=b, max_ig=max_ig, max_skip=s + 1, weight_mode=op.STALE_LINEAR, on_round=chk)
    assert tops[0] == lead                                      # before A's first step: the bounded lead
    assert tops[1] == lead + more                               # A jumped to their iteration: as many iterations again
    assert tops[2] == lead + 2 * more
    jumps = [(k, i) for k in range(40) for i in range(3) if tr.op[k, i] == op.JUMP]
    assert jumps and all(i == 0 for _, i in jumps)
