"""Oracle, part 1: the Hop queue protocol, tick by tick (TEST INFRASTRUCTURE ONLY).

Follows the paper's worker loop literally:
  * Train() of Fig. alg2 (token insert -> Send -> Compute -> Recv -> Reduce -> Apply ->
    token acquire), with the update queue and its tagged enqueue / dequeue / size of
    Section 4.1, the token queues of Section 4.2 (max_ig - 1 initial tokens plus one per
    entered iteration), Recv of Fig. alg4 (backup workers) and of Fig. alg3 (bounded
    staleness), the Reduce weights of Fig. alg4 (plain mean) and Eq. 2, and the skipping
    rule of Section 5.
  * Every worker is a little state machine; simulated time is an integer tick counter.

Readings taken where the paper is silent (listed once more in the design notes):
  R1  Compute of (i, k) lasts ticks[i][k] >= 1 ticks; every other operation lasts 0 ticks and
      a sent update is visible at once.
  R2  At level k a worker may take from in-neighbour j the newest update of j with
      iter <= k (Section 6: one queue per iteration slot keeps newer iterations out of
      reach); it is satisfactory iff iter >= k - s.  The newest update seen so far from j
      is remembered (Fig. alg3 iter_rcv; Section 4.4: an earlier update still inside the bound
      needs no new arrival, so it never blocks the worker).
  R2' Which satisfactory updates enter the Reduce (stale_reduce).  NEW_ONLY, the default, is what
      the paper prints three times: Eq. 2 sums over the in-neighbours whose update received in
      iteration k is satisfactory, Fig. alg3's Recv appends an update only when the newest
      iteration among what this call dequeued is inside the bound, and Section 4.4 reduces what
      has arrived since the last Reduce.  An in-neighbour whose newest update was already taken out of the
      queue by an earlier Recv of this worker still counts for the blocking test but adds no
      term; the own update is new in every iteration.  REUSE adds such an update again, with the
      lower weight Eq. 2 gives its age (every satisfactory in-neighbour contributes at every
      level).
  R3  Recv(k, i) completes at the first moment at least |N_in(i)| - b_i in-neighbours (self
      included) are satisfactory, and then takes every satisfactory one (Fig. alg4: the
      required number, then whatever else is there), subject to R2'.  b = 0 is Fig. alg3, s = 0 is
      Fig. alg4 (an update of iteration k is first dequeued by Recv(k), so R2' changes nothing
      there), both 0 is Fig. alg1; both > 0 is the "hybrid" row of Table 1.
  R3' serial=True is the serial approach of Section 3.2 (Compute, Apply, Send, Recv, Reduce): the update of
      iteration k is enqueued when Compute(k) ends, not when the iteration is entered; tokens are still inserted
      at the start of the iteration (Fig. alg2).  The default is the parallel approach the paper adopts.
  R4  Same-tick ordering: rounds.  In a round every worker decides its transition from the
      state left by the previous round; then all decisions are committed in worker order.
      One transition per worker per round; rounds repeat until nothing moves.
  R5  Skipping (max_skip > 0): a worker that has applied iteration k0 and attempts to enter
      k0+1 reads its out-neighbours' token counts (Section 5); behind = min_j size(TokenQ(j->i))
      - max_ig - 1 = min_j Iter(j) - (k0+1).  If behind >= 1 it jumps to
      k = k0 + 1 + min(behind, max_skip, last - (k0+1)): it first completes Recv(k-1) under
      R2/R3, its own current parameters x_{k0+1,i} standing in for its update of iteration
      k-1, and Reduces (a JUMP record at level k-1), then moves k-k0 tokens each way and enters
      k.  Levels k0+1 .. k-2 are IDLE; its updates k0+1 .. k-1 are never sent.
  R6  A worker that applied its last iteration stops (no token acquire after it).
  R8  notify_ack=True replaces the token queues by the NOTIFY-ACK scheme of Section 3.3 (prior work, the paper's
      baseline): after the Reduce of iteration k a worker sends ACK(k) to its in-neighbours, and a worker enters
      iteration k+1 only with ACK(k-1) from every out-neighbour.  That is the reading that reproduces the bounds
      the paper states for it (Table 1: a receiver at most 1 ahead of its sender, a sender at most 2 ahead of its
      receiver) and the Section 3.4 example (B and C stuck in iteration 1 waiting for ACK(0)); the Section 3.5
      remark that they could not even enter iteration 1 is at odds with both and is not followed.
  R7  backup_exact (off by default; Fig. alg4 takes the required number, then whatever else is queued): Recv completes at the
      same moment as under R3 but keeps exactly |N_in(i)| - b_i updates: its own, plus those in-neighbours
      whose first satisfactory update (iter in [k-s, k]) arrived earliest in UpdateQ(i) (FIFO order of
      Fig. alg4's dequeue); the version taken from a kept neighbour is still its newest one with iter <= k.
      Under NEW_ONLY the kept set is chosen first and R2' then drops the kept ones that are not new.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

IDLE, NORMAL, JUMP = 0, 1, 2
UNIFORM, STALE_LINEAR = 0, 1
NEW_ONLY, REUSE = 0, 1

_COMPUTE, _RECV, _TOKEN, _JUMPRECV, _DONE = range(5)


class Deadlock(RuntimeError):
    pass


@dataclass
class Trace:
    """Consumption trace: for every (level k, worker i) an op and the list of consumed
    (in-neighbour, version, weight numerator) with a common weight denominator."""
    N: int
    levels: int
    op: np.ndarray                                   # [levels][N]
    rec: dict = field(default_factory=dict)          # (k, i) -> [(nbr, ver, num), ...]
    den: dict = field(default_factory=dict)          # (k, i) -> int
    makespan: int = 0

    def to_arrays(self):
        ptr = [0]
        nbr, ver, num = [], [], []
        den = np.zeros((self.levels, self.N), np.int32)
        for k in range(self.levels):
            for i in range(self.N):
                for (j, v, w) in self.rec.get((k, i), ()):
                    nbr.append(j)
                    ver.append(v)
                    num.append(w)
                ptr.append(len(nbr))
                den[k, i] = self.den.get((k, i), 0)
        return dict(op=self.op.astype(np.int32), ptr=np.asarray(ptr, np.int64),
                    nbr=np.asarray(nbr, np.int32), ver=np.asarray(ver, np.int32),
                    num=np.asarray(num, np.int32), den=den)


def reduce_weights(vers, level, s, weight_mode):
    """Integer weight numerators and their sum.  UNIFORM: Fig. alg4 Reduce (plain mean over
    what was received).  STALE_LINEAR: Eq. 2, numerator Iter(u) - (k - s) + 1."""
    if weight_mode == UNIFORM:
        nums = [1 for _ in vers]
    else:
        nums = [v - (level - s) + 1 for v in vers]
    return nums, sum(nums)


class HopProtocol:
    def __init__(self, n_in, ticks, iters, s=0, b=0, max_ig=None, max_skip=0,
                 weight_mode=UNIFORM, on_round=None, backup_exact=False, notify_ack=False,
                 stale_reduce=NEW_ONLY, serial=False):
        self.N = N = len(n_in)
        self.serial = serial
        self.n_in = [list(nb) for nb in n_in]
        for i, nb in enumerate(self.n_in):
            if i not in nb:
                raise ValueError("every node needs a self-loop (Section 3.1)")
        self.n_out = [[] for _ in range(N)]
        for i, nb in enumerate(self.n_in):
            for j in nb:
                self.n_out[j].append(i)
        self.ticks = ticks
        self.iters = iters
        self.s = s
        self.b = [b] * N if np.isscalar(b) else list(b)
        for i in range(N):
            if not (0 <= self.b[i] < len(self.n_in[i])):
                raise ValueError("N_buw(i) < |N_in(i)| required (Fig. alg4)")
        self.max_ig = max_ig
        self.max_skip = max_skip
        if max_skip > 0 and max_ig is None:
            raise ValueError("skipping reads token counts: token queues required")
        self.weight_mode = weight_mode
        self.on_round = on_round
        # ---- literal queues
        self.notify_ack = notify_ack
        if notify_ack and (max_ig is not None or max_skip > 0):
            raise ValueError("NOTIFY-ACK replaces the token queues (max_ig=None) and has no skipping")
        self.acks = {(j, i): [] for i in range(N) for j in self.n_out[i] if j != i}   # ACKs from j received at i
        self.backup_exact = backup_exact
        self.arrivals = [0] * N                                # entries ever enqueued into UpdateQ(i)
        self.arrival_pos = {}                                  # (w_id, i) -> {iter: position in UpdateQ(i)'s arrival order}
        self.update_q = [[] for _ in range(N)]                 # FIFO of (iter, w_id) tags
        self.iter_rcv = {(j, i): -1 for i in range(N) for j in self.n_in[i]}
        self.stale_reduce = stale_reduce
        # iter_rcv as it stood when worker i last completed a Recv: what that call (or an earlier one) dequeued
        self.iter_reduced = {(j, i): -1 for i in range(N) for j in self.n_in[i]}
        self.token_q = {}
        if max_ig is not None:
            for i in range(N):
                for j in self.n_in[i]:
                    if j != i:
                        self.token_q[(i, j)] = [0] * (max_ig - 1)   # TokenQ(i -> j), kept at i
        self.Iter = [0] * N
        self.phase = [_COMPUTE] * N
        self.end = [0] * N
        self.jump_to = [0] * N
        self.now = 0
        self.trace = Trace(N, iters, np.zeros((iters, N), np.int32))

    # ---------------------------------------------------------------- paper operations
    def _send(self, i, k):
        for j in self.n_out[i]:
            self.update_q[j].append((k, i))                     # UpdateQ(j).enqueue(x_{k,i}, iter=k, w_id=i)
            self.arrival_pos.setdefault((i, j), {})[k] = self.arrivals[j]
            self.arrivals[j] += 1

    def _enter(self, i, k, n_tokens=1):
        """Start of iteration k at worker i (Fig. alg2): insert tokens, Send (parallel approach), start Compute."""
        if self.max_ig is not None:
            for j in self.n_in[i]:
                if j != i:
                    self.token_q[(i, j)].extend([k] * n_tokens)
        if not self.serial:
            self._send(i, k)
        self.Iter[i] = k
        self.phase[i] = _COMPUTE
        self.end[i] = self.now + int(self.ticks[i][k])

    def _drain(self, i, level):
        """Take every queued update with iter <= level out of UpdateQ(i), remembering per
        sender the newest iteration seen (Fig. alg3 iter_rcv; Section 6, one pass per w_id)."""
        keep = []
        for (it, w) in self.update_q[i]:
            if it <= level:
                if it > self.iter_rcv[(w, i)]:
                    self.iter_rcv[(w, i)] = it
            else:
                keep.append((it, w))
        self.update_q[i] = keep

    def _try_recv(self, i, level, own_version=None):
        """Recv(level, i).  Returns the consumed [(nbr, ver)] or None while it must block."""
        self._drain(i, level)
        got = []
        for j in self.n_in[i]:
            if j == i and own_version is not None:
                got.append((j, own_version))                     # jumper's current parameters
            elif self.iter_rcv[(j, i)] >= max(level - self.s, 0):         # -1: nothing received from j yet (Fig. alg3)
                got.append((j, self.iter_rcv[(j, i)]))
        need = len(self.n_in[i]) - self.b[i]
        if len(got) < need:
            return None
        if self.backup_exact and len(got) > need:
            def first_satisfactory_arrival(j):
                seen = self.arrival_pos[(j, i)]
                return min(seen[it] for it in range(level - self.s, level + 1) if it in seen)
            others = sorted((jv for jv in got if jv[0] != i), key=lambda jv: (first_satisfactory_arrival(jv[0]), jv[0]))
            keep = {i} | {j for j, _ in others[:need - 1]}
            got = [jv for jv in got if jv[0] in keep]
        if self.stale_reduce == NEW_ONLY:
            # Fig. alg3: only what this Recv call itself dequeued is appended (max(l_iter) >= min_iter)
            got = [(j, v) for (j, v) in got if j == i or v > self.iter_reduced[(j, i)]]
        return got

    def _recv_done(self, i):
        """Recv of worker i returned: everything it dequeued, used or not, is gone from the queue."""
        for j in self.n_in[i]:
            self.iter_reduced[(j, i)] = self.iter_rcv[(j, i)]

    def _record(self, op, level, i, got, own_as=None):
        vers = [(own_as if (j == i and own_as is not None) else v) for (j, v) in got]
        nums, den = reduce_weights(vers, level, self.s, self.weight_mode)
        self.trace.op[level, i] = op
        self.trace.rec[(level, i)] = [(j, v, w) for (j, v), w in zip(got, nums)]
        self.trace.den[(level, i)] = den

    def _tokens_available(self, i, n):
        if self.notify_ack:                                       # ACK(k-1) from every out-neighbour
            k = self.Iter[i]
            return k - 1 < 0 or all((k - 1) in self.acks[(j, i)] for j in self.n_out[i] if j != i)
        if self.max_ig is None:
            return True
        return all(len(self.token_q[(j, i)]) >= n for j in self.n_out[i] if j != i)

    def _take_tokens(self, i, n):
        if self.max_ig is None:
            return
        for j in self.n_out[i]:
            if j != i:
                q = self.token_q[(j, i)]
                assert len(q) >= n
                del q[:n]                                        # TokenQ(j -> i).dequeue(n)

    # ---------------------------------------------------------------- one round
    def _decide(self, i):
        ph = self.phase[i]
        k = self.Iter[i]
        if ph == _RECV:
            got = self._try_recv(i, k)
            if got is not None:
                return ("applied", got)
        elif ph == _TOKEN:
            outs = [j for j in self.n_out[i] if j != i]
            if self.max_skip > 0 and outs:
                behind = min(len(self.token_q[(j, i)]) for j in outs) - self.max_ig - 1
                skip = min(behind, self.max_skip, (self.iters - 1) - (k + 1))
                if behind >= 1 and skip >= 1:
                    return ("plan_jump", k + 1 + skip)
            if self._tokens_available(i, 1):
                return ("enter", k + 1)
        elif ph == _JUMPRECV:
            target = self.jump_to[i]
            got = self._try_recv(i, target - 1, own_version=k + 1)
            if got is not None:
                return ("jump", target, got)
        return None

    def _commit(self, i, act):
        k = self.Iter[i]
        if act[0] == "applied":
            self._record(NORMAL, k, i, act[1])
            self._recv_done(i)
            if self.notify_ack:
                for j in self.n_in[i]:
                    if j != i:
                        self.acks[(i, j)].append(k)              # ACK(k) after the Reduce, to every in-neighbour
            self.phase[i] = _DONE if k == self.iters - 1 else _TOKEN
        elif act[0] == "enter":
            self._take_tokens(i, 1)
            self._enter(i, act[1])
        elif act[0] == "plan_jump":
            self.jump_to[i] = act[1]
            self.phase[i] = _JUMPRECV                            # levels k+1 .. target-2 stay IDLE
        elif act[0] == "jump":
            target, got = act[1], act[2]
            self._record(JUMP, target - 1, i, got, own_as=target - 1)
            self._recv_done(i)
            self._take_tokens(i, target - k)
            self._enter(i, target, n_tokens=target - k)

    def run(self):
        for i in range(self.N):
            self._enter(i, 0)
        while True:
            computing = [i for i in range(self.N) if self.phase[i] == _COMPUTE]
            if not computing:
                if all(p == _DONE for p in self.phase):
                    break
                raise Deadlock(f"no worker can move at tick {self.now}: Iter={self.Iter}")
            self.now = min(self.end[i] for i in computing)
            for i in computing:
                if self.end[i] == self.now:
                    if self.serial:
                        self._send(i, self.Iter[i])               # Compute, Apply, then Send (Section 3.2)
                    self.phase[i] = _RECV
            while True:
                acts = [(i, self._decide(i)) for i in range(self.N)]
                acts = [(i, a) for (i, a) in acts if a is not None]
                if not acts:
                    break
                for i, a in acts:
                    self._commit(i, a)
                if self.on_round is not None:
                    self.on_round(self)
        self.trace.makespan = self.now
        return self.trace


def simulate(n_in, ticks, iters, s=0, b=0, max_ig=None, max_skip=0, weight_mode=UNIFORM, on_round=None,
             backup_exact=False, notify_ack=False, stale_reduce=NEW_ONLY, serial=False):
    return HopProtocol(n_in, ticks, iters, s, b, max_ig, max_skip, weight_mode, on_round, backup_exact, notify_ack,
                       stale_reduce, serial).run()


# -------------------------------------------------------------------- graph helpers for the invariants
def shortest_paths(n_in):
    """dist[a][b] = length of the shortest directed path a -> b (edge (j, i) for j in N_in(i))."""
    N = len(n_in)
    INF = 10 ** 9
    n_out = [[] for _ in range(N)]
    for i, nb in enumerate(n_in):
        for j in nb:
            if j != i:
                n_out[j].append(i)
    dist = [[INF] * N for _ in range(N)]
    for a in range(N):
        dist[a][a] = 0
        frontier = [a]
        while frontier:
            nxt = []
            for u in frontier:
                for v in n_out[u]:
                    if dist[a][v] == INF:
                        dist[a][v] = dist[a][u] + 1
                        nxt.append(v)
            frontier = nxt
    return dist


def token_identity_holds(p: HopProtocol) -> bool:
    """Section 4.2 proof: TokenQ(j -> i).size() == Iter(j) - Iter(i) + max_ig for every edge i -> j."""
    for (j, i), q in p.token_q.items():
        if len(q) != p.Iter[j] - p.Iter[i] + p.max_ig:
            return False
    return True
