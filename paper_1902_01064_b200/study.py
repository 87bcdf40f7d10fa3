"""Protocol study in simulated time (host only): how fast do iterations go under the paper's slowdowns?

    python -m paper_1902_01064_b200.study

Runs the C++ protocol simulator (hop_sim_run) on the paper's three 16-worker graphs (ring, ring-based,
double-ring; Section 7, Fig. "Graphs used in experiments") under its two heterogeneity models -- every worker
6x slower with probability 1/n in each iteration (Section 7.3.1), one worker always 4x slower (Section 7.3.5) --
for NOTIFY-ACK, standard decentralized training, backup workers, bounded staleness and skipping, and prints the
iteration speed (iterations per unit of compute time, averaged over workers) relative to standard training.
Only Compute takes time here (no network, no Reduce cost), so the numbers say what the *protocol* allows, not what
the paper's cluster measured; the paper's own figures (1.81x for one backup worker, a 4x straggler's effect on the
iteration duration cut from 3.9x to 1.1x by skipping) are printed beside them as context.
"""
from __future__ import annotations

import numpy as np

from . import hop, inputs

UNIT = 1 << 10


def iteration_speed(n_in, ticks, iters, s=0, b=0, max_ig=1, max_skip=0, notify_ack=False):
    """(mean executed iterations per worker) / makespan, in iterations per unit of compute time."""
    ptr, idx = inputs.graph_to_csr(n_in)
    h = hop.Hop(ptr, idx, len(n_in), 4, s, b, max_skip)
    h.set_option(hop.OPT_MAX_IG, max_ig)
    h.set_option(hop.OPT_NOTIFY_ACK, 1 if notify_ack else 0)
    tr = h.sim_run(ticks, iters).to_arrays()
    h.close()
    return iters / (tr["makespan"] / UNIT), int((tr["op"] == hop.OP_JUMP).sum())


def settings():
    return [("NOTIFY-ACK", dict(notify_ack=True)),
            ("standard", dict(max_ig=1)),
            ("backup b=1, max_ig=4", dict(b=1, max_ig=4)),
            ("staleness s=5", dict(s=5, max_ig=5)),
            ("backup b=1 + skip<=2", dict(s=1, b=1, max_ig=4, max_skip=2)),
            ("staleness s=9 + skip<=10", dict(s=9, max_ig=9, max_skip=10))]


def run(n=16, iters=400, seed=1902):
    graphs = [("ring", inputs.ring(n)), ("ring-based", inputs.ring_based(n)), ("double-ring", inputs.double_ring(n))]
    rng = np.random.default_rng(seed)
    random6 = np.where(rng.random((n, iters)) < 1.0 / n, 6, 1).astype(np.uint64) * UNIT
    straggler = np.ones((n, iters), np.uint64) * UNIT
    straggler[3, :] *= 4
    rows = []
    for gname, n_in in graphs:
        for tname, ticks in (("6x w.p. 1/n", random6), ("one worker 4x", straggler)):
            base = None
            for sname, kw in settings():
                speed, jumps = iteration_speed(n_in, ticks, iters, **kw)
                if sname == "standard":
                    base = speed
                rows.append((gname, tname, sname, speed, jumps))
            for k in range(len(rows) - len(settings()), len(rows)):
                rows[k] = rows[k] + (rows[k][3] / base,)
    return rows


def main():
    rows = run()
    print(f"{'graph':12s} {'slowdown':14s} {'protocol':26s} {'iter/time':>10s} {'vs standard':>12s} {'jumps':>6s}")
    for g, t, s, speed, jumps, rel in rows:
        print(f"{g:12s} {t:14s} {s:26s} {speed:10.3f} {rel:12.2f} {jumps:6d}")
    print("paper (CPU cluster, VGG11): backup workers up to 1.81x iteration speed under the random 6x slowdown (Section 7.3.3);"
          " a 4x straggler slows iterations 3.9x without and 1.1x with skipping (Section 7.3.5)")


if __name__ == "__main__":
    main()
