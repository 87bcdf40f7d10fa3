"""Protocol study in simulated time (host only): how fast do iterations go under the paper's slowdowns?

    python -m paper_1902_01064_b200.study                  # iteration speed per protocol (no GPU)
    python -m paper_1902_01064_b200.study --reduce-set     # what the two readings of the Reduce set do to training (GPU)

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


def reduce_set_study(P=8192, iters=2000, cfg=2, lr=2.0):
    """What do the readings of the bounded-staleness Reduce set change in training?  (Needs a GPU: the levels run through
    the library.)  Configuration `cfg` (default 2: 16 workers, CSR hinge SVM, s = 2, one backup worker, random 5x
    slowdowns) with `P` features for `iters` iterations under {only updates that arrived since the previous Recv, every
    update inside the bound} x {Eq. 2 weights, plain mean} with learning rate `lr`; returns rows (reduce set, weights, mean hinge loss of the
    workers' average model over all shards, largest distance of a worker from that average, consumed entries per record)."""
    import torch
    w = inputs.make_workload(cfg, P=P, iters=iters)
    w.lr = lr                   # the configuration's own rate (0.05) barely moves the loss in a run this short
    sv = w.svm
    rows_total = w.N * sv.rows_per_worker
    nnz = sv.row_ptr[1] - sv.row_ptr[0]
    assert (np.diff(sv.row_ptr) == nnz).all()
    col = sv.col.reshape(rows_total, nnz)
    val = sv.val.reshape(rows_total, nnz).astype(np.float64)
    y = sv.y.reshape(rows_total).astype(np.float64)
    dev = torch.device("cuda", torch.cuda.current_device())
    data = [torch.from_numpy(a).to(dev) for a in (sv.row_ptr, sv.col, sv.val, sv.y)]
    out = []
    for reduce_name, reduce in (("since previous Recv", hop.STALE_NEW_ONLY), ("all inside the bound", hop.STALE_REUSE)):
        for weight_name, mode in (("Eq. 2", hop.W_STALE_LINEAR), ("plain mean", hop.W_UNIFORM)):
            X = torch.zeros((w.N, w.s + 1, w.P), dtype=torch.float32, device=dev)
            h = hop.from_workload(w)
            h.set_option(hop.OPT_STALE_REDUCE, reduce)
            h.set_option(hop.OPT_WEIGHT_MODE, mode)
            h.bind_buffers(X, None, None, torch.cuda.current_stream().cuda_stream)
            h.bind_svm_csr(*data, sv.rows_per_worker, sv.batch)
            trace = h.sim_run(w.ticks, w.iters)
            entries = trace.dims()[2] / max(1, int((trace.to_arrays()["op"] != hop.OP_IDLE).sum()))
            h.load_trace(trace)
            h.write_params(-1, 0, w.p0())
            for _ in range(w.iters):
                h.step()
            if h.read_status() != 0:
                raise RuntimeError("device status")
            xs = np.stack([h.read_params(i) for i in range(w.N)]).astype(np.float64)
            h.close()
            mean = xs.mean(axis=0)
            margins = (val * mean[col]).sum(axis=1)
            loss = float(np.maximum(0.0, 1.0 - y * margins).mean())
            out.append((reduce_name, weight_name, loss, float(np.abs(xs - mean).max()), entries))
    return out


def main():
    import sys
    if "--reduce-set" in sys.argv:
        print(f"{'Reduce set':22s} {'weights':11s} {'hinge loss':>11s} {'max |x_i - mean|':>17s} {'entries/record':>15s}")
        for r, wname, loss, spread, entries in reduce_set_study():
            print(f"{r:22s} {wname:11s} {loss:11.4f} {spread:17.3e} {entries:15.2f}")
        return
    rows = run()
    print(f"{'graph':12s} {'slowdown':14s} {'protocol':26s} {'iter/time':>10s} {'vs standard':>12s} {'jumps':>6s}")
    for g, t, s, speed, jumps, rel in rows:
        print(f"{g:12s} {t:14s} {s:26s} {speed:10.3f} {rel:12.2f} {jumps:6d}")
    print("paper (CPU cluster, VGG11): backup workers up to 1.81x iteration speed under the random 6x slowdown (Section 7.3.3);"
          " a 4x straggler slows iterations 3.9x without and 1.1x with skipping (Section 7.3.5)")


if __name__ == "__main__":
    main()
