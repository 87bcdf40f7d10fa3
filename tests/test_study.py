"""The protocol study (simulated time, host only) runs and shows the effects the paper reports, qualitatively."""
from paper_1902_01064_b200 import study


def test_protocol_study_orders_protocols_like_the_paper():
    rows = {(g, t, s): (speed, rel) for g, t, s, speed, jumps, rel in study.run(iters=200)}
    for g in ("ring", "ring-based", "double-ring"):
        rnd, det = "6x w.p. 1/n", "one worker 4x"
        # random slowdown: backup workers and staleness beat standard training (Sections 7.3.3, 7.3.4)
        assert rows[(g, rnd, "backup b=1, max_ig=4")][1] > 1.15
        assert rows[(g, rnd, "staleness s=5")][1] > 1.15
        # NOTIFY-ACK never beats the token-queue protocol
        assert rows[(g, rnd, "NOTIFY-ACK")][0] <= rows[(g, rnd, "standard")][0] + 1e-12
        # deterministic straggler: neither helps (Section 5), skipping does (Section 7.3.5: 3.9x -> 1.1x)
        assert abs(rows[(g, det, "standard")][0] - 0.25) < 0.01
        assert abs(rows[(g, det, "backup b=1, max_ig=4")][1] - 1.0) < 0.02
        assert rows[(g, det, "staleness s=9 + skip<=10")][0] > 0.9
