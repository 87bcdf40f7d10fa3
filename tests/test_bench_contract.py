"""The oracle arm of bench.py runs without a GPU: its JSON line must carry the keys the benchmark contract names."""
import json
import os
import subprocess
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "3",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "worker_iterations_per_s" and d["unit"] == "worker-iterations/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["data"] == "synthetic" and d["dtype"] == "f64"
    assert d["value"] > 0 and d["n_gpus"] == 1 and d["steps"] == 1 and d["warmup"] == 0
    assert d["config"]["workload"].startswith("config 3") and d["config"]["N"] == 32
    import bench
    from paper_1902_01064_b200 import inputs
    w = inputs.make_workload(3)
    assert d["config"] == bench.workload_config(3, w, w.P)          # the same object the GPU arm prints
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == 1 and cb["value"] == d["value"] and "columns" in cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_other_ranks_of_the_reference_arm_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_ncu_traffic_tables_cover_every_level_of_their_workloads():
    """roofline.traffic is summed over the levels the timed region ran: the per-level tables must have one value per level
    of the configuration's trace, be plausible against the algorithmic bytes of that level, and name the trace they
    were captured on."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import bench
    from paper_1902_01064_b200 import hop, inputs
    for cfg, cap in bench.NCU_LEVEL_TRAFFIC.items():
        w = inputs.make_workload(cfg, P=cap["P"])
        assert len(cap["bytes"]) == w.iters and cap["stale_reduce"] == w.stale_reduce
        h = hop.from_workload(w)
        t = h.sim_run(w.ticks, w.iters).to_arrays()
        h.close()
        for k in range(w.iters):
            lo, hi = t["ptr"][k * w.N], t["ptr"][(k + 1) * w.N]
            U = len(set(zip(t["nbr"][lo:hi].tolist(), t["ver"][lo:hi].tolist())))
            alg = 4 * cap["P"] * (U + int((t["op"][k] == 1).sum()) + int((t["op"][k] != 0).sum()))
            assert 0.9 < cap["bytes"][k] / alg < 1.05, (cfg, k, cap["bytes"][k] / alg)
