"""The shared library loads, exports every symbol include/hop.h declares, and its host-side
checks reject bad graphs and bad traces.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1902_01064_b200 import hop, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hop_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    syms = declared_symbols()
    assert len(syms) >= 20
    lib = ctypes.CDLL(hop.LIB_PATH)
    for s in syms:
        assert hasattr(lib, s), s
        assert s in hop.SIGNATURES, f"{s} has no Python binding"
    assert sorted(hop.SIGNATURES) == syms


def test_create_rejects_bad_graphs():
    ptr, idx = inputs.graph_to_csr(inputs.ring(4))
    with pytest.raises(hop.HopError) as e:
        hop.Hop(ptr, idx, 4, 16, 1, 3, 0)                # b >= |N_in|
    assert e.value.code == hop.E_GRAPH
    with pytest.raises(hop.HopError) as e:
        hop.Hop(ptr, idx, 4, 16, 1, 0, 3)                # max_skip > s + 1
    assert e.value.code == hop.E_GRAPH
    bad_ptr, bad_idx = np.array([0, 1, 3], np.int32), np.array([1, 0, 1], np.int32)
    with pytest.raises(hop.HopError) as e:
        hop.Hop(bad_ptr, bad_idx, 2, 16, 0, 0, 0)        # worker 0 has no self-loop
    assert e.value.code == hop.E_GRAPH and "self-loop" in str(e.value)
    with pytest.raises(hop.HopError):
        hop.Hop(ptr, idx, 4, 0, 0, 0, 0)                 # P = 0


def test_options_are_validated():
    ptr, idx = inputs.graph_to_csr(inputs.ring(4))
    h = hop.Hop(ptr, idx, 4, 16, 1, 0, 0)
    for key, val in [(hop.OPT_MAX_IG, -1), (hop.OPT_WEIGHT_MODE, 7), (hop.OPT_GRAD_MODE, 9), (hop.OPT_COL_OFFSET, 6),
                     (hop.OPT_BACKUP_OF_WORKER + 1, 3), (hop.OPT_BACKUP_OF_WORKER + 9, 0), (77, 1),
                     (hop.OPT_LR, float("nan")), (hop.OPT_GRAD_SIGMA, float("inf"))]:
        with pytest.raises(hop.HopError):
            h.set_option(key, val)
    h.set_option(hop.OPT_BACKUP_OF_WORKER + 2, 2)
    with pytest.raises(hop.HopError) as e:
        h.sim_run(np.zeros((4, 3), np.uint64), 3)        # zero-length compute
    assert e.value.code == hop.E_ARG
    with pytest.raises(hop.HopError) as e:
        h.step()                                         # nothing bound
    assert e.value.code == hop.E_STATE


def test_per_worker_backup_matches_oracle():
    from oracle import protocol as op
    n_in = inputs.ring_chords(8, 3)
    ptr, idx = inputs.graph_to_csr(n_in)
    h = hop.Hop(ptr, idx, 8, 16, 1, 0, 0)
    b = [0, 1, 2, 0, 3, 1, 0, 2]
    for i, bi in enumerate(b):
        h.set_option(hop.OPT_BACKUP_OF_WORKER + i, bi)
    h.set_option(hop.OPT_MAX_IG, 2)
    rng = np.random.default_rng(0)
    ticks = rng.integers(1, 30, size=(8, 20)).astype(np.uint64)
    got = h.sim_run(ticks, 20).to_arrays()
    want = op.simulate(n_in, ticks, 20, 1, b, 2, 0, op.UNIFORM).to_arrays()
    for k in ("op", "ptr", "nbr", "ver", "num", "den"):
        assert np.array_equal(got[k], want[k])


def test_trace_roundtrip():
    w = inputs.make_workload(3, P=64, iters=30)
    h = hop.from_workload(w)
    a = h.sim_run(w.ticks, w.iters).to_arrays()
    t2 = hop.Trace.from_arrays(a["op"], a["ptr"], a["nbr"], a["ver"], a["num"], a["den"])
    b = t2.to_arrays()
    for k in ("op", "ptr", "nbr", "ver", "num", "den"):
        assert np.array_equal(a[k], b[k])
    assert t2.dims()[:3] == (30, 32, len(a["nbr"]))


def test_python_constants_match_the_header():
    """hop.py repeats the header's enumerators by hand: they must not drift apart."""
    text = open(os.path.join(ROOT, "include", "hop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    enums = {name: int(val) for name, val in re.findall(r"\b(HOP_[A-Z0-9_]+)\s*=\s*(-?\d+)", text)}
    assert len(enums) > 45
    missing = []
    for name, val in enums.items():
        py = name[len("HOP_"):]
        if not hasattr(hop, py):
            missing.append(name)
            continue
        assert getattr(hop, py) == val, name
    assert not missing, missing
    assert hop.STATIC_MAX_ROWS == int(re.search(r"#define HOP_STATIC_MAX_ROWS (\d+)", text).group(1))
