"""The bounds-checked build of the library (the sanitizer's place on this path): the same parity cases run through it
with every global-memory source of the mix kernels' copies and every CSR gather / atomic tested against the bound buffers
first, and must finish with a clean status word; a column index outside the ring is refused and reported, not accessed."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_1902_01064_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _env():
    lib = build.build(checked=True)
    return dict(os.environ, HOP_B200_LIBRARY=lib)


def test_parity_cases_pass_through_the_checked_build_with_a_clean_status():
    select = ("cfg1 or cfg2_reduced or cfg3_reduced or cfg4_reduced or cfg5_reduced or tiny or unaligned or hazard or "
              "jump_records or csr_svm_variants or streaming_levels or no_kernel_writes")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-m", "gpu", "-x", "-q",
                        "-k", select], capture_output=True, text=True, timeout=1500, cwd=ROOT, env=_env())
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


def test_an_index_outside_the_bound_buffers_is_refused_and_reported():
    script = textwrap.dedent("""
        import numpy as np, torch
        from paper_1902_01064_b200 import hop, inputs
        assert hop.build_is_checked(), "this input must only ever reach the checked build"
        w = inputs.make_workload(2, P=4096, iters=3)
        S = w.s + 1
        w.svm.col[7] = w.N * S * w.P + 1000                  # far past the end of the ring, for every worker's slot
        X = torch.zeros((w.N, S, w.P), dtype=torch.float32, device="cuda:0")
        h = hop.from_workload(w)
        h.bind_buffers(X, None, None, torch.cuda.current_stream().cuda_stream)
        keep = [torch.from_numpy(a).to("cuda:0") for a in (w.svm.row_ptr, w.svm.col, w.svm.val, w.svm.y)]
        h.bind_svm_csr(*keep, w.svm.rows_per_worker, w.svm.batch)
        h.load_trace(h.sim_run(w.ticks, w.iters))
        h.write_params(-1, 0, w.p0())
        h.step()
        rc, word = h.read_status_word()
        assert rc == hop.E_DEVICE and word >> 24 == 4 and (word & 0xffffff) in (4, 5), (rc, word)
        h.clear_status()
        torch.cuda.synchronize()                             # no fault: the access was never made
        assert bool(torch.isfinite(X).all())
        print("refused and reported", word)
    """)
    r = subprocess.run([sys.executable, "-c", script], capture_output=True, text=True, timeout=600, cwd=ROOT, env=_env())
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-3000:]
    assert "refused and reported" in r.stdout
