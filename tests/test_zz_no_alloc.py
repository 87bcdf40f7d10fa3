"""hop_svm_csr_sgd_static -- the entry point for callers that may not allocate device memory (code
running where cudaMalloc is forbidden or would stall the device, or under a fixed memory budget).
Its coefficient scratch is a fixed array inside the library, so the test checks that it gives the
same parameters as the ordinary path (hop_bind_svm_csr + hop_step, whose scratch is allocated), on
two calls in a row that share that array.  Collected last on purpose: a failure here cannot hide
another test's result in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

from paper_1902_01064_b200 import hop, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def csr_batch(rng, rows, P, nnz):
    col = np.stack([np.sort(rng.choice(P, nnz, replace=False)) for _ in range(rows)]).astype(np.int32)
    val = rng.lognormal(0, 1, (rows, nnz))
    val = (val / np.sqrt((val * val).sum(1, keepdims=True))).astype(np.float32)
    y = np.where(rng.random(rows) < 0.5, -1.0, 1.0).astype(np.float32)
    row_ptr = (np.arange(rows + 1) * nnz).astype(np.int64)
    return row_ptr, col.reshape(-1), val.reshape(-1), y


def ordinary_path(x0, row_ptr, col, val, y, rows, lr):
    """One worker with only its self-loop: Reduce is the identity, so hop_step is x <- x - lr * g."""
    P = x0.size
    X = torch.zeros((1, 1, P), dtype=torch.float32, device=DEV)
    h = hop.Hop(np.array([0, 1], np.int32), np.array([0], np.int32), 1, P, 0, 0, 0)
    h.set_option(hop.OPT_LR, lr)
    h.set_option(hop.OPT_GRAD_MODE, hop.GRAD_SVM_CSR)
    h.bind_buffers(X, None, None, torch.cuda.current_stream().cuda_stream)
    dev = [torch.from_numpy(a).to(DEV) for a in (row_ptr, col, val, y)]
    h.bind_svm_csr(*dev, rows, rows)
    h.load_trace(h.sim_run(np.ones((1, 1), np.uint64), 1))
    h.write_params(0, 0, x0)
    h.step()
    assert h.read_status() == 0
    out = h.read_params(0)
    h.close()
    return out


def static_path(x0, row_ptr, col, val, y, rows, lr):
    x = torch.from_numpy(x0).to(DEV)
    x_out = x.clone()
    dev = [torch.from_numpy(a).to(DEV) for a in (row_ptr, col, val, y)]
    torch.cuda.synchronize()
    hop.svm_csr_sgd_static(x, x_out, x0.size, *dev, rows, lr, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return x_out.cpu().numpy()


def test_static_scratch_entry_matches_ordinary_path_twice_in_a_row():
    rng = np.random.default_rng(2024)
    P = 50000
    # the second call uses fewer rows than the first: stale coefficients of the first call stay in the
    # shared array beyond its rows and must not leak into the result
    for rows, nnz, lr in [(384, 60, 0.05), (130, 100, 0.2)]:
        x0 = (rng.standard_normal(P) * 2.0).astype(np.float32)
        batch = csr_batch(rng, rows, P, nnz)
        want = ordinary_path(x0, *batch, rows, lr)
        got = static_path(x0, *batch, rows, lr)
        assert np.abs(want - x0).max() > 0                          # the step did something
        assert np.abs(got - want).max() <= 1e-6 * np.abs(want).max()


def test_static_scratch_entry_rejects_oversized_minibatches():
    x = torch.zeros(8, dtype=torch.float32, device=DEV)
    rp = torch.zeros(hop.STATIC_MAX_ROWS + 2, dtype=torch.int64, device=DEV)
    col = torch.zeros(1, dtype=torch.int32, device=DEV)
    val = torch.zeros(1, dtype=torch.float32, device=DEV)
    y = torch.ones(hop.STATIC_MAX_ROWS + 1, dtype=torch.float32, device=DEV)
    with pytest.raises(hop.HopError) as e:
        hop.svm_csr_sgd_static(x, x, 8, rp, col, val, y, hop.STATIC_MAX_ROWS + 1, 0.1)
    assert e.value.code == hop.E_ARG and "exceed" in str(e.value)
