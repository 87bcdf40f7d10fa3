"""Pins for the fp64 update-rule oracle and the gradient generators (CPU only)."""
import os

import numpy as np
import pytest
import torch

from oracle import philox, protocol as op, update as up
from paper_1902_01064_b200 import inputs


def uniform_W(n_in):
    """Eq. 1: W[j][i] = 1/|N_in(i)| for j in N_in(i)."""
    N = len(n_in)
    W = np.zeros((N, N))
    for i, nb in enumerate(n_in):
        for j in nb:
            W[j, i] = 1.0 / len(nb)
    return W


def trace_equal_speed(n_in, iters, s=0, mode=op.UNIFORM, max_ig=None):
    N = len(n_in)
    return op.simulate(n_in, np.ones((N, iters), np.uint64), iters, s=s, max_ig=max_ig, weight_mode=mode).to_arrays()


# ------------------------------------------------------------------ Fig. alg0 == library matmul
@pytest.mark.parametrize("n_in", [inputs.ring(5), inputs.torus(3, 3), inputs.directed_cycle(4), inputs.complete(4)])
def test_standard_training_is_matrix_recursion(n_in):
    rng = np.random.default_rng(0)
    N, C, iters, lr = len(n_in), 17, 6, 0.3
    x0 = rng.standard_normal((N, C))
    G = rng.standard_normal((iters, N, C))
    tr = trace_equal_speed(n_in, iters)
    X, newest = up.run_updates(tr, N, lr, 0.0, x0, up.GradExternal(G), keep_all=True)
    W = uniform_W(n_in)
    Xk = x0.copy()
    for k in range(iters):
        Xk = W.T @ Xk - lr * G[k]                      # x_{k+1,i} = sum_j W_ji x_{k,j} - lr g_{k,i}
        for i in range(N):
            np.testing.assert_allclose(X[(i, k + 1)], Xk[i], rtol=0, atol=1e-12)
    assert newest == [iters] * N


def test_complete_graph_is_allreduce_average():
    rng = np.random.default_rng(1)
    N, C, lr = 6, 9, 0.05
    x0 = rng.standard_normal((N, C))
    G = rng.standard_normal((1, N, C))
    tr = trace_equal_speed(inputs.complete(N), 1, s=2, mode=op.STALE_LINEAR, max_ig=2)
    X, _ = up.run_updates(tr, N, lr, 0.0, x0, up.GradExternal(G), keep_all=True)
    for i in range(N):
        np.testing.assert_allclose(X[(i, 1)], x0.mean(axis=0) - lr * G[0, i], atol=1e-13)


def test_zero_gradient_hull_and_mean_conservation():
    rng = np.random.default_rng(2)
    n_in = inputs.ring_chords(8, 3)
    N, C, iters = 8, 11, 15
    x0 = rng.standard_normal((N, C))
    T = rng.integers(1, 7, size=(N, iters)).astype(np.uint64)
    tr = op.simulate(n_in, T, iters, s=2, b=1, max_ig=2, weight_mode=op.STALE_LINEAR).to_arrays()
    X, newest = up.run_updates(tr, N, 0.1, 0.0, x0, up.GradExternal(np.zeros((iters, N, C))), keep_all=True)
    lo, hi = x0.min(axis=0) - 1e-12, x0.max(axis=0) + 1e-12
    for x in X.values():
        assert (x >= lo).all() and (x <= hi).all()          # convex combinations only
    # equal speeds + symmetric graph: W doubly stochastic -> the worker mean is conserved
    tr = trace_equal_speed(n_in, iters, s=2, mode=op.STALE_LINEAR, max_ig=2)
    X, _ = up.run_updates(tr, N, 0.1, 0.0, x0, up.GradExternal(np.zeros((iters, N, C))), keep_all=True)
    for k in range(iters + 1):
        np.testing.assert_allclose(np.mean([X[(i, k)] for i in range(N)], axis=0), x0.mean(axis=0), atol=1e-12)


def test_stale_weights_follow_eq2_by_hand():
    # one worker (1) consumes: itself at version 3, worker 0 at version 1, worker 2 at version 2; s = 2
    N, C = 3, 4
    rng = np.random.default_rng(3)
    xs = {(j, v): rng.standard_normal(C) for j in range(3) for v in range(4)}
    k, s = 3, 2
    vers = {0: 1, 1: 3, 2: 2}
    num = {j: vers[j] - (k - s) + 1 for j in vers}         # 1, 3, 2
    expect = sum(num[j] * xs[(j, vers[j])] for j in vers) / sum(num.values())
    nums, den = op.reduce_weights([vers[0], vers[1], vers[2]], k, s, op.STALE_LINEAR)
    assert nums == [1, 3, 2] and den == 6
    # drive run_updates with a hand-built one-level trace placed at level 0 of a shifted problem
    tr = dict(op=np.array([[0, 2, 0]], np.int32), ptr=np.array([0, 0, 3, 3], np.int64),
              nbr=np.array([0, 1, 2], np.int32), ver=np.array([0, 0, 0], np.int32),
              num=np.array(nums, np.int32), den=np.array([[0, den, 0]], np.int32))
    x0 = np.stack([xs[(0, 1)], xs[(1, 3)], xs[(2, 2)]])
    X, _ = up.run_updates(tr, 3, 0.0, 0.0, x0, up.GradExternal(np.zeros((1, 3, C))), keep_all=True)
    np.testing.assert_allclose(X[(1, 1)], expect, atol=1e-14)


def test_momentum_matches_torch_sgd_single_worker():
    # one worker with only its self-loop: Reduce is the identity, so the rule must be textbook
    # momentum SGD (buf = mu*buf + g; x -= lr*buf), i.e. torch.optim.SGD without dampening.
    rng = np.random.default_rng(4)
    C, iters, lr, mu = 13, 12, 0.1, 0.9
    x0 = rng.standard_normal((1, C))
    G = rng.standard_normal((iters, 1, C))
    tr = trace_equal_speed([[0]], iters)
    X, _ = up.run_updates(tr, 1, lr, mu, x0, up.GradExternal(G), keep_all=True)
    p = torch.tensor(x0[0], dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=mu)
    for k in range(iters):
        p.grad = torch.tensor(G[k, 0], dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(X[(0, k + 1)], p.detach().numpy(), atol=1e-12)


def test_momentum_buffer_is_local_and_gradient_uses_pre_reduce_parameters():
    # two workers, complete graph: mix is the mean, each keeps its own buffer; the gradient
    # function sees x_{k,i} (before the Reduce), as in the parallel approach of Section 3.2.
    lr, mu = 0.5, 0.5
    x0 = np.array([[1.0], [3.0]])
    seen = []

    def grad(k, i, x):
        seen.append((k, i, float(x[0])))
        return x.copy()                                   # g = x  (F = x^2 / 2)
    tr = trace_equal_speed(inputs.complete(2), 2)
    X, _ = up.run_updates(tr, 2, lr, mu, x0, grad, keep_all=True)
    # level 0: mean 2; m = (1, 3); x1 = (2 - .5, 2 - 1.5) = (1.5, 0.5)
    assert X[(0, 1)][0] == 1.5 and X[(1, 1)][0] == 0.5
    # level 1: mean 1; m = (.5*1 + 1.5, .5*3 + .5) = (2, 2); x2 = (0, 0)
    assert X[(0, 2)][0] == 0.0 and X[(1, 2)][0] == 0.0
    assert seen == [(0, 0, 1.0), (0, 1, 3.0), (1, 0, 1.5), (1, 1, 0.5)]


def test_jump_record_has_no_gradient_and_uses_held_version():
    tr = dict(op=np.array([[1, 1], [0, 1], [2, 1]], np.int32),
              ptr=np.array([0, 1, 2, 2, 3, 5, 6], np.int64),
              nbr=np.array([0, 1, 1, 0, 1, 1], np.int32),
              ver=np.array([0, 0, 1, 1, 2, 2], np.int32),
              num=np.array([1, 1, 1, 1, 1, 1], np.int32),
              den=np.array([[1, 1], [0, 1], [2, 1]], np.int32))
    x0 = np.array([[10.0], [20.0]])
    calls = []

    def grad(k, i, x):
        calls.append((k, i))
        return np.ones(1)
    X, newest = up.run_updates(tr, 2, 1.0, 0.0, x0, grad, keep_all=True)
    assert X[(0, 1)][0] == 9.0 and X[(1, 1)][0] == 19.0 and X[(1, 2)][0] == 18.0
    assert X[(0, 3)][0] == (9.0 + 18.0) / 2                # JUMP at level 2: own version 1 + neighbour version 2
    assert (0, 2) not in X and newest == [3, 3]
    assert (2, 0) not in calls and (1, 0) not in calls


# ------------------------------------------------------------------ SVM gradient
def test_hinge_gradient_at_zero_closed_form():
    w = inputs.make_workload(1)
    A, y = w.svm.dense[0, :32], w.svm.y[0, :32]
    g = up.svm_gradient_dense(A, y, np.zeros(64))
    np.testing.assert_allclose(g, -(y[:, None].astype(np.float64) * A).sum(axis=0) / 32, atol=1e-14)


def test_hinge_gradient_finite_differences():
    rng = np.random.default_rng(5)
    A = rng.standard_normal((32, 10)).astype(np.float32)
    y = np.where(rng.random(32) < 0.5, -1.0, 1.0).astype(np.float32)
    x = rng.standard_normal(10) * 0.3
    assert np.abs(1 - y * (A.astype(np.float64) @ x)).min() > 1e-3          # away from the kinks
    g = up.svm_gradient_dense(A, y, x)
    h = 1e-6
    for p in range(10):
        e = np.zeros(10)
        e[p] = h
        fd = (up.mean_hinge_loss(A, y, x + e) - up.mean_hinge_loss(A, y, x - e)) / (2 * h)
        assert abs(fd - g[p]) < 1e-7


def test_hinge_kink_is_inactive_and_csr_equals_dense():
    A = np.array([[1.0, 0.0], [0.0, 2.0]], np.float32)
    y = np.array([1.0, -1.0], np.float32)
    x = np.array([1.0, 0.25])                               # margins 1 (kink, inactive) and .5 (y*m = -.5 < 1)
    np.testing.assert_allclose(up.svm_gradient_dense(A, y, x), [0.0, 1.0])
    rng = np.random.default_rng(6)
    D = rng.standard_normal((8, 30)) * (rng.random((8, 30)) < 0.2)
    yy = np.where(rng.random(8) < 0.5, -1.0, 1.0)
    row_ptr, col, val = [0], [], []
    for r in range(8):
        nz = np.nonzero(D[r])[0]
        col += nz.tolist()
        val += D[r, nz].tolist()
        row_ptr.append(len(col))
    xx = rng.standard_normal(30)
    coef, g = up.svm_gradient_csr(np.array(row_ptr), np.array(col), np.array(val, np.float32), yy, xx)
    np.testing.assert_allclose(g, up.svm_gradient_dense(D.astype(np.float32), yy, xx), atol=1e-7)


# ------------------------------------------------------------------ Philox + Box-Muller
def test_philox_known_answers():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        out = philox.philox4x32_10([v[0]], [v[1]], [v[2]], [v[3]], v[4], v[5])
        assert [int(o[0]) for o in out] == v[6:10]
        n += 1
    assert n == 3


def test_box_muller_inverts_and_is_standard_normal():
    from scipy import stats
    rng = np.random.default_rng(8)
    ra = rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32)
    rb = rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32)
    z0, z1 = philox.box_muller(ra, rb)
    u1 = ((ra >> 9).astype(np.float64) + 0.5) / 2 ** 23
    u2 = ((rb >> 9).astype(np.float64) + 0.5) / 2 ** 23
    np.testing.assert_allclose(np.exp(-(z0 ** 2 + z1 ** 2) / 2), u1, rtol=1e-9)      # radius
    np.testing.assert_allclose(np.mod(np.arctan2(z1, z0) / (2 * np.pi), 1.0), u2, atol=1e-9)   # angle
    assert stats.kstest(np.concatenate([z0, z1]), "norm").pvalue > 1e-3


def test_synthetic_gradient_is_a_pure_function_of_its_indices():
    cols = np.arange(0, 64)
    g = philox.synthetic_gradient(12345678901, 3, 7, cols, 1e-3)
    sub = philox.synthetic_gradient(12345678901, 3, 7, cols[[5, 17, 40]], 1e-3)
    np.testing.assert_array_equal(g[[5, 17, 40]], sub)                                 # column-separable
    assert not np.allclose(g, philox.synthetic_gradient(12345678901, 4, 7, cols, 1e-3))
    assert not np.allclose(g, philox.synthetic_gradient(12345678901, 3, 8, cols, 1e-3))
    big = philox.synthetic_gradient(99, 0, 0, np.arange(400000), 1e-3)
    assert abs(big.mean()) < 1e-5 and abs(big.std() - 1e-3) < 1e-5


# ------------------------------------------------------------------ log loss, weight decay, serial approach
def test_log_loss_gradient_matches_autograd_and_finite_differences():
    rng = np.random.default_rng(11)
    A = rng.standard_normal((32, 10)).astype(np.float32)
    y = np.where(rng.random(32) < 0.5, -1.0, 1.0).astype(np.float32)
    x = rng.standard_normal(10)
    g = up.svm_gradient_dense(A, y, x, loss="log")
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    loss = torch.nn.functional.softplus(-torch.tensor(y, dtype=torch.float64) * (torch.tensor(A, dtype=torch.float64) @ xt)).mean()
    loss.backward()
    np.testing.assert_allclose(g, xt.grad.numpy(), atol=1e-13)
    h = 1e-6
    for p in range(10):
        e = np.zeros(10)
        e[p] = h
        fd = (up.mean_log_loss(A, y, x + e) - up.mean_log_loss(A, y, x - e)) / (2 * h)
        assert abs(fd - g[p]) < 1e-8


def test_weight_decay_and_momentum_match_torch_sgd_single_worker():
    rng = np.random.default_rng(12)
    C, iters, lr, mu, wd = 9, 10, 0.1, 0.9, 0.05
    x0 = rng.standard_normal((1, C))
    G = rng.standard_normal((iters, 1, C))
    tr = trace_equal_speed([[0]], iters)
    for serial in (False, True):                        # with one worker Reduce is the identity: both orders coincide
        X, _ = up.run_updates(tr, 1, lr, mu, x0, up.GradExternal(G), keep_all=True, weight_decay=wd, serial=serial)
        p = torch.tensor(x0[0], dtype=torch.float64, requires_grad=True)
        opt = torch.optim.SGD([p], lr=lr, momentum=mu, weight_decay=wd)
        for k in range(iters):
            p.grad = torch.tensor(G[k, 0], dtype=torch.float64)
            opt.step()
            # serial: version k is replaced by what the worker sent, x'_k = x_k - lr d_k (= the optimiser's state)
            np.testing.assert_allclose(X[(0, k)] if serial else X[(0, k + 1)], p.detach().numpy(), atol=1e-12)
        np.testing.assert_allclose(X[(0, iters)], p.detach().numpy(), atol=1e-12)


@pytest.mark.parametrize("n_in", [inputs.ring(5), inputs.torus(3, 3), inputs.complete(4)])
def test_serial_approach_is_apply_then_average(n_in):
    # serial approach of Section 3.2 with equal speeds: X_{k+1} = W^T (X_k - lr G_k)
    rng = np.random.default_rng(13)
    N, C, iters, lr = len(n_in), 7, 5, 0.2
    x0 = rng.standard_normal((N, C))
    G = rng.standard_normal((iters, N, C))
    tr = trace_equal_speed(n_in, iters)
    X, _ = up.run_updates(tr, N, lr, 0.0, x0, up.GradExternal(G), keep_all=True, serial=True)
    W = uniform_W(n_in)
    Xk = x0.copy()
    for k in range(iters):
        sent = Xk - lr * G[k]
        for i in range(N):
            np.testing.assert_allclose(X[(i, k)], sent[i], atol=1e-12)        # version k as sent
        Xk = W.T @ sent
    for i in range(N):
        np.testing.assert_allclose(X[(i, iters)], Xk[i], atol=1e-12)
    # and it differs from the parallel approach as soon as replicas differ
    Xp, _ = up.run_updates(tr, N, lr, 0.0, x0, up.GradExternal(G), keep_all=True)
    assert np.abs(Xp[(0, iters)] - X[(0, iters)]).max() > 1e-3
