"""Oracle, part 2: Reduce / Apply and the gradients, in float64 (TEST INFRASTRUCTURE ONLY).

Given a consumption trace, the parameters have a plain definition (Fig. alg0 / Fig. alg2
Train(), Reduce of Fig. alg4 or Eq. 2):

    NORMAL at level k, worker i:  x_{k+1,i} = sum_{(j,v) consumed} (num/den) x_{v,j} - lr * d_{k,i}
        d = g_{k,i}                      plain SGD (Fig. alg0: gradient of the pre-Reduce parameters,
                                         the "parallel approach" of Section 3.2)
        d = m <- mu*m + g_{k,i}          momentum; the buffer m is local and never averaged
    weight decay lambda adds lambda * x_{k,i} to g (the experiments' regulariser, Section 7.2).
    Serial approach (Section 3.2): Compute, Apply, then Send: x'_{k,i} = x_{k,i} - lr * d is what the worker sends
    (it replaces version k), and x_{k+1,i} = sum (num/den) x'_{v,j}; all Applies of a level precede its Reduces.
    JUMP at level k (Section 5):  x_{k+1,i} = sum (num/den) x_{v,j}, no gradient; the worker's own
                                  entry names the version it actually holds.
    IDLE: nothing.

Versions are kept in a dictionary keyed (worker, version): there is no ring buffer here.
The synthetic-gradient workloads are separable by parameter index, so `cols` may select any
subset of columns and the result is exact for those columns.
"""
from __future__ import annotations

import numpy as np

from . import philox

IDLE, NORMAL, JUMP = 0, 1, 2


def hinge_coefficients(margins: np.ndarray, y: np.ndarray) -> np.ndarray:
    """d/d(margin) of the mean hinge loss (1/B) sum_r max(0, 1 - y_r m_r); zero at the kink."""
    B = len(y)
    return np.where(y * margins < 1.0, -y / B, 0.0)


def log_coefficients(margins: np.ndarray, y: np.ndarray) -> np.ndarray:
    """d/d(margin) of the mean log loss (1/B) sum_r log(1 + exp(-y_r m_r)) (the loss of the paper's SVM runs)."""
    B = len(y)
    return -y / (B * (1.0 + np.exp(y * margins)))


def loss_coefficients(margins, y, loss="hinge"):
    return hinge_coefficients(margins, y) if loss == "hinge" else log_coefficients(margins, y)


def svm_gradient_dense(A: np.ndarray, y: np.ndarray, x: np.ndarray, loss="hinge") -> np.ndarray:
    """(Sub-)gradient of the mean hinge or log loss of a linear model (no bias, no regulariser) at x."""
    A = A.astype(np.float64)
    y = y.astype(np.float64)
    coef = loss_coefficients(A @ x, y, loss)
    return A.T @ coef


def svm_gradient_csr(row_ptr, col, val, y, x: np.ndarray, loss="hinge"):
    """Same for CSR rows; returns (coef per row, dense gradient)."""
    y = y.astype(np.float64)
    B = len(y)
    margins = np.empty(B)
    for r in range(B):
        a, e = row_ptr[r], row_ptr[r + 1]
        margins[r] = np.dot(val[a:e].astype(np.float64), x[col[a:e]])
    coef = loss_coefficients(margins, y, loss)
    g = np.zeros_like(x)
    for r in range(B):
        if coef[r] != 0.0:
            a, e = row_ptr[r], row_ptr[r + 1]
            np.add.at(g, col[a:e], coef[r] * val[a:e].astype(np.float64))
    return coef, g


def mean_hinge_loss(A, y, x):
    return np.maximum(0.0, 1.0 - y.astype(np.float64) * (A.astype(np.float64) @ x)).mean()


def mean_log_loss(A, y, x):
    return np.logaddexp(0.0, -y.astype(np.float64) * (A.astype(np.float64) @ x)).mean()


class GradSynthetic:
    def __init__(self, seed, sigma, cols):
        self.seed, self.sigma, self.cols = seed, sigma, np.asarray(cols, np.int64)

    def __call__(self, k, i, x):
        return philox.synthetic_gradient(self.seed, i, k, self.cols, self.sigma)


class GradSvmDense:
    """Minibatch of iteration k = rows [(k mod R/B)*B, +B) of the worker's shard."""
    def __init__(self, A, y, batch, loss="hinge"):
        self.A, self.y, self.B, self.loss = A, y, batch, loss

    def __call__(self, k, i, x):
        R = self.A.shape[1]
        r0 = (k % (R // self.B)) * self.B
        return svm_gradient_dense(self.A[i, r0:r0 + self.B], self.y[i, r0:r0 + self.B], x, self.loss)


class GradSvmCsr:
    def __init__(self, row_ptr, col, val, y, rows_per_worker, batch, loss="hinge"):
        self.row_ptr, self.col, self.val, self.y = row_ptr, col, val, y
        self.R, self.B, self.loss = rows_per_worker, batch, loss

    def __call__(self, k, i, x):
        r0 = i * self.R + (k % (self.R // self.B)) * self.B
        rp = self.row_ptr[r0:r0 + self.B + 1]
        yy = self.y[i, (r0 - i * self.R):(r0 - i * self.R) + self.B]
        _, g = svm_gradient_csr(rp, self.col, self.val, yy, x, self.loss)
        return g


class GradExternal:
    """Gradients handed in as arrays: G[k][i] -> vector."""
    def __init__(self, G):
        self.G = G

    def __call__(self, k, i, x):
        return np.asarray(self.G[k][i], np.float64)


def run_updates(tr: dict, N: int, lr: float, momentum: float, x0: np.ndarray, grad_fn,
                levels=None, keep_all=False, s=None, weight_decay=0.0, serial=False):
    """Execute levels 0..levels-1 of the trace arrays `tr` (see Trace.to_arrays).

    x0: [N][C] float64, version 0 of every worker.  Returns (X, newest) where X maps
    (worker, version) -> float64[C] and newest[i] is the newest version worker i holds."""
    op, ptr, nbr, ver, num, den = tr["op"], tr["ptr"], tr["nbr"], tr["ver"], tr["num"], tr["den"]
    L = op.shape[0] if levels is None else levels
    X = {(i, 0): np.array(x0[i], np.float64) for i in range(N)}
    newest = [0] * N
    M = [np.zeros(x0.shape[1]) for _ in range(N)] if momentum != 0.0 else None
    def direction(k, i):
        g = grad_fn(k, i, X[(i, k)])
        if weight_decay != 0.0:
            g = g + weight_decay * X[(i, k)]
        if M is not None:
            M[i] = momentum * M[i] + g
            g = M[i]
        return g

    for k in range(L):
        if serial:                                   # Compute -> Apply -> Send: version k becomes x' before any Reduce
            applied = {i: X[(i, k)] - lr * direction(k, i) for i in range(N) if op[k, i] == NORMAL}
            for i, x in applied.items():
                X[(i, k)] = x
        new = {}
        for i in range(N):
            o = op[k, i]
            if o == IDLE:
                continue
            a, e = ptr[k * N + i], ptr[k * N + i + 1]
            mix = np.zeros(x0.shape[1])
            for t in range(a, e):
                mix += (float(num[t]) / float(den[k, i])) * X[(int(nbr[t]), int(ver[t]))]
            if o == NORMAL and not serial:
                mix = mix - lr * direction(k, i)
            new[(i, k + 1)] = mix
        for (i, v), x in new.items():
            X[(i, v)] = x
            newest[i] = v
        if not keep_all and s is not None:
            for key in [key for key in X if key[1] < k - s - 1 and key[1] != newest[key[0]]]:
                del X[key]
    return X, newest
