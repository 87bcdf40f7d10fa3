"""ctypes binding of the C ABI in include/hop.h.  Argument marshalling only: every step of the
path runs inside libhop_b200.so.  Importing this module loads the library and raises ImportError
when it has not been built (python -m paper_1902_01064_b200.build); there is no CPU fallback."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# HOP_B200_LIBRARY selects another build of the same sources (the bounds-checked one the tests use)
LIB_PATH = os.environ.get("HOP_B200_LIBRARY") or os.path.join(_HERE, "libhop_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1902_01064_b200.build` "
                      "(the Hop hot path has no CPU fallback)")
lib = C.CDLL(LIB_PATH)

OK, E_ARG, E_GRAPH, E_TRACE, E_STATE, E_DEADLOCK, E_CUDA, E_DEVICE, E_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6, -7, -8
OP_IDLE, OP_NORMAL, OP_JUMP = 0, 1, 2
W_UNIFORM, W_STALE_LINEAR = 0, 1
GRAD_EXTERNAL, GRAD_SYNTHETIC, GRAD_SVM_DENSE, GRAD_SVM_CSR = 0, 1, 2, 3
MIX_AUTO, MIX_STAGED, MIX_BULK, MIX_TENSOR = 0, 1, 2, 3
(OPT_MAX_IG, OPT_LR, OPT_MOMENTUM, OPT_WEIGHT_MODE, OPT_GRAD_MODE, OPT_GRAD_SEED, OPT_GRAD_SIGMA,
 OPT_MIX_KERNEL, OPT_COL_OFFSET, OPT_USE_GRAPH, OPT_BACKUP_MODE, OPT_NOTIFY_ACK, OPT_WEIGHT_DECAY, OPT_LOSS,
 OPT_APPROACH, OPT_STALE_REDUCE, OPT_NVTX) = range(1, 18)
STALE_NEW_ONLY, STALE_REUSE = 0, 1
LOSS_HINGE, LOSS_LOG = 0, 1
APPROACH_PARALLEL, APPROACH_SERIAL = 0, 1
BACKUP_AT_LEAST, BACKUP_EXACT = 0, 1
OPT_BACKUP_OF_WORKER = 1000

_p = C.c_void_p
_i32, _i64, _u64, _f64 = C.c_int32, C.c_int64, C.c_uint64, C.c_double

SIGNATURES = {
    "hop_create": [C.POINTER(_p), _p, _p, _i32, _i64, _i32, _i32, _i32],
    "hop_destroy": [_p],
    "hop_last_error": [_p],
    "hop_set_option": [_p, C.c_int, _f64],
    "hop_sim_run": [_p, _p, _i32, C.POINTER(_p)],
    "hop_trace_create": [C.POINTER(_p), _i32, _i32, _p, _p, _p, _p, _p, _p],
    "hop_trace_dims": [_p, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i64), C.POINTER(_u64)],
    "hop_trace_export": [_p, _p, _p, _p, _p, _p, _p],
    "hop_trace_destroy": [_p],
    "hop_bind_buffers": [_p, _p, _p, _p, _p],
    "hop_bind_svm_dense": [_p, _p, _p, _i32, _i32],
    "hop_bind_svm_csr": [_p, _p, _p, _p, _p, _i32, _i32],
    "hop_load_trace": [_p, _p],
    "hop_write_params": [_p, _i32, _i32, _p],
    "hop_read_params": [_p, _i32, _i32, _p],
    "hop_newest_version": [_p, _i32, C.POINTER(_i32)],
    "hop_set_level": [_p, _i32],
    "hop_step": [_p],
    "hop_run": [_p, _i32],
    "hop_step_begin": [_p, C.POINTER(_p), C.POINTER(_i64)],
    "hop_step_end": [_p],
    "hop_step_host": [_p, _p, _p, _p, _p, _p, _p, _p, _i64],
    "hop_read_status": [_p, C.POINTER(_i32)],
    "hop_clear_status": [_p],
    "hop_build_is_checked": [],
    "hop_selftest_bounded_wait": [_p, _i32, _i32],
    "hop_level_stats": [_p, _i32, _p],
    "hop_timing_enable": [_p, _i32],
    "hop_timing_read": [_p, _p, _p, C.POINTER(_i64)],
    "hop_launch_count": [_p, C.POINTER(_i64)],
    "hop_svm_csr_sgd_static": [_p, _p, _i64, _p, _p, _p, _p, _i32, C.c_float, _p, C.c_char_p, _i64],
}
for _name, _args in SIGNATURES.items():
    _f = getattr(lib, _name)
    _f.argtypes = _args
    _f.restype = C.c_char_p if _name == "hop_last_error" else C.c_int


def build_is_checked() -> bool:
    return bool(lib.hop_build_is_checked())


class DeviceSpan:
    """A context-owned run of device memory, described through the CUDA array interface so that
    torch.as_tensor(span, device=...) wraps it without a copy (for a collective on it)."""

    def __init__(self, ptr: int, count: int, typestr: str = "<f8"):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 3}


class HopError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"hop error {code}: {msg}")
        self.code = code


def _ptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    if hasattr(a, "data_ptr"):          # torch tensor (device or pinned host memory)
        return a.data_ptr()
    return a


def _arr(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


class Trace:
    """Owns a hop_trace*."""

    def __init__(self, handle):
        self.h = handle

    @classmethod
    def from_arrays(cls, op, ptr, nbr, ver, num, den):
        op, den = _arr(op, np.int32), _arr(den, np.int32)
        ptr = _arr(ptr, np.int64)
        nbr, ver, num = _arr(nbr, np.int32), _arr(ver, np.int32), _arr(num, np.int32)
        levels, N = op.shape
        h = _p()
        rc = lib.hop_trace_create(C.byref(h), levels, N, _ptr(op), _ptr(ptr), _ptr(nbr), _ptr(ver), _ptr(num), _ptr(den))
        if rc:
            raise HopError(rc, (lib.hop_last_error(None) or b"").decode())
        return cls(h)

    def dims(self):
        L, N, E, mk = _i32(), _i32(), _i64(), _u64()
        lib.hop_trace_dims(self.h, C.byref(L), C.byref(N), C.byref(E), C.byref(mk))
        return L.value, N.value, E.value, mk.value

    def to_arrays(self):
        L, N, E, mk = self.dims()
        out = dict(op=np.zeros((L, N), np.int32), ptr=np.zeros(L * N + 1, np.int64), nbr=np.zeros(E, np.int32),
                   ver=np.zeros(E, np.int32), num=np.zeros(E, np.int32), den=np.zeros((L, N), np.int32))
        lib.hop_trace_export(self.h, *[_ptr(out[k]) for k in ("op", "ptr", "nbr", "ver", "num", "den")])
        out["makespan"] = mk
        return out

    def __del__(self):
        if getattr(self, "h", None):
            lib.hop_trace_destroy(self.h)
            self.h = None


class Hop:
    """Owns a hop_ctx*.  Method names mirror the C entry points without the hop_ prefix."""

    def __init__(self, in_ptr, in_idx, N, P, s, b, max_skip):
        self.h = _p()
        self.N, self.P, self.s = N, P, s
        in_ptr, in_idx = _arr(in_ptr, np.int32), _arr(in_idx, np.int32)
        rc = lib.hop_create(C.byref(self.h), _ptr(in_ptr), _ptr(in_idx), N, P, s, b, max_skip)
        if rc:
            self.h = None
            raise HopError(rc, (lib.hop_last_error(None) or b"").decode())
        self._keep = []

    def _chk(self, rc):
        if rc:
            raise HopError(rc, (lib.hop_last_error(self.h) or b"").decode())

    def set_option(self, key, value):
        self._chk(lib.hop_set_option(self.h, key, float(value)))

    def sim_run(self, ticks, iters) -> Trace:
        ticks = _arr(ticks, np.uint64)
        assert ticks.shape == (self.N, iters)
        h = _p()
        self._chk(lib.hop_sim_run(self.h, _ptr(ticks), iters, C.byref(h)))
        return Trace(h)

    def bind_buffers(self, X, M=None, G=None, stream=None):
        self._keep = [X, M, G]
        self._chk(lib.hop_bind_buffers(self.h, _ptr(X), _ptr(M), _ptr(G), stream))

    def bind_svm_dense(self, A, y, rows_per_worker, batch):
        self._keep += [A, y]
        self._chk(lib.hop_bind_svm_dense(self.h, _ptr(A), _ptr(y), rows_per_worker, batch))

    def bind_svm_csr(self, row_ptr, col, val, y, rows_per_worker, batch):
        self._keep += [row_ptr, col, val, y]
        self._chk(lib.hop_bind_svm_csr(self.h, _ptr(row_ptr), _ptr(col), _ptr(val), _ptr(y), rows_per_worker, batch))

    def load_trace(self, trace: Trace):
        self._chk(lib.hop_load_trace(self.h, trace.h))

    def write_params(self, worker, version, host_src):
        src = _arr(host_src, np.float32)
        assert src.size == self.P
        self._chk(lib.hop_write_params(self.h, worker, version, _ptr(src)))

    def read_params(self, worker, version=-1):
        dst = np.empty(self.P, np.float32)
        self._chk(lib.hop_read_params(self.h, worker, version, _ptr(dst)))
        return dst

    def newest_version(self, worker):
        v = _i32()
        self._chk(lib.hop_newest_version(self.h, worker, C.byref(v)))
        return v.value

    def set_level(self, level):
        self._chk(lib.hop_set_level(self.h, level))

    def step(self):
        self._chk(lib.hop_step(self.h))

    def step_begin(self):
        """Returns (device address of the partial margins, count of doubles); (None, 0) outside the SVM modes."""
        ptr, n = _p(), _i64()
        self._chk(lib.hop_step_begin(self.h, C.byref(ptr), C.byref(n)))
        return ptr.value, n.value

    def step_end(self):
        self._chk(lib.hop_step_end(self.h))

    def run(self, n_levels):
        self._chk(lib.hop_run(self.h, n_levels))

    def step_host(self, op, ptr, nbr, ver, num, den, probe=None):
        """One level from host arrays (already contiguous int32/int64 numpy); probe: float32 numpy or None."""
        n = 0 if probe is None else probe.size
        self._chk(lib.hop_step_host(self.h, _ptr(op), _ptr(ptr), _ptr(nbr), _ptr(ver), _ptr(num), _ptr(den), _ptr(probe), n))

    def read_status(self):
        w = _i32()
        self._chk(lib.hop_read_status(self.h, C.byref(w)))
        return w.value

    def read_status_word(self):
        """(return code, status word) without raising: HOP_E_DEVICE and the word a kernel left when it gave up a wait."""
        w = _i32()
        rc = lib.hop_read_status(self.h, C.byref(w))
        return rc, w.value

    def clear_status(self):
        self._chk(lib.hop_clear_status(self.h))

    def selftest_bounded_wait(self, polls=256, detail=0):
        self._chk(lib.hop_selftest_bounded_wait(self.h, polls, detail))

    def level_stats(self, level):
        out = np.zeros(10, np.int64)
        self._chk(lib.hop_level_stats(self.h, level, _ptr(out)))
        return dict(zip(("U", "normal", "jump", "entries", "tile_w", "kernel", "stage_rows", "alg_bytes", "mma_flops", "k_padded"),
                        out.tolist()))

    def timing_enable(self, on=True):
        self._chk(lib.hop_timing_enable(self.h, 1 if on else 0))

    def timing_read(self):
        ms, n, b = np.zeros(3, np.float64), np.zeros(3, np.int64), _i64()
        self._chk(lib.hop_timing_read(self.h, _ptr(ms), _ptr(n), C.byref(b)))
        return dict(ms_grad=ms[0], ms_mix=ms[1], ms_apply=ms[2], spans=n.tolist(), mix_bytes=b.value)

    def launch_count(self):
        n = _i64()
        self._chk(lib.hop_launch_count(self.h, C.byref(n)))
        return n.value

    def close(self):
        if getattr(self, "h", None):
            lib.hop_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()


STATIC_MAX_ROWS = 16384


def svm_csr_sgd_static(x, x_out, P, row_ptr, col, val, y, rows, lr, stream=None):
    """hop_svm_csr_sgd_static: context-free hinge-SVM minibatch step that allocates nothing (its
    coefficient scratch is a fixed array inside the library).  All array arguments are device buffers."""
    buf = C.create_string_buffer(512)
    rc = lib.hop_svm_csr_sgd_static(_ptr(x), _ptr(x_out), P, _ptr(row_ptr), _ptr(col), _ptr(val), _ptr(y), rows,
                                    float(lr), stream, buf, len(buf))
    if rc:
        raise HopError(rc, buf.value.decode())


def from_workload(w, mix_kernel=MIX_AUTO) -> Hop:
    """Context configured from a paper_1902_01064_b200.inputs.Workload (options only; no buffers)."""
    h = Hop(w.in_ptr, w.in_idx, w.N, w.P, w.s, w.b, w.max_skip)
    h.set_option(OPT_MAX_IG, w.max_ig)
    h.set_option(OPT_LR, w.lr)
    h.set_option(OPT_MOMENTUM, w.momentum)
    h.set_option(OPT_WEIGHT_MODE, w.weight_mode)
    h.set_option(OPT_GRAD_MODE, w.grad_mode)
    h.set_option(OPT_GRAD_SEED, w.grad_seed)
    h.set_option(OPT_GRAD_SIGMA, w.sigma)
    h.set_option(OPT_MIX_KERNEL, mix_kernel)
    h.set_option(OPT_STALE_REDUCE, w.stale_reduce)
    return h
