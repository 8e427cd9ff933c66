"""TEST INFRASTRUCTURE -- ctypes front end of the CPU oracle (asgd_oracle.cpp).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It knows nothing about the CUDA library and imports nothing from it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "asgd_oracle.cpp")
_LIB = os.path.join(_HERE, "libasgd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP on, used only when more than one thread is asked for)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-fopenmp", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u64, i64, i32, f32, vp = C.c_uint64, C.c_int64, C.c_int32, C.c_float, C.c_void_p
        L.oracle_sm64.restype = u64
        L.oracle_sm64.argtypes = [u64]
        L.oracle_draw.restype = u64
        L.oracle_draw.argtypes = [u64] * 5
        L.oracle_batch_order.argtypes = [u64, i32, i32, i64, vp]
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [i64, i32, i32, i32, i32, f32, i32, i32, i32, i32, i32, u64, vp, vp]
        L.oracle_destroy.argtypes = [vp]
        L.oracle_set_threads.argtypes = [vp, C.c_int]
        L.oracle_set_threads.restype = C.c_int
        L.oracle_rounds.argtypes = [vp, i64]
        L.oracle_get_state.argtypes = [vp, i32, vp]
        L.oracle_set_state.argtypes = [vp, i32, vp]
        L.oracle_put.argtypes = [vp, i32, i32, vp]
        L.oracle_get_mail.argtypes = [vp, i32, i32, vp, vp]
        L.oracle_get_stats.argtypes = [vp, i32, vp]
        L.oracle_get_perm.argtypes = [vp, i32, vp]
        L.oracle_batches_per_pass.argtypes = [vp]
        L.oracle_batches_per_pass.restype = i64
        L.oracle_shard_rows.argtypes = [vp]
        L.oracle_shard_rows.restype = i64
        L.oracle_recipients.argtypes = [vp, i32, u64, vp, vp]
        L.oracle_last_step.argtypes = [vp, i32] + [vp] * 7
        L.oracle_assign.argtypes = [vp, i64, i32, vp, i32, vp, vp, vp]
        L.oracle_eval.argtypes = [vp, i64, i32, vp, i32, C.c_int]
        L.oracle_eval.restype = C.c_double
        L.oracle_max_threads.restype = C.c_int
        L.oracle_set_partial_rows.argtypes = [vp, i32]
        L.oracle_set_partial_rows.restype = C.c_int
        L.oracle_put_rows.argtypes = [vp, i32, i32, vp, vp]
        L.oracle_put_row_flags.argtypes = [vp, i32, u64, i32, vp]
        L.oracle_last_step_rows.argtypes = [vp, i32, vp, vp, vp]
        L.oracle_get_mail_rows.argtypes = [vp, i32, i32, vp]
        _lib = L
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def sm64(x: int) -> int:
    return lib().oracle_sm64(x & (2**64 - 1))


def draw(seed: int, tag: int, a: int, b: int, c: int) -> int:
    return lib().oracle_draw(seed, tag, a, b, c)


def batch_order(seed: int, worker: int, B: int, shuffle: int = 1):
    """The worker's seeded order of its B mini-batches (Algorithm 5: shuffle, then draw in turn)."""
    out = np.empty(B, np.int32)
    lib().oracle_batch_order(int(seed), int(shuffle), int(worker), int(B), _p(out))
    return out


def assign(X, w):
    """Nearest prototype of every row of X (Eq. 8 text) -> (index, smallest, second smallest sq. distance)."""
    X = _f32(X)
    w = _f32(w)
    n, d = X.shape
    k = w.shape[0]
    a = np.empty(n, np.int32)
    d1 = np.empty(n, np.float64)
    d2 = np.empty(n, np.float64)
    lib().oracle_assign(_p(X), n, d, _p(w), k, _p(a), _p(d1), _p(d2))
    return a, d1, d2


def quantization_error(X, w, threads: int = 1) -> float:
    """E(w) of Eq. 8 over all rows of X."""
    X = _f32(X)
    w = _f32(w)
    return float(lib().oracle_eval(_p(X), X.shape[0], X.shape[1], _p(w), w.shape[0], threads))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


class Oracle:
    """Deterministic, round-synchronous ASGD over W workers on the host."""

    def __init__(self, X, w0, *, W, b, eps, comm_interval=0, fanout=0, slots=None, parzen=1,
                 shuffle=1, seed=0, threads=1, partial_rows=0):
        self.X = _f32(X)
        w0 = _f32(w0)
        self.N, self.d = self.X.shape
        self.k = w0.shape[0]
        assert w0.shape[1] == self.d
        self.W, self.b = int(W), int(b)
        self.S = int(slots) if slots else max(1, int(fanout))
        self.fanout = int(fanout)
        self._h = lib().oracle_create(self.N, self.d, self.k, self.W, self.b, float(eps), int(comm_interval),
                                      self.fanout, self.S, int(parzen), int(shuffle), int(seed), _p(self.X), _p(w0))
        if not self._h:
            raise ValueError("oracle_create rejected the configuration")
        self.threads = lib().oracle_set_threads(self._h, int(threads))
        self.partial_rows = int(partial_rows)
        if lib().oracle_set_partial_rows(self._h, self.partial_rows) != 0:
            raise ValueError("partial_rows must lie in 0..k")
        self.H = int(lib().oracle_shard_rows(self._h))
        self.B = int(lib().oracle_batches_per_pass(self._h))

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def rounds(self, n: int):
        lib().oracle_rounds(self._h, int(n))

    def state(self, worker: int = 0):
        out = np.empty((self.k, self.d), np.float32)
        lib().oracle_get_state(self._h, worker, _p(out))
        return out

    def states(self):
        return np.stack([self.state(i) for i in range(self.W)])

    def set_state(self, worker: int, w):
        w = _f32(w)
        assert w.shape == (self.k, self.d)
        lib().oracle_set_state(self._h, worker, _p(w))

    def put(self, worker: int, slot: int, payload):
        v = _f32(payload)
        assert v.shape == (self.k, self.d)
        lib().oracle_put(self._h, worker, slot, _p(v))

    def mail(self, worker: int, slot: int):
        out = np.empty((self.k, self.d), np.float32)
        ss = np.zeros(2, np.uint64)
        lib().oracle_get_mail(self._h, worker, slot, _p(out), _p(ss))
        return out, int(ss[0]), int(ss[1])

    def stats(self, worker: int):
        out = np.zeros(5, np.uint64)
        lib().oracle_get_stats(self._h, worker, _p(out))
        return dict(zip(("steps", "sent", "received", "accepted", "overwritten"), (int(x) for x in out)))

    def perm(self, worker: int):
        out = np.empty(self.B, np.int32)
        lib().oracle_get_perm(self._h, worker, _p(out))
        return out

    def recipients(self, worker: int, t: int):
        f = max(1, self.fanout)
        peers = np.zeros(f, np.int32)
        slots = np.zeros(f, np.int32)
        lib().oracle_recipients(self._h, worker, int(t), _p(peers), _p(slots))
        return peers[: self.fanout].copy(), slots[: self.fanout].copy()

    def last_step(self, worker: int):
        """Trace of the worker's most recent step."""
        a = np.empty(self.b, np.int32)
        d1 = np.empty(self.b, np.float64)
        d2 = np.empty(self.b, np.float64)
        cnt = np.empty(self.k, np.int64)
        acc = np.empty(self.S, np.int32)
        lhs = np.empty(self.S, np.float64)
        rhs = np.empty(self.S, np.float64)
        lib().oracle_last_step(self._h, worker, _p(a), _p(d1), _p(d2), _p(cnt), _p(acc), _p(lhs), _p(rhs))
        return dict(assign=a, d1=d1, d2=d2, counts=cnt, accept=acc, lhs=lhs, rhs=rhs)

    # ---- per-centre messages (Section 4.4) ----
    def put_rows(self, worker: int, slot: int, payload, has):
        """External put that carries only the centre rows flagged in has[k]."""
        v = _f32(payload)
        assert v.shape == (self.k, self.d)
        hs = np.ascontiguousarray(np.asarray(has, dtype=np.uint8))
        assert hs.shape == (self.k,)
        lib().oracle_put_rows(self._h, worker, slot, _p(v), _p(hs))

    def put_row_flags(self, worker: int, t: int, j: int):
        """Rows (k flags) of the j-th message of the put worker makes after its step t."""
        out = np.zeros(self.k, np.uint8)
        lib().oracle_put_row_flags(self._h, worker, int(t), int(j), _p(out))
        return out

    def mail_rows(self, worker: int, slot: int):
        out = np.zeros(self.k, np.uint8)
        lib().oracle_get_mail_rows(self._h, worker, slot, _p(out))
        return out

    def last_step_rows(self, worker: int):
        """Per-row trace of the last step in per-centre mode: accept[S, k] (-1 = row not in a new message), lhs, rhs."""
        acc = np.full((self.S, self.k), -1, np.int32)
        lhs = np.zeros((self.S, self.k), np.float64)
        rhs = np.zeros((self.S, self.k), np.float64)
        lib().oracle_last_step_rows(self._h, worker, _p(acc), _p(lhs), _p(rhs))
        return dict(accept=acc, lhs=lhs, rhs=rhs)
