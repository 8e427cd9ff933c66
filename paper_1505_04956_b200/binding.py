"""ctypes binding of libasgd.so: same names as the C ABI (include/asgd.h), argument marshalling only.

torch is used for device memory and the stream handle; every step of the method runs inside the
library's CUDA kernels.  There is no fallback: if the library is missing, loading fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libasgd.so")

ASGD_OK, ASGD_EINVAL, ASGD_ENOMEM, ASGD_ECUDA, ASGD_EUNSUPPORTED, ASGD_ETIMEOUT = 0, -1, -2, -3, -4, -5
PATH_AUTO, PATH_FP32, PATH_TC_FP16, PATH_TC_BF16, PATH_FP32_GENERAL = 0, 1, 2, 3, 4

EXPORTS = (
    "asgd_workspace_bytes", "asgd_init", "asgd_step", "asgd_run", "asgd_get_state", "asgd_set_state",
    "asgd_put", "asgd_put_rows", "asgd_get_accept_rows", "asgd_eval", "asgd_get_stats", "asgd_get_assign", "asgd_get_accept", "asgd_sync",
    "asgd_set_wait_drill", "asgd_launch_count", "asgd_path_name", "asgd_last_cuda_error", "asgd_strerror", "asgd_destroy",
    "asgd_fit_host_bytes", "asgd_fit_host", "asgd_eval_noalloc",
)


class AsgdConfig(C.Structure):
    """Mirror of `asgd_config`."""
    _fields_ = [
        ("N", C.c_int64), ("d", C.c_int32), ("k", C.c_int32), ("W", C.c_int32), ("b", C.c_int32),
        ("eps", C.c_float), ("comm_interval", C.c_int32), ("fanout", C.c_int32), ("slots", C.c_int32),
        ("parzen", C.c_int32), ("dist_path", C.c_int32), ("shuffle", C.c_int32),
        ("record_assign", C.c_int32), ("partial_rows", C.c_int32), ("seed", C.c_uint64),
    ]


class AsgdError(RuntimeError):
    def __init__(self, status, where, cuda=0):
        self.status = status
        msg = "%s: %s (%d)" % (where, strerror(status), status)
        if cuda:
            msg += " [cudaError %d]" % cuda
        super().__init__(msg)


_lib = None


def load():
    """Load libasgd.so.  Raises if it has not been built: there is no other implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("libasgd.so is not built (run `python -m paper_1505_04956_b200.build`); "
                          "this package has no CPU or PyTorch fallback")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
    cfgp = C.POINTER(AsgdConfig)
    L.asgd_workspace_bytes.argtypes = [cfgp, C.POINTER(sz)]
    L.asgd_init.argtypes = [C.POINTER(vp), cfgp, vp, vp, vp, vp, sz, vp]
    L.asgd_step.argtypes = [vp, i64]
    L.asgd_run.argtypes = [vp, i64]
    L.asgd_get_state.argtypes = [vp, i32, vp]
    L.asgd_set_state.argtypes = [vp, i32, vp]
    L.asgd_put.argtypes = [vp, i32, i32, vp]
    L.asgd_put_rows.argtypes = [vp, i32, i32, vp, i32, i32]
    L.asgd_get_accept_rows.argtypes = [vp, i32, C.POINTER(C.c_int32)]
    L.asgd_eval.argtypes = [vp, i32, C.POINTER(C.c_double)]
    L.asgd_get_stats.argtypes = [vp, i32, C.POINTER(C.c_uint64)]
    L.asgd_get_assign.argtypes = [vp, vp]
    L.asgd_get_accept.argtypes = [vp, i32, C.POINTER(C.c_int32)]
    L.asgd_sync.argtypes = [vp]
    L.asgd_set_wait_drill.argtypes = [vp, C.c_uint32, i64]
    L.asgd_launch_count.argtypes = [vp]
    L.asgd_launch_count.restype = i64
    L.asgd_path_name.argtypes = [vp]
    L.asgd_path_name.restype = C.c_char_p
    L.asgd_last_cuda_error.argtypes = [vp]
    L.asgd_strerror.argtypes = [C.c_int]
    L.asgd_strerror.restype = C.c_char_p
    L.asgd_destroy.argtypes = [vp]
    L.asgd_destroy.restype = None
    L.asgd_fit_host_bytes.argtypes = [cfgp, C.POINTER(sz)]
    L.asgd_fit_host.argtypes = [cfgp, vp, vp, i64, i32, vp, vp, sz, vp]
    L.asgd_eval_noalloc.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    _lib = L
    return L


def strerror(status: int) -> str:
    return load().asgd_strerror(int(status)).decode()


def make_config(*, N, d, k, W, b, eps, comm_interval=0, fanout=0, slots=None, parzen=1,
                dist_path=PATH_AUTO, shuffle=1, record_assign=0, seed=0, partial_rows=0) -> AsgdConfig:
    return AsgdConfig(int(N), int(d), int(k), int(W), int(b), float(eps), int(comm_interval), int(fanout),
                      int(slots) if slots else max(1, int(fanout)), int(parzen), int(dist_path), int(shuffle),
                      int(record_assign), int(partial_rows), int(seed))


def asgd_workspace_bytes(cfg: AsgdConfig) -> int:
    n = C.c_size_t(0)
    rc = load().asgd_workspace_bytes(C.byref(cfg), C.byref(n))
    if rc != ASGD_OK:
        raise AsgdError(rc, "asgd_workspace_bytes")
    return int(n.value)


def asgd_fit_host_bytes(cfg: AsgdConfig) -> int:
    n = C.c_size_t(0)
    rc = load().asgd_fit_host_bytes(C.byref(cfg), C.byref(n))
    if rc != ASGD_OK:
        raise AsgdError(rc, "asgd_fit_host_bytes")
    return int(n.value)


def _stream_handle(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def asgd_fit_host(cfg: AsgdConfig, X_host, w0_host, steps_per_worker: int, mode_async: bool, w_out_host,
                  scratch_dev, stream=None) -> None:
    """Whole job from host tensors (X_host, w0_host, w_out_host: CPU fp32; scratch_dev: CUDA uint8)."""
    rc = load().asgd_fit_host(C.byref(cfg), C.c_void_p(X_host.data_ptr()), C.c_void_p(w0_host.data_ptr()),
                              int(steps_per_worker), 1 if mode_async else 0, C.c_void_p(w_out_host.data_ptr()),
                              C.c_void_p(scratch_dev.data_ptr()), scratch_dev.numel(), _stream_handle(stream))
    if rc != ASGD_OK:
        raise AsgdError(rc, "asgd_fit_host")


def asgd_eval_noalloc(X, w, E_out, stream=None) -> int:
    """E(w) over the rows of X into the one-element float64 CUDA tensor `E_out`, using only the
    library's built-in scratch array (for callers that may not allocate device memory).  Returns the
    status code instead of raising, so that a caller can probe the size limits."""
    n, d = X.shape
    return int(load().asgd_eval_noalloc(C.c_void_p(X.data_ptr()), int(n), int(d), int(w.shape[0]),
                                        C.c_void_p(w.data_ptr()), C.c_void_p(E_out.data_ptr()),
                                        _stream_handle(stream)))


class Asgd:
    """One library context.  Methods carry the C function's name without the prefix."""

    def __init__(self, cfg: AsgdConfig, X, w0, X_bf16=None, stream=None):
        import torch
        if not (X.is_cuda and w0.is_cuda):
            raise ValueError("X and w0 must be CUDA tensors: the library has no host path")
        assert X.dtype == torch.float32 and X.is_contiguous() and w0.dtype == torch.float32 and w0.is_contiguous()
        self._L = load()
        self.cfg = cfg
        self.X, self.w0, self.X_bf16 = X, w0, X_bf16          # keep the borrowed buffers alive
        self.k, self.d, self.W, self.b, self.S = cfg.k, cfg.d, cfg.W, cfg.b, cfg.slots
        self.stream = stream
        self.workspace = torch.empty(asgd_workspace_bytes(cfg) + 256, dtype=torch.uint8, device=X.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        h = C.c_void_p()
        rc = self._L.asgd_init(C.byref(h), C.byref(cfg), C.c_void_p(X.data_ptr()),
                               C.c_void_p(X_bf16.data_ptr()) if X_bf16 is not None else None,
                               C.c_void_p(w0.data_ptr()), C.c_void_p(base), self.workspace.numel() - 256,
                               _stream_handle(stream))
        if rc != ASGD_OK:
            raise AsgdError(rc, "asgd_init")
        self._h = h

    def _chk(self, rc, where):
        if rc != ASGD_OK:
            raise AsgdError(rc, where, self._L.asgd_last_cuda_error(self._h))

    def step(self, rounds: int = 1):
        self._chk(self._L.asgd_step(self._h, int(rounds)), "asgd_step")

    def run(self, steps_per_worker: int):
        self._chk(self._L.asgd_run(self._h, int(steps_per_worker)), "asgd_run")

    def get_state(self, worker: int = 0, out=None):
        import torch
        if out is None:
            out = torch.empty((self.k, self.d), dtype=torch.float32, device=self.X.device)
        self._chk(self._L.asgd_get_state(self._h, int(worker), C.c_void_p(out.data_ptr())), "asgd_get_state")
        return out

    def set_state(self, worker: int, w):
        assert w.is_cuda and w.is_contiguous() and w.numel() == self.k * self.d
        self._chk(self._L.asgd_set_state(self._h, int(worker), C.c_void_p(w.data_ptr())), "asgd_set_state")

    def put(self, worker: int, slot: int, payload):
        assert payload.is_cuda and payload.is_contiguous() and payload.numel() == self.k * self.d
        self._chk(self._L.asgd_put(self._h, int(worker), int(slot), C.c_void_p(payload.data_ptr())), "asgd_put")

    def put_rows(self, worker: int, slot: int, payload, first_row: int, n_rows: int):
        assert payload.is_cuda and payload.is_contiguous() and payload.numel() == self.k * self.d
        self._chk(self._L.asgd_put_rows(self._h, int(worker), int(slot), C.c_void_p(payload.data_ptr()), int(first_row),
                                        int(n_rows)), "asgd_put_rows")

    def get_accept_rows(self, worker: int):
        """[S][k] per-row acceptance of the worker's last step in per-centre mode (-1, 0, 1)."""
        out = (C.c_int32 * (self.S * self.k))()
        self._chk(self._L.asgd_get_accept_rows(self._h, int(worker), out), "asgd_get_accept_rows")
        return [[int(out[s * self.k + a]) for a in range(self.k)] for s in range(self.S)]

    def eval(self, worker: int = 0) -> float:
        e = C.c_double(0.0)
        self._chk(self._L.asgd_eval(self._h, int(worker), C.byref(e)), "asgd_eval")
        return float(e.value)

    def get_stats(self, worker: int):
        out = (C.c_uint64 * 5)()
        self._chk(self._L.asgd_get_stats(self._h, int(worker), out), "asgd_get_stats")
        return dict(zip(("steps", "sent", "received", "accepted", "overwritten"), (int(v) for v in out)))

    def get_assign(self, out=None):
        import torch
        if out is None:
            out = torch.empty((self.W, self.b), dtype=torch.int32, device=self.X.device)
        self._chk(self._L.asgd_get_assign(self._h, C.c_void_p(out.data_ptr())), "asgd_get_assign")
        return out

    def get_accept(self, worker: int):
        out = (C.c_int32 * self.S)()
        self._chk(self._L.asgd_get_accept(self._h, int(worker), out), "asgd_get_accept")
        return [int(v) for v in out]

    def sync(self):
        self._chk(self._L.asgd_sync(self._h), "asgd_sync")

    def set_wait_drill(self, wait_limit: int, withhold_step: int = -1):
        self._chk(self._L.asgd_set_wait_drill(self._h, int(wait_limit), int(withhold_step)), "asgd_set_wait_drill")

    def launch_count(self) -> int:
        return int(self._L.asgd_launch_count(self._h))

    def path_name(self) -> str:
        return self._L.asgd_path_name(self._h).decode()

    def destroy(self):
        if getattr(self, "_h", None):
            self._L.asgd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
