"""ctypes binding of the C ABI in ``include/sketched_amsgrad.h``.

Argument marshalling only: every step of the optimiser runs in the CUDA library.  There is no fallback; if the
library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# SKETCHED_AMSGRAD_LIB selects another build of the same library (e.g. the bounds-checked one)
LIB_PATH = os.environ.get("SKETCHED_AMSGRAD_LIB") or os.path.join(_HERE, "libsketched_amsgrad.so")

EXPORTS = ["sk_create", "sk_step", "sk_set_lr", "sk_step_host", "sk_step_host_sparse", "sk_destroy", "sk_set_stream", "sk_sync", "sk_set_option",
           "sk_get_option", "sk_hash", "sk_get", "sk_set", "sk_algorithmic_bytes", "sk_get_timing", "sk_select_static",
           "sk_exchange_floats", "sk_step_local", "sk_step_select", "sk_step_finish", "sk_last_error", "sk_version",
           "sk_get_stats", "sk_test_fail_allocation", "sk_debug_check"]
NUM_STATS = 6
STAT_NAMES = ["threshold", "threshold_bin_count", "tie_group_count", "emitted", "floats_on_the_wire", "status"]
STATIC_MAX_D = 262144
NUM_STAGES = 8
STAGE_NAMES = ["zero_tables", "second_moment", "moment_sketch", "sum_tables", "unsketch_hist",
               "unsketch_emit", "refine", "apply"]

_lib = None


class SkError(RuntimeError):
    pass


def lib() -> C.CDLL:
    """Loads the built library (build it with ``python -m paper_2210_07454_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SkError(f"{LIB_PATH} is missing: build the CUDA library first (there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        u64, u32, f32, vp, i64 = C.c_uint64, C.c_uint32, C.c_float, C.c_void_p, C.c_int64
        L.sk_create.restype = vp
        L.sk_create.argtypes = [u64, u32, u32, u32, u64, u64, f32, f32, f32, f32]
        L.sk_step.restype = C.c_int; L.sk_step.argtypes = [vp, vp, vp]
        L.sk_set_lr.restype = C.c_int; L.sk_set_lr.argtypes = [vp, f32]
        L.sk_step_host.restype = C.c_int; L.sk_step_host.argtypes = [vp, vp, vp]
        L.sk_step_host_sparse.restype = C.c_int; L.sk_step_host_sparse.argtypes = [vp, vp, vp, vp]
        L.sk_destroy.restype = None; L.sk_destroy.argtypes = [vp]
        L.sk_set_stream.restype = C.c_int; L.sk_set_stream.argtypes = [vp, vp]
        L.sk_sync.restype = C.c_int; L.sk_sync.argtypes = [vp]
        L.sk_set_option.restype = C.c_int; L.sk_set_option.argtypes = [vp, C.c_char_p, i64]
        L.sk_get_option.restype = C.c_int; L.sk_get_option.argtypes = [vp, C.c_char_p, C.POINTER(i64)]
        L.sk_hash.restype = C.c_int; L.sk_hash.argtypes = [vp, u32, u64, u64, vp, vp]
        L.sk_get.restype = C.c_int; L.sk_get.argtypes = [vp, C.c_char_p, vp, u64]
        L.sk_set.restype = C.c_int; L.sk_set.argtypes = [vp, C.c_char_p, vp, u64]
        L.sk_algorithmic_bytes.restype = u64; L.sk_algorithmic_bytes.argtypes = [vp]
        L.sk_get_timing.restype = C.c_int
        L.sk_get_timing.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(u64)]
        L.sk_select_static.restype = C.c_int; L.sk_select_static.argtypes = [vp, vp]
        L.sk_get_stats.restype = C.c_int; L.sk_get_stats.argtypes = [vp, C.POINTER(C.c_double), u32]
        L.sk_test_fail_allocation.restype = C.c_int; L.sk_test_fail_allocation.argtypes = [i64]
        L.sk_debug_check.restype = C.c_int; L.sk_debug_check.argtypes = [vp, u32]
        L.sk_exchange_floats.restype = u64; L.sk_exchange_floats.argtypes = [vp, C.c_int]
        L.sk_step_local.restype = C.c_int; L.sk_step_local.argtypes = [vp, vp, vp]
        L.sk_step_select.restype = C.c_int; L.sk_step_select.argtypes = [vp, vp, vp]
        L.sk_step_finish.restype = C.c_int; L.sk_step_finish.argtypes = [vp, vp, vp]
        L.sk_last_error.restype = C.c_char_p; L.sk_last_error.argtypes = []
        L.sk_version.restype = C.c_char_p; L.sk_version.argtypes = []
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc < 0:
        raise SkError(f"error {rc}: {lib().sk_last_error().decode()}")


def _ptr(t) -> int:
    """Address of a torch tensor (device or host) or a numpy array."""
    if isinstance(t, np.ndarray):
        assert t.flags.c_contiguous
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def _nbytes(t) -> int:
    return t.nbytes if isinstance(t, np.ndarray) else t.numel() * t.element_size()


class SketchedAMSGrad:
    """Handle over ``sk_create`` / ``sk_step`` / ``sk_destroy`` and the auxiliary calls."""

    _FIELD_SHAPES = {"m": "nd", "e": "nd", "v": "d", "vhat": "d", "est": "d", "x": "d", "tables": "nrc", "sum": "rc",
                     "vw": "nd", "vhatw": "nd"}

    def __init__(self, d, n, r, c, k, seed=0, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, log2g=None,
                 window_lines=None, variant="ga", P=1, workers_total=None):
        self.d, self.n, self.r, self.c, self.k = d, n, r, c, k
        self.stream_ptr = 0               # the CUDA stream the handle launches on (0 = the default stream)
        self._h = lib().sk_create(d, n, r, c, k, seed, lr, beta1, beta2, eps)
        if not self._h:
            raise SkError(f"sk_create failed: {lib().sk_last_error().decode()}")
        if log2g is not None:
            self.set_option("log2g", log2g)
        if window_lines is not None:
            self.set_option("window_lines", window_lines)
        if variant not in ("ga", "pa"):
            raise SkError("variant must be 'ga' (Algorithm 2, gradient averaging) or 'pa' (Algorithm 1)")
        if variant == "pa":
            self.set_option("variant", 1)
        self.P = P
        if P != 1:
            self.set_option("P", P)
        if workers_total is not None:     # this handle holds n of the workers of a partitioned step
            self.set_option("workers_total", workers_total)

    def close(self):
        if getattr(self, "_h", None):
            lib().sk_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    # -- the hot path -----------------------------------------------------------------------------------
    def step(self, grads, x) -> None:
        """grads: CUDA float32 tensor of n*d elements (worker-major); x: CUDA float32 tensor of d, in place."""
        _check(lib().sk_step(_ptr(grads), _ptr(x), self._h))

    def set_lr(self, lr: float) -> None:
        """Step size of the steps taken from now on; e_{t-1} is weighted by alpha_{t-1}/alpha_t (Algorithms 1, 2)."""
        _check(lib().sk_set_lr(self._h, float(lr)))

    def step_host(self, grads, x) -> None:
        """Same step with host buffers (numpy arrays or CPU tensors, ideally pinned); x is updated in place."""
        _check(lib().sk_step_host(_ptr(grads), _ptr(x), self._h))

    def step_host_sparse(self, grads, idx_out, values_out) -> None:
        """Host gradients in, sparse update out (k indices of I_t and the new values of x there); the parameters stay
        on the device (field "x").  idx_out: k uint32, values_out: k float32, host arrays."""
        _check(lib().sk_step_host_sparse(_ptr(grads), _ptr(idx_out), _ptr(values_out), self._h))

    # -- one iteration in three phases, the workers partitioned over processes (see partitioned.py) ----
    def exchange_floats(self, which: int) -> int:
        return int(lib().sk_exchange_floats(self._h, which))

    def step_local(self, grads, exchange1) -> None:
        _check(lib().sk_step_local(_ptr(grads), _ptr(exchange1), self._h))

    def step_select(self, exchange1, exchange2) -> None:
        _check(lib().sk_step_select(_ptr(exchange1), _ptr(exchange2), self._h))

    def step_finish(self, exchange2, x) -> None:
        _check(lib().sk_step_finish(_ptr(exchange2), _ptr(x), self._h))

    # -- auxiliaries ------------------------------------------------------------------------------------
    def sync(self) -> None:
        _check(lib().sk_sync(self._h))

    def set_stream(self, cuda_stream_ptr: int) -> None:
        _check(lib().sk_set_stream(self._h, cuda_stream_ptr))
        self.stream_ptr = int(cuda_stream_ptr or 0)

    def set_option(self, key: str, value: int) -> None:
        _check(lib().sk_set_option(self._h, key.encode(), int(value)))

    def get_option(self, key: str) -> int:
        out = C.c_int64(0)
        _check(lib().sk_get_option(self._h, key.encode(), C.byref(out)))
        return int(out.value)

    def hash(self, row: int, i0: int, count: int, idx_out, sign_out) -> None:
        """Writes buckets (uint32 / int32 CUDA tensor) and signs (int8 CUDA tensor) of `count` coordinates."""
        _check(lib().sk_hash(self._h, row, i0, count, _ptr(idx_out), _ptr(sign_out)))

    def get(self, field: str, out=None):
        """Copies a state field into `out` (numpy array or tensor) or into a new numpy array."""
        if out is None:
            if field == "I":
                out = np.empty(self._count_I(), np.uint32)
            elif field == "cand":
                out = np.empty(self.P * self.k if (self.P > 1 and self._count_I()) else 0, np.uint32)
            elif field == "t":
                out = np.empty(1, np.uint64)
            elif field == "keys":
                out = np.empty(self.d, np.uint32)
            else:
                if field not in self._FIELD_SHAPES:
                    raise SkError(f"unknown field '{field}'")
                dims = {"n": self.n, "d": self.d, "r": self.r, "c": self.c}
                out = np.empty(tuple(dims[ch] for ch in self._FIELD_SHAPES[field]), np.float32)
        _check(lib().sk_get(self._h, field.encode(), _ptr(out) if _nbytes(out) else 0, _nbytes(out)))
        return out

    def _count_I(self) -> int:
        return self.get_option("I_count")

    def set(self, field: str, value) -> None:
        _check(lib().sk_set(self._h, field.encode(), _ptr(value) if _nbytes(value) else 0, _nbytes(value)))

    def stats(self) -> dict:
        """Statistics of the last step's selection and the exchange volume (see sk_get_stats)."""
        out = (C.c_double * NUM_STATS)()
        _check(lib().sk_get_stats(self._h, out, NUM_STATS))
        return dict(zip(STAT_NAMES, [float(v) for v in out]))

    def debug_check(self, kind: int) -> None:
        """Debug build: makes the device record a bounds violation of `kind` (1..5) without any access."""
        _check(lib().sk_debug_check(self._h, kind))

    def select_static(self, idx_out) -> None:
        """Re-runs the last step's top-k selection into `idx_out` (CUDA tensor of k int32/uint32) without
        allocating: for callers that may not call cudaMalloc.  Shares one static scratch array with every other
        call, so calls must not overlap on the GPU; handles with d > STATIC_MAX_D are rejected."""
        _check(lib().sk_select_static(self._h, _ptr(idx_out)))

    def algorithmic_bytes(self) -> int:
        return int(lib().sk_algorithmic_bytes(self._h))

    def timing(self):
        """(steps, ms per stage, launches per stage) accumulated since the last call; clears the counters."""
        ms = (C.c_double * NUM_STAGES)()
        ln = (C.c_uint64 * NUM_STAGES)()
        steps = lib().sk_get_timing(self._h, ms, ln)
        _check(steps)
        return steps, list(ms), [int(v) for v in ln]


def version() -> str:
    return lib().sk_version().decode()
