"""CPU oracle for the SketchedAMSGrad step: TEST INFRASTRUCTURE ONLY.

A ctypes wrapper over ``sk_oracle.c`` / ``sk_oracle_step.c`` (plain C, fp64 arithmetic, fp32 storage).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA
library never does, and this package imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, f) for f in ("sk_oracle.c", "sk_oracle_step.c")]
_HDR = os.path.join(_HERE, "sk_oracle.h")
_LIB = os.path.join(_HERE, "libsk_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (FP contraction off, OpenMP on) if the library is missing or stale."""
    newest = max(os.path.getmtime(p) for p in _SRC + [_HDR])
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", tmp] + _SRC + ["-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u64, u32, f32, vp = C.c_uint64, C.c_uint32, C.c_float, C.c_void_p
        L.ora_mix64.restype = u64; L.ora_mix64.argtypes = [u64]
        L.ora_stream.restype = u64; L.ora_stream.argtypes = [u64, u64]
        L.ora_row_key.restype = u64; L.ora_row_key.argtypes = [u64, u32]
        L.ora_hash.restype = None; L.ora_hash.argtypes = [u64, u32, u32, u32, u64, u64, vp, vp]
        L.ora_hash_w.restype = None; L.ora_hash_w.argtypes = [u64, u32, u32, u32, u32, u64, u64, vp, vp]
        L.ora_sketch.restype = None; L.ora_sketch.argtypes = [vp, u64, u32, u32, vp, vp, vp]
        L.ora_median.restype = f32; L.ora_median.argtypes = [vp, u32]
        L.ora_unsketch.restype = None; L.ora_unsketch.argtypes = [vp, u64, u32, u32, vp, vp, vp, vp]
        L.ora_topk.restype = None; L.ora_topk.argtypes = [vp, u64, u64, vp]
        L.ora_create.restype = vp
        L.ora_create.argtypes = [u64, u32, u32, u32, u64, u64, u32, f32, f32, f32, f32]
        L.ora_destroy.restype = None; L.ora_destroy.argtypes = [vp]
        L.ora_set_hash.restype = None; L.ora_set_hash.argtypes = [vp, vp, vp]
        L.ora_set_option.restype = None; L.ora_set_option.argtypes = [vp, C.c_char_p, C.c_int]
        L.ora_set_lr.restype = None; L.ora_set_lr.argtypes = [vp, f32]
        L.ora_step.restype = C.c_int; L.ora_step.argtypes = [vp, vp, vp]
        L.ora_field.restype = vp; L.ora_field.argtypes = [vp, C.c_char_p]
        L.ora_count.restype = u64; L.ora_count.argtypes = [vp, C.c_char_p]
        L.ora_comm_floats.restype = C.c_double; L.ora_comm_floats.argtypes = [u64, u64, u64, u64]
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def mix64(z: int) -> int:
    return int(lib().ora_mix64(z & (2**64 - 1)))


def stream(s0: int, t: int) -> int:
    return int(lib().ora_stream(s0 & (2**64 - 1), t))


def hash_family(seed: int, log2g: int, c: int, row: int, i0: int, count: int, window_lines: int = 0):
    """Buckets (uint32) and signs (int8) of coordinates i0..i0+count-1 in one row."""
    b = np.empty(count, np.uint32)
    s = np.empty(count, np.int8)
    lib().ora_hash_w(seed, log2g, window_lines, c, row, i0, count, _p(b), _p(s))
    return b, s


def sketch(a, r: int, c: int, idx, sgn) -> np.ndarray:
    a = np.ascontiguousarray(a, np.float32)
    idx = np.ascontiguousarray(idx, np.uint32).reshape(r, a.size)
    sgn = np.ascontiguousarray(sgn, np.int8).reshape(r, a.size)
    out = np.empty((r, c), np.float32)
    lib().ora_sketch(_p(a), a.size, r, c, _p(idx), _p(sgn), _p(out))
    return out


def median(q) -> float:
    q = np.ascontiguousarray(q, np.float32)
    return float(lib().ora_median(_p(q), q.size))


def unsketch(table, d: int, idx, sgn, vhat=None) -> np.ndarray:
    table = np.ascontiguousarray(table, np.float32)
    r, c = table.shape
    idx = np.ascontiguousarray(idx, np.uint32).reshape(r, d)
    sgn = np.ascontiguousarray(sgn, np.int8).reshape(r, d)
    est = np.empty(d, np.float32)
    vh = None if vhat is None else np.ascontiguousarray(vhat, np.float32)
    lib().ora_unsketch(_p(table), d, r, c, _p(idx), _p(sgn), 0 if vh is None else _p(vh), _p(est))
    return est


def topk(est, k: int) -> np.ndarray:
    est = np.ascontiguousarray(est, np.float32)
    out = np.empty(k, np.uint32)
    lib().ora_topk(_p(est), est.size, k, _p(out))
    return out


def comm_floats(r: int, c: int, k: int, P: int) -> float:
    return float(lib().ora_comm_floats(r, c, k, P))


class Oracle:
    """One SketchedAMSGrad (gradient averaging) optimiser; `step` advances it by one iteration."""

    def __init__(self, d, n, r, c, k, seed=0, log2g=0, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8,
                 hash_idx=None, hash_sgn=None, v_keep=False, threads=1, window_lines=0, variant="ga", P=1,
                 freeze_v=False):
        self.d, self.n, self.r, self.c, self.k, self.P = d, n, r, c, k, P
        self._h = lib().ora_create(d, n, r, c, k, seed, log2g, lr, beta1, beta2, eps)
        if not self._h:
            raise ValueError("ora_create rejected the arguments")
        self._keep = None
        if hash_idx is not None:
            hi = np.ascontiguousarray(hash_idx, np.uint32).reshape(r, d)
            hs = np.ascontiguousarray(hash_sgn, np.int8).reshape(r, d)
            self._keep = (hi, hs)
            lib().ora_set_hash(self._h, _p(hi), _p(hs))
        if window_lines:
            if log2g != 5 or 32 * window_lines > c:
                raise ValueError("the windowed family needs g = 32 and 32 * window_lines <= c")
            lib().ora_set_option(self._h, b"window_lines", int(window_lines))
        if variant not in ("ga", "pa"):
            raise ValueError("variant must be 'ga' (Algorithm 2) or 'pa' (Algorithm 1)")
        lib().ora_set_option(self._h, b"variant_pa", int(variant == "pa"))
        if P != 1:
            if P < 1 or P * k > d:
                raise ValueError("P must be >= 1 with P*k <= d")
            lib().ora_set_option(self._h, b"P", int(P))
        if freeze_v and variant != "ga":
            raise ValueError("freeze_v applies to Algorithm 2 (gradient averaging) only")
        lib().ora_set_option(self._h, b"freeze_v", int(freeze_v))
        lib().ora_set_option(self._h, b"v_keep", int(v_keep))
        lib().ora_set_option(self._h, b"threads", int(threads))

    def close(self):
        if self._h:
            lib().ora_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_lr(self, lr: float) -> None:
        """Step size alpha_t of the steps taken from now on."""
        lib().ora_set_lr(self._h, float(lr))

    def set_freeze_v(self, on: bool) -> None:
        """Algorithm 2 without h_t and the update of v, vhat (on), or with them (off), from the next step."""
        lib().ora_set_option(self._h, b"freeze_v", int(on))

    def step(self, grads: np.ndarray, x: np.ndarray) -> None:
        """grads: (n, d) float32, C-contiguous; x: (d,) float32, updated in place."""
        assert grads.dtype == np.float32 and grads.flags.c_contiguous and grads.size == self.n * self.d
        assert x.dtype == np.float32 and x.flags.c_contiguous and x.size == self.d
        rc = lib().ora_step(self._h, _p(grads), _p(x))
        if rc != 0:
            raise RuntimeError(f"ora_step failed: {rc}")

    _SHAPES = {"m": "nd", "e": "nd", "v": "d", "vhat": "d", "est": "d", "tables": "nrc", "sum": "rc",
               "vw": "nd", "vhatw": "nd"}

    def field(self, name: str) -> np.ndarray:
        """A numpy VIEW of the oracle's own buffer (writable: teacher forcing writes through it)."""
        ptr = lib().ora_field(self._h, name.encode())
        if not ptr:
            raise KeyError(name)
        if name in ("I", "I_prev", "cand"):
            cnt = int(lib().ora_count(self._h, name.encode()))
            buf = (C.c_uint32 * max(cnt, 1)).from_address(ptr)
            return np.frombuffer(buf, np.uint32, cnt)
        dims = {"n": self.n, "d": self.d, "r": self.r, "c": self.c}
        shape = tuple(dims[ch] for ch in self._SHAPES[name])
        size = int(np.prod(shape))
        buf = (C.c_float * size).from_address(ptr)
        return np.frombuffer(buf, np.float32, size).reshape(shape)

    @property
    def t(self) -> int:
        return int(lib().ora_count(self._h, b"t"))
