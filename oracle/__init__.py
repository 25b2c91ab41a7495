"""ctypes loader for the CPU oracle (``tf_oracle.cpp``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only ``tests/``, the smoke check and the benchmark's
CPU-baseline leg import this package.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.

Arrays are numpy, C-contiguous, shape ``[rows, cols]``; bf16 tensors travel as ``uint16`` bit
patterns.  Every function returns freshly allocated outputs.
"""
from __future__ import annotations

import ctypes
import fcntl
import hashlib
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tf_oracle.cpp"
_LIB = _HERE / "libtf_oracle.so"

F32, BF16 = 0, 1
_NP = {F32: np.float32, BF16: np.uint16}


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no fast-math, no CUDA) unless a build of the same source exists."""
    stamp = _HERE / ".libtf_oracle.stamp"
    digest = hashlib.sha256(_SRC.read_bytes()).hexdigest()
    with open(_HERE / ".build.lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        if force or not _LIB.exists() or not stamp.exists() or stamp.read_text().strip() != digest:
            tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
            subprocess.run(
                ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", "-o", str(tmp), str(_SRC)],
                check=True,
            )
            os.replace(tmp, _LIB)
            stamp.write_text(digest)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        vp, i64, f32, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_int
        lib.oracle_softmax.argtypes = [vp, vp, vp, i64, i64, i32, i32]
        lib.oracle_softmax.restype = i32
        lib.oracle_layernorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, f32, i32, i32]
        lib.oracle_layernorm.restype = i32
        lib.oracle_rmsnorm.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, f32, i32, i32]
        lib.oracle_rmsnorm.restype = i32
        lib.oracle_sin.argtypes = [vp, vp, vp, i64, i32]
        lib.oracle_sin.restype = i32
        lib.oracle_bvecmat.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i32, i32]
        lib.oracle_bvecmat.restype = i32
        lib.oracle_softmax_len.argtypes = [vp, vp, vp, vp, i64, i64, i32, i32]
        lib.oracle_softmax_len.restype = i32
        lib.oracle_log_softmax.argtypes = [vp, vp, vp, i64, i64, i32, i32]
        lib.oracle_log_softmax.restype = i32
        lib.oracle_softmax_bwd.argtypes = [vp, vp, vp, vp, vp, i64, i64, i32, i32]
        lib.oracle_softmax_bwd.restype = i32
        lib.oracle_log_softmax_bwd.argtypes = [vp, vp, vp, vp, vp, i64, i64, i32, i32]
        lib.oracle_log_softmax_bwd.restype = i32
        lib.oracle_norm_bwd.argtypes = [vp] * 14 + [i64, i64, i32, i32, i32]
        lib.oracle_norm_bwd.restype = i32
        lib.oracle_add.argtypes = [vp, vp, vp, vp, i64, i32]
        lib.oracle_add.restype = i32
        lib.oracle_bf16_from_double.argtypes = [vp, vp, i64]
        lib.oracle_bf16_from_double.restype = None
        lib.oracle_bf16_to_double.argtypes = [vp, vp, i64]
        lib.oracle_bf16_to_double.restype = None
        _lib = lib
    return _lib


def _check(a: np.ndarray, dt: int, name: str) -> np.ndarray:
    if a.dtype != _NP[dt] or not a.flags.c_contiguous:
        raise TypeError(f"{name}: want C-contiguous {_NP[dt].__name__}, got {a.dtype}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def softmax(x: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """Row softmax.  Returns ``y`` (and the unrounded float64 result if ``want64``)."""
    _check(x, dt, "x")
    rows, cols = x.shape
    y = np.empty_like(x)
    y64 = np.empty((rows, cols), np.float64) if want64 else None
    rc = _load().oracle_softmax(_p(x), _p(y), _p(y64), rows, cols, dt, nthreads)
    if rc:
        raise ValueError("oracle_softmax: bad argument")
    return (y, y64) if want64 else y


def softmax_len(x: np.ndarray, lengths: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """Row softmax over the first ``lengths[r]`` entries of row r; the rest of the output row is +0 and the rest of
    the input row is not read.  ``lengths``: int32 [rows]."""
    _check(x, dt, "x")
    rows, cols = x.shape
    if lengths.dtype != np.int32 or lengths.shape != (rows,) or not lengths.flags.c_contiguous:
        raise TypeError("lengths: want C-contiguous int32 [rows]")
    y = np.empty_like(x)
    y64 = np.empty((rows, cols), np.float64) if want64 else None
    if _load().oracle_softmax_len(_p(x), _p(lengths), _p(y), _p(y64), rows, cols, dt, nthreads):
        raise ValueError("oracle_softmax_len: bad argument")
    return (y, y64) if want64 else y


def log_softmax(x: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """Row log-softmax.  Returns ``y`` (and the unrounded float64 result if ``want64``)."""
    _check(x, dt, "x")
    rows, cols = x.shape
    y = np.empty_like(x)
    y64 = np.empty((rows, cols), np.float64) if want64 else None
    if _load().oracle_log_softmax(_p(x), _p(y), _p(y64), rows, cols, dt, nthreads):
        raise ValueError("oracle_log_softmax: bad argument")
    return (y, y64) if want64 else y


def softmax_bwd(y: np.ndarray, dy: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """Softmax backward ``dx = y * (dy - sum(y * dy))`` per row.  Returns ``dx`` plus ``(dx64, scale64)`` if ``want64``."""
    _check(y, dt, "y"), _check(dy, dt, "dy")
    if y.shape != dy.shape:
        raise ValueError("y and dy must have the same shape")
    rows, cols = y.shape
    dx = np.empty_like(y)
    dx64 = np.empty((rows, cols), np.float64) if want64 else None
    sc = np.empty((rows, cols), np.float64) if want64 else None
    if _load().oracle_softmax_bwd(_p(y), _p(dy), _p(dx), _p(dx64), _p(sc), rows, cols, dt, nthreads):
        raise ValueError("oracle_softmax_bwd: bad argument")
    return (dx, dx64, sc) if want64 else dx


def log_softmax_bwd(y: np.ndarray, dy: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """Log-softmax backward ``dx = dy - exp(y) * sum(dy)`` per row.  Returns ``dx`` plus ``(dx64, scale64)`` if ``want64``."""
    _check(y, dt, "y"), _check(dy, dt, "dy")
    if y.shape != dy.shape:
        raise ValueError("y and dy must have the same shape")
    rows, cols = y.shape
    dx = np.empty_like(y)
    dx64 = np.empty((rows, cols), np.float64) if want64 else None
    sc = np.empty((rows, cols), np.float64) if want64 else None
    if _load().oracle_log_softmax_bwd(_p(y), _p(dy), _p(dx), _p(dx64), _p(sc), rows, cols, dt, nthreads):
        raise ValueError("oracle_log_softmax_bwd: bad argument")
    return (dx, dx64, sc) if want64 else dx


def layernorm(x, gamma, beta, eps: float, dt: int, want64: bool = False, nthreads: int = 1):
    """Row LayerNorm.  Returns ``(y, mean_f32, rstd_f32)`` plus ``(y64, stats64[rows, 2])`` if ``want64``."""
    _check(x, dt, "x"), _check(gamma, dt, "gamma"), _check(beta, dt, "beta")
    rows, cols = x.shape
    if gamma.shape != (cols,) or beta.shape != (cols,):
        raise ValueError("gamma/beta must have shape [cols]")
    y = np.empty_like(x)
    mean = np.empty(rows, np.float32)
    rstd = np.empty(rows, np.float32)
    y64 = np.empty((rows, cols), np.float64) if want64 else None
    st = np.empty((rows, 2), np.float64) if want64 else None
    rc = _load().oracle_layernorm(_p(x), _p(gamma), _p(beta), _p(y), _p(y64), _p(mean), _p(rstd), _p(st),
                                  rows, cols, eps, dt, nthreads)
    if rc:
        raise ValueError("oracle_layernorm: bad argument")
    return (y, mean, rstd, y64, st) if want64 else (y, mean, rstd)


def rmsnorm(x, w, eps: float, dt: int, want64: bool = False, nthreads: int = 1):
    """Row RMSNorm.  Returns ``(y, rstd_f32)`` plus ``(y64, rstd64[rows])`` if ``want64``."""
    _check(x, dt, "x"), _check(w, dt, "w")
    rows, cols = x.shape
    if w.shape != (cols,):
        raise ValueError("w must have shape [cols]")
    y = np.empty_like(x)
    rstd = np.empty(rows, np.float32)
    y64 = np.empty((rows, cols), np.float64) if want64 else None
    st = np.empty(rows, np.float64) if want64 else None
    rc = _load().oracle_rmsnorm(_p(x), _p(w), _p(y), _p(y64), _p(rstd), _p(st), rows, cols, eps, dt, nthreads)
    if rc:
        raise ValueError("oracle_rmsnorm: bad argument")
    return (y, rstd, y64, st) if want64 else (y, rstd)


def sin(x: np.ndarray, dt: int, want64: bool = False):
    """Element-wise sine of any-shape array.  Returns ``y`` (and the unrounded float64 result if ``want64``)."""
    _check(x, dt, "x")
    y = np.empty_like(x)
    y64 = np.empty(x.shape, np.float64) if want64 else None
    if _load().oracle_sin(_p(x), _p(y), _p(y64), x.size, dt):
        raise ValueError("oracle_sin: bad argument")
    return (y, y64) if want64 else y


def bvecmat(a: np.ndarray, b: np.ndarray, dt: int, want64: bool = False, nthreads: int = 1):
    """C[m,n] = sum_k a[m,k] * b[m,n,k].  Returns ``c`` plus ``(c64, scale64)`` if ``want64``, where
    ``scale64[m,n] = sum_k |a[m,k] * b[m,n,k]|``."""
    _check(a, dt, "a"), _check(b, dt, "b")
    if a.ndim != 2 or b.ndim != 3 or b.shape[0] != a.shape[0] or b.shape[2] != a.shape[1]:
        raise ValueError("want a [M, K] and b [M, N, K]")
    M, K = a.shape
    N = b.shape[1]
    c = np.empty((M, N), _NP[dt])
    c64 = np.empty((M, N), np.float64) if want64 else None
    sc = np.empty((M, N), np.float64) if want64 else None
    if _load().oracle_bvecmat(_p(a), _p(b), _p(c), _p(c64), _p(sc), M, N, K, dt, nthreads):
        raise ValueError("oracle_bvecmat: bad argument")
    return (c, c64, sc) if want64 else c


def add(x: np.ndarray, r: np.ndarray, dt: int, want64: bool = False):
    """h = x + r rounded once to the storage type (the residual add of a fused add-and-normalise)."""
    _check(x, dt, "x"), _check(r, dt, "r")
    if x.shape != r.shape:
        raise ValueError("x and r must have the same shape")
    h = np.empty_like(x)
    h64 = np.empty(x.shape, np.float64) if want64 else None
    if _load().oracle_add(_p(x), _p(r), _p(h), _p(h64), x.size, dt):
        raise ValueError("oracle_add: bad argument")
    return (h, h64) if want64 else h


def add_layernorm(x, r, gamma, beta, eps: float, dt: int, want64: bool = False, nthreads: int = 1):
    """Fused residual add + LayerNorm: ``h = add(x, r)`` then ``layernorm(h)``.  Returns ``(h,) + layernorm(h, ...)``."""
    h = add(x, r, dt)
    return (h,) + tuple(layernorm(h, gamma, beta, eps, dt, want64=want64, nthreads=nthreads))


def add_rmsnorm(x, r, w, eps: float, dt: int, want64: bool = False, nthreads: int = 1):
    """Fused residual add + RMSNorm: ``h = add(x, r)`` then ``rmsnorm(h)``.  Returns ``(h,) + rmsnorm(h, ...)``."""
    h = add(x, r, dt)
    return (h,) + tuple(rmsnorm(h, w, eps, dt, want64=want64, nthreads=nthreads))


def norm_bwd(x, gamma, dy, mean, rstd, dt: int, rms: bool, nthreads: int = 1) -> dict:
    """Backward pass of LayerNorm (``rms=False``) or RMSNorm (``rms=True``) from the forward pass's stored fp32
    ``mean`` / ``rstd`` ([rows]; ``mean`` may be None for RMSNorm).  Returns a dict with ``dx, dgamma, dbeta`` in the
    storage type (``dbeta`` None for RMSNorm), their unrounded float64 versions ``dx64, dg64, db64`` and the condition
    scales ``dx_scale, dg_scale, db_scale``."""
    _check(x, dt, "x"), _check(gamma, dt, "gamma"), _check(dy, dt, "dy")
    rows, cols = x.shape
    if dy.shape != x.shape or gamma.shape != (cols,):
        raise ValueError("shape mismatch")
    rstd = np.ascontiguousarray(rstd, np.float32)
    mean = None if mean is None else np.ascontiguousarray(mean, np.float32)
    out = {"dx": np.empty_like(x), "dgamma": np.empty_like(gamma), "dbeta": None if rms else np.empty_like(gamma),
           "dx64": np.empty((rows, cols)), "dg64": np.empty(cols), "db64": np.empty(cols),
           "dx_scale": np.empty((rows, cols)), "dg_scale": np.empty(cols), "db_scale": np.empty(cols)}
    rc = _load().oracle_norm_bwd(_p(x), _p(gamma), _p(dy), _p(mean), _p(rstd), _p(out["dx"]), _p(out["dgamma"]), _p(out["dbeta"]),
                                 _p(out["dx64"]), _p(out["dg64"]), _p(out["db64"]), _p(out["dx_scale"]), _p(out["dg_scale"]),
                                 _p(out["db_scale"]), rows, cols, int(rms), dt, nthreads)
    if rc:
        raise ValueError("oracle_norm_bwd: bad argument")
    return out


def bf16_from_double(v: np.ndarray) -> np.ndarray:
    """Round float64 values to bf16 bit patterns (nearest-even, subnormals kept)."""
    v = np.ascontiguousarray(v, np.float64)
    out = np.empty(v.shape, np.uint16)
    _load().oracle_bf16_from_double(_p(v), _p(out), v.size)
    return out


def bf16_to_double(h: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float64 (exact)."""
    h = np.ascontiguousarray(h, np.uint16)
    out = np.empty(h.shape, np.float64)
    _load().oracle_bf16_to_double(_p(h), _p(out), h.size)
    return out
