"""Seeded synthetic workloads (numpy, host memory) for the three row-wise ops and the batched vector-matrix product.

Data generation only: nothing here computes a softmax or a norm.  The generator is a small C file
(``gen.c``, built with gcc + OpenMP) so that the 2 GiB workload is produced in seconds; every element
is a pure function of (seed, stream, global index), hence ``generate(row0, nrows)`` returns exactly
the rows ``[row0, row0 + nrows)`` of the full tensor.

bf16 tensors are ``uint16`` bit patterns; view them with ``torch.from_numpy(a).view(torch.bfloat16)``.
"""
from __future__ import annotations

import ctypes
import fcntl
import hashlib
import os
import subprocess
from dataclasses import dataclass, field
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gen.c"
_LIB = _HERE / "libtf_inputs.so"

F32, BF16 = 0, 1
NP_DTYPE = {F32: np.float32, BF16: np.uint16}
ELEM_SIZE = {F32: 4, BF16: 2}
OPS = ("softmax", "layernorm", "rmsnorm")


def build(force: bool = False) -> Path:
    """Compile the generator with gcc + OpenMP unless a build of the same source exists."""
    stamp = _HERE / ".libtf_inputs.stamp"
    digest = hashlib.sha256(_SRC.read_bytes()).hexdigest()
    with open(_HERE / ".build.lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        if force or not _LIB.exists() or not stamp.exists() or stamp.read_text().strip() != digest:
            tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
            subprocess.run(["gcc", "-std=c11", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"],
                           check=True)
            os.replace(tmp, _LIB)
            stamp.write_text(digest)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        vp, i64, u64, i32, f64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_int, ctypes.c_double
        lib.tfgen_normal.argtypes = [vp, i64, i32, u64, u64, f64, f64, i64]
        lib.tfgen_uniform.argtypes = [vp, i64, i32, u64, u64, f64, f64, i64]
        lib.tfgen_normal_outliers.argtypes = [vp, i64, i32, u64, f64, f64, f64, f64, i64]
        lib.tfgen_tail_mask.argtypes = [vp, i64, i64, i32, i64, i64]
        for f in (lib.tfgen_normal, lib.tfgen_uniform, lib.tfgen_normal_outliers, lib.tfgen_tail_mask):
            f.restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def normal(shape, dt: int, seed: int, stream: int, mean: float, std: float, idx0: int = 0) -> np.ndarray:
    out = np.empty(shape, NP_DTYPE[dt])
    _load().tfgen_normal(_ptr(out), out.size, dt, seed, stream, mean, std, idx0)
    return out


def uniform(shape, dt: int, seed: int, stream: int, lo: float, hi: float, idx0: int = 0) -> np.ndarray:
    out = np.empty(shape, NP_DTYPE[dt])
    _load().tfgen_uniform(_ptr(out), out.size, dt, seed, stream, lo, hi, idx0)
    return out


def normal_outliers(shape, dt: int, seed: int, mean: float, std: float, p: float, factor: float,
                    idx0: int = 0) -> np.ndarray:
    out = np.empty(shape, NP_DTYPE[dt])
    _load().tfgen_normal_outliers(_ptr(out), out.size, dt, seed, mean, std, p, factor, idx0)
    return out


def tail_mask_(x: np.ndarray, dt: int, step: int, row0: int = 0) -> np.ndarray:
    """In place: global row r = row0 + i has its last (r*step mod cols) columns set to -inf."""
    rows, cols = x.shape
    _load().tfgen_tail_mask(_ptr(x), rows, cols, dt, step, row0)
    return x


@dataclass(frozen=True)
class Workload:
    """One (op, dtype, shape, distribution) point.  ``params`` describes gamma/beta/w as
    ``("uniform", lo, hi)`` or ``("normal", mean, std)``."""
    name: str
    op: str
    dt: int
    rows: int
    cols: int
    seed: int
    x_mean: float = 0.0
    x_std: float = 1.0
    eps: float = 0.0
    outlier_p: float = 0.0
    outlier_factor: float = 1.0
    mask_step: int = 0
    scale: tuple = ("uniform", 0.5, 1.5)      # gamma (LayerNorm) / weight (RMSNorm)
    shift: tuple = ("uniform", 0.5, 1.5)      # beta (LayerNorm)
    extra: dict = field(default_factory=dict, compare=False)

    @property
    def elem_size(self) -> int:
        return ELEM_SIZE[self.dt]

    @property
    def dtype_name(self) -> str:
        return "f32" if self.dt == F32 else "bf16"

    def algorithmic_bytes(self, rows: int | None = None, with_rms_rstd: bool = False) -> int:
        """Bytes the method must move: x in once, y out once, parameters once, row statistics once."""
        r = self.rows if rows is None else rows
        es, c = self.elem_size, self.cols
        if self.op == "softmax":
            return 2 * r * c * es
        if self.op == "layernorm":
            return 2 * r * c * es + 2 * c * es + 8 * r
        return 2 * r * c * es + c * es + (4 * r if with_rms_rstd else 0)

    def _param(self, spec, stream):
        kind, a, b = spec
        if kind == "uniform":
            return uniform((self.cols,), self.dt, self.seed, stream, a, b)
        return normal((self.cols,), self.dt, self.seed, stream, a, b)

    def generate(self, row0: int = 0, nrows: int | None = None) -> dict:
        """Rows ``[row0, row0 + nrows)`` of x plus the full parameter vectors."""
        n = self.rows - row0 if nrows is None else nrows
        if row0 < 0 or n < 0 or row0 + n > self.rows:
            raise ValueError("row range outside the workload")
        idx0 = row0 * self.cols
        if self.outlier_p > 0.0:
            x = normal_outliers((n, self.cols), self.dt, self.seed, self.x_mean, self.x_std, self.outlier_p,
                                self.outlier_factor, idx0)
        else:
            x = normal((n, self.cols), self.dt, self.seed, 0, self.x_mean, self.x_std, idx0)
        if self.mask_step:
            tail_mask_(x, self.dt, self.mask_step, row0)
        out = {"x": x}
        if self.op == "layernorm":
            out["gamma"] = self._param(self.scale, 1)
            out["beta"] = self._param(self.shift, 2)
        elif self.op == "rmsnorm":
            out["w"] = self._param(self.scale, 1)
        return out


def config(i: int) -> Workload:
    """The four fixed configurations (0-based): small fp32 softmax, bf16 LayerNorm, bf16 RMSNorm with
    outliers, bf16 tail-masked softmax with 131,072 columns."""
    if i == 0:
        return Workload("softmax_f32_1024x1024", "softmax", F32, 1024, 1024, seed=0)
    if i == 1:
        return Workload("layernorm_bf16_8192x4096", "layernorm", BF16, 8192, 4096, seed=1, x_mean=0.5, x_std=3.0,
                        eps=1e-5, scale=("uniform", 0.5, 1.5), shift=("normal", 0.0, 0.1))
    if i == 2:
        return Workload("rmsnorm_bf16_16384x8192_outliers", "rmsnorm", BF16, 16384, 8192, seed=2, eps=1e-6,
                        outlier_p=0.01, outlier_factor=100.0, scale=("normal", 1.0, 0.1))
    if i == 3:
        return Workload("masked_softmax_bf16_4096x131072", "softmax", BF16, 4096, 131072, seed=3, x_std=10.0,
                        mask_step=32)
    raise IndexError(i)


SWEEP_COLS = (64, 128, 256, 512, 1000, 1024, 2048, 4096, 5120, 8192, 12288, 16384, 32768, 65536)
SWEEP_BYTES = 256 << 20


def sweep_point(op: str, dt: int, cols: int, input_bytes: int = SWEEP_BYTES) -> Workload:
    """One point of the shape sweep: rows = floor(input_bytes / (cols * elem_size)), x ~ N(0,1),
    affine parameters ~ U(0.5, 1.5), seed = cols, eps as in the fixed configurations."""
    rows = input_bytes // (cols * ELEM_SIZE[dt])
    eps = {"softmax": 0.0, "layernorm": 1e-5, "rmsnorm": 1e-6}[op]
    name = f"sweep_{op}_{'f32' if dt == F32 else 'bf16'}_{rows}x{cols}"
    return Workload(name, op, dt, rows, cols, seed=cols, eps=eps)


def sweep(input_bytes: int = SWEEP_BYTES):
    return [sweep_point(op, dt, c, input_bytes) for op in OPS for dt in (F32, BF16) for c in SWEEP_COLS]


def shard_rows(rows: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous row block ``(row0, nrows)`` of rank ``rank`` when ``rows`` independent rows are split
    over ``world`` ranks (the first ``rows % world`` ranks get one extra row)."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("bad rank/world")
    q, r = divmod(rows, world)
    n = q + (1 if rank < r else 0)
    return rank * q + min(rank, r), n


@dataclass(frozen=True)
class VecMat:
    """One point of the batched vector-matrix workload  C[m,n] = sum_k A[m,k] * B[m,n,k]:  A [M, K] ~ N(0, 1),
    B [M, N, K] ~ N(0, 1) (streams 0 and 1 of the counter-based generator)."""
    name: str
    dt: int
    M: int
    N: int
    K: int
    seed: int

    @property
    def elem_size(self) -> int:
        return ELEM_SIZE[self.dt]

    @property
    def dtype_name(self) -> str:
        return "f32" if self.dt == F32 else "bf16"

    def algorithmic_bytes(self) -> int:
        """A in once, B in once, C out once."""
        return (self.M * self.K + self.M * self.N * self.K + self.M * self.N) * self.elem_size

    def generate(self) -> dict:
        return {"a": normal((self.M, self.K), self.dt, self.seed, 0, 0.0, 1.0),
                "b": normal((self.M, self.N, self.K), self.dt, self.seed, 1, 0.0, 1.0)}


VECMAT_KS = (64, 256, 1000, 1024, 4096, 16384)
VECMAT_BYTES = 512 << 20


def vecmat_point(dt: int, K: int, M: int = 64, b_bytes: int = VECMAT_BYTES) -> VecMat:
    """N = floor(b_bytes / (M * K * elem_size)): B holds about b_bytes whatever K is."""
    N = max(1, b_bytes // (M * K * ELEM_SIZE[dt]))
    return VecMat(f"bvecmat_{'f32' if dt == F32 else 'bf16'}_{M}x{N}x{K}", dt, M, N, K, seed=K)


def vecmat_headline() -> VecMat:
    """bf16, B = 1.5 GiB: the traffic that the paper's reported runtime and memory throughput for this kernel imply."""
    return VecMat("bvecmat_bf16_96x2048x4096", BF16, 96, 2048, 4096, seed=96)


def vecmat_sweep():
    return [vecmat_headline()] + [vecmat_point(dt, K) for dt in (F32, BF16) for K in VECMAT_KS]
