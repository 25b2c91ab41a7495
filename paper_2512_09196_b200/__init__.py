"""Row-wise softmax / LayerNorm / RMSNorm forward kernels for B200 behind a C ABI (``libtf.so``).

This module is the thin binding: it marshals torch tensors (used only as device memory and for the
current stream) into the C calls declared in ``include/tf.h`` and does no arithmetic of its own.
There is no fallback: if ``libtf.so`` has not been built, every call raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libtf.so"

TF_F32, TF_BF16 = 0, 1
TF_OP_SOFTMAX, TF_OP_LAYERNORM, TF_OP_RMSNORM = 0, 1, 2
OP_CODE = {"softmax": TF_OP_SOFTMAX, "layernorm": TF_OP_LAYERNORM, "rmsnorm": TF_OP_RMSNORM}
TF_OK = 0
STATUS_NAMES = {0: "TF_OK", 1: "TF_ERR_INVALID_ARG", 2: "TF_ERR_UNSUPPORTED", 3: "TF_ERR_CUDA", 4: "TF_ERR_TIMEOUT",
                5: "TF_ERR_NOMEM"}

# every symbol include/tf.h declares
EXPORTS = ("tf_softmax_fwd", "tf_softmax_fwd_noalloc", "tf_layernorm_fwd", "tf_rmsnorm_fwd", "tf_tune", "tf_tune_like", "tf_tune_report", "tf_copy", "tf_sin_fwd", "tf_bvecmat_fwd", "tf_add_layernorm_fwd", "tf_add_rmsnorm_fwd", "tf_tune_add", "tf_softmax_len_fwd", "tf_log_softmax_fwd", "tf_softmax_bwd", "tf_log_softmax_bwd", "tf_norm_bwd_workspace_bytes", "tf_layernorm_bwd", "tf_rmsnorm_bwd", "tf_norm_bwd_force", "tf_softmax_variants_force", "tf_tune_norm_bwd", "tf_tune_norm_bwd_report", "tf_norm_bwd_choice",
           "tf_status_string",
           "tf_last_cuda_error", "tf_device_status", "tf_force_plan", "tf_query_choice", "tf_candidate_count",
           "tf_candidate", "tf_clear_cache", "tf_launch_count", "tf_debug_wait_probe", "tf_debug_tune_inject_timeout", "tf_refine_hint", "tf_tune_last_hint")


class TfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == 3 and _lib is not None:
            detail = f" (cudaError {_lib.tf_last_cuda_error()})"
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}{detail}")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (``python -m paper_2512_09196_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_2512_09196_b200.build); "
                               "there is no fallback path")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i64, i32, f32, cp, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_char_p,
                                     ctypes.c_size_t)
        L.tf_softmax_fwd.argtypes = [vp, vp, i64, i64, i32, vp]
        L.tf_softmax_fwd_noalloc.argtypes = [vp, vp, i64, i64, i32, vp]
        L.tf_layernorm_fwd.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, f32, i32, vp]
        L.tf_rmsnorm_fwd.argtypes = [vp, vp, vp, vp, i64, i64, f32, i32, vp]
        L.tf_tune.argtypes = [i32, i64, i64, i32]
        L.tf_copy.argtypes = [vp, vp, i64, vp]
        L.tf_add_layernorm_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, f32, i32, vp]
        L.tf_add_rmsnorm_fwd.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, f32, i32, vp]
        L.tf_tune_add.argtypes = [i32, i64, i64, i32]
        L.tf_softmax_len_fwd.argtypes = [vp, vp, vp, i64, i64, i32, vp]
        L.tf_log_softmax_fwd.argtypes = [vp, vp, i64, i64, i32, vp]
        L.tf_softmax_bwd.argtypes = [vp, vp, vp, i64, i64, i32, vp]
        L.tf_log_softmax_bwd.argtypes = [vp, vp, vp, i64, i64, i32, vp]
        L.tf_norm_bwd_workspace_bytes.argtypes = [i64, i64]
        L.tf_norm_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.tf_layernorm_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, i64, i64, i32, vp]
        L.tf_norm_bwd_force.argtypes = [i32, i32, i32]
        L.tf_tune_norm_bwd.argtypes = [i32, i64, i64, i32]
        L.tf_tune_norm_bwd_report.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(f32), ctypes.POINTER(f32)]
        L.tf_norm_bwd_choice.argtypes = [i32, i64, i64, i32, ctypes.c_char_p, ctypes.c_size_t]
        L.tf_softmax_variants_force.argtypes = [i32]
        L.tf_rmsnorm_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, i64, i64, i32, vp]
        L.tf_bvecmat_fwd.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, i32, vp]
        L.tf_sin_fwd.argtypes = [vp, vp, i64, i32, i32, i32, vp]
        L.tf_tune_like.argtypes = [i32, vp, vp, vp, i64, i64, i32]
        L.tf_tune_report.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(f32), ctypes.POINTER(f32)]
        L.tf_status_string.argtypes = [i32]
        L.tf_status_string.restype = cp
        L.tf_last_cuda_error.argtypes = []
        L.tf_device_status.argtypes = []
        L.tf_force_plan.argtypes = [i32, cp]
        L.tf_query_choice.argtypes = [i32, i64, i64, i32, i32, ctypes.c_char_p, sz]
        L.tf_candidate_count.argtypes = [i32, i64, i64, i32]
        L.tf_candidate.argtypes = [i32, i64, i64, i32, i32, ctypes.c_char_p, sz]
        L.tf_debug_wait_probe.argtypes = [vp, i64, vp, vp]
        L.tf_debug_wait_probe.restype = i32
        L.tf_debug_tune_inject_timeout.argtypes = [cp]
        L.tf_debug_tune_inject_timeout.restype = i32
        L.tf_refine_hint.argtypes = [i32, i64, i64, i32, cp, ctypes.c_char_p, sz]
        L.tf_refine_hint.restype = i32
        L.tf_tune_last_hint.argtypes = [ctypes.c_char_p, sz]
        L.tf_tune_last_hint.restype = i32
        L.tf_clear_cache.argtypes = []
        L.tf_clear_cache.restype = None
        L.tf_launch_count.argtypes = []
        L.tf_launch_count.restype = i64
        for name in ("tf_softmax_fwd", "tf_softmax_fwd_noalloc", "tf_layernorm_fwd", "tf_rmsnorm_fwd", "tf_tune", "tf_tune_like", "tf_tune_report", "tf_copy", "tf_sin_fwd", "tf_bvecmat_fwd", "tf_add_layernorm_fwd", "tf_add_rmsnorm_fwd", "tf_tune_add", "tf_softmax_len_fwd", "tf_log_softmax_fwd", "tf_softmax_bwd", "tf_layernorm_bwd", "tf_rmsnorm_bwd",
                     "tf_last_cuda_error", "tf_device_status", "tf_force_plan", "tf_query_choice",
                     "tf_candidate_count", "tf_candidate"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def _dt(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return TF_F32
    if t.dtype == torch.bfloat16:
        return TF_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: fp32 and bf16 only")


def _check2d(x, name="x"):
    if not x.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if x.dim() != 2 or not x.is_contiguous():
        raise ValueError(f"{name} must be a contiguous [rows, cols] tensor")


def _like(x, t, name, shape=None, dtype=None):
    """``t`` must be a contiguous tensor on ``x``'s device with this shape and dtype (default: ``x``'s own).  The C ABI sees
    only pointers, so a tensor that is too small, of another type or on another GPU would make a kernel read or write out
    of bounds: it is refused here, before the call."""
    shape = tuple(x.shape) if shape is None else tuple(shape)
    dtype = x.dtype if dtype is None else dtype
    if not t.is_cuda or t.device != x.device:
        raise ValueError(f"{name} must be on the same CUDA device as x ({x.device}), got {t.device}")
    if t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if tuple(t.shape) != shape:
        raise ValueError(f"{name} must have shape {shape}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


def _param(x, t, name):
    """An affine parameter vector: [cols], x's dtype and device."""
    return _like(x, t, name, shape=(x.shape[1],))


def _stat(x, t, name):
    """A per-row statistic: fp32 [rows] on x's device."""
    import torch
    return _like(x, t, name, shape=(x.shape[0],), dtype=torch.float32)


def _stream(x) -> int:
    import torch
    try:                                    # raw handle of the current stream without building a Stream object
        return torch._C._cuda_getCurrentRawStream(x.device.index)
    except AttributeError:
        return torch.cuda.current_stream(x.device).cuda_stream


class _on_device:
    """Makes x's device current for the call; free when it already is."""
    __slots__ = ("guard",)

    def __init__(self, x):
        import torch
        self.guard = None if x.device.index == torch.cuda.current_device() else torch.cuda.device(x.device)

    def __enter__(self):
        if self.guard is not None:
            self.guard.__enter__()

    def __exit__(self, *exc):
        if self.guard is not None:
            self.guard.__exit__(*exc)


def _ok(status: int, where: str):
    if status != TF_OK:
        raise TfError(status, where)


def tf_softmax_fwd(x, y=None):
    """Softmax over the last axis of a contiguous CUDA [rows, cols] tensor (fp32 or bf16); ``y`` may alias ``x``."""
    import torch
    _check2d(x)
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    rows, cols = x.shape
    with _on_device(x):
        _ok(lib().tf_softmax_fwd(x.data_ptr(), y.data_ptr(), rows, cols, _dt(x), _stream(x)), "tf_softmax_fwd")
    return y


def tf_softmax_len_fwd(x, lengths, y=None):
    """Softmax of row r over its first ``lengths[r]`` entries (int32 CUDA tensor [rows]); the rest of the output row is
    +0 and the rest of the input row is never read.  ``y`` may alias ``x``."""
    import torch
    _check2d(x)
    rows, cols = x.shape
    if not lengths.is_cuda or lengths.dtype != torch.int32 or lengths.shape != (rows,) or not lengths.is_contiguous():
        raise ValueError("lengths must be a contiguous int32 CUDA tensor of shape [rows]")
    if lengths.device != x.device:
        raise ValueError("lengths must be on x's device")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    with _on_device(x):
        _ok(lib().tf_softmax_len_fwd(x.data_ptr(), lengths.data_ptr(), y.data_ptr(), rows, cols, _dt(x), _stream(x)),
            "tf_softmax_len_fwd")
    return y


def tf_log_softmax_fwd(x, y=None):
    """Log-softmax over the last axis of a contiguous CUDA [rows, cols] tensor (fp32 or bf16); ``y`` may alias ``x``."""
    import torch
    _check2d(x)
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    rows, cols = x.shape
    with _on_device(x):
        _ok(lib().tf_log_softmax_fwd(x.data_ptr(), y.data_ptr(), rows, cols, _dt(x), _stream(x)), "tf_log_softmax_fwd")
    return y


def tf_softmax_bwd(y, dy, dx=None):
    """Softmax backward ``dx = y * (dy - sum(y * dy, -1))`` from the stored forward output ``y`` and the gradient ``dy``."""
    import torch
    _check2d(y, "y")
    _check2d(dy, "dy")
    _like(y, dy, "dy")
    dx = torch.empty_like(y) if dx is None else _like(y, dx, "dx")
    rows, cols = y.shape
    with _on_device(y):
        _ok(lib().tf_softmax_bwd(y.data_ptr(), dy.data_ptr(), dx.data_ptr(), rows, cols, _dt(y), _stream(y)), "tf_softmax_bwd")
    return dx


def tf_log_softmax_bwd(y, dy, dx=None):
    """Log-softmax backward ``dx = dy - exp(y) * sum(dy, -1)`` from the stored log-probabilities ``y`` and the gradient ``dy``."""
    import torch
    _check2d(y, "y")
    _check2d(dy, "dy")
    _like(y, dy, "dy")
    dx = torch.empty_like(y) if dx is None else _like(y, dx, "dx")
    rows, cols = y.shape
    with _on_device(y):
        _ok(lib().tf_log_softmax_bwd(y.data_ptr(), dy.data_ptr(), dx.data_ptr(), rows, cols, _dt(y), _stream(y)), "tf_log_softmax_bwd")
    return dx


def _norm_bwd_workspace(x):
    import torch
    rows, cols = x.shape
    n = lib().tf_norm_bwd_workspace_bytes(rows, cols)
    return torch.empty(max(1, n // 4), dtype=torch.float32, device=x.device), n


def tf_layernorm_bwd(x, gamma, dy, mean, rstd, dx=None, dgamma=None, dbeta=None):
    """LayerNorm backward from the forward pass's stored fp32 ``mean`` / ``rstd``.  Returns ``(dx, dgamma, dbeta)``."""
    import torch
    _check2d(x)
    _like(x, dy, "dy")
    _param(x, gamma, "gamma")
    _stat(x, mean, "mean")
    _stat(x, rstd, "rstd")
    rows, cols = x.shape
    dx = torch.empty_like(x) if dx is None else _like(x, dx, "dx")
    dgamma = torch.empty_like(gamma) if dgamma is None else _param(x, dgamma, "dgamma")
    dbeta = torch.empty_like(gamma) if dbeta is None else _param(x, dbeta, "dbeta")
    ws, n = _norm_bwd_workspace(x)
    with _on_device(x):
        _ok(lib().tf_layernorm_bwd(x.data_ptr(), gamma.data_ptr(), dy.data_ptr(), mean.data_ptr(), rstd.data_ptr(), dx.data_ptr(),
                                   dgamma.data_ptr(), dbeta.data_ptr(), ws.data_ptr(), n, rows, cols, _dt(x), _stream(x)),
            "tf_layernorm_bwd")
    return dx, dgamma, dbeta


def tf_rmsnorm_bwd(x, weight, dy, rstd, dx=None, dweight=None):
    """RMSNorm backward from the forward pass's stored fp32 ``rstd``.  Returns ``(dx, dweight)``."""
    import torch
    _check2d(x)
    _like(x, dy, "dy")
    _param(x, weight, "weight")
    _stat(x, rstd, "rstd")
    rows, cols = x.shape
    dx = torch.empty_like(x) if dx is None else _like(x, dx, "dx")
    dweight = torch.empty_like(weight) if dweight is None else _param(x, dweight, "dweight")
    ws, n = _norm_bwd_workspace(x)
    with _on_device(x):
        _ok(lib().tf_rmsnorm_bwd(x.data_ptr(), weight.data_ptr(), dy.data_ptr(), rstd.data_ptr(), dx.data_ptr(), dweight.data_ptr(),
                                 ws.data_ptr(), n, rows, cols, _dt(x), _stream(x)), "tf_rmsnorm_bwd")
    return dx, dweight


def tf_tune_norm_bwd(op, rows: int, cols: int, dt: int):
    """Measure-and-keep over the forms of the norm backward pass (``op``: "layernorm" or "rmsnorm") on this shape; later
    calls use the winner.  Returns ``(forms_timed, automatic_us, best_us)``."""
    _ok(lib().tf_tune_norm_bwd(OP_CODE[op] if isinstance(op, str) else int(op), rows, cols, dt), "tf_tune_norm_bwd")
    n, a, b = ctypes.c_int32(0), ctypes.c_float(0), ctypes.c_float(0)
    _ok(lib().tf_tune_norm_bwd_report(ctypes.byref(n), ctypes.byref(a), ctypes.byref(b)), "tf_tune_norm_bwd_report")
    return n.value, a.value, b.value


def tf_norm_bwd_choice(op, rows: int, cols: int, dt: int) -> str:
    """What the norm backward pass of ``op`` would use now for this shape (forced > tuned > automatic)."""
    buf = ctypes.create_string_buffer(64)
    _ok(lib().tf_norm_bwd_choice(OP_CODE[op] if isinstance(op, str) else int(op), rows, cols, dt, buf, 64), "tf_norm_bwd_choice")
    return buf.value.decode()


def tf_softmax_variants_force(cluster=0):
    """Test and bench hook: CTAs per row of ``tf_log_softmax_fwd`` / ``tf_softmax_bwd`` (0 = automatic, 1 = never a cluster)."""
    _ok(lib().tf_softmax_variants_force(int(cluster)), "tf_softmax_variants_force")


def tf_norm_bwd_force(path=0, stages=0, cluster=0):
    """Test and bench hook: which form of the norm backward passes runs (0 = automatic everywhere); see ``tf.h``."""
    _ok(lib().tf_norm_bwd_force(int(path), int(stages), int(cluster)), "tf_norm_bwd_force")


def tf_softmax_fwd_noalloc(x, y):
    """Softmax through the entry point that never allocates device memory: for processes that gave all free device
    memory to their own pool at start-up, or loops that cannot afford an allocation call's possible synchronisation.
    ``y`` must be preallocated (it may alias ``x``); rows <= 8192, 16-byte aligned tensors.  Calls that may overlap on
    the GPU share one fixed scratch array inside the library and must be ordered by the caller."""
    _check2d(x)
    _like(x, y, "y")
    rows, cols = x.shape
    with _on_device(x):
        _ok(lib().tf_softmax_fwd_noalloc(x.data_ptr(), y.data_ptr(), rows, cols, _dt(x), _stream(x)), "tf_softmax_fwd_noalloc")
    return y


def tf_copy(x, y=None):
    """Calibration copy of a contiguous CUDA tensor with the library's own streaming kernel."""
    import torch
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA tensor")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    with _on_device(x):
        _ok(lib().tf_copy(x.data_ptr(), y.data_ptr(), x.numel() * x.element_size(), _stream(x)), "tf_copy")
    return y


def tf_sin_fwd(x, y=None, threads: int = 0, vectors_per_thread: int = 0):
    """Element-wise sine of a contiguous CUDA tensor (fp32 or bf16); ``threads`` and ``vectors_per_thread`` (1, 2, 4, 8)
    are the launch geometry (0 = defaults)."""
    import torch
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA tensor")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    with _on_device(x):
        _ok(lib().tf_sin_fwd(x.data_ptr(), y.data_ptr(), x.numel(), _dt(x), threads, vectors_per_thread, _stream(x)), "tf_sin_fwd")
    return y


def tf_bvecmat_fwd(a, b, c=None, threads: int = 0, lanes: int = 0, rows: int = 0, ksplit: int = 0):
    """C[m,n] = sum_k A[m,k] * B[m,n,k] for contiguous CUDA tensors a [M, K], b [M, N, K] (fp32 or bf16)."""
    import torch
    if not (a.is_cuda and b.is_cuda and a.is_contiguous() and b.is_contiguous()) or a.dim() != 2 or b.dim() != 3:
        raise ValueError("a must be a contiguous CUDA [M, K] tensor and b a contiguous CUDA [M, N, K] tensor")
    M, K = a.shape
    if b.shape[0] != M or b.shape[2] != K or b.dtype != a.dtype:
        raise ValueError("shape or dtype mismatch between a and b")
    N = b.shape[1]
    if b.device != a.device:
        raise ValueError("a and b must be on the same device")
    c = torch.empty((M, N), dtype=a.dtype, device=a.device) if c is None else _like(a, c, "c", shape=(M, N))
    with _on_device(a):
        _ok(lib().tf_bvecmat_fwd(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, _dt(a), threads, lanes, rows, ksplit,
                                 _stream(a)),
            "tf_bvecmat_fwd")
    return c


def tf_layernorm_fwd(x, gamma, beta, eps: float, y=None, mean=None, rstd=None, want_stats: bool = True):
    """LayerNorm forward; returns ``(y, mean, rstd)`` (fp32 [rows] statistics, or None if ``want_stats`` is False
    and none were passed in)."""
    import torch
    _check2d(x)
    rows, cols = x.shape
    _param(x, gamma, "gamma")
    _param(x, beta, "beta")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    if mean is not None:
        _stat(x, mean, "mean")
    elif want_stats:
        mean = torch.empty(rows, dtype=torch.float32, device=x.device)
    if rstd is not None:
        _stat(x, rstd, "rstd")
    elif want_stats:
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device)
    with _on_device(x):
        _ok(lib().tf_layernorm_fwd(x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), y.data_ptr(),
                                   mean.data_ptr() if mean is not None else None,
                                   rstd.data_ptr() if rstd is not None else None,
                                   rows, cols, eps, _dt(x), _stream(x)), "tf_layernorm_fwd")
    return y, mean, rstd


def tf_add_layernorm_fwd(x, r, gamma, beta, eps: float, h=None, y=None, want_stats: bool = True, mean=None, rstd=None):
    """Fused residual add + LayerNorm: ``h = x + r`` (rounded to the storage type), ``y = layernorm(h)``.
    Returns ``(h, y, mean, rstd)``; pass ``h=r`` to update the residual stream in place."""
    import torch
    _check2d(x)
    _like(x, r, "r")
    _param(x, gamma, "gamma")
    _param(x, beta, "beta")
    rows, cols = x.shape
    h = torch.empty_like(x) if h is None else _like(x, h, "h")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    if mean is not None:
        _stat(x, mean, "mean")
    elif want_stats:
        mean = torch.empty(rows, dtype=torch.float32, device=x.device)
    if rstd is not None:
        _stat(x, rstd, "rstd")
    elif want_stats:
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device)
    with _on_device(x):
        _ok(lib().tf_add_layernorm_fwd(x.data_ptr(), r.data_ptr(), gamma.data_ptr(), beta.data_ptr(), h.data_ptr(), y.data_ptr(),
                                       mean.data_ptr() if mean is not None else None, rstd.data_ptr() if rstd is not None else None,
                                       rows, cols, eps, _dt(x), _stream(x)), "tf_add_layernorm_fwd")
    return h, y, mean, rstd


def tf_add_rmsnorm_fwd(x, r, weight, eps: float, h=None, y=None, want_rstd: bool = False, rstd=None):
    """Fused residual add + RMSNorm: ``h = x + r`` (rounded to the storage type), ``y = rmsnorm(h)``.
    Returns ``(h, y, rstd)``; pass ``h=r`` to update the residual stream in place."""
    import torch
    _check2d(x)
    _like(x, r, "r")
    _param(x, weight, "weight")
    rows, cols = x.shape
    h = torch.empty_like(x) if h is None else _like(x, h, "h")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    if rstd is not None:
        _stat(x, rstd, "rstd")
    elif want_rstd:
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device)
    with _on_device(x):
        _ok(lib().tf_add_rmsnorm_fwd(x.data_ptr(), r.data_ptr(), weight.data_ptr(), h.data_ptr(), y.data_ptr(),
                                     rstd.data_ptr() if rstd is not None else None, rows, cols, eps, _dt(x), _stream(x)),
            "tf_add_rmsnorm_fwd")
    return h, y, rstd


def tf_rmsnorm_fwd(x, weight, eps: float, y=None, rstd=None, want_rstd: bool = False):
    """RMSNorm forward; returns ``(y, rstd)`` (``rstd`` is None unless requested or passed in)."""
    import torch
    _check2d(x)
    rows, cols = x.shape
    _param(x, weight, "weight")
    y = torch.empty_like(x) if y is None else _like(x, y, "y")
    if rstd is not None:
        _stat(x, rstd, "rstd")
    elif want_rstd:
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device)
    with _on_device(x):
        _ok(lib().tf_rmsnorm_fwd(x.data_ptr(), weight.data_ptr(), y.data_ptr(),
                                 rstd.data_ptr() if rstd is not None else None, rows, cols, eps, _dt(x), _stream(x)),
            "tf_rmsnorm_fwd")
    return y, rstd


def tf_tune(op, rows: int, cols: int, dt: int, like=None) -> dict:
    """Times the candidate plans for this problem on the current device, caches the winner, and returns
    ``{"timed": n, "heuristic_us": a, "best_us": b, "plan": "..."}``.  ``like=(x, p0, p1)`` (CUDA tensors, p0/p1 may be
    None) times on a copy of the caller's data instead of synthetic values."""
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    if like is None:
        _ok(lib().tf_tune(code, rows, cols, dt), "tf_tune")
    else:
        x, p0, p1 = like
        _check2d(x)
        if tuple(x.shape) != (rows, cols) or _dt(x) != dt:
            raise ValueError("like[0] must be the [rows, cols] tensor of this dtype")
        for q, nm in ((p0, "like[1]"), (p1, "like[2]")):
            if q is not None:
                _param(x, q, nm)
        _ok(lib().tf_tune_like(code, x.data_ptr(), p0.data_ptr() if p0 is not None else None,
                               p1.data_ptr() if p1 is not None else None, rows, cols, dt), "tf_tune_like")
    n, a, b = ctypes.c_int(), ctypes.c_float(), ctypes.c_float()
    lib().tf_tune_report(ctypes.byref(n), ctypes.byref(a), ctypes.byref(b))
    return {"timed": n.value, "heuristic_us": a.value, "best_us": b.value, "plan": tf_query_choice(code, rows, cols, dt)}


def tf_tune_add(op, rows: int, cols: int, dt: int) -> dict:
    """``tf_tune`` for the fused residual-add form of LayerNorm / RMSNorm (own cache entry).  Returns
    ``{"timed": n, "heuristic_us": a, "best_us": b}``; raises TfError(TF_ERR_UNSUPPORTED) when only the two-kernel route
    can serve the shape."""
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    _ok(lib().tf_tune_add(code, rows, cols, dt), "tf_tune_add")
    n, a, b = ctypes.c_int(), ctypes.c_float(), ctypes.c_float()
    lib().tf_tune_report(ctypes.byref(n), ctypes.byref(a), ctypes.byref(b))
    return {"timed": n.value, "heuristic_us": a.value, "best_us": b.value}


def tf_force_plan(op, plan: str | None):
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    _ok(lib().tf_force_plan(code, plan.encode() if plan else None), "tf_force_plan")


def tf_query_choice(op, rows: int, cols: int, dt: int, aligned: bool = True) -> str:
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    buf = ctypes.create_string_buffer(256)
    _ok(lib().tf_query_choice(code, rows, cols, dt, int(aligned), buf, 256), "tf_query_choice")
    return buf.value.decode()


def tf_candidates(op, rows: int, cols: int, dt: int) -> list[str]:
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    n = lib().tf_candidate_count(code, rows, cols, dt)
    if n < 0:
        raise TfError(1, "tf_candidate_count")
    out = []
    buf = ctypes.create_string_buffer(256)
    for i in range(n):
        _ok(lib().tf_candidate(code, rows, cols, dt, i, buf, 256), "tf_candidate")
        out.append(buf.value.decode())
    return out


def tf_device_status():
    _ok(lib().tf_device_status(), "tf_device_status")


def _parse_hint(text: str) -> dict:
    out = {}
    for part in text.split(" "):
        if "=" in part:
            k, v = part.split("=", 1)
            if k == "first":
                out[k] = [q for q in v.split(";") if q]
            elif k == "rule":
                out[k] = v
            else:
                out[k] = float(v)
    return out


def tf_refine_hint(op, rows: int, cols: int, dt: int, plan: str) -> dict:
    """The refinement hint for ``plan`` on this shape: ``{"rule": ..., "regs": ..., "ctas_per_sm": ..., "occupancy": ...,
    "waves": ..., "tail": ..., "inflight_kb": ..., "vs_copy": ..., "first": [plans the refinement would try first]}``."""
    code = OP_CODE[op] if isinstance(op, str) else int(op)
    buf = ctypes.create_string_buffer(1024)
    _ok(lib().tf_refine_hint(code, rows, cols, dt, plan.encode(), buf, 1024), "tf_refine_hint")
    return _parse_hint(buf.value.decode())


def tf_tune_last_hint() -> dict:
    """The hint ``tf_tune`` computed for the heuristic plan in its last run on this thread."""
    buf = ctypes.create_string_buffer(256)
    _ok(lib().tf_tune_last_hint(buf, 256), "tf_tune_last_hint")
    return _parse_hint(buf.value.decode())


def tf_debug_wait_probe(src, budget_cycles: int = 2_000_000) -> bool:
    """Test hook: runs the library's bounded wait on a barrier that cannot complete; returns True if the wait gave up
    (the status word is then set: ``tf_device_status()`` raises TF_ERR_TIMEOUT once).  ``src``: any CUDA tensor of at
    least 16 bytes."""
    import torch
    if not src.is_cuda or src.numel() * src.element_size() < 16:
        raise ValueError("src must be a CUDA tensor of at least 16 bytes")
    flag = torch.zeros(1, dtype=torch.int32, device=src.device)
    with _on_device(src):
        _ok(lib().tf_debug_wait_probe(src.data_ptr(), int(budget_cycles), flag.data_ptr(), _stream(src)), "tf_debug_wait_probe")
    return bool(flag.item())


def tf_debug_tune_inject_timeout(plan_prefix: str | None):
    """Test hook: ``tf_tune`` treats candidates whose plan starts with ``plan_prefix`` as timed out (None switches it off)."""
    _ok(lib().tf_debug_tune_inject_timeout(plan_prefix.encode() if plan_prefix else None), "tf_debug_tune_inject_timeout")


def tf_clear_cache():
    lib().tf_clear_cache()


def tf_launch_count() -> int:
    return int(lib().tf_launch_count())
