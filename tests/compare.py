"""Element-by-element comparators between a candidate output and the CPU oracle.

Tolerances (written here so that every parity test uses the same ones):

* fp32 outputs: ``|g - o| <= 1e-5 * c`` where ``o`` is the oracle's unrounded float64 value and ``c`` the
  condition scale of the expression.  For softmax and RMSNorm nothing cancels, so ``c = |o|`` (the literal
  max-relative-error rule).  LayerNorm's ``(x - mu)*rstd*gamma + beta`` crosses zero, where a relative error
  against the cancelled result is unattainable in any fp32 pipeline, so ``c = (|x|+|mu|)*rstd*|gamma| + |beta|``
  (always >= |o|).  One fp32 subnormal quantum (2^-149) of absolute slack covers results the oracle rounds to
  zero or a subnormal.
* bf16 outputs: at most 1 ulp between the candidate's and the oracle's bf16 patterns (distance of the monotone
  integer images, +0 and -0 identified).  LayerNorm additionally passes where
  ``|g - o| <= ulp_bf16(o)/2 + 1e-5 * c`` (same cancellation argument).
* Where x is -inf (masked) a softmax output must be the bit pattern of +0 exactly.
* Row statistics (fp32): mean within ``1e-5 * mean|x|`` of the oracle's, rstd within 1e-5 relative.
"""
from __future__ import annotations

import numpy as np

F32, BF16 = 0, 1
REL = 1e-5
F32_QUANTUM = 2.0 ** -149


def bf16_to_f64(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def to_f64(a: np.ndarray, dt: int) -> np.ndarray:
    return a.astype(np.float64) if dt == F32 else bf16_to_f64(a)


def bf16_key(h: np.ndarray) -> np.ndarray:
    """Monotone integer image of bf16 patterns: -0 and +0 both map to 0."""
    k = (h & 0x7FFF).astype(np.int32)
    return np.where(h & 0x8000, -k, k)


def bf16_ulp_dist(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    return np.abs(bf16_key(a) - bf16_key(b))


def bf16_ulp_of(v64: np.ndarray) -> np.ndarray:
    """Spacing of the bf16 grid at |v| (2^-133 in the subnormal range)."""
    a = np.abs(v64)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return np.exp2(np.maximum(e, -126.0) - 7.0)


class Report(dict):
    @property
    def ok(self) -> bool:
        return self["fail"] == 0

    def __str__(self) -> str:
        return ", ".join(f"{k}={v}" for k, v in self.items())


def _finish(bad: np.ndarray, err: np.ndarray, extra: dict) -> Report:
    r = Report(fail=int(bad.sum()), n=int(bad.size), max_err=float(err.max()) if err.size else 0.0)
    if r["fail"]:
        r["first_bad"] = tuple(int(i) for i in np.argwhere(bad)[0])
    r.update(extra)
    return r


def compare_values(g: np.ndarray, o: np.ndarray, o64: np.ndarray, dt: int, cond: np.ndarray | None = None) -> Report:
    """g, o: candidate / oracle outputs in storage type; o64: oracle before rounding; cond: condition scale
    (None = |o64|, the literal rule)."""
    g64 = to_f64(g, dt)
    diff = np.abs(g64 - o64)
    diff = np.where(np.isnan(diff), np.inf, diff)
    c = np.abs(o64) if cond is None else cond
    if dt == F32:
        bad = diff > REL * c + F32_QUANTUM
        with np.errstate(divide="ignore", invalid="ignore"):
            rel = np.where(c > 0, diff / c, np.where(diff > F32_QUANTUM, np.inf, 0.0))
        return _finish(bad, rel, {"kind": "rel"})
    d = bf16_ulp_dist(g, o)
    bad = d > 1
    if cond is not None:
        bad &= diff > 0.5 * bf16_ulp_of(o64) + REL * c
    lit = int((d > 1).sum())
    return _finish(bad, d, {"kind": "ulp", "literal_fail": lit})


def compare_softmax(g, o, o64, x, dt) -> Report:
    r = compare_values(g, o, o64, dt)
    masked = np.isneginf(to_f64(x, dt))
    nz = int(np.count_nonzero(g.view(np.uint32 if dt == F32 else np.uint16)[masked]))
    r["masked_nonzero"] = nz
    r["fail"] += nz
    return r


def layernorm_cond(x, gamma, beta, stats64, dt) -> np.ndarray:
    x64, g64, b64 = to_f64(x, dt), to_f64(gamma, dt), to_f64(beta, dt)
    mu, rs = stats64[:, 0:1], stats64[:, 1:2]
    return (np.abs(x64) + np.abs(mu)) * rs * np.abs(g64)[None, :] + np.abs(b64)[None, :]


def compare_layernorm(g, o, o64, x, gamma, beta, stats64, dt) -> Report:
    return compare_values(g, o, o64, dt, layernorm_cond(x, gamma, beta, stats64, dt))


def compare_mean(g_mean, stats64, x, dt) -> Report:
    scale = np.abs(to_f64(x, dt)).mean(axis=1)
    diff = np.abs(g_mean.astype(np.float64) - stats64[:, 0])
    diff = np.where(np.isnan(diff), np.inf, diff)
    bad = diff > REL * scale + F32_QUANTUM
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(scale > 0, diff / scale, 0.0)
    return _finish(bad, rel, {"kind": "mean"})


def compare_rstd(g_rstd, rstd64) -> Report:
    diff = np.abs(g_rstd.astype(np.float64) - rstd64)
    diff = np.where(np.isnan(diff), np.inf, diff)
    bad = diff > REL * np.abs(rstd64)
    return _finish(bad, diff / np.abs(rstd64), {"kind": "rstd"})
