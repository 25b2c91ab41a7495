"""Pins for the oracle's log-softmax, softmax backward and log-softmax backward passes.  CPU only."""
from __future__ import annotations

import math

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F32


def f32(a):
    return np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))


def bf(a):
    t = torch.from_numpy(np.asarray(a, np.float64).astype(np.float32)).to(torch.bfloat16)
    return np.ascontiguousarray(t.view(torch.uint16).numpy())


def test_log_softmax_closed_forms_and_invariants():
    # two elements: y = (-log1p(e^(b-a)), (b-a) - log1p(e^(b-a))) for a >= b
    rng = np.random.default_rng(41)
    a, b = rng.uniform(-5, 5, 200), rng.uniform(-5, 5, 200)
    hi, lo = np.maximum(a, b), np.minimum(a, b)
    x = f32(np.stack([hi, lo], axis=1))
    d = x[:, 1].astype(np.float64) - x[:, 0].astype(np.float64)
    _, y64 = oracle.log_softmax(x, F32, want64=True)
    np.testing.assert_allclose(y64[:, 0], -np.log1p(np.exp(d)), rtol=1e-14, atol=1e-15)    # ln(1 + t) in double: absolute 2^-53
    np.testing.assert_allclose(y64[:, 1], d - np.log1p(np.exp(d)), rtol=1e-14, atol=1e-15)
    # uniform rows: -ln n exactly the same for every element; [0, ln 3] -> [ln(1/4), ln(3/4)]
    for n in (1, 2, 7, 1000):
        _, u = oracle.log_softmax(f32(np.full((1, n), 3.25)), F32, want64=True)
        np.testing.assert_allclose(u, -math.log(n), rtol=1e-15, atol=1e-300)
    _, g = oracle.log_softmax(f32([[0.0, math.log(3.0)]]), F32, want64=True)
    x3 = float(np.float32(math.log(3.0)))
    np.testing.assert_allclose(g[0], [-math.log1p(math.exp(x3)), x3 - math.log1p(math.exp(x3))], rtol=1e-15)
    # equals the logarithm of the (separately pinned) softmax, exp sums to one, shift by a representable constant is exact
    xr = f32(rng.standard_normal((9, 301)) * 4)
    _, y64 = oracle.log_softmax(xr, F32, want64=True)
    _, s64 = oracle.softmax(xr, F32, want64=True)
    np.testing.assert_allclose(y64, np.log(s64), rtol=0, atol=1e-13)
    np.testing.assert_allclose(np.exp(y64).sum(axis=1), 1.0, rtol=1e-13)
    shifted = f32(xr.astype(np.float64) * 0 + (xr + np.float32(64.0)))
    if np.array_equal(shifted.astype(np.float64) - 64.0, xr.astype(np.float64)):
        np.testing.assert_array_equal(oracle.log_softmax(shifted, F32, want64=True)[1], y64)
    assert (y64 <= 0).all()
    # no overflow at large offsets
    _, big = oracle.log_softmax(f32([[1e30, 1e30, -1e30]]), F32, want64=True)
    np.testing.assert_allclose(big[0, :2], -math.log(2.0), rtol=1e-15)
    assert big[0, 2] < -1e30


@pytest.mark.parametrize("dt", [F32, BF16])
def test_log_softmax_masks_rounding_and_library(dt):
    rng = np.random.default_rng(42 + dt)
    enc = f32 if dt == F32 else bf
    xv = rng.standard_normal((11, 130)) * 3
    xv[2, 50:] = -np.inf
    xv[3, :] = -np.inf
    xv[4, 0] = 40.0
    x = enc(xv)
    y, y64 = oracle.log_softmax(x, dt, want64=True, nthreads=3)
    wide = x.astype(np.float64) if dt == F32 else oracle.bf16_to_double(x)
    assert np.isneginf(y64[2, 50:]).all() and np.isfinite(y64[2, :50]).all()
    assert np.isneginf(y64[3]).all()                                            # fully masked row: -inf everywhere
    live = [r for r in range(11) if r != 3]
    ref = torch.log_softmax(torch.from_numpy(wide[live]), dim=1).numpy()
    np.testing.assert_allclose(y64[live], ref, rtol=1e-13, atol=1e-13)
    if dt == F32:
        np.testing.assert_array_equal(y[live], y64[live].astype(np.float32))
    else:
        np.testing.assert_array_equal(y, oracle.bf16_from_double(y64))
    np.testing.assert_array_equal(oracle.log_softmax(x, dt, nthreads=1), y)


def test_softmax_bwd_jacobian_finite_differences_and_library():
    rng = np.random.default_rng(43)
    rows, n = 4, 9
    x = f32(rng.standard_normal((rows, n)) * 2)
    _, y64 = oracle.softmax(x, F32, want64=True)
    y = f32(y64)                                                                # the stored forward output
    yd = y.astype(np.float64)
    # (1) one-hot dy = e_i gives column i of the Jacobian: dx_j = y_j (delta_ij - y_i)
    for i in (0, 3, n - 1):
        dy = np.zeros((rows, n)); dy[:, i] = 1.0
        _, dx64, _ = oracle.softmax_bwd(y, f32(dy), F32, want64=True)
        want = yd * ((np.arange(n)[None, :] == i) - yd[:, i:i + 1])
        np.testing.assert_allclose(dx64, want, rtol=1e-14, atol=1e-17)
    # (2) constant dy: dx = y c (1 - sum y), zero up to how far the stored y is from summing to one
    _, dx64, sc = oracle.softmax_bwd(y, f32(np.full((rows, n), 2.5)), F32, want64=True)
    np.testing.assert_allclose(dx64, yd * 2.5 * (1.0 - yd.sum(axis=1, keepdims=True)), rtol=1e-9, atol=1e-18)
    assert np.abs(dx64).max() < 1e-6
    # (3) central differences of the pinned forward pass in double: d softmax(x)^T dy / dx
    dyv = f32(rng.standard_normal((rows, n)))
    xd = x.astype(np.float64)
    def fwd(z):
        e = np.exp(z - z.max(axis=1, keepdims=True)); return e / e.sum(axis=1, keepdims=True)
    num = np.zeros((rows, n))
    h = 1e-6
    for j in range(n):
        zp, zm = xd.copy(), xd.copy()
        zp[:, j] += h; zm[:, j] -= h
        num[:, j] = ((fwd(zp) - fwd(zm)) / (2 * h) * dyv.astype(np.float64)).sum(axis=1)
    _, exact, _ = oracle.softmax_bwd(f32(fwd(xd)), dyv, F32, want64=True)       # y rounded to fp32: error ~1e-7
    np.testing.assert_allclose(exact, num, rtol=0, atol=5e-7)
    # (4) torch autograd in float64 on the same stored y, linearity in dy, and the condition scale
    yt = torch.from_numpy(yd)
    gt = torch.from_numpy(dyv.astype(np.float64))
    ref = (yt * (gt - (yt * gt).sum(dim=1, keepdim=True))).numpy()
    xt = torch.from_numpy(xd).requires_grad_(True)
    torch.softmax(xt, dim=1).backward(gt)
    _, dx64, sc = oracle.softmax_bwd(y, dyv, F32, want64=True, nthreads=2)
    np.testing.assert_allclose(dx64, ref, rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(dx64, xt.grad.numpy(), rtol=0, atol=3e-7)         # autograd uses the unrounded y
    np.testing.assert_allclose(sc, np.abs(yd) * (np.abs(dyv) + (np.abs(yd * dyv)).sum(axis=1, keepdims=True)), rtol=1e-13)
    _, dx2, _ = oracle.softmax_bwd(y, f32(2.0 * dyv.astype(np.float64)), F32, want64=True)
    np.testing.assert_array_equal(dx2, 2.0 * dx64)
    # (5) bf16: stored result is the single rounding of the double
    yb, gb = bf(yd), bf(dyv)
    dxb, dxb64, _ = oracle.softmax_bwd(yb, gb, BF16, want64=True)
    np.testing.assert_array_equal(dxb, oracle.bf16_from_double(dxb64))
    ybd, gbd = oracle.bf16_to_double(yb), oracle.bf16_to_double(gb)
    np.testing.assert_allclose(dxb64, ybd * (gbd - (ybd * gbd).sum(axis=1, keepdims=True)), rtol=1e-13, atol=1e-17)


def test_log_softmax_bwd_jacobian_finite_differences_and_library():
    rng = np.random.default_rng(47)
    rows, n = 4, 9
    x = f32(rng.standard_normal((rows, n)) * 2)
    _, y64 = oracle.log_softmax(x, F32, want64=True)
    y = f32(y64)                                                                # the stored log-probabilities
    yd = y.astype(np.float64)
    p = np.exp(yd)
    # (1) one-hot dy = e_i gives row i of the Jacobian of log-softmax: dx_j = delta_ij - p_j
    for i in (0, 4, n - 1):
        dy = np.zeros((rows, n)); dy[:, i] = 1.0
        _, dx64, _ = oracle.log_softmax_bwd(y, f32(dy), F32, want64=True)
        np.testing.assert_allclose(dx64, (np.arange(n)[None, :] == i) - p, rtol=1e-14, atol=1e-17)
    # (2) the loss -y_t of a cross entropy: dy = -e_t gives p - e_t, whose entries sum to zero as far as p sums to one
    dy = np.zeros((rows, n)); dy[np.arange(rows), [1, 0, 8, 3]] = -1.0
    _, dx64, _ = oracle.log_softmax_bwd(y, f32(dy), F32, want64=True)
    np.testing.assert_allclose(dx64, p + dy, rtol=1e-14, atol=1e-17)
    np.testing.assert_allclose(dx64.sum(axis=1), p.sum(axis=1) - 1.0, rtol=0, atol=1e-15)
    assert np.abs(dx64.sum(axis=1)).max() < 1e-6
    # (3) a gradient that sums to zero passes through unchanged, exactly
    z = rng.standard_normal((rows, n)); z[:, -1] = 0; z = f32(z)
    z[:, -1] = 0
    zs = z.astype(np.float64); zs[:, -1] = -zs[:, :-1].sum(axis=1)
    if np.array_equal(f32(zs).astype(np.float64), zs) and (f32(zs).astype(np.float64).sum(axis=1) == 0).all():
        np.testing.assert_array_equal(oracle.log_softmax_bwd(y, f32(zs), F32, want64=True)[1], zs)
    # (4) central differences of the pinned forward pass in double
    dyv = f32(rng.standard_normal((rows, n)))
    xd = x.astype(np.float64)
    def fwd(zz):
        m = zz.max(axis=1, keepdims=True); return (zz - m) - np.log(np.exp(zz - m).sum(axis=1, keepdims=True))
    num = np.zeros((rows, n))
    h = 1e-6
    for j in range(n):
        zp, zm = xd.copy(), xd.copy()
        zp[:, j] += h; zm[:, j] -= h
        num[:, j] = ((fwd(zp) - fwd(zm)) / (2 * h) * dyv.astype(np.float64)).sum(axis=1)
    _, exact, _ = oracle.log_softmax_bwd(f32(fwd(xd)), dyv, F32, want64=True)   # y rounded to fp32: error ~1e-6
    np.testing.assert_allclose(exact, num, rtol=0, atol=5e-6)
    # (5) torch autograd in float64, the formula re-evaluated on the stored y, linearity in dy, the condition scale
    gt = torch.from_numpy(dyv.astype(np.float64))
    xt = torch.from_numpy(xd).requires_grad_(True)
    torch.log_softmax(xt, dim=1).backward(gt)
    _, dx64, sc = oracle.log_softmax_bwd(y, dyv, F32, want64=True, nthreads=2)
    gd = dyv.astype(np.float64)
    np.testing.assert_allclose(dx64, gd - p * gd.sum(axis=1, keepdims=True), rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(dx64, xt.grad.numpy(), rtol=0, atol=3e-6)         # autograd uses the unrounded y
    np.testing.assert_allclose(sc, np.abs(gd) + p * np.abs(gd).sum(axis=1, keepdims=True), rtol=1e-13)
    _, dx2, _ = oracle.log_softmax_bwd(y, f32(2.0 * gd), F32, want64=True)
    np.testing.assert_array_equal(dx2, 2.0 * dx64)
    # (6) masked entries (y = -inf) pass their gradient through; a fully masked row passes dy through entirely
    ym = y.copy(); ym[1, 3:] = -np.inf; ym[2, :] = -np.inf
    _, dxm, _ = oracle.log_softmax_bwd(ym, dyv, F32, want64=True)
    np.testing.assert_array_equal(dxm[1, 3:], gd[1, 3:])
    np.testing.assert_array_equal(dxm[2], gd[2])
    # (7) bf16: stored result is the single rounding of the double
    yb, gb = bf(yd), bf(dyv)
    dxb, dxb64, _ = oracle.log_softmax_bwd(yb, gb, BF16, want64=True)
    np.testing.assert_array_equal(dxb, oracle.bf16_from_double(dxb64))
    ybd, gbd = oracle.bf16_to_double(yb), oracle.bf16_to_double(gb)
    np.testing.assert_allclose(dxb64, gbd - np.exp(ybd) * gbd.sum(axis=1, keepdims=True), rtol=1e-13, atol=1e-17)
