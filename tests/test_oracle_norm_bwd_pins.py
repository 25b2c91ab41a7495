"""Pins for the oracle's LayerNorm / RMSNorm backward passes.  CPU only."""
from __future__ import annotations

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


def forward64(x, g, b, eps, rms):
    if rms:
        r = 1.0 / np.sqrt((x * x).mean(axis=1, keepdims=True) + eps)
        return x * r * g, None, r[:, 0]
    mu = x.mean(axis=1, keepdims=True)
    r = 1.0 / np.sqrt(((x - mu) ** 2).mean(axis=1, keepdims=True) + eps)
    return (x - mu) * r * g + b, mu[:, 0], r[:, 0]


@pytest.mark.parametrize("rms", [False, True])
def test_central_differences_of_the_forward_pass(rms):
    rng = np.random.default_rng(51 + rms)
    rows, n, eps = 3, 7, 1e-5
    x = f32(rng.standard_normal((rows, n)) * 2 + 0.5).astype(np.float64)
    g = f32(rng.uniform(0.5, 1.5, n)).astype(np.float64)
    b = f32(rng.standard_normal(n) * 0.1).astype(np.float64)
    dy = f32(rng.standard_normal((rows, n))).astype(np.float64)
    _, mu, r = forward64(x, g, b, eps, rms)
    out = oracle.norm_bwd(f32(x), f32(g), f32(dy), None if rms else mu, r, F32, rms)
    loss = lambda xx, gg, bb: (forward64(xx, gg, bb, eps, rms)[0] * dy).sum()
    h = 1e-6
    num_dx = np.zeros_like(x)
    for i in range(rows):
        for j in range(n):
            xp, xm = x.copy(), x.copy()
            xp[i, j] += h; xm[i, j] -= h
            num_dx[i, j] = (loss(xp, g, b) - loss(xm, g, b)) / (2 * h)
    num_dg, num_db = np.zeros(n), np.zeros(n)
    for j in range(n):
        gp, gm = g.copy(), g.copy(); gp[j] += h; gm[j] -= h
        num_dg[j] = (loss(x, gp, b) - loss(x, gm, b)) / (2 * h)
        bp, bm = b.copy(), b.copy(); bp[j] += h; bm[j] -= h
        num_db[j] = (loss(x, g, bp) - loss(x, g, bm)) / (2 * h)
    # the oracle uses the statistics rounded to fp32 (as stored by the forward pass): agreement to about 1e-6
    np.testing.assert_allclose(out["dx64"], num_dx, rtol=0, atol=3e-6)
    np.testing.assert_allclose(out["dg64"], num_dg, rtol=0, atol=3e-6)
    if not rms:
        np.testing.assert_allclose(out["db64"], num_db, rtol=0, atol=3e-6)


@pytest.mark.parametrize("rms", [False, True])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_invariants_library_and_rounding(rms, dt):
    rng = np.random.default_rng(53 + 2 * rms + dt)
    rows, n, eps = 19, 96, 1e-5
    enc = f32 if dt == F32 else bf
    wide = (lambda a: a.astype(np.float64)) if dt == F32 else oracle.bf16_to_double
    x, g, dy = enc(rng.standard_normal((rows, n)) * 3 + 1), enc(rng.uniform(0.5, 1.5, n)), enc(rng.standard_normal((rows, n)))
    xd, gd, dyd = wide(x), wide(g), wide(dy)
    _, mu, r = forward64(xd, gd, 0.0, eps, rms)
    mu32 = None if rms else mu.astype(np.float32)
    r32 = r.astype(np.float32)
    out = oracle.norm_bwd(x, g, dy, mu32, r32, dt, rms, nthreads=3)
    rr = r32.astype(np.float64)[:, None]
    xh = xd * rr if rms else (xd - mu32.astype(np.float64)[:, None]) * rr
    # identities of the formula: sum_j dx_j xh_j = rstd (sum g xh) (1 - mean xh^2) - rstd mean(g) sum xh, which vanishes when the
    # statistics are exact and eps = 0 (dx orthogonal to the normalised row); for LayerNorm sum_j dx_j = -rstd mean(g xh) sum xh
    gg = dyd * gd
    sgx, sx, sg = (gg * xh).sum(axis=1), xh.sum(axis=1), gg.sum(axis=1)
    mg = 0.0 if rms else sg / n
    want = rr[:, 0] * (sgx * (1.0 - (xh * xh).mean(axis=1)) - mg * sx)
    np.testing.assert_allclose((out["dx64"] * xh).sum(axis=1), want, rtol=0, atol=1e-12 * n)
    assert np.abs(want).max() < 1e-3                       # small: the stored statistics are nearly exact, eps is small
    if not rms:
        np.testing.assert_allclose(out["dx64"].sum(axis=1), -rr[:, 0] * (sgx / n) * sx, rtol=0, atol=1e-12 * n)
        np.testing.assert_allclose(out["db64"], dyd.sum(axis=0), rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(out["db_scale"], np.abs(dyd).sum(axis=0), rtol=1e-13)
    np.testing.assert_allclose(out["dg64"], (dyd * xh).sum(axis=0), rtol=1e-12, atol=1e-12)
    # torch float64 autograd on the same inputs (its statistics are unrounded: agreement to fp32 rounding of mean/rstd)
    xt = torch.from_numpy(xd).requires_grad_(True)
    gt = torch.from_numpy(gd).requires_grad_(True)
    if rms:
        yt = xt * torch.rsqrt((xt * xt).mean(dim=1, keepdim=True) + eps) * gt
    else:
        bt = torch.zeros(n, dtype=torch.float64, requires_grad=True)
        yt = torch.nn.functional.layer_norm(xt, (n,), gt, bt, eps)
    yt.backward(torch.from_numpy(dyd))
    np.testing.assert_allclose(out["dx64"], xt.grad.numpy(), rtol=0, atol=2e-6)
    np.testing.assert_allclose(out["dg64"], gt.grad.numpy(), rtol=0, atol=2e-5)
    # stored outputs are single roundings; threads change nothing
    if dt == F32:
        np.testing.assert_array_equal(out["dx"], out["dx64"].astype(np.float32))
        np.testing.assert_array_equal(out["dgamma"], out["dg64"].astype(np.float32))
    else:
        np.testing.assert_array_equal(out["dx"], oracle.bf16_from_double(out["dx64"]))
        np.testing.assert_array_equal(out["dgamma"], oracle.bf16_from_double(out["dg64"]))
    one = oracle.norm_bwd(x, g, dy, mu32, r32, dt, rms, nthreads=1)
    np.testing.assert_array_equal(one["dx64"], out["dx64"])
    np.testing.assert_array_equal(one["dg64"], out["dg64"])
    assert (out["dbeta"] is None) == bool(rms)
