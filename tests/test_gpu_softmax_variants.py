"""Log-softmax forward and softmax backward through the C ABI against the CPU oracle, element by element.

Tolerances (derived from the arithmetic, fp32 throughout):
* log-softmax: |g - o| <= 1e-5 * (|x_j - m| + |ln S|) + 32 * 2^-24.  The relative part is the rule of the other ops on
  the two terms that are subtracted; the absolute part covers ln S, whose argument S >= 1 is an fp32 sum of up to
  2^17 terms (a few 2^-24 of absolute error however small ln S itself is).  bf16 outputs add half a bf16 ulp.
  Where x_j = -inf the output must be -inf.
* softmax backward: |g - o| <= 1e-5 * |y_j| (|dy_j| + sum_k |y_k dy_k|) -- dy_j - sum y dy cancels, so the bound is
  stated against what is subtracted -- plus one fp32 subnormal quantum; bf16 outputs add half a bf16 ulp.
* log-softmax backward: |g - o| <= 1e-5 * (|dy_j| + exp(y_j) sum_k |dy_k|), the same rule on dy_j - exp(y_j) sum dy (the
  exponential is one rounding of y log2 e + 64 and one MUFU op: at most 6e-6 relative at |y| ~ 100, 1e-6 at |y| ~ 20)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import compare
import oracle
import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu
F32, BF16 = inputs.F32, inputs.BF16


def check_close(g, o, o64, cond, dt, abs_extra, what):
    g64 = compare.to_f64(g, dt)
    both_ninf = np.isneginf(g64) & np.isneginf(o64)
    with np.errstate(invalid="ignore"):
        diff = np.where(both_ninf, 0.0, np.abs(g64 - o64))
    diff = np.where(np.isnan(diff), np.inf, diff)
    tol = compare.REL * cond + abs_extra + compare.F32_QUANTUM
    if dt == BF16:
        with np.errstate(invalid="ignore"):
            tol = tol + 0.5 * compare.bf16_ulp_of(np.where(np.isfinite(o64), o64, 1.0))
        bad = (diff > tol) & (compare.bf16_ulp_dist(g, o) > 1)
    else:
        bad = diff > tol
    assert not bad.any(), (what, int(bad.sum()), tuple(int(i) for i in np.argwhere(bad)[0]), float(diff[bad].max()))


def run_log_softmax(dt, rows, cols, seed=1, offset=0, std=3.0, mask=False, inplace=False):
    x = inputs.normal((rows, cols), dt, seed, 0, 0.0, std)
    if mask:
        ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
        x[::3, cols // 2:] = ninf
        if rows > 1:
            x[1, :] = ninf                                        # a fully masked row
    ref, ref64 = oracle.log_softmax(x, dt, want64=True, nthreads=8)
    xd = parity.to_dev(x, dt, offset)
    y = tf.tf_log_softmax_fwd(xd, xd if inplace else parity.guarded(tuple(xd.shape), xd.dtype, offset, name="y"))
    torch.cuda.synchronize()
    x64 = compare.to_f64(x, dt)
    with np.errstate(invalid="ignore"):
        m = x64.max(axis=1, keepdims=True)
        d = np.where(np.isfinite(x64), np.abs(x64 - m), 0.0)
        lns = np.where(np.isfinite(m), np.abs(ref64 - (x64 - m)), 0.0)
    cond = np.where(np.isfinite(ref64), d + np.nan_to_num(lns, nan=0.0, posinf=0.0, neginf=0.0), 0.0)
    got = parity.to_host(y, dt)
    assert np.array_equal(np.isneginf(compare.to_f64(got, dt)), np.isneginf(ref64)), "masked entries must come out as -inf"
    check_close(got, ref, ref64, cond, dt, 32 * 2.0 ** -24, ("log_softmax", dt, rows, cols, offset))


def run_softmax_bwd(dt, rows, cols, seed=1, offset=0, inplace=False):
    x = inputs.normal((rows, cols), dt, seed, 0, 0.0, 2.0)
    y = oracle.softmax(x, dt, nthreads=8)                         # a real forward output as the stored y
    dy = inputs.normal((rows, cols), dt, seed + 7, 1, 0.1, 1.5)
    ref, ref64, sc = oracle.softmax_bwd(y, dy, dt, want64=True, nthreads=8)
    yd, gd = parity.to_dev(y, dt, offset), parity.to_dev(dy, dt, offset)
    dx = tf.tf_softmax_bwd(yd, gd, gd if inplace else parity.guarded(tuple(yd.shape), yd.dtype, offset, name="dx"))
    torch.cuda.synchronize()
    check_close(parity.to_host(dx, dt), ref, ref64, sc, dt, 0.0, ("softmax_bwd", dt, rows, cols, offset))


def run_log_softmax_bwd(dt, rows, cols, seed=1, offset=0, inplace=False, mask=False, std=2.0):
    x = inputs.normal((rows, cols), dt, seed, 0, 0.0, std)
    if mask:
        ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
        x[::3, cols // 2:] = ninf
        if rows > 1:
            x[1, :] = ninf                                        # a fully masked row: y = -inf, dx = dy
    y = oracle.log_softmax(x, dt, nthreads=8)                     # real stored log-probabilities
    dy = inputs.normal((rows, cols), dt, seed + 7, 1, 0.1, 1.5)
    ref, ref64, sc = oracle.log_softmax_bwd(y, dy, dt, want64=True, nthreads=8)
    yd, gd = parity.to_dev(y, dt, offset), parity.to_dev(dy, dt, offset)
    dx = tf.tf_log_softmax_bwd(yd, gd, gd if inplace else parity.guarded(tuple(yd.shape), yd.dtype, offset, name="dx"))
    torch.cuda.synchronize()
    check_close(parity.to_host(dx, dt), ref, ref64, sc, dt, 0.0, ("log_softmax_bwd", dt, rows, cols, offset))


@pytest.mark.parametrize("dt", [F32, BF16])
def test_log_softmax_bwd_over_edge_widths(dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 3 * ne, 64, 256, 1000 // ne * ne, 1024, 2048 + ne, 4096, 5120, 16384, 32768 + ne, 65536, 200000 // ne * ne):
        for rows in (1, 9, 300):
            if rows * cols > (1 << 22):
                rows = max(3, (1 << 22) // cols)
            run_log_softmax_bwd(dt, rows, cols, seed=cols + rows, mask=cols >= 64)
    run_log_softmax_bwd(dt, 2000, 512)
    run_log_softmax_bwd(dt, 40, 2048, inplace=True)
    run_log_softmax_bwd(dt, 20, 4096, std=30.0)                   # log-probabilities down to -100 and below: tiny and zero exp(y)
    for cols, offset in ((1001, 0), (7, 0), (1024, 1), (4099, 3)):
        run_log_softmax_bwd(dt, 9, cols, offset=offset)
    assert tf.tf_log_softmax_bwd(torch.empty(0, 64, device="cuda"), torch.empty(0, 64, device="cuda")).shape == (0, 64)


def test_log_softmax_bwd_is_the_cross_entropy_gradient():
    torch.manual_seed(0)
    x = torch.randn(300, 5000, device="cuda", requires_grad=True)
    t = torch.randint(0, 5000, (300,), device="cuda")
    torch.nn.functional.cross_entropy(x, t, reduction="sum").backward()
    y = tf.tf_log_softmax_fwd(x.detach())
    dy = torch.zeros_like(y); dy[torch.arange(300), t] = -1.0
    dx = tf.tf_log_softmax_bwd(y, dy)
    assert (dx - x.grad).abs().max().item() < 2e-6


@pytest.mark.parametrize("dt", [F32, BF16])
def test_log_softmax_over_edge_widths(dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 2 * ne, 64, 256, 1000 // ne * ne, 1024, 2048, 4096, 5120, 8192, 16384, 32768, 65536, 131072, 200000 // ne * ne):
        run_log_softmax(dt, max(3, min(200, (1 << 21) // cols)), cols, seed=cols)
    run_log_softmax(dt, 0, 64)
    # many rows of 8-64 KiB (the form that stages the row in shared memory): rows that fill one to four steps exactly, ragged
    # ones, masks and a fully masked row, in place; 295 rows of the same width take the register forms
    es = 4 if dt == F32 else 2
    for kib, rows in ((8, 320), (12, 300), (16, 333), (24, 296), (32, 300), (48, 297), (64, 296)):
        cols = kib * 1024 // es
        run_log_softmax(dt, rows, cols, seed=kib, mask=True)
        run_log_softmax(dt, rows, cols - ne, seed=kib + 1, mask=kib % 16 == 0, std=12.0)
    run_log_softmax(dt, 310, 10240 // es + 3 * ne, seed=5, inplace=True)
    run_log_softmax(dt, 295, 16384 // es, seed=6, mask=True)
    run_log_softmax(dt, 301, 1024, mask=True)
    run_log_softmax(dt, 9, 40000, mask=True, std=20.0)
    run_log_softmax(dt, 50, 2048, inplace=True)
    for cols, offset in ((1001, 0), (7, 0), (1024, 1), (4099, 3)):           # odd widths and misaligned bases: scalar passes
        run_log_softmax(dt, 9, cols, offset=offset, mask=True)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_softmax_bwd_over_edge_widths(dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 2 * ne, 64, 256, 1000 // ne * ne, 1024, 2048, 4096, 5120, 8192, 16384, 32768, 65536, 200000 // ne * ne):
        run_softmax_bwd(dt, max(3, min(200, (1 << 21) // cols)), cols, seed=cols)
    run_softmax_bwd(dt, 0, 64)
    run_softmax_bwd(dt, 50, 2048, inplace=True)
    for cols, offset in ((1001, 0), (7, 0), (1024, 1), (4099, 3)):
        run_softmax_bwd(dt, 9, cols, offset=offset)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_cluster_per_row_and_streamed_forms(dt):
    """A thread-block cluster shares a row: forced on short rows (ragged slices, empty slices, masked slices) and chosen by
    itself beyond 32 KiB; with clusters switched off the same long rows take the streamed passes."""
    ne = 4 if dt == F32 else 8
    try:
        for cluster in (2, 4, 8):
            tf.tf_softmax_variants_force(cluster)
            for rows, cols in ((1, ne), (5, 3 * ne), (33, 256), (700, 1000 // ne * ne), (64, 4096), (9, 40000 // ne * ne)):
                run_log_softmax(dt, rows, cols, seed=cols + cluster, mask=True)
                run_softmax_bwd(dt, rows, cols, seed=cols + cluster)
                run_log_softmax_bwd(dt, rows, cols, seed=cols + cluster, mask=True)
            run_log_softmax(dt, 40, 2048, seed=3, inplace=True)
            run_softmax_bwd(dt, 40, 2048, seed=3, inplace=True)
        tf.tf_softmax_variants_force(1)
        for rows, cols in ((6, 32768), (3, 200000 // ne * ne)):
            run_log_softmax(dt, rows, cols, seed=cols, mask=True)
            run_softmax_bwd(dt, rows, cols, seed=cols)
            run_log_softmax_bwd(dt, rows, cols, seed=cols, mask=True)
    finally:
        tf.tf_softmax_variants_force(0)
    for rows, cols in ((70, 16384), (6, 32768), (5, 65536 + ne), (3, 131072)):      # automatic: clusters where the slices fit
        run_log_softmax(dt, rows, cols, seed=cols, mask=True)
        run_softmax_bwd(dt, rows, cols, seed=cols)
        run_log_softmax_bwd(dt, rows, cols, seed=cols, mask=True)
    with pytest.raises(tf.TfError):
        tf.tf_softmax_variants_force(3)


def test_peaked_rows_and_closed_forms():
    # one dominant entry: y_max = -ln S is tiny and must still be right to the absolute part of the tolerance
    x = torch.full((4, 1024), -20.0, device="cuda")
    x[:, 5] = 10.0
    y = tf.tf_log_softmax_fwd(x).cpu().numpy().astype(np.float64)
    lns = np.log1p(1023 * np.exp(-30.0))
    assert np.abs(y[:, 5] + lns).max() < 4 * 2.0 ** -24
    np.testing.assert_allclose(y[:, 0], -30.0 - lns, rtol=1e-6)
    # uniform rows: -ln n; softmax backward of a constant gradient is zero to rounding
    u = tf.tf_log_softmax_fwd(torch.zeros(2, 4096, device="cuda")).cpu().numpy()
    np.testing.assert_allclose(u, -np.log(4096.0), rtol=1e-6)
    ysm = torch.softmax(torch.randn(8, 512, device="cuda"), dim=1)
    dx = tf.tf_softmax_bwd(ysm, torch.full_like(ysm, 3.0)).cpu().numpy()
    assert np.abs(dx).max() < 1e-6
    # against torch autograd in fp32 (context, loose)
    xt = torch.randn(16, 1000, device="cuda", requires_grad=True)
    g = torch.randn(16, 1000, device="cuda")
    yt = torch.softmax(xt, dim=1)
    yt.backward(g)
    ours = tf.tf_softmax_bwd(yt.detach().contiguous(), g)
    assert (ours - xt.grad).abs().max().item() < 1e-6


def test_bad_arguments():
    L = tf.lib()
    p = torch.zeros(64, device="cuda").data_ptr()
    assert L.tf_log_softmax_fwd(None, p, 1, 8, 0, None) == 1
    assert L.tf_log_softmax_fwd(p, p, 1, 0, 0, None) == 1
    assert L.tf_log_softmax_fwd(p, p, 1, 8, 3, None) == 1
    assert L.tf_log_softmax_fwd(p, p, 0, 8, 0, None) == 0
    assert L.tf_softmax_bwd(p, None, p, 1, 8, 0, None) == 1
    assert L.tf_softmax_bwd(p, p, None, 1, 8, 0, None) == 1
    assert L.tf_softmax_bwd(p, p, p, 0, 8, 1, None) == 0


@pytest.mark.parametrize("dt,rows,cols", [(BF16, 16384, 8192), (BF16, 32768, 4096), (F32, 65536, 1024), (BF16, 524288, 256), (BF16, 2048, 32768),
                                          (F32, 1024, 131072)])
def test_shapes_of_the_bench_table_every_element(dt, rows, cols):
    """The shapes `bench.py --table softmaxvariants` times (the two widest on a quarter / half of their rows), both ops,
    every element against the oracle."""
    run_log_softmax(dt, rows, cols, seed=cols)
    run_softmax_bwd(dt, rows, cols, seed=cols)
    run_log_softmax_bwd(dt, rows, cols, seed=cols)
