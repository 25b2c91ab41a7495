"""LayerNorm / RMSNorm backward through the C ABI against the CPU oracle.

Tolerances (fp32 arithmetic; written against what is subtracted or summed, as for the other ops):
* dx: |g - o| <= 1e-5 * rstd (|g_j| + mean|g| + |xh_j| mean|g xh|) plus half a bf16 ulp for bf16 outputs.
* dgamma / dbeta: |g - o| <= 1e-5 * sum_rows |term| plus half a bf16 ulp: the fp32 column sums run over at most a few
  thousand rows per accumulator, so their summation error stays two orders below that."""
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


def close(g, o, o64, cond, dt, what):
    g64 = compare.to_f64(g, dt)
    diff = np.abs(g64 - o64)
    diff = np.where(np.isnan(diff), np.inf, diff)
    tol = compare.REL * cond + compare.F32_QUANTUM
    if dt == BF16:
        bad = (diff > tol + 0.5 * compare.bf16_ulp_of(o64)) & (compare.bf16_ulp_dist(g, o) > 1)
    else:
        bad = diff > tol
    assert not bad.any(), (what, int(bad.sum()), tuple(int(i) for i in np.argwhere(bad)[0]), float(diff[bad].max()))


def run_case(rms, dt, rows, cols, seed=1, offset=0, inplace=False):
    op = "rmsnorm" if rms else "layernorm"
    w = inputs.Workload(f"bwd-{op}-{dt}-{rows}x{cols}", op, dt, rows, cols, seed=seed, eps=1e-6 if rms else 1e-5, x_mean=0.4, x_std=2.0)
    data = w.generate()
    gamma = data["w"] if rms else data["gamma"]
    dy = inputs.normal((rows, cols), dt, seed + 99, 3, 0.05, 1.0)
    # the stored statistics of the forward pass, as the oracle's forward produces them
    if rms:
        _, rstd = oracle.rmsnorm(data["x"], gamma, w.eps, dt, nthreads=8)
        mean = None
    else:
        _, mean, rstd = oracle.layernorm(data["x"], gamma, data["beta"], w.eps, dt, nthreads=8)
    ref = oracle.norm_bwd(data["x"], gamma, dy, mean, rstd, dt, rms, nthreads=8)
    xd, gd, dyd = parity.to_dev(data["x"], dt, offset), parity.to_dev(gamma, dt, offset), parity.to_dev(dy, dt, offset)
    rs = torch.from_numpy(rstd).cuda()
    dxg = dyd if inplace else parity.guarded(tuple(xd.shape), xd.dtype, offset, name="dx")      # every output between guard bands
    pg = lambda name: parity.guarded(tuple(gd.shape), gd.dtype, offset, name=name)
    if rms:
        dx, dg = tf.tf_rmsnorm_bwd(xd, gd, dyd, rs, dx=dxg, dweight=pg("dweight"))
        db = None
    else:
        dx, dg, db = tf.tf_layernorm_bwd(xd, gd, dyd, torch.from_numpy(mean).cuda(), rs, dx=dxg, dgamma=pg("dgamma"), dbeta=pg("dbeta"))
    torch.cuda.synchronize()
    tf.tf_device_status()
    what = (op, dt, rows, cols, offset)
    if rows:
        close(parity.to_host(dx, dt), ref["dx"], ref["dx64"], ref["dx_scale"], dt, what + ("dx",))
    close(parity.to_host(dg, dt), ref["dgamma"], ref["dg64"], ref["dg_scale"], dt, what + ("dgamma",))
    if not rms:
        close(parity.to_host(db, dt), ref["dbeta"], ref["db64"], ref["db_scale"], dt, what + ("dbeta",))


@pytest.mark.parametrize("rms", [False, True])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_edge_shapes(rms, dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 3 * ne, 64, 256, 1000 // ne * ne, 1024, 2048, 4096, 5120, 8192, 8192 + ne, 16384, 40000 // ne * ne):
        for rows in (1, 7, 700):
            if rows * cols > (1 << 22):
                rows = max(3, (1 << 22) // cols)
            run_case(rms, dt, rows, cols, seed=cols + rows)
    run_case(rms, dt, 5000, 512)                                   # more rows than CTAs: several rows per accumulator
    run_case(rms, dt, 0, 64)
    run_case(rms, dt, 300, 2048, inplace=True)
    for cols, offset in ((1001, 0), (7, 0), (1024, 1), (4099, 3)):           # odd widths and misaligned bases: the plain kernels
        run_case(rms, dt, 9, cols, offset=offset)


@pytest.mark.parametrize("rms", [False, True])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_every_form_on_shapes_both_serve(rms, dt):
    """The register form and the staged form (both group widths, several ring depths) give the oracle's result."""
    ne = 4 if dt == F32 else 8
    try:
        for path, stages in ((1, 0), (2, 0), (2, 2), (3, 3), (3, 8), (4, 0), (4, 2)):
            tf.tf_norm_bwd_force(path, stages)
            for rows, cols in ((1, ne), (5, 3 * ne), (77, 256), (1500, 512), (700, 1024), (333, 4096), (130, 5120), (64, 8192)):
                run_case(rms, dt, rows, cols, seed=rows + cols + path)
            run_case(rms, dt, 300, 2048, inplace=True)
    finally:
        tf.tf_norm_bwd_force(0, 0, 0)
    with pytest.raises(tf.TfError):
        tf.tf_norm_bwd_force(5, 0)
    with pytest.raises(tf.TfError):
        tf.tf_norm_bwd_force(2, 9)
    with pytest.raises(tf.TfError):
        tf.tf_norm_bwd_force(0, 0, 3)


@pytest.mark.parametrize("rms", [False, True])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_cluster_per_row(rms, dt):
    """A thread-block cluster shares each row: forced on short rows (ragged slices, an empty slice, one row, fewer rows
    than clusters, many rows per cluster) and chosen by itself beyond what one CTA holds."""
    ne = 4 if dt == F32 else 8
    try:
        for cluster, stages in ((2, 0), (4, 2), (8, 0)):
            tf.tf_norm_bwd_force(0, stages, cluster)
            for rows, cols in ((1, ne), (3, 5 * ne), (40, 256), (2000, 512), (300, 1024 + ne), (100, 4096), (37, 8192)):
                run_case(rms, dt, rows, cols, seed=rows + cols + cluster)
            run_case(rms, dt, 64, 2048, inplace=True)
    finally:
        tf.tf_norm_bwd_force(0, 0, 0)
    for rows, cols in ((200, 16384), (31, 16384 + ne), (20, 32768), (9, 65536)):
        run_case(rms, dt, rows, cols, seed=cols)
    try:                                                           # the same long rows without clusters: the streamed form
        tf.tf_norm_bwd_force(0, 0, 1)
        run_case(rms, dt, 50, 16384, seed=5)
    finally:
        tf.tf_norm_bwd_force(0, 0, 0)


def test_matches_torch_autograd_in_fp32():
    torch.manual_seed(0)
    x = torch.randn(257, 1024, device="cuda", requires_grad=True)
    g = (torch.rand(1024, device="cuda") + 0.5).requires_grad_(True)
    b = torch.zeros(1024, device="cuda", requires_grad=True)
    dy = torch.randn(257, 1024, device="cuda")
    y = torch.nn.functional.layer_norm(x, (1024,), g, b, 1e-5)
    y.backward(dy)
    _, mean, rstd = tf.tf_layernorm_fwd(x.detach(), g.detach(), b.detach(), 1e-5)
    dx, dg, db = tf.tf_layernorm_bwd(x.detach(), g.detach(), dy, mean, rstd)
    assert (dx - x.grad).abs().max().item() < 2e-5
    assert (dg - g.grad).abs().max().item() < 2e-4 and (db - b.grad).abs().max().item() < 2e-4


def test_deterministic_and_bad_arguments():
    x = torch.randn(999, 2048, device="cuda", dtype=torch.bfloat16)
    w = torch.ones(2048, device="cuda", dtype=torch.bfloat16)
    dy = torch.randn_like(x)
    _, rstd = tf.tf_rmsnorm_fwd(x, w, 1e-6, want_rstd=True)
    a = tf.tf_rmsnorm_bwd(x, w, dy, rstd)
    b = tf.tf_rmsnorm_bwd(x, w, dy, rstd)
    assert torch.equal(a[0].view(torch.uint16), b[0].view(torch.uint16)) and torch.equal(a[1].view(torch.uint16), b[1].view(torch.uint16))
    L = tf.lib()
    p = torch.zeros(4096, device="cuda").data_ptr()
    assert L.tf_norm_bwd_workspace_bytes(999, 2048) >= 4 * 2048 * 2 * 4
    assert L.tf_rmsnorm_bwd(p, p, p, p, p, p, None, 0, 4, 64, 0, None) == 1          # workspace missing for an aligned shape
    assert L.tf_rmsnorm_bwd(p, p, p, p, p, p, p, 16, 4, 64, 0, None) == 1            # workspace too small
    assert L.tf_rmsnorm_bwd(p, p, p, None, p, p, p, 1 << 20, 4, 64, 0, None) == 1    # rstd missing
    assert L.tf_layernorm_bwd(p, p, p, None, p, p, p, p, p, 1 << 20, 4, 64, 0, None) == 1   # mean missing
    assert L.tf_layernorm_bwd(p, p, p, p, p, p, p, None, p, 1 << 20, 4, 64, 0, None) == 1   # dbeta missing
    assert L.tf_rmsnorm_bwd(p, p, p, p, p, p, p, 1 << 20, 4, 0, 0, None) == 1


def test_workspace_needs_only_4_byte_alignment():
    """Wide parts are added with 16-byte reads when the workspace allows them: a workspace that is only 4-byte aligned gives
    the same bits (same order of additions) through the 4-byte reads."""
    rows, cols = 40, 32768
    x = torch.randn(rows, cols, device="cuda", dtype=torch.bfloat16)
    dy = torch.randn_like(x)
    g = (torch.rand(cols, device="cuda") + 0.5).to(torch.bfloat16)
    _, mean, rstd = tf.tf_layernorm_fwd(x, g, torch.zeros_like(g), 1e-5)
    dx0, dg0, db0 = tf.tf_layernorm_bwd(x, g, dy, mean, rstd)
    L = tf.lib()
    n = L.tf_norm_bwd_workspace_bytes(rows, cols)
    ws = torch.empty(n // 4 + 8, dtype=torch.float32, device="cuda")
    dx, dg, db = torch.empty_like(x), torch.empty_like(g), torch.empty_like(g)
    st = L.tf_layernorm_bwd(x.data_ptr(), g.data_ptr(), dy.data_ptr(), mean.data_ptr(), rstd.data_ptr(), dx.data_ptr(), dg.data_ptr(),
                            db.data_ptr(), ws.data_ptr() + 4, n, rows, cols, BF16, torch.cuda.current_stream().cuda_stream)
    assert st == 0
    torch.cuda.synchronize()
    tf.tf_device_status()
    for a, b in ((dx0, dx), (dg0, dg), (db0, db)):
        assert torch.equal(a.view(torch.uint16), b.view(torch.uint16))


@pytest.mark.parametrize("rms,dt,rows,cols", [(True, BF16, 16384, 4096), (True, BF16, 16384, 8192), (True, F32, 16384, 4096), (False, BF16, 16384, 4096),
                                              (False, BF16, 65536, 1024), (False, F32, 8192, 8192), (False, BF16, 4096, 16384), (False, F32, 4096, 16384),
                                              (False, BF16, 2048, 32768)])
def test_shapes_of_the_bench_table_every_element(rms, dt, rows, cols):
    """The shapes `bench.py --table normbwd` times, in the form it times (automatic): dx element by element, the parameter
    gradients summed over all rows."""
    run_case(rms, dt, rows, cols, seed=cols)


@pytest.mark.parametrize("op,dt,rows,cols", [("layernorm", BF16, 4096, 4096), ("rmsnorm", BF16, 3000, 1024), ("layernorm", F32, 2048, 8192),
                                              ("rmsnorm", BF16, 700, 16384), ("layernorm", BF16, 50, 1000)])
def test_tuned_form_is_used_and_still_exact(op, dt, rows, cols):
    """tf_tune_norm_bwd times the forms on the shape and keeps one only if it is measured faster; whatever it keeps must
    be what later calls use, and must still meet the oracle."""
    rms = op == "rmsnorm"
    try:
        assert tf.tf_norm_bwd_choice(op, rows, cols, dt) == "path=0,stages=0,cluster=0"
        timed, auto_us, best_us = tf.tf_tune_norm_bwd(op, rows, cols, dt)
        if cols * (4 if dt == F32 else 2) % 16 == 0:
            assert timed >= 2 and 0 < best_us <= auto_us
        else:
            assert timed == 0                                      # only the plain kernels serve such rows
        kept = tf.tf_norm_bwd_choice(op, rows, cols, dt)
        if best_us == auto_us:
            assert kept == "path=0,stages=0,cluster=0"            # nothing was more than 2 % faster
        run_case(rms, dt, rows, cols, seed=7)
        assert tf.tf_norm_bwd_choice(op, rows + 1, cols, dt) == "path=0,stages=0,cluster=0"   # another shape: automatic
        tf.tf_norm_bwd_force(1, 0, 1)                              # a forced choice wins over the tuned one
        assert tf.tf_norm_bwd_choice(op, rows, cols, dt) == "path=1,stages=0,cluster=1"
        tf.tf_norm_bwd_force(0, 0, 0)
        assert tf.tf_norm_bwd_choice(op, rows, cols, dt) == kept
        tf.tf_clear_cache()
        assert tf.tf_norm_bwd_choice(op, rows, cols, dt) == "path=0,stages=0,cluster=0"
    finally:
        tf.tf_norm_bwd_force(0, 0, 0)
        tf.tf_clear_cache()
    with pytest.raises(tf.TfError):
        tf.tf_tune_norm_bwd("softmax", 8, 64, dt)
