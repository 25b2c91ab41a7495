"""Fused residual add + LayerNorm / RMSNorm through the C ABI against the CPU oracle: h must equal the oracle's rounded
sum bit for bit, y and the statistics must meet the tolerances of the unfused ops computed on that h."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import compare
import oracle
import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
from paper_2512_09196_b200.inputs import Workload
import parity

pytestmark = pytest.mark.gpu
F32, BF16 = inputs.F32, inputs.BF16
EPS = {"layernorm": 1e-5, "rmsnorm": 1e-6}
OPS = ("layernorm", "rmsnorm")


@pytest.fixture(autouse=True)
def _auto_plans():
    yield
    for op in OPS:
        tf.tf_force_plan(op, None)


def run_case(op, dt, rows, cols, seed=3, offset=0, inplace=False, r_scale=1.0):
    w = Workload(f"add-{op}-{dt}-{rows}x{cols}", op, dt, rows, cols, seed=seed, eps=EPS[op], x_mean=0.3, x_std=2.0)
    data = w.generate()
    r_host = inputs.normal((rows, cols), dt, seed + 1000, 7, -0.2, r_scale)
    h_ref = oracle.add(data["x"], r_host, dt)
    x, r = parity.to_dev(data["x"], dt, offset), parity.to_dev(r_host, dt, offset)
    # the usual use: the residual stream is updated in place; every output sits between guard bands
    h = r if inplace else parity.guarded(tuple(x.shape), x.dtype, offset, name="h")
    yg = parity.guarded(tuple(x.shape), x.dtype, offset, name="y")
    st = lambda name: parity.guarded((rows,), torch.float32, name=name)
    got = {}
    if op == "layernorm":
        hh, y, mean, rstd = tf.tf_add_layernorm_fwd(x, r, parity.to_dev(data["gamma"], dt, offset), parity.to_dev(data["beta"], dt, offset),
                                                    w.eps, h=h, y=yg, mean=st("mean"), rstd=st("rstd"))
        got["mean"], got["rstd"] = mean.cpu().numpy(), rstd.cpu().numpy()
    else:
        hh, y, rstd = tf.tf_add_rmsnorm_fwd(x, r, parity.to_dev(data["w"], dt, offset), w.eps, h=h, y=yg, rstd=st("rstd"))
        got["rstd"] = rstd.cpu().numpy()
    torch.cuda.synchronize()
    tf.tf_device_status()
    got["y"] = parity.to_host(y, dt)
    np.testing.assert_array_equal(parity.to_host(hh, dt), h_ref, err_msg=f"h of {w.name}")       # bit-exact
    ref_data = dict(data, x=h_ref)
    fails = parity.check(w, ref_data, got, parity.run_oracle(w, ref_data))
    assert not fails, (w.name, offset, inplace, fails)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_automatic_plan_over_edge_widths(op, dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 2 * ne, 64, 128, 256, 1000 // ne * ne, 1024, 4096, 5120, 8192, 12288, 16384, 40960, 65536, 131072):
        rows = max(3, min(300, (1 << 21) // cols))
        run_case(op, dt, rows, cols, seed=cols)
    run_case(op, dt, 0, 64)
    run_case(op, dt, 1, 4096)
    run_case(op, dt, 2000, 512, inplace=True)
    run_case(op, dt, 77, 8192, inplace=True, r_scale=100.0)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_unaligned_odd_and_very_long_rows_take_the_two_kernel_route(op, dt):
    ne = 4 if dt == F32 else 8
    run_case(op, dt, 9, 1001)                        # cols * es not a multiple of 16
    run_case(op, dt, 9, 1024, offset=1)              # misaligned base pointers
    run_case(op, dt, 7, 1024, offset=3, inplace=True)
    run_case(op, dt, 3, 600000 // ne * ne)           # beyond what a cluster of register-resident CTAs holds


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_register_plans(op, dt):
    ne = 4 if dt == F32 else 8
    for lanes, vpt, rpg in ((8, 1, 1), (8, 2, 2), (16, 1, 4), (32, 2, 2), (32, 4, 1), (32, 8, 1)):
        cap = lanes * vpt
        for nvec in (cap, max(1, cap - 1)):
            tf.tf_force_plan(op, f"warp:threads=128,lanes={lanes},vpt={vpt},rpg={rpg},persist=0")
            run_case(op, dt, 301, nvec * ne, seed=nvec)
    for cluster in (1, 2, 8):
        for vpt, threads in ((1, 64), (2, 1024), (4, 256), (8, 512)):
            cap = threads * vpt * cluster
            for nvec, persist in ((cap, 0), (max(1, cap - threads - 3), 1)):
                tf.tf_force_plan(op, f"cta:threads={threads},vpt={vpt},cluster={cluster},persist={persist}")
                run_case(op, dt, 9 if nvec >= 4096 else 170, nvec * ne, seed=nvec)
    # a forced plan that the fused kernels do not have (the pipeline) falls back to their own choice: still exact
    # x and r staged in shared memory: rows of one to four steps, exact and ragged, in place, one row
    for threads, stages in ((32, 2), (64, 4), (128, 2), (256, 3)):
        st = threads * 4
        for nvec, rows in ((st * stages, 9), (st * stages - 1, 170), (st + 1, 301), (1, 5), (st, 1)):
            tf.tf_force_plan(op, f"twopass:threads={threads},persist=0,regcap=0,stages={stages},u=4")
            run_case(op, dt, min(rows, max(3, (1 << 21) // (nvec * ne))), nvec * ne, seed=nvec + threads)
        run_case(op, dt, 23, st * 2 * ne, seed=st, inplace=True)
    tf.tf_force_plan(op, None)
    es = 4 if dt == F32 else 2
    for kib in (8, 16, 24, 32):                          # the default for many rows of 8-32 KiB
        run_case(op, dt, 300, kib * 1024 // es, seed=kib)
        run_case(op, dt, 297, kib * 1024 // es - ne, seed=kib + 1, inplace=True)
    tf.tf_force_plan(op, "pipe:threads=512,lanes=64,vpt=8,rpg=1,stages=2,chunk=8192,persist=1")
    run_case(op, dt, 100, 512 * ne)


def test_tuned_plan_is_used_and_still_exact():
    for op, dt, rows, cols in (("rmsnorm", BF16, 2048, 4096), ("layernorm", F32, 1024, 1024)):
        tf.tf_clear_cache()
        rep = tf.tf_tune_add(op, rows, cols, dt)
        assert rep["timed"] >= 2 and rep["best_us"] <= rep["heuristic_us"] * 1.0001
        run_case(op, dt, rows, cols, seed=5)
        tf.tf_clear_cache()
    with pytest.raises(tf.TfError):
        tf.tf_tune_add("softmax", 64, 64, F32)
    with pytest.raises(tf.TfError):
        tf.tf_tune_add("rmsnorm", 4, 1 << 20, F32)            # no register-resident plan holds 4 MiB rows


def test_rounding_of_h_decides_the_statistics():
    # x + r lands between bf16 values: the norm must see the ROUNDED h (ties to even), as the unfused pair of calls would
    cols = 1024
    x = torch.full((4, cols), 1.0, dtype=torch.bfloat16, device="cuda")
    r = torch.full((4, cols), 2.0 ** -8, dtype=torch.bfloat16, device="cuda")       # 1 + 2^-8 ties down to 1.0
    r[:, ::2] = 2.0 ** -8 + 2.0 ** -9                                               # above the tie: rounds up to 1 + 2^-7
    w = torch.ones(cols, dtype=torch.bfloat16, device="cuda")
    h, y, rstd = tf.tf_add_rmsnorm_fwd(x, r, w, 0.0, want_rstd=True)
    hh = h.float().cpu().numpy()
    assert (hh[:, 1::2] == 1.0).all() and (hh[:, ::2] == 1.0 + 2.0 ** -7).all()
    ms = 0.5 * (1.0 + (1.0 + 2.0 ** -7) ** 2)
    np.testing.assert_allclose(rstd.cpu().numpy(), 1.0 / np.sqrt(ms), rtol=1e-6)
    y2, _ = tf.tf_rmsnorm_fwd(h, w, 0.0)
    assert torch.equal(y.view(torch.uint16), y2.view(torch.uint16)) or (y.float() - y2.float()).abs().max() <= 2.0 ** -7


def test_bad_arguments():
    L = tf.lib()
    p = torch.zeros(64, device="cuda").data_ptr()
    assert L.tf_add_rmsnorm_fwd(p, None, p, p, p, None, 1, 8, 1e-6, 0, None) == 1           # r missing
    assert L.tf_add_rmsnorm_fwd(p, p, p, None, p, None, 1, 8, 1e-6, 0, None) == 1           # h missing
    assert L.tf_add_layernorm_fwd(p, p, p, None, p, p, None, None, 1, 8, 1e-5, 0, None) == 1  # beta missing
    assert L.tf_add_layernorm_fwd(p, p, p, p, p, p, None, None, 1, 8, -1.0, 0, None) == 1
    assert L.tf_add_layernorm_fwd(p, p, p, p, p, p, None, None, 0, 8, 1e-5, 0, None) == 0


@pytest.mark.parametrize("op,dt,rows,cols", [("rmsnorm", BF16, 16384, 4096), ("layernorm", BF16, 16384, 4096), ("rmsnorm", BF16, 4096, 16384),
                                              ("layernorm", F32, 16384, 4096), ("rmsnorm", BF16, 256, 8192)])
def test_shapes_of_the_bench_table_every_element(op, dt, rows, cols):
    """The shapes `bench.py --table addnorm` times, in the plan it times (automatic), every element against the oracle."""
    run_case(op, dt, rows, cols, seed=cols)
