"""Parity at the full sizes of the fixed configurations, in the launch configuration the bench times (the tuned
plan): configurations 0-2 are compared on every row, block by block; the 2 GiB masked softmax on sampled rows
(each row is an independent problem, so a row sample is an exact check of those rows)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu


def _run_full(w, data):
    dt = w.dt
    x = parity.to_dev(data["x"], dt)
    out = {}
    if w.op == "softmax":
        out["y"] = tf.tf_softmax_fwd(x)
    elif w.op == "layernorm":
        y, mean, rstd = tf.tf_layernorm_fwd(x, parity.to_dev(data["gamma"], dt), parity.to_dev(data["beta"], dt), w.eps)
        out.update(y=y, mean=mean.cpu().numpy(), rstd=rstd.cpu().numpy())
    else:
        y, rstd = tf.tf_rmsnorm_fwd(x, parity.to_dev(data["w"], dt), w.eps, want_rstd=True)
        out.update(y=y, rstd=rstd.cpu().numpy())
    torch.cuda.synchronize()
    tf.tf_device_status()
    return out


def _check_rows(w, data, got, rows):
    """Oracle + comparison on the given row indices (a slice or an index array)."""
    sub = dict(data)
    sub["x"] = np.ascontiguousarray(data["x"][rows])
    g = {"y": parity.to_host(got["y"][rows], w.dt)}
    for k in ("mean", "rstd"):
        if k in got:
            g[k] = got[k][rows]
    return parity.check(w, sub, g, parity.run_oracle(w, sub, nthreads=16))


@pytest.mark.parametrize("i", [0, 1, 2])
def test_full_configuration_every_row(i):
    w = inputs.config(i)
    tf.tf_tune(w.op, w.rows, w.cols, w.dt)
    data = w.generate()
    got = _run_full(w, data)
    block = max(1, (1 << 23) // w.cols)
    for r0 in range(0, w.rows, block):
        fails = _check_rows(w, data, got, slice(r0, min(w.rows, r0 + block)))
        assert not fails, (w.name, tf.tf_query_choice(w.op, w.rows, w.cols, w.dt), r0, fails)


def test_masked_softmax_2gib_sampled_rows():
    w = inputs.config(3)
    data = w.generate()
    x_dev = parity.to_dev(data["x"], w.dt)
    tuned = tf.tf_tune(w.op, w.rows, w.cols, w.dt, like=(x_dev, None, None))      # timed on the masked data itself, as the bench does
    tf.tf_force_plan(w.op, tuned["plan"])            # the winner (a listed proposal or a refinement of one) is a valid plan
    tf.tf_force_plan(w.op, None)
    del x_dev
    got = _run_full(w, data)
    rows = np.unique(np.concatenate([np.arange(0, w.rows, 61), [0, 1, 2047, 2048, w.rows - 2, w.rows - 1]]))
    fails = _check_rows(w, data, got, rows)
    assert not fails, (tf.tf_query_choice(w.op, w.rows, w.cols, w.dt), fails)
    # properties that hold for every row: masked tail is +0 everywhere, nothing else is NaN, rows sum to about 1
    y = got["y"]
    assert not torch.isnan(y).any()
    sums = y.float().sum(dim=1)
    assert (sums > 0.97).all() and (sums < 1.03).all()
    for r in (1, 1000, 4095):
        k = (r * 32) % w.cols
        assert (y[r, w.cols - k:].view(torch.int16) == 0).all()


def test_tune_is_idempotent_and_candidates_all_pass_parity():
    w = inputs.Workload("tune_case", "layernorm", inputs.BF16, 600, 2048, seed=9, x_mean=0.5, x_std=3.0, eps=1e-5)
    tf.tf_clear_cache()
    first = tf.tf_tune(w.op, w.rows, w.cols, w.dt)
    cands = tf.tf_candidates(w.op, w.rows, w.cols, w.dt)
    assert first["timed"] >= 2 and first["best_us"] <= first["heuristic_us"] * 1.0001
    variants = {c.split(":")[0] for c in cands}
    assert first["plan"].split(":")[0] in variants        # a listed proposal or a one-parameter refinement of one
    assert tf.tf_query_choice(w.op, w.rows, w.cols, w.dt) == first["plan"]          # later calls hit the cache
    second = tf.tf_tune(w.op, w.rows, w.cols, w.dt)
    assert second["plan"].split(":")[0] in variants
    tf.tf_force_plan(w.op, second["plan"])
    assert not parity.parity(w)                            # the refined winner passes parity like any plan
    data = w.generate()
    ref = parity.run_oracle(w, data)
    try:
        for plan in cands[:: max(1, len(cands) // 24)]:
            tf.tf_force_plan(w.op, plan)
            fails = parity.check(w, data, parity.run_gpu(w, data), ref)
            assert not fails, (plan, fails)
    finally:
        tf.tf_force_plan(w.op, None)
        tf.tf_clear_cache()


def test_host_pipeline_matches_single_call():
    """The overlapped host path (row blocks on three streams) gives exactly the single-call result."""
    from paper_2512_09196_b200.host import HostPipeline
    w = inputs.Workload("host_case", "layernorm", inputs.BF16, 1037, 2048, seed=4, x_mean=0.5, x_std=3.0, eps=1e-5)
    data = w.generate()
    pin = lambda a: torch.from_numpy(a).view(torch.bfloat16).pin_memory()
    hx, hg, hb = pin(data["x"]), pin(data["gamma"]), pin(data["beta"])
    hy = torch.empty_like(hx).pin_memory()
    hmean, hrstd = torch.empty(w.rows).pin_memory(), torch.empty(w.rows).pin_memory()
    dev = torch.device("cuda", 0)
    dp = {"gamma": torch.empty_like(hg, device=dev), "beta": torch.empty_like(hb, device=dev)}
    pipe = HostPipeline("layernorm", w.rows, w.cols, torch.bfloat16, dev, blocks=5)
    for _ in range(2):
        pipe.run(hx, hy, {"gamma": hg, "beta": hb}, dp, w.eps, hmean, hrstd)
    torch.cuda.synchronize()
    tf.tf_device_status()
    got = {"y": hy.view(torch.uint16).numpy(), "mean": hmean.numpy(), "rstd": hrstd.numpy()}
    assert not parity.check(w, data, got, parity.run_oracle(w, data))


def test_host_pipeline_overlapped_calls_keep_their_results_apart():
    """Consecutive calls without a join reuse the device staging buffers block by block: each call's host outputs must
    still be exactly its own result."""
    from paper_2512_09196_b200.host import HostPipeline
    dev = torch.device("cuda", 0)
    pin = lambda a: torch.from_numpy(a).view(torch.bfloat16).pin_memory()
    cases = []
    for seed in (11, 12, 13):
        w = inputs.Workload(f"host_case_{seed}", "rmsnorm", inputs.BF16, 2051, 4096, seed=seed, x_std=float(seed - 9), eps=1e-6)
        data = w.generate()
        cases.append((w, data, pin(data["x"]), pin(data["w"]), torch.empty(w.rows, w.cols, dtype=torch.bfloat16).pin_memory()))
    pipe = HostPipeline("rmsnorm", 2051, 4096, torch.bfloat16, dev, blocks=7)
    dps = [{"w": torch.empty(4096, dtype=torch.bfloat16, device=dev)} for _ in cases]
    for rep in range(2):
        for (w, data, hx, hw, hy), dp in zip(cases, dps):
            pipe.run(hx, hy, {"w": hw}, dp, w.eps, join=False)
    pipe.finish()
    torch.cuda.synchronize()
    tf.tf_device_status()
    for w, data, hx, hw, hy in cases:
        assert not parity.check(w, data, {"y": hy.view(torch.uint16).numpy()}, parity.run_oracle(w, data)), w.name
