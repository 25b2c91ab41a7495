"""Parity at the 84 points of the shape sweep at their full size (256 MiB of input each): every row of every point,
in the plan an untuned call takes, and for a spread of points also in the plan ``tf_tune`` ends up with (the one the
sweep table reports).  The oracle runs row-parallel on the host (bit-identical to its single-threaded run); the
element-by-element comparison of ``compare.py`` is applied block by block on a thread pool."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import pytest
import torch

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu

SWEEP = inputs.sweep()
TUNED = list(range(3, len(SWEEP), 7))            # 12 points spread over ops, types and widths


def _gpu(w, data):
    dt = w.dt
    x = parity.to_dev(data["x"], dt)
    y = parity.guarded(tuple(x.shape), x.dtype, name="y")
    out = {}
    if w.op == "softmax":
        tf.tf_softmax_fwd(x, y)
    elif w.op == "layernorm":
        _, mean, rstd = tf.tf_layernorm_fwd(x, parity.to_dev(data["gamma"], dt), parity.to_dev(data["beta"], dt), w.eps, y,
                                            mean=parity.guarded((w.rows,), torch.float32, name="mean"),
                                            rstd=parity.guarded((w.rows,), torch.float32, name="rstd"))
        out.update(mean=mean.cpu().numpy(), rstd=rstd.cpu().numpy())
    else:
        _, rstd = tf.tf_rmsnorm_fwd(x, parity.to_dev(data["w"], dt), w.eps, y, rstd=parity.guarded((w.rows,), torch.float32, name="rstd"))
        out.update(rstd=rstd.cpu().numpy())
    torch.cuda.synchronize()
    tf.tf_device_status()
    out["y"] = parity.to_host(y, dt)
    parity.check_guards()
    return out


def _check_all_rows(w, data, got, ref, block_elems=1 << 21):
    rows_per = max(1, block_elems // w.cols)

    def one(r0):
        sl = slice(r0, min(w.rows, r0 + rows_per))
        d = dict(data)
        d["x"] = data["x"][sl]
        return [f"rows {r0}+: {f}" for f in parity.check(w, d, {k: v[sl] for k, v in got.items()}, {k: v[sl] for k, v in ref.items()})]

    fails = []
    with ThreadPoolExecutor(os.cpu_count() or 4) as ex:
        for f in ex.map(one, range(0, w.rows, rows_per)):
            fails += f
    return fails


@pytest.mark.parametrize("i", range(len(SWEEP)), ids=[w.name for w in SWEEP])
def test_sweep_point_every_row(i):
    w = SWEEP[i]
    assert w.rows * w.cols * w.elem_size > 250 << 20                 # the table's size, not a reduced one
    data = w.generate()
    ref = parity.run_oracle(w, data, nthreads=os.cpu_count() or 4)
    tf.tf_clear_cache()
    plans = [tf.tf_query_choice(w.op, w.rows, w.cols, w.dt)]          # what an untuned call runs
    fails = _check_all_rows(w, data, _gpu(w, data), ref)
    assert not fails, (w.name, plans[0], fails[:3])
    if i in TUNED:
        x = parity.to_dev(data["x"], w.dt)
        p0 = data.get("gamma", data.get("w"))
        like = (x, parity.to_dev(p0, w.dt) if p0 is not None else None, parity.to_dev(data["beta"], w.dt) if "beta" in data else None)
        tuned = tf.tf_tune(w.op, w.rows, w.cols, w.dt, like=like)    # on the workload's own data, as the table does
        del x, like
        plans.append(tuned["plan"])
        fails = _check_all_rows(w, data, _gpu(w, data), ref)
        tf.tf_clear_cache()
        assert not fails, (w.name, plans[1], fails[:3])
