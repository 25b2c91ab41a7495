"""Shared driver for the GPU parity tests: run one op through the C ABI on seeded inputs, run the oracle on the
same inputs, compare element by element with the tolerances of ``compare.py``."""
from __future__ import annotations

import numpy as np
import torch

import compare
import oracle
import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs

BF16, F32 = inputs.BF16, inputs.F32


def to_dev(a: np.ndarray, dt: int, offset_elems: int = 0) -> torch.Tensor:
    """Upload; with offset_elems the tensor starts that many elements into a larger allocation (misaligned base)."""
    t = torch.from_numpy(a)
    if dt == BF16:
        t = t.view(torch.bfloat16)
    if offset_elems == 0:
        return t.cuda()
    big = torch.empty(t.numel() + offset_elems + 64, dtype=t.dtype, device="cuda")
    view = big[offset_elems:offset_elems + t.numel()].view(t.shape)
    view.copy_(t)
    return view


def to_host(t: torch.Tensor, dt: int) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dt == BF16 else t.numpy()


def run_gpu(w: inputs.Workload, data: dict, offset: int = 0, inplace: bool = False, rms_rstd: bool = True):
    """Returns dict of host arrays: y (+ mean, rstd)."""
    dt = w.dt
    x = to_dev(data["x"], dt, offset)
    y = x if inplace else None
    out = {}
    if w.op == "softmax":
        yy = tf.tf_softmax_fwd(x, y)
    elif w.op == "layernorm":
        yy, mean, rstd = tf.tf_layernorm_fwd(x, to_dev(data["gamma"], dt, offset), to_dev(data["beta"], dt, offset), w.eps, y)
        out["mean"], out["rstd"] = mean.cpu().numpy(), rstd.cpu().numpy()
    else:
        yy, rstd = tf.tf_rmsnorm_fwd(x, to_dev(data["w"], dt, offset), w.eps, y, want_rstd=rms_rstd)
        if rstd is not None:
            out["rstd"] = rstd.cpu().numpy()
    torch.cuda.synchronize()
    tf.tf_device_status()
    out["y"] = to_host(yy, dt)
    return out


def run_oracle(w: inputs.Workload, data: dict, nthreads: int = 8):
    dt = w.dt
    if w.op == "softmax":
        y, y64 = oracle.softmax(data["x"], dt, want64=True, nthreads=nthreads)
        return {"y": y, "y64": y64}
    if w.op == "layernorm":
        y, mean, rstd, y64, st = oracle.layernorm(data["x"], data["gamma"], data["beta"], w.eps, dt, want64=True,
                                                  nthreads=nthreads)
        return {"y": y, "y64": y64, "stats64": st}
    y, rstd, y64, st = oracle.rmsnorm(data["x"], data["w"], w.eps, dt, want64=True, nthreads=nthreads)
    return {"y": y, "y64": y64, "rstd64": st}


def check(w: inputs.Workload, data: dict, got: dict, ref: dict) -> list[str]:
    """Returns a list of failure descriptions (empty = parity holds)."""
    dt = w.dt
    fails = []
    if w.op == "softmax":
        r = compare.compare_softmax(got["y"], ref["y"], ref["y64"], data["x"], dt)
        if not r.ok:
            fails.append(f"y: {r}")
    elif w.op == "layernorm":
        r = compare.compare_layernorm(got["y"], ref["y"], ref["y64"], data["x"], data["gamma"], data["beta"],
                                      ref["stats64"], dt)
        if not r.ok:
            fails.append(f"y: {r}")
        rm = compare.compare_mean(got["mean"], ref["stats64"], data["x"], dt)
        if not rm.ok:
            fails.append(f"mean: {rm}")
        rs = compare.compare_rstd(got["rstd"], ref["stats64"][:, 1])
        if not rs.ok:
            fails.append(f"rstd: {rs}")
    else:
        r = compare.compare_values(got["y"], ref["y"], ref["y64"], dt)
        if not r.ok:
            fails.append(f"y: {r}")
        if "rstd" in got:
            rs = compare.compare_rstd(got["rstd"], ref["rstd64"])
            if not rs.ok:
                fails.append(f"rstd: {rs}")
    return fails


def parity(w: inputs.Workload, row0: int = 0, nrows: int | None = None, **kw) -> list[str]:
    data = w.generate(row0, nrows)
    return check(w, data, run_gpu(w, data, **kw), run_oracle(w, data))
