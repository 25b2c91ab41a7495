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


# Guard bands: every tensor these drivers hand to the library is carved out of a larger allocation with GUARD bytes of a
# known pattern on both sides; check_guards() (run after every GPU test by conftest.py) fails if a kernel wrote into a
# band.  This stands in for a memory checker: a store one vector before or past any tensor shows here.
GUARD = 4096
GUARD_BYTE = 0xA5
_guards: list[tuple[torch.Tensor, int, int, str]] = []


def guarded(shape, dtype, offset_elems: int = 0, name: str = "tensor") -> torch.Tensor:
    """An uninitialised CUDA tensor of this shape between two guard bands (offset_elems: start that many elements later,
    for misaligned-base cases)."""
    es = torch.empty(0, dtype=dtype).element_size()
    n = int(np.prod(shape)) if len(shape) else 1
    start = GUARD + offset_elems * es
    raw = torch.full((start + n * es + GUARD,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
    _guards.append((raw, start, start + n * es, name))
    return raw[start:start + n * es].view(dtype).view(tuple(shape))


def guarded_like(t: torch.Tensor, name: str = "tensor") -> torch.Tensor:
    return guarded(tuple(t.shape), t.dtype, name=name)


def check_guards():
    """Asserts that no guard band of any tensor made since the last call was written to."""
    bad = []
    for raw, lo, hi, name in _guards:
        for band, what in ((raw[lo - GUARD:lo], "before"), (raw[hi:hi + GUARD], "behind")):
            wrong = (band != GUARD_BYTE).nonzero()
            if wrong.numel():
                bad.append(f"{name} [{hi - lo} bytes]: {wrong.numel()} bytes written {what} it, first at offset {int(wrong[0])} of the band")
    _guards.clear()
    assert not bad, "out-of-bounds writes: " + "; ".join(bad)


def to_dev(a: np.ndarray, dt: int, offset_elems: int = 0) -> torch.Tensor:
    """Upload between guard bands; with offset_elems the tensor starts that many elements later (misaligned base)."""
    t = torch.from_numpy(a)
    if dt == BF16:
        t = t.view(torch.bfloat16)
    view = guarded(tuple(t.shape), t.dtype, offset_elems, name="input")
    view.copy_(t)
    return view


def to_host(t: torch.Tensor, dt: int) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    return t.view(torch.uint16).numpy() if dt == BF16 else t.numpy()


def run_gpu(w: inputs.Workload, data: dict, offset: int = 0, inplace: bool = False, rms_rstd: bool = True):
    """Returns dict of host arrays: y (+ mean, rstd)."""
    dt = w.dt
    x = to_dev(data["x"], dt, offset)
    y = x if inplace else guarded(tuple(x.shape), x.dtype, offset, name="y")
    rows = x.shape[0]
    out = {}
    if w.op == "softmax":
        yy = tf.tf_softmax_fwd(x, y)
    elif w.op == "layernorm":
        yy, mean, rstd = tf.tf_layernorm_fwd(x, to_dev(data["gamma"], dt, offset), to_dev(data["beta"], dt, offset), w.eps, y,
                                             mean=guarded((rows,), torch.float32, name="mean"), rstd=guarded((rows,), torch.float32, name="rstd"))
        out["mean"], out["rstd"] = mean.cpu().numpy(), rstd.cpu().numpy()
    else:
        yy, rstd = tf.tf_rmsnorm_fwd(x, to_dev(data["w"], dt, offset), w.eps, y,
                                     rstd=guarded((rows,), torch.float32, name="rstd") if rms_rstd else None)
        if rstd is not None:
            out["rstd"] = rstd.cpu().numpy()
    torch.cuda.synchronize()
    tf.tf_device_status()
    out["y"] = to_host(yy, dt)
    check_guards()
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
