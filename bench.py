#!/usr/bin/env python
"""Benchmark of the row-wise reduce-then-normalise library on B200.

Default run (``python bench.py [--gpus N --steps K --warmup W]``): one step = one pass of the hot path
(``tf_softmax_fwd`` through the C ABI) over the largest fixed configuration, the tail-masked bf16 softmax
[4096, 131072] (2 GiB of algorithmic bytes per step), already resident in HBM.  The timed span is R back-to-back
regions of K steps each with an event between regions and no synchronisation inside; the line reports the median
region and the spread.  Prints ONE JSON line: achieved HBM GB/s (algorithmic bytes / device time), the roofline
fraction against the measured copy bandwidth of this machine, the end-to-end figure with host<->device copies inside the
timed region, the CPU oracle timed on this machine's host cores as a reported baseline, and (one GPU only) a record per
fixed configuration (``per_config``) and a summary of the 84-point shape sweep (``sweep_summary``).

``--impl reference`` times the CPU oracle alone (the reference arm).
``--table configs|sweep|...`` measure tables (not bench lines) and write them under ``--out``.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

NOMINAL_HBM_GBS = 8000.0          # the "~8 TB/s" the 80% bar is quoted against
FALLBACK_HBM_GBS = 6650.0         # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
L2_BYTES = 126 << 20
HEADLINE_CONFIG = 3               # the largest fixed configuration that fits one GPU: masked softmax bf16 [4096, 131072]

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel of each fixed
# configuration, from profiler captures of cases too large for the 126 MB L2 to hide the writes; None where no capture
# exists.  Value = (bytes of the captured case, factor to a full launch of the configuration).
NCU_TRAFFIC_BYTES = {
    # LayerNorm bf16 [8192, 4096] itself (k_twopass_fit, untuned plan): 67.2 MB read (= the algorithmic reads) + 15.7 MB
    # written inside an isolated launch; the rest of y is still dirty in L2 when the kernel ends (the problem is the size of L2)
    "layernorm_bf16_8192x4096": (67_156_224 + 15_669_760, 1.0),
    # RMSNorm bf16 [16384, 8192] itself (k_twopass_fit, untuned plan), a one-pass capture of the two DRAM counters:
    # 268.5 MB read (= the algorithmic reads) + 212.1 MB written inside the kernel
    "rmsnorm_bf16_16384x8192_outliers": (268_470_528 + 212_073_472, 1.0),
    # the 2 GiB masked softmax itself, a one-pass capture of the two DRAM counters on the full 4096 rows (untuned plan):
    # 1091.0 MB read (the algorithmic reads are 1073.7 MB) + 1013.4 MB written inside the kernel
    "masked_softmax_bf16_4096x131072": (1_090_978_560 + 1_013_370_112, 1.0),
}


def traffic_of(name):
    t = NCU_TRAFFIC_BYTES.get(name)
    return None if t is None else int(t[0] * t[1])


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------------------
# clocks: sampled through NVML while the timed region runs (reading only)
# ---------------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, cuda_index: int, period_s: float = 0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            try:        # CUDA and NVML may number the GPUs differently: match by UUID
                uuid = "GPU-" + str(torch.cuda.get_device_properties(cuda_index).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self.period = period_s

    def sample(self):
        if self._h is None:
            return
        try:
            self.samples.append(int(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM)))
            mask = int(self._nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            for bit, name in self.REASONS.items():
                if mask & bit and name != "gpu_idle":
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample()
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()
        self.sample()

    def summary(self) -> dict:
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------------------------
# one workload on one device
# ---------------------------------------------------------------------------------------------------------
class DeviceCase:
    """K rotating (x, y) buffer sets of one workload in HBM, so that no launch finds its lines in L2."""

    def __init__(self, w, data, device, min_total_bytes=1 << 30, max_sets=128):
        import torch
        from paper_2512_09196_b200 import inputs
        self.w, self.torch = w, torch
        tdt = torch.float32 if w.dt == inputs.F32 else torch.bfloat16

        def dev(a):
            t = torch.from_numpy(a)
            return (t.view(torch.bfloat16) if w.dt == inputs.BF16 else t).to(device)

        x0 = dev(data["x"])
        foot = 2 * x0.numel() * x0.element_size()
        self.sets = max(2, min(max_sets, -(-min_total_bytes // foot)))
        if foot >= 4 * L2_BYTES:
            self.sets = 2
        self.x = [x0] + [x0.clone() for _ in range(self.sets - 1)]
        self.y = [torch.empty_like(x0) for _ in range(self.sets)]
        self.params = {k: dev(v) for k, v in data.items() if k != "x"}
        rows = x0.shape[0]
        self.mean = torch.empty(rows, dtype=torch.float32, device=device)
        self.rstd = torch.empty(rows, dtype=torch.float32, device=device)
        self.i = 0
        self.bytes_per_step = w.algorithmic_bytes(rows)
        self.footprint = foot
        _ = tdt

    def step(self):
        import paper_2512_09196_b200 as tf
        k = self.i % self.sets
        self.i += 1
        w = self.w
        if w.op == "softmax":
            tf.tf_softmax_fwd(self.x[k], self.y[k])
        elif w.op == "layernorm":
            tf.tf_layernorm_fwd(self.x[k], self.params["gamma"], self.params["beta"], w.eps, self.y[k], self.mean, self.rstd)
        else:
            tf.tf_rmsnorm_fwd(self.x[k], self.params["w"], w.eps, self.y[k])

    def time_regions(self, steps: int, regions: int, warmup: int, step=None):
        """`regions` back-to-back regions of `steps` launches each, an event between regions, no synchronisation inside.
        Returns the region times in milliseconds."""
        torch = self.torch
        step = step or self.step
        for _ in range(warmup):
            step()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(regions + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for r in range(regions):
            for _ in range(steps):
                step()
            evs[r + 1].record()
        torch.cuda.synchronize()
        return [evs[r].elapsed_time(evs[r + 1]) for r in range(regions)]

    def copy_step(self):
        """The library's own streaming copy of the same tensors (x -> y): the practical ceiling at this size."""
        import paper_2512_09196_b200 as tf
        k = self.i % self.sets
        self.i += 1
        tf.tf_copy(self.x[k], self.y[k])

    def time_steps(self, steps: int, warmup: int) -> float:
        """Milliseconds for `steps` back-to-back launches (CUDA events on the launching stream)."""
        torch = self.torch
        for _ in range(warmup):
            self.step()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps):
            self.step()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)


def sample_rows(w, n: int):
    """n row indices spread evenly over the workload (the tail mask of the 2 GiB softmax grows with the row index, so
    the first rows alone would not be a fair sample)."""
    import numpy as np
    n = max(1, min(n, w.rows))
    return np.unique((np.arange(n, dtype=np.int64) * w.rows) // n)


def time_oracle(w, data, rows, reps: int = 1) -> float:
    """Seconds (best of reps) for the single-threaded oracle on the given rows (a count = the first rows, or indices)."""
    import numpy as np
    import oracle
    x = data["x"][:rows] if isinstance(rows, (int, np.integer)) else np.ascontiguousarray(data["x"][rows])
    best = float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        if w.op == "softmax":
            oracle.softmax(x, w.dt)
        elif w.op == "layernorm":
            oracle.layernorm(x, data["gamma"], data["beta"], w.eps, w.dt)
        else:
            oracle.rmsnorm(x, data["w"], w.eps, w.dt)
        best = min(best, time.perf_counter() - t0)
    return best


def cpu_baseline(w, data, budget_s: float = 12.0) -> dict:
    """The oracle as it stands, one thread, on a bounded sample of the workload: rows spread evenly over it."""
    probe = sample_rows(w, 16)
    t_probe = max(time_oracle(w, data, probe), 1e-6) / len(probe)
    n = int(max(1, min(w.rows, budget_s / 2 / t_probe)))
    rows = sample_rows(w, n)
    reps = 3 if len(rows) == w.rows and t_probe * w.rows * 3 < budget_s else 1
    t = time_oracle(w, data, rows, reps)
    gbs = w.algorithmic_bytes(len(rows)) / t / 1e9
    sample = (f"full batch [{w.rows}, {w.cols}], best of {reps}" if len(rows) == w.rows
              else f"{len(rows)} of {w.rows} rows spread evenly over the batch, one pass, GB/s of those rows' bytes")
    return {"value": gbs, "unit": "GB/s", "cores": 1, "cores_available": os.cpu_count(), "kind": "oracle", "sample": sample,
            "seconds": t}


# ---------------------------------------------------------------------------------------------------------
# end to end: pinned host buffers, H2D + kernel + D2H inside the timed region
# ---------------------------------------------------------------------------------------------------------
def time_e2e(w, data, device, steps: int, warmup: int, blocks: int = 8):
    """Pinned host buffers in, pinned host buffers out; every step copies x and the parameters to the device,
    runs the op through the C ABI and copies y (and the row statistics) back, all inside the timed region.
    The three legs are overlapped over row blocks by paper_2512_09196_b200.host.HostPipeline."""
    import torch
    from paper_2512_09196_b200 import inputs
    from paper_2512_09196_b200.host import HostPipeline

    def pin(a):
        t = torch.from_numpy(a)
        return (t.view(torch.bfloat16) if w.dt == inputs.BF16 else t).pin_memory()

    hx = pin(data["x"])
    hp = {k: pin(v) for k, v in data.items() if k != "x"}
    hy = torch.empty_like(hx).pin_memory()
    rows = hx.shape[0]
    hmean = torch.empty(rows, dtype=torch.float32).pin_memory()
    hrstd = torch.empty(rows, dtype=torch.float32).pin_memory()
    dp = {k: torch.empty_like(v, device=device) for k, v in hp.items()}
    pipe = HostPipeline(w.op, rows, w.cols, hx.dtype, device, blocks)
    h2d = hx.numel() * hx.element_size() + sum(v.numel() * v.element_size() for v in hp.values())
    d2h = hy.numel() * hy.element_size() + (8 * rows if w.op == "layernorm" else 0)

    def step():                  # consecutive steps overlap block by block; every step moves all of its inputs and results
        pipe.run(hx, hy, hp, dp, w.eps, hmean, hrstd, join=False)

    for _ in range(warmup):
        step()
    pipe.finish()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(steps):
        step()
    pipe.finish()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b), h2d, d2h


# ---------------------------------------------------------------------------------------------------------
# arms
# ---------------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def _spread(ms_regions, steps):
    """Median / min / max time per step over the timed regions."""
    per = sorted(m / steps for m in ms_regions)
    return per[len(per) // 2], per[0], per[-1]


def _tune_or_query(tf, w, case, no_tune):
    like = (case.x[0], case.params.get("gamma", case.params.get("w")), case.params.get("beta"))
    if no_tune:
        return {"plan": tf.tf_query_choice(w.op, w.rows, w.cols, w.dt), "timed": 0}
    return tf.tf_tune(w.op, w.rows, w.cols, w.dt, like=like)


def measure_config(tf, w, data, device, peak, no_tune, regions=25):
    """One fixed configuration: tuned plan, `regions` regions sized to a few milliseconds each, and the library's own
    streaming copy of the same tensors as the ceiling at that size."""
    case = DeviceCase(w, data, device)
    tuned = _tune_or_query(tf, w, case, no_tune)
    est = max(case.bytes_per_step / 6e12, 2e-6)
    steps = int(max(4, min(2000, 3e-3 / est)))
    med, lo, hi = _spread(case.time_regions(steps, regions, 5), steps)
    cmed, _, _ = _spread(case.time_regions(steps, 7, 3, step=case.copy_step), steps)
    gbs = case.bytes_per_step / (med * 1e-3) / 1e9
    copy_bytes = 2 * case.x[0].numel() * case.x[0].element_size()
    rec = {"workload": w.name, "op": w.op, "storage": w.dtype_name, "rows": w.rows, "cols": w.cols,
           "algorithmic_bytes": case.bytes_per_step, "plan": tuned["plan"], "us_per_launch": 1e3 * med,
           "us_min": 1e3 * lo, "us_max": 1e3 * hi, "launches_per_region": steps, "regions": regions, "gbs": gbs,
           "frac": gbs / peak, "pct_of_nominal_8000": 100 * gbs / NOMINAL_HBM_GBS,
           "tf_copy_gbs": copy_bytes / (cmed * 1e-3) / 1e9, "traffic": traffic_of(w.name),
           "tune": {k: tuned[k] for k in tuned if k != "plan"},
           "l2": f"rotating {case.sets} buffer sets ({case.sets * case.footprint / 1e9:.2f} GB)"}
    if case.footprint <= L2_BYTES // 4:
        rec["note"] = "latency-bound: the whole problem is a fraction of L2 and takes a few microseconds"
    return rec, case


def sweep_summary(tf, device, peak, tune: bool):
    """The 84-point shape sweep (256 MiB of input per point) in one pass: GB/s per point, how many reach 80 % of the
    nominal 8 TB/s, and the worst point.  x depends on (type, width) only, so it is generated once per pair."""
    import torch
    from paper_2512_09196_b200 import inputs
    pts, cache = [], {}
    for w in inputs.sweep():
        key = (w.dt, w.cols)
        if key not in cache:
            cache.clear()
            cache[key] = w.generate()["x"]
        data = dict(w.generate(0, 0), x=cache[key])
        case = DeviceCase(w, data, device)
        tf.tf_clear_cache()
        plan = _tune_or_query(tf, w, case, not tune)["plan"]
        steps = 20
        med, lo, hi = _spread(case.time_regions(steps, 5, 4), steps)
        gbs = case.bytes_per_step / (med * 1e-3) / 1e9
        pts.append({"workload": w.name, "us": 1e3 * med, "gbs": gbs, "plan": plan})
        del case
        torch.cuda.empty_cache()
    tf.tf_clear_cache()
    worst = min(pts, key=lambda r: r["gbs"])
    srt = sorted(r["gbs"] for r in pts)
    return {"points": len(pts), "input_bytes_per_point": inputs.SWEEP_BYTES, "plans": "tf_tune per point" if tune else "untuned defaults",
            "reach_6400": sum(r["gbs"] >= 0.8 * NOMINAL_HBM_GBS for r in pts), "reach_90pct_of_peak": sum(r["gbs"] >= 0.9 * peak for r in pts),
            "median_gbs": srt[len(srt) // 2], "worst": worst,
            "below_6400": [{"workload": r["workload"], "gbs": round(r["gbs"], 1)} for r in sorted(pts, key=lambda r: r["gbs"]) if r["gbs"] < 0.8 * NOMINAL_HBM_GBS]}


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs

    rank, local_rank, world = dist_env()
    if args.gpus != world and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)
    peak, peak_kind = measured_peak()

    # weak scaling: every rank owns one full batch (rows are independent; there is no exchange step)
    base = inputs.config(HEADLINE_CONFIG)
    w = inputs.Workload(base.name, base.op, base.dt, base.rows, base.cols, seed=base.seed + 1000 * rank, x_mean=base.x_mean,
                        x_std=base.x_std, eps=base.eps, outlier_p=base.outlier_p, outlier_factor=base.outlier_factor,
                        mask_step=base.mask_step, scale=base.scale, shift=base.shift)
    data = w.generate()
    case = DeviceCase(w, data, device)
    tuned = _tune_or_query(tf, w, case, args.no_tune)

    steps, warmup = args.steps, max(args.warmup, 3)
    # R regions of `steps` launches each: at least 25, and enough of them for about 100 ms of device time
    est_ms = 1e3 * case.bytes_per_step / 6e12
    regions = int(max(25, min(400, 100.0 / max(steps * est_ms, 1e-3))))
    for _ in range(warmup):
        case.step()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(regions + 1)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = tf.tf_launch_count()
    with ClockSampler(local_rank) as clk:
        torch.cuda.nvtx.range_push("BIG_OP")         # the label the paper's profiling step filters on (Section 3.3)
        evs[0].record()
        for r in range(regions):
            for _ in range(steps):
                case.step()
            evs[r + 1].record()
        torch.cuda.synchronize()
        torch.cuda.nvtx.range_pop()
    launches = tf.tf_launch_count() - launches0
    med, lo, hi = _spread([evs[r].elapsed_time(evs[r + 1]) for r in range(regions)], steps)
    if world > 1:
        t = torch.tensor([med, lo, hi], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        med, lo, hi = (float(v) for v in t.tolist())
    tf.tf_device_status()

    e2e_steps = max(3, min(steps, 6))
    blocks = 4
    e2e_ms, h2d, d2h = time_e2e(w, data, device, e2e_steps, 3, blocks)
    if world > 1:
        t = torch.tensor([e2e_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())

    if rank == 0:
        bytes_step = case.bytes_per_step
        per_launch_gbs = bytes_step / (med * 1e-3) / 1e9
        line = {
            "metric": "achieved HBM GB/s (algorithmic bytes / device time)", "value": world * per_launch_gbs, "unit": "GB/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": med, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "op": w.op, "storage": w.dtype_name, "rows_per_gpu": w.rows, "cols": w.cols,
                       "algorithmic_bytes_per_step": bytes_step, "plan": tuned["plan"],
                       "l2": f"rotating {case.sets} buffer sets ({case.sets * case.footprint / 1e9:.2f} GB) > 126 MB L2",
                       "sharding": "independent row batches per GPU, no collective"},
            "timing": {"regions": regions, "steps_per_region": steps, "statistic": "median region / steps",
                       "ms_per_step_min": lo, "ms_per_step_max": hi, "spread_pct": 100 * (hi - lo) / med},
            "pct_of_nominal_8000": 100 * per_launch_gbs / NOMINAL_HBM_GBS,
            "pct_of_measured_peak": 100 * per_launch_gbs / peak,
            "roofline": {"bound": "hbm", "achieved": per_launch_gbs, "peak": peak, "peak_kind": f"of {peak_kind}",
                         "unit": "GB/s", "frac": per_launch_gbs / peak, "traffic": traffic_of(w.name)},
            "e2e": {"value": world * bytes_step * e2e_steps / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps,
                    "how": f"pinned host -> device -> pinned host, {blocks} row blocks overlapped on three streams, consecutive steps overlapped block by block"},
            "gpu_launches": launches,
            "clocks": clk.summary(),
            "tune": {k: tuned[k] for k in tuned if k != "plan"},
        }
        line["cpu_baseline"] = cpu_baseline(w, data) if world == 1 else None
        if world == 1 and not args.no_extras:
            del case
            torch.cuda.empty_cache()
            per = []
            for i in range(4):
                if i == HEADLINE_CONFIG:
                    per.append({"workload": w.name, "op": w.op, "storage": w.dtype_name, "rows": w.rows, "cols": w.cols,
                                "algorithmic_bytes": bytes_step, "plan": tuned["plan"], "us_per_launch": 1e3 * med, "us_min": 1e3 * lo,
                                "us_max": 1e3 * hi, "launches_per_region": steps, "regions": regions, "gbs": per_launch_gbs,
                                "frac": per_launch_gbs / peak, "pct_of_nominal_8000": 100 * per_launch_gbs / NOMINAL_HBM_GBS,
                                "tf_copy_gbs": None, "traffic": traffic_of(w.name), "note": "the headline measurement above"})
                    continue
                wi = inputs.config(i)
                rec, c = measure_config(tf, wi, wi.generate(), device, peak, args.no_tune)
                per.append(rec)
                del c
                torch.cuda.empty_cache()
            # the copy ceiling of the headline configuration, on fresh buffers
            hc = DeviceCase(w, data, device)
            cm, _, _ = _spread(hc.time_regions(10, 7, 3, step=hc.copy_step), 10)
            per[HEADLINE_CONFIG]["tf_copy_gbs"] = 2 * hc.x[0].numel() * hc.x[0].element_size() / (cm * 1e-3) / 1e9
            del hc
            torch.cuda.empty_cache()
            line["per_config"] = per
            line["sweep_summary"] = sweep_summary(tf, device, peak, args.sweep_tune)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores, on the headline workload; every step is a
    bounded sample of it (rows spread evenly over the batch)."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import numpy as np
    from paper_2512_09196_b200 import inputs
    w = inputs.config(HEADLINE_CONFIG)
    steps, warmup = args.steps, args.warmup
    # a quarter of a second per step, found on a few rows first; only the sampled rows are generated
    probe_rows = sample_rows(w, 4)
    probe = {"x": np.concatenate([w.generate(int(r), 1)["x"] for r in probe_rows])}
    per_row = max(time_oracle(w, probe, len(probe_rows)), 1e-6) / len(probe_rows)
    budget = 120.0 / max(1, steps + warmup)
    rows = sample_rows(w, int(max(1, min(w.rows, min(0.25, budget) / per_row))))
    data = {"x": np.concatenate([w.generate(int(r), 1)["x"] for r in rows])}
    n = len(rows)
    for _ in range(warmup):
        time_oracle(w, data, n)
    t0 = time.perf_counter()
    for _ in range(steps):
        time_oracle(w, data, n)
    sec = time.perf_counter() - t0
    value = w.algorithmic_bytes(n) * steps / sec / 1e9
    sample = f"{n} of {w.rows} rows spread evenly over the batch per step"
    print(json.dumps({
        "impl": "reference", "metric": "achieved HBM GB/s (algorithmic bytes / device time)", "value": value, "unit": "GB/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * sec / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "op": w.op, "storage": w.dtype_name, "rows_per_step": n, "cols": w.cols},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


# ---------------------------------------------------------------------------------------------------------
# tables: the other configurations and the shape sweep (not bench lines)
# ---------------------------------------------------------------------------------------------------------
def run_table(args):
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peak, peak_kind = measured_peak()
    if args.table == "configs":
        points = [inputs.config(i) for i in range(4)]
    else:
        points = inputs.sweep()
        if args.filter:
            points = [p for p in points if args.filter in p.name]
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    rows_out = []
    for w in points:
        data = w.generate()
        case = DeviceCase(w, data, device)
        heur = tf.tf_query_choice(w.op, w.rows, w.cols, w.dt)
        reps = max(20, min(400, int(0.05 / max(1e-6, case.bytes_per_step / 5e12))))
        tf.tf_clear_cache()
        ms_h = case.time_steps(reps, 5)
        like = (case.x[0], case.params.get("gamma", case.params.get("w")), case.params.get("beta"))
        tuned = tf.tf_tune(w.op, w.rows, w.cols, w.dt, like=like) if not args.no_tune else {"plan": heur, "timed": 0}
        ms_t = case.time_steps(reps, 5)
        us = 1e3 * ms_t / reps
        gbs = case.bytes_per_step / (us * 1e-6) / 1e9
        # calibration: a plain device copy of the same tensors (x -> y), same rotation, same timing loop
        for k in range(min(5, case.sets)):
            case.y[k].copy_(case.x[k])
        ca, cb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ca.record()
        for k in range(reps):
            case.y[k % case.sets].copy_(case.x[k % case.sets])
        cb.record()
        torch.cuda.synchronize()
        copy_us = 1e3 * ca.elapsed_time(cb) / reps
        copy_gbs = 2 * case.x[0].numel() * case.x[0].element_size() / (copy_us * 1e-6) / 1e9
        # and the library's own streaming copy (same load/store style as the row kernels)
        for k in range(min(5, case.sets)):
            tf.tf_copy(case.x[k], case.y[k])
        torch.cuda.synchronize()
        ca.record()
        for k in range(reps):
            tf.tf_copy(case.x[k % case.sets], case.y[k % case.sets])
        cb.record()
        torch.cuda.synchronize()
        tf_copy_gbs = 2 * case.x[0].numel() * case.x[0].element_size() / (ca.elapsed_time(cb) / reps * 1e-3) / 1e9
        row = {"workload": w.name, "op": w.op, "dtype": w.dtype_name, "rows": w.rows, "cols": w.cols,
               "bytes": case.bytes_per_step, "heuristic_plan": heur, "heuristic_us": 1e3 * ms_h / reps,
               "plan": tuned["plan"], "timed_candidates": tuned.get("timed"), "us": us, "gbs": gbs,
               "pct_of_8000": 100 * gbs / NOMINAL_HBM_GBS, f"pct_of_{peak_kind}_{peak:.0f}": 100 * gbs / peak,
               "copy_us": copy_us, "copy_gbs": copy_gbs, "tf_copy_gbs": tf_copy_gbs}
        if args.cpu:
            cb = cpu_baseline(w, data, budget_s=6.0)
            row["oracle_gbs"], row["oracle_sample"] = cb["value"], cb["sample"]
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del case
        torch.cuda.empty_cache()
    (out_dir / f"table_{args.table}.json").write_text(json.dumps(rows_out, indent=1))


def run_vecmat_table(args):
    """Batched vector-matrix product (the paper's second case study) over the K sweep: automatic geometry, every forced
    geometry, and torch's library routine for the same contraction as context.  B is far larger than L2."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    points = inputs.vecmat_sweep()
    if args.filter:
        points = [p for p in points if args.filter in p.name]
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)

    def timed(fn, reps):
        for _ in range(5):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return 1e3 * a.elapsed_time(b) / reps

    rows_out = []
    for w in points:
        data = w.generate()
        conv = (lambda t: t.view(torch.bfloat16)) if w.dt == inputs.BF16 else (lambda t: t)
        A, B = conv(torch.from_numpy(data["a"])).cuda(), conv(torch.from_numpy(data["b"])).cuda()
        C = torch.empty((w.M, w.N), dtype=A.dtype, device="cuda")
        nbytes = w.algorithmic_bytes()
        reps = max(20, min(200, int(0.05 / (nbytes / 5e12))))
        us_auto = timed(lambda: tf.tf_bvecmat_fwd(A, B, C), reps)
        grid, kvec = {}, w.K * w.elem_size // 16
        ks_ok = lambda th: th >= 128
        if not args.no_tune:
            for threads in (128, 256, 512, 1024):
                for lanes in (4, 8, 16, 32):
                    if w.dt == inputs.F32 and lanes <= kvec and (lanes == 32 or kvec <= 16 * lanes):
                        for rows in (1, 2, 4):
                            for ks in ((1, 2, 4) if lanes == 32 and kvec >= 1024 and ks_ok(threads) else (1,)):
                                grid[f"{threads},{lanes},{rows},{ks}"] = timed(lambda: tf.tf_bvecmat_fwd(A, B, C, threads, lanes, rows, ks), reps)
                if threads == 128 and kvec >= 64:
                    grid["staged"] = timed(lambda: tf.tf_bvecmat_fwd(A, B, C, 0, 1), reps)
                if w.dt == inputs.BF16 and threads < 1024:
                    for rows in (16, 32):
                        for ks in (1, 2, 4, 8):
                            if ks * 32 <= threads:
                                grid[f"{threads},0,{rows},{ks}"] = timed(lambda: tf.tf_bvecmat_fwd(A, B, C, threads, 0, rows, ks), reps)
        best = min(grid, key=grid.get) if grid else None
        us_lib = timed(lambda: torch.bmm(B, A.unsqueeze(-1)), max(5, reps // 4))
        tf.tf_device_status()
        row = {"workload": w.name, "dtype": w.dtype_name, "M": w.M, "N": w.N, "K": w.K, "bytes": nbytes, "us": us_auto,
               "gbs": nbytes / us_auto / 1e3, f"pct_of_{peak_kind}_{peak:.0f}": 100 * nbytes / us_auto / 1e3 / peak,
               "best_geometry": best, "best_us": grid.get(best), "best_gbs": nbytes / grid[best] / 1e3 if best else None,
               "torch_bmm_us": us_lib, "torch_bmm_gbs": nbytes / us_lib / 1e3,
               "grid_us": {k: round(v, 2) for k, v in sorted(grid.items(), key=lambda kv: kv[1])[:8]}}
        if args.cpu:
            import numpy as np
            import oracle
            sub = max(1, min(w.N, int(2e8 / (w.M * w.K))))
            sub_b = np.ascontiguousarray(data["b"][:, :sub])
            t0 = time.perf_counter()
            oracle.bvecmat(data["a"], sub_b, w.dt, nthreads=os.cpu_count() or 1)
            dt_s = time.perf_counter() - t0
            row["oracle_gbs"] = (w.M * w.K + w.M * sub * w.K + w.M * sub) * w.elem_size / dt_s / 1e9
            row["oracle_sample"] = f"first {sub} of {w.N} columns n of every batch entry"
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del A, B, C
        torch.cuda.empty_cache()
    (out_dir / "table_vecmat.json").write_text(json.dumps(rows_out, indent=1))


def run_addnorm_table(args):
    """Fused residual add + norm against the same work as two calls (torch add into h, then the unfused op)."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    shapes = [("rmsnorm", inputs.BF16, 16384, 4096), ("rmsnorm", inputs.BF16, 16384, 8192), ("rmsnorm", inputs.BF16, 4096, 16384),
              ("rmsnorm", inputs.F32, 8192, 8192), ("layernorm", inputs.BF16, 16384, 4096), ("layernorm", inputs.BF16, 65536, 1024),
              ("layernorm", inputs.F32, 16384, 4096), ("rmsnorm", inputs.BF16, 256, 8192)]
    rows_out = []
    for op, dt, rows, cols in shapes:
        w = inputs.Workload(f"add_{op}_{'f32' if dt == inputs.F32 else 'bf16'}_{rows}x{cols}", op, dt, rows, cols, seed=cols,
                            eps=1e-5 if op == "layernorm" else 1e-6)
        data = w.generate()
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        es = w.elem_size
        sets = max(2, min(16, int((1 << 30) // (4 * rows * cols * es)) + 1))         # rotate so that no launch finds its lines in L2
        xs = [conv(torch.from_numpy(data["x"])).cuda() for _ in range(sets)]
        rs = [conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols + 1, 7, 0.0, 1.0))).cuda() for _ in range(sets)]
        hs = [torch.empty_like(xs[0]) for _ in range(sets)]
        ys = [torch.empty_like(xs[0]) for _ in range(sets)]
        g = conv(torch.from_numpy(data["gamma"] if op == "layernorm" else data["w"])).cuda()
        b = conv(torch.from_numpy(data["beta"])).cuda() if op == "layernorm" else None
        tf.tf_tune(op, rows, cols, dt, like=(xs[0], g, b))
        tuned = tf.tf_tune_add(op, rows, cols, dt)

        def fused(k):
            if op == "layernorm":
                tf.tf_add_layernorm_fwd(xs[k], rs[k], g, b, w.eps, h=hs[k], y=ys[k], want_stats=False)
            else:
                tf.tf_add_rmsnorm_fwd(xs[k], rs[k], g, w.eps, h=hs[k], y=ys[k])

        def unfused(k):
            torch.add(xs[k], rs[k], out=hs[k])
            if op == "layernorm":
                tf.tf_layernorm_fwd(hs[k], g, b, w.eps, y=ys[k], want_stats=False)
            else:
                tf.tf_rmsnorm_fwd(hs[k], g, w.eps, y=ys[k])

        def timed(fn, reps):
            for k in range(5):
                fn(k % sets)
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for k in range(reps):
                fn(k % sets)
            e.record()
            torch.cuda.synchronize()
            return 1e3 * a.elapsed_time(e) / reps

        nbytes = 4 * rows * cols * es + (2 if op == "layernorm" else 1) * cols * es
        reps = max(20, min(400, int(0.05 / (nbytes / 5e12))))
        us_f, us_u = timed(fused, reps), timed(unfused, reps)
        tf.tf_device_status()
        row = {"workload": w.name, "op": op, "dtype": w.dtype_name, "rows": rows, "cols": cols, "bytes": nbytes, "us": us_f,
               "gbs": nbytes / us_f / 1e3, f"pct_of_{peak_kind}_{peak:.0f}": 100 * nbytes / us_f / 1e3 / peak,
               "unfused_us": us_u, "speedup_vs_two_calls": us_u / us_f, "tune": tuned, "base_plan": tf.tf_query_choice(op, rows, cols, dt)}
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del xs, rs, hs, ys
        torch.cuda.empty_cache()
    (out_dir / "table_addnorm.json").write_text(json.dumps(rows_out, indent=1))


def run_softmaxlen_table(args):
    """Softmax with per-row valid lengths against the same rows with the mask stored in the data (-inf tails)."""
    import numpy as np
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    shapes = [("tail 32 r mod cols (the mask of the 2 GiB configuration)", inputs.BF16, 4096, 131072), ("uniform lengths", inputs.BF16, 16384, 8192),
              ("uniform lengths", inputs.F32, 65536, 1024), ("uniform lengths", inputs.BF16, 262144, 256), ("full lengths", inputs.BF16, 16384, 8192)]
    rows_out = []
    for kind, dt, rows, cols in shapes:
        es = inputs.ELEM_SIZE[dt]
        r = np.arange(rows, dtype=np.int64)
        if kind.startswith("tail"):
            lens = (cols - (32 * r) % cols).astype(np.int32)
        elif kind.startswith("full"):
            lens = np.full(rows, cols, np.int32)
        else:
            lens = np.random.default_rng(cols).integers(1, cols + 1, rows).astype(np.int32)
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        sets = max(1, min(8, int((1 << 30) // (2 * rows * cols * es))))
        x = conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols, 0, 0.0, 3.0))).cuda()
        ld = torch.from_numpy(lens).cuda()
        xm = x.clone()
        xm[torch.arange(cols, device="cuda")[None, :] >= ld[:, None]] = float("-inf")
        xs = [x] + [x.clone() for _ in range(sets - 1)]
        xms = [xm] + [xm.clone() for _ in range(sets - 1)]
        ys = [torch.empty_like(x) for _ in range(sets)]
        tf.tf_tune("softmax", rows, cols, dt, like=(xm, None, None))

        def timed(fn, reps):
            for k in range(3):
                fn(k % sets)
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for k in range(reps):
                fn(k % sets)
            e.record()
            torch.cuda.synchronize()
            return 1e3 * a.elapsed_time(e) / reps

        nbytes = int(lens.astype(np.int64).sum()) * es + rows * cols * es + 4 * rows
        reps = max(10, min(200, int(0.05 / (2 * rows * cols * es / 5e12))))
        us_len = timed(lambda k: tf.tf_softmax_len_fwd(xs[k], ld, ys[k]), reps)
        us_data = timed(lambda k: tf.tf_softmax_fwd(xms[k], ys[k]), reps)
        tf.tf_device_status()
        row = {"workload": f"softmax_len_{'f32' if dt == inputs.F32 else 'bf16'}_{rows}x{cols}", "lengths": kind, "dtype": "f32" if dt == inputs.F32 else "bf16",
               "rows": rows, "cols": cols, "live_fraction": float(lens.mean() / cols), "bytes": nbytes, "us": us_len, "gbs": nbytes / us_len / 1e3,
               f"pct_of_{peak_kind}_{peak:.0f}": 100 * nbytes / us_len / 1e3 / peak, "mask_in_data_us": us_data,
               "speedup_vs_mask_in_data": us_data / us_len, "plain_plan": tf.tf_query_choice("softmax", rows, cols, dt)}
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del xs, xms, ys, x, xm
        torch.cuda.empty_cache()
    (out_dir / "table_softmaxlen.json").write_text(json.dumps(rows_out, indent=1))


def run_softmax_variants_table(args):
    """Log-softmax forward and softmax backward: achieved bandwidth of their algorithmic bytes, torch's routines as context."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    shapes = [(inputs.BF16, 16384, 8192), (inputs.BF16, 32768, 4096), (inputs.F32, 65536, 1024), (inputs.BF16, 524288, 256),
              (inputs.BF16, 8192, 32768), (inputs.F32, 4096, 32768), (inputs.F32, 2048, 131072)]
    rows_out = []
    for dt, rows, cols in shapes:
        es = inputs.ELEM_SIZE[dt]
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        sets = max(2, min(8, int((1 << 30) // (3 * rows * cols * es))))
        xs = [conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols, 0, 0.0, 3.0))).cuda() for _ in range(sets)]
        gs = [conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols + 1, 1, 0.0, 1.0))).cuda() for _ in range(sets)]
        ys = [torch.softmax(x.float(), dim=1).to(x.dtype) for x in xs]
        lys = [torch.log_softmax(x.float(), dim=1).to(x.dtype) for x in xs]
        outs = [torch.empty_like(x) for x in xs]

        def timed(fn, reps):
            for k in range(3):
                fn(k % sets)
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for k in range(reps):
                fn(k % sets)
            e.record()
            torch.cuda.synchronize()
            return 1e3 * a.elapsed_time(e) / reps

        reps = max(10, min(200, int(0.05 / (3 * rows * cols * es / 5e12))))
        for op, nbytes, ours, lib in (
                ("log_softmax_fwd", 2 * rows * cols * es, lambda k: tf.tf_log_softmax_fwd(xs[k], outs[k]),
                 lambda k: torch.log_softmax(xs[k], dim=1, out=outs[k]) if False else torch.log_softmax(xs[k], dim=1)),
                ("softmax_bwd", 3 * rows * cols * es, lambda k: tf.tf_softmax_bwd(ys[k], gs[k], outs[k]),
                 lambda k: torch._softmax_backward_data(gs[k], ys[k], 1, ys[k].dtype)),
                ("log_softmax_bwd", 3 * rows * cols * es, lambda k: tf.tf_log_softmax_bwd(lys[k], gs[k], outs[k]),
                 lambda k: torch._log_softmax_backward_data(gs[k], lys[k], 1, lys[k].dtype))):
            us, us_lib = timed(ours, reps), timed(lib, max(5, reps // 2))
            row = {"op": op, "dtype": "f32" if dt == inputs.F32 else "bf16", "rows": rows, "cols": cols, "bytes": nbytes, "us": us,
                   "gbs": nbytes / us / 1e3, f"pct_of_{peak_kind}_{peak:.0f}": 100 * nbytes / us / 1e3 / peak, "torch_us": us_lib,
                   "torch_gbs": nbytes / us_lib / 1e3}
            rows_out.append(row)
            print(json.dumps(row), flush=True)
        tf.tf_device_status()
        del xs, gs, ys, lys, outs
        torch.cuda.empty_cache()
    (out_dir / "table_softmaxvariants.json").write_text(json.dumps(rows_out, indent=1))


def run_sine_table(args):
    """The element-wise sine (the paper's Case Study 1): time over its one tuning knob, the launch geometry
    (threads per CTA x 16-byte vectors per thread = the "block size"), on 256 MiB of input per storage type."""
    import torch
    import paper_2512_09196_b200 as tf
    torch.cuda.set_device(0)
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    rows_out = []
    for dt, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        n = (256 << 20) // torch.empty(0, dtype=dt).element_size()
        sets = 2                                              # 1 GiB of x and y in rotation: no launch finds its lines in L2
        gen = torch.Generator(device="cuda").manual_seed(7)
        xs = [(torch.rand(n, device="cuda", generator=gen) * 200.0 - 100.0).to(dt) for _ in range(sets)]
        ys = [torch.empty_like(x) for x in xs]
        nbytes = 2 * n * xs[0].element_size()

        def timed(fn, reps=20):
            for k in range(3):
                fn(k % sets)
            best = None
            for _ in range(3):
                a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                a.record()
                for k in range(reps):
                    fn(k % sets)
                e.record()
                torch.cuda.synchronize()
                us = 1e3 * a.elapsed_time(e) / reps
                best = us if best is None else min(best, us)
            return best

        us_default = timed(lambda k: tf.tf_sin_fwd(xs[k], ys[k]))
        grid = {}
        for threads in (32, 64, 128, 256, 512, 1024):
            for vpt in (1, 2, 4, 8):
                grid[(threads, vpt)] = timed(lambda k: tf.tf_sin_fwd(xs[k], ys[k], threads, vpt))
        us_default = min(us_default, timed(lambda k: tf.tf_sin_fwd(xs[k], ys[k])))      # before and after the grid, like every entry the best region
        us_torch = timed(lambda k: torch.sin(xs[k], out=ys[k]))
        us_copy = timed(lambda k: tf.tf_copy(xs[k], ys[k]))
        tf.tf_device_status()
        best, worst = min(grid, key=grid.get), max(grid, key=grid.get)
        row = {"dtype": name, "elements": n, "bytes": nbytes, "default_us": us_default, "default_gbs": nbytes / us_default / 1e3,
               "best_geometry": list(best), "best_us": grid[best], "best_gbs": nbytes / grid[best] / 1e3,
               "worst_geometry": list(worst), "worst_us": grid[worst], "worst_over_best": grid[worst] / grid[best],
               "torch_sin_us": us_torch, "tf_copy_us": us_copy,
               "grid_us": {f"{t}x{v}": grid[(t, v)] for (t, v) in sorted(grid)}}
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del xs, ys
        torch.cuda.empty_cache()
    (out_dir / "table_sine.json").write_text(json.dumps(rows_out, indent=1))


def run_launch_table(args):
    """Launch-bound shapes: time per call made eagerly through the Python binding and as one CUDA graph of 32 captured calls."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    sets, per_graph = 8, 32
    bf = torch.bfloat16
    rows_out = []

    def softmax_case():
        w = inputs.config(0)
        xs = [torch.from_numpy(inputs.normal((w.rows, w.cols), w.dt, k, 0, 0.0, 1.0)).cuda() for k in range(sets)]
        ys = [torch.empty_like(x) for x in xs]
        return "softmax f32 [1024, 1024] (configuration 0)", 2 * w.rows * w.cols * 4, lambda k: tf.tf_softmax_fwd(xs[k], ys[k])

    def add_case():
        rows, cols = 256, 8192
        xs = [torch.randn(rows, cols, device="cuda").to(bf) for _ in range(sets)]
        rs = [torch.randn(rows, cols, device="cuda").to(bf) for _ in range(sets)]
        hs, ys = [torch.empty_like(x) for x in xs], [torch.empty_like(x) for x in xs]
        wt = (torch.rand(cols, device="cuda") + 0.5).to(bf)
        return "add + rmsnorm bf16 [256, 8192] (a decode batch)", 4 * rows * cols * 2, lambda k: tf.tf_add_rmsnorm_fwd(xs[k], rs[k], wt, 1e-6, h=hs[k], y=ys[k])

    def lsm_case(rows, cols, dt, label):
        def make():
            xs = [torch.randn(rows, cols, device="cuda").to(dt) for _ in range(sets)]
            ys = [torch.empty_like(x) for x in xs]
            return label, 2 * rows * cols * xs[0].element_size(), lambda k: tf.tf_log_softmax_fwd(xs[k], ys[k])
        return make

    for make in (softmax_case, add_case, lsm_case(64, 32768, bf, "log-softmax bf16 [64, 32768] (logits of a decode batch)"),
                 lsm_case(8, 131072, torch.float32, "log-softmax f32 [8, 131072] (fp32 logits, 128 Ki vocabulary)"),
                 lsm_case(1, 262144, bf, "log-softmax bf16 [1, 262144] (one sequence, 256 Ki vocabulary)")):
        name, nbytes, call = make()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):                         # first use outside the capture
            for k in range(sets):
                call(k)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for k in range(per_graph):
                call(k % sets)

        def timed(fn, reps):
            for _ in range(3):
                fn()
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(reps):
                fn()
            e.record()
            torch.cuda.synchronize()
            return 1e3 * a.elapsed_time(e) / reps

        def eager():
            for k in range(per_graph):
                call(k % sets)
        us_eager = min(timed(eager, 20) for _ in range(3)) / per_graph
        us_graph = min(timed(graph.replay, 20) for _ in range(3)) / per_graph
        tf.tf_device_status()
        row = {"case": name, "bytes": nbytes, "eager_us_per_call": us_eager, "graph_us_per_call": us_graph,
               "graph_gbs": nbytes / us_graph / 1e3, "calls_per_graph": per_graph}
        rows_out.append(row)
        print(json.dumps(row), flush=True)
    (out_dir / "table_launch.json").write_text(json.dumps(rows_out, indent=1))


def run_normbwd_table(args):
    """LayerNorm / RMSNorm backward: achieved bandwidth of x, dy in and dx out; torch's native backward as context."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    out_dir = Path(args.out)
    out_dir.mkdir(exist_ok=True)
    shapes = [("rmsnorm", inputs.BF16, 16384, 4096), ("rmsnorm", inputs.BF16, 16384, 8192), ("rmsnorm", inputs.F32, 16384, 4096),
              ("layernorm", inputs.BF16, 16384, 4096), ("layernorm", inputs.BF16, 16384, 8192), ("layernorm", inputs.BF16, 65536, 1024),
              ("layernorm", inputs.F32, 8192, 8192),
              ("layernorm", inputs.BF16, 4096, 16384), ("rmsnorm", inputs.BF16, 4096, 16384), ("layernorm", inputs.F32, 4096, 16384),
              ("layernorm", inputs.BF16, 2048, 32768)]
    rows_out = []
    for op, dt, rows, cols in shapes:
        es = inputs.ELEM_SIZE[dt]
        tdt = torch.bfloat16 if dt == inputs.BF16 else torch.float32
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        sets = max(2, min(8, int((1 << 30) // (3 * rows * cols * es))))
        xs = [conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols, 0, 0.3, 2.0))).cuda() for _ in range(sets)]
        dys = [conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols + 1, 3, 0.0, 1.0))).cuda() for _ in range(sets)]
        dxs = [torch.empty_like(x) for x in xs]
        g = (torch.rand(cols, device="cuda") + 0.5).to(tdt)
        b = torch.zeros(cols, device="cuda", dtype=tdt)
        if op == "layernorm":
            stats = [tf.tf_layernorm_fwd(x, g, b, 1e-5)[1:] for x in xs]
        else:
            stats = [(None, tf.tf_rmsnorm_fwd(x, g, 1e-6, want_rstd=True)[1]) for x in xs]

        def ours(k):
            if op == "layernorm":
                tf.tf_layernorm_bwd(xs[k], g, dys[k], stats[k][0], stats[k][1], dx=dxs[k])
            else:
                tf.tf_rmsnorm_bwd(xs[k], g, dys[k], stats[k][1], dx=dxs[k])

        def lib(k):
            if op == "layernorm":
                torch.ops.aten.native_layer_norm_backward(dys[k], xs[k], [cols], stats[k][0].view(rows, 1), stats[k][1].view(rows, 1), g, b,
                                                          [True, True, True])
            else:
                xf = xs[k].float()
                xh = xf * stats[k][1][:, None]
                gg = dys[k].float() * g.float()
                (stats[k][1][:, None] * (gg - xh * (gg * xh).mean(dim=1, keepdim=True))).to(tdt)
                (dys[k].float() * xh).sum(dim=0).to(tdt)

        def timed(fn, reps):
            for k in range(3):
                fn(k % sets)
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for k in range(reps):
                fn(k % sets)
            e.record()
            torch.cuda.synchronize()
            return 1e3 * a.elapsed_time(e) / reps

        nbytes = 3 * rows * cols * es + (3 if op == "layernorm" else 2) * cols * es + (8 if op == "layernorm" else 4) * rows
        reps = max(10, min(200, int(0.05 / (nbytes / 5e12))))
        tf.tf_clear_cache()
        us_auto, us_lib = timed(ours, reps), timed(lib, max(5, reps // 4))
        timed_forms, _, _ = tf.tf_tune_norm_bwd(op, rows, cols, dt)                 # measure the forms, keep the fastest
        choice = tf.tf_norm_bwd_choice(op, rows, cols, dt)
        us = min(timed(ours, reps), us_auto) if choice != "path=0,stages=0,cluster=0" else us_auto
        tf.tf_device_status()
        row = {"op": op + "_bwd", "dtype": "f32" if dt == inputs.F32 else "bf16", "rows": rows, "cols": cols, "bytes": nbytes, "us": us,
               "automatic_us": us_auto, "forms_timed": timed_forms, "kept": choice,
               "gbs": nbytes / us / 1e3, f"pct_of_{peak_kind}_{peak:.0f}": 100 * nbytes / us / 1e3 / peak, "torch_us": us_lib,
               "torch_what": "aten native_layer_norm_backward" if op == "layernorm" else "eager fp32 expression (no fused kernel in torch)"}
        rows_out.append(row)
        print(json.dumps(row), flush=True)
        del xs, dys, dxs
        torch.cuda.empty_cache()
    (out_dir / "table_normbwd.json").write_text(json.dumps(rows_out, indent=1))


def run_case(args):
    """A few launches of one op/shape (for profiler captures): --case op:dtype:rows:cols or --case config:<i>[:rows[:mask_step]]
    (fewer rows of a fixed configuration; mask_step 128 on 1024 rows of the masked softmax spreads the tail mask over the
    whole range of lengths, like the full 4096 rows with their step of 32)."""
    import torch
    import paper_2512_09196_b200 as tf
    from paper_2512_09196_b200 import inputs
    torch.cuda.set_device(0)
    parts = args.case.split(":")
    if parts[0] == "vecmat":                  # vecmat:dtype:M:N:K[:threads:lanes:rows:ksplit]
        dt = inputs.F32 if parts[1] == "f32" else inputs.BF16
        M, N, K = (int(v) for v in parts[2:5])
        knobs = [int(v) for v in parts[5:9]] + [0] * (4 - len(parts[5:9]))
        w = inputs.VecMat(f"case_bvecmat_{parts[1]}_{M}x{N}x{K}", dt, M, N, K, seed=K)
        data = w.generate()
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        A, B = conv(torch.from_numpy(data["a"])).cuda(), conv(torch.from_numpy(data["b"])).cuda()
        C = torch.empty((M, N), dtype=A.dtype, device="cuda")
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(max(1, args.warmup)):
            tf.tf_bvecmat_fwd(A, B, C, *knobs)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            tf.tf_bvecmat_fwd(A, B, C, *knobs)
        b.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(b) / args.steps
        print(json.dumps({"case": w.name, "knobs": knobs, "launches": args.steps, "us_per_launch": us,
                          "gbs": w.algorithmic_bytes() / us / 1e3}))
        return
    if parts[0] == "softmaxlen":              # softmaxlen:dtype:rows:cols -- softmax with uniform per-row lengths
        import numpy as np
        dts, rows, cols = parts[1], int(parts[2]), int(parts[3])
        dt = inputs.F32 if dts == "f32" else inputs.BF16
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        x = conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols, 0, 0.0, 3.0))).cuda()
        lens = torch.from_numpy(np.random.default_rng(cols).integers(0, cols + 1, rows).astype(np.int32)).cuda()
        y = torch.empty_like(x)
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(max(1, args.warmup)):
            tf.tf_softmax_len_fwd(x, lens, y)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            tf.tf_softmax_len_fwd(x, lens, y)
        e.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(e) / args.steps
        live = int(lens.sum().item()) * inputs.ELEM_SIZE[dt]
        nbytes = live + rows * cols * inputs.ELEM_SIZE[dt] + 4 * rows
        print(json.dumps({"case": f"case_softmax_len_{dts}_{rows}x{cols}", "launches": args.steps, "us_per_launch": us, "gbs": nbytes / us / 1e3}))
        return
    if parts[0] == "normbwd":                 # normbwd:op:dtype:rows:cols -- the backward pass of a norm
        op, dts, rows, cols = parts[1], parts[2], int(parts[3]), int(parts[4])
        dt = inputs.F32 if dts == "f32" else inputs.BF16
        tdt = torch.float32 if dt == inputs.F32 else torch.bfloat16
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        x = conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols, 0, 0.3, 2.0))).cuda()
        dy = conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols + 1, 3, 0.0, 1.0))).cuda()
        g = (torch.rand(cols, device="cuda") + 0.5).to(tdt)
        dx = torch.empty_like(x)
        if op == "layernorm":
            _, mean, rstd = tf.tf_layernorm_fwd(x, g, torch.zeros_like(g), 1e-5)
            call = lambda: tf.tf_layernorm_bwd(x, g, dy, mean, rstd, dx=dx)
        else:
            _, rstd = tf.tf_rmsnorm_fwd(x, g, 1e-6, want_rstd=True)
            call = lambda: tf.tf_rmsnorm_bwd(x, g, dy, rstd, dx=dx)
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(max(1, args.warmup)):
            call()
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            call()
        e.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(e) / args.steps
        nbytes = 3 * rows * cols * inputs.ELEM_SIZE[dt]
        print(json.dumps({"case": f"case_{op}_bwd_{dts}_{rows}x{cols}", "launches": args.steps, "us_per_launch": us, "gbs": nbytes / us / 1e3}))
        return
    if parts[0] == "sine":                    # sine:dtype:elements[:threads:vectors] -- the element-wise sine, inputs as in the sine table
        dts, n = parts[1], int(parts[2])
        threads, vectors = (int(parts[3]), int(parts[4])) if len(parts) > 4 else (0, 0)
        tdt = torch.float32 if dts == "f32" else torch.bfloat16
        gen = torch.Generator(device="cuda").manual_seed(n)
        x = (torch.rand(n, device="cuda", generator=gen) * 200.0 - 100.0).to(tdt)
        y = torch.empty_like(x)
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(max(1, args.warmup)):
            tf.tf_sin_fwd(x, y, threads, vectors)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            tf.tf_sin_fwd(x, y, threads, vectors)
        e.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(e) / args.steps
        print(json.dumps({"case": f"case_sin_{dts}_{n}", "launches": args.steps, "us_per_launch": us, "gbs": 2 * n * x.element_size() / us / 1e3}))
        return
    if parts[0] == "addnorm":                 # addnorm:op:dtype:rows:cols -- the fused residual add + norm, heuristic plan
        op, dts, rows, cols = parts[1], parts[2], int(parts[3]), int(parts[4])
        dt = inputs.F32 if dts == "f32" else inputs.BF16
        w = inputs.Workload(f"case_add_{op}_{dts}_{rows}x{cols}", op, dt, rows, cols, seed=cols, eps=1e-5 if op == "layernorm" else 1e-6)
        data = w.generate()
        conv = (lambda t: t.view(torch.bfloat16)) if dt == inputs.BF16 else (lambda t: t)
        x = conv(torch.from_numpy(data["x"])).cuda()
        r = conv(torch.from_numpy(inputs.normal((rows, cols), dt, cols + 1, 7, 0.0, 1.0))).cuda()
        g = conv(torch.from_numpy(data["gamma"] if op == "layernorm" else data["w"])).cuda()
        b = conv(torch.from_numpy(data["beta"])).cuda() if op == "layernorm" else None
        h, y = torch.empty_like(x), torch.empty_like(x)
        if not args.no_tune:
            tf.tf_tune_add(op, rows, cols, dt)
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def call():
            if op == "layernorm":
                tf.tf_add_layernorm_fwd(x, r, g, b, w.eps, h=h, y=y, want_stats=False)
            else:
                tf.tf_add_rmsnorm_fwd(x, r, g, w.eps, h=h, y=y)
        for _ in range(max(1, args.warmup)):
            call()
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            call()
        e.record()
        torch.cuda.synchronize()
        us = 1e3 * a.elapsed_time(e) / args.steps
        nbytes = 4 * rows * cols * w.elem_size + (2 if op == "layernorm" else 1) * cols * w.elem_size
        print(json.dumps({"case": w.name, "launches": args.steps, "us_per_launch": us, "gbs": nbytes / us / 1e3}))
        return
    if parts[0] == "config":
        w = inputs.config(int(parts[1]))
        if len(parts) > 2:
            w = inputs.Workload(w.name, w.op, w.dt, int(parts[2]), w.cols, seed=w.seed, x_mean=w.x_mean, x_std=w.x_std, eps=w.eps,
                                outlier_p=w.outlier_p, outlier_factor=w.outlier_factor,
                                mask_step=int(parts[3]) if len(parts) > 3 else w.mask_step, scale=w.scale, shift=w.shift)
    else:
        op, dt, rows, cols = parts
        eps = {"softmax": 0.0, "layernorm": 1e-5, "rmsnorm": 1e-6}[op]
        w = inputs.Workload(f"case_{op}_{dt}_{rows}x{cols}", op, inputs.F32 if dt == "f32" else inputs.BF16, int(rows), int(cols),
                            seed=int(cols), eps=eps)
    case = DeviceCase(w, w.generate(), torch.device("cuda", 0), min_total_bytes=0)
    if args.plan:
        tf.tf_force_plan(w.op, args.plan)
    elif not args.no_tune:
        tf.tf_tune(w.op, w.rows, w.cols, w.dt, like=(case.x[0], case.params.get("gamma", case.params.get("w")), case.params.get("beta")))
    ms = case.time_steps(args.steps, max(1, args.warmup))
    tf.tf_device_status()
    print(json.dumps({"case": w.name, "plan": args.plan or tf.tf_query_choice(w.op, w.rows, w.cols, w.dt), "launches": args.steps,
                      "us_per_launch": 1e3 * ms / args.steps, "gbs": case.bytes_per_step / (ms * 1e-3 / args.steps) / 1e9}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--table", choices=["configs", "sweep", "vecmat", "addnorm", "softmaxlen", "softmaxvariants", "normbwd", "launch", "sine"], default=None)
    ap.add_argument("--filter", default=None)
    ap.add_argument("--out", default=str(ROOT / "bench_out"), help="folder for the JSON files the --table modes write")
    ap.add_argument("--no-extras", action="store_true", help="default run: skip per_config and sweep_summary")
    ap.add_argument("--sweep-tune", action="store_true", help="default run: tune every sweep point before timing it")
    ap.add_argument("--no-tune", action="store_true")
    ap.add_argument("--cpu", action="store_true", help="with --table: also time the oracle")
    ap.add_argument("--case", default=None, help="op:dtype:rows:cols, config:<i>[:rows], vecmat:..., addnorm:op:dtype:rows:cols, normbwd:op:dtype:rows:cols, softmaxlen:dtype:rows:cols, sine:dtype:elements[:threads:vectors] -- a few launches of one shape")
    ap.add_argument("--plan", default=None, help="with --case: force this launch plan")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        return run_reference(args)
    args.steps = 20 if args.steps is None else args.steps
    args.warmup = 5 if args.warmup is None else args.warmup
    import __graft_entry__
    __graft_entry__.build()
    if args.case:
        return run_case(args)
    if args.table == "vecmat":
        return run_vecmat_table(args)
    if args.table == "addnorm":
        return run_addnorm_table(args)
    if args.table == "softmaxlen":
        return run_softmaxlen_table(args)
    if args.table == "softmaxvariants":
        return run_softmax_variants_table(args)
    if args.table == "normbwd":
        return run_normbwd_table(args)
    if args.table == "launch":
        return run_launch_table(args)
    if args.table == "sine":
        return run_sine_table(args)
    if args.table:
        return run_table(args)
    run_ours(args)


if __name__ == "__main__":
    main()
