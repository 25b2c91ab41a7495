"""GPU parity: every variant forced explicitly and the automatic choice, both dtypes, edge shapes, against the
CPU oracle, through the C ABI."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
from paper_2512_09196_b200.inputs import BF16, F32, Workload
import parity

pytestmark = pytest.mark.gpu

OPS = ("softmax", "layernorm", "rmsnorm")
EPS = {"softmax": 0.0, "layernorm": 1e-5, "rmsnorm": 1e-6}


def wl(op, dt, rows, cols, seed=7, **kw):
    kw.setdefault("x_mean", 0.3)
    kw.setdefault("x_std", 2.0)
    return Workload(f"{op}-{dt}-{rows}x{cols}", op, dt, rows, cols, seed=seed, eps=EPS[op], **kw)


@pytest.fixture(autouse=True)
def _auto_plans():
    yield
    for op in OPS:
        tf.tf_force_plan(op, None)


# ------------------------------------------------------------------ automatic choice over edge shapes

@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("cols", [1, 2, 3, 7, 8, 31, 32, 33, 64, 100, 256, 1000, 1001, 1024, 4096, 4097, 5120, 12288, 40000])
def test_auto_edge_cols(op, dt, cols):
    for rows in (1, 37):
        fails = parity.parity(wl(op, dt, rows, cols, seed=cols))
        assert not fails, f"{tf.tf_query_choice(op, rows, cols, dt, (cols * (4 if dt == F32 else 2)) % 16 == 0)}: {fails}"


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("rows", [2, 147, 148, 149, 1000])
def test_auto_edge_rows(op, rows):
    for dt, cols in ((F32, 520), (BF16, 2048)):
        assert not parity.parity(wl(op, dt, rows, cols, seed=rows))


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_long_rows_take_the_cluster_path(op, dt):
    cols = 131072 if dt == BF16 else 65536 + 64
    w = wl(op, dt, 21, cols)
    assert tf.tf_query_choice(op, 21, cols, dt).startswith(("ring:", "twopass:", "split:"))
    assert not parity.parity(w)
    w2 = wl(op, dt, 3, 1 << 20)          # 2-4 MiB rows: more than a cluster of shared memory holds
    assert tf.tf_query_choice(op, 3, 1 << 20, dt).startswith(("ring:", "tma:", "twopass:", "split:"))
    assert not parity.parity(w2)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_misaligned_base_and_inplace(op, dt):
    for cols in (64, 1000, 4096):
        w = wl(op, dt, 19, cols)
        assert not parity.parity(w, offset=1), "misaligned base"
        assert not parity.parity(w, inplace=True), "in place"
        assert not parity.parity(w, offset=3, inplace=True), "misaligned and in place"


def test_rows_zero_is_a_noop_and_bad_args_are_rejected():
    x = torch.empty((0, 16), device="cuda")
    tf.tf_softmax_fwd(x)
    L = tf.lib()
    buf = torch.zeros(64, device="cuda")
    p = buf.data_ptr()
    assert L.tf_softmax_fwd(None, p, 2, 8, 0, None) == 1
    assert L.tf_softmax_fwd(p, p, -1, 8, 0, None) == 1
    assert L.tf_softmax_fwd(p, p, 2, 0, 0, None) == 1
    assert L.tf_softmax_fwd(p, p, 2, 8, 5, None) == 1
    assert L.tf_layernorm_fwd(p, None, p, p, None, None, 2, 8, 1e-5, 0, None) == 1
    assert L.tf_layernorm_fwd(p, p, p, p, None, None, 2, 8, -1.0, 0, None) == 1
    assert L.tf_layernorm_fwd(p, p, p, p, None, None, 2, 8, float("nan"), 0, None) == 1
    assert L.tf_rmsnorm_fwd(p, None, p, None, 2, 8, 1e-6, 0, None) == 1
    assert L.tf_softmax_fwd(p, p, 1 << 40, 1 << 40, 0, None) == 2
    assert L.tf_tune(7, 2, 8, 0) == 1
    assert L.tf_force_plan(0, b"nonsense:threads=3") == 1
    assert L.tf_status_string(2) == b"unsupported size or plan"


# ------------------------------------------------------------------ special values

@pytest.mark.parametrize("dt", [F32, BF16])
def test_softmax_masks_fully_masked_rows_and_subnormals(dt):
    for cols, plan in ((64, None), (4096, None), (131072, None), (4096, "stream:threads=256,lanes=0")):
        tf.tf_force_plan("softmax", plan)
        w = Workload("m", "softmax", dt, 24, cols, seed=5, x_std=10.0, mask_step=max(1, cols // 16 + 3))
        data = w.generate()
        x = data["x"]
        ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
        x[3, :] = ninf                                     # fully masked row -> all +0
        x[5, : cols // 2] = ninf                           # masked head instead of tail
        x[7, ::2] = ninf                                   # alternating
        x[9, 0] = np.float32(75.0) if dt == F32 else np.uint16(0x4296)   # 75.0: pushes much of the row to e^-88 and below
        got, ref = parity.run_gpu(w, data), parity.run_oracle(w, data)
        assert not parity.check(w, data, got, ref)
        assert not got["y"][3].any()
        if dt == BF16 and cols >= 4096:
            sub = (ref["y"] > 0) & (ref["y"] < 0x0080)
            assert sub.any(), "the case is meant to produce bf16 subnormal outputs"


@pytest.mark.parametrize("op", ["layernorm", "rmsnorm"])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_norm_degenerate_rows(op, dt):
    for cols in (8, 512, 8192):
        w = wl(op, dt, 6, cols)
        data = w.generate()
        x = data["x"]
        x[1, :] = x[1, 0]                                  # constant row: variance 0
        x[2, :] = 0                                        # all zeros
        if dt == F32:
            x[3, :] *= np.float32(1e4)
        got, ref = parity.run_gpu(w, data), parity.run_oracle(w, data)
        assert not parity.check(w, data, got, ref)


def test_rmsnorm_outliers_and_optional_rstd():
    w = Workload("o", "rmsnorm", BF16, 64, 8192, seed=2, eps=1e-6, outlier_p=0.01, outlier_factor=100.0,
                 scale=("normal", 1.0, 0.1))
    assert not parity.parity(w)
    assert not parity.parity(w, rms_rstd=False)


def test_nan_row_does_not_leak_into_other_rows():
    w = wl("softmax", F32, 8, 1024)
    data = w.generate()
    data["x"][4, 100] = np.nan
    got, ref = parity.run_gpu(w, data), parity.run_oracle(w, data)
    keep = [r for r in range(8) if r != 4]
    sub = {"x": data["x"][keep]}
    assert not parity.check(w, sub, {"y": got["y"][keep]}, {"y": ref["y"][keep], "y64": ref["y64"][keep]})
    assert np.isnan(got["y"][4]).any()


# ------------------------------------------------------------------ every variant, forced

WARP_PLANS = [(l, v, r) for (l, v, r) in [(8, 1, 1), (8, 1, 2), (8, 1, 4), (8, 2, 1), (8, 2, 2), (16, 1, 1), (16, 1, 2),
                                           (16, 1, 4), (16, 2, 1), (16, 2, 2), (32, 1, 1), (32, 1, 2), (32, 1, 4),
                                           (32, 2, 1), (32, 2, 2), (32, 4, 1), (32, 4, 2), (32, 8, 1)]]


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_warp_variants(op, dt):
    ne = 4 if dt == F32 else 8
    for lanes, vpt, rpg in WARP_PLANS:
        cap = lanes * vpt                               # vectors the group can hold
        for nvec in {cap, max(1, cap - 1), max(1, cap // 2 + 1)}:
            for threads, persist in ((128, 0), (256, 1)):
                tf.tf_force_plan(op, f"warp:threads={threads},lanes={lanes},vpt={vpt},rpg={rpg},persist={persist}")
                fails = parity.parity(wl(op, dt, 301, nvec * ne, seed=nvec))
                assert not fails, (lanes, vpt, rpg, nvec, threads, fails)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_forced_cta_variants(op, dt, cluster):
    ne = 4 if dt == F32 else 8
    for vpt in (1, 2, 4, 8):
        for threads in (64, 256) + ((1024,) if vpt <= 2 else (512,)):
            cap = threads * vpt * cluster
            for nvec in {cap, cap - 1, cap - threads - 3, max(1, cap // 2 + 5)}:
                if nvec < 1:
                    continue
                for persist in (0, 1):
                    tf.tf_force_plan(op, f"cta:threads={threads},vpt={vpt},cluster={cluster},persist={persist}")
                    rows = 9 if persist == 0 else min(700, max(160, (1 << 20) // (nvec * ne)))   # > 148 clusters' worth
                    fails = parity.parity(wl(op, dt, rows if nvec < 4096 else 5, nvec * ne, seed=nvec))
                    assert not fails, (vpt, threads, cluster, nvec, persist, fails)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_forced_tma_variants(op, dt, cluster):
    ne = 4 if dt == F32 else 8
    for nvec in (cluster * 512, cluster * 4096 - 1, cluster * 2048 + 77, 1000):
        for threads, stages, chunk, persist, rows in ((128, 1, 4096, 0, 7), (512, 1, 8192, 0, 7), (1024, 2, 32768, 1, 400),
                                                       (256, 3, 16384, 1, 900), (256, 2, 1024, 2, 1300)):
            tf.tf_force_plan(op, f"tma:threads={threads},cluster={cluster},stages={stages},chunk={chunk},persist={persist}")
            rows = min(rows, max(7 if persist == 0 else 2 * 148 // cluster + 9, (1 << 21) // (nvec * ne)))
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec))
            assert not fails, (cluster, nvec, threads, stages, chunk, persist, fails)


PIPE_COMBOS = [(8, 1), (16, 1), (32, 1), (32, 2), (32, 4), (32, 8), (64, 2), (64, 4), (64, 8), (128, 2), (128, 4), (128, 8),
               (256, 2), (256, 4), (256, 8), (512, 4), (512, 8), (160, 4), (160, 8), (320, 4), (192, 8), (384, 4), (384, 8)]


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_pipe_variants(op, dt):
    ne = 4 if dt == F32 else 8
    ran = 0
    for ci, (lanes, vpt) in enumerate(PIPE_COMBOS):
        cap = lanes * vpt
        ut = max(32, lanes)
        threads = (512 if ci % 2 else max(256, ut)) // ut * ut
        # rows chosen so that a unit wraps its ring several times and the last tile is ragged
        for nvec, stages, chunk, persist, rows in ((cap, 2, 4096, 1, 4001), (max(1, cap - 1), 3, 16384, 2, 2999),
                                                   (max(1, cap // 2 + 1), 1, 2048, 1, 1777), (cap, 4, 512, 8, 77)):
            chunk = max(chunk, nvec * 16 * (ut // lanes))
            rpg = 2 if (vpt <= 4 and nvec == cap and stages != 3) else 1        # two rows per pass needs a full row
            plan = f"pipe:threads={threads},lanes={lanes},vpt={vpt},rpg={rpg},stages={stages},chunk={chunk},persist={persist}"
            tf.tf_force_plan(op, plan)
            if nvec * 16 > 8192:
                rows = max(40, rows // 16)
            w = wl(op, dt, rows, nvec * ne, seed=nvec)
            try:
                fails = parity.parity(w)
            except tf.TfError as e:
                assert e.status == 2, plan                     # ring does not fit shared memory: refused, not wrong
                continue
            ran += 1
            assert not fails, (plan, nvec, fails)
    assert ran >= 30


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_forced_ring_variants(op, dt, cluster):
    ne = 4 if dt == F32 else 8
    for vpt, threads in ((1, 128), (2, 256), (4, 1024), (8, 512), (4, 96)):
        cap = threads * vpt * cluster
        for nvec, stages, persist, rows in ((cap, 2, 1, 2 * 148 // cluster + 11), (cap - 1, 3, 2, 700 // cluster + 5),
                                            (max(1, cap - threads - 3), 1, 1, 19), (max(1, cap // 2 + 5), 4, 1, 3)):
            if nvec * 16 * stages // cluster > 180 * 1024 // persist:
                continue
            rows = min(rows, max(3, (1 << 22) // (nvec * ne)))
            for psmem in ((0, 1) if vpt == 8 and op != "softmax" and nvec * 16 * (stages + 2) // cluster <= 180 * 1024 // persist else (0,)):
                tf.tf_force_plan(op, f"ring:threads={threads},vpt={vpt},cluster={cluster},stages={stages},persist={persist},psmem={psmem}")
                fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec))
                assert not fails, (vpt, threads, cluster, nvec, stages, persist, psmem, rows, fails)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_srows_variants(op, dt):
    # rows resident in shared memory, 1-8 lanes per row: rows that fill the lanes exactly and ragged ones, a single vector,
    # blocks of rows with a ragged last block, one row, in place
    ne = 4 if dt == F32 else 8
    ran = 0
    for threads in (64, 128, 256):
        for lanes in (1, 2, 4, 8):
            for vpt in (4, 8, 16):
                cap = lanes * vpt
                rpc = threads // lanes
                if op == "softmax" and vpt != 4:                   # softmax keeps its exponentials in registers: four vectors per lane
                    tf.tf_force_plan(op, f"srows:threads={threads},lanes={lanes},vpt={vpt}")
                    with pytest.raises(tf.TfError) as e:
                        parity.parity(wl(op, dt, 5, cap * ne, seed=1))
                    assert e.value.status == 2
                    continue
                for nvec, rows in ((cap, 3 * rpc + 5), (cap, 1), (cap - 1, rpc + 1), (max(1, cap // 2 + 1), 2 * rpc - 1), (1, 7)):
                    tf.tf_force_plan(op, f"srows:threads={threads},lanes={lanes},vpt={vpt}")
                    fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec + rows))
                    assert not fails, (threads, lanes, vpt, nvec, rows, fails)
                    ran += 1
                fails = parity.parity(wl(op, dt, rpc + 3, cap * ne, seed=cap), inplace=True)
                assert not fails, ("in place", threads, lanes, vpt, fails)
    assert ran == (60 if op == "softmax" else 180)
    tf.tf_force_plan(op, "srows:threads=128,lanes=8,vpt=8")        # a row longer than the lanes hold: refused
    with pytest.raises(tf.TfError):
        parity.parity(wl(op, dt, 4, 65 * ne, seed=1))


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_twopass_variants(op, dt):
    ne = 4 if dt == F32 else 8
    for threads, persist, regcap in ((32, 0, 0), (256, 1, 0), (1024, 0, 0), (512, 0, 1), (768, 0, 1), (96, 2, 1)):
        for nvec, rows in ((1, 5), (threads * 4, 9), (threads * 4 + 1, 9), (threads * 9 - 3, 300), (70001, 3)):
            tf.tf_force_plan(op, f"twopass:threads={threads},persist={persist},regcap={regcap}")
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec))
            assert not fails, (threads, persist, regcap, nvec, rows, fails)
    # a thread-block cluster per row: ragged and empty slices, one row, rows left over after the last full pass, heads in shared memory
    for cluster, threads, persist, regcap, cache in ((2, 256, 0, 0, 0), (4, 512, 0, 1, 4096), (8, 128, 1, 0, 0), (8, 1024, 2, 0, 16384), (2, 768, 0, 1, 49152)):
        for nvec, rows in ((cluster, 5), (cluster + 1, 3), (threads * 4 * cluster + 1, 9), (threads * 9 - 3, 150), (70001, 3), (9, 1)):
            tf.tf_force_plan(op, f"twopass:threads={threads},cache={cache},persist={persist},regcap={regcap},cluster={cluster}")
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec + cluster))
            assert not fails, (cluster, threads, persist, regcap, cache, nvec, rows, fails)
    # the ring form (asynchronous copies into a private shared-memory ring): rows shorter than the ring, exactly one ring,
    # ragged last steps, rows taken in interleaved order, every hint combination, persistent grids
    for threads, stages, u, persist, regcap, groups, hints in ((32, 2, 4, 0, 0, 1, 3), (256, 3, 2, 1, 1, 8, 0), (512, 2, 4, 0, 1, 3, 1),
                                                               (1024, 2, 2, 0, 0, 1, 2), (384, 4, 4, 2, 1, 16, 3), (128, 8, 2, 0, 1, 2, 3)):
        for nvec, rows in ((1, 5), (threads * u, 9), (threads * u * stages, 7), (threads * u * stages + 1, 9), (threads * 9 - 3, 300), (70001, 3)):
            plan = f"twopass:threads={threads},persist={persist},regcap={regcap},groups={groups},hints={hints},stages={stages},u={u}"
            tf.tf_force_plan(op, plan)
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec + stages))
            assert not fails, (plan, nvec, rows, fails)
            fails = parity.parity(wl(op, dt, min(rows, 11), nvec * ne, seed=nvec + stages), inplace=True)
            assert not fails, ("in place", plan, nvec, rows, fails)
    # the ring form with the CTAs of a cluster sharing a row step by step: rows shorter than one CTA's step (CTAs without
    # work), ragged steps falling to every rank, persistent clusters, one row
    for cluster, threads, stages, u, persist, regcap in ((2, 128, 2, 4, 0, 1), (4, 256, 3, 2, 0, 0), (8, 64, 2, 4, 1, 1), (2, 512, 3, 4, 0, 0)):
        st = threads * u
        for nvec, rows in ((1, 3), (st, 5), (st + 1, 5), (st * cluster - 1, 9), (st * cluster * stages + 5, 9), (st * (cluster + 1) + 7, 150), (70001, 3), (st * 3, 1)):
            plan = f"twopass:threads={threads},persist={persist},regcap={regcap},cluster={cluster},stages={stages},u={u}"
            tf.tf_force_plan(op, plan)
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec + cluster))
            assert not fails, (plan, nvec, rows, fails)
    # rows that fit the ring (straight-line build, one row per CTA or per cluster): a single vector, steps without work,
    # rows that fill the steps exactly and by one vector less, a last CTA that falls short, one row; one vector more than
    # fits goes to the general ring form
    for cluster, threads, stages in ((1, 64, 2), (1, 96, 3), (1, 256, 4), (1, 128, 2), (2, 128, 2), (4, 64, 4), (8, 32, 3), (2, 512, 2)):
        st, cap = threads * 4, threads * 4 * cluster * stages
        for nvec, rows in ((1, 3), (st - 1, 5), (st, 150), (st * cluster, 9), (cap, 9), (cap - 1, 300), (cap - st - 3, 9),
                           (cap - st * cluster + 5, 1), (cap + 1, 5)):
            plan = f"twopass:threads={threads},persist=0,regcap=0,cluster={cluster},stages={stages},u=4"
            tf.tf_force_plan(op, plan)
            fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec + cluster))
            assert not fails, (plan, nvec, rows, fails)
            fails = parity.parity(wl(op, dt, min(rows, 7), nvec * ne, seed=nvec + stages), inplace=True)
            assert not fails, ("in place", plan, nvec, rows, fails)
    for groups in (2, 8, 1000):                            # the direct form with interleaved row order
        tf.tf_force_plan(op, f"twopass:threads=256,persist=0,groups={groups},hints=0")
        assert not parity.parity(wl(op, dt, 37, 5000 * ne, seed=groups)), groups
    if op == "softmax":                                    # masks, a fully masked row and outputs in the subnormal range
        for plan in ("twopass:threads=256,persist=0,cluster=4", "twopass:threads=512,cache=8192,persist=0,regcap=1,cluster=8",
                     "twopass:threads=256,persist=0,stages=2,u=4", "twopass:threads=128,persist=0,regcap=1,stages=3,u=2,groups=4",
                     "twopass:threads=128,persist=0,regcap=1,stages=2,u=4,cluster=2", "twopass:threads=64,persist=0,stages=3,u=2,cluster=8",
                     "twopass:threads=512,persist=0,stages=4,u=4", "twopass:threads=256,persist=0,stages=3,u=4,cluster=4"):
            tf.tf_force_plan(op, plan)
            w = Workload("m", "softmax", dt, 12, 40000, seed=5, x_std=10.0, mask_step=3001)
            data = w.generate()
            ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
            data["x"][3, :] = ninf                                   # fully masked row
            data["x"][5, :20000] = ninf                              # whole slices masked
            data["x"][7, 0] = np.float32(75.0) if dt == F32 else np.uint16(0x4296)
            assert not parity.check(w, data, parity.run_gpu(w, data), parity.run_oracle(w, data)), plan
        tf.tf_force_plan(op, "twopass:threads=256,persist=0")
        w = Workload("m", "softmax", dt, 12, 40000, seed=5, x_std=10.0, mask_step=3001)
        data = w.generate()
        ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
        data["x"][3, :] = ninf
        data["x"][5, :20000] = ninf
        data["x"][7, 0] = np.float32(75.0) if dt == F32 else np.uint16(0x4296)
        assert not parity.check(w, data, parity.run_gpu(w, data), parity.run_oracle(w, data))


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_split_variants_and_few_long_rows(op, dt):
    ne = 4 if dt == F32 else 8
    for threads, splits, nvec, rows in ((32, 2, 5, 3), (256, 7, 4099, 4), (512, 64, 40000, 2), (1024, 300, 70001, 1), (128, 8, 8, 5)):
        tf.tf_force_plan(op, f"split:threads={threads},splits={splits}")
        fails = parity.parity(wl(op, dt, rows, nvec * ne, seed=nvec))
        assert not fails, (threads, splits, nvec, rows, fails)
    tf.tf_force_plan(op, None)
    for rows, cols in ((1, 262144), (3, 524288), (8, 131072), (64, 32768)):  # what a decode-time vocabulary softmax looks like
        if rows <= 4:
            assert tf.tf_query_choice(op, rows, cols, dt).startswith("split:")
        assert not parity.parity(wl(op, dt, rows, cols, seed=rows))
    if op == "softmax":
        tf.tf_force_plan(op, "split:threads=256,splits=16")
        w = Workload("m", "softmax", dt, 6, 40000, seed=5, x_std=10.0, mask_step=3001)
        data = w.generate()
        ninf = np.float32(-np.inf) if dt == F32 else np.uint16(0xFF80)
        data["x"][1, :] = ninf                                   # fully masked row
        data["x"][2, :30000] = ninf                              # whole segments masked
        data["x"][3, 0] = np.float32(75.0) if dt == F32 else np.uint16(0x4296)
        assert not parity.check(w, data, parity.run_gpu(w, data), parity.run_oracle(w, data))


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_stream_variants(op, dt):
    for lanes in (32, 0):
        for threads in (64, 1024):
            for cols in (1, 5, 999, 4099):
                tf.tf_force_plan(op, f"stream:threads={threads},lanes={lanes},persist=0")
                assert not parity.parity(wl(op, dt, 41, cols, seed=cols), offset=1)
            tf.tf_force_plan(op, f"stream:threads={threads},lanes={lanes},persist=1")
            assert not parity.parity(wl(op, dt, 5000, 40, seed=1))


def test_forced_plan_that_cannot_hold_the_row_is_refused():
    tf.tf_force_plan("softmax", "warp:threads=256,lanes=8,vpt=1,rpg=1")
    x = torch.zeros((4, 4096), device="cuda")
    with pytest.raises(tf.TfError) as e:
        tf.tf_softmax_fwd(x)
    assert e.value.status == 2
    tf.tf_force_plan("softmax", "cta:threads=64,vpt=1,cluster=1")
    with pytest.raises(tf.TfError):
        tf.tf_softmax_fwd(x)
    tf.tf_force_plan("softmax", "tma:threads=256,cluster=1,stages=3,chunk=8192")
    with pytest.raises(tf.TfError):
        tf.tf_softmax_fwd(torch.zeros((2, 1 << 16), device="cuda"))        # 3 x 256 KiB of shared memory
    tf.tf_force_plan("softmax", "warp:threads=256,lanes=8,vpt=1,rpg=1")
    xu = torch.zeros(4 * 32 + 1, device="cuda")[1:].view(4, 32)             # misaligned: vector plans refuse
    with pytest.raises(tf.TfError):
        tf.tf_softmax_fwd(xu)
