"""Softmax with per-row valid lengths through the C ABI against the CPU oracle.  The tails of x hold NaN in every
test: a kernel that read them would poison its row."""
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
NAN = {F32: np.float32(np.nan), BF16: np.uint16(0x7FC0)}
NINF = {F32: np.float32(-np.inf), BF16: np.uint16(0xFF80)}


@pytest.fixture(autouse=True)
def _auto_plans():
    yield
    tf.tf_force_plan("softmax", None)


def lengths_for(rows, cols, seed):
    rng = np.random.default_rng(seed)
    ne = 8
    lens = rng.integers(0, cols + 1, rows).astype(np.int32)
    special = [0, 1, cols, max(0, cols - 1), min(cols, ne), min(cols, ne + 1), min(cols, max(0, ne - 1)), cols // 2]
    lens[:min(rows, len(special))] = special[:min(rows, len(special))]
    return lens


def run_case(dt, rows, cols, seed=1, offset=0, inplace=False, x_std=3.0, compare_plain=False):
    x = inputs.normal((rows, cols), dt, seed, 0, 0.0, x_std)
    lens = lengths_for(rows, cols, seed)
    poisoned, masked = x.copy(), x.copy()
    for r in range(rows):
        poisoned[r, lens[r]:] = NAN[dt]
        masked[r, lens[r]:] = NINF[dt]
    ref, ref64 = oracle.softmax_len(poisoned, lens, dt, want64=True, nthreads=8)
    xd = parity.to_dev(poisoned, dt, offset)
    ld = torch.from_numpy(lens).cuda()
    y = tf.tf_softmax_len_fwd(xd, ld, xd if inplace else parity.guarded(tuple(xd.shape), xd.dtype, offset, name="y"))
    torch.cuda.synchronize()
    tf.tf_device_status()
    got = parity.to_host(y, dt)
    rep = compare.compare_softmax(got, ref, ref64, masked, dt)          # masked positions must hold the bits of +0
    assert rep.ok, (dt, rows, cols, offset, inplace, str(rep))
    if compare_plain:                                                   # same plan, mask in the data: the same bits
        plain = parity.to_host(tf.tf_softmax_fwd(parity.to_dev(masked, dt, offset)), dt)
        np.testing.assert_array_equal(got, plain)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_automatic_plan_over_edge_widths(dt):
    ne = 4 if dt == F32 else 8
    for cols in (ne, 2 * ne, 3 * ne, 64, 256, 1000 // ne * ne, 1024, 4096, 5120, 12288, 32768, 65536, 200000 // ne * ne):
        rows = max(9, min(200, (1 << 21) // cols))
        run_case(dt, rows, cols, seed=cols)
    run_case(dt, 0, 64)
    run_case(dt, 1, 4096)
    run_case(dt, 500, 2048, inplace=True)
    run_case(dt, 9, 65536, inplace=True, x_std=20.0)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_unaligned_and_odd_widths_take_the_scalar_kernel(dt):
    run_case(dt, 9, 1001)
    run_case(dt, 9, 7)
    run_case(dt, 11, 1024, offset=1)
    run_case(dt, 11, 4099, offset=3, inplace=True)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_forced_plans_and_bitwise_equality_with_the_masked_plain_softmax(dt):
    ne = 4 if dt == F32 else 8
    for lanes, vpt, rpg in ((8, 1, 1), (8, 2, 2), (16, 1, 4), (32, 2, 2), (32, 4, 1), (32, 8, 1)):
        cap = lanes * vpt
        for nvec in (cap, max(1, cap - 1)):
            tf.tf_force_plan("softmax", f"warp:threads=128,lanes={lanes},vpt={vpt},rpg={rpg},persist=0")
            run_case(dt, 301, nvec * ne, seed=nvec, compare_plain=True)
    for cluster in (1, 2, 8):
        for vpt, threads in ((1, 64), (2, 1024), (4, 256), (8, 512)):
            cap = threads * vpt * cluster
            for nvec, persist in ((cap, 0), (max(1, cap - threads - 3), 1)):
                tf.tf_force_plan("softmax", f"cta:threads={threads},vpt={vpt},cluster={cluster},persist={persist}")
                run_case(dt, 9 if nvec >= 4096 else 170, nvec * ne, seed=nvec, compare_plain=vpt <= 4 or dt == F32)   # bf16 x 8 vectors: own choice
    for threads, cache, regcap, persist in ((32, 0, 0, 0), (256, 4096, 1, 0), (512, 49152, 1, 0), (1024, 0, 0, 2)):
        for nvec, rows in ((1, 9), (threads * 4 + 1, 9), (threads * 9 - 3, 60), (70001, 9)):
            tf.tf_force_plan("softmax", f"twopass:threads={threads},cache={cache},persist={persist},regcap={regcap}")
            run_case(dt, rows, nvec * ne, seed=nvec, compare_plain=True)
    for cluster, threads, cache in ((2, 256, 0), (4, 512, 8192), (8, 128, 0)):           # lengths that end inside any slice, or before the first
        for nvec, rows in ((cluster + 1, 9), (threads * 4 * cluster + 1, 9), (70001, 9)):
            tf.tf_force_plan("softmax", f"twopass:threads={threads},cache={cache},persist=0,regcap=0,cluster={cluster}")
            run_case(dt, rows, nvec * ne, seed=nvec + cluster)
    # the pipeline: only the live part of a row is copied; exact and ragged fits, few and many rows per unit, every ring depth
    for lanes, vpt, threads, stages, persist in ((32, 2, 128, 2, 1), (32, 8, 512, 4, 2), (64, 8, 512, 2, 1), (128, 4, 256, 3, 0), (256, 8, 512, 1, 1),
                                                 (512, 4, 512, 8, 1)):
        cap = lanes * vpt
        for nvec, rows in ((cap, 9), (cap - 1, 700), (max(1, cap // 2 + 1), 3000)):
            rows = min(rows, max(3, (1 << 22) // (nvec * ne)))
            tf.tf_force_plan("softmax", f"pipe:threads={threads},lanes={lanes},vpt={vpt},rpg=1,stages={stages},chunk=16,persist={persist}")
            run_case(dt, rows, nvec * ne, seed=nvec + lanes, compare_plain=False)
    # rows that fit the ring of one CTA: only the live vectors are copied; exact and ragged fits, one to four steps
    for threads, stages in ((32, 3), (64, 2), (128, 4), (256, 2), (512, 1 + 1)):
        st = threads * 4
        for nvec, rows in ((st * stages, 9), (st * stages - 1, 170), (st + 1, 170), (1, 9), (max(1, st // 2), 301)):
            rows = min(rows, max(3, (1 << 22) // (nvec * ne)))
            tf.tf_force_plan("softmax", f"twopass:threads={threads},persist=0,regcap=0,stages={stages},u=4")
            run_case(dt, rows, nvec * ne, seed=nvec + threads)
        run_case(dt, 23, st * ne, seed=st, inplace=True)
    # ... and the rings of the CTAs of a cluster: lengths that end in any CTA's steps, or before the first
    for cluster, threads, stages in ((2, 128, 2), (4, 64, 4), (8, 32, 3), (2, 256, 1 + 1)):
        cap = threads * 4 * cluster * stages
        for nvec, rows in ((cap, 9), (cap - 1, 60), (threads * 4 * cluster + 1, 60), (cluster + 1, 9)):
            rows = min(rows, max(3, (1 << 22) // (nvec * ne)))
            tf.tf_force_plan("softmax", f"twopass:threads={threads},persist=0,regcap=0,cluster={cluster},stages={stages},u=4")
            run_case(dt, rows, nvec * ne, seed=nvec + cluster)
    # the general ring form (rows longer than the ring): lengths that end in a whole step, a ragged one, the first step, nowhere
    # (length 0), with and without a cluster, persistent grids, both register builds
    for cluster, threads, stages, persist, regcap in ((1, 64, 2, 0, 0), (1, 256, 3, 0, 1), (2, 128, 2, 0, 1), (4, 64, 4, 0, 0), (8, 32, 2, 1, 0), (2, 384, 3, 2, 1)):
        st = threads * 4
        for nvec, rows in ((st * cluster * stages + 1, 60), (st * (cluster * stages + 3) + 5, 60), (st * cluster * 9, 33), (70001, 9)):
            rows = min(rows, max(3, (1 << 22) // (nvec * ne)))
            tf.tf_force_plan("softmax", f"twopass:threads={threads},persist={persist},regcap={regcap},cluster={cluster},stages={stages},u=4")
            run_case(dt, rows, nvec * ne, seed=nvec + cluster)
        run_case(dt, 11, (st * cluster * stages * 2 + 7) * ne, seed=st, inplace=True, x_std=20.0)
    # a forced plan without a length mode (the cluster ring) falls back to the length-aware choice
    tf.tf_force_plan("softmax", "ring:threads=256,vpt=4,cluster=2,stages=2,persist=1")
    run_case(dt, 100, 2048 * ne)


def test_bad_arguments():
    L = tf.lib()
    p = torch.zeros(64, device="cuda").data_ptr()
    assert L.tf_softmax_len_fwd(p, None, p, 1, 8, 0, None) == 1
    assert L.tf_softmax_len_fwd(None, p, p, 1, 8, 0, None) == 1
    assert L.tf_softmax_len_fwd(p, p, p, 1, 0, 0, None) == 1
    assert L.tf_softmax_len_fwd(p, p, p, 1, 8, 5, None) == 1
    assert L.tf_softmax_len_fwd(p, p, p, 0, 8, 0, None) == 0
    with pytest.raises(ValueError):
        tf.tf_softmax_len_fwd(torch.zeros(4, 8, device="cuda"), torch.zeros(4, dtype=torch.int64, device="cuda"))


@pytest.mark.parametrize("dt,rows,cols", [(BF16, 16384, 8192), (F32, 65536, 1024), (BF16, 262144, 256), (BF16, 1024, 131072)])
def test_shapes_of_the_bench_table_every_element(dt, rows, cols):
    """The shapes `bench.py --table softmaxlen` times (the 128 Ki-column one on a quarter of its rows), every element."""
    run_case(dt, rows, cols, seed=cols)
