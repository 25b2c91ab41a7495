"""Batched vector-matrix product through the C ABI against the CPU oracle, element by element.

Tolerance: fp32 accumulation of K exact products in any order errs by at most (chain length) * 2^-24 * sum_k|a_k b_k|,
and no lane chain of the kernel is longer than K / 64 + 8 additions, so  |g - o| <= 1e-5 * sum_k |a_k b_k|  (o the oracle's
unrounded double) holds with margin up to K of several 10^4; bf16 outputs add half a bf16 ulp of o for the final rounding
(or sit within 1 ulp of the oracle's pattern)."""
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


def check(w: inputs.VecMat, threads=0, lanes=0, offset=0, data=None, ksplit=0, rows=0):
    data = data or w.generate()
    c, c64, sc = oracle.bvecmat(data["a"], data["b"], w.dt, want64=True, nthreads=8)
    a, b = parity.to_dev(data["a"], w.dt, offset), parity.to_dev(data["b"], w.dt, offset)
    g = tf.tf_bvecmat_fwd(a, b, parity.guarded((w.M, w.N), a.dtype, offset, name="c"), threads, lanes, rows, ksplit)
    torch.cuda.synchronize()
    r = compare.compare_values(parity.to_host(g, w.dt), c, c64, w.dt, cond=sc)
    assert r.ok, (w.name, threads, lanes, rows, ksplit, offset, str(r))
    return r


SHAPES = [(1, 1, 4), (1, 1, 1), (3, 5, 8), (2, 7, 64), (4, 33, 256), (5, 17, 1000), (3, 9, 1024), (2, 3, 4096), (7, 129, 520),
          (1, 300, 16384), (2, 2, 65536), (16, 1000, 72), (6, 11, 1001), (3, 4, 7)]


@pytest.mark.parametrize("dt", [F32, BF16])
def test_shapes_automatic_geometry(dt):
    for M, N, K in SHAPES:
        check(inputs.VecMat(f"t_{M}x{N}x{K}", dt, M, N, K, seed=M * 1000 + K))


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("lanes", [0, 4, 8, 16, 32])
def test_every_geometry(dt, lanes):
    for threads in (32, 128, 1024):
        for M, N, K in ((3, 37, 8), (2, 65, 200), (5, 129, 1032), (1, 19, 8200), (2, 16, 640), (1, 1, 32768)):
            for rows in ((0,) if lanes == 0 else (1, 2, 4)):
                check(inputs.VecMat(f"t_{M}x{N}x{K}", dt, M, N, K, seed=K + lanes), threads, lanes, rows=rows)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_every_k_split_of_the_plain_path(dt):
    for ksplit in (1, 2, 4, 8):
        for threads in (64, 256, 1024):
            for rows in (1, 2, 4):
                for M, N, K in ((3, 37, 8), (2, 65, 200), (5, 129, 1032), (1, 19, 8200), (1, 1, 32768)):
                    check(inputs.VecMat(f"t_{M}x{N}x{K}", dt, M, N, K, seed=K + ksplit), threads, 32, ksplit=ksplit, rows=rows)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_staged_path(dt):
    # lanes = 1: the shared-memory staged kernel; row lengths around the 1 KiB stage, tiles with fewer than 16 rows
    ne = 4 if dt == F32 else 8
    for M, N, K in ((1, 1, ne), (3, 37, 2 * ne), (2, 16, 1024 // (16 // ne)), (2, 33, 1024 // (16 // ne) + ne), (5, 129, 1032), (1, 19, 8200),
                    (2, 15, 640), (1, 1, 32768), (4, 64, 4096), (2, 100, 5000 // ne * ne)):
        check(inputs.VecMat(f"t_{M}x{N}x{K}", dt, M, N, K, seed=K + 1), lanes=1)


def test_every_k_split_of_the_tensor_core_path():
    for ksplit in (1, 2, 4, 8):
        for threads in (128, 256, 512):
            for M, N, K in ((3, 37, 8), (2, 65, 200), (5, 129, 1032), (1, 19, 8200), (2, 16, 640), (1, 1, 32768), (2, 32, 72), (3, 48, 136)):
                for rows in (16, 32):
                    check(inputs.VecMat(f"t_{M}x{N}x{K}", BF16, M, N, K, seed=K + ksplit), threads, 0, ksplit=ksplit, rows=rows)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_misaligned_and_odd_k_take_the_scalar_path(dt):
    for M, N, K in ((3, 37, 8), (2, 65, 201), (4, 9, 1031)):
        for offset in (0, 1, 3):
            check(inputs.VecMat(f"t_{M}x{N}x{K}", dt, M, N, K, seed=K), offset=offset)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_same_sign_terms_long_rows(dt):
    # nothing cancels: the sum equals the condition scale, so any biased rounding in a long accumulation chain shows
    for M, N, K in ((2, 40, 16384), (1, 5, 65536)):
        w = inputs.VecMat(f"pos_{M}x{N}x{K}", dt, M, N, K, seed=K)
        a = inputs.uniform((M, K), dt, K, 0, 0.5, 1.5)
        b = inputs.uniform((M, N, K), dt, K, 1, 0.5, 1.5)
        for threads in (0, 128, 512):
            check(w, threads=threads, data={"a": a, "b": b})


def test_exact_on_small_integers_and_selection():
    # integers: every fp32 partial sum is exact, so the result must equal the oracle bit for bit in any order
    rng = np.random.default_rng(3)
    M, N, K = 4, 50, 512
    a = rng.integers(-16, 17, (M, K)).astype(np.float32)
    b = rng.integers(-16, 17, (M, N, K)).astype(np.float32)
    c = oracle.bvecmat(a, b, F32)
    g = tf.tf_bvecmat_fwd(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda())
    np.testing.assert_array_equal(g.cpu().numpy(), c)
    ab, bb = torch.from_numpy(a).cuda().bfloat16(), torch.from_numpy(b).cuda().bfloat16()       # same integers, tensor-core path
    gb = tf.tf_bvecmat_fwd(ab, bb).float().cpu().numpy()
    np.testing.assert_array_equal(gb, torch.from_numpy(c).bfloat16().float().numpy())
    # a unit vector per batch entry selects one k slice: catches a wrong A row (m versus n) or a transposed B
    a[:] = 0
    for m in range(M):
        a[m, 37 * (m + 1)] = 1.0
    g = tf.tf_bvecmat_fwd(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()).cpu().numpy()
    for m in range(M):
        np.testing.assert_array_equal(g[m], b[m, :, 37 * (m + 1)])


def test_sweep_points_on_sampled_outputs():
    # full-size points: the oracle computes sampled (m, n) outputs one by one
    rng = np.random.default_rng(4)
    for w in (inputs.vecmat_headline(), inputs.vecmat_point(F32, 16384), inputs.vecmat_point(BF16, 64)):
        data = w.generate()
        a, b = parity.to_dev(data["a"], w.dt), parity.to_dev(data["b"], w.dt)
        g = parity.to_host(tf.tf_bvecmat_fwd(a, b), w.dt)
        del a, b
        ms = rng.integers(0, w.M, 256)
        ns = np.concatenate([[0, w.N - 1], rng.integers(0, w.N, 254)])
        sub_b = np.ascontiguousarray(data["b"][ms, ns][:, None, :])                 # [256, 1, K]: one output per batch entry
        sub_a = np.ascontiguousarray(data["a"][ms])
        c, c64, sc = oracle.bvecmat(sub_a, sub_b, w.dt, want64=True, nthreads=8)
        r = compare.compare_values(np.ascontiguousarray(g[ms, ns][:, None]), c, c64, w.dt, cond=sc)
        assert r.ok, (w.name, str(r))


def test_empty_and_refusals():
    L = tf.lib()
    p = torch.zeros(64, device="cuda").data_ptr()
    assert L.tf_bvecmat_fwd(p, p, p, 0, 4, 8, 0, 0, 0, 0, 0, None) == 0
    assert L.tf_bvecmat_fwd(p, p, p, 4, 0, 8, 0, 0, 0, 0, 0, None) == 0
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 0, 0, 0, 0, 0, 0, None) == 1              # K must be positive
    assert L.tf_bvecmat_fwd(None, p, p, 1, 1, 8, 0, 0, 0, 0, 0, None) == 1
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 0, 48, 0, 0, 0, None) == 1             # threads not a multiple of 32
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 0, 0, 5, 0, 0, None) == 1              # lanes must be 4, 8, 16 or 32
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 1, 0, 0, 0, 3, None) == 1           # ksplit must be 1, 2, 4 or 8
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 1, 0, 0, 4, 0, None) == 1           # tensor-core path: rows 16 or 32
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 0, 0, 0, 16, 0, None) == 1          # plain path: rows 1, 2 or 4
    assert L.tf_bvecmat_fwd(p, p, p, 1, 1, 8, 2, 0, 0, 0, 0, None) == 1              # unknown element type
    out = tf.tf_bvecmat_fwd(torch.zeros(0, 8, device="cuda"), torch.zeros(0, 3, 8, device="cuda"))
    assert out.shape == (0, 3)
