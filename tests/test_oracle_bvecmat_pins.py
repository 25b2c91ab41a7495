"""Pins for the oracle's batched vector-matrix product  C[m,n] = sum_k A[m,k] * B[m,n,k]  (the paper's Case Study 2):
closed forms, index-order traps, exact integer brute force in Python integers, linearity, numpy's float64 einsum, and
the single rounding of the stored result.  CPU only."""
from __future__ import annotations

from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F32


def f32(a):
    return np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))


def bf(a):
    t = torch.from_numpy(np.asarray(a, np.float64).astype(np.float32)).to(torch.bfloat16)
    return np.ascontiguousarray(t.view(torch.uint16).numpy())


def test_all_ones_and_ramp_closed_forms():
    M, N, K = 3, 5, 37
    _, c64, sc = oracle.bvecmat(f32(np.ones((M, K))), f32(np.ones((M, N, K))), F32, want64=True)
    np.testing.assert_array_equal(c64, np.full((M, N), float(K)))                   # sum of K ones
    np.testing.assert_array_equal(sc, c64)
    ramp = np.arange(1, K + 1, dtype=np.float64)
    a = np.broadcast_to(ramp, (M, K))
    _, c64, _ = oracle.bvecmat(f32(a), f32(np.ones((M, N, K))), F32, want64=True)
    np.testing.assert_array_equal(c64, np.full((M, N), K * (K + 1) / 2))            # 1 + 2 + ... + K
    _, c64, _ = oracle.bvecmat(f32(a), f32(np.broadcast_to(ramp, (M, N, K))), F32, want64=True)
    np.testing.assert_array_equal(c64, np.full((M, N), K * (K + 1) * (2 * K + 1) / 6))   # sum of squares
    # alternating signs cancel to zero while the condition scale counts every term
    alt = np.where(np.arange(K - 1) % 2 == 0, 1.0, -1.0)
    _, c64, sc = oracle.bvecmat(f32(alt[None]), f32(np.ones((1, 2, K - 1))), F32, want64=True)
    np.testing.assert_array_equal(c64, [[0.0, 0.0]])
    np.testing.assert_array_equal(sc, [[K - 1.0, K - 1.0]])


def test_unit_vector_selects_one_k_slice_per_batch_entry():
    # A[m,:] = e_{k(m)} picks B[m,:,k(m)]: fails if the contraction ran over n, or used A of another batch entry
    M, N, K = 4, 6, 5
    rng = np.random.default_rng(11)
    b = rng.integers(-50, 50, (M, N, K)).astype(np.float64)
    ks = [3, 0, 4, 1]
    a = np.zeros((M, K))
    for m, k in enumerate(ks):
        a[m, k] = 1.0
    _, c64, _ = oracle.bvecmat(f32(a), f32(b), F32, want64=True)
    for m, k in enumerate(ks):
        np.testing.assert_array_equal(c64[m], b[m, :, k])


def test_index_order_trap_with_distinct_powers():
    # B[m,n,k] = 2^(m*N*K + n*K + k) (all distinct bits, exact in double), A[m,k] = 1 only at k = m + 1:
    # the result names the exact element used, so any transposition of B's axes or A's shows up bit for bit
    M, N, K = 2, 3, 4
    idx = np.arange(M * N * K).reshape(M, N, K)
    b = 2.0 ** idx
    a = np.zeros((M, K))
    a[0, 1] = 1.0
    a[1, 2] = 1.0
    _, c64, _ = oracle.bvecmat(f32(a), f32(b), F32, want64=True)
    want = np.array([[2.0 ** idx[m, n, m + 1] for n in range(N)] for m in range(M)])
    np.testing.assert_array_equal(c64, want)
    # and with two active k the sum holds exactly both bits
    a[0, 3] = 1.0
    _, c64, _ = oracle.bvecmat(f32(a), f32(b), F32, want64=True)
    np.testing.assert_array_equal(c64[0], [2.0 ** idx[0, n, 1] + 2.0 ** idx[0, n, 3] for n in range(N)])


@pytest.mark.parametrize("dt", [F32, BF16])
def test_exact_integer_bruteforce(dt):
    # small integers: every product and partial sum is an integer below 2^53, so double arithmetic is exact and must
    # equal Python's unbounded integers
    M, N, K = 3, 4, 29
    rng = np.random.default_rng(12 + dt)
    lim = 100 if dt == BF16 else 2000                    # integers up to 256 are exact in bf16
    ai = rng.integers(-lim, lim + 1, (M, K))
    bi = rng.integers(-lim, lim + 1, (M, N, K))
    enc = f32 if dt == F32 else bf
    c, c64, sc = oracle.bvecmat(enc(ai), enc(bi), dt, want64=True)
    for m in range(M):
        for n in range(N):
            exact = sum(int(ai[m, k]) * int(bi[m, n, k]) for k in range(K))
            assert c64[m, n] == float(exact)
            assert sc[m, n] == float(sum(abs(int(ai[m, k]) * int(bi[m, n, k])) for k in range(K)))
    if dt == F32:
        np.testing.assert_array_equal(c, c64.astype(np.float32))
    else:
        np.testing.assert_array_equal(c, oracle.bf16_from_double(c64))


def test_exact_rational_bruteforce_on_random_floats():
    # fp32 inputs are dyadic rationals: the exact sum is a Fraction; the double result must be within the classic
    # recursive-summation bound K * 2^-53 * sum|a b| of it (and for K this small, far inside)
    M, N, K = 2, 3, 17
    rng = np.random.default_rng(13)
    a = f32(rng.standard_normal((M, K)))
    b = f32(rng.standard_normal((M, N, K)))
    _, c64, sc = oracle.bvecmat(a, b, F32, want64=True)
    for m in range(M):
        for n in range(N):
            exact = sum(Fraction(float(a[m, k])) * Fraction(float(b[m, n, k])) for k in range(K))
            scale = sum(abs(Fraction(float(a[m, k])) * Fraction(float(b[m, n, k]))) for k in range(K))
            assert abs(Fraction(float(c64[m, n])) - exact) <= K * Fraction(1, 2 ** 53) * scale
            assert abs(Fraction(float(sc[m, n])) - scale) <= K * Fraction(1, 2 ** 53) * scale


def test_linearity_and_batch_independence():
    M, N, K = 3, 4, 64
    rng = np.random.default_rng(14)
    a = f32(rng.standard_normal((M, K)))
    b1 = f32(rng.integers(-8, 8, (M, N, K)))
    b2 = f32(rng.integers(-8, 8, (M, N, K)))
    _, c1, _ = oracle.bvecmat(a, b1, F32, want64=True)
    _, c2, _ = oracle.bvecmat(a, b2, F32, want64=True)
    _, c12, sc = oracle.bvecmat(a, f32(b1.astype(np.float64) + b2), F32, want64=True)
    assert (np.abs(c12 - (c1 + c2)) <= 4 * K * 2.0 ** -53 * (sc + 1)).all()
    _, c4, _ = oracle.bvecmat(f32(4.0 * a.astype(np.float64)), b1, F32, want64=True)
    np.testing.assert_array_equal(c4, 4.0 * c1)                                      # scaling by 4 is exact
    # changing batch entry 1 leaves entries 0 and 2 bit-identical
    a2, b3 = a.copy(), b1.copy()
    a2[1] += 1.0
    b3[1] *= 2.0
    _, c3, _ = oracle.bvecmat(a2, b3, F32, want64=True)
    np.testing.assert_array_equal(c3[[0, 2]], c1[[0, 2]])
    assert (c3[1] != c1[1]).any()


@pytest.mark.parametrize("dt", [F32, BF16])
def test_against_numpy_einsum_float64(dt):
    M, N, K = 5, 33, 257
    rng = np.random.default_rng(15 + dt)
    enc = f32 if dt == F32 else bf
    a, b = enc(rng.standard_normal((M, K))), enc(rng.standard_normal((M, N, K)) * 3.0)
    wide = (lambda v: v.astype(np.float64)) if dt == F32 else oracle.bf16_to_double
    c, c64, sc = oracle.bvecmat(a, b, dt, want64=True, nthreads=3)
    ref = np.einsum("mk,mnk->mn", wide(a), wide(b))
    assert (np.abs(c64 - ref) <= 2 * K * 2.0 ** -53 * sc).all()
    np.testing.assert_allclose(sc, np.einsum("mk,mnk->mn", np.abs(wide(a)), np.abs(wide(b))), rtol=1e-13)
    # threads only spread rows: bit-identical to the single-thread run
    c1, c641, _ = oracle.bvecmat(a, b, dt, want64=True, nthreads=1)
    np.testing.assert_array_equal(c64, c641)
    np.testing.assert_array_equal(c, c1)
    # stored result is the single rounding of the double
    if dt == F32:
        np.testing.assert_array_equal(c, c64.astype(np.float32))
    else:
        np.testing.assert_array_equal(c, oracle.bf16_from_double(c64))


def test_empty_and_bad_arguments():
    c = oracle.bvecmat(f32(np.zeros((0, 8))), f32(np.zeros((0, 4, 8))), F32)
    assert c.shape == (0, 4)
    c = oracle.bvecmat(f32(np.zeros((2, 8))), f32(np.zeros((2, 0, 8))), F32)
    assert c.shape == (2, 0)
    with pytest.raises(ValueError):
        oracle.bvecmat(f32(np.zeros((2, 8))), f32(np.zeros((3, 4, 8))), F32)
    with pytest.raises(ValueError):
        oracle.bvecmat(f32(np.zeros((2, 8))), f32(np.zeros((2, 4, 7))), F32)
    with pytest.raises(TypeError):
        oracle.bvecmat(np.zeros((2, 8)), f32(np.zeros((2, 4, 8))), F32)
