"""Pins that hold the CPU oracle to something other than itself: closed forms, hand rows, invariants,
brute force in extended precision, torch-CPU float64 library routines, and an exhaustive bf16 codec walk.
CPU only."""
from __future__ import annotations

import math
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F32

GOLDEN = Path(__file__).resolve().parent / "golden" / "closed_forms.txt"
ONES = lambda n: np.ones(n, np.float32)
ZEROS = lambda n: np.zeros(n, np.float32)


def f32(a):
    return np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))


def bf(a):
    """float64 -> bf16 patterns through torch (an independent codec), exact for values already on the grid."""
    t = torch.from_numpy(np.asarray(a, np.float64).astype(np.float32)).to(torch.bfloat16)
    return np.ascontiguousarray(t.view(torch.uint16).numpy())


# ------------------------------------------------------------------ golden closed forms (hand-derived)

def _golden_cases():
    out = []
    for line in GOLDEN.read_text().splitlines():
        line = line.split("#")[0].strip()
        if not line:
            continue
        op, eps, x, y, st = [s.strip() for s in line.split("|")]
        out.append((op, float(eps), [float(v) for v in x.split()], [float(v) for v in y.split()],
                    [float(v) for v in st.split()]))
    return out


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: f"{c[0]}-{len(c[2])}")
def test_golden_closed_forms(case):
    op, eps, x, y, st = case
    xr = f32(x)[None, :]
    n = xr.shape[1]
    if op == "softmax":
        got, got64 = oracle.softmax(xr, F32, want64=True)
        stats = []
    elif op == "layernorm":
        got, mean, rstd, got64, s64 = oracle.layernorm(xr, ONES(n), ZEROS(n), eps, F32, want64=True)
        stats = [s64[0, 0], s64[0, 1]]
        assert mean[0] == np.float32(s64[0, 0]) and rstd[0] == np.float32(s64[0, 1])
    else:
        got, rstd, got64, s64 = oracle.rmsnorm(xr, ONES(n), eps, F32, want64=True)
        stats = [s64[0]]
        assert rstd[0] == np.float32(s64[0])
    # inputs are fp32 roundings of the listed decimals, hence 1e-6 rather than 1e-15
    np.testing.assert_allclose(got64[0], y, rtol=1e-6, atol=1e-300)
    np.testing.assert_allclose(stats, st, rtol=1e-6)
    np.testing.assert_array_equal(got[0], got64[0].astype(np.float32))
    # exact zeros are +0
    z = np.asarray(y) == 0.0
    if op == "softmax":
        assert not np.signbit(got[0][z]).any() and (got[0][z] == 0).all()


# ------------------------------------------------------------------ softmax

def test_softmax_two_element_closed_form():
    rng = np.random.default_rng(1)
    for _ in range(200):
        a, b = f32(rng.normal(0, 20, 2))
        _, y64 = oracle.softmax(np.array([[a, b]], np.float32), F32, want64=True)
        d = float(b) - float(a)
        assert abs(d) < 700
        assert y64[0, 0] == pytest.approx(1.0 / (1.0 + math.exp(d)), rel=1e-14)
        assert y64[0, 1] == pytest.approx(1.0 / (1.0 + math.exp(-d)), rel=1e-14)


def test_softmax_row_sum_shift_monotone():
    rng = np.random.default_rng(2)
    x = f32(rng.normal(0, 3, (37, 1000)))
    y, y64 = oracle.softmax(x, F32, want64=True)
    np.testing.assert_allclose(y64.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    # shift by an exactly representable constant that keeps x + c exact: multiples of 2^-10, c = 8
    xq = f32(np.round(x * 1024) / 1024)
    _, a = oracle.softmax(xq, F32, want64=True)
    _, b = oracle.softmax(f32(xq.astype(np.float64) + 8.0), F32, want64=True)
    assert (xq.astype(np.float64) + 8.0 == f32(xq.astype(np.float64) + 8.0).astype(np.float64)).all()
    np.testing.assert_array_equal(a, b)
    # monotone: ordering of outputs follows ordering of inputs
    order = np.argsort(x[0], kind="stable")
    assert (np.diff(y64[0][order]) >= 0).all()
    assert (y64 > 0).all() and (y64 <= 1).all()


def test_softmax_masked_and_fully_masked():
    x = f32([[0.0, -np.inf, 1.0, -np.inf], [-np.inf] * 4, [3.0, 3.0, -np.inf, 3.0]])
    y, y64 = oracle.softmax(x, F32, want64=True)
    assert y.view(np.uint32)[0, 1] == 0 and y.view(np.uint32)[0, 3] == 0
    assert (y.view(np.uint32)[1] == 0).all()
    np.testing.assert_allclose(y64[2], [1 / 3, 1 / 3, 0, 1 / 3], rtol=1e-15)
    e = math.e
    np.testing.assert_allclose(y64[0], [1 / (1 + e), 0, e / (1 + e), 0], rtol=1e-15)
    xb = bf([[0.0, -np.inf, 1.0, -np.inf], [-np.inf] * 4])
    yb = oracle.softmax(xb, BF16)
    assert yb[0, 1] == 0 and yb[0, 3] == 0 and (yb[1] == 0).all()


def test_softmax_no_overflow_and_extreme_range():
    x = f32([[1e30, 1e30], [-1e30, 0.0], [88.0, -88.0]])
    _, y64 = oracle.softmax(x, F32, want64=True)
    np.testing.assert_array_equal(y64[0], [0.5, 0.5])
    np.testing.assert_array_equal(y64[1], [0.0, 1.0])
    assert y64[2, 1] == pytest.approx(math.exp(-176.0), rel=1e-13)


def test_softmax_subnormal_bf16_outputs_kept():
    # y = exp(-90)/(1+tiny) ~ 8.2e-40 lies below 2^-126 ~ 1.18e-38: must come out as a bf16 subnormal, not 0
    xb = bf([[0.0, -90.0, -95.0]])
    yb, y64 = oracle.softmax(xb, BF16, want64=True)
    assert 0 < yb[0, 1] < 0x0080
    q = 2.0 ** -133
    assert yb[0, 1] == round(y64[0, 1] / q)
    assert yb[0, 2] == round(y64[0, 2] / q)


# ------------------------------------------------------------------ LayerNorm

def test_layernorm_eps_closed_form_invariants():
    rng = np.random.default_rng(3)
    x = f32(rng.normal(0.5, 3.0, (29, 777)))
    n = x.shape[1]
    for eps in (0.0, 1e-5, 0.5):
        _, _, _, y64, st = oracle.layernorm(x, ONES(n), ZEROS(n), eps, F32, want64=True)
        var = x.astype(np.float64).var(axis=1)      # numpy's population variance: an independent routine
        np.testing.assert_allclose(y64.mean(axis=1), 0.0, atol=1e-13)
        e = float(np.float32(eps))
        np.testing.assert_allclose(y64.var(axis=1), var / (var + e), rtol=1e-12)
        np.testing.assert_allclose(st[:, 0], x.astype(np.float64).mean(axis=1), rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(st[:, 1], 1.0 / np.sqrt(var + e), rtol=1e-13)


def test_layernorm_affine_linearity_and_constant_row():
    rng = np.random.default_rng(4)
    x = f32(rng.normal(0, 1, (11, 64)))
    g, b = f32(rng.uniform(0.5, 1.5, 64)), f32(rng.normal(0, 0.1, 64))
    _, _, _, y_plain, _ = oracle.layernorm(x, ONES(64), ZEROS(64), 1e-5, F32, want64=True)
    _, _, _, y_aff, _ = oracle.layernorm(x, g, b, 1e-5, F32, want64=True)
    np.testing.assert_allclose(y_aff, y_plain * g.astype(np.float64) + b.astype(np.float64), rtol=1e-14, atol=1e-16)
    xc = np.full((2, 64), 3.25, np.float32)
    y, mean, rstd, y64, st = oracle.layernorm(xc, g, b, 1e-5, F32, want64=True)
    np.testing.assert_array_equal(y, np.broadcast_to(b, (2, 64)))
    assert mean[0] == np.float32(3.25)
    assert st[0, 1] == pytest.approx(1.0 / math.sqrt(float(np.float32(1e-5))), rel=1e-15)
    # cols = 1: variance 0, output = beta
    y1, m1, r1 = oracle.layernorm(f32([[5.0]]), f32([2.0]), f32([0.75]), 1e-5, F32)
    assert y1[0, 0] == np.float32(0.75) and m1[0] == 5.0


def test_layernorm_eps_is_the_fp32_value():
    # 1e-5f != 1e-5: a constant row makes rstd = 1/sqrt(eps), which tells the two apart at 1e-9
    _, _, _, _, st = oracle.layernorm(np.zeros((1, 8), np.float32), ONES(8), ZEROS(8), 1e-5, F32, want64=True)
    e32 = float(np.float32(1e-5))
    assert st[0, 1] == pytest.approx(1 / math.sqrt(e32), rel=1e-15)
    assert abs(st[0, 1] - 1 / math.sqrt(1e-5)) / st[0, 1] > 1e-9


# ------------------------------------------------------------------ RMSNorm

def test_rmsnorm_closed_form_and_scale_equivariance():
    rng = np.random.default_rng(5)
    x = f32(rng.normal(0, 1, (13, 515)))
    n = x.shape[1]
    w = f32(rng.normal(1.0, 0.1, n))
    for eps in (0.0, 1e-6, 2.0):
        _, _, y64, rr = oracle.rmsnorm(x, ONES(n), eps, F32, want64=True)
        ms = (x.astype(np.float64) ** 2).mean(axis=1)
        e = float(np.float32(eps))
        np.testing.assert_allclose(np.sqrt((y64 ** 2).mean(axis=1)), np.sqrt(ms / (ms + e)), rtol=1e-13)
        np.testing.assert_allclose(rr, 1 / np.sqrt(ms + e), rtol=1e-13)
    _, _, a, _ = oracle.rmsnorm(x, w, 0.0, F32, want64=True)
    _, _, b, _ = oracle.rmsnorm(f32(x.astype(np.float64) * 4.0), w, 0.0, F32, want64=True)   # c = 2^2: exact scaling
    np.testing.assert_allclose(a, b, rtol=1e-15)
    _, _, ones_out, _ = oracle.rmsnorm(np.ones((1, n), np.float32), w, 0.0, F32, want64=True)
    np.testing.assert_array_equal(ones_out[0], w.astype(np.float64))
    # sign is kept, no mean is subtracted
    _, _, s, _ = oracle.rmsnorm(f32([[2.0, 2.0, 2.0]]), ONES(3), 0.0, F32, want64=True)
    np.testing.assert_array_equal(s[0], [1.0, 1.0, 1.0])


# ------------------------------------------------------------------ element-wise sine (calibration kernel)

def test_sin_closed_forms_symmetry_and_library():
    x = f32([0.0, -0.0, 0.5, 1.0, 2.0, 3.0, 10.0, 100.0, 1e6, -7.25])
    y, y64 = oracle.sin(x, F32, want64=True)
    assert y[0] == 0.0 and not np.signbit(y[0]) and np.signbit(y[1])             # sin(+-0) = +-0
    # closed forms at exactly representable arguments of the half-angle chain: sin(2a) = 2 sin a cos a, sin^2 + cos^2 = 1
    a = x.astype(np.float64)
    s_half, c_half = np.sin(a / 2), np.cos(a / 2)
    np.testing.assert_allclose(y64, 2 * s_half * c_half, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(y64, [math.sin(float(v)) for v in x], rtol=1e-15)       # libm through Python, value by value
    _, neg = oracle.sin(f32(-a), F32, want64=True)
    np.testing.assert_array_equal(neg, -y64)                                        # odd
    assert (np.abs(y64) <= 1).all()
    # small-angle series: sin x = x - x^3/6 + x^5/120 - ... for |x| <= 2^-10 agrees to 1e-16 relative
    small = f32([2.0 ** -10, 2.0 ** -15, -2.0 ** -20])
    _, ys = oracle.sin(small, F32, want64=True)
    sd = small.astype(np.float64)
    np.testing.assert_allclose(ys, sd - sd ** 3 / 6 + sd ** 5 / 120, rtol=1e-15)
    yb, yb64 = oracle.sin(bf([0.5, 1.5]), BF16, want64=True)
    np.testing.assert_array_equal(yb, oracle.bf16_from_double(yb64))


# ------------------------------------------------------------------ brute force on tiny rows (long double)

def test_bruteforce_longdouble_tiny_rows():
    rng = np.random.default_rng(6)
    L = np.longdouble
    for n in (1, 2, 3, 5, 8):
        x = f32(rng.normal(0, 2, (4, n)))
        g, b = f32(rng.uniform(0.5, 1.5, n)), f32(rng.normal(0, 0.3, n))
        _, s64 = oracle.softmax(x, F32, want64=True)
        _, _, _, l64, lst = oracle.layernorm(x, g, b, 1e-5, F32, want64=True)
        _, _, r64, rst = oracle.rmsnorm(x, g, 1e-6, F32, want64=True)
        for r in range(4):
            xs = [L(float(v)) for v in x[r]]
            m = max(xs)
            es = [np.exp(v - m) for v in xs]
            tot = sum(es, L(0))
            for j in range(n):
                assert float(es[j] / tot) == pytest.approx(s64[r, j], rel=1e-14)
            mu = sum(xs, L(0)) / L(n)
            var = sum(((v - mu) ** 2 for v in xs), L(0)) / L(n)
            rs = L(1) / np.sqrt(var + L(float(np.float32(1e-5))))
            assert float(mu) == pytest.approx(lst[r, 0], rel=1e-14, abs=1e-16)
            assert float(rs) == pytest.approx(lst[r, 1], rel=1e-13)
            for j in range(n):
                want = float((xs[j] - mu) * rs * L(float(g[j])) + L(float(b[j])))
                assert want == pytest.approx(l64[r, j], rel=1e-12, abs=1e-14)
            rr = L(1) / np.sqrt(sum((v * v for v in xs), L(0)) / L(n) + L(float(np.float32(1e-6))))
            assert float(rr) == pytest.approx(rst[r], rel=1e-14)
            for j in range(n):
                assert float(xs[j] * rr * L(float(g[j]))) == pytest.approx(r64[r, j], rel=1e-14)


# ------------------------------------------------------------------ reduces to library routines (torch CPU float64)

@pytest.mark.parametrize("cols", [1, 2, 7, 64, 1000, 4097])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_matches_torch_float64(cols, dt):
    rng = np.random.default_rng(cols + dt)
    rows = 9
    raw = rng.normal(0.3, 2.5, (rows, cols))
    g_raw, b_raw = rng.uniform(0.5, 1.5, cols), rng.normal(0, 0.1, cols)
    conv = f32 if dt == F32 else bf
    x, g, b = conv(raw), conv(g_raw), conv(b_raw)
    wide = (lambda a: torch.from_numpy(a).double()) if dt == F32 else \
        (lambda a: torch.from_numpy(a).view(torch.bfloat16).double())
    xt, gt, bt = wide(x), wide(g), wide(b)
    _, y64 = oracle.softmax(x, dt, want64=True)
    np.testing.assert_allclose(y64, torch.softmax(xt, -1).numpy(), rtol=1e-12, atol=1e-300)
    eps = float(np.float32(1e-5))
    yl, mean, rstd, l64, st = oracle.layernorm(x, g, b, 1e-5, dt, want64=True)
    ref = torch.nn.functional.layer_norm(xt, (cols,), gt, bt, eps).numpy()
    np.testing.assert_allclose(l64, ref, rtol=1e-11, atol=1e-12)
    eps6 = float(np.float32(1e-6))
    yr, rr, r64, _ = oracle.rmsnorm(x, g, 1e-6, dt, want64=True)
    refr = (xt * torch.rsqrt((xt * xt).mean(-1, keepdim=True) + eps6) * gt).numpy()
    np.testing.assert_allclose(r64, refr, rtol=1e-12)
    # the stored outputs are the single rounding of the float64 results
    if dt == F32:
        np.testing.assert_array_equal(yl, l64.astype(np.float32))
        np.testing.assert_array_equal(yr, r64.astype(np.float32))
    else:
        np.testing.assert_array_equal(yl, oracle.bf16_from_double(l64))
        np.testing.assert_array_equal(yr, oracle.bf16_from_double(r64))


def test_threaded_driver_is_bit_identical():
    rng = np.random.default_rng(7)
    x = f32(rng.normal(0, 1, (101, 333)))
    g, b = f32(rng.uniform(0.5, 1.5, 333)), f32(rng.normal(0, 0.1, 333))
    np.testing.assert_array_equal(oracle.softmax(x, F32), oracle.softmax(x, F32, nthreads=5))
    for a, c in zip(oracle.layernorm(x, g, b, 1e-5, F32), oracle.layernorm(x, g, b, 1e-5, F32, nthreads=4)):
        np.testing.assert_array_equal(a, c)
    for a, c in zip(oracle.rmsnorm(x, g, 1e-6, F32), oracle.rmsnorm(x, g, 1e-6, F32, nthreads=200)):
        np.testing.assert_array_equal(a, c)


# ------------------------------------------------------------------ bf16 codec

def test_bf16_roundtrip_all_patterns():
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    v = oracle.bf16_to_double(h)
    with np.errstate(invalid="ignore"):
        ref = (h.astype(np.uint32) << 16).view(np.float32).astype(np.float64)     # bit-level definition
    np.testing.assert_array_equal(np.isnan(v), np.isnan(ref))
    ok = ~np.isnan(ref)
    np.testing.assert_array_equal(v[ok], ref[ok])
    back = oracle.bf16_from_double(v)
    np.testing.assert_array_equal(back[ok], h[ok])
    assert ((back[~ok] & 0x7F80) == 0x7F80).all() and ((back[~ok] & 0x007F) != 0).all()


def test_bf16_midpoints_go_to_even_and_neighbours():
    # all adjacent pairs of finite non-negative bf16 values, including subnormals and the step into infinity
    h = np.arange(0, 0x7F80, dtype=np.uint16)
    lo = oracle.bf16_to_double(h)
    hi = np.where(h + 1 == 0x7F80, 2.0 ** 128, oracle.bf16_to_double((h + 1).astype(np.uint16)))
    mid = 0.5 * (lo + hi)                       # exact in double
    even = np.where(h & 1, h + 1, h).astype(np.uint16)
    np.testing.assert_array_equal(oracle.bf16_from_double(mid), even)
    np.testing.assert_array_equal(oracle.bf16_from_double(-mid), even | 0x8000)
    above, below = np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf)
    np.testing.assert_array_equal(oracle.bf16_from_double(above), (h + 1).astype(np.uint16))
    np.testing.assert_array_equal(oracle.bf16_from_double(below), h)
    # the overflow threshold (2 - 2^-8) * 2^127 is the midpoint between max finite and 2^128: ties to "even" = inf
    thr = (2.0 - 2.0 ** -8) * 2.0 ** 127
    got = oracle.bf16_from_double(np.array([thr, np.nextafter(thr, 0), 1e300, -1e300, 2.0 ** -134, 2.0 ** -134 * 1.0001,
                                            2.0 ** -140, -0.0, 0.0]))
    assert list(got) == [0x7F80, 0x7F7F, 0x7F80, 0xFF80, 0x0000, 0x0001, 0x0000, 0x8000, 0x0000]


def test_bf16_matches_torch_on_random_fp32_patterns():
    rng = np.random.default_rng(8)
    bits = rng.integers(0, 2 ** 32, 5_000_000, dtype=np.uint64).astype(np.uint32)
    f = bits.view(np.float32)
    f = f[np.isfinite(f)]
    ours = oracle.bf16_from_double(f.astype(np.float64))
    theirs = torch.from_numpy(f).to(torch.bfloat16).view(torch.uint16).numpy()
    np.testing.assert_array_equal(ours, theirs)


def test_bf16_rounds_directly_from_double():
    # 1 + 2^-8 + 2^-30 lies just above the midpoint of [1, 1 + 2^-7]; via float it would first fall ON the
    # midpoint (2^-30 is below fp32 resolution at 1) and then tie to even = 1.0.  Direct rounding goes up.
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert oracle.bf16_from_double(np.array([v]))[0] == 0x3F81
    assert np.float32(v) == np.float32(1.0 + 2.0 ** -8)


# ------------------------------------------------------------------ residual add of the fused add-and-normalise

def test_add_exact_cases_ties_and_library():
    x = f32([1.0, 2.5, -3.0, 1e30, 0.0, -0.0, 16777216.0, 1.0])
    r = f32([2.0, 0.25, 3.0, 1e30, 0.0, -0.0, 1.0, 2.0 ** -30])
    h, h64 = oracle.add(x, r, F32, want64=True)
    np.testing.assert_array_equal(h64[:4], [3.0, 2.75, 0.0, 2.0 * float(np.float32(1e30))])
    assert not np.signbit(h[2])                                  # x + (-x) = +0 in round-to-nearest
    assert np.signbit(h[5]) and not np.signbit(h[4])             # (-0) + (-0) = -0, (+0) + (+0) = +0
    assert h[6] == np.float32(16777216.0)                        # 2^24 + 1 is a tie in fp32: goes to the even 2^24
    assert h[7] == np.float32(1.0)
    np.testing.assert_array_equal(oracle.add(r, x, F32), h)      # commutative
    np.testing.assert_array_equal(oracle.add(x, ZEROS(8), F32)[[0, 1, 2, 3, 6, 7]], x[[0, 1, 2, 3, 6, 7]])
    # bf16: ties to even at 1 + 2^-8 (down to 1) and 1 + 2^-7 + 2^-8 (up to 1 + 2^-6); a sum that needs more than 8 bits
    xb = bf([1.0, 1.0 + 2.0 ** -7, 256.0, 3.0])
    rb = bf([2.0 ** -8, 2.0 ** -8, 1.0, -3.0])
    hb, hb64 = oracle.add(xb, rb, BF16, want64=True)
    np.testing.assert_array_equal(hb64, [1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7 + 2.0 ** -8, 257.0, 0.0])
    np.testing.assert_array_equal(oracle.bf16_to_double(hb), [1.0, 1.0 + 2.0 ** -6, 256.0, 0.0])
    # against torch's CPU add on random finite inputs, both types (an independent library route), and the bf16 codec
    rng = np.random.default_rng(21)
    a = rng.standard_normal(200_000) * np.exp(rng.uniform(-20, 20, 200_000))
    b = rng.standard_normal(200_000) * np.exp(rng.uniform(-20, 20, 200_000))
    np.testing.assert_array_equal(oracle.add(f32(a), f32(b), F32), (torch.from_numpy(f32(a)) + torch.from_numpy(f32(b))).numpy())
    ab, bb = bf(a), bf(b)
    tb = (torch.from_numpy(ab).view(torch.bfloat16) + torch.from_numpy(bb).view(torch.bfloat16)).view(torch.uint16).numpy()
    got, got64 = oracle.add(ab, bb, BF16, want64=True)
    np.testing.assert_array_equal(got, tb)
    np.testing.assert_array_equal(got, oracle.bf16_from_double(oracle.bf16_to_double(ab) + oracle.bf16_to_double(bb)))
    np.testing.assert_array_equal(got64, oracle.bf16_to_double(ab) + oracle.bf16_to_double(bb))


def test_add_then_norm_is_the_composition():
    rng = np.random.default_rng(22)
    for dt, enc in ((F32, f32), (BF16, bf)):
        x, r = enc(rng.standard_normal((5, 96)) * 3), enc(rng.standard_normal((5, 96)))
        g, b = enc(rng.uniform(0.5, 1.5, 96)), enc(rng.standard_normal(96) * 0.1)
        h, y, mean, rstd = oracle.add_layernorm(x, r, g, b, 1e-5, dt)
        np.testing.assert_array_equal(h, oracle.add(x, r, dt))
        y2, mean2, rstd2 = oracle.layernorm(h, g, b, 1e-5, dt)
        np.testing.assert_array_equal(y, y2), np.testing.assert_array_equal(mean, mean2), np.testing.assert_array_equal(rstd, rstd2)
        h, y, rs = oracle.add_rmsnorm(x, r, g, 1e-6, dt)
        y2, rs2 = oracle.rmsnorm(oracle.add(x, r, dt), g, 1e-6, dt)
        np.testing.assert_array_equal(y, y2), np.testing.assert_array_equal(rs, rs2)
        # the statistics come from the ROUNDED h: feeding the unrounded sum would change mean in the last bits for bf16
        if dt == BF16:
            exact = oracle.bf16_to_double(x) + oracle.bf16_to_double(r)
            assert np.abs(mean.astype(np.float64) - oracle.bf16_to_double(h).mean(axis=1)).max() < 1e-6
            assert np.abs(oracle.bf16_to_double(h) - exact).max() > 0          # rounding did happen


# ------------------------------------------------------------------ softmax with per-row valid lengths

@pytest.mark.parametrize("dt", [F32, BF16])
def test_softmax_len_equals_masked_softmax_and_never_reads_the_tail(dt):
    rng = np.random.default_rng(31 + dt)
    rows, cols = 23, 77
    enc = f32 if dt == F32 else bf
    xv = rng.standard_normal((rows, cols)) * 4
    lens = rng.integers(0, cols + 1, rows).astype(np.int32)
    lens[:4] = [0, 1, cols, cols - 1]
    x = enc(xv)
    y, y64 = oracle.softmax_len(x, lens, dt, want64=True)
    # (1) the plain softmax on a copy whose tails hold -inf: bit for bit
    masked = xv.copy()
    for r in range(rows):
        masked[r, lens[r]:] = -np.inf
    ym, ym64 = oracle.softmax(enc(masked), dt, want64=True)
    np.testing.assert_array_equal(y, ym)
    np.testing.assert_array_equal(y64, ym64)
    # (2) the tail of the input is never read: NaN and +inf there leave no trace
    poisoned = xv.copy()
    for r in range(rows):
        poisoned[r, lens[r]:] = np.nan if r % 2 else np.inf
    yp = oracle.softmax_len(enc(poisoned), lens, dt)
    np.testing.assert_array_equal(yp, y)
    # (3) special lengths: 0 -> all +0 bits; 1 -> a single 1; cols -> the plain softmax; sums are 1 over the live part
    bits = y.view(np.uint32) if dt == F32 else y
    assert not bits[0].any()
    one = np.float32(1.0).view(np.uint32) if dt == F32 else 0x3F80
    assert bits[1, 0] == one and not bits[1, 1:].any()
    np.testing.assert_array_equal(y[2], oracle.softmax(x[2:3], dt)[0])
    for r in range(rows):
        assert not bits[r, lens[r]:].any()
        if lens[r]:
            assert abs(y64[r, :lens[r]].sum() - 1.0) < 1e-12
    # (4) lengths outside [0, cols] are clamped; threads only spread rows
    wild = lens.copy()
    wild[5], wild[6] = -7, cols + 100
    ref = lens.copy()
    ref[5], ref[6] = 0, cols
    np.testing.assert_array_equal(oracle.softmax_len(x, wild, dt), oracle.softmax_len(x, ref, dt))
    np.testing.assert_array_equal(oracle.softmax_len(x, lens, dt, nthreads=4), y)
