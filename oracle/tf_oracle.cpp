// CPU oracle for the row-wise reduce-then-normalise forward ops (softmax, LayerNorm, RMSNorm).
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test suite, the smoke check and the
// benchmark's CPU-baseline leg may call it.  It shares no code, header, table or helper with the
// CUDA library and includes no CUDA header.
//
// Form: plain C++17, no SIMD intrinsics, one thread per call (the *_mt drivers only spread whole
// rows over std::thread workers around the very same per-row functions, so their results are
// bit-identical to the single-thread run).  Inputs are widened exactly to double, every operation
// is done in double in the order the textbook definition states, and the result is rounded ONCE,
// round-to-nearest-even, to the output type (subnormals kept, never flushed).
//
// The paper (TritonForge) names this kernel class only in passing (Section 2, the list of
// hand-optimised Triton kernels: fused operators, attention, softmax variants) and defines none of
// the three ops, so each function below is the standard definition written out; the readings of
// every open point (fully masked rows, variance divisor, where eps goes, one final rounding) are
// stated beside the code that takes them.
//
// Pins (tests that hold this file to something other than itself): closed forms and hand rows,
// row-sum / shift / scale invariants, the eps closed forms for variance and RMS, brute force in
// long double on tiny rows, agreement with torch-CPU float64 library routines before rounding, and
// for the bf16 codec an exhaustive walk over all 65,536 patterns and every midpoint.  The element-wise
// sine (the kernel of the paper's Case Study 1, used as a calibration workload) is std::sin in double;
// it is pinned by sin(+-0), oddness, the double-angle identity, the small-angle series and libm
// through another route.  The batched vector-matrix product (the paper's Case Study 2) is the plain
// triple loop in double; it is pinned by all-ones and ramp closed forms, unit-vector selection, an
// index-order trap (B[m,n,k] versus B[m,k,n] and A[m,k] versus A[n,k]), exact integer brute force,
// linearity, and numpy's float64 einsum.  The residual add that precedes a fused add-and-normalise
// (h = x + r, rounded once to the storage type; the norm is then the ordinary one applied to h) is
// pinned by exact small sums, x + 0, x - x, commutativity, bf16 ties to even, and torch's CPU add.
// Softmax with per-row valid lengths (row r is normalised over its first len[r] entries, the rest of the
// output row is +0, the rest of the input row is never read) is pinned by equality with the plain softmax on
// a copy whose tails hold -inf, by len = cols, len = 0, len = 1, and by NaN-filled tails leaving no trace.
// Log-softmax (y = (x - m) - ln sum exp(x - m)) is pinned by the logarithm of the pinned softmax, by
// sum exp(y) = 1, exact shift invariance, the two-element closed form -log1p(e^(b-a)), uniform rows (-ln n),
// masked entries (-inf) and torch's float64 routine.  The softmax backward pass (dx = y (dy - sum y dy)) is
// pinned by the analytic Jacobian on one-hot dy, by central differences of the pinned softmax in double,
// by dx = 0 for constant dy, by linearity in dy and by torch's float64 autograd.
// The backward passes of LayerNorm and RMSNorm (dx per row from the stored statistics, parameter gradients
// as column sums over the rows) are pinned by central differences of the pinned forward passes in double, by
// the orthogonality invariants of dx (it sums to zero and is orthogonal to the normalised row for LayerNorm,
// orthogonal to x for RMSNorm with unit weight), by plain column sums for dbeta, and by torch's float64 autograd.
// tf_tune has
// no oracle function here: which candidate wins is hardware-dependent ("parity unpinned" for the
// winner's identity; its output is checked like any other launch).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

enum Dtype : int { F32 = 0, BF16 = 1 };

// ---------------------------------------------------------------------------------------------
// bf16 codec.  bf16 = 1 sign, 8 exponent (bias 127), 7 mantissa bits: the top half of an fp32.
// ---------------------------------------------------------------------------------------------

// Exact widening: place the 16 bits in the top half of an fp32 pattern, then float -> double.
double bf16_to_double(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// Round a double straight to bf16 (never through float, which would round twice).
// Nearest, ties to even; values below 2^-126 land on the subnormal grid of spacing 2^-133;
// anything that rounds to 2^128 or above becomes infinity; NaN becomes a quiet NaN.
uint16_t bf16_from_double(double v) {
    if (std::isnan(v)) return 0x7FC0;
    const uint16_t sign = std::signbit(v) ? 0x8000 : 0x0000;
    const double a = std::fabs(v);
    if (a == 0.0) return sign;
    if (std::isinf(a)) return sign | 0x7F80;
    int e2;
    std::frexp(a, &e2);            // a = f * 2^e2 with f in [0.5, 1)  =>  a in [2^(e2-1), 2^e2)
    int E = e2 - 1;                // binade of a
    if (E < -126) E = -126;        // subnormals share the grid of the lowest normal binade
    if (E > 127) return sign | 0x7F80;
    // In binade E the representable values are r * 2^(E-7), r = 128..255 (r < 128: subnormal).
    const double q = std::ldexp(a, -(E - 7));      // exact: scaling by a power of two
    const double r = std::nearbyint(q);            // default rounding mode: nearest, ties to even
    // bits = (E+127)<<7 | (r-128); written as ((E+126)<<7) + r it also carries r = 256 into the
    // next binade and covers the subnormal case E = -126 (bits = r).
    const uint32_t bits = (static_cast<uint32_t>(E + 126) << 7) + static_cast<uint32_t>(r);
    if (bits >= 0x7F80u) return sign | 0x7F80;
    return sign | static_cast<uint16_t>(bits);
}

float f32_from_double(double v) { return static_cast<float>(v); }   // RNE, subnormals kept

inline double load(const void* p, int64_t i, int dt) {
    if (dt == F32) return static_cast<double>(static_cast<const float*>(p)[i]);
    return bf16_to_double(static_cast<const uint16_t*>(p)[i]);
}

inline void store(void* p, int64_t i, int dt, double v) {
    if (dt == F32) static_cast<float*>(p)[i] = f32_from_double(v);
    else           static_cast<uint16_t*>(p)[i] = bf16_from_double(v);
}

// ---------------------------------------------------------------------------------------------
// Per-row definitions.  x points at the row's first element; y likewise; y64 (nullable) receives
// the unrounded double result for tests that check invariants below the output type's resolution.
// ---------------------------------------------------------------------------------------------

// softmax over the last axis, no temperature:  y_j = exp(x_j - m) / sum_k exp(x_k - m), m = max x.
// Reading for a fully masked row (every x_j = -inf, where the plain formula gives NaN): all +0.
// exp(-inf) is exactly 0, so masked entries of a live row come out as +0.
void softmax_row(const void* x, void* y, double* y64, int64_t n, int dt, int64_t base) {
    double m = -std::numeric_limits<double>::infinity();
    for (int64_t j = 0; j < n; ++j) {
        const double v = load(x, base + j, dt);
        if (v > m || std::isnan(v)) m = v;       // a NaN poisons the row (outside the parity contract)
    }
    if (m == -std::numeric_limits<double>::infinity()) {
        for (int64_t j = 0; j < n; ++j) {
            if (y64) y64[base + j] = 0.0;
            if (y) store(y, base + j, dt, 0.0);
        }
        return;
    }
    double S = 0.0;
    for (int64_t j = 0; j < n; ++j) S += std::exp(load(x, base + j, dt) - m);
    for (int64_t j = 0; j < n; ++j) {
        const double v = std::exp(load(x, base + j, dt) - m) / S;
        if (y64) y64[base + j] = v;
        if (y) store(y, base + j, dt, v);
    }
}

// LayerNorm:  mu = mean(x);  var = mean((x - mu)^2)  (two passes, divisor n: the population
// variance, which is what makes "variance 1" hold for the output);  rstd = 1/sqrt(var + eps),
// eps being the caller's fp32 value widened to double and added inside the root;
// y_j = (x_j - mu) * rstd * gamma_j + beta_j.  mean/rstd outputs are fp32 roundings of mu/rstd;
// y is computed from the unrounded ones.
void layernorm_row(const void* x, const void* gamma, const void* beta, void* y, double* y64,
                   float* mean, float* rstd, double* stats64, int64_t n, double eps, int dt,
                   int64_t row) {
    const int64_t base = row * n;
    double s = 0.0;
    for (int64_t j = 0; j < n; ++j) s += load(x, base + j, dt);
    const double mu = s / static_cast<double>(n);
    double m2 = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const double d = load(x, base + j, dt) - mu;
        m2 += d * d;
    }
    const double var = m2 / static_cast<double>(n);
    const double rs = 1.0 / std::sqrt(var + eps);
    if (mean) mean[row] = f32_from_double(mu);
    if (rstd) rstd[row] = f32_from_double(rs);
    if (stats64) { stats64[2 * row] = mu; stats64[2 * row + 1] = rs; }
    for (int64_t j = 0; j < n; ++j) {
        const double v = (load(x, base + j, dt) - mu) * rs * load(gamma, j, dt) + load(beta, j, dt);
        if (y64) y64[base + j] = v;
        if (y) store(y, base + j, dt, v);
    }
}

// RMSNorm:  ms = mean(x^2);  rrms = 1/sqrt(ms + eps);  y_j = x_j * rrms * w_j, rounded once
// (not the flavour that rounds x*rrms to the storage type before the weight, and not (1 + w)).
void rmsnorm_row(const void* x, const void* w, void* y, double* y64, float* rstd, double* stats64,
                 int64_t n, double eps, int dt, int64_t row) {
    const int64_t base = row * n;
    double ss = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const double v = load(x, base + j, dt);
        ss += v * v;
    }
    const double rr = 1.0 / std::sqrt(ss / static_cast<double>(n) + eps);
    if (rstd) rstd[row] = f32_from_double(rr);
    if (stats64) stats64[row] = rr;
    for (int64_t j = 0; j < n; ++j) {
        const double v = load(x, base + j, dt) * rr * load(w, j, dt);
        if (y64) y64[base + j] = v;
        if (y) store(y, base + j, dt, v);
    }
}

// Spread rows [0, rows) over nthreads workers in contiguous blocks; fn(row) does one row.
template <class Fn>
void for_rows(int64_t rows, int nthreads, Fn fn) {
    if (nthreads <= 1 || rows < 2) {
        for (int64_t r = 0; r < rows; ++r) fn(r);
        return;
    }
    if (nthreads > rows) nthreads = static_cast<int>(rows);
    std::vector<std::thread> pool;
    pool.reserve(nthreads);
    for (int t = 0; t < nthreads; ++t) {
        const int64_t lo = rows * t / nthreads, hi = rows * (t + 1) / nthreads;
        pool.emplace_back([=] { for (int64_t r = lo; r < hi; ++r) fn(r); });
    }
    for (auto& th : pool) th.join();
}

bool bad(int64_t rows, int64_t cols, int dt) { return rows < 0 || cols <= 0 || (dt != F32 && dt != BF16); }

}  // namespace

extern "C" {

// All pointers are host memory, row-major [rows, cols], element type per dt (0 = fp32, 1 = bf16 as
// uint16 bit patterns).  y, y64, mean, rstd, stats64 are nullable outputs.  Returns 0, or -1 on a
// bad argument.  nthreads <= 1 runs on the calling thread.

int oracle_softmax(const void* x, void* y, double* y64, int64_t rows, int64_t cols, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x) return -1;
    for_rows(rows, nthreads, [=](int64_t r) { softmax_row(x, y, y64, cols, dt, r * cols); });
    return 0;
}

int oracle_layernorm(const void* x, const void* gamma, const void* beta, void* y, double* y64,
                     float* mean, float* rstd, double* stats64, int64_t rows, int64_t cols,
                     float eps, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x || !gamma || !beta) return -1;
    const double e = static_cast<double>(eps);
    for_rows(rows, nthreads, [=](int64_t r) {
        layernorm_row(x, gamma, beta, y, y64, mean, rstd, stats64, cols, e, dt, r);
    });
    return 0;
}

int oracle_rmsnorm(const void* x, const void* w, void* y, double* y64, float* rstd, double* stats64,
                   int64_t rows, int64_t cols, float eps, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x || !w) return -1;
    const double e = static_cast<double>(eps);
    for_rows(rows, nthreads, [=](int64_t r) { rmsnorm_row(x, w, y, y64, rstd, stats64, cols, e, dt, r); });
    return 0;
}

// Softmax over the first len[r] entries of row r (0 <= len[r] <= cols, values outside are clamped): the
// definition above applied to x[r, 0:len[r]]; y[r, j] = +0 for j >= len[r]; x[r, j >= len[r]] is not read.
// len[r] = 0 gives an all +0 row (the fully masked reading above).
int oracle_softmax_len(const void* x, const int32_t* len, void* y, double* y64, int64_t rows, int64_t cols, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x || !len) return -1;
    for_rows(rows, nthreads, [=](int64_t r) {
        const int64_t n = len[r] < 0 ? 0 : (len[r] > cols ? cols : len[r]);
        if (n > 0) softmax_row(x, y, y64, n, dt, r * cols);
        for (int64_t j = n; j < cols; ++j) {
            if (y64) y64[r * cols + j] = 0.0;
            if (y) store(y, r * cols + j, dt, 0.0);
        }
    });
    return 0;
}

// Log-softmax over the last axis:  y_j = (x_j - m) - ln sum_k exp(x_k - m), m = max x.  Entries with x_j = -inf
// give y_j = -inf; a fully masked row gives -inf everywhere (the logarithm of the all-zero reading of softmax).
int oracle_log_softmax(const void* x, void* y, double* y64, int64_t rows, int64_t cols, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x) return -1;
    for_rows(rows, nthreads, [=](int64_t r) {
        const int64_t base = r * cols;
        double m = -std::numeric_limits<double>::infinity();
        for (int64_t j = 0; j < cols; ++j) {
            const double v = load(x, base + j, dt);
            if (v > m || std::isnan(v)) m = v;
        }
        double S = 0.0;
        if (m != -std::numeric_limits<double>::infinity())
            for (int64_t j = 0; j < cols; ++j) S += std::exp(load(x, base + j, dt) - m);
        const double lnS = std::log(S);                      // S >= 1 for a live row
        for (int64_t j = 0; j < cols; ++j) {
            const double v = (m == -std::numeric_limits<double>::infinity()) ? m : (load(x, base + j, dt) - m) - lnS;
            if (y64) y64[base + j] = v;
            if (y) store(y, base + j, dt, v);
        }
    });
    return 0;
}

// Softmax backward:  dx_j = y_j * (dy_j - sum_k y_k dy_k), y the forward output as stored, dy the incoming
// gradient.  scale64 (nullable) receives |y_j| * (|dy_j| + sum_k |y_k dy_k|), the quantity an error bound for the
// cancelling difference is stated against.
int oracle_softmax_bwd(const void* y, const void* dy, void* dx, double* dx64, double* scale64, int64_t rows, int64_t cols,
                       int dt, int nthreads) {
    if (bad(rows, cols, dt) || !y || !dy) return -1;
    for_rows(rows, nthreads, [=](int64_t r) {
        const int64_t base = r * cols;
        double s = 0.0, sa = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double p = load(y, base + j, dt) * load(dy, base + j, dt);
            s += p;
            sa += std::fabs(p);
        }
        for (int64_t j = 0; j < cols; ++j) {
            const double yj = load(y, base + j, dt), gj = load(dy, base + j, dt);
            const double v = yj * (gj - s);
            if (dx64) dx64[base + j] = v;
            if (scale64) scale64[base + j] = std::fabs(yj) * (std::fabs(gj) + sa);
            if (dx) store(dx, base + j, dt, v);
        }
    });
    return 0;
}

// Log-softmax backward:  dx_j = dy_j - exp(y_j) * sum_k dy_k, y the forward output (log-probabilities) as stored, dy the
// incoming gradient; exp(-inf) = 0, so masked entries pass their gradient through.  scale64 (nullable) receives
// |dy_j| + exp(y_j) * sum_k |dy_k|, the quantity an error bound for the difference is stated against.
int oracle_log_softmax_bwd(const void* y, const void* dy, void* dx, double* dx64, double* scale64, int64_t rows, int64_t cols,
                           int dt, int nthreads) {
    if (bad(rows, cols, dt) || !y || !dy) return -1;
    for_rows(rows, nthreads, [=](int64_t r) {
        const int64_t base = r * cols;
        double s = 0.0, sa = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double g = load(dy, base + j, dt);
            s += g;
            sa += std::fabs(g);
        }
        for (int64_t j = 0; j < cols; ++j) {
            const double p = std::exp(load(y, base + j, dt)), gj = load(dy, base + j, dt);
            const double v = gj - p * s;
            if (dx64) dx64[base + j] = v;
            if (scale64) scale64[base + j] = std::fabs(gj) + p * sa;
            if (dx) store(dx, base + j, dt, v);
        }
    });
    return 0;
}

// Backward pass of LayerNorm (rms = 0) or RMSNorm (rms = 1) from the forward pass's stored fp32 statistics.
//   xh_j = (x_j - mean) * rstd   (RMSNorm: x_j * rstd),   g_j = dy_j * gamma_j
//   LayerNorm:  dx_j = rstd * (g_j - mean_k g_k - xh_j * mean_k (g_k xh_k))
//   RMSNorm:    dx_j = rstd * (g_j - xh_j * mean_k (g_k xh_k))
//   dgamma_j = sum_rows dy_j * xh_j,   dbeta_j = sum_rows dy_j   (LayerNorm only)
// Everything in double, sums in increasing index, one rounding to the storage type.  dx_scale64 (nullable) receives
// rstd * (|g_j| + mean|g| + |xh_j| mean|g xh|), dg_scale64 / db_scale64 the sums of absolute terms.
int oracle_norm_bwd(const void* x, const void* gamma, const void* dy, const float* mean, const float* rstd, void* dx,
                    void* dgamma, void* dbeta, double* dx64, double* dg64, double* db64, double* dx_scale64,
                    double* dg_scale64, double* db_scale64, int64_t rows, int64_t cols, int rms, int dt, int nthreads) {
    if (bad(rows, cols, dt) || !x || !gamma || !dy || !rstd || (!rms && !mean)) return -1;
    const double n = static_cast<double>(cols);
    for_rows(rows, nthreads, [=](int64_t r) {
        const int64_t base = r * cols;
        const double mu = rms ? 0.0 : static_cast<double>(mean[r]), rs = static_cast<double>(rstd[r]);
        double sg = 0.0, sgx = 0.0, ag = 0.0, agx = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double xh = (load(x, base + j, dt) - mu) * rs, g = load(dy, base + j, dt) * load(gamma, j, dt);
            sg += g; sgx += g * xh; ag += std::fabs(g); agx += std::fabs(g * xh);
        }
        const double mg = rms ? 0.0 : sg / n, mgx = sgx / n;
        for (int64_t j = 0; j < cols; ++j) {
            const double xh = (load(x, base + j, dt) - mu) * rs, g = load(dy, base + j, dt) * load(gamma, j, dt);
            const double v = rs * (g - mg - xh * mgx);
            if (dx64) dx64[base + j] = v;
            if (dx_scale64) dx_scale64[base + j] = rs * (std::fabs(g) + (rms ? 0.0 : ag / n) + std::fabs(xh) * agx / n);
            if (dx) store(dx, base + j, dt, v);
        }
    });
    // parameter gradients: column sums over the rows (columns spread over the workers)
    for_rows(cols, nthreads, [=](int64_t j) {
        double sg = 0.0, sb = 0.0, ag = 0.0, ab = 0.0;
        for (int64_t r = 0; r < rows; ++r) {
            const double mu = rms ? 0.0 : static_cast<double>(mean[r]), rs = static_cast<double>(rstd[r]);
            const double d = load(dy, r * cols + j, dt), t = d * ((load(x, r * cols + j, dt) - mu) * rs);
            sg += t; sb += d; ag += std::fabs(t); ab += std::fabs(d);
        }
        if (dg64) dg64[j] = sg;
        if (db64) db64[j] = sb;
        if (dg_scale64) dg_scale64[j] = ag;
        if (db_scale64) db_scale64[j] = ab;
        if (dgamma) store(dgamma, j, dt, sg);
        if (dbeta && !rms) store(dbeta, j, dt, sb);
    });
    return 0;
}

// Element-wise sine (the kernel of the paper's Case Study 1): y_i = sin(x_i) in double, rounded once.
int oracle_sin(const void* x, void* y, double* y64, int64_t n, int dt) {
    if (n < 0 || (dt != F32 && dt != BF16) || !x) return -1;
    for (int64_t i = 0; i < n; ++i) {
        const double v = std::sin(load(x, i, dt));
        if (y64) y64[i] = v;
        if (y) store(y, i, dt, v);
    }
    return 0;
}

// Batched vector-matrix product (the paper's Case Study 2):  C[m,n] = sum_k A[m,k] * B[m,n,k],
// A [M,K], B [M,N,K] (k fastest), C [M,N].  Inputs widened exactly, products and the running sum in
// double in increasing k, one rounding to the output type.  scale64 (nullable) receives
// sum_k |A[m,k] * B[m,n,k]|, the quantity any summation-order error bound is stated against.
int oracle_bvecmat(const void* A, const void* B, void* C, double* c64, double* scale64, int64_t M, int64_t N,
                   int64_t K, int dt, int nthreads) {
    if (M < 0 || N < 0 || K <= 0 || (dt != F32 && dt != BF16) || ((M > 0 && N > 0) && (!A || !B))) return -1;
    for_rows(M * N, nthreads, [=](int64_t r) {
        const int64_t m = r / N;
        double s = 0.0, t = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double p = load(A, m * K + k, dt) * load(B, r * K + k, dt);
            s += p;
            t += std::fabs(p);
        }
        if (c64) c64[r] = s;
        if (scale64) scale64[r] = t;
        if (C) store(C, r, dt, s);
    });
    return 0;
}

// Residual add of a fused add-and-normalise:  h_i = x_i + r_i in double (exact for every pair of
// fp32 or bf16 inputs whose exponents differ by less than 29), rounded once to the storage type.
// Reading: the statistics and the output of the norm that follows are computed from this ROUNDED h,
// i.e. the fused op equals the two ops called one after the other.
int oracle_add(const void* x, const void* r, void* h, double* h64, int64_t n, int dt) {
    if (n < 0 || (dt != F32 && dt != BF16) || (n > 0 && (!x || !r))) return -1;
    for (int64_t i = 0; i < n; ++i) {
        const double v = load(x, i, dt) + load(r, i, dt);
        if (h64) h64[i] = v;
        if (h) store(h, i, dt, v);
    }
    return 0;
}

void oracle_bf16_from_double(const double* in, uint16_t* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_from_double(in[i]);
}

void oracle_bf16_to_double(const uint16_t* in, double* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_double(in[i]);
}

}  // extern "C"
