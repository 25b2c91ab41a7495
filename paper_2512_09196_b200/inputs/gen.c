/* Seeded synthetic inputs for the row-wise softmax / LayerNorm / RMSNorm workloads.
 *
 * This module holds data generation only: none of the three ops' arithmetic lives here.  Every
 * element is a pure function of (seed, stream, global element index), so a shard or a sample of
 * rows can be generated on its own and equals the same slice of the full tensor, whatever the
 * thread count.  Values are produced in double, rounded once to the tensor's storage type
 * (fp32, or bf16 as uint16 bit patterns), and that rounded array is what both the CUDA library and
 * the CPU oracle are fed.
 *
 * Streams: 0 = x, 1 = gamma / weight, 2 = beta, 3 = outlier coin flips.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define TF_GEN_F32 0
#define TF_GEN_BF16 1

static inline uint64_t mix64(uint64_t z) {          /* splitmix64 finaliser */
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* 64 bits for counter idx of (seed, stream). */
static inline uint64_t bits_at(uint64_t seed, uint64_t stream, uint64_t idx) {
    return mix64(mix64(seed * 0xD1342543DE82EF95ull + stream) + idx);
}

/* Uniform in (0, 1]: 53 bits, never 0, so log() below is finite. */
static inline double unit_at(uint64_t seed, uint64_t stream, uint64_t idx) {
    return (double)((bits_at(seed, stream, idx) >> 11) + 1) * 0x1.0p-53;
}

/* Standard normal for element i: Box-Muller on the uniforms at counters 2k and 2k+1, k = i / 2;
 * even i takes the cosine branch, odd i the sine branch. */
static inline double normal_at(uint64_t seed, uint64_t stream, uint64_t i) {
    const uint64_t k = i >> 1;
    const double u1 = unit_at(seed, stream, 2 * k), u2 = unit_at(seed, stream, 2 * k + 1);
    const double r = sqrt(-2.0 * log(u1)), t = 6.283185307179586476925286766559 * u2;
    return (i & 1) ? r * sin(t) : r * cos(t);
}

static inline uint16_t to_bf16(double v) {          /* via float, nearest-even; finite inputs only */
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static inline void put(void* out, int64_t i, int dt, double v) {
    if (dt == TF_GEN_F32) ((float*)out)[i] = (float)v;
    else ((uint16_t*)out)[i] = to_bf16(v);
}

/* out[i] = mean + std * N(0,1) at global index idx0 + i, i in [0, n). */
void tfgen_normal(void* out, int64_t n, int dt, uint64_t seed, uint64_t stream, double mean, double std,
                  int64_t idx0) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) put(out, i, dt, mean + std * normal_at(seed, stream, (uint64_t)(idx0 + i)));
}

/* out[i] = lo + (hi - lo) * U at global index idx0 + i. */
void tfgen_uniform(void* out, int64_t n, int dt, uint64_t seed, uint64_t stream, double lo, double hi,
                   int64_t idx0) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) put(out, i, dt, lo + (hi - lo) * unit_at(seed, stream, (uint64_t)(idx0 + i)));
}

/* N(mean, std^2) on stream 0 with an independent coin of probability p per element on stream 3;
 * where the coin lands the value is multiplied by factor before the one rounding. */
void tfgen_normal_outliers(void* out, int64_t n, int dt, uint64_t seed, double mean, double std, double p,
                           double factor, int64_t idx0) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        const uint64_t g = (uint64_t)(idx0 + i);
        double v = mean + std * normal_at(seed, 0, g);
        if (unit_at(seed, 3, g) <= p) v *= factor;
        put(out, i, dt, v);
    }
}

/* Causal-like tail mask: global row r = row0 + i gets its last (r * step mod cols) columns set to
 * -infinity.  x holds rows_local rows of cols elements. */
void tfgen_tail_mask(void* x, int64_t rows_local, int64_t cols, int dt, int64_t step, int64_t row0) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows_local; ++i) {
        const int64_t k = ((row0 + i) * step) % cols;
        for (int64_t j = cols - k; j < cols; ++j) {
            if (dt == TF_GEN_F32) ((float*)x)[i * cols + j] = -INFINITY;
            else ((uint16_t*)x)[i * cols + j] = 0xFF80u;
        }
    }
}
