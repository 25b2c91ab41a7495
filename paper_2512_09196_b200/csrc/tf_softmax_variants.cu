// Three more row-wise reduce-then-normalise ops on the softmax family:
//   log-softmax forward    y_j  = (x_j - m) - ln sum_k exp(x_k - m),  m = max_k x_k
//   softmax backward       dx_j = y_j * (dy_j - sum_k y_k dy_k)
//   log-softmax backward   dx_j = dy_j - exp(y_j) * sum_k dy_k
// One kernel shape serves all of them: a CTA owns a row and holds it in registers (VPT 16-byte vectors per thread, loaded at
// once), reduces across the CTA, finishes and stores -- one read of every input element, one write of every output
// element.  Rows of up to 2 KiB are owned by lane groups instead (several rows per warp).  Rows beyond 32 KiB are
// streamed in two passes of 16-byte loads, the second from L2; when such rows are too few to give every SM a CTA (logits
// of a decode batch), the CTAs of a thread-block cluster share each row, slices in registers where they fit and streamed
// where not, with one exchange of partials through distributed shared memory.  Unaligned tensors and odd widths take
// scalar passes.
//
// Log-softmax keeps x - m as a difference (exact for bf16 inputs, one rounding for fp32) and subtracts ln S computed
// from S = sum 2^((x - m) log2 e) with the accurate logarithm; the term of the maximum is exactly 1, so S >= 1 and its
// fp32 summation error is a few 2^-24 absolute, which is the absolute part of the tolerance the tests use.
#include <cooperative_groups.h>

#include <algorithm>

#include "../../include/tf.h"
#include "tf_streamrow.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace {

constexpr int kOpLogSoftmax = 0, kOpSoftmaxBwd = 1, kOpLogSoftmaxBwd = 2;

// The two backward passes share every kernel: both reduce one number per row from (y, dy) and finish element-wise.
//   softmax backward       term y dy,  dx = y (dy - sum)
//   log-softmax backward   term dy,    dx = dy - exp(y) sum
// exp(y) is one MUFU op on a biased exponent (2^(y log2 e + 64), flushing only below a true value of 2^-190) scaled back
// by an exact, non-flushing 2^-64: probabilities in the subnormal range stay exact to rounding; exp(-inf) = 0.
template <int WHICH> __device__ __forceinline__ float bwd_accumulate(float y, float g, float s) {
    return WHICH == kOpSoftmaxBwd ? fmaf(y, g, s) : s + g;
}
template <int WHICH> __device__ __forceinline__ float bwd_finish(float y, float g, float s) {
    if (WHICH == kOpSoftmaxBwd) return y * (g - s);
    const float p = ex2_ftz(fmaf(y, kLog2e, 64.f)) * 0x1p-64f;
    return fmaf(-p, s, g);
}

// fp32 values a thread holds for its share of a row; up to 32 of them leave room for 1024 threads, up to 64 for 512.
template <int WHICH, int DT, int VPT> constexpr int row2_floats() { return VPT * Elem<DT>::NE * (WHICH != kOpLogSoftmax ? 2 : 1); }
template <int WHICH, int DT, int VPT> constexpr int row2_max_threads() { return row2_floats<WHICH, DT, VPT>() <= 32 ? 1024 : 512; }

template <int WHICH, int DT, int VPT>
__global__ void __launch_bounds__(row2_max_threads<WHICH, DT, VPT>()) k_row2(const uint4* in0, const uint4* in1, uint4* out,
                                               int64_t rows, int nvec) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    __shared__ float buf[2][32];
    pdl_wait();
    pdl_trigger();
    const int T = blockDim.x, t = threadIdx.x;
    const int64_t row = blockIdx.x;
    if (row >= rows) return;
    const uint4* a = in0 + row * nvec + t;
    uint4* o = out + row * nvec + t;
    bool valid[VPT];
    uint4 ra[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = t + v * T < nvec;
        ra[v] = valid[v] ? ld_stream(a + v * T) : make_uint4(0, 0, 0, 0);
    }
    if constexpr (WHICH == kOpLogSoftmax) {
        float m = kNegInf;
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) m = fmaxf(m, vec_max<DT>(ra[v]));
        m = cta_reduce<MaxOp>(m, buf[0]);
        float d[VPT][NE];
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float x[NE];
            E::unpack(ra[v], x);
#pragma unroll
            for (int i = 0; i < NE; ++i) {
                d[v][i] = x[i] - m;                                       // -inf for masked entries; NaN only if the whole row is masked
                if (valid[v]) s += ex2_ftz(d[v][i] * kLog2e);             // 2^0 = 1 exactly for the maximum
            }
        }
        s = cta_reduce<SumOp>(s, buf[1]);
        const float lns = logf(s);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float y[NE];
#pragma unroll
            for (int i = 0; i < NE; ++i) y[i] = (m == kNegInf) ? kNegInf : d[v][i] - lns;
            if (valid[v]) st_stream(o + v * T, E::pack(y));
        }
    } else {
        const uint4* b = in1 + row * nvec + t;
        float y[VPT][NE], g[VPT][NE];
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            const uint4 rb = valid[v] ? ld_stream(b + v * T) : make_uint4(0, 0, 0, 0);
            E::unpack(ra[v], y[v]);
            E::unpack(rb, g[v]);
#pragma unroll
            for (int i = 0; i < NE; ++i) s = bwd_accumulate<WHICH>(y[v][i], g[v][i], s);    // absent vectors hold zeros
        }
        s = cta_reduce<SumOp>(s, buf[0]);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float dx[NE];
#pragma unroll
            for (int i = 0; i < NE; ++i) dx[i] = bwd_finish<WHICH>(y[v][i], g[v][i], s);
            if (valid[v]) st_stream(o + v * T, E::pack(dx));
        }
    }
}

// Rows beyond what one CTA should hold in registers: a thread-block cluster of `cs` CTAs owns a row, each CTA a slice of
// it in registers (the same VPT vectors per thread, loaded at once).  One exchange: every CTA writes its partial --
// (slice maximum, sum of 2^((x - slice maximum) log2 e)) for log-softmax, sum y dy for the backward pass -- into every
// peer's shared memory, one cluster barrier, and every CTA combines the partials in rank order (the same bits in all of
// them): M = max m_k, S = sum_k s_k 2^((m_k - M) log2 e).  Still one read of every input element and one write of every
// output element, and small slices keep several CTAs on an SM, which is what the long rows lacked.
template <int WHICH, int DT, int VPT>
__global__ void __launch_bounds__(row2_max_threads<WHICH, DT, VPT>()) k_row2_cluster(const uint4* in0, const uint4* in1,
                                                                                     uint4* out, int64_t rows, int nvec, int cs) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    __shared__ float buf[2][32];
    __shared__ float xch[kMaxCluster][2];
    pdl_wait();
    pdl_trigger();
    cg::cluster_group cl = cg::this_cluster();
    const int T = blockDim.x, t = threadIdx.x;
    const int rank = static_cast<int>(blockIdx.x % cs);
    const int64_t row = blockIdx.x / cs;                          // the grid is rows x cs CTAs
    const int per = (nvec + cs - 1) / cs;
    const int first = rank * per;
    const int len = max(0, min(per, nvec - first));
    const uint4* a = in0 + row * nvec + first + t;
    uint4* o = out + row * nvec + first + t;
    bool valid[VPT];
    uint4 ra[VPT], rb[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = t + v * T < len;
        ra[v] = valid[v] ? ld_stream(a + v * T) : make_uint4(0, 0, 0, 0);
        if (WHICH != kOpLogSoftmax) rb[v] = valid[v] ? ld_stream(in1 + row * nvec + first + t + v * T) : make_uint4(0, 0, 0, 0);
    }
    cl.sync();                     // every CTA of the cluster is resident before any remote write (the loads are already under way)
    if constexpr (WHICH == kOpLogSoftmax) {
        float m = kNegInf;
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) m = fmaxf(m, vec_max<DT>(ra[v]));
        m = cta_reduce<MaxOp>(m, buf[0]);
        float s = 0.f;
        if (m != kNegInf) {
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                float x[NE];
                E::unpack(ra[v], x);
#pragma unroll
                for (int i = 0; i < NE; ++i)
                    if (valid[v]) s += ex2_ftz((x[i] - m) * kLog2e);
            }
        }
        s = cta_reduce<SumOp>(s, buf[1]);
        if (t < cs) {
            float* dst = cl.map_shared_rank(&xch[rank][0], t);
            dst[0] = m; dst[1] = s;
        }
        cl.sync();                                                 // release our writes, acquire the peers'
        float M = kNegInf, S = 0.f;
        for (int k = 0; k < cs; ++k) M = fmaxf(M, xch[k][0]);
        for (int k = 0; k < cs; ++k)
            if (xch[k][0] != kNegInf) S += xch[k][1] * ex2_ftz((xch[k][0] - M) * kLog2e);      // the slice of the maximum contributes exactly s_k
        const float lns = logf(S);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float x[NE], y[NE];
            E::unpack(ra[v], x);
#pragma unroll
            for (int i = 0; i < NE; ++i) y[i] = (M == kNegInf) ? kNegInf : (x[i] - M) - lns;
            if (valid[v]) st_stream(o + v * T, E::pack(y));
        }
    } else {
        float y[VPT][NE], g[VPT][NE];
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            E::unpack(ra[v], y[v]);
            E::unpack(rb[v], g[v]);
#pragma unroll
            for (int i = 0; i < NE; ++i) s = bwd_accumulate<WHICH>(y[v][i], g[v][i], s);    // absent vectors hold zeros
        }
        s = cta_reduce<SumOp>(s, buf[0]);
        if (t < cs) {
            float* dst = cl.map_shared_rank(&xch[rank][0], t);
            dst[0] = s; dst[1] = 0.f;
        }
        cl.sync();
        float total = 0.f;
        for (int k = 0; k < cs; ++k) total += xch[k][0];
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float dx[NE];
#pragma unroll
            for (int i = 0; i < NE; ++i) dx[i] = bwd_finish<WHICH>(y[v][i], g[v][i], total);
            if (valid[v]) st_stream(o + v * T, E::pack(dx));
        }
    }
}

// Short rows (up to 2 KiB): a group of LANES lanes owns a row, a CTA of 128 threads covers 128 / LANES consecutive
// rows, reductions are shuffles.  Every lane runs every step (the shuffles need the whole warp); rows past the end
// are loaded as zeros and not stored.
template <int WHICH, int DT, int LANES, int VPT>
__global__ void __launch_bounds__(128) k_row2_group(const uint4* in0, const uint4* in1, uint4* out,
                                                    int64_t rows, int nvec) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x % LANES;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x / LANES) + threadIdx.x / LANES;
    const bool live = row < rows;
    const int64_t base = (live ? row : 0) * nvec + lane;
    bool valid[VPT];
    uint4 ra[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = live && lane + v * LANES < nvec;
        ra[v] = valid[v] ? ld_stream(in0 + base + v * LANES) : make_uint4(0, 0, 0, 0);
    }
    if constexpr (WHICH == kOpLogSoftmax) {
        float m = kNegInf;
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) m = fmaxf(m, vec_max<DT>(ra[v]));
        m = group_reduce<MaxOp, LANES>(m);
        float d[VPT][NE];
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float x[NE];
            E::unpack(ra[v], x);
#pragma unroll
            for (int i = 0; i < NE; ++i) {
                d[v][i] = x[i] - m;
                if (valid[v]) s += ex2_ftz(d[v][i] * kLog2e);
            }
        }
        s = group_reduce<SumOp, LANES>(s);
        const float lns = logf(s);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float y[NE];
#pragma unroll
            for (int i = 0; i < NE; ++i) y[i] = (m == kNegInf) ? kNegInf : d[v][i] - lns;
            if (valid[v]) st_stream(out + base + v * LANES, E::pack(y));
        }
    } else {
        float y[VPT][NE], g[VPT][NE];
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            const uint4 rb = valid[v] ? ld_stream(in1 + base + v * LANES) : make_uint4(0, 0, 0, 0);
            E::unpack(ra[v], y[v]);
            E::unpack(rb, g[v]);
#pragma unroll
            for (int i = 0; i < NE; ++i) s = bwd_accumulate<WHICH>(y[v][i], g[v][i], s);
        }
        s = group_reduce<SumOp, LANES>(s);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float dx[NE];
#pragma unroll
            for (int i = 0; i < NE; ++i) dx[i] = bwd_finish<WHICH>(y[v][i], g[v][i], s);
            if (valid[v]) st_stream(out + base + v * LANES, E::pack(dx));
        }
    }
}

// Rows too long for registers (aligned): a CTA per row, passes of four independent 16-byte loads per thread; the first
// pass comes from HBM, the later ones find the row in L2 (a row is at most a few MiB).
// CL: the row is shared by the `cs` CTAs of a thread-block cluster (few rows of many columns: one CTA per row would leave
// most of the device idle); each streams its own slice and the partials meet as in k_row2_cluster, between the passes.
template <int WHICH, int DT, bool CL>
__global__ void __launch_bounds__(512) k_row2_stream(const uint4* in0, const uint4* in1, uint4* out,
                                                     int64_t rows, int64_t row_vecs, int cs) {
    using E = Elem<DT>;
    constexpr int NE = E::NE, U = 4;
    __shared__ float buf[2][32];
    __shared__ float xch[kMaxCluster][2];
    pdl_wait();
    pdl_trigger();
    const int T = blockDim.x, t = threadIdx.x;
    const int rank = CL ? static_cast<int>(blockIdx.x % cs) : 0;
    const int64_t row = CL ? blockIdx.x / cs : blockIdx.x;
    if (!CL && row >= rows) return;
    // the output may alias an input (in-place calls), so the first pass reads with ordinary coherent loads (not the
    // read-only path) and asks L2 to keep the lines for the passes that follow
    const uint64_t keep = policy_evict_last();
    const int64_t per = CL ? (row_vecs + cs - 1) / cs : row_vecs, first = rank * per;
    const int64_t nvec = per < row_vecs - first ? per : (row_vecs - first > 0 ? row_vecs - first : 0);      // this CTA's slice
    const uint4* a = in0 + row * row_vecs + first;
    uint4* o = out + row * row_vecs + first;
    if constexpr (CL) cg::this_cluster().sync();                  // every CTA of the cluster is resident before any remote write
    const int64_t step = static_cast<int64_t>(T) * U;
    if constexpr (WHICH == kOpLogSoftmax) {
        // one pass for both statistics: every thread keeps (running max, sum relative to it) and rescales the sum when
        // its maximum grows; exponents are formed from differences, never from a rounded offset
        float mt = kNegInf, st = 0.f;
        for (int64_t b0 = t; b0 < nvec; b0 += step) {
            uint4 r[U];
            float cm = kNegInf;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = b0 + u * T < nvec;
                r[u] = ok ? ld_hint(a + b0 + u * T, keep) : make_uint4(0, 0, 0, 0);
                if (ok) cm = fmaxf(cm, vec_max<DT>(r[u]));
            }
            if (cm > mt) {
                st = (mt == kNegInf) ? 0.f : st * ex2_ftz((mt - cm) * kLog2e);
                mt = cm;
            }
            if (mt != kNegInf) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float x[NE];
                    E::unpack(r[u], x);
                    if (b0 + u * T < nvec) {
#pragma unroll
                        for (int i = 0; i < NE; ++i) st += ex2_ftz((x[i] - mt) * kLog2e);
                    }
                }
            }
        }
        float m = cta_reduce<MaxOp>(mt, buf[0]);
        float s = (mt == kNegInf) ? 0.f : st * ex2_ftz((mt - m) * kLog2e);          // 2^0 = 1 exactly for the thread that holds the maximum
        s = cta_reduce<SumOp>(s, buf[1]);
        if constexpr (CL) {
            cg::cluster_group cl = cg::this_cluster();
            if (t < cs) {
                float* dst = cl.map_shared_rank(&xch[rank][0], t);
                dst[0] = m; dst[1] = s;
            }
            cl.sync();
            m = kNegInf; s = 0.f;
            for (int k = 0; k < cs; ++k) m = fmaxf(m, xch[k][0]);
            for (int k = 0; k < cs; ++k)
                if (xch[k][0] != kNegInf) s += xch[k][1] * ex2_ftz((xch[k][0] - m) * kLog2e);
        }
        const float lns = logf(s);
        for (int64_t b0 = t; b0 < nvec; b0 += step) {
            uint4 r[U];
#pragma unroll
            for (int u = 0; u < U; ++u) r[u] = b0 + u * T < nvec ? ld_stream(a + b0 + u * T) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float x[NE];
                E::unpack(r[u], x);
#pragma unroll
                for (int i = 0; i < NE; ++i) x[i] = (m == kNegInf) ? kNegInf : (x[i] - m) - lns;
                if (b0 + u * T < nvec) st_stream(o + b0 + u * T, E::pack(x));
            }
        }
    } else {
        const uint4* b = in1 + row * row_vecs + first;
        float s = 0.f;
        for (int64_t b0 = t; b0 < nvec; b0 += step) {
            uint4 ry[U], rg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = b0 + u * T < nvec;
                ry[u] = ok ? ld_hint(a + b0 + u * T, keep) : make_uint4(0, 0, 0, 0);
                rg[u] = ok ? ld_hint(b + b0 + u * T, keep) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float y[NE], g[NE];
                E::unpack(ry[u], y);
                E::unpack(rg[u], g);
#pragma unroll
                for (int i = 0; i < NE; ++i) s = bwd_accumulate<WHICH>(y[i], g[i], s);
            }
        }
        s = cta_reduce<SumOp>(s, buf[0]);
        if constexpr (CL) {
            cg::cluster_group cl = cg::this_cluster();
            if (t < cs) {
                float* dst = cl.map_shared_rank(&xch[rank][0], t);
                dst[0] = s; dst[1] = 0.f;
            }
            cl.sync();
            s = 0.f;
            for (int k = 0; k < cs; ++k) s += xch[k][0];
        }
        for (int64_t b0 = t; b0 < nvec; b0 += step) {
            uint4 ry[U], rg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = b0 + u * T < nvec;
                ry[u] = ok ? ld_stream(a + b0 + u * T) : make_uint4(0, 0, 0, 0);
                rg[u] = ok ? ld_stream(b + b0 + u * T) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float y[NE], g[NE];
                E::unpack(ry[u], y);
                E::unpack(rg[u], g);
#pragma unroll
                for (int i = 0; i < NE; ++i) y[i] = bwd_finish<WHICH>(y[i], g[i], s);
                if (b0 + u * T < nvec) st_stream(o + b0 + u * T, E::pack(y));
            }
        }
    }
}

// Any alignment, any width, any length: a CTA per row, scalar passes.
template <int WHICH, int DT>
__global__ void __launch_bounds__(256) k_row2_scalar(const typename Elem<DT>::scalar* in0, const typename Elem<DT>::scalar* in1,
                                                     typename Elem<DT>::scalar* out, int64_t rows, int64_t cols) {
    using E = Elem<DT>;
    __shared__ float buf[2][32];
    const int64_t row = blockIdx.x;
    if (row >= rows) return;
    const typename E::scalar* a = in0 + row * cols;
    typename E::scalar* o = out + row * cols;
    if constexpr (WHICH == kOpLogSoftmax) {
        float m = kNegInf;
        for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) m = fmaxf(m, E::to_float(a[j]));
        m = cta_reduce<MaxOp>(m, buf[0]);
        float s = 0.f;
        if (m != kNegInf)
            for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) s += expf(E::to_float(a[j]) - m);
        s = cta_reduce<SumOp>(s, buf[1]);
        const float lns = logf(s);
        for (int64_t j = threadIdx.x; j < cols; j += blockDim.x)
            o[j] = E::from_float(m == kNegInf ? kNegInf : (E::to_float(a[j]) - m) - lns);
    } else {
        const typename E::scalar* b = in1 + row * cols;
        float s = 0.f;
        for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) s = bwd_accumulate<WHICH>(E::to_float(a[j]), E::to_float(b[j]), s);
        s = cta_reduce<SumOp>(s, buf[0]);
        for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) o[j] = E::from_float(bwd_finish<WHICH>(E::to_float(a[j]), E::to_float(b[j]), s));
    }
}

bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Log-softmax forward on rows of 8-64 KiB: the row is copied into shared memory by 16-byte asynchronous copies that are
// all requested at once (NS steps of four vectors per thread, a warp taking 128 consecutive vectors per step), then swept
// three times out of shared memory -- maximum, sum of exponentials, result -- with the arithmetic of the register forms
// above ((x - m) first, then minus ln S).  The row costs no registers, so a dozen small CTAs are resident per SM and
// the copies of the next rows are in flight while this one is worked on.  FULL: the row fills the steps exactly.
__device__ __forceinline__ void lsm_cp_async16(uint4* dst, const uint4* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
template <int N> __device__ __forceinline__ void lsm_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int DT, int NS, bool FULL>
__global__ void __launch_bounds__(256, 4) k_logsoftmax_smem(const uint4* x, uint4* y, int64_t rows, int nvec) {
    using E = Elem<DT>;
    constexpr int NE = E::NE, U = 4;
    __shared__ float buf[2][32];
    extern __shared__ __align__(16) unsigned char lsm_smem[];
    pdl_wait();
    pdl_trigger();
    const int t = threadIdx.x;
    const int step = (blockDim.x >> 5) * U * 32;
    const int toff = (t >> 5) * U * 32 + (t & 31);
    const int64_t row = blockIdx.x;
    const uint4* const xr = x + row * nvec + toff;
    uint4* const yr = y + row * nvec + toff;
    const uint4* const ring = reinterpret_cast<const uint4*>(lsm_smem) + toff;
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (FULL || s * step + toff + u * 32 < nvec) lsm_cp_async16(const_cast<uint4*>(ring) + s * step + u * 32, xr + s * step + u * 32);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    float m = kNegInf;
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        if (s == 0) lsm_cp_async_wait<NS - 1>();
        else if (s == 1) lsm_cp_async_wait<(NS > 2 ? NS - 2 : 0)>();
        else if (s == 2) lsm_cp_async_wait<(NS > 3 ? NS - 3 : 0)>();
        else lsm_cp_async_wait<0>();
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (FULL || s * step + toff + u * 32 < nvec) m = fmaxf(m, vec_max<DT>(ring[s * step + u * 32]));
    }
    m = cta_reduce<MaxOp>(m, buf[0]);
    float acc[U] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (FULL || s * step + toff + u * 32 < nvec) {
                float v[NE];
                E::unpack(ring[s * step + u * 32], v);
#pragma unroll
                for (int i = 0; i < NE; ++i) acc[u] += ex2_ftz((v[i] - m) * kLog2e);     // 2^0 = 1 exactly for the maximum
            }
        }
    }
    const float sum = cta_reduce<SumOp>((acc[0] + acc[1]) + (acc[2] + acc[3]), buf[1]);
    const float lns = logf(sum);
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (FULL || s * step + toff + u * 32 < nvec) {
                float v[NE];
                E::unpack(ring[s * step + u * 32], v);
#pragma unroll
                for (int i = 0; i < NE; ++i) v[i] = (m == kNegInf) ? kNegInf : (v[i] - m) - lns;
                st_stream(yr + s * step + u * 32, E::pack(v));
            }
        }
    }
}

template <int DT, int NS, bool FULL>
cudaError_t launch_logsoftmax_smem(int threads, cudaStream_t st, const void* in0, void* out, int64_t rows, int nvec) {
    auto fn = k_logsoftmax_smem<DT, NS, FULL>;
    const size_t smem = static_cast<size_t>(NS) * threads * 4 * 16;
    static bool raised = false;                                  // per instantiation; the limit is a property of the function
    if (smem > 40 * 1024 && !raised) {                           // the default limit counts the static buffers as well
        const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e != cudaSuccess) return e;
        raised = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(rows));
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, static_cast<const uint4*>(in0), static_cast<uint4*>(out), rows, nvec);
}

template <int DT>
cudaError_t launch_logsoftmax_smem_dt(cudaStream_t st, const void* in0, void* out, int64_t rows, int nvec) {
    const int threads = std::min(256, std::max(32, ((nvec + 7) / 8 + 31) / 32 * 32));
    const int steps = (nvec + threads * 4 - 1) / (threads * 4);
    const bool full = steps * threads * 4 == nvec;
    switch (steps) {
        case 1: return full ? launch_logsoftmax_smem<DT, 1, true>(threads, st, in0, out, rows, nvec) : launch_logsoftmax_smem<DT, 1, false>(threads, st, in0, out, rows, nvec);
        case 2: return full ? launch_logsoftmax_smem<DT, 2, true>(threads, st, in0, out, rows, nvec) : launch_logsoftmax_smem<DT, 2, false>(threads, st, in0, out, rows, nvec);
        case 3: return full ? launch_logsoftmax_smem<DT, 3, true>(threads, st, in0, out, rows, nvec) : launch_logsoftmax_smem<DT, 3, false>(threads, st, in0, out, rows, nvec);
        case 4: return full ? launch_logsoftmax_smem<DT, 4, true>(threads, st, in0, out, rows, nvec) : launch_logsoftmax_smem<DT, 4, false>(threads, st, in0, out, rows, nvec);
    }
    return cudaErrorInvalidValue;
}

int sm_count() {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

template <int WHICH, int DT, int VPT>
cudaError_t launch_vpt(int threads, cudaStream_t st, const void* in0, const void* in1, void* out, int64_t rows, int nvec) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(rows));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_row2<WHICH, DT, VPT>, static_cast<const uint4*>(in0), static_cast<const uint4*>(in1),
                              static_cast<uint4*>(out), rows, nvec);
}

template <class... T>
cudaError_t launch_pdl(void (*fn)(T...), int64_t grid, int threads, cudaStream_t st, T... args) {
    if (grid > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, args...);
}

template <int WHICH, int DT, int LANES, int VPT>
cudaError_t launch_group(cudaStream_t st, const void* in0, const void* in1, void* out, int64_t rows, int nvec) {
    const int rpc = 128 / LANES;
    return launch_pdl(k_row2_group<WHICH, DT, LANES, VPT>, (rows + rpc - 1) / rpc, 128, st, static_cast<const uint4*>(in0),
                      static_cast<const uint4*>(in1), static_cast<uint4*>(out), rows, nvec);
}

// Test and bench hook: 0 = automatic, 1 = never a cluster per row, 2 / 4 / 8 = that many CTAs per row wherever the slices fit.
int g_force_cluster = 0;

template <int WHICH, int DT, int VPT>
cudaError_t launch_cluster_vpt(int threads, int cs, cudaStream_t st, const void* in0, const void* in1, void* out, int64_t rows, int nvec) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(rows * cs));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, k_row2_cluster<WHICH, DT, VPT>, static_cast<const uint4*>(in0), static_cast<const uint4*>(in1),
                              static_cast<uint4*>(out), rows, nvec, cs);
}

// Geometry of a register-resident slice of `nv` vectors: the fewest vectors per thread that keep the CTA at 128 threads
// or fewer; else the most the register budget allows.  vpt = 0: does not fit.
template <int WHICH, int DT>
void slice_geometry(int nv, int& vpt, int& threads) {
    vpt = 0; threads = 0;
    const int fl[4] = {row2_floats<WHICH, DT, 1>(), row2_floats<WHICH, DT, 2>(), row2_floats<WHICH, DT, 4>(), row2_floats<WHICH, DT, 8>()};
    for (int k = 0; k < 4; ++k) {
        const int v = 1 << k;
        if (fl[k] > 64) break;
        const int th = std::max(32, ((nv + v - 1) / v + 31) / 32 * 32);
        if (th > (fl[k] <= 32 ? 1024 : 512)) continue;
        vpt = v; threads = th;
        if (th <= 128) break;
    }
}

template <int WHICH, int DT>
cudaError_t launch_dt(cudaStream_t st, const void* in0, const void* in1, void* out, int64_t rows, int64_t cols) {
    using S = typename Elem<DT>::scalar;
    if (rows > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
    {
        const int64_t b = cols * Elem<DT>::SIZE;
        const bool al = al16(in0) && al16(out) && (WHICH == kOpLogSoftmax || al16(in1)) && b % 16 == 0;
        if (al && b / 16 <= 128 && g_force_cluster <= 1) {          // rows up to 2 KiB: lane groups
            const int nv = static_cast<int>(b / 16);
            if (nv <= 8) return launch_group<WHICH, DT, 8, 1>(st, in0, in1, out, rows, nv);
            if (nv <= 16) return launch_group<WHICH, DT, 8, 2>(st, in0, in1, out, rows, nv);
            if (nv <= 32) return launch_group<WHICH, DT, 16, 2>(st, in0, in1, out, rows, nv);
            if (nv <= 64) return launch_group<WHICH, DT, 32, 2>(st, in0, in1, out, rows, nv);
            return launch_group<WHICH, DT, 32, 4>(st, in0, in1, out, rows, nv);
        }
    }
    const int64_t bytes = cols * Elem<DT>::SIZE;
    const bool aligned = al16(in0) && al16(out) && (WHICH == kOpLogSoftmax || al16(in1)) && bytes % 16 == 0;
    if constexpr (WHICH == kOpLogSoftmax) {
        // the forward pass on many rows of 8-64 KiB: the row staged in shared memory by asynchronous copies
        if (aligned && g_force_cluster == 0 && bytes >= 8 * 1024 && bytes <= 64 * 1024 && rows >= 2LL * sm_count())
            return launch_logsoftmax_smem_dt<DT>(st, in0, out, rows, static_cast<int>(bytes / 16));
    }
    int vpt = 0, threads = 0;
    // a cluster per row: rows beyond 32 KiB when there are too few of them to fill the device with one CTA each -- as many
    // CTAs per row (2, 4 or 8) as keep the launch within about two CTAs per SM.  With more rows of up to 128 KiB the
    // streamed passes of one CTA are faster (bf16 [8192, 32768]: 5.4 TB/s streamed, 3.6 with clusters).  Or where the hook asks.
    // Rows of 256 KiB and more are shared whatever their number, in streamed slices of about 128 KiB: one CTA per row in
    // flight on every SM is more than L2 holds of such rows, so the second pass went back to HBM (fp32 [2048, 131072]:
    // 4.4 -> 6.0 TB/s with four CTAs per row).
    int cs = g_force_cluster > 1 ? g_force_cluster : 0;
    if (g_force_cluster == 0 && bytes / 16 > 2048) {
        const int64_t room = 2 * static_cast<int64_t>(sm_count()) / rows;
        cs = room >= 8 ? 8 : room >= 4 ? 4 : room >= 2 ? 2 : 0;
        const int64_t pieces = bytes / (128 * 1024);
        cs = std::max(cs, pieces >= 8 ? 8 : pieces >= 4 ? 4 : pieces >= 2 ? 2 : 0);
    }
    if (aligned && cs >= 2 && rows * kMaxCluster <= 0x7FFFFFFF) {
        const int64_t nv = bytes / 16;
        int64_t per = (nv + cs - 1) / cs;
        if (per > 2048) {                                           // slices too long for registers: every CTA streams its own
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(static_cast<unsigned>(rows * cs));
            cfg.blockDim = dim3(512);
            cfg.stream = st;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[1].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            const cudaError_t e = cudaLaunchKernelEx(&cfg, k_row2_stream<WHICH, DT, true>, static_cast<const uint4*>(in0), static_cast<const uint4*>(in1),
                                                     static_cast<uint4*>(out), rows, nv, cs);
            if (e == cudaSuccess) return e;
            cudaGetLastError();
        } else {
            slice_geometry<WHICH, DT>(static_cast<int>(per), vpt, threads);
            if (vpt) {
                const int nvec = static_cast<int>(nv);
                cudaError_t e = cudaErrorInvalidValue;
                switch (vpt) {
                    case 1: e = launch_cluster_vpt<WHICH, DT, 1>(threads, cs, st, in0, in1, out, rows, nvec); break;
                    case 2: e = launch_cluster_vpt<WHICH, DT, 2>(threads, cs, st, in0, in1, out, rows, nvec); break;
                    case 4: e = launch_cluster_vpt<WHICH, DT, 4>(threads, cs, st, in0, in1, out, rows, nvec); break;
                    default:
                        if constexpr (row2_floats<WHICH, DT, 8>() <= 64) e = launch_cluster_vpt<WHICH, DT, 8>(threads, cs, st, in0, in1, out, rows, nvec);
                }
                if (e == cudaSuccess) return e;
                cudaGetLastError();                                 // the cluster could not be launched here: the forms below serve the shape
                vpt = 0;
            }
        }
    }
    // beyond 32 KiB a single CTA that holds the row in registers is alone on its SM for too long (measured at 64 KiB:
    // log-softmax 4.1 TB/s held, 5.4 streamed), so such rows are streamed when no cluster took them
    if (aligned && bytes / 16 <= 2048) slice_geometry<WHICH, DT>(static_cast<int>(bytes / 16), vpt, threads);
    if (vpt == 0 && aligned)
        return launch_pdl(k_row2_stream<WHICH, DT, false>, rows, 512, st, static_cast<const uint4*>(in0), static_cast<const uint4*>(in1),
                          static_cast<uint4*>(out), rows, bytes / 16, 1);
    if (vpt == 0) {
        k_row2_scalar<WHICH, DT><<<static_cast<unsigned>(rows), 256, 0, st>>>(static_cast<const S*>(in0), static_cast<const S*>(in1),
                                                                             static_cast<S*>(out), rows, cols);
        return cudaGetLastError();
    }
    const int nvec = static_cast<int>(bytes / 16);
    switch (vpt) {
        case 1: return launch_vpt<WHICH, DT, 1>(threads, st, in0, in1, out, rows, nvec);
        case 2: return launch_vpt<WHICH, DT, 2>(threads, st, in0, in1, out, rows, nvec);
        case 4: return launch_vpt<WHICH, DT, 4>(threads, st, in0, in1, out, rows, nvec);
        default:
            if constexpr (row2_floats<WHICH, DT, 8>() <= 64) return launch_vpt<WHICH, DT, 8>(threads, st, in0, in1, out, rows, nvec);
            else return cudaErrorInvalidValue;
    }
}

template <int WHICH>
tf_status run2(const void* in0, const void* in1, void* out, int64_t rows, int64_t cols, int dt, void* stream) {
    if (rows < 0 || cols <= 0 || (dt != DT_F32 && dt != DT_BF16)) return TF_ERR_INVALID_ARG;
    if (rows > 0 && (!in0 || !out || (WHICH != kOpLogSoftmax && !in1))) return TF_ERR_INVALID_ARG;
    if (rows == 0) return TF_OK;
    if (cols > (INT64_MAX / 8) / rows) return TF_ERR_UNSUPPORTED;
    count_launches(1);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const cudaError_t e = dt == DT_F32 ? launch_dt<WHICH, DT_F32>(st, in0, in1, out, rows, cols)
                                       : launch_dt<WHICH, DT_BF16>(st, in0, in1, out, rows, cols);
    if (e == cudaErrorInvalidConfiguration) return TF_ERR_UNSUPPORTED;
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}

}  // namespace
}  // namespace tf

using namespace tf;

extern "C" tf_status tf_softmax_variants_force(int cluster) {
    if (cluster != 0 && cluster != 1 && cluster != 2 && cluster != 4 && cluster != 8) return TF_ERR_INVALID_ARG;
    g_force_cluster = cluster;
    return TF_OK;
}

extern "C" tf_status tf_log_softmax_fwd(const void* x, void* y, int64_t rows, int64_t cols, tf_dtype dt, void* stream) {
    return run2<kOpLogSoftmax>(x, nullptr, y, rows, cols, dt, stream);
}

extern "C" tf_status tf_log_softmax_bwd(const void* y, const void* dy, void* dx, int64_t rows, int64_t cols, tf_dtype dt, void* stream) {
    return run2<kOpLogSoftmaxBwd>(y, dy, dx, rows, cols, dt, stream);
}

extern "C" tf_status tf_softmax_bwd(const void* y, const void* dy, void* dx, int64_t rows, int64_t cols, tf_dtype dt, void* stream) {
    return run2<kOpSoftmaxBwd>(y, dy, dx, rows, cols, dt, stream);
}
