// Register-level row arithmetic shared by the variants that hold a row (or a slice of one) in registers:
// the per-op math on NV 16-byte vectors per thread, written on packed fp32 pairs, parameterised by how
// partials are reduced across the threads that share the data and by where the affine parameters come from.
#pragma once

#include "tf_common.cuh"

namespace tf {

template <int DT> __device__ __forceinline__ uint4 fill_vec(int op) {
    if (op == OP_SOFTMAX) {
        const uint32_t w = (DT == DT_F32) ? 0xFF800000u : 0xFF80FF80u;     // -inf in every element
        return make_uint4(w, w, w, w);
    }
    return make_uint4(0, 0, 0, 0);
}

// Reducers: how a per-thread partial becomes the value for everything the group holds.
template <int LANES> struct GroupRed {
    __device__ __forceinline__ float sum(float v, int) const { return group_reduce<SumOp, LANES>(v); }
    __device__ __forceinline__ float max(float v, int) const { return group_reduce<MaxOp, LANES>(v); }
};
struct CtaRed {
    float* buf;      // [4][32] floats of shared memory
    __device__ __forceinline__ float sum(float v, int slot) const { return cta_reduce<SumOp>(v, buf + 32 * slot); }
    __device__ __forceinline__ float max(float v, int slot) const { return cta_reduce<MaxOp>(v, buf + 32 * slot); }
};

// Parameter access: held in registers, or fetched (L1/L2 or shared memory) when the normalise pass needs them.
template <int NV> struct HeldParams {
    uint4 g[NV], b[NV];
    __device__ __forceinline__ uint4 gamma(int v) const { return g[v]; }
    __device__ __forceinline__ uint4 beta(int v) const { return b[v]; }
};
struct LazyParams {
    const uint4* p0;
    const uint4* p1;
    int first, stride;
    __device__ __forceinline__ uint4 gamma(int v) const { return ld_param(p0 + first + v * stride); }
    __device__ __forceinline__ uint4 beta(int v) const { return ld_param(p1 + first + v * stride); }
};

// Parameters of a persistent thread's own columns, widened to fp32 pairs once and kept in registers (worth it where a
// thread owns one or two vectors per row: a 2-byte gamma / beta then costs neither a load nor a widening per row).
template <int DT, int NV> struct HeldWideParams {
    F2 g[NV][Pairs<DT>::NP], b[NV][Pairs<DT>::NP];
};

// gamma / beta of vector v as fp32 pairs, whatever the provider keeps them as.
template <int DT, class Par>
__device__ __forceinline__ void load_gamma(const Par& par, int v, F2 (&g)[Pairs<DT>::NP]) { Pairs<DT>::unpack(par.gamma(v), g); }
template <int DT, class Par>
__device__ __forceinline__ void load_beta(const Par& par, int v, F2 (&b)[Pairs<DT>::NP]) { Pairs<DT>::unpack(par.beta(v), b); }
template <int DT, int NV>
__device__ __forceinline__ void load_gamma(const HeldWideParams<DT, NV>& par, int v, F2 (&g)[Pairs<DT>::NP]) {
#pragma unroll
    for (int i = 0; i < Pairs<DT>::NP; ++i) g[i] = par.g[v][i];
}
template <int DT, int NV>
__device__ __forceinline__ void load_beta(const HeldWideParams<DT, NV>& par, int v, F2 (&b)[Pairs<DT>::NP]) {
#pragma unroll
    for (int i = 0; i < Pairs<DT>::NP; ++i) b[i] = par.b[v][i];
}

// Keeps the first `keep` (1 .. NE-1) elements of a vector and replaces the rest by -inf.
template <int DT> __device__ __forceinline__ uint4 mask_tail(const uint4& v, int keep) {
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) if (i >= keep) w[i] = 0xFF800000u;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (2 * i >= keep) w[i] = (w[i] & 0xFFFF0000u) | 0x0000FF80u;
            if (2 * i + 1 >= keep) w[i] = (w[i] & 0x0000FFFFu) | 0xFF800000u;
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Parameters copied once into shared memory by the thread that will use them (a persistent CTA always owns the same
// columns): no barrier is needed between the copy and the reads.
struct OwnedSmemParams {
    const uint4* g;
    const uint4* b;
    int first, stride;
    __device__ __forceinline__ uint4 gamma(int v) const { return g[first + v * stride]; }
    __device__ __forceinline__ uint4 beta(int v) const { return b[first + v * stride]; }
};

// ---- slice math ---------------------------------------------------------------------------------------
// A group holds one SLICE of a row (possibly the whole row) as NV vectors per thread; invalid vectors are
// filled with -inf (softmax) / 0 (norms).  Inside the slice the statistics are exact two-pass ones.  Slices
// of one row that live in groups which cannot shuffle with one another (the warps of a multi-warp unit, the
// CTAs of a cluster) are merged afterwards: (offset, sum) for softmax, (mean, M2) with Chan's update for
// LayerNorm, the plain sum of squares for RMSNorm.
struct Part { float a, b; };
struct Total { float a, b; };        // softmax: (rescale of my slice, 1/S); LayerNorm: (mean, rstd); RMSNorm: (rrms, rrms)

// `slot0` picks the reducer's shared buffers (CTA reducers alternate them between rows).  `w` receives the
// widened values (softmax: the exponentials) for slice_finish.
// ALLV: every vector of every thread is valid (the row fills the group exactly), so no predicate is needed.
template <int OP, int DT, int NV, class Red, bool ALLV = false>
__device__ __forceinline__ Part slice_stats(const uint4 (&raw)[NV], const bool (&valid)[NV], const Red& red, int slot0,
                                            float n_slice, F2 (&w)[NV][Pairs<DT>::NP]) {
    using P = Pairs<DT>;
    constexpr int NP = P::NP;
    if constexpr (OP == OP_SOFTMAX) {
        // vectors that are absent (or, with a row length, entirely behind it) hold -inf and contribute exact zeros: their
        // exponentials are not evaluated
        float m = kNegInf;
#pragma unroll
        for (int v = 0; v < NV; ++v)
            if (ALLV || valid[v]) m = fmaxf(m, vec_max<DT>(raw[v]));
        m = red.max(m, slot0);
        const F2 off = f2(exp_offset(m)), l2e = f2(kLog2e);
        F2 s = f2(0.f);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (ALLV || valid[v]) {
                P::unpack(raw[v], w[v]);
#pragma unroll
                for (int i = 0; i < NP; ++i) { w[v][i] = ex2_ftz2(fma2(w[v][i], l2e, off)); s = add2(s, w[v][i]); }
            } else {
#pragma unroll
                for (int i = 0; i < NP; ++i) w[v][i] = f2(0.f);
            }
        }
        return Part{(m == kNegInf) ? -kNegInf : exp_offset(m), red.sum(hsum(s), slot0 + 1)};
    } else if constexpr (OP == OP_LAYERNORM) {
        F2 s = f2(0.f);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            P::unpack(raw[v], w[v]);
#pragma unroll
            for (int i = 0; i < NP; ++i) s = add2(s, w[v][i]);
        }
        const float tot = red.sum(hsum(s), slot0);
        const float mean = (n_slice > 0.f) ? fast_div(tot, n_slice) : 0.f;
        const F2 mm = f2(mean);
        F2 m2 = f2(0.f);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (ALLV || valid[v]) {
#pragma unroll
                for (int i = 0; i < NP; ++i) { const F2 d = sub2(w[v][i], mm); m2 = fma2(d, d, m2); }
            }
        }
        return Part{mean, red.sum(hsum(m2), slot0 + 1)};
    } else {
        F2 ss = f2(0.f);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            P::unpack(raw[v], w[v]);
#pragma unroll
            for (int i = 0; i < NP; ++i) ss = fma2(w[v][i], w[v][i], ss);
        }
        return Part{red.sum(hsum(ss), slot0), 0.f};
    }
}

// Merges K slice partials (read through get(k), element counts through count(k)) in slice order, so that
// every holder of the same partials computes bit-identical totals.
template <int OP, class Get, class Count>
__device__ __forceinline__ Total combine_parts(int K, int mine, const Get& get, const Count& count, float n, float eps) {
    if constexpr (OP == OP_SOFTMAX) {
        float O = -kNegInf;
        for (int k = 0; k < K; ++k) O = fminf(O, get(k).a);
        float S = 0.f;
        for (int k = 0; k < K; ++k) { const Part p = get(k); S = fmaf(p.b, softmax_rescale(O, p.a), S); }
        return Total{softmax_rescale(O, get(mine).a), (S == 0.f) ? 0.f : fast_rcp(S)};
    } else if constexpr (OP == OP_LAYERNORM) {
        MomentPartial acc{0.f, 0.f, 0.f};
        for (int k = 0; k < K; ++k) { const Part p = get(k); acc = chan_combine(acc, MomentPartial{count(k), p.a, p.b}); }
        return Total{acc.mean, fast_rsqrt(fast_div(acc.m2, n) + eps)};
    } else {
        float tot = 0.f;
        for (int k = 0; k < K; ++k) tot += get(k).a;
        const float rr = fast_rsqrt(fast_div(tot, n) + eps);
        return Total{rr, rr};
    }
}

// The single-slice case of combine_parts (the group holds the whole row).
template <int OP>
__device__ __forceinline__ Total total_of(const Part& p, float n, float eps) {
    if constexpr (OP == OP_SOFTMAX) return Total{1.0f, (p.b == 0.f) ? 0.f : fast_rcp(p.b)};
    else if constexpr (OP == OP_LAYERNORM) return Total{p.a, fast_rsqrt(fast_div(p.b, n) + eps)};
    else { const float rr = fast_rsqrt(fast_div(p.a, n) + eps); return Total{rr, rr}; }
}

// Normalises R rows that share this thread's columns: the parameters of a vector are fetched and widened once
// and applied to every row.  SINGLE: the slice is the whole row, so softmax needs no slice rescale.
template <int OP, int DT, int NV, int R, bool SINGLE, bool ALLV, class Par>
__device__ __forceinline__ void slice_finish_rows(const bool (&valid)[NV], F2 (&w)[R][NV][Pairs<DT>::NP], const Total (&t)[R],
                                                  const Par& par, uint4 (&out)[R][NV]) {
    using P = Pairs<DT>;
    constexpr int NP = P::NP;
    F2 ta[R], tb[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        // LayerNorm: (x - mean) rstd gamma + beta as two fused multiply-adds, x rstd + (-mean rstd) first: ta holds -mean rstd
        ta[r] = f2(OP == OP_LAYERNORM ? -t[r].a * t[r].b : t[r].a);
        tb[r] = f2(t[r].b);
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        if constexpr (OP == OP_SOFTMAX) {
            // two factors when slices are merged: the slice rescale may be subnormal (a slice far below the row
            // maximum) while 1/S carries 2^-bias; their product could lose the subnormal bits.
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (ALLV || valid[v]) {
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[r][v][i] = SINGLE ? mul2(w[r][v][i], tb[r]) : mul2(mul2(w[r][v][i], ta[r]), tb[r]);
                    out[r][v] = P::pack(w[r][v]);
                } else {
                    out[r][v] = make_uint4(0, 0, 0, 0);               // +0 in either element type
                }
            }
        } else if constexpr (OP == OP_LAYERNORM) {
            if (ALLV || valid[v]) {
                F2 g[NP], b[NP];
                load_gamma<DT>(par, v, g);
                load_beta<DT>(par, v, b);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[r][v][i] = fma2(fma2(w[r][v][i], tb[r], ta[r]), g[i], b[i]);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) out[r][v] = P::pack(w[r][v]);
        } else {
            if (ALLV || valid[v]) {
                F2 g[NP];
                load_gamma<DT>(par, v, g);
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[r][v][i] = mul2(mul2(w[r][v][i], ta[r]), g[i]);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) out[r][v] = P::pack(w[r][v]);
        }
    }
}

template <int OP, int DT, int NV, bool SINGLE, class Par>
__device__ __forceinline__ void slice_finish(const bool (&valid)[NV], F2 (&w)[NV][Pairs<DT>::NP], const Total& t, const Par& par,
                                             uint4 (&out)[NV]) {
    slice_finish_rows<OP, DT, NV, 1, SINGLE, false>(valid, reinterpret_cast<F2 (&)[1][NV][Pairs<DT>::NP]>(w),
                                                    reinterpret_cast<const Total (&)[1]>(t), par, reinterpret_cast<uint4 (&)[1][NV]>(out));
}

// Whole row in one group: statistics, totals and outputs in one call.  st0/st1: mean & rstd (LayerNorm), rrms (RMSNorm).
template <int OP, int DT, int NV, class Red, class Par>
__device__ __forceinline__ void row_math(const uint4 (&raw)[NV], const bool (&valid)[NV], const Red& red, const Par& par,
                                         int slot0, float n, float eps, uint4 (&out)[NV], float& st0, float& st1) {
    F2 w[NV][Pairs<DT>::NP];
    const Part part = slice_stats<OP, DT, NV>(raw, valid, red, slot0, n, w);
    const Total t = total_of<OP>(part, n, eps);
    st0 = t.a; st1 = t.b;
    slice_finish<OP, DT, NV, true>(valid, w, t, par, out);
}

}  // namespace tf
