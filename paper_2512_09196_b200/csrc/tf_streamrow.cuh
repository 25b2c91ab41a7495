// Streaming a row segment straight from global memory with 16-byte loads: running per-thread statistics
// (pass A), their CTA-wide merge into a segment partial, and the normalise-and-store pass (pass B).
// Shared by V_TWOPASS (segment = whole row, one CTA per row) and V_SPLIT (a row cut into segments, one CTA
// each, partials merged through global scratch).
#pragma once

#include "tf_rowmath.cuh"

namespace tf {

// L2 cache policies for 16-byte loads (the plain eviction-priority qualifiers exist only for 32-byte loads).
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 ld_hint(const uint4* p, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
    return v;
}

template <int DT> __device__ __forceinline__ bool all_neg_inf_vec(const uint4& v) {
    const uint32_t w = (DT == DT_F32) ? 0xFF800000u : 0xFF80FF80u;
    return (v.x == w) & (v.y == w) & (v.z == w) & (v.w == w);
}

constexpr int kStreamU = 4;          // independent 16-byte loads per thread per step

// Per-thread running statistics over the vectors a thread meets while streaming a segment.
//   softmax   (offset of the running max, sum at that offset), rescaled online when the max grows
//   LayerNorm (n, mean, M2): each step's exact two-pass statistics merged with Chan's update
//   RMSNorm   sum of squares
template <int OP, int DT> struct Running {
    float s_off = 0.f, s_sum = 0.f, s_max = kNegInf;
    float c_n = 0.f, c_mean = 0.f, c_m2 = 0.f;
    F2 q2 = f2(0.f);
    int64_t live_end = 0;            // softmax: one past the last vector of THIS thread that held anything but -inf

    __device__ __forceinline__ void update(const uint4 (&raw)[kStreamU], const bool (&ok)[kStreamU]) {
        using P = Pairs<DT>;
        constexpr int NE = Elem<DT>::NE, NP = P::NP, U = kStreamU;
        if constexpr (OP == OP_SOFTMAX) {
            float cm = kNegInf;
#pragma unroll
            for (int u = 0; u < U; ++u) cm = fmaxf(cm, vec_max<DT>(raw[u]));       // absent vectors are filled with -inf
            if (cm > s_max) {                                                     // new running max: move the sum to its offset
                const float noff = exp_offset(cm);
                s_sum = (s_max == kNegInf) ? 0.f : s_sum * ex2_ftz(noff - s_off);
                s_off = noff; s_max = cm;
            }
            const F2 off = f2(s_off), l2e = f2(kLog2e);
            F2 acc = f2(0.f);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (!all_neg_inf_vec<DT>(raw[u])) {                               // masked vectors cost no exponentials
                    F2 w[NP]; P::unpack(raw[u], w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) acc = add2(acc, ex2_ftz2(fma2(w[i], l2e, off)));
                }
            }
            s_sum += hsum(acc);
        } else if constexpr (OP == OP_LAYERNORM) {
            F2 w[U][NP];
            F2 s2 = f2(0.f);
            int cnt = 0;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                P::unpack(raw[u], w[u]);                                          // absent vectors are filled with 0
                cnt += ok[u] ? NE : 0;
#pragma unroll
                for (int i = 0; i < NP; ++i) s2 = add2(s2, w[u][i]);
            }
            const float nc = static_cast<float>(cnt);
            const float mc = fast_div(hsum(s2), nc);                              // cnt > 0: a step has at least one vector
            const F2 mc2 = f2(mc);
            F2 d2 = f2(0.f);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (ok[u]) {
#pragma unroll
                    for (int i = 0; i < NP; ++i) { const F2 d = sub2(w[u][i], mc2); d2 = fma2(d, d, d2); }
                }
            }
            const MomentPartial m = chan_combine(MomentPartial{c_n, c_mean, c_m2}, MomentPartial{nc, mc, hsum(d2)});
            c_n = m.n; c_mean = m.mean; c_m2 = m.m2;
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                F2 w[NP]; P::unpack(raw[u], w);
#pragma unroll
                for (int i = 0; i < NP; ++i) q2 = fma2(w[i], w[i], q2);
            }
        }
    }
};

// Pass A over `nvec` vectors starting at xs (all threads of the CTA take part).  The first `cache_vecs` vectors
// are also parked in shared memory (`cache`), each by the thread that will want it back in pass B -- the same
// thread meets the same vectors in both passes, so no barrier is needed between them.
// len >= 0 (softmax with a valid length, in elements): only the first ceil(len / NE) vectors are read and the one that
// straddles the length has its tail replaced by -inf.
template <int OP, int DT>
__device__ __forceinline__ Running<OP, DT> stream_stats(const uint4* xs, int64_t nvec, uint64_t policy, uint4* cache = nullptr,
                                                        int64_t cache_vecs = 0, int64_t len = -1) {
    constexpr int U = kStreamU, NE = Elem<DT>::NE;
    const int T = blockDim.x, t = threadIdx.x;
    const uint4 fill = fill_vec<DT>(OP);
    Running<OP, DT> run;
    if (len >= 0) nvec = (len + NE - 1) / NE;
    const int64_t straddle = (len >= 0 && len % NE) ? nvec - 1 : -1;
    for (int64_t base = t; base < nvec; base += static_cast<int64_t>(T) * U) {
        uint4 raw[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t idx = base + static_cast<int64_t>(u) * T;
            ok[u] = idx < nvec;
            raw[u] = ok[u] ? ld_hint(xs + idx, policy) : fill;
            if (idx == straddle) raw[u] = mask_tail<DT>(raw[u], static_cast<int>(len % NE));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t idx = base + static_cast<int64_t>(u) * T;
            if (idx < cache_vecs) cache[idx] = raw[u];          // cache_vecs <= nvec
            if (OP == OP_SOFTMAX && ok[u] && !all_neg_inf_vec<DT>(raw[u])) run.live_end = idx + 1;
        }
        run.update(raw, ok);
    }
    return run;
}

// CTA-wide merge of the threads' running statistics into the segment's partial (every thread gets it):
// softmax (offset of the segment max, or +inf for an all -inf segment; sum at that offset),
// LayerNorm (segment mean, segment M2) for `count` elements, RMSNorm (sum of squares, 0).
// rb: 64 floats of shared memory not used by the previous merge of this CTA.
template <int OP, int DT>
__device__ __forceinline__ Part merge_running(const Running<OP, DT>& run, float count, float* rb) {
    if constexpr (OP == OP_SOFTMAX) {
        const float M = cta_reduce<MaxOp>(run.s_max, rb);
        const float O = exp_offset(M);
        const float mine = (run.s_max == kNegInf) ? 0.f : run.s_sum * ex2(O - run.s_off);       // O <= s_off: factor <= 1
        const float S = cta_reduce<SumOp>(mine, rb + 32);
        return Part{(M == kNegInf) ? -kNegInf : O, S};
    } else if constexpr (OP == OP_LAYERNORM) {
        const float mean = fast_div(cta_reduce<SumOp>(run.c_n * run.c_mean, rb), count);
        const float d = run.c_mean - mean;
        return Part{mean, cta_reduce<SumOp>(fmaf(run.c_n * d, d, run.c_m2), rb + 32)};           // sum of M2_t + n_t (mean_t - mean)^2
    } else {
        return Part{cta_reduce<SumOp>(hsum(run.q2), rb), 0.f};
    }
}

// What pass B needs: softmax (row offset O, 1/S); LayerNorm (mean, rstd); RMSNorm (rrms, rrms).
struct RowScale { float a, b; };

template <int OP>
__device__ __forceinline__ RowScale scale_of_row(const Part& p, float n, float eps) {       // p covers the whole row
    if constexpr (OP == OP_SOFTMAX) return RowScale{(p.a == -kNegInf) ? 0.f : p.a, (p.b == 0.f) ? 0.f : fast_rcp(p.b)};
    else if constexpr (OP == OP_LAYERNORM) return RowScale{p.a, fast_rsqrt(fast_div(p.b, n) + eps)};
    else { const float rr = fast_rsqrt(fast_div(p.a, n) + eps); return RowScale{rr, rr}; }
}

// Pass B over `nvec` vectors: xs/ys point at the segment, g/b at the parameters of its first column.
// live_end: this thread's Running::live_end when the same thread ran pass A over the same vectors (softmax): vectors
// from there on are known to be all -inf, so their zeros are written without reading x again.
template <int OP, int DT>
__device__ __forceinline__ void stream_apply(const uint4* xs, uint4* ys, const uint4* g, const uint4* b, int64_t nvec,
                                             const RowScale& sc, uint64_t policy, const uint4* cache = nullptr,
                                             int64_t cache_vecs = 0, int64_t live_end = INT64_MAX, int64_t len = -1) {
    using P = Pairs<DT>;
    constexpr int NP = P::NP, U = kStreamU, NE = Elem<DT>::NE;
    const int64_t straddle = (len >= 0 && len % NE) ? len / NE : -1;      // live_end already ends at ceil(len / NE)
    const int T = blockDim.x, t = threadIdx.x;
    const uint4 fill = fill_vec<DT>(OP);
    const F2 ta2 = f2(sc.a), tb2 = f2(sc.b), l2e = f2(kLog2e);
    // back to front: the end of the segment is what pass A touched last, hence what L2 most likely still holds
    const int64_t step = static_cast<int64_t>(T) * U;
    for (int64_t base = (nvec - 1) / step * step + t; base >= 0; base -= step) {
        uint4 raw[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t idx = base + static_cast<int64_t>(u) * T;
            ok[u] = idx < nvec;
            raw[u] = (!ok[u] || idx >= live_end) ? fill : (idx < cache_vecs ? cache[idx] : ld_hint(xs + idx, policy));
            if (idx == straddle) raw[u] = mask_tail<DT>(raw[u], static_cast<int>(len % NE));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            const int64_t idx = base + static_cast<int64_t>(u) * T;
            F2 w[NP];
            uint4 out = make_uint4(0, 0, 0, 0);
            if constexpr (OP == OP_SOFTMAX) {
                if (!all_neg_inf_vec<DT>(raw[u]) && sc.b != 0.f) {
                    P::unpack(raw[u], w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[i] = mul2(ex2_ftz2(fma2(w[i], l2e, ta2)), tb2);
                    out = P::pack(w);
                }
            } else if constexpr (OP == OP_LAYERNORM) {
                F2 gg[NP], bb[NP];
                P::unpack(raw[u], w);
                P::unpack(ld_param(g + idx), gg);
                P::unpack(ld_param(b + idx), bb);
#pragma unroll
                for (int i = 0; i < NP; ++i) w[i] = fma2(mul2(sub2(w[i], ta2), tb2), gg[i], bb[i]);
                out = P::pack(w);
            } else {
                F2 gg[NP];
                P::unpack(raw[u], w);
                P::unpack(ld_param(g + idx), gg);
#pragma unroll
                for (int i = 0; i < NP; ++i) w[i] = mul2(mul2(w[i], ta2), gg[i]);
                out = P::pack(w);
            }
            st_stream(ys + idx, out);
        }
    }
}

}  // namespace tf
