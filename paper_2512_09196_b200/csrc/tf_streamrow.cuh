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
__device__ __forceinline__ uint64_t policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
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

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {       // NaNs are ignored, as by fmaxf
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// Per-thread running statistics over the vectors a thread meets while streaming a segment.
//   softmax   (offset of the running max, packed pair of sums at that offset), rescaled online when the max grows
//   LayerNorm (n, mean, M2): each step's exact two-pass statistics merged with Chan's update
//   RMSNorm   sum of squares
// A thread's vectors are numbered by SLOT = step * U_ + u (U_ vectors per step) in row order.
template <int OP, int DT, int U_ = kStreamU> struct Running {
    float s_off = 0.f, s_max = kNegInf;
    F2 s_sum2 = f2(0.f);
    float c_n = 0.f, c_mean = 0.f, c_m2 = 0.f;
    F2 q2 = f2(0.f);
    int live_slots = 0;              // softmax: one past the last slot of the last STEP of this thread that held anything but -inf

    // raw: the step's vectors, absent ones already replaced by the fill value (-inf for softmax, 0 for the norms);
    // PRED: some may be absent, ok[] says which exist; count: elements that exist (LayerNorm's divisor); slot0: slot of raw[0].
    template <bool PRED>
    __device__ __forceinline__ void update(const uint4 (&raw)[U_], const bool (&ok)[U_], int count, int slot0) {
        using P = Pairs<DT>;
        constexpr int NP = P::NP, U = U_;
        if constexpr (OP == OP_SOFTMAX) {
            // maximum of the step, on the packed values; a step of nothing but -inf is skipped as a whole (no exponentials,
            // one test per step instead of one per vector: masks are runs, so mixed steps are rare, and the -inf elements
            // of a mixed step contribute exact zeros)
            float cm;
            if constexpr (DT == DT_BF16) {
                uint32_t pa = bf16x2_max(bf16x2_max(raw[0].x, raw[0].y), bf16x2_max(raw[0].z, raw[0].w));
#pragma unroll
                for (int u = 1; u < U; ++u) pa = bf16x2_max(pa, bf16x2_max(bf16x2_max(raw[u].x, raw[u].y), bf16x2_max(raw[u].z, raw[u].w)));
                cm = fmaxf(__uint_as_float(pa << 16), __uint_as_float(pa & 0xFFFF0000u));
            } else {
                cm = vec_max<DT>(raw[0]);
#pragma unroll
                for (int u = 1; u < U; ++u) cm = fmaxf(cm, vec_max<DT>(raw[u]));
            }
            if (cm != kNegInf) {
                if (cm > s_max) {                                                 // new running max: move the sums to its offset
                    const float noff = exp_offset(cm);
                    s_sum2 = (s_max == kNegInf) ? f2(0.f) : mul2(s_sum2, f2(ex2_ftz(noff - s_off)));
                    s_off = noff; s_max = cm;
                }
                const F2 off = f2(s_off), l2e = f2(kLog2e);
                F2 acc[U];                                                        // independent chains: the exponentials overlap
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    F2 w[NP]; P::unpack(raw[u], w);
                    acc[u] = ex2_ftz2(fma2(w[0], l2e, off));
#pragma unroll
                    for (int i = 1; i < NP; ++i) acc[u] = add2(acc[u], ex2_ftz2(fma2(w[i], l2e, off)));
                }
#pragma unroll
                for (int u = 0; u < U; ++u) s_sum2 = add2(s_sum2, acc[u]);
                live_slots = max(live_slots, slot0 + U);                          // pass A may walk the row in either direction
            }
        } else if constexpr (OP == OP_LAYERNORM) {
            F2 w[U][NP];
            F2 s2 = f2(0.f);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                P::unpack(raw[u], w[u]);
#pragma unroll
                for (int i = 0; i < NP; ++i) s2 = add2(s2, w[u][i]);
            }
            const float nc = static_cast<float>(count);                           // > 0: a step has at least one vector
            const float mc = fast_div(hsum(s2), nc);
            const F2 mc2 = f2(mc);
            F2 d2 = f2(0.f);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (!PRED || ok[u]) {
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

// Pass A over `nvec` vectors starting at xs (all threads of the CTA take part).  Whole steps (every thread has all of its
// kStreamU vectors) run without predicates; one ragged step follows where the row does not end on a step.
// CACHE: the first `cache_vecs` vectors are also parked in shared memory (`cache`), each by the thread that will want it
// back in pass B -- the same thread meets the same vectors in both passes, so no barrier is needed between them.
// LEN (softmax with a valid length `len`, in elements): only the first ceil(len / NE) vectors are read and the one that
// straddles the length has its tail replaced by -inf.
template <int OP, int DT, bool LEN = false, bool CACHE = false>
__device__ __forceinline__ Running<OP, DT> stream_stats(const uint4* xs, int64_t nvec, uint64_t policy, uint4* cache = nullptr,
                                                        int64_t cache_vecs = 0, int64_t len = -1) {
    constexpr int U = kStreamU, NE = Elem<DT>::NE;
    const int T = blockDim.x, t = threadIdx.x;
    Running<OP, DT> run;
    int64_t straddle = -1;
    if constexpr (LEN) {
        nvec = (len + NE - 1) / NE;
        if (len % NE) straddle = nvec - 1;
    }
    const int64_t step = static_cast<int64_t>(T) * U;
    // the straddling vector is the last one: it is left to the ragged step
    const int nfull = static_cast<int>((nvec - (LEN && straddle >= 0 ? 1 : 0)) / step);
    const uint4* p = xs + t;
    for (int s = 0; s < nfull; ++s, p += step) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = ld_hint(p + u * T, policy);
        if constexpr (CACHE) {
            const int64_t idx0 = s * step + t;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (idx0 + u * T < cache_vecs) cache[idx0 + u * T] = raw[u];          // cache_vecs <= nvec
        }
        const bool all[U] = {true, true, true, true};
        run.template update<false>(raw, all, U * NE, s * U);
    }
    const int64_t base = nfull * step + t;
    if (base < nvec) {                                                               // the ragged step
        const uint4 fill = fill_vec<DT>(OP);
        uint4 raw[U];
        bool ok[U];
        int count = 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t idx = base + static_cast<int64_t>(u) * T;
            ok[u] = idx < nvec;
            raw[u] = ok[u] ? ld_hint(xs + idx, policy) : fill;
            count += ok[u] ? NE : 0;
            if (LEN && idx == straddle) raw[u] = mask_tail<DT>(raw[u], static_cast<int>(len % NE));
            if (CACHE && idx < cache_vecs) cache[idx] = raw[u];
        }
        run.template update<true>(raw, ok, count, nfull * U);
    }
    return run;
}

// CTA-wide merge of the threads' running statistics into the segment's partial (every thread gets it):
// softmax (offset of the segment max, or +inf for an all -inf segment; sum at that offset),
// LayerNorm (segment mean, segment M2) for `count` elements, RMSNorm (sum of squares, 0).
// rb: 64 floats of shared memory not used by the previous merge of this CTA.
template <int OP, int DT, int U_ = kStreamU>
__device__ __forceinline__ Part merge_running(const Running<OP, DT, U_>& run, float count, float* rb) {
    if constexpr (OP == OP_SOFTMAX) {
        const float M = cta_reduce<MaxOp>(run.s_max, rb);
        const float O = exp_offset(M);
        const float mine = (run.s_max == kNegInf) ? 0.f : hsum(run.s_sum2) * ex2(O - run.s_off);       // O <= s_off: factor <= 1
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

__device__ __forceinline__ float ta2_lo(F2 a) { float lo, hi; split(a, lo, hi); return lo; }

// The normalised form of one vector: softmax 2^(x log2e + O) / S (ta2 = O, tb2 = 1/S; -inf elements need no test:
// 2^(-inf) is +0, and +0 times 1/S is +0), LayerNorm (x - mean) rstd gamma + beta, RMSNorm x rrms w.
// g, b: the parameter vectors of this column (read only for the norms).
// SMEM: g and b point into shared memory (parameters staged there by the caller), else into global memory.
template <int OP, int DT, bool SMEM = false>
__device__ __forceinline__ uint4 apply_vec(const uint4& raw, const uint4* g, const uint4* b, const F2 ta2, const F2 tb2) {
    using P = Pairs<DT>;
    constexpr int NP = P::NP;
    F2 w[NP];
    P::unpack(raw, w);
    if constexpr (OP == OP_SOFTMAX) {
        const F2 l2e = f2(kLog2e);
#pragma unroll
        for (int i = 0; i < NP; ++i) w[i] = mul2(ex2_ftz2(fma2(w[i], l2e, ta2)), tb2);
    } else if constexpr (OP == OP_LAYERNORM) {
        // (x - mean) rstd gamma + beta as two fused multiply-adds: x rstd + (-mean rstd), then times gamma plus beta
        F2 gg[NP], bb[NP];
        P::unpack(SMEM ? *g : ld_param(g), gg);
        P::unpack(SMEM ? *b : ld_param(b), bb);
        const F2 nmr2 = f2(-ta2_lo(ta2) * ta2_lo(tb2));
#pragma unroll
        for (int i = 0; i < NP; ++i) w[i] = fma2(fma2(w[i], tb2, nmr2), gg[i], bb[i]);
    } else {
        F2 gg[NP];
        P::unpack(SMEM ? *g : ld_param(g), gg);
#pragma unroll
        for (int i = 0; i < NP; ++i) w[i] = mul2(mul2(w[i], ta2), gg[i]);
    }
    return P::pack(w);
}

// One step of pass B: kStreamU vectors of this thread starting at vector idx0 (stride T).  PRED: vectors at or beyond
// nvec do not exist.  live[u] (softmax): the vector may hold something other than -inf; the others become zeros unread.
// nlive (LEN): vectors from there on lie behind the row's length: never read, always zeros.
template <int OP, int DT, bool PRED, bool LEN, bool CACHE>
__device__ __forceinline__ void apply_step(const uint4* xs, uint4* ys, const uint4* g, const uint4* b, int64_t idx0, int T, int64_t nvec,
                                           const F2 ta2, const F2 tb2, uint64_t policy, const uint4* cache, int64_t cache_vecs,
                                           const bool (&live)[kStreamU], int64_t straddle, int keep, int64_t nlive) {
    constexpr int U = kStreamU;
    uint4 raw[U];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int64_t idx = idx0 + static_cast<int64_t>(u) * T;
        ok[u] = !PRED || idx < nvec;
        const bool want = ok[u] && (OP != OP_SOFTMAX || (live[u] && (!LEN || idx < nlive)));
        if (want) raw[u] = (CACHE && idx < cache_vecs) ? cache[idx] : ld_hint(xs + idx, policy);
        else raw[u] = fill_vec<DT>(OP);
        if (LEN && idx == straddle) raw[u] = mask_tail<DT>(raw[u], keep);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        const int64_t idx = idx0 + static_cast<int64_t>(u) * T;
        uint4 out = make_uint4(0, 0, 0, 0);
        if (OP != OP_SOFTMAX || (live[u] && (!LEN || idx < nlive))) out = apply_vec<OP, DT>(raw[u], g + idx, b + idx, ta2, tb2);
        st_stream(ys + idx, out);
    }
}

// Pass B over `nvec` vectors: xs/ys point at the segment, g/b at the parameters of its first column.
// live_slots: this thread's Running::live_slots when the same thread ran pass A over the same vectors (softmax): its
// vectors from that slot on are known to be all -inf, so their zeros are written without reading x again.
// A fully masked row (1/S = 0) passes live_slots = 0.
template <int OP, int DT, bool LEN = false, bool CACHE = false>
__device__ __forceinline__ void stream_apply(const uint4* xs, uint4* ys, const uint4* g, const uint4* b, int64_t nvec,
                                             const RowScale& sc, uint64_t policy, const uint4* cache = nullptr,
                                             int64_t cache_vecs = 0, int live_slots = 0x7FFFFFFF, int64_t len = -1) {
    constexpr int U = kStreamU, NE = Elem<DT>::NE;
    const int64_t straddle = (LEN && len % NE) ? len / NE : -1;           // live_slots already ends at ceil(len / NE)
    const int keep = LEN ? static_cast<int>(len % NE) : 0;
    const int64_t nlive = LEN ? (len + NE - 1) / NE : nvec;
    const int T = blockDim.x, t = threadIdx.x;
    const F2 ta2 = f2(sc.a), tb2 = f2(sc.b);
    // back to front: the end of the segment is what pass A touched last, hence what L2 most likely still holds
    const int64_t step = static_cast<int64_t>(T) * U;
    const int nfull = static_cast<int>(nvec / step);
    if (nfull * step + t < nvec) {                                        // the ragged step
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; ++u) live[u] = nfull * U + u < live_slots;
        apply_step<OP, DT, true, LEN, CACHE>(xs, ys, g, b, nfull * step + t, T, nvec, ta2, tb2, policy, cache, cache_vecs, live, straddle, keep, nlive);
    }
    for (int s = nfull - 1; s >= 0; --s) {
        const int64_t idx0 = s * step + t;
        if (OP == OP_SOFTMAX && s * U >= live_slots) {                    // nothing but -inf here: zeros, x is not read again
#pragma unroll
            for (int u = 0; u < U; ++u) st_stream(ys + idx0 + u * T, make_uint4(0, 0, 0, 0));
            continue;
        }
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; ++u) live[u] = s * U + u < live_slots;
        apply_step<OP, DT, false, LEN, CACHE>(xs, ys, g, b, idx0, T, nvec, ta2, tb2, policy, cache, cache_vecs, live, straddle, keep, nlive);
    }
}

}  // namespace tf
