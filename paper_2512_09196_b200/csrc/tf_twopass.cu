// V_TWOPASS: long rows of any length, streamed twice with 16-byte vector loads.
//
// A CTA owns a row.  Pass A streams the row from HBM and keeps only per-thread running statistics in
// registers -- (max offset, sum) rescaled online for softmax, (n, mean, M2) merged chunk by chunk with Chan's
// update for LayerNorm, the sum of squares for RMSNorm -- so no cross-thread communication happens inside the
// row; one CTA-wide merge follows.  Pass B streams the row again, this time from L2 (a row is at most a few
// MiB and was just read; the loads of pass A carry an L2 evict-last policy, those of pass B an
// evict-first one), normalises and writes y with streaming stores.  HBM still sees x once and y once.
// There is no shared-memory staging, no cluster and no limit on the row length; many resident CTAs with
// several independent loads per thread keep the memory system busy.
#include <algorithm>

#include "tf_rowmath.cuh"

namespace tf {
namespace {

struct WArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t rows;
    int64_t nvec;
    float n, eps;
};

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

constexpr int kTwoU = 4;             // independent 16-byte loads per thread per step

template <int OP, int DT>
__global__ void __launch_bounds__(1024) k_twopass(const WArgs a) {
    using E = Elem<DT>;
    using P = Pairs<DT>;
    constexpr int NE = E::NE, NP = P::NP, U = kTwoU;
    __shared__ float red_buf[4 * 32];
    pdl_wait();
    pdl_trigger();
    const int T = blockDim.x, t = threadIdx.x;
    const uint4 fill = fill_vec<DT>(OP);
    const F2 l2e = f2(kLog2e);
    const uint64_t keep = policy_evict_last(), last = policy_evict_first();     // pass A keeps x in L2, pass B lets it go

    int it = 0;
    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x, ++it) {
        const uint4* xr = a.x + row * a.nvec;
        uint4* yr = a.y + row * a.nvec;
        float* rb = red_buf + 64 * (it & 1);
        // ---------------- pass A: per-thread running statistics ----------------
        float s_off = 0.f, s_sum = 0.f, s_max = kNegInf;      // softmax: offset of the running max, sum at that offset
        float c_n = 0.f, c_mean = 0.f, c_m2 = 0.f;            // LayerNorm
        F2 q2 = f2(0.f);                                      // RMSNorm
        for (int64_t base = t; base < a.nvec; base += static_cast<int64_t>(T) * U) {
            uint4 raw[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                ok[u] = base + static_cast<int64_t>(u) * T < a.nvec;
                raw[u] = ok[u] ? ld_hint(xr + base + static_cast<int64_t>(u) * T, keep) : fill;
            }
            if constexpr (OP == OP_SOFTMAX) {
                float cm = kNegInf;
#pragma unroll
                for (int u = 0; u < U; ++u) cm = fmaxf(cm, vec_max<DT>(raw[u]));
                if (cm > s_max) {                             // new running max: move the sum to its offset
                    const float noff = exp_offset(cm);
                    s_sum = (s_max == kNegInf) ? 0.f : s_sum * ex2_ftz(noff - s_off);
                    s_off = noff; s_max = cm;
                }
                const F2 off = f2(s_off);
                F2 acc = f2(0.f);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (!all_neg_inf_vec<DT>(raw[u])) {
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
                    P::unpack(raw[u], w[u]);
                    cnt += ok[u] ? NE : 0;
#pragma unroll
                    for (int i = 0; i < NP; ++i) s2 = add2(s2, w[u][i]);
                }
                const float nc = static_cast<float>(cnt);
                const float mc = fast_div(hsum(s2), nc);                // cnt > 0: base < nvec
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
        // ---------------- CTA-wide merge ----------------
        float ta, tb;
        if constexpr (OP == OP_SOFTMAX) {
            const float M = cta_reduce<MaxOp>(s_max, rb);
            const float O = exp_offset(M);
            const float mine = (s_max == kNegInf) ? 0.f : s_sum * ex2(O - s_off);       // O <= s_off: factor <= 1
            const float S = cta_reduce<SumOp>(mine, rb + 32);
            ta = O; tb = (S == 0.f) ? 0.f : fast_rcp(S);
        } else if constexpr (OP == OP_LAYERNORM) {
            const float mean = fast_div(cta_reduce<SumOp>(c_n * c_mean, rb), a.n);
            const float d = c_mean - mean;
            const float m2 = cta_reduce<SumOp>(fmaf(c_n * d, d, c_m2), rb + 32);          // sum of M2_t + n_t (mean_t - mean)^2
            ta = mean; tb = fast_rsqrt(fast_div(m2, a.n) + a.eps);
        } else {
            const float tot = cta_reduce<SumOp>(hsum(q2), rb);
            ta = tb = fast_rsqrt(fast_div(tot, a.n) + a.eps);
        }
        if (t == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = ta;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = tb;
        }
        // ---------------- pass B: normalise from L2, store ----------------
        const F2 ta2 = f2(ta), tb2 = f2(tb);
        for (int64_t base = t; base < a.nvec; base += static_cast<int64_t>(T) * U) {
            uint4 raw[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                ok[u] = base + static_cast<int64_t>(u) * T < a.nvec;
                raw[u] = ok[u] ? ld_hint(xr + base + static_cast<int64_t>(u) * T, last) : fill;
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (!ok[u]) continue;
                const int64_t idx = base + static_cast<int64_t>(u) * T;
                F2 w[NP];
                uint4 out = make_uint4(0, 0, 0, 0);
                if constexpr (OP == OP_SOFTMAX) {
                    if (!all_neg_inf_vec<DT>(raw[u]) && tb != 0.f) {
                        P::unpack(raw[u], w);
#pragma unroll
                        for (int i = 0; i < NP; ++i) w[i] = mul2(ex2_ftz2(fma2(w[i], l2e, ta2)), tb2);
                        out = P::pack(w);
                    }
                } else if constexpr (OP == OP_LAYERNORM) {
                    F2 g[NP], b[NP];
                    P::unpack(raw[u], w);
                    P::unpack(ld_param(a.p0 + idx), g);
                    P::unpack(ld_param(a.p1 + idx), b);
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[i] = fma2(mul2(sub2(w[i], ta2), tb2), g[i], b[i]);
                    out = P::pack(w);
                } else {
                    F2 g[NP];
                    P::unpack(raw[u], w);
                    P::unpack(ld_param(a.p0 + idx), g);
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[i] = mul2(mul2(w[i], ta2), g[i]);
                    out = P::pack(w);
                }
                st_stream(yr + idx, out);
            }
        }
    }
}

using TwoFn = void (*)(const WArgs);

TwoFn two_fn(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_twopass<OP_SOFTMAX, DT_F32>;
        case 1: return k_twopass<OP_SOFTMAX, DT_BF16>;
        case 2: return k_twopass<OP_LAYERNORM, DT_F32>;
        case 3: return k_twopass<OP_LAYERNORM, DT_BF16>;
        case 4: return k_twopass<OP_RMSNORM, DT_F32>;
        case 5: return k_twopass<OP_RMSNORM, DT_BF16>;
    }
    return nullptr;
}

}  // namespace

bool supports_twopass(const Plan& p, const Args& a, const DeviceInfo&) {
    return vector_ok(a) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0;
}

cudaError_t launch_twopass(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    TwoFn fn = two_fn(a.op, a.dt);
    if (!fn) return cudaErrorInvalidValue;
    int64_t grid = a.rows;
    if (p.persist > 0) grid = std::min<int64_t>(grid, static_cast<int64_t>(p.persist) * d.sms);
    grid = std::min<int64_t>(grid, 0x7FFFFFFF);
    WArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = a.cols * elem_size(a.dt) / 16;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(p.threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
