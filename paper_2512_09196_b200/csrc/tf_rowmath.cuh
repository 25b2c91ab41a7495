// Register-level row arithmetic shared by the variants that hold a row (or a slice) in registers:
// the per-op math on NV 16-byte vectors per thread, parameterised by how partials are reduced across
// the threads that share the row and by where the affine parameters come from.
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

// Reducers: how a per-thread partial becomes the value for everything this group holds.
template <int LANES> struct GroupRed {
    __device__ __forceinline__ float sum(float v, int) const { return group_reduce<SumOp, LANES>(v); }
    __device__ __forceinline__ float max(float v, int) const { return group_reduce<MaxOp, LANES>(v); }
};
struct CtaRed {
    float* buf;      // [4][32] floats of shared memory
    __device__ __forceinline__ float sum(float v, int slot) const { return cta_reduce<SumOp>(v, buf + 32 * slot); }
    __device__ __forceinline__ float max(float v, int slot) const { return cta_reduce<MaxOp>(v, buf + 32 * slot); }
};

// Parameter access: either held in registers (V_WARP) or fetched from L1/L2 when the normalise pass needs them.
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

// ---- single-group math: the group holds the entire row -----------------------------------------------
// raw[v] invalid => filled with -inf (softmax) / 0 (norms).  slot0 alternates between calls so that a CTA
// reducer never reuses a shared buffer that slow threads may still be reading.
template <int OP, int DT, int NV, class Red, class Par>
__device__ __forceinline__ void row_math(const uint4 (&raw)[NV], const bool (&valid)[NV], const Red& red, const Par& par,
                                         int slot0, float n, float eps, uint4 (&out)[NV], float& st0, float& st1) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    if constexpr (OP == OP_SOFTMAX) {
        float f[NV][NE];
        float m = kNegInf;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            E::unpack(raw[v], f[v]);
#pragma unroll
            for (int e = 0; e < NE; ++e) m = fmaxf(m, f[v][e]);
        }
        m = red.max(m, slot0);
        const float off = exp_offset(m);
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < NE; ++e) { f[v][e] = ex2_ftz(fmaf(f[v][e], kLog2e, off)); s += f[v][e]; }
        s = red.sum(s, slot0 + 1);
        const float inv = (s == 0.f) ? 0.f : 1.0f / s;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
#pragma unroll
            for (int e = 0; e < NE; ++e) f[v][e] *= inv;
            out[v] = E::pack(f[v]);
        }
    } else if constexpr (OP == OP_LAYERNORM) {
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float f[NE]; E::unpack(raw[v], f);
#pragma unroll
            for (int e = 0; e < NE; ++e) s += f[e];
        }
        const float mean = red.sum(s, slot0) / n;
        float m2 = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float f[NE]; E::unpack(raw[v], f);
            if (valid[v]) {
#pragma unroll
                for (int e = 0; e < NE; ++e) { const float d = f[e] - mean; m2 = fmaf(d, d, m2); }
            }
        }
        const float var = red.sum(m2, slot0 + 1) / n;
        const float rstd = 1.0f / sqrtf(var + eps);
        st0 = mean; st1 = rstd;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float f[NE], g[NE], b[NE];
            E::unpack(raw[v], f);
            if (valid[v]) { E::unpack(par.gamma(v), g); E::unpack(par.beta(v), b); }
#pragma unroll
            for (int e = 0; e < NE; ++e) f[e] = valid[v] ? fmaf((f[e] - mean) * rstd, g[e], b[e]) : 0.f;
            out[v] = E::pack(f);
        }
    } else {
        float ss = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float f[NE]; E::unpack(raw[v], f);
#pragma unroll
            for (int e = 0; e < NE; ++e) ss = fmaf(f[e], f[e], ss);
        }
        const float rr = 1.0f / sqrtf(red.sum(ss, slot0) / n + eps);
        st0 = rr; st1 = rr;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            float f[NE], w[NE];
            E::unpack(raw[v], f);
            if (valid[v]) E::unpack(par.gamma(v), w);
#pragma unroll
            for (int e = 0; e < NE; ++e) f[e] = valid[v] ? (f[e] * rr) * w[e] : 0.f;
            out[v] = E::pack(f);
        }
    }
}

}  // namespace tf
