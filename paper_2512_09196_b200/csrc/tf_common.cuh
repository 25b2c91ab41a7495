// Device-side building blocks shared by the kernel files: 16-byte vector access, bf16 <-> fp32,
// the exponential used by softmax, warp and CTA reductions, and the per-op partial-combine rules.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tf_plan.h"

namespace tf {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -__builtin_huge_valf();

// ---------------------------------------------------------------------------------------------
// Element traits: a 16-byte vector holds NE elements.
// ---------------------------------------------------------------------------------------------
template <int DT> struct Elem;

template <> struct Elem<DT_F32> {
    static constexpr int NE = 4;
    static constexpr int SIZE = 4;
    using scalar = float;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[NE]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[NE]) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
    static __device__ __forceinline__ float to_float(float s) { return s; }
    static __device__ __forceinline__ float from_float(float f) { return f; }
};

template <> struct Elem<DT_BF16> {
    static constexpr int NE = 8;
    static constexpr int SIZE = 2;
    using scalar = uint16_t;
    // a bf16 is the upper half of an fp32: widening is a shift (exact)
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[NE]) {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
    }
    // round-to-nearest-even, subnormals kept (cvt.rn.bf16x2.f32)
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&p);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[NE]) {
        return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
    }
    static __device__ __forceinline__ float to_float(uint16_t s) { return __uint_as_float(static_cast<uint32_t>(s) << 16); }
    static __device__ __forceinline__ uint16_t from_float(float f) {
        __nv_bfloat16 b = __float2bfloat16_rn(f);
        return *reinterpret_cast<uint16_t*>(&b);
    }
};

// ---------------------------------------------------------------------------------------------
// Packed pairs of fp32 (Blackwell's .f32x2 arithmetic: one instruction, two IEEE results, no flushing).
// The row arithmetic below is written on pairs, which halves its FP instruction count.
// ---------------------------------------------------------------------------------------------
struct F2 { unsigned long long v; };
__device__ __forceinline__ F2 f2(float lo, float hi) { F2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ F2 f2(float both) { return f2(both, both); }
__device__ __forceinline__ void split(F2 a, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v)); }
__device__ __forceinline__ float hsum(F2 a) { float lo, hi; split(a, lo, hi); return lo + hi; }
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) { F2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r; }
__device__ __forceinline__ F2 add2(F2 a, F2 b) { F2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ F2 sub2(F2 a, F2 b) { F2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ F2 mul2(F2 a, F2 b) { F2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }

// A 16-byte vector as NP pairs.
template <int DT> struct Pairs;
template <> struct Pairs<DT_F32> {
    static constexpr int NP = 2;
    static __device__ __forceinline__ void unpack(const uint4& v, F2 (&p)[NP]) {
        p[0] = f2(__uint_as_float(v.x), __uint_as_float(v.y));
        p[1] = f2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
    static __device__ __forceinline__ uint4 pack(const F2 (&p)[NP]) {
        float a, b, c, d;
        split(p[0], a, b); split(p[1], c, d);
        return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
    }
};
template <> struct Pairs<DT_BF16> {
    static constexpr int NP = 4;
    static __device__ __forceinline__ F2 widen(uint32_t w) { return f2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)); }
    static __device__ __forceinline__ void unpack(const uint4& v, F2 (&p)[NP]) {
        p[0] = widen(v.x); p[1] = widen(v.y); p[2] = widen(v.z); p[3] = widen(v.w);
    }
    static __device__ __forceinline__ uint32_t narrow(F2 a) { float lo, hi; split(a, lo, hi); return Elem<DT_BF16>::pack2(lo, hi); }
    static __device__ __forceinline__ uint4 pack(const F2 (&p)[NP]) {
        return make_uint4(narrow(p[0]), narrow(p[1]), narrow(p[2]), narrow(p[3]));
    }
};

// ---------------------------------------------------------------------------------------------
// Global memory access.  x is read once and y written once: both bypass L1 allocation / are marked
// streaming so that they do not push the (re-read) parameter vectors out of the caches.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_param(const uint4* p) { return __ldg(p); }

// 2^t with subnormal results kept (no .ftz): ex2.approx.f32, relative error about 2^-22.  Used once per row.
__device__ __forceinline__ float ex2(float t) {
    float r;
    asm("ex2.approx.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}
// 2^t as a single MUFU operation; results below 2^-126 are flushed to zero.  The softmax paths use it
// per element on exponents that carry a bias of +kExpBias (folded into the constant of the FMA that forms
// the exponent): the largest term is then 2^64, a term is only flushed when its true value is below
// 2^-190 (zero in fp32 and bf16 anyway), and the bias cancels in e / sum(e) -- the final, non-flushing
// multiply by 1/sum produces subnormal outputs correctly.
constexpr float kExpBias = 64.0f;
__device__ __forceinline__ float ex2_ftz(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}
__device__ __forceinline__ F2 ex2_ftz2(F2 t) { float lo, hi; split(t, lo, hi); return f2(ex2_ftz(lo), ex2_ftz(hi)); }
// Exponent offset of a slice whose maximum is m: exponents are x*log2e + exp_offset(m).  One rounding,
// shared by every element of the slice, so it cancels between numerator and denominator.
__device__ __forceinline__ float exp_offset(float m) { return (m == kNegInf) ? 0.f : fmaf(-m, kLog2e, kExpBias); }

// Largest element of a 16-byte vector (NaNs are ignored, as by fmaxf).
template <int DT> __device__ __forceinline__ float vec_max(const uint4& v) {
    if constexpr (DT == DT_F32) {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)), fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    } else {
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&v.x), b = *reinterpret_cast<const __nv_bfloat162*>(&v.y);
        const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&v.z), d = *reinterpret_cast<const __nv_bfloat162*>(&v.w);
        const __nv_bfloat162 m = __hmax2(__hmax2(a, b), __hmax2(c, d));
        const uint32_t w = *reinterpret_cast<const uint32_t*>(&m);
        return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    }
}

// Per-row scalars (1/n, 1/sqrt(var + eps), 1/sum) use the approximate MUFU forms: their relative error is about
// 2^-22, two orders below the 1e-5 tolerance, and the IEEE sequences would cost 10-20 instructions per row in
// every thread, which matters for rows of a few hundred bytes.  None of them flushes subnormals.
__device__ __forceinline__ float fast_div(float a, float b) { return __fdividef(a, b); }      // |b| < 2^126
__device__ __forceinline__ float fast_rsqrt(float v) { return rsqrtf(v); }
__device__ __forceinline__ float fast_rcp(float v) { return __frcp_rn(v); }

// Programmatic dependent launch: every kernel is launched with programmatic stream serialisation, so its
// CTAs may be scheduled while the previous kernel of the stream drains.  pdl_wait() orders all later global
// accesses after that kernel's completion; pdl_trigger() lets the next kernel start being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// mbarrier and bulk-copy primitives (shared-memory staging variants).  Every wait is bounded by a clock
// budget: a wait that runs out returns false, the caller records TF_ERR_TIMEOUT and carries on without
// hanging anybody.
// ---------------------------------------------------------------------------------------------
constexpr long long kWaitBudgetCycles = 400000000LL;      // about 0.2 s at 2 GHz

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long budget = kWaitBudgetCycles) {       // false: the clock budget ran out
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > budget) return false;
    return true;
}
// Bulk copy global -> this CTA's shared memory (no multicast); dst, src 16-byte aligned, bytes a multiple of 16;
// completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Reductions.
// ---------------------------------------------------------------------------------------------
struct SumOp { static __device__ __forceinline__ float apply(float a, float b) { return a + b; } static __device__ __forceinline__ float identity() { return 0.f; } };
struct MaxOp { static __device__ __forceinline__ float apply(float a, float b) { return fmaxf(a, b); } static __device__ __forceinline__ float identity() { return kNegInf; } };

template <class Op, int LANES>
__device__ __forceinline__ float group_reduce(float v) {      // all LANES lanes of the group get the result
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) v = Op::apply(v, __shfl_xor_sync(0xFFFFFFFFu, v, o, LANES));
    return v;
}

// CTA-wide reduction through `buf` (>= 32 floats of shared memory, private to this call site until the
// next __syncthreads after a later use of a DIFFERENT buffer).  Every thread gets the result.
template <class Op>
__device__ __forceinline__ float cta_reduce(float v, float* buf) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    v = group_reduce<Op, 32>(v);
    if (lane == 0) buf[warp] = v;
    __syncthreads();
    float r = (lane < nwarp) ? buf[lane] : Op::identity();
    return group_reduce<Op, 32>(r);
}

// ---------------------------------------------------------------------------------------------
// Combining per-slice partial results of one row (used across the CTAs of a cluster).
// ---------------------------------------------------------------------------------------------

// softmax: partial k is (o_k, s_k) with o_k = exp_offset(slice max) (+inf marks an all -inf slice) and
// s_k = sum_j 2^(x_j*log2e + o_k).  With O = min_k o_k (the offset of the row maximum) the row total is
// S = sum_k s_k * 2^(O - o_k), and slice k's terms rescale by 2^(O - o_k): every exponent is then
// x_j*log2e + O, the same expression in numerator and denominator.
__device__ __forceinline__ float softmax_rescale(float O, float ok) { return (ok == -kNegInf) ? 0.f : ex2(O - ok); }

// LayerNorm (Chan et al. pairwise update): (n, mean, M2) of the union of two disjoint slices.
struct MomentPartial { float n, mean, m2; };
__device__ __forceinline__ MomentPartial chan_combine(const MomentPartial& a, const MomentPartial& b) {
    if (b.n == 0.f) return a;
    if (a.n == 0.f) return b;
    const float n = a.n + b.n, d = b.mean - a.mean, f = fast_div(b.n, n);
    return MomentPartial{n, fmaf(d, f, a.mean), a.m2 + b.m2 + d * d * a.n * f};
}

}  // namespace tf
