// V_SROWS: narrow rows (128 B ... 2 KiB) of LayerNorm and RMSNorm (softmax: up to 512 B), resident in shared memory,
// G lanes per row.
//
// The register-resident forms give a thread one or two vectors of such a row, so the per-row work -- two reductions
// over 8-32 lanes, the row scalars, the statistics stores -- is paid once per vector or two, and bf16 LayerNorm rows
// of 64-1000 columns are bound by instruction issue (about 150 warp instructions per 32 vectors).  Here a CTA copies a
// block of consecutive rows into shared memory with 16-byte asynchronous copies, all issued at once, and then G = 1, 2,
// 4 or 8 lanes own a row and walk its vectors out of shared memory three times (sum, squared deviations, normalise):
// with one lane per row nothing is shuffled at all, with eight a reduction is three shuffles per eight vectors.  The
// row lives in shared memory, not in registers, so a thread can own 8-16 vectors.  y is written over x in the block
// and leaves as ONE bulk copy (shared memory -> global) issued by one thread; mean and rstd of consecutive rows are
// stored by consecutive lanes.
// Bank conflicts: the lanes of a quarter warp read 16-byte words that are a row (or G-th of a row) apart; each lane
// starts its walk at a different vector (rotation by its row index) so that the eight words fall into different banks.
#include <algorithm>

#include "tf_streamrow.cuh"

namespace tf {
namespace {

struct SArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t rows;
    int nvec;
    int rpc;          // rows per CTA: threads / G
    float n, eps;
};

__device__ __forceinline__ void cp_async16_plain(uint4* dst, const uint4* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all_plain() {
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}
// What the threads of this CTA wrote to shared memory becomes visible to the bulk-copy engine.
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // shared memory may be released once it has been read
}

// A 16-byte read of shared memory that the compiler may neither merge with an earlier read of the same word nor keep
// in registers from pass to pass: the row stays in shared memory, the kernel stays at 32-48 registers.
__device__ __forceinline__ uint4 lds_again(const uint4* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
    return v;
}

// G lanes per row, VPT vectors per lane (VPT a power of two); FULL: nvec == G * VPT.
template <int OP, int DT, int G, int VPT, bool FULL>
__global__ void __launch_bounds__(256, 4) k_srows(const SArgs a) {       // 64 registers: the rows are in shared memory, residency is what hides the copies
    using P = Pairs<DT>;
    constexpr int NP = P::NP;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    const int t = threadIdx.x, T = blockDim.x;
    const int nvec = FULL ? G * VPT : a.nvec;
    const int rpc = a.rpc;
    uint4* const tile = reinterpret_cast<uint4*>(dyn_smem);
    uint4* const params = tile + rpc * nvec;              // gamma / weight at [0, nvec), beta at [nvec, 2 nvec)
    const int64_t row0 = static_cast<int64_t>(blockIdx.x) * rpc;
    const int rows_here = static_cast<int>(min(static_cast<int64_t>(rpc), a.rows - row0));
    const int tile_vecs = rows_here * nvec;
    pdl_wait();
    pdl_trigger();
    const uint4* const src = a.x + row0 * nvec;
    for (int i = t; i < tile_vecs; i += T) cp_async16_plain(tile + i, src + i);
    if (OP != OP_SOFTMAX) {
        for (int i = t; i < nvec; i += T) {
            params[i] = ld_param(a.p0 + i);
            if (OP == OP_LAYERNORM) params[nvec + i] = ld_param(a.p1 + i);
        }
    }
    cp_async_wait_all_plain();
    __syncthreads();
    const int r = t / G, g = t % G;
    const bool live = r < rows_here;                       // lanes behind the last row of a ragged block walk its last row and
    {                                                      // write nothing (the shuffles below want whole warps)
        uint4* const rowp = tile + (live ? r : rows_here - 1) * nvec;
        // lane g owns the vectors g, g + G, ...; it visits them starting at its row's rotation, so that the lanes of a
        // quarter warp (8 / G rows) touch different banks in every step
        const int rot = (G < 8) ? (r & (VPT - 1)) : 0;
        // (the walks are unrolled four vectors at a time: fully unrolled, the compiler hoists all of a pass's reads and spills)
        auto vec_of = [&](int k) { return g + G * ((k + rot) & (VPT - 1)); };
        // the norms walk only the vectors the lane owns: all VPT of them in a full row (rotated), ceil((nvec - g) / G) in a
        // ragged one (in order; no test per vector)
        const int kend = FULL ? VPT : max(0, (nvec - g + G - 1) / G);
        auto vec_at = [&](int k) { return FULL ? vec_of(k) : g + G * k; };
        const GroupRed<G> red;
        float mean = 0.f, scale = 0.f;
        if constexpr (OP == OP_SOFTMAX) {
            // softmax (VPT <= 4 only): the exponentials stay in registers between the sum and the normalisation, one MUFU
            // per element; vectors behind the end of a ragged row contribute nothing
            float m = kNegInf;
#pragma unroll
            for (int k = 0; k < VPT; ++k) {
                const int j = vec_of(k);
                if (FULL || j < nvec) m = fmaxf(m, vec_max<DT>(lds_again(rowp + j)));
            }
            m = red.max(m, 0);
            const F2 off = f2(exp_offset(m)), l2e = f2(kLog2e);
            F2 e[VPT][NP];
            F2 s0 = f2(0.f);
#pragma unroll
            for (int k = 0; k < VPT; ++k) {
                const int j = vec_of(k);
                if (FULL || j < nvec) {
                    P::unpack(lds_again(rowp + j), e[k]);
#pragma unroll
                    for (int i = 0; i < NP; ++i) { e[k][i] = ex2_ftz2(fma2(e[k][i], l2e, off)); s0 = add2(s0, e[k][i]); }
                } else {
#pragma unroll
                    for (int i = 0; i < NP; ++i) e[k][i] = f2(0.f);
                }
            }
            const float sum = red.sum(hsum(s0), 0);
            const F2 inv = f2(sum == 0.f ? 0.f : fast_rcp(sum));
#pragma unroll
            for (int k = 0; k < VPT; ++k) {
                const int j = vec_of(k);
                if (live && (FULL || j < nvec)) {
#pragma unroll
                    for (int i = 0; i < NP; ++i) e[k][i] = mul2(e[k][i], inv);
                    rowp[j] = P::pack(e[k]);
                }
            }
        } else if constexpr (OP == OP_LAYERNORM) {
            F2 s0 = f2(0.f), s1 = f2(0.f);
#pragma unroll 4
            for (int k = 0; k < kend; ++k) {
                F2 w[NP];
                P::unpack(lds_again(rowp + vec_at(k)), w);
#pragma unroll
                for (int i = 0; i < NP; i += 2) { s0 = add2(s0, w[i]); s1 = add2(s1, w[i + 1]); }
            }
            mean = fast_div(red.sum(hsum(add2(s0, s1)), 0), a.n);
            const F2 mm = f2(mean);
            F2 q0 = f2(0.f), q1 = f2(0.f);
#pragma unroll 4
            for (int k = 0; k < kend; ++k) {
                F2 w[NP];
                P::unpack(lds_again(rowp + vec_at(k)), w);
#pragma unroll
                for (int i = 0; i < NP; i += 2) {
                    const F2 d0 = sub2(w[i], mm), d1 = sub2(w[i + 1], mm);
                    q0 = fma2(d0, d0, q0); q1 = fma2(d1, d1, q1);
                }
            }
            scale = fast_rsqrt(fast_div(red.sum(hsum(add2(q0, q1)), 0), a.n) + a.eps);
        } else {
            F2 q0 = f2(0.f), q1 = f2(0.f);
#pragma unroll 4
            for (int k = 0; k < kend; ++k) {
                F2 w[NP];
                P::unpack(lds_again(rowp + vec_at(k)), w);
#pragma unroll
                for (int i = 0; i < NP; i += 2) { q0 = fma2(w[i], w[i], q0); q1 = fma2(w[i + 1], w[i + 1], q1); }
            }
            scale = fast_rsqrt(fast_div(red.sum(hsum(add2(q0, q1)), 0), a.n) + a.eps);
        }
        if constexpr (OP != OP_SOFTMAX) {
            if (g == 0 && live) {
                const int64_t row = row0 + r;
                if (OP == OP_LAYERNORM && a.mean) a.mean[row] = mean;
                if (a.rstd) a.rstd[row] = scale;
            }
            // LayerNorm: (mean, rstd); RMSNorm: (rrms, rrms)
            const F2 ta2 = f2(OP == OP_LAYERNORM ? mean : scale), tb2 = f2(scale);
            if (live) {
#pragma unroll 4
                for (int k = 0; k < kend; ++k) {
                    const int j = vec_at(k);
                    rowp[j] = apply_vec<OP, DT, true>(lds_again(rowp + j), params + j, params + nvec + j, ta2, tb2);
                }
            }
        }
    }
    fence_async_proxy();
    __syncthreads();
    if (t == 0 && tile_vecs > 0) bulk_s2g(a.y + row0 * nvec, tile, static_cast<uint32_t>(tile_vecs) * 16u);
}

using SFn = void (*)(const SArgs);

template <int G, int VPT, bool FULL>
SFn srows_fn_c(int op, int dt) {
    if (op == OP_LAYERNORM) return dt == DT_F32 ? k_srows<OP_LAYERNORM, DT_F32, G, VPT, FULL> : k_srows<OP_LAYERNORM, DT_BF16, G, VPT, FULL>;
    if (op == OP_RMSNORM) return dt == DT_F32 ? k_srows<OP_RMSNORM, DT_F32, G, VPT, FULL> : k_srows<OP_RMSNORM, DT_BF16, G, VPT, FULL>;
    if constexpr (VPT <= 4) {
        if (op == OP_SOFTMAX) return dt == DT_F32 ? k_srows<OP_SOFTMAX, DT_F32, G, VPT, FULL> : k_srows<OP_SOFTMAX, DT_BF16, G, VPT, FULL>;
    }
    return nullptr;
}
SFn srows_fn(int op, int dt, int g, int vpt, bool full) {
#define TF_S(GG, VV) if (g == GG && vpt == VV) return full ? srows_fn_c<GG, VV, true>(op, dt) : srows_fn_c<GG, VV, false>(op, dt);
    TF_S(1, 4) TF_S(1, 8) TF_S(1, 16) TF_S(2, 4) TF_S(2, 8) TF_S(2, 16) TF_S(4, 4) TF_S(4, 8) TF_S(4, 16) TF_S(8, 4) TF_S(8, 8) TF_S(8, 16)
#undef TF_S
    return nullptr;
}

size_t srows_smem(const Plan& p, const Args& a) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    return static_cast<size_t>((p.threads / p.lanes) * nvec + nvec * (a.op == OP_LAYERNORM ? 2 : a.op == OP_RMSNORM ? 1 : 0)) * 16;
}

}  // namespace

// Plan fields: `threads` (64, 128 or 256), `lanes` = lanes per row (1, 2, 4, 8), `vpt` = vectors per lane (4, 8, 16).
bool supports_srows(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || a.len || a.r) return false;                  // (softmax: rows of up to lanes x 4 vectors)
    if (p.threads != 64 && p.threads != 128 && p.threads != 256) return false;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (p.lanes < 1 || p.vpt < 1 || nvec < 1 || nvec > static_cast<int64_t>(p.lanes) * p.vpt) return false;
    if (!srows_fn(a.op, a.dt, p.lanes, p.vpt, nvec == static_cast<int64_t>(p.lanes) * p.vpt)) return false;
    const int64_t rpc = p.threads / p.lanes;
    if ((a.rows + rpc - 1) / rpc > 0x7FFFFFFF) return false;
    return d.smem_optin == 0 || srows_smem(p, a) + 1024 <= static_cast<size_t>(d.smem_optin);
}

cudaError_t launch_srows(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    SFn fn = srows_fn(a.op, a.dt, p.lanes, p.vpt, nvec == static_cast<int64_t>(p.lanes) * p.vpt);
    if (!fn) return cudaErrorInvalidValue;
    const size_t smem = srows_smem(p, a);
    cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
    if (e != cudaSuccess) return e;
    SArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(nvec); k.rpc = p.threads / p.lanes;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    const int64_t grid = (a.rows + k.rpc - 1) / k.rpc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch(reinterpret_cast<const void*>(fn), grid, p.threads, smem, 1);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
