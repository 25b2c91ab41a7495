// Fused residual add + LayerNorm / RMSNorm:  h = x + r (fp32 add, one rounding to the storage type, written out),
// y = norm(h) with the statistics taken from the ROUNDED h -- bit for bit what calling an add and then the norm would
// give, with x, r read once and h, y written once (4 row-widths of traffic instead of 6).
//
// Served by the register-resident kernels (a lane group or a CTA, optionally a cluster, holds the row): the add is
// two more instructions per pair on values that are in registers anyway.  Rows that those kernels cannot hold, or
// tensors that are not 16-byte aligned, take an element-wise add kernel followed by the ordinary norm.
#include <algorithm>

#include "tf_rowreg.cuh"
#include "tf_streamrow.cuh"

namespace tf {
namespace {

using namespace rowreg;

// Rows of 8-32 KiB, many of them (plan variant V_TWOPASS with `stages` >= the steps a row takes): x and r are copied into
// shared memory by 16-byte asynchronous copies requested all at once; the first sweep forms h = x + r (rounded once),
// writes it out, keeps it in place of x and takes the statistics from it; the second sweep normalises from shared memory.
// The row costs no registers, so a dozen small CTAs are resident per SM (the register forms hold x, r and the widened h).
struct AArgs {
    const uint4* x;
    const uint4* r;
    const uint4* p0;
    const uint4* p1;
    uint4* h;
    uint4* y;
    float* mean;
    float* rstd;
    int nvec;
    float n, eps;
};

__device__ __forceinline__ void add_cp_async16(uint4* dst, const uint4* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
template <int N> __device__ __forceinline__ void add_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int OP, int DT, int NS, bool FULL>
__global__ void __launch_bounds__(256, 4) k_addnorm_smem(const AArgs a) {
    constexpr int NE = Elem<DT>::NE, U = 4;
    __shared__ float red_buf[2 * 32];
    extern __shared__ __align__(16) unsigned char add_smem[];
    pdl_wait();
    pdl_trigger();
    const int t = threadIdx.x;
    const int nvec = a.nvec;
    const int step = (blockDim.x >> 5) * U * 32;
    const int toff = (t >> 5) * U * 32 + (t & 31);
    const int64_t base = static_cast<int64_t>(blockIdx.x) * nvec + toff;
    uint4* const xs = reinterpret_cast<uint4*>(add_smem) + toff;          // x, then h, of this thread's vectors: step s at xs + s * step (+ u * 32)
    uint4* const rs = xs + NS * step;                                     // r
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = s * step + u * 32;
            if (FULL || o + toff < nvec) { add_cp_async16(xs + o, a.x + base + o); add_cp_async16(rs + o, a.r + base + o); }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    Running<OP, DT, U> run;
    const uint4 fill = fill_vec<DT>(OP);
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        if (s == 0) add_cp_async_wait<NS - 1>();
        else if (s == 1) add_cp_async_wait<(NS > 2 ? NS - 2 : 0)>();
        else if (s == 2) add_cp_async_wait<(NS > 3 ? NS - 3 : 0)>();
        else add_cp_async_wait<0>();
        const int first = s * step + toff;
        uint4 raw[U];
        bool ok[U];
        int count = 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = s * step + u * 32;
            ok[u] = FULL || first + u * 32 < nvec;
            raw[u] = fill;
            if (ok[u]) {
                raw[u] = add_round<DT>(xs[o], rs[o]);
                xs[o] = raw[u];
                st_stream(a.h + base + o, raw[u]);
            }
            count += ok[u] ? NE : 0;
        }
        if (FULL) run.template update<false>(raw, ok, U * NE, s * U);
        else if (count > 0) run.template update<true>(raw, ok, count, s * U);
    }
    const Part part = merge_running<OP, DT, U>(run, a.n, red_buf);
    const RowScale sc = scale_of_row<OP>(part, a.n, a.eps);
    if (t == 0) {
        if (OP == OP_LAYERNORM && a.mean) a.mean[blockIdx.x] = sc.a;
        if (a.rstd) a.rstd[blockIdx.x] = sc.b;
    }
    const F2 ta2 = f2(sc.a), tb2 = f2(sc.b);
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = s * step + u * 32;
            if (FULL || o + toff < nvec) st_stream(a.y + base + o, apply_vec<OP, DT>(xs[o], a.p0 + toff + o, a.p1 + toff + o, ta2, tb2));
        }
    }
}

using AddFn = void (*)(const AArgs);
template <int NS, bool FULL>
AddFn add_smem_fn_c(int op, int dt) {
    switch (op * 2 + dt) {
        case 2: return k_addnorm_smem<OP_LAYERNORM, DT_F32, NS, FULL>;
        case 3: return k_addnorm_smem<OP_LAYERNORM, DT_BF16, NS, FULL>;
        case 4: return k_addnorm_smem<OP_RMSNORM, DT_F32, NS, FULL>;
        case 5: return k_addnorm_smem<OP_RMSNORM, DT_BF16, NS, FULL>;
    }
    return nullptr;
}
AddFn add_smem_fn(int op, int dt, int steps, bool full) {
    switch (steps) {
        case 1: return full ? add_smem_fn_c<1, true>(op, dt) : add_smem_fn_c<1, false>(op, dt);
        case 2: return full ? add_smem_fn_c<2, true>(op, dt) : add_smem_fn_c<2, false>(op, dt);
        case 3: return full ? add_smem_fn_c<3, true>(op, dt) : add_smem_fn_c<3, false>(op, dt);
        case 4: return full ? add_smem_fn_c<4, true>(op, dt) : add_smem_fn_c<4, false>(op, dt);
    }
    return nullptr;
}
// steps a row takes with this plan's CTA size, or 0 when the plan is not of this form
int add_smem_steps(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (p.variant != V_TWOPASS || p.stages < 2 || p.cluster != 1 || p.persist != 0 || p.threads < 32 || p.threads > 256 || p.threads % 32) return 0;
    if (!vector_ok(a) || a.rows > 0x7FFFFFFF) return 0;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    const int64_t steps = (nvec + 4 * p.threads - 1) / (4 * p.threads);
    if (steps > std::min(p.stages, 4)) return 0;
    if (d.smem_optin && 2 * steps * p.threads * 64 + 1024 > d.smem_optin) return 0;
    return add_smem_fn(a.op, a.dt, static_cast<int>(steps), steps * 4 * p.threads == nvec) ? static_cast<int>(steps) : 0;
}

WarpFn warp_fn_add(int op, int dt, int l, int v, int r) {
    switch (op * 2 + dt) {
        case 2: return pick_warp<OP_LAYERNORM, DT_F32, kModeAdd>(l, v, r);
        case 3: return pick_warp<OP_LAYERNORM, DT_BF16, kModeAdd>(l, v, r);
        case 4: return pick_warp<OP_RMSNORM, DT_F32, kModeAdd>(l, v, r);
        case 5: return pick_warp<OP_RMSNORM, DT_BF16, kModeAdd>(l, v, r);
    }
    return nullptr;
}
CtaFn cta_fn_add(int op, int dt, int v, bool c) {
    switch (op * 2 + dt) {
        case 2: return pick_cta<OP_LAYERNORM, DT_F32, kModeAdd>(v, c);
        case 3: return pick_cta<OP_LAYERNORM, DT_BF16, kModeAdd>(v, c);
        case 4: return pick_cta<OP_RMSNORM, DT_F32, kModeAdd>(v, c);
        case 5: return pick_cta<OP_RMSNORM, DT_BF16, kModeAdd>(v, c);
    }
    return nullptr;
}

bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// h = x + r, any alignment: 16-byte vectors where all three pointers allow it, scalars otherwise.
template <int DT>
__global__ void __launch_bounds__(256) k_add_vec(const uint4* x, const uint4* r, uint4* h, int64_t nvec) {
    pdl_wait();
    pdl_trigger();
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < nvec) st_stream(h + i, add_round<DT>(ld_stream(x + i), ld_stream(r + i)));
}
template <int DT>
__global__ void __launch_bounds__(256) k_add_scalar(const typename Elem<DT>::scalar* x, const typename Elem<DT>::scalar* r,
                                                    typename Elem<DT>::scalar* h, int64_t n) {
    using E = Elem<DT>;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) h[i] = E::from_float(E::to_float(x[i]) + E::to_float(r[i]));
}

int round_up32(int64_t v) { return static_cast<int>((v + 31) / 32 * 32); }

}  // namespace

bool supports_addnorm(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!a.r || !a.h || !al16(a.r) || !al16(a.h)) return false;
    if (p.variant == V_WARP) return warp_geometry_ok(p, a) && warp_fn_add(a.op, a.dt, p.lanes, p.vpt, p.rpg) != nullptr;
    if (p.variant == V_CTA) return cta_geometry_ok(p, a, d) && cta_fn_add(a.op, a.dt, p.vpt, p.cluster > 1) != nullptr;
    if (p.variant == V_TWOPASS) return add_smem_steps(p, a, d) > 0;
    return false;
}

cudaError_t launch_addnorm(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    count_launches(1);
    if (p.variant == V_TWOPASS) {
        const int steps = add_smem_steps(p, a, d);
        const int64_t nvec = a.cols * elem_size(a.dt) / 16;
        AddFn fn = steps ? add_smem_fn(a.op, a.dt, steps, static_cast<int64_t>(steps) * 4 * p.threads == nvec) : nullptr;
        if (!fn) return cudaErrorInvalidValue;
        cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
        if (e != cudaSuccess) return e;
        AArgs k;
        k.x = static_cast<const uint4*>(a.x); k.r = static_cast<const uint4*>(a.r); k.p0 = static_cast<const uint4*>(a.p0);
        k.p1 = static_cast<const uint4*>(a.p1); k.h = static_cast<uint4*>(a.h); k.y = static_cast<uint4*>(a.y);
        k.mean = a.mean; k.rstd = a.rstd; k.nvec = static_cast<int>(nvec); k.n = static_cast<float>(a.cols); k.eps = a.eps;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(a.rows));
        cfg.blockDim = dim3(p.threads);
        cfg.dynamicSmemBytes = static_cast<size_t>(2) * steps * p.threads * 64;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        note_launch(reinterpret_cast<const void*>(fn), a.rows, p.threads, cfg.dynamicSmemBytes, 1);
        return cudaLaunchKernelEx(&cfg, fn, k);
    }
    if (p.variant == V_WARP) return launch_warp_fn(warp_fn_add(a.op, a.dt, p.lanes, p.vpt, p.rpg), p, a, d, st);
    return launch_cta_fn(cta_fn_add(a.op, a.dt, p.vpt, p.cluster > 1), p, a, d, st);
}

// Default register-resident plan by row size (read off what tf_tune_add ends up with: the add costs registers, so the
// fused kernels like many threads with one or two vectors each); `variant` is -1 when no such plan holds the row.
Plan heuristic_addnorm(const Args& a, const DeviceInfo& d) {
    Plan p;
    p.variant = -1;
    if (!vector_ok(a)) return p;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    Plan q;
    if (nvec >= 512 && nvec <= 2048 && a.rows >= 2LL * d.sms) {
        // many rows of 8-32 KiB: x and r staged in shared memory, CTAs of an eighth of the row's vectors
        q.variant = V_TWOPASS; q.chunk = 0; q.lanes = 1; q.vpt = 3; q.persist = 0; q.rpg = 1; q.cluster = 1; q.unroll = 4;
        q.threads = static_cast<int>(std::min<int64_t>(256, std::max<int64_t>(32, round_up32((nvec + 7) / 8))));
        q.stages = static_cast<int>(std::max<int64_t>(2, (nvec + 4 * q.threads - 1) / (4 * q.threads)));
        if (supports_addnorm(q, a, d)) return q;
        q = Plan();
    }
    // rows beyond 64 KiB: the register-resident cluster forms lose to the plain add followed by the op's own long-row
    // kernels (five tensors moved instead of four, but at the copy rate: bf16 LayerNorm [3276, 40960] 602 us fused)
    if (nvec > 4096) return p;
    if (nvec <= 32) {
        q.variant = V_WARP; q.threads = 128; q.vpt = 1; q.rpg = 1;
        q.lanes = nvec <= 8 ? 8 : nvec <= 16 ? 16 : 32;
    } else {
        q.variant = V_CTA;
        int cl = 1;
        while (cl < kMaxCluster && nvec > 2048LL * cl) cl *= 2;          // up to 32 KiB of a row per CTA
        const int64_t per = (nvec + cl - 1) / cl;
        q.cluster = cl;
        if (per < 256) { q.vpt = 2; q.threads = std::max(64, round_up32((per + 1) / 2)); }
        else if (per <= 512) { q.threads = 256; q.vpt = per <= 256 ? 1 : 2; }
        else if (per <= 2048 && cl == 1) { q.threads = 1024; q.vpt = per <= 1024 ? 1 : 2; }
        else { q.threads = 512; q.vpt = 4; }
    }
    if (supports_addnorm(q, a, d)) return q;
    // anything the rules above do not hold: the widest register-resident geometry that does
    q = Plan();
    q.variant = V_CTA;
    int cl = 1;
    while (cl < kMaxCluster && nvec > 4096LL * cl) cl *= 2;
    const int64_t per = (nvec + cl - 1) / cl;
    q.cluster = cl;
    q.vpt = per <= 1024 ? 2 : per <= 2048 ? 4 : 8;
    q.threads = std::max(64, round_up32((per + q.vpt - 1) / q.vpt));
    if (supports_addnorm(q, a, d)) return q;
    return p;
}

cudaError_t launch_add_elementwise(const void* x, const void* r, void* h, int64_t n, int dt, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    count_launches(1);
    const int es = elem_size(dt);
    if (al16(x) && al16(r) && al16(h) && (n * es) % 16 == 0) {
        const int64_t nvec = n * es / 16, grid = (nvec + 255) / 256;
        if (grid > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
        if (dt == DT_F32) k_add_vec<DT_F32><<<static_cast<unsigned>(grid), 256, 0, st>>>(static_cast<const uint4*>(x), static_cast<const uint4*>(r), static_cast<uint4*>(h), nvec);
        else k_add_vec<DT_BF16><<<static_cast<unsigned>(grid), 256, 0, st>>>(static_cast<const uint4*>(x), static_cast<const uint4*>(r), static_cast<uint4*>(h), nvec);
    } else {
        const int64_t grid = (n + 255) / 256;
        if (grid > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
        if (dt == DT_F32) k_add_scalar<DT_F32><<<static_cast<unsigned>(grid), 256, 0, st>>>(static_cast<const float*>(x), static_cast<const float*>(r), static_cast<float*>(h), n);
        else k_add_scalar<DT_BF16><<<static_cast<unsigned>(grid), 256, 0, st>>>(static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(r), static_cast<uint16_t*>(h), n);
    }
    return cudaGetLastError();
}

}  // namespace tf
