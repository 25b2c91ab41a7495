// Fused residual add + LayerNorm / RMSNorm:  h = x + r (fp32 add, one rounding to the storage type, written out),
// y = norm(h) with the statistics taken from the ROUNDED h -- bit for bit what calling an add and then the norm would
// give, with x, r read once and h, y written once (4 row-widths of traffic instead of 6).
//
// Served by the register-resident kernels (a lane group or a CTA, optionally a cluster, holds the row): the add is
// two more instructions per pair on values that are in registers anyway.  Rows that those kernels cannot hold, or
// tensors that are not 16-byte aligned, take an element-wise add kernel followed by the ordinary norm.
#include "tf_rowreg.cuh"

namespace tf {
namespace {

using namespace rowreg;

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
    return false;
}

cudaError_t launch_addnorm(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    count_launches(1);
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
