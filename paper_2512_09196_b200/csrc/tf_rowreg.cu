// Register-resident variants: the whole row (or, in a cluster, this CTA's slice of it) is loaded once into
// registers with 16-byte coalesced loads, reduced, normalised and stored.  One HBM read and one HBM write
// per element; the reductions and the exponentials run on values that never leave the register file.
//
//   V_WARP  a group of 8, 16 or 32 lanes owns a row; a warp therefore covers 4, 2 or 1 rows per load
//           instruction, which keeps narrow rows (128 B .. 4 KiB) coalesced; each group keeps `rpg` rows in
//           flight; parameters are loaded once per thread and reused for every row the thread meets.
//   V_CTA   a CTA of `threads` threads owns a row (vpt vectors per thread); with cluster > 1 the row is split
//           over the CTAs of a thread-block cluster and the per-slice partials (max,sum | mean,M2 | sumsq) are
//           exchanged through distributed shared memory with one cluster barrier per row.
#include "tf_rowreg.cuh"

namespace tf {
namespace {

using namespace rowreg;

WarpFn warp_fn(int op, int dt, int l, int v, int r) {
    switch (op * 2 + dt) {
        case 0: return pick_warp<OP_SOFTMAX, DT_F32, kModePlain>(l, v, r);
        case 1: return pick_warp<OP_SOFTMAX, DT_BF16, kModePlain>(l, v, r);
        case 2: return pick_warp<OP_LAYERNORM, DT_F32, kModePlain>(l, v, r);
        case 3: return pick_warp<OP_LAYERNORM, DT_BF16, kModePlain>(l, v, r);
        case 4: return pick_warp<OP_RMSNORM, DT_F32, kModePlain>(l, v, r);
        case 5: return pick_warp<OP_RMSNORM, DT_BF16, kModePlain>(l, v, r);
    }
    return nullptr;
}
CtaFn cta_fn(int op, int dt, int v, bool c) {
    switch (op * 2 + dt) {
        case 0: return pick_cta<OP_SOFTMAX, DT_F32, kModePlain>(v, c);
        case 1: return pick_cta<OP_SOFTMAX, DT_BF16, kModePlain>(v, c);
        case 2: return pick_cta<OP_LAYERNORM, DT_F32, kModePlain>(v, c);
        case 3: return pick_cta<OP_LAYERNORM, DT_BF16, kModePlain>(v, c);
        case 4: return pick_cta<OP_RMSNORM, DT_F32, kModePlain>(v, c);
        case 5: return pick_cta<OP_RMSNORM, DT_BF16, kModePlain>(v, c);
    }
    return nullptr;
}

}  // namespace

bool supports_warp(const Plan& p, const Args& a, const DeviceInfo&) {
    return warp_geometry_ok(p, a) && warp_fn(a.op, a.dt, p.lanes, p.vpt, p.rpg) != nullptr;
}

cudaError_t launch_warp(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    return launch_warp_fn(warp_fn(a.op, a.dt, p.lanes, p.vpt, p.rpg), p, a, d, st);
}

bool supports_cta(const Plan& p, const Args& a, const DeviceInfo& d) {
    return cta_geometry_ok(p, a, d) && cta_fn(a.op, a.dt, p.vpt, p.cluster > 1) != nullptr;
}

cudaError_t launch_cta(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    return launch_cta_fn(cta_fn(a.op, a.dt, p.vpt, p.cluster > 1), p, a, d, st);
}

}  // namespace tf
