// Host side of V_PIPE (see tf_pipe.cuh for the kernel): stage geometry, plan checks, launch.
#include <algorithm>

#include "tf_pipe.cuh"

namespace tf {
namespace {

using pipe::PArgs;
using pipe::PipeFn;
using pipe::kPipeMaxBarriers;
using pipe::kPipeMaxThreads;

PipeFn pipe_fn(int op, int dt, int l, int v, int rpg, bool full) {
    switch (op) {
        case OP_SOFTMAX: return pipe::pipe_fn_softmax(dt, l, v, rpg, full);
        case OP_LAYERNORM: return pipe::pipe_fn_layernorm(dt, l, v, rpg, full);
        case OP_RMSNORM: return pipe::pipe_fn_rmsnorm(dt, l, v, rpg, full);
    }
    return nullptr;
}

bool row_fills(const Plan& p, const Args& a) { return a.cols * elem_size(a.dt) / 16 == static_cast<int64_t>(p.lanes) * p.vpt; }

struct PipeGeometry { int tile_rows; size_t smem; };

// Rows per unit stage: as many whole passes as fit the plan's stage budget (`chunk` bytes), at least one pass.
bool pipe_geometry(const Plan& p, const Args& a, const DeviceInfo& d, PipeGeometry& g) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    const int64_t row_bytes = nvec * 16;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    const int rpp = ut / p.lanes * std::max(1, p.rpg);       // rows a unit takes per pass
    const int units = p.threads / ut;
    int64_t rows = std::max<int64_t>(rpp, p.chunk / row_bytes / rpp * rpp);
    if (a.len) rows = rpp;                                    // length-aware: one row per tile
    const int64_t rows_per_unit = (a.rows + static_cast<int64_t>(units) * d.sms - 1) / (static_cast<int64_t>(units) * d.sms);
    rows = std::min<int64_t>(rows, std::max<int64_t>(rpp, (rows_per_unit + rpp - 1) / rpp * rpp));   // small problems: spread over all SMs
    const size_t param_bytes = a.op == OP_SOFTMAX ? 0 : static_cast<size_t>(row_bytes) * (a.op == OP_LAYERNORM ? 2 : 1);
    g.tile_rows = static_cast<int>(rows);
    g.smem = static_cast<size_t>(units) * p.stages * rows * row_bytes + param_bytes;
    if (rows * row_bytes >= (1 << 20)) return false;          // mbarrier transaction-count limit
    const size_t static_smem = 8 * kPipeMaxBarriers + 1024 + 1024;
    return g.smem + static_smem <= static_cast<size_t>(d.smem_optin) / std::max(1, p.persist);      // persist = 0: any ring that fits
}

}  // namespace

bool supports_pipe(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || p.lanes < 8 || p.threads < 32 || p.threads > kPipeMaxThreads || p.threads % 32) return false;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    if (a.len) {                                              // softmax with lengths: a row per tile, a row per pass
        if (a.op != OP_SOFTMAX || p.lanes < 32 || p.rpg != 1 || p.threads % ut || !pipe::pipe_fn_softmax_len(a.dt, p.lanes, p.vpt)) return false;
    } else if (p.threads % ut || p.rpg < 1 || !pipe_fn(a.op, a.dt, p.lanes, p.vpt, p.rpg, row_fills(p, a))) return false;
    const int units = p.threads / ut;
    if (p.stages < 1 || units * p.stages > kPipeMaxBarriers || p.persist < 0 || p.persist > 8 || p.chunk < 16) return false;
    if (ut > 32 && units > 15) return false;                  // one named barrier per multi-warp unit
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (nvec > static_cast<int64_t>(p.lanes) * p.vpt) return false;
    PipeGeometry g;
    return pipe_geometry(p, a, d, g);
}

cudaError_t launch_pipe(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    PipeFn fn = a.len ? pipe::pipe_fn_softmax_len(a.dt, p.lanes, p.vpt) : pipe_fn(a.op, a.dt, p.lanes, p.vpt, p.rpg, row_fills(p, a));
    PipeGeometry g;
    if (!fn || !pipe_geometry(p, a, d, g)) return cudaErrorInvalidValue;
    cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
    if (e != cudaSuccess) return e;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    const int units = p.threads / ut;
    const int64_t tiles = (a.rows + g.tile_rows - 1) / g.tile_rows;
    // persist = k: k CTAs per SM walk all tiles.  persist = 0: as many CTAs as it takes for every unit to get at most
    // `stages` tiles, all requested in its prologue -- no refill, the hardware replaces finished CTAs.
    int64_t grid = (tiles + units - 1) / units;
    if (p.persist > 0) grid = std::min<int64_t>(grid, static_cast<int64_t>(p.persist) * d.sms);
    else grid = std::min<int64_t>((grid + p.stages - 1) / p.stages, 0x7FFFFFFF);
    PArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.tile_rows = g.tile_rows; k.nstage = p.stages; k.status = a.status; k.len = a.len;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch(reinterpret_cast<const void*>(fn), grid, p.threads, g.smem, 1);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
