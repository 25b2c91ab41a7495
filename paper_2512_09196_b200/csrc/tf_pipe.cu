// V_PIPE: persistent self-feeding pipeline for rows that fit a shared-memory stage (128 B .. 64 KiB).
//
// Rows are dense and row-major, so a tile of R consecutive rows is one contiguous range of global memory
// and arrives with one bulk asynchronous copy (cp.async.bulk global -> shared, completion counted on an
// mbarrier; no multicast).  A CTA is a set of independent UNITS (a warp, or a few warps for wide rows); each
// unit owns a small ring of stages and walks its own sequence of tiles: wait for a stage, take the rows into
// registers, reduce, and -- as soon as the reduction has consumed the stage -- let its first lane refill
// that same stage with the unit's tile after next, then normalise and write y with 16-byte streaming stores.
// There is no producer warp and no "empty" barrier: the refill is issued by a thread that has just finished
// with the data.  The bytes in flight are the rings (up to ~200 KiB per SM), not what the register file can
// hold, and no unit ever waits for another.  HBM sees each element once in and once out.
//
// Inside a unit a row belongs to LANES threads: 8 or 16 (a warp then covers 4 or 2 rows at a time), 32, or
// several warps that merge their partials (max,sum | mean,M2 | sum of squares) through shared memory and one
// named barrier per row.  LayerNorm / RMSNorm parameters are copied to shared memory once per CTA.
//
// The kernel is launched with programmatic stream serialisation: its prologue (barrier init) overlaps the
// tail of the previous kernel in the stream, and griddepcontrol.wait orders every global access after it.
//
// All mbarrier waits are bounded by a clock budget; a unit that gives up records TF_ERR_TIMEOUT in the status
// word, stops issuing copies and finishes its loop without waiting again (control flow stays uniform, so no
// named barrier is left hanging).
#include <algorithm>

#include "tf_rowmath.cuh"

namespace tf {
namespace {

struct PArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t rows;
    int nvec;          // 16-byte vectors per row
    float n, eps;
    int tile_rows;     // rows per stage of a unit
    int nstage;        // stages per unit
    int* status;
};

constexpr int kPipeMaxBarriers = 128;                    // units x stages per CTA
constexpr long long kPipeWaitBudget = 400000000LL;      // about 0.2 s

__device__ __forceinline__ uint32_t sm_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(sm_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, long long budget) {   // false: gave up
    if (bar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!bar_try_wait(bar, parity))
        if (clock64() - t0 > budget) return false;
    return true;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(sm_u32(dst)), "l"(src), "r"(bytes), "r"(sm_u32(bar)) : "memory");
}

// Parameters staged in shared memory: gamma at [0, nvec), beta at [nvec, 2 nvec).
struct SmemParams {
    const uint4* base;
    int nvec, first, stride;
    __device__ __forceinline__ uint4 gamma(int v) const { return base[first + v * stride]; }
    __device__ __forceinline__ uint4 beta(int v) const { return base[nvec + first + v * stride]; }
};

constexpr int kPipeMaxThreads = 512;

template <int OP, int DT, int LANES, int VPL>
__global__ void __launch_bounds__(kPipeMaxThreads) k_pipe(const PArgs a) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    constexpr int UT = LANES < 32 ? 32 : LANES;          // threads per unit
    constexpr int RPP = UT / LANES;                      // rows a unit takes per pass
    constexpr int W = UT / 32;                           // warps per unit
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[kPipeMaxBarriers];
    __shared__ float xch[W > 1 ? (kPipeMaxThreads / UT) * 2 * W * 2 : 1];     // [unit][parity][warp][2]

    const int t = threadIdx.x;
    const int units = blockDim.x / UT;
    const int unit = t / UT, ut = t % UT;               // unit index, thread index within the unit
    const int sub = ut / LANES, lane = ut % LANES;      // row slot within a pass, lane within the row
    const int S = a.nstage;
    const size_t tile_vecs = static_cast<size_t>(a.tile_rows) * a.nvec;
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem) + tile_vecs * S * unit;
    uint4* const params = reinterpret_cast<uint4*>(dyn_smem) + tile_vecs * S * units;
    uint64_t* const bars = full_bar + unit * S;
    const int64_t num_tiles = (a.rows + a.tile_rows - 1) / a.tile_rows;
    const int64_t gu = static_cast<int64_t>(blockIdx.x) * units + unit;          // global unit index
    const int64_t GU = static_cast<int64_t>(gridDim.x) * units;

    if (ut == 0) {
        for (int s = 0; s < S; ++s) bar_init(&bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");   // everything below may read what the previous kernel wrote

    auto issue = [&](int64_t tile, int s) {              // first thread of the unit only
        const int64_t row0 = tile * a.tile_rows;
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
        const uint32_t bytes = static_cast<uint32_t>(rows_here) * a.nvec * 16u;
        bar_expect_tx(&bars[s], bytes);
        bulk_load(ring + tile_vecs * s, a.x + row0 * a.nvec, bytes, &bars[s]);
    };
    if (ut == 0)
        for (int s = 0; s < S; ++s) {
            const int64_t tile = gu + s * GU;
            if (tile < num_tiles) issue(tile, s);
        }
    if (OP != OP_SOFTMAX) {
        for (int i = t; i < a.nvec; i += blockDim.x) {
            params[i] = ld_param(a.p0 + i);
            if (OP == OP_LAYERNORM) params[a.nvec + i] = ld_param(a.p1 + i);
        }
    }
    __syncthreads();                                      // barriers initialised, parameters staged
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    bool valid[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) valid[v] = (lane + v * LANES) < a.nvec;
    const GroupRed<(LANES < 32 ? LANES : 32)> red;
    const SmemParams par{params, a.nvec, lane, LANES};
    const uint4 fill = fill_vec<DT>(OP);
    // element count of warp w's slice of a row (multi-warp units): lanes 32w .. 32w+31 own vectors l + v*LANES
    auto slice_count = [&](int w) {
        int c = 0;
#pragma unroll
        for (int v = 0; v < VPL; ++v) c += max(0, min(32, a.nvec - (w * 32 + v * LANES)));
        return static_cast<float>(c * NE);
    };
    const int my_warp = ut >> 5;
    const float my_count = (W > 1) ? slice_count(my_warp) : a.n;

    bool failed = false;
    int i = 0, xpar = 0;
    for (int64_t tile = gu; tile < num_tiles; tile += GU, ++i) {
        const int s = i % S;
        if (!failed && !bar_wait(&bars[s], static_cast<uint32_t>(i / S) & 1u, kPipeWaitBudget)) {
            failed = true;
            atomicExch(a.status, 4);
            bar_wait(&bars[s], static_cast<uint32_t>(i / S) & 1u, kPipeWaitBudget);    // one more bounded wait for the copy
        }
        const int64_t row0 = tile * a.tile_rows;
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
        const uint4* stage = ring + tile_vecs * s;
        const int64_t next = tile + static_cast<int64_t>(S) * GU;
        // same trip count for every thread of the unit; slots past the tile compute on fill values and store nothing
        for (int r0 = 0; r0 < rows_here; r0 += RPP) {
            const int r = r0 + sub;
            const bool live = r < rows_here;
            const uint4* xr = stage + static_cast<size_t>(live ? r : 0) * a.nvec + lane;
            uint4 raw[VPL], out[VPL];
#pragma unroll
            for (int v = 0; v < VPL; ++v) raw[v] = (live && valid[v]) ? xr[v * LANES] : fill;
            F2 w[VPL][Pairs<DT>::NP];
            const Part part = slice_stats<OP, DT, VPL>(raw, valid, red, 0, my_count, w);
            Total tot;
            if constexpr (W > 1) {
                float* slot = xch + ((unit * 2 + xpar) * W) * 2;
                if ((ut & 31) == 0) { slot[my_warp * 2] = part.a; slot[my_warp * 2 + 1] = part.b; }
                asm volatile("bar.sync %0, %1;" ::"r"(1 + unit), "r"(UT) : "memory");
                tot = combine_parts<OP>(W, my_warp, [&](int k) { return Part{slot[k * 2], slot[k * 2 + 1]}; }, slice_count, a.n, a.eps);
                xpar ^= 1;
            } else {
                tot = total_of<OP>(part, a.n, a.eps);
            }
            // The reduction above consumed every value this unit read from the stage (shuffle results and the
            // named barrier both depend on all of its loads): after the tile's last pass the stage is refilled.
            if (r0 + RPP >= rows_here && ut == 0 && !failed && next < num_tiles) issue(next, s);
            slice_finish<OP, DT, VPL, (W == 1)>(valid, w, tot, par, out);
            if (live) {
                const int64_t row = row0 + r;
                uint4* yr = a.y + row * a.nvec + lane;
#pragma unroll
                for (int v = 0; v < VPL; ++v)
                    if (valid[v]) st_stream(yr + v * LANES, out[v]);
                if (lane == 0) {
                    if (OP == OP_LAYERNORM && a.mean) a.mean[row] = tot.a;
                    if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = tot.b;
                }
            }
        }
    }
}

using PipeFn = void (*)(const PArgs);

template <int OP, int DT> PipeFn pick_pipe(int lanes, int vpl) {
#define TF_P(L, V) if (lanes == L && vpl == V) return k_pipe<OP, DT, L, V>;
    TF_P(8, 1) TF_P(16, 1) TF_P(32, 1) TF_P(32, 2) TF_P(32, 4) TF_P(32, 8)
    TF_P(64, 2) TF_P(64, 4) TF_P(64, 8) TF_P(128, 2) TF_P(128, 4) TF_P(128, 8) TF_P(256, 2) TF_P(256, 4) TF_P(256, 8)
    TF_P(512, 4) TF_P(512, 8)
#undef TF_P
    return nullptr;
}

PipeFn pipe_fn(int op, int dt, int l, int v) {
    switch (op * 2 + dt) {
        case 0: return pick_pipe<OP_SOFTMAX, DT_F32>(l, v);
        case 1: return pick_pipe<OP_SOFTMAX, DT_BF16>(l, v);
        case 2: return pick_pipe<OP_LAYERNORM, DT_F32>(l, v);
        case 3: return pick_pipe<OP_LAYERNORM, DT_BF16>(l, v);
        case 4: return pick_pipe<OP_RMSNORM, DT_F32>(l, v);
        case 5: return pick_pipe<OP_RMSNORM, DT_BF16>(l, v);
    }
    return nullptr;
}

struct PipeGeometry { int tile_rows; size_t smem; };

// Rows per unit stage: as many whole passes as fit the plan's stage budget (`chunk` bytes), at least one pass.
bool pipe_geometry(const Plan& p, const Args& a, const DeviceInfo& d, PipeGeometry& g) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    const int64_t row_bytes = nvec * 16;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    const int rpp = ut / p.lanes;
    const int units = p.threads / ut;
    int64_t rows = std::max<int64_t>(rpp, p.chunk / row_bytes / rpp * rpp);
    const int64_t rows_per_unit = (a.rows + static_cast<int64_t>(units) * d.sms - 1) / (static_cast<int64_t>(units) * d.sms);
    rows = std::min<int64_t>(rows, std::max<int64_t>(rpp, (rows_per_unit + rpp - 1) / rpp * rpp));   // small problems: spread over all SMs
    const size_t param_bytes = a.op == OP_SOFTMAX ? 0 : static_cast<size_t>(row_bytes) * (a.op == OP_LAYERNORM ? 2 : 1);
    g.tile_rows = static_cast<int>(rows);
    g.smem = static_cast<size_t>(units) * p.stages * rows * row_bytes + param_bytes;
    if (rows * row_bytes >= (1 << 20)) return false;          // mbarrier transaction-count limit
    const size_t static_smem = 8 * kPipeMaxBarriers + 1024 + 1024;
    return g.smem + static_smem <= static_cast<size_t>(d.smem_optin) / std::max(1, p.persist);
}

}  // namespace

bool supports_pipe(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || p.lanes < 8 || p.threads < 32 || p.threads > kPipeMaxThreads || p.threads % 32) return false;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    if (p.threads % ut || !pipe_fn(a.op, a.dt, p.lanes, p.vpt)) return false;
    const int units = p.threads / ut;
    if (p.stages < 1 || units * p.stages > kPipeMaxBarriers || p.persist < 1 || p.persist > 8 || p.chunk < 16) return false;
    if (ut > 32 && units > 15) return false;                  // one named barrier per multi-warp unit
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (nvec > static_cast<int64_t>(p.lanes) * p.vpt) return false;
    PipeGeometry g;
    return pipe_geometry(p, a, d, g);
}

cudaError_t launch_pipe(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    PipeFn fn = pipe_fn(a.op, a.dt, p.lanes, p.vpt);
    PipeGeometry g;
    if (!fn || !pipe_geometry(p, a, d, g)) return cudaErrorInvalidValue;
    cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
    if (e != cudaSuccess) return e;
    const int ut = p.lanes < 32 ? 32 : p.lanes;
    const int units = p.threads / ut;
    const int64_t tiles = (a.rows + g.tile_rows - 1) / g.tile_rows;
    const int64_t grid = std::min<int64_t>((tiles + units - 1) / units, static_cast<int64_t>(p.persist) * d.sms);
    PArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.tile_rows = g.tile_rows; k.nstage = p.stages; k.status = a.status;
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
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
