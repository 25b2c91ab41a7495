// V_PIPE: persistent, warp-specialised pipeline for rows that fit a shared-memory stage (128 B .. 64 KiB).
//
// Rows are dense and row-major, so a tile of R consecutive rows is one contiguous range of global memory.
// One producer thread per CTA streams tiles into a ring of shared-memory stages with bulk asynchronous
// copies (cp.async.bulk, completion counted on a "full" mbarrier per stage; no multicast); the consumer
// warps take each tile from shared memory into registers, reduce, normalise and write y with 16-byte
// streaming stores, then release the stage through an "empty" mbarrier.  The bytes in flight are the ring
// (about 190 KiB per SM) rather than what the register file can hold, and loading never waits for the
// arithmetic of the previous rows.  HBM still sees each element once in and once out.
//
// Inside a tile a row belongs to a group of LANES consumer threads (8 .. 512): sub-warp groups for narrow
// rows, one warp, or several warps that combine their partials through shared memory and a named barrier.
// LayerNorm / RMSNorm parameters are copied to shared memory once per CTA.
//
// All mbarrier waits are bounded by a clock budget; a CTA that gives up records TF_ERR_TIMEOUT in the status
// word and skips its remaining tiles (no CTA waits on another CTA here).
#include <algorithm>
#include <mutex>

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
    int tile_rows;     // rows per stage
    int nstage;
    int* status;
};

constexpr int kPipeMaxStages = 8;
constexpr int kPipeMaxGroups = 64;
constexpr long long kPipeWaitBudget = 400000000LL;      // about 0.2 s

__device__ __forceinline__ uint32_t sm_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sm_u32(bar)) : "memory");
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
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity) {       // false: the clock budget ran out
    if (bar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!bar_try_wait(bar, parity))
        if (clock64() - t0 > kPipeWaitBudget) return false;
    return true;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(sm_u32(dst)), "l"(src), "r"(bytes), "r"(sm_u32(bar)) : "memory");
}

// Reduction across a group of LANES threads.  Up to a warp: shuffles.  Beyond: warp shuffles, one slot per
// warp in shared memory, a named barrier over the group's threads, then every thread combines the slots.
// The slot buffer alternates between calls: a warp can only reach the call after next by passing the next
// call's barrier, which all warps of the group pass only after they have read this call's slots.
template <int LANES> struct PipeRed {
    float* slots;        // [2][LANES / 32] floats of this group
    int bar_id;          // named barrier of this group (1 .. 15)
    mutable int flip;
    template <class Op> __device__ __forceinline__ float run(float v) const {
        if constexpr (LANES <= 32) {
            return group_reduce<Op, LANES>(v);
        } else {
            constexpr int W = LANES / 32;
            v = group_reduce<Op, 32>(v);
            float* s = slots + flip * W;
            if ((threadIdx.x & 31) == 0) s[(threadIdx.x >> 5) % W] = v;
            asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(LANES) : "memory");
            float r = Op::identity();
#pragma unroll
            for (int w = 0; w < W; ++w) r = Op::apply(r, s[w]);
            flip ^= 1;
            return r;
        }
    }
    __device__ __forceinline__ float sum(float v, int) const { return run<SumOp>(v); }
    __device__ __forceinline__ float max(float v, int) const { return run<MaxOp>(v); }
};

// Parameters staged in shared memory: gamma at [0, nvec), beta at [nvec, 2 nvec).
struct SmemParams {
    const uint4* base;
    int nvec, first, stride;
    __device__ __forceinline__ uint4 gamma(int v) const { return base[first + v * stride]; }
    __device__ __forceinline__ uint4 beta(int v) const { return base[nvec + first + v * stride]; }
};

constexpr int pipe_max_threads(int vpl) { return vpl <= 4 ? 544 : 288; }     // producer warp + 512 / 256 consumers

template <int OP, int DT, int LANES, int VPL>
__global__ void __launch_bounds__(pipe_max_threads(VPL)) k_pipe(const PArgs a) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[kPipeMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kPipeMaxStages];
    __shared__ float red_slots[LANES > 32 ? 16 * 2 * (LANES / 32) : 1];

    const int t = threadIdx.x;
    const int NC = blockDim.x - 32;                     // consumer threads
    const int consumer_warps = NC >> 5;
    const size_t tile_vecs = static_cast<size_t>(a.tile_rows) * a.nvec;
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem);
    uint4* const params = ring + tile_vecs * a.nstage;
    const int64_t num_tiles = (a.rows + a.tile_rows - 1) / a.tile_rows;

    if (t == 0) {
        for (int s = 0; s < a.nstage; ++s) { bar_init(&full_bar[s], 1); bar_init(&empty_bar[s], consumer_warps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (OP != OP_SOFTMAX) {
        for (int i = t; i < a.nvec; i += blockDim.x) {
            params[i] = ld_param(a.p0 + i);
            if (OP == OP_LAYERNORM) params[a.nvec + i] = ld_param(a.p1 + i);
        }
    }
    __syncthreads();

    if (t < 32) {
        // ---------------- producer: one thread keeps the ring full ----------------
        if (t == 0) {
            int i = 0;
            for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++i) {
                const int s = i % a.nstage, use = i / a.nstage;
                if (use > 0 && !bar_wait(&empty_bar[s], static_cast<uint32_t>(use - 1) & 1u)) { atomicExch(a.status, 4); break; }
                const int64_t row0 = tile * a.tile_rows;
                const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
                const size_t bytes = static_cast<size_t>(rows_here) * a.nvec * 16;
                bar_expect_tx(&full_bar[s], static_cast<uint32_t>(bytes));
                const char* src = reinterpret_cast<const char*>(a.x + row0 * a.nvec);
                char* dst = reinterpret_cast<char*>(ring + tile_vecs * s);
                for (size_t off = 0; off < bytes; off += 32768) {
                    const uint32_t nb = static_cast<uint32_t>(min(static_cast<size_t>(32768), bytes - off));
                    bulk_load(dst + off, src + off, nb, &full_bar[s]);
                }
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    const int ct = t - 32;                              // consumer thread index
    const int group = ct / LANES, lane = ct % LANES;
    const int groups = NC / LANES;
    bool valid[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) valid[v] = (lane + v * LANES) < a.nvec;
    const PipeRed<LANES> red{red_slots + group * 2 * (LANES > 32 ? LANES / 32 : 1), 1 + group, 0};
    const SmemParams par{params, a.nvec, lane, LANES};
    const uint4 fill = fill_vec<DT>(OP);

    int i = 0;
    for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++i) {
        const int s = i % a.nstage;
        if (!bar_wait(&full_bar[s], static_cast<uint32_t>(i / a.nstage) & 1u)) { atomicExch(a.status, 4); return; }
        const int64_t row0 = tile * a.tile_rows;
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
        const uint4* stage = ring + tile_vecs * s;
        // The trip count is the same for every group (sub-warp groups share a warp and its shuffles): a group
        // whose row index falls past the tile computes on fill values and stores nothing.
        for (int r0 = 0; r0 < rows_here; r0 += groups) {
            const int r = r0 + group;
            const bool live = r < rows_here;
            const uint4* xr = stage + static_cast<size_t>(live ? r : 0) * a.nvec + lane;
            uint4 raw[VPL], out[VPL];
#pragma unroll
            for (int v = 0; v < VPL; ++v) raw[v] = (live && valid[v]) ? xr[v * LANES] : fill;
            float st0 = 0.f, st1 = 0.f;
            row_math<OP, DT, VPL>(raw, valid, red, par, 0, a.n, a.eps, out, st0, st1);
            if (live) {
                const int64_t row = row0 + r;
                uint4* yr = a.y + row * a.nvec + lane;
#pragma unroll
                for (int v = 0; v < VPL; ++v)
                    if (valid[v]) st_stream(yr + v * LANES, out[v]);
                if (lane == 0) {
                    if (OP == OP_LAYERNORM && a.mean) a.mean[row] = st0;
                    if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = st1;
                }
            }
        }
        __syncwarp();
        if ((t & 31) == 0) bar_arrive(&empty_bar[s]);     // this warp has read everything it needs from the stage
    }
}

using PipeFn = void (*)(const PArgs);

template <int OP, int DT> PipeFn pick_pipe(int lanes, int vpl) {
#define TF_P(L, V) if (lanes == L && vpl == V) return k_pipe<OP, DT, L, V>;
    TF_P(8, 1) TF_P(16, 1) TF_P(32, 1) TF_P(32, 2) TF_P(32, 4) TF_P(32, 8)
    TF_P(64, 2) TF_P(64, 4) TF_P(64, 8) TF_P(128, 2) TF_P(128, 4) TF_P(128, 8) TF_P(256, 2) TF_P(256, 4) TF_P(256, 8) TF_P(512, 4)
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

// Rows per stage: as many as fit the plan's stage budget (`chunk` bytes), in whole rounds of the CTA's groups
// when possible so that no group idles.
bool pipe_geometry(const Plan& p, const Args& a, const DeviceInfo& d, PipeGeometry& g) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    const int64_t row_bytes = nvec * 16;
    const int groups = p.threads / p.lanes;
    int64_t rows = std::max<int64_t>(1, p.chunk / row_bytes);
    if (rows >= groups) rows = rows / groups * groups;
    rows = std::min<int64_t>(rows, std::max<int64_t>(1, a.rows));
    const size_t param_bytes = a.op == OP_SOFTMAX ? 0 : static_cast<size_t>(row_bytes) * (a.op == OP_LAYERNORM ? 2 : 1);
    g.tile_rows = static_cast<int>(rows);
    g.smem = static_cast<size_t>(p.stages) * rows * row_bytes + param_bytes;
    if (rows * row_bytes >= (1 << 20)) return false;          // mbarrier transaction count limit
    const size_t static_smem = 16 * kPipeMaxStages + 16 * 2 * 16 * 4 + 1024;
    return g.smem + static_smem <= static_cast<size_t>(d.smem_optin) / std::max(1, p.persist);
}

}  // namespace

bool supports_pipe(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || p.lanes < 8 || p.threads < p.lanes || p.threads % 32 || p.threads % p.lanes) return false;
    if (!pipe_fn(a.op, a.dt, p.lanes, p.vpt) || p.threads + 32 > pipe_max_threads(p.vpt)) return false;
    if (p.stages < 2 || p.stages > kPipeMaxStages || p.persist < 1 || p.persist > 4 || p.chunk < 16) return false;
    const int groups = p.threads / p.lanes;
    if (groups > kPipeMaxGroups || (p.lanes > 32 && groups > 15)) return false;
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
    const int64_t tiles = (a.rows + g.tile_rows - 1) / g.tile_rows;
    const int64_t grid = std::min<int64_t>(tiles, static_cast<int64_t>(p.persist) * d.sms);
    PArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.tile_rows = g.tile_rows; k.nstage = p.stages; k.status = a.status;
    fn<<<static_cast<unsigned>(grid), p.threads + 32, g.smem, st>>>(k);
    return cudaGetLastError();
}

}  // namespace tf
