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
#pragma once

#include "tf_rowmath.cuh"

namespace tf {
namespace pipe {

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
    const int* len;    // LEN builds: valid elements per row (softmax over x[r, 0:len[r]], zeros behind)
};

constexpr int kPipeMaxBarriers = 128;                    // units x stages per CTA
// Parameters staged in shared memory: gamma at [0, nvec), beta at [nvec, 2 nvec).
struct SmemParams {
    const uint4* base;
    int nvec, first, stride;
    __device__ __forceinline__ uint4 gamma(int v) const { return base[first + v * stride]; }
    __device__ __forceinline__ uint4 beta(int v) const { return base[nvec + first + v * stride]; }
};

constexpr int kPipeMaxThreads = 512;

// RPG: rows of the same columns a thread carries through one pass (parameters, barriers and shuffle latency are
// shared by them).  FULL: the row fills LANES x VPL vectors exactly, so no vector needs a predicate.
// LEN (softmax, one row per tile): only the live part of a row is copied -- the bulk copy of a tile is as long as its
// row's length says, so bytes behind the length never leave HBM and the bytes in flight are all live; the length of a
// tile travels with its stage (written by the issuing lane before it arms the barrier) and the issuing lane requests
// the length of the tile after next an iteration early, so that no copy waits for a length.
template <int OP, int DT, int LANES, int VPL, int RPG, bool FULL, bool LEN = false>
__global__ void __launch_bounds__(kPipeMaxThreads) k_pipe(const PArgs a) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    constexpr int UT = LANES < 32 ? 32 : LANES;          // threads per unit
    constexpr int RPP = UT / LANES;                      // rows a unit takes per pass
    constexpr int W = UT / 32;                           // warps per unit
    constexpr int RPU = RPP * RPG;                       // rows a unit takes per pass
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[kPipeMaxBarriers];
    __shared__ float xch[W > 1 ? (kPipeMaxThreads / UT) * 2 * RPG * W * 2 : 1];     // [unit][parity][row][warp][2]
    __shared__ int tile_len[LEN ? kPipeMaxBarriers : 1];                            // LEN: the length of the row in each stage

    const int t = threadIdx.x;
    const int nvec = FULL ? LANES * VPL : a.nvec;        // FULL builds: the row fills the unit, so its length is a constant
    const int units = blockDim.x / UT;
    const int unit = t / UT, ut = t % UT;               // unit index, thread index within the unit
    const int sub = ut / LANES, lane = ut % LANES;      // row slot within a pass, lane within the row
    const int S = a.nstage;
    const size_t tile_vecs = static_cast<size_t>(a.tile_rows) * nvec;
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem) + tile_vecs * S * unit;
    uint4* const params = reinterpret_cast<uint4*>(dyn_smem) + tile_vecs * S * units;
    uint64_t* const bars = full_bar + unit * S;
    const int64_t num_tiles = (a.rows + a.tile_rows - 1) / a.tile_rows;
    const int64_t gu = static_cast<int64_t>(blockIdx.x) * units + unit;          // global unit index
    const int64_t GU = static_cast<int64_t>(gridDim.x) * units;

    if (ut == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
        mbar_fence_init();
    }
    pdl_wait();   // everything below may read what the previous kernel wrote

    auto len_of = [&](int64_t tile) {                    // LEN: a tile is a row
        return tile < num_tiles ? min(max(__ldg(a.len + tile), 0), nvec * NE) : 0;
    };
    auto issue = [&](int64_t tile, int s, int len) {     // first thread of the unit only
        const int64_t row0 = tile * a.tile_rows;
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
        uint32_t bytes = static_cast<uint32_t>(rows_here) * nvec * 16u;
        if constexpr (LEN) {
            tile_len[unit * S + s] = len;
            bytes = static_cast<uint32_t>((len + NE - 1) / NE) * 16u;              // the live vectors only
        }
        mbar_expect_tx(&bars[s], bytes);                 // also publishes tile_len to the threads that wait on the barrier
        if (bytes) bulk_g2s(ring + tile_vecs * s, a.x + row0 * nvec, bytes, &bars[s]);
    };
    int pref_len = 0;                                    // LEN, issuing lane: the length of the tile it will issue next
    if (ut == 0) {
        if constexpr (LEN) {                             // at most eight stages: the lengths are all requested before any is used
            int first_len[8];
#pragma unroll
            for (int s = 0; s < 8; ++s) first_len[s] = s < S ? len_of(gu + s * GU) : 0;
            pref_len = len_of(gu + static_cast<int64_t>(S) * GU);
#pragma unroll
            for (int s = 0; s < 8; ++s)
                if (s < S && gu + s * GU < num_tiles) issue(gu + s * GU, s, first_len[s]);
        } else {
            for (int s = 0; s < S; ++s) {
                const int64_t tile = gu + s * GU;
                if (tile < num_tiles) issue(tile, s, 0);
            }
        }
    }
    if (OP != OP_SOFTMAX) {
        for (int i = t; i < nvec; i += blockDim.x) {
            params[i] = ld_param(a.p0 + i);
            if (OP == OP_LAYERNORM) params[nvec + i] = ld_param(a.p1 + i);
        }
    }
    __syncthreads();                                      // barriers initialised, parameters staged
    pdl_trigger();

    bool valid[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) valid[v] = FULL || (lane + v * LANES) < nvec;
    const GroupRed<(LANES < 32 ? LANES : 32)> red;
    const SmemParams par{params, nvec, lane, LANES};
    // a thread that owns one or two vectors per row (lane groups of narrow rows) keeps its parameters widened in registers
    constexpr bool kHeldWide = OP != OP_SOFTMAX && VPL <= 2 && LANES <= 32;
    HeldWideParams<DT, kHeldWide ? VPL : 1> wide;
    if constexpr (kHeldWide) {
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const bool have = valid[v];
            Pairs<DT>::unpack(have ? par.gamma(v) : make_uint4(0, 0, 0, 0), wide.g[v]);
            Pairs<DT>::unpack((have && OP == OP_LAYERNORM) ? par.beta(v) : make_uint4(0, 0, 0, 0), wide.b[v]);
        }
    }
    const uint4 fill = fill_vec<DT>(OP);
    // element count of warp w's slice of a row (multi-warp units): lanes 32w .. 32w+31 own vectors l + v*LANES
    auto slice_count = [&](int w) {
        int c = 0;
#pragma unroll
        for (int v = 0; v < VPL; ++v) c += max(0, min(32, nvec - (w * 32 + v * LANES)));
        return static_cast<float>(c * NE);
    };
    const int my_warp = ut >> 5;
    const float my_count = (W > 1) ? slice_count(my_warp) : a.n;
    (void)my_warp;

    bool failed = false;
    int s = 0, xpar = 0;                                  // stage of the current tile; its barrier's phase parity
    uint32_t phase = 0;
    for (int64_t tile = gu; tile < num_tiles; tile += GU, s = (s + 1 == S ? 0 : s + 1), phase ^= (s == 0)) {
        if (!failed && !mbar_wait(&bars[s], phase)) {
            failed = true;
            atomicExch(a.status, 4);
            mbar_wait(&bars[s], phase);                    // one more bounded wait for the copy
        }
        const int64_t row0 = tile * a.tile_rows;
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(a.tile_rows), a.rows - row0));
        const uint4* const stage = ring + tile_vecs * s + lane;          // this lane's column of the stage's first row
        uint4* const ytile = a.y + row0 * nvec + lane;                  // ... and of the tile's first row of y (offsets inside a tile fit 32 bits)
        const int64_t next = tile + static_cast<int64_t>(S) * GU;
        // same trip count for every thread of the unit; slots past the tile compute on fill values and store nothing
        for (int r0 = 0; r0 < rows_here; r0 += RPU) {
            int r[RPG];
            bool live[RPG];
            uint4 raw[RPG][VPL], out[RPG][VPL];
#pragma unroll
            for (int q = 0; q < RPG; ++q) {
                r[q] = r0 + q * RPP + sub;
                live[q] = (RPU == 1) || r[q] < rows_here;
                const uint4* xr = stage + (live[q] ? r[q] : 0) * nvec;
                if constexpr (LEN) {
                    const int len = tile_len[unit * S + s];
#pragma unroll
                    for (int v = 0; v < VPL; ++v) raw[q][v] = (live[q] && valid[v] && (lane + v * LANES) * NE < len) ? xr[v * LANES] : fill;
                    const int tail = len % NE, off = len / NE - lane;            // the vector that straddles the length: one thread's
                    if (tail != 0 && off >= 0 && off % LANES == 0 && off / LANES < VPL) {
                        const int mine = off / LANES;
#pragma unroll
                        for (int v = 0; v < VPL; ++v)
                            if (v == mine) raw[q][v] = mask_tail<DT>(raw[q][v], tail);
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < VPL; ++v) raw[q][v] = (live[q] && valid[v]) ? xr[v * LANES] : fill;
                }
            }
            F2 w[RPG][VPL][Pairs<DT>::NP];
            Part part[RPG];
            bool livev[VPL];      // vectors the arithmetic visits: LEN: those in front of the length; plain softmax: all (absent ones hold -inf)
#pragma unroll
            for (int v = 0; v < VPL; ++v) livev[v] = LEN ? (valid[v] && (lane + v * LANES) * NE < tile_len[unit * S + s]) : (OP == OP_SOFTMAX || valid[v]);
#pragma unroll
            for (int q = 0; q < RPG; ++q) part[q] = slice_stats<OP, DT, VPL, decltype(red), FULL>(raw[q], livev, red, 0, my_count, w[q]);
            Total tot[RPG];
            if constexpr (W > 1) {
                float* slot = xch + ((unit * 2 + xpar) * RPG) * W * 2;
                if ((ut & 31) == 0) {
#pragma unroll
                    for (int q = 0; q < RPG; ++q) { slot[(q * W + my_warp) * 2] = part[q].a; slot[(q * W + my_warp) * 2 + 1] = part[q].b; }
                }
                asm volatile("bar.sync %0, %1;" ::"r"(1 + unit), "r"(UT) : "memory");
#pragma unroll
                for (int q = 0; q < RPG; ++q)
                    tot[q] = combine_parts<OP>(W, my_warp, [&](int k) { return Part{slot[(q * W + k) * 2], slot[(q * W + k) * 2 + 1]}; },
                                               slice_count, a.n, a.eps);
                xpar ^= 1;
            } else {
#pragma unroll
                for (int q = 0; q < RPG; ++q) tot[q] = total_of<OP>(part[q], a.n, a.eps);
            }
            // The reductions above consumed every value this unit read from the stage (shuffle results and the
            // named barrier both depend on all of its loads): after the tile's last pass the stage is refilled.
            if (r0 + RPU >= rows_here && ut == 0 && !failed && next < num_tiles) {
                issue(next, s, pref_len);
                if constexpr (LEN) pref_len = len_of(next + GU);
            }
            if constexpr (kHeldWide) slice_finish_rows<OP, DT, VPL, RPG, (W == 1), FULL>(livev, w, tot, wide, out);
            else slice_finish_rows<OP, DT, VPL, RPG, (W == 1), FULL>(livev, w, tot, par, out);
#pragma unroll
            for (int q = 0; q < RPG; ++q) {
                if (live[q]) {
                    const int64_t row = row0 + r[q];
                    uint4* yr = ytile + r[q] * nvec;
#pragma unroll
                    for (int v = 0; v < VPL; ++v)
                        if (valid[v]) st_stream(yr + v * LANES, out[q][v]);
                    if (lane == 0) {
                        if (OP == OP_LAYERNORM && a.mean) a.mean[row] = tot[q].a;
                        if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = tot[q].b;
                    }
                }
            }
        }
    }
}

using PipeFn = void (*)(const PArgs);

template <int OP, int DT> PipeFn pick_pipe(int lanes, int vpl, int rpg, bool full) {
#define TF_P(L, V)                                                                     \
    if (lanes == L && vpl == V) {                                                      \
        if (rpg == 1) return full ? k_pipe<OP, DT, L, V, 1, true> : k_pipe<OP, DT, L, V, 1, false>; \
        if (rpg == 2 && V <= 4 && full) return k_pipe<OP, DT, L, (V <= 4 ? V : 1), 2, true>;       \
        return nullptr;                                                                \
    }
    TF_P(8, 1) TF_P(16, 1) TF_P(32, 1) TF_P(32, 2) TF_P(32, 4) TF_P(32, 8)
    TF_P(64, 2) TF_P(64, 4) TF_P(64, 8) TF_P(128, 2) TF_P(128, 4) TF_P(128, 8) TF_P(256, 2) TF_P(256, 4) TF_P(256, 8)
    TF_P(512, 4) TF_P(512, 8)
    // rows of 5120 and 12288 elements (640 / 1280 / 1536 / 3072 vectors) fill these exactly
    TF_P(160, 4) TF_P(160, 8) TF_P(320, 4) TF_P(192, 8) TF_P(384, 4) TF_P(384, 8)
#undef TF_P
    return nullptr;
}

template <int OP> PipeFn pipe_fn_op(int dt, int lanes, int vpl, int rpg, bool full) {
    return dt == DT_F32 ? pick_pipe<OP, DT_F32>(lanes, vpl, rpg, full) : pick_pipe<OP, DT_BF16>(lanes, vpl, rpg, full);
}

// The length-aware builds: softmax, one row per tile (units of at least a warp per row), one row per pass.
template <int DT> PipeFn pick_pipe_len(int lanes, int vpl) {
#define TF_PL(L, V) if (lanes == L && vpl == V) return k_pipe<OP_SOFTMAX, DT, L, V, 1, false, true>;
    TF_PL(32, 2) TF_PL(32, 4) TF_PL(32, 8) TF_PL(64, 2) TF_PL(64, 4) TF_PL(64, 8) TF_PL(128, 2) TF_PL(128, 4) TF_PL(128, 8)
    TF_PL(256, 2) TF_PL(256, 4) TF_PL(256, 8) TF_PL(512, 4) TF_PL(512, 8)
#undef TF_PL
    return nullptr;
}

// one translation unit per op instantiates the kernels
PipeFn pipe_fn_softmax(int dt, int lanes, int vpl, int rpg, bool full);
PipeFn pipe_fn_layernorm(int dt, int lanes, int vpl, int rpg, bool full);
PipeFn pipe_fn_rmsnorm(int dt, int lanes, int vpl, int rpg, bool full);
PipeFn pipe_fn_softmax_len(int dt, int lanes, int vpl);

}  // namespace pipe
}  // namespace tf
