// Kernel templates of the register-resident variants (V_WARP, V_CTA), shared by the plain row ops and by the fused
// residual-add forms (MODE = kModeAdd: h = x + r is formed in fp32, rounded to the storage type, written out, and the
// row op then runs on the rounded h, exactly as if the two ops had been called one after the other) and by softmax with
// per-row valid lengths (MODE = kModeLen: vectors past the row's length are not loaded, the vector that straddles it
// has its tail replaced by -inf; the stores still cover the whole row, so the tail of y is +0).
#pragma once

#include <cooperative_groups.h>

#include <algorithm>

#include "tf_rowmath.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace rowreg {

struct KArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    const uint4* r;  // kModeAdd: residual input
    uint4* h;        // kModeAdd: x + r, rounded to the storage type
    const int* len;  // kModeLen: valid length of every row, in elements
    float* mean;
    float* rstd;
    int64_t rows;
    int nvec;        // 16-byte vectors per row
    float n;         // cols as float
    float eps;
};

constexpr int kModePlain = 0, kModeAdd = 1, kModeLen = 2;

// Row length in elements, clamped to [0, cols].
__device__ __forceinline__ int row_len(const int* len, int64_t row, int cols) { return min(max(__ldg(len + row), 0), cols); }

// What the loaded vectors of a row are worth when only the row's first `len` elements count (NE per vector): this thread
// holds vectors i0, i0 + stride, ...  Vectors entirely behind the length become the fill value (one compare and a
// select per vector); the one vector of a row that straddles the length is patched in a branch that a single thread per
// row takes -- written per vector, the element-wise patch was a fifth of the instructions of a bf16 row and cost 18 %.
template <int DT, int NV>
__device__ __forceinline__ void apply_len(uint4 (&raw)[NV], int i0, int stride, int len, const uint4& fill) {
    constexpr int NE = Elem<DT>::NE;
#pragma unroll
    for (int v = 0; v < NV; ++v)
        if ((i0 + v * stride) * NE >= len) raw[v] = fill;
    const int tail = len % NE, off = len / NE - i0;               // the straddling vector is `off` vectors after my first
    if (tail != 0 && off >= 0 && off % stride == 0 && off / stride < NV) {
        const int mine = off / stride;
#pragma unroll
        for (int v = 0; v < NV; ++v)
            if (v == mine) raw[v] = mask_tail<DT>(raw[v], tail);
    }
}
// Rows of at least this many vectors (16 KiB) do not read what lies behind their length: their loads wait for the row's
// length to arrive first, which pays off from about this size on (measured at 16 KiB, half of every row live: 90 us
// skipping, 96 us reading everything).  Shorter rows load the whole row at once, like the plain kernels, and discard.
constexpr int kLenSkipVecs = 1024;

template <int DT>
__device__ __forceinline__ uint4 add_round(const uint4& a, const uint4& b) {
    using P = Pairs<DT>;
    F2 x[P::NP], y[P::NP];
    P::unpack(a, x);
    P::unpack(b, y);
#pragma unroll
    for (int i = 0; i < P::NP; ++i) x[i] = add2(x[i], y[i]);          // fp32 round-to-nearest, subnormals kept
    return P::pack(x);                                                // one rounding to the storage type
}

// Largest CTA each kernel is compiled for (bounds the registers a thread may use).
constexpr int kWarpMaxThreads = 256;
constexpr int cta_max_threads(int vpt) { return vpt <= 2 ? 1024 : 512; }

// =====================================================================================================
// V_WARP
// =====================================================================================================
template <int OP, int DT, int LANES, int VPT, int RPG, int MODE>
__global__ void __launch_bounds__(kWarpMaxThreads) k_warp(const KArgs a) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x % LANES;
    const int gpc = blockDim.x / LANES;                                   // groups per CTA
    const int64_t g = static_cast<int64_t>(blockIdx.x) * gpc + threadIdx.x / LANES;
    const int64_t G = static_cast<int64_t>(gridDim.x) * gpc;

    bool valid[VPT];
    HeldParams<VPT> par;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        const int idx = lane + v * LANES;
        valid[v] = idx < a.nvec;
        par.g[v] = make_uint4(0, 0, 0, 0); par.b[v] = make_uint4(0, 0, 0, 0);
        if (OP != OP_SOFTMAX && valid[v]) par.g[v] = ld_param(a.p0 + idx);
        if (OP == OP_LAYERNORM && valid[v]) par.b[v] = ld_param(a.p1 + idx);
    }
    const GroupRed<LANES> red;
    const uint4 fill = fill_vec<DT>(OP);

    for (int64_t base = 0; base < a.rows; base += G * RPG) {
        uint4 raw[RPG][VPT];
#pragma unroll
        for (int rr = 0; rr < RPG; ++rr) {
            const int64_t row = base + rr * G + g;                          // adjacent groups -> adjacent rows
            const int len_row = (MODE == kModeLen && row < a.rows) ? row_len(a.len, row, a.nvec * Elem<DT>::NE) : 0;
            (void)len_row;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                const bool ok = row < a.rows && valid[v];
                const int64_t idx = row * a.nvec + lane + v * LANES;
                raw[rr][v] = ok ? ld_stream(a.x + idx) : fill;
                if constexpr (MODE == kModeAdd) {
                    if (ok) {
                        raw[rr][v] = add_round<DT>(raw[rr][v], ld_stream(a.r + idx));
                        st_stream(a.h + idx, raw[rr][v]);
                    }
                }
            }
            if constexpr (MODE == kModeLen) apply_len<DT, VPT>(raw[rr], lane, LANES, len_row, fill);
        }
#pragma unroll
        for (int rr = 0; rr < RPG; ++rr) {
            const int64_t row = base + rr * G + g;
            uint4 out[VPT];
            float st0 = 0.f, st1 = 0.f;
            // which vectors the arithmetic visits: for softmax all of them (absent or masked ones hold -inf and give exact
            // zeros; a test per vector cost these latency-bound kernels 4-10 %), for the norms the ones that exist
            bool visit[VPT];
#pragma unroll
            for (int v = 0; v < VPT; ++v) visit[v] = OP == OP_SOFTMAX || valid[v];
            row_math<OP, DT, VPT>(raw[rr], visit, red, par, 0, a.n, a.eps, out, st0, st1);
            if (row < a.rows) {
#pragma unroll
                for (int v = 0; v < VPT; ++v)
                    if (valid[v]) st_stream(a.y + row * a.nvec + lane + v * LANES, out[v]);
                if (lane == 0) {
                    if (OP == OP_LAYERNORM && a.mean) a.mean[row] = st0;
                    if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = st1;
                }
            }
        }
    }
}

// =====================================================================================================
// V_CTA (optionally split over a cluster)
// =====================================================================================================
template <int OP, int DT, int VPT, bool CLUSTER, int MODE>
__global__ void __launch_bounds__(cta_max_threads(VPT)) k_cta(const KArgs a, const int cs) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    __shared__ float red_buf[4 * 32];
    __shared__ float xch[2][kMaxCluster][2];          // partials pushed by the peers, double-buffered by row parity

    pdl_wait();
    pdl_trigger();
    const int T = blockDim.x, t = threadIdx.x;
    const int rank = CLUSTER ? static_cast<int>(blockIdx.x % cs) : 0;
    const int64_t cluster_id = CLUSTER ? blockIdx.x / cs : blockIdx.x;
    const int64_t num_clusters = CLUSTER ? gridDim.x / cs : gridDim.x;
    const int per = CLUSTER ? (a.nvec + cs - 1) / cs : a.nvec;         // vectors per slice
    const int first = rank * per;
    const int len = max(0, min(per, a.nvec - first));                   // this CTA's slice length

    bool valid[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) valid[v] = (t + v * T) < len;
    const CtaRed red{red_buf};
    const LazyParams par{a.p0, a.p1, first + t, T};
    const uint4 fill = fill_vec<DT>(OP);

    if constexpr (CLUSTER) cg::this_cluster().sync();      // every CTA of the cluster is resident before any remote write

    int it = 0;
    // the length of a row is requested one row ahead: the loads of a long row wait for it (a persistent CTA would
    // otherwise pay that latency at the top of every iteration)
    int next_len = (MODE == kModeLen && cluster_id < a.rows) ? row_len(a.len, cluster_id, a.nvec * NE) : 0;
    for (int64_t row = cluster_id; row < a.rows; row += num_clusters, ++it) {
        const uint4* xr = a.x + row * a.nvec + first + t;
        uint4* yr = a.y + row * a.nvec + first + t;
        uint4 raw[VPT], out[VPT];
        const int len_row = next_len;
        if (MODE == kModeLen && row + num_clusters < a.rows) next_len = row_len(a.len, row + num_clusters, a.nvec * NE);
        (void)len_row;
        if (MODE == kModeLen && a.nvec >= kLenSkipVecs) {              // long rows: nothing behind the length is read
#pragma unroll
            for (int v = 0; v < VPT; ++v) raw[v] = (valid[v] && (first + t + v * T) * NE < len_row) ? ld_stream(xr + v * T) : fill;
        } else {
#pragma unroll
            for (int v = 0; v < VPT; ++v) raw[v] = valid[v] ? ld_stream(xr + v * T) : fill;
        }
        if constexpr (MODE == kModeLen) apply_len<DT, VPT>(raw, first + t, T, len_row, fill);
        if constexpr (MODE == kModeAdd) {
            const uint4* rr = a.r + row * a.nvec + first + t;
            uint4* hr = a.h + row * a.nvec + first + t;
#pragma unroll
            for (int v = 0; v < VPT; ++v)
                if (valid[v]) {
                    raw[v] = add_round<DT>(raw[v], ld_stream(rr + v * T));
                    st_stream(hr + v * T, raw[v]);
                }
        }
        float st0 = 0.f, st1 = 0.f;
        const int slot0 = (it & 1) * 2;
        bool livev[VPT];                                          // softmax visits every vector (see k_warp); the norms the ones that exist
#pragma unroll
        for (int v = 0; v < VPT; ++v) livev[v] = (OP == OP_SOFTMAX && MODE != kModeAdd) || valid[v];

        if constexpr (!CLUSTER) {
            row_math<OP, DT, VPT>(raw, livev, red, par, slot0, a.n, a.eps, out, st0, st1);
        } else {
            cg::cluster_group cl = cg::this_cluster();
            const int par_buf = it & 1;
            F2 w[VPT][Pairs<DT>::NP];
            const Part part = slice_stats<OP, DT, VPT>(raw, livev, red, slot0, static_cast<float>(len) * NE, w);
            if (t < cs) {                                             // push my partial into every CTA of the cluster
                float* dst = cl.map_shared_rank(&xch[par_buf][rank][0], t);
                dst[0] = part.a; dst[1] = part.b;
            }
            cl.sync();                                                // release our writes, acquire the peers'
            const Total tot = combine_parts<OP>(
                cs, rank, [&](int k) { return Part{xch[par_buf][k][0], xch[par_buf][k][1]}; },
                [&](int k) { return static_cast<float>(max(0, min(per, a.nvec - k * per))) * NE; }, a.n, a.eps);
            st0 = tot.a; st1 = tot.b;
            slice_finish<OP, DT, VPT, false>(livev, w, tot, par, out);
        }
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) st_stream(yr + v * T, out[v]);
        if (t == 0 && rank == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = st0;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = st1;
        }
    }
}

inline KArgs make_kargs(const Args& a) {
    KArgs k;
    k.r = static_cast<const uint4*>(a.r); k.h = static_cast<uint4*>(a.h); k.len = a.len;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    return k;
}

using WarpFn = void (*)(const KArgs);
using CtaFn = void (*)(const KArgs, const int);

template <int OP, int DT, int MODE> WarpFn pick_warp(int lanes, int vpt, int rpg) {
#define TF_W(L, V, R) if (lanes == L && vpt == V && rpg == R) return k_warp<OP, DT, L, V, R, MODE>;
    TF_W(8, 1, 1) TF_W(8, 1, 2) TF_W(8, 1, 4) TF_W(8, 2, 1) TF_W(8, 2, 2)
    TF_W(16, 1, 1) TF_W(16, 1, 2) TF_W(16, 1, 4) TF_W(16, 2, 1) TF_W(16, 2, 2)
    TF_W(32, 1, 1) TF_W(32, 1, 2) TF_W(32, 1, 4) TF_W(32, 2, 1) TF_W(32, 2, 2) TF_W(32, 4, 1) TF_W(32, 4, 2) TF_W(32, 8, 1)
#undef TF_W
    return nullptr;
}

template <int OP, int DT, int MODE> CtaFn pick_cta(int vpt, bool cluster) {
#define TF_C(V) if (vpt == V) return cluster ? k_cta<OP, DT, V, true, MODE> : k_cta<OP, DT, V, false, MODE>;
    TF_C(1) TF_C(2) TF_C(4) TF_C(8)
#undef TF_C
    return nullptr;
}

inline bool threads_ok(int t) { return t >= 32 && t <= 1024 && t % 32 == 0; }

inline bool warp_geometry_ok(const Plan& p, const Args& a) {
    if (!vector_ok(a) || !threads_ok(p.threads) || p.threads > kWarpMaxThreads || p.lanes < 1 || p.threads % p.lanes) return false;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    return nvec <= static_cast<int64_t>(p.lanes) * p.vpt;
}

inline bool cta_geometry_ok(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || !threads_ok(p.threads)) return false;
    if (p.cluster < 1 || p.cluster > kMaxCluster || p.cluster > d.max_cluster || (p.cluster & (p.cluster - 1))) return false;
    if (p.threads > cta_max_threads(p.vpt)) return false;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (nvec > 0x7FFFFFFF) return false;
    const int64_t per = (nvec + p.cluster - 1) / p.cluster;
    return per <= static_cast<int64_t>(p.threads) * p.vpt;
}

inline cudaError_t launch_warp_fn(WarpFn fn, const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    if (!fn) return cudaErrorInvalidValue;
    const int64_t rows_per_cta = static_cast<int64_t>(p.threads / p.lanes) * p.rpg;
    int64_t grid = (a.rows + rows_per_cta - 1) / rows_per_cta;
    if (p.persist > 0) grid = std::min<int64_t>(grid, static_cast<int64_t>(p.persist) * d.sms);
    grid = std::min<int64_t>(grid, 0x7FFFFFFF);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(p.threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch(reinterpret_cast<const void*>(fn), grid, p.threads, 0, 1);
    return cudaLaunchKernelEx(&cfg, fn, make_kargs(a));
}

inline cudaError_t launch_cta_fn(CtaFn fn, const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    if (!fn) return cudaErrorInvalidValue;
    int64_t clusters = a.rows;
    if (p.persist > 0) clusters = std::min<int64_t>(clusters, std::max<int64_t>(1, static_cast<int64_t>(p.persist) * d.sms / p.cluster));
    clusters = std::min<int64_t>(clusters, 0x7FFFFFFF / p.cluster);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(clusters * p.cluster));
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = p.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.cluster > 1 ? 2 : 1;
    note_launch(reinterpret_cast<const void*>(fn), clusters * p.cluster, p.threads, 0, p.cluster);
    return cudaLaunchKernelEx(&cfg, fn, make_kargs(a), p.cluster);
}

}  // namespace rowreg
}  // namespace tf
