// V_TMA: shared-memory-staged split-row variant for long rows.
//
// A row is cut into `cluster` slices, one per CTA of a thread-block cluster.  Each CTA brings its slice into
// shared memory with bulk asynchronous copies (cp.async.bulk global -> shared, completion counted on an
// mbarrier per chunk; no multicast: every CTA fetches a different slice), so the bytes in flight cost no
// registers and the first reduction pass starts on chunk 0 while the later chunks are still landing.  The
// per-slice partials (max,sum | mean,M2 | sum of squares) are pushed into every peer's shared memory and
// combined after one cluster barrier; the normalise pass re-reads the slice from shared memory and writes y
// with 16-byte streaming stores.  HBM sees each element once in and once out.
//
// With stages > 1 a CTA that loops over several rows keeps the next rows' slices in flight while it works
// on the current one.
//
// Every wait on an mbarrier is bounded by a clock budget: when it runs out the CTA records TF_ERR_TIMEOUT in
// the status word, keeps taking part in the barriers (so that its peers never hang), and leaves its rows
// undefined.
#include <cooperative_groups.h>

#include <algorithm>
#include <mutex>

#include "tf_rowmath.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace {

struct TArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t rows;
    int nvec;
    float n, eps;
    int cs;          // CTAs per row
    int nstage;      // slices in flight per CTA
    int cv;          // vectors per bulk copy
    int* status;
};

template <int DT> __device__ __forceinline__ bool all_neg_inf(const uint4& v) {
    const uint32_t w = (DT == DT_F32) ? 0xFF800000u : 0xFF80FF80u;
    return (v.x == w) & (v.y == w) & (v.z == w) & (v.w == w);
}

template <int OP, int DT>
__global__ void __launch_bounds__(1024) k_tma(const TArgs a) {
    using E = Elem<DT>;
    using P = Pairs<DT>;
    constexpr int NE = E::NE, NP = P::NP;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t mbar[kMaxStages][kMaxChunks];
    __shared__ float red_buf[4 * 32];
    __shared__ float xch[2][kMaxCluster][2];

    const int T = blockDim.x, t = threadIdx.x, cs = a.cs;
    const int rank = static_cast<int>(blockIdx.x % cs);
    const int64_t cluster_id = blockIdx.x / cs, num_clusters = gridDim.x / cs;
    const int per = (a.nvec + cs - 1) / cs;
    const int first = rank * per;
    const int len = max(0, min(per, a.nvec - first));
    const int nchunk = (len + a.cv - 1) / a.cv;
    uint4* const slices = reinterpret_cast<uint4*>(dyn_smem);
    cg::cluster_group cl = cg::this_cluster();

    if (t == 0) {
        for (int s = 0; s < a.nstage; ++s)
            for (int c = 0; c < nchunk; ++c) mbar_init(&mbar[s][c], 1);
        mbar_fence_init();
    }
    pdl_wait();
    pdl_trigger();
    __syncthreads();
    if (cs > 1) cl.sync();                 // all CTAs of the cluster resident before any remote shared-memory write

    auto issue = [&](int64_t row, int stage) {       // thread 0 only
        const uint4* src = a.x + row * a.nvec + first;
        uint4* dst = slices + static_cast<size_t>(stage) * per;
        for (int c = 0; c < nchunk; ++c) {
            const int v0 = c * a.cv, nv = min(a.cv, len - v0);
            mbar_expect_tx(&mbar[stage][c], static_cast<uint32_t>(nv) * 16u);
            bulk_g2s(dst + v0, src + v0, static_cast<uint32_t>(nv) * 16u, &mbar[stage][c]);
        }
    };
    if (t == 0)
        for (int s = 0; s < a.nstage; ++s) {
            const int64_t row = cluster_id + s * num_clusters;
            if (row < a.rows) issue(row, s);
        }

    bool failed = false;
    int it = 0;
    for (int64_t row = cluster_id; row < a.rows; row += num_clusters, ++it) {
        const int stage = it % a.nstage;
        const uint32_t parity = static_cast<uint32_t>(it / a.nstage) & 1u;
        const uint4* buf = slices + static_cast<size_t>(stage) * per;
        uint4* yr = a.y + row * a.nvec + first;
        const int xb = it & 1;                       // exchange / reduction buffers alternate by row
        float* rb0 = red_buf + 64 * xb;
        float* rb1 = rb0 + 32;
        auto push = [&](float p0v, float p1v) {
            if (cs > 1) {
                if (t < cs) {
                    float* dst = cl.map_shared_rank(&xch[xb][rank][0], t);
                    dst[0] = p0v; dst[1] = p1v;
                }
                cl.sync();
            } else {
                if (t == 0) { xch[xb][0][0] = p0v; xch[xb][0][1] = p1v; }
                __syncthreads();
            }
        };
        float st0 = 0.f, st1 = 0.f;

        auto wait_chunk = [&](int c) {
            if (!mbar_wait(&mbar[stage][c], parity)) { failed = true; mbar_wait(&mbar[stage][c], parity); }
        };
        auto slice_count = [&](int k) { return static_cast<float>(max(0, min(per, a.nvec - k * per))) * NE; };
        auto get_part = [&](int k) { return Part{xch[xb][k][0], xch[xb][k][1]}; };
        const F2 l2e = f2(kLog2e);

        if constexpr (OP == OP_SOFTMAX) {
            // pass 1 (consumes chunks as they land): slice max
            float m = kNegInf;
            for (int c = 0; c < nchunk; ++c) {
                wait_chunk(c);
                const int end = min(len, (c + 1) * a.cv);
#pragma unroll 4
                for (int v = c * a.cv + t; v < end; v += T) m = fmaxf(m, vec_max<DT>(buf[v]));
            }
            m = cta_reduce<MaxOp>(m, rb0);
            // pass 2: slice sum of 2^(x*log2e + off); vectors that are -inf throughout contribute nothing
            const F2 off = f2(exp_offset(m));
            F2 s2 = f2(0.f);
#pragma unroll 4
            for (int v = t; v < len; v += T) {
                const uint4 raw = buf[v];
                if (!all_neg_inf<DT>(raw)) {
                    F2 w[NP]; P::unpack(raw, w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) s2 = add2(s2, ex2_ftz2(fma2(w[i], l2e, off)));
                }
            }
            const float s = cta_reduce<SumOp>(hsum(s2), rb1);
            push((m == kNegInf) ? -kNegInf : exp_offset(m), s);
            float O = -kNegInf;
            for (int k = 0; k < cs; ++k) O = fminf(O, xch[xb][k][0]);
            float S = 0.f;
            for (int k = 0; k < cs; ++k) S = fmaf(xch[xb][k][1], softmax_rescale(O, xch[xb][k][0]), S);
            const float inv = (S == 0.f) ? 0.f : fast_rcp(S);
            // pass 3: y = 2^(x*log2e + O) / S with the row-wide offset O; store
            const F2 O2 = f2(O), inv2 = f2(inv);
#pragma unroll 4
            for (int v = t; v < len; v += T) {
                const uint4 raw = buf[v];
                uint4 out = make_uint4(0, 0, 0, 0);
                if (!all_neg_inf<DT>(raw) && inv != 0.f) {
                    F2 w[NP]; P::unpack(raw, w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) w[i] = mul2(ex2_ftz2(fma2(w[i], l2e, O2)), inv2);
                    out = P::pack(w);
                }
                st_stream(yr + v, out);
            }
        } else if constexpr (OP == OP_LAYERNORM) {
            F2 s2 = f2(0.f);
            for (int c = 0; c < nchunk; ++c) {
                wait_chunk(c);
                const int end = min(len, (c + 1) * a.cv);
#pragma unroll 4
                for (int v = c * a.cv + t; v < end; v += T) {
                    F2 w[NP]; P::unpack(buf[v], w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) s2 = add2(s2, w[i]);
                }
            }
            const float s = cta_reduce<SumOp>(hsum(s2), rb0);
            const float mk = (len > 0) ? fast_div(s, slice_count(rank)) : 0.f;
            const F2 mk2 = f2(mk);
            F2 q2 = f2(0.f);
#pragma unroll 4
            for (int v = t; v < len; v += T) {
                F2 w[NP]; P::unpack(buf[v], w);
#pragma unroll
                for (int i = 0; i < NP; ++i) { const F2 d = sub2(w[i], mk2); q2 = fma2(d, d, q2); }
            }
            push(mk, cta_reduce<SumOp>(hsum(q2), rb1));
            const Total tot = combine_parts<OP>(cs, rank, get_part, slice_count, a.n, a.eps);
            st0 = tot.a; st1 = tot.b;
            const F2 mean2 = f2(tot.a), rstd2 = f2(tot.b);
#pragma unroll 2
            for (int v = t; v < len; v += T) {
                F2 w[NP], g[NP], b[NP];
                P::unpack(buf[v], w);
                P::unpack(ld_param(a.p0 + first + v), g);
                P::unpack(ld_param(a.p1 + first + v), b);
#pragma unroll
                for (int i = 0; i < NP; ++i) w[i] = fma2(mul2(sub2(w[i], mean2), rstd2), g[i], b[i]);
                st_stream(yr + v, P::pack(w));
            }
        } else {
            F2 q2 = f2(0.f);
            for (int c = 0; c < nchunk; ++c) {
                wait_chunk(c);
                const int end = min(len, (c + 1) * a.cv);
#pragma unroll 4
                for (int v = c * a.cv + t; v < end; v += T) {
                    F2 w[NP]; P::unpack(buf[v], w);
#pragma unroll
                    for (int i = 0; i < NP; ++i) q2 = fma2(w[i], w[i], q2);
                }
            }
            push(cta_reduce<SumOp>(hsum(q2), rb0), 0.f);
            const Total tot = combine_parts<OP>(cs, rank, get_part, slice_count, a.n, a.eps);
            st0 = tot.a; st1 = tot.b;
            const F2 rr2 = f2(tot.a);
#pragma unroll 4
            for (int v = t; v < len; v += T) {
                F2 w[NP], g[NP];
                P::unpack(buf[v], w);
                P::unpack(ld_param(a.p0 + first + v), g);
#pragma unroll
                for (int i = 0; i < NP; ++i) w[i] = mul2(mul2(w[i], rr2), g[i]);
                st_stream(yr + v, P::pack(w));
            }
        }
        if (t == 0 && rank == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = st0;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = st1;
        }
        __syncthreads();                              // the slice buffer is free: refill it with a later row
        const int64_t next = row + static_cast<int64_t>(a.nstage) * num_clusters;
        if (t == 0 && next < a.rows) issue(next, stage);
    }
    if (failed) atomicExch(a.status, 4);
}

using TmaFn = void (*)(const TArgs);

TmaFn tma_fn(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_tma<OP_SOFTMAX, DT_F32>;
        case 1: return k_tma<OP_SOFTMAX, DT_BF16>;
        case 2: return k_tma<OP_LAYERNORM, DT_F32>;
        case 3: return k_tma<OP_LAYERNORM, DT_BF16>;
        case 4: return k_tma<OP_RMSNORM, DT_F32>;
        case 5: return k_tma<OP_RMSNORM, DT_BF16>;
    }
    return nullptr;
}

struct Geometry { int per, cv, nchunk; size_t smem; };

bool geometry(const Plan& p, const Args& a, Geometry& g) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (nvec > 0x7FFFFFFF) return false;
    g.per = static_cast<int>((nvec + p.cluster - 1) / p.cluster);
    int cv = std::max(1, p.chunk / 16);
    cv = std::max(cv, (g.per + kMaxChunks - 1) / kMaxChunks);
    g.cv = cv;
    g.nchunk = (g.per + cv - 1) / cv;
    g.smem = static_cast<size_t>(p.stages) * g.per * 16;
    return true;
}

}  // namespace

bool supports_tma(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || p.threads < 32 || p.threads > 1024 || p.threads % 32) return false;
    if (p.cluster < 1 || p.cluster > kMaxCluster || p.cluster > d.max_cluster || (p.cluster & (p.cluster - 1))) return false;
    if (p.stages < 1 || p.stages > kMaxStages || p.chunk < 16 || p.chunk % 16) return false;
    Geometry g;
    if (!geometry(p, a, g)) return false;
    const size_t static_smem = sizeof(uint64_t) * kMaxStages * kMaxChunks + 4 * 32 * 4 + 2 * kMaxCluster * 2 * 4 + 256;
    return g.smem + static_smem <= static_cast<size_t>(d.smem_optin);
}

cudaError_t launch_tma(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    TmaFn fn = tma_fn(a.op, a.dt);
    Geometry g;
    if (!fn || !geometry(p, a, g)) return cudaErrorInvalidValue;
    cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
    if (e != cudaSuccess) return e;
    int64_t clusters = a.rows;
    if (p.persist > 0) clusters = std::min<int64_t>(clusters, std::max<int64_t>(1, static_cast<int64_t>(p.persist) * d.sms / p.cluster));
    clusters = std::min<int64_t>(clusters, 0x7FFFFFFF / p.cluster);
    TArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.cs = p.cluster; k.nstage = p.stages; k.cv = g.cv; k.status = a.status;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(clusters * p.cluster));
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = p.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.cluster > 1 ? 2 : 1;
    note_launch(reinterpret_cast<const void*>(fn), clusters * p.cluster, p.threads, g.smem, p.cluster);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
