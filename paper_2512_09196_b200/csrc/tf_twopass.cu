// V_TWOPASS: long rows of any length, streamed twice with 16-byte vector loads.
//
// A CTA owns a row.  Pass A streams the row from HBM and keeps only per-thread running statistics in
// registers -- (max offset, sum) rescaled online for softmax, (n, mean, M2) merged chunk by chunk with Chan's
// update for LayerNorm, the sum of squares for RMSNorm -- so no cross-thread communication happens inside the
// row; one CTA-wide merge follows.  Pass B streams the row again, back to front, this time from L2 (a row is at most a few
// MiB and was just read; the loads of pass A carry an L2 evict-last policy, those of pass B an
// evict-first one), normalises and writes y with streaming stores.  The head of the row -- the part pass A read
// first and L2 is most likely to have dropped -- can be parked in shared memory instead (plan field `cache`).
// HBM still sees x once and y once.
// There is no shared-memory staging and no limit on the row length; many resident CTAs with several independent
// loads per thread keep the memory system busy.
// Optionally the 2-8 CTAs of a thread-block cluster share a row (plan field `cluster`): each streams its own slice in
// both passes and the slices' partials meet between the passes through distributed shared memory and one cluster
// barrier.  With rows of 256 KiB and more this keeps what is in flight between the passes within L2 (one CTA per row
// on every SM is more than L2 holds of such rows, and the second pass then goes back to HBM), and with few rows it
// gives every SM a share.
#include <cooperative_groups.h>

#include <algorithm>

#include "tf_streamrow.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace {

struct WArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t rows;
    int64_t nvec;
    const int* len;       // softmax with per-row valid lengths (elements), or null
    int64_t cache_vecs;   // vectors at the head of a row (of a CTA's slice of it) parked in shared memory between the passes
    float n, eps;
    int cs;               // CTAs per row (CL builds)
};

// MAXT / MINB: the launch bounds.  Besides the unconstrained form (1024, 0) there are (768, 2) and (512, 3), which hold
// the kernel to 40 registers so that 1536 threads are resident per SM instead of 1024-1280.
template <int OP, int DT, int MAXT, int MINB, bool CL>
__global__ void __launch_bounds__(MAXT, MINB) k_twopass(const WArgs a) {
    constexpr int NE = Elem<DT>::NE;
    __shared__ float red_buf[4 * 32];
    __shared__ float xch[CL ? 2 : 1][CL ? kMaxCluster : 1][2];   // partials of the peers, by row parity
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    uint4* const cache = reinterpret_cast<uint4*>(dyn_smem);
    pdl_wait();
    pdl_trigger();
    const uint64_t keep = policy_evict_last(), last = policy_evict_first();     // pass A keeps x in L2, pass B lets it go
    const int cs = CL ? a.cs : 1;
    const int rank = CL ? static_cast<int>(blockIdx.x % cs) : 0;
    const int64_t first_row = CL ? blockIdx.x / cs : blockIdx.x, row_step = CL ? gridDim.x / cs : gridDim.x;
    const int64_t per = CL ? (a.nvec + cs - 1) / cs : a.nvec, first = rank * per;        // this CTA's slice of every row
    const int64_t seg = max(int64_t{0}, min(per, a.nvec - first));
    const int64_t cache_vecs = min(a.cache_vecs, seg);
    auto count_of = [&](int k) { return static_cast<float>(max(int64_t{0}, min(per, a.nvec - k * per)) * NE); };
    if constexpr (CL) cg::this_cluster().sync();                  // every CTA of the cluster is resident before any remote write
    int it = 0;
    for (int64_t row = first_row; row < a.rows; row += row_step, ++it) {
        const uint4* xr = a.x + row * a.nvec + first;
        int64_t len = -1;
        if (OP == OP_SOFTMAX && a.len) {
            const int64_t whole = min(max(static_cast<int64_t>(__ldg(a.len + row)), int64_t{0}), a.nvec * NE);
            len = min(max(whole - first * NE, int64_t{0}), seg * NE);
        }
        const Running<OP, DT> run = stream_stats<OP, DT>(xr, seg, keep, cache, cache_vecs, len);
        Part part = merge_running<OP, DT>(run, CL ? fmaxf(count_of(rank), 1.f) : a.n, red_buf + 64 * (it & 1));
        if constexpr (CL) {
            cg::cluster_group cl = cg::this_cluster();
            const int xb = it & 1;
            if (threadIdx.x < cs) {                               // my partial into every CTA of the cluster
                float* dst = cl.map_shared_rank(&xch[xb][rank][0], threadIdx.x);
                dst[0] = part.a; dst[1] = part.b;
            }
            cl.sync();                                            // release our writes, acquire the peers'
            // the row's partial from the slices', in rank order (the same bits in every CTA)
            if constexpr (OP == OP_SOFTMAX) {
                float O = -kNegInf, S = 0.f;
                for (int k = 0; k < cs; ++k) O = fminf(O, xch[xb][k][0]);
                for (int k = 0; k < cs; ++k) S = fmaf(xch[xb][k][1], softmax_rescale(O, xch[xb][k][0]), S);
                part = Part{O, S};
            } else if constexpr (OP == OP_LAYERNORM) {
                float sum = 0.f, m2 = 0.f;
                for (int k = 0; k < cs; ++k) sum = fmaf(count_of(k), xch[xb][k][0], sum);
                const float mean = fast_div(sum, a.n);
                for (int k = 0; k < cs; ++k) { const float d = xch[xb][k][0] - mean; m2 += fmaf(count_of(k) * d, d, xch[xb][k][1]); }
                part = Part{mean, m2};
            } else {
                float q = 0.f;
                for (int k = 0; k < cs; ++k) q += xch[xb][k][0];
                part = Part{q, 0.f};
            }
        }
        const RowScale sc = scale_of_row<OP>(part, a.n, a.eps);
        if (threadIdx.x == 0 && rank == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = sc.a;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = sc.b;
        }
        stream_apply<OP, DT>(xr, a.y + row * a.nvec + first, a.p0 + first, a.p1 + first, seg, sc, last, cache, cache_vecs,
                             OP == OP_SOFTMAX ? run.live_end : INT64_MAX, len);
    }
}

using TwoFn = void (*)(const WArgs);

template <int MAXT, int MINB, bool CL>
TwoFn two_fn_b(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_twopass<OP_SOFTMAX, DT_F32, MAXT, MINB, CL>;
        case 1: return k_twopass<OP_SOFTMAX, DT_BF16, MAXT, MINB, CL>;
        case 2: return k_twopass<OP_LAYERNORM, DT_F32, MAXT, MINB, CL>;
        case 3: return k_twopass<OP_LAYERNORM, DT_BF16, MAXT, MINB, CL>;
        case 4: return k_twopass<OP_RMSNORM, DT_F32, MAXT, MINB, CL>;
        case 5: return k_twopass<OP_RMSNORM, DT_BF16, MAXT, MINB, CL>;
    }
    return nullptr;
}

TwoFn two_fn(int op, int dt, int threads, bool capped, bool cl) {
    if (capped && threads <= 512) return cl ? two_fn_b<512, 3, true>(op, dt) : two_fn_b<512, 3, false>(op, dt);
    if (capped && threads <= 768) return cl ? two_fn_b<768, 2, true>(op, dt) : two_fn_b<768, 2, false>(op, dt);
    return cl ? two_fn_b<1024, 0, true>(op, dt) : two_fn_b<1024, 0, false>(op, dt);
}

}  // namespace

// Plan field `chunk`: bytes of each row's head kept in shared memory between the passes (0 = none); `rpg` = 2 selects
// the register-capped build (threads <= 768).
bool supports_twopass(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (p.cluster != 1 && p.cluster != 2 && p.cluster != 4 && p.cluster != 8) return false;
    if (p.cluster > 1 && (p.cluster > d.max_cluster || a.cols * elem_size(a.dt) / 16 < p.cluster || a.rows * p.cluster > 0x7FFFFFFF)) return false;
    return vector_ok(a) && (p.rpg == 1 || (p.rpg == 2 && p.threads <= 768)) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 && p.chunk >= 0 && p.chunk % 16 == 0 &&
           (d.smem_optin == 0 || p.chunk + 2048 <= d.smem_optin);
}

cudaError_t launch_twopass(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    const int cs = std::max(1, p.cluster);
    TwoFn fn = two_fn(a.op, a.dt, p.threads, p.rpg == 2, cs > 1);
    if (!fn) return cudaErrorInvalidValue;
    int64_t grid = a.rows;                                         // in rows (clusters)
    if (p.persist > 0) grid = std::min<int64_t>(grid, std::max<int64_t>(1, static_cast<int64_t>(p.persist) * d.sms / cs));
    grid = std::min<int64_t>(grid, 0x7FFFFFFF / cs);
    WArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows; k.len = a.len;
    k.nvec = a.cols * elem_size(a.dt) / 16;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.cs = cs;
    k.cache_vecs = std::min<int64_t>((k.nvec + cs - 1) / cs, p.chunk / 16);
    if (p.chunk > 0) {
        cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = static_cast<size_t>(k.cache_vecs) * 16;
    cfg.gridDim = dim3(static_cast<unsigned>(grid * cs));
    cfg.blockDim = dim3(p.threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    int na = 1;
    if (cs > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = cs; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
