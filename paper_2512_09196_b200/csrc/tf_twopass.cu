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
// There is no shared-memory staging, no cluster and no limit on the row length; many resident CTAs with
// several independent loads per thread keep the memory system busy.
#include <algorithm>

#include "tf_streamrow.cuh"

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
    int64_t cache_vecs;   // vectors at the head of a row parked in shared memory between the passes
    float n, eps;
};

// MAXT / MINB: the launch bounds.  Besides the unconstrained form (1024, 0) there are (768, 2) and (512, 3), which hold
// the kernel to 40 registers so that 1536 threads are resident per SM instead of 1024-1280.
template <int OP, int DT, int MAXT, int MINB>
__global__ void __launch_bounds__(MAXT, MINB) k_twopass(const WArgs a) {
    __shared__ float red_buf[4 * 32];
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    uint4* const cache = reinterpret_cast<uint4*>(dyn_smem);
    pdl_wait();
    pdl_trigger();
    const uint64_t keep = policy_evict_last(), last = policy_evict_first();     // pass A keeps x in L2, pass B lets it go
    int it = 0;
    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x, ++it) {
        const uint4* xr = a.x + row * a.nvec;
        int64_t len = -1;
        if (OP == OP_SOFTMAX && a.len) len = min(max(static_cast<int64_t>(__ldg(a.len + row)), int64_t{0}), a.nvec * Elem<DT>::NE);
        const Running<OP, DT> run = stream_stats<OP, DT>(xr, a.nvec, keep, cache, a.cache_vecs, len);
        const Part part = merge_running<OP, DT>(run, a.n, red_buf + 64 * (it & 1));
        const RowScale sc = scale_of_row<OP>(part, a.n, a.eps);
        if (threadIdx.x == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = sc.a;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = sc.b;
        }
        stream_apply<OP, DT>(xr, a.y + row * a.nvec, a.p0, a.p1, a.nvec, sc, last, cache, a.cache_vecs,
                             OP == OP_SOFTMAX ? run.live_end : INT64_MAX, len);
    }
}

using TwoFn = void (*)(const WArgs);

template <int MAXT, int MINB>
TwoFn two_fn_b(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_twopass<OP_SOFTMAX, DT_F32, MAXT, MINB>;
        case 1: return k_twopass<OP_SOFTMAX, DT_BF16, MAXT, MINB>;
        case 2: return k_twopass<OP_LAYERNORM, DT_F32, MAXT, MINB>;
        case 3: return k_twopass<OP_LAYERNORM, DT_BF16, MAXT, MINB>;
        case 4: return k_twopass<OP_RMSNORM, DT_F32, MAXT, MINB>;
        case 5: return k_twopass<OP_RMSNORM, DT_BF16, MAXT, MINB>;
    }
    return nullptr;
}

TwoFn two_fn(int op, int dt, int threads, bool capped) {
    if (capped && threads <= 512) return two_fn_b<512, 3>(op, dt);
    if (capped && threads <= 768) return two_fn_b<768, 2>(op, dt);
    return two_fn_b<1024, 0>(op, dt);
}

}  // namespace

// Plan field `chunk`: bytes of each row's head kept in shared memory between the passes (0 = none); `rpg` = 2 selects
// the register-capped build (threads <= 768).
bool supports_twopass(const Plan& p, const Args& a, const DeviceInfo& d) {
    return vector_ok(a) && (p.rpg == 1 || (p.rpg == 2 && p.threads <= 768)) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 && p.chunk >= 0 && p.chunk % 16 == 0 &&
           (d.smem_optin == 0 || p.chunk + 2048 <= d.smem_optin);
}

cudaError_t launch_twopass(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    TwoFn fn = two_fn(a.op, a.dt, p.threads, p.rpg == 2);
    if (!fn) return cudaErrorInvalidValue;
    int64_t grid = a.rows;
    if (p.persist > 0) grid = std::min<int64_t>(grid, static_cast<int64_t>(p.persist) * d.sms);
    grid = std::min<int64_t>(grid, 0x7FFFFFFF);
    WArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows; k.len = a.len;
    k.nvec = a.cols * elem_size(a.dt) / 16;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.cache_vecs = std::min<int64_t>(k.nvec, p.chunk / 16);
    if (p.chunk > 0) {
        cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = static_cast<size_t>(k.cache_vecs) * 16;
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(p.threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
