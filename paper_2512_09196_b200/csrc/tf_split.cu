// V_SPLIT: few, very long rows (small-batch softmax over a vocabulary, for instance).
//
// With fewer rows than SMs a CTA or a cluster per row leaves most of the GPU idle, so a row is cut into
// `splits` segments and every (row, segment) gets its own CTA.  Kernel 1 streams the segments once and writes
// one partial per segment -- (offset, sum) | (mean, M2) | sum of squares -- to a small scratch array in global
// memory (8 bytes per segment); kernel 2 merges a row's partials (every CTA of the row computes the same
// totals, in the same order), streams its segment again (from L2: the whole problem is a few MiB) and writes y.
// The scratch is the only global memory beyond inputs and outputs that any plan of this library touches; the
// ordinary entry points take it from the stream-ordered allocator for the duration of the call.
#include <algorithm>

#include "tf_streamrow.cuh"

namespace tf {
namespace {

struct SplitArgs {
    const uint4* x;
    const uint4* p0;
    const uint4* p1;
    uint4* y;
    float* mean;
    float* rstd;
    int64_t nvec;        // 16-byte vectors per row
    int64_t seg;         // vectors per segment
    int splits;
    float n, eps;
    float2* scratch;     // [rows][splits] partials
};

template <int DT> __device__ __forceinline__ float seg_count(const SplitArgs& a, int k) {
    const int64_t len = max(static_cast<int64_t>(0), min(a.seg, a.nvec - k * a.seg));
    return static_cast<float>(len * Elem<DT>::NE);
}

template <int OP, int DT>
__global__ void __launch_bounds__(1024) k_split_stats(const SplitArgs a) {
    __shared__ float red_buf[64];
    pdl_wait();
    pdl_trigger();
    const int k = blockIdx.x;
    const int64_t row = blockIdx.y, first = k * a.seg;
    const int64_t len = max(static_cast<int64_t>(0), min(a.seg, a.nvec - first));
    const Running<OP, DT> run = stream_stats<OP, DT>(a.x + row * a.nvec + first, len, policy_evict_last());
    Part part = merge_running<OP, DT>(run, fmaxf(seg_count<DT>(a, k), 1.f), red_buf);
    if (threadIdx.x == 0) a.scratch[row * a.splits + k] = make_float2(part.a, part.b);
}

template <int OP, int DT>
__global__ void __launch_bounds__(1024) k_split_apply(const SplitArgs a) {
    __shared__ float red_buf[64];
    pdl_wait();                                  // the partials of kernel 1 are complete and visible
    pdl_trigger();
    const int k = blockIdx.x, T = blockDim.x, t = threadIdx.x;
    const int64_t row = blockIdx.y, first = k * a.seg;
    const int64_t len = max(static_cast<int64_t>(0), min(a.seg, a.nvec - first));
    const float2* parts = a.scratch + row * a.splits;
    RowScale sc;
    if constexpr (OP == OP_SOFTMAX) {
        float o = -kNegInf;                      // +inf marks "no finite element yet"
        for (int j = t; j < a.splits; j += T) o = fminf(o, parts[j].x);
        const float O = -cta_reduce<MaxOp>(-o, red_buf);
        float s = 0.f;
        for (int j = t; j < a.splits; j += T) { const float2 p = parts[j]; s = fmaf(p.y, softmax_rescale(O, p.x), s); }
        const float S = cta_reduce<SumOp>(s, red_buf + 32);
        sc = RowScale{(O == -kNegInf) ? 0.f : O, (S == 0.f) ? 0.f : fast_rcp(S)};
    } else if constexpr (OP == OP_LAYERNORM) {
        float s = 0.f;
        for (int j = t; j < a.splits; j += T) s = fmaf(seg_count<DT>(a, j), parts[j].x, s);
        const float mean = fast_div(cta_reduce<SumOp>(s, red_buf), a.n);
        float m2 = 0.f;
        for (int j = t; j < a.splits; j += T) { const float2 p = parts[j]; const float d = p.x - mean; m2 += fmaf(seg_count<DT>(a, j) * d, d, p.y); }
        sc = RowScale{mean, fast_rsqrt(fast_div(cta_reduce<SumOp>(m2, red_buf + 32), a.n) + a.eps)};
    } else {
        float s = 0.f;
        for (int j = t; j < a.splits; j += T) s += parts[j].x;
        const float rr = fast_rsqrt(fast_div(cta_reduce<SumOp>(s, red_buf), a.n) + a.eps);
        sc = RowScale{rr, rr};
    }
    if (t == 0 && k == 0) {
        if (OP == OP_LAYERNORM && a.mean) a.mean[row] = sc.a;
        if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = sc.b;
    }
    stream_apply<OP, DT>(a.x + row * a.nvec + first, a.y + row * a.nvec + first, a.p0 + first, a.p1 + first, len, sc,
                         policy_evict_first());
}

using SplitFn = void (*)(const SplitArgs);

template <int OP, int DT> void pick(SplitFn& s, SplitFn& ap) { s = k_split_stats<OP, DT>; ap = k_split_apply<OP, DT>; }

bool split_fns(int op, int dt, SplitFn& s, SplitFn& ap) {
    switch (op * 2 + dt) {
        case 0: pick<OP_SOFTMAX, DT_F32>(s, ap); return true;
        case 1: pick<OP_SOFTMAX, DT_BF16>(s, ap); return true;
        case 2: pick<OP_LAYERNORM, DT_F32>(s, ap); return true;
        case 3: pick<OP_LAYERNORM, DT_BF16>(s, ap); return true;
        case 4: pick<OP_RMSNORM, DT_F32>(s, ap); return true;
        case 5: pick<OP_RMSNORM, DT_BF16>(s, ap); return true;
    }
    return false;
}

cudaError_t launch_one(SplitFn fn, const SplitArgs& k, dim3 grid, int threads, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch(reinterpret_cast<const void*>(fn), static_cast<int64_t>(grid.x) * grid.y, threads, 0, 1);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace

bool supports_split(const Plan& p, const Args& a, const DeviceInfo&) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    return vector_ok(a) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 && p.cluster >= 1 && p.cluster <= 65535 &&
           p.cluster <= nvec && a.rows <= 65535 && a.rows * p.cluster <= (1 << 24);
}

// Both kernels of the split plan with the partials in `scratch` (rows * splits float2, device memory).
cudaError_t launch_split_with_scratch(const Plan& p, const Args& a, void* scratch, cudaStream_t st) {
    SplitFn stats = nullptr, apply = nullptr;
    if (!split_fns(a.op, a.dt, stats, apply)) return cudaErrorInvalidValue;
    SplitArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd;
    k.nvec = a.cols * elem_size(a.dt) / 16;
    k.splits = p.cluster;
    k.seg = (k.nvec + k.splits - 1) / k.splits;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.scratch = static_cast<float2*>(scratch);
    const dim3 grid(static_cast<unsigned>(k.splits), static_cast<unsigned>(a.rows));
    cudaError_t e = launch_one(stats, k, grid, p.threads, st);
    if (e != cudaSuccess) return e;
    return launch_one(apply, k, grid, p.threads, st);
}

size_t split_scratch_bytes(const Plan& p, const Args& a) { return static_cast<size_t>(a.rows) * p.cluster * sizeof(float2); }

cudaError_t launch_split(const Plan& p, const Args& a, const DeviceInfo&, cudaStream_t st) {
    void* scratch = nullptr;
    cudaError_t e = cudaMallocAsync(&scratch, split_scratch_bytes(p, a), st);       // stream-ordered: no race between streams
    if (e != cudaSuccess) return e;
    e = launch_split_with_scratch(p, a, scratch, st);
    const cudaError_t f = cudaFreeAsync(scratch, st);
    return e != cudaSuccess ? e : f;
}

}  // namespace tf

// =====================================================================================================
// tf_softmax_fwd_noalloc: the split plan with its scratch in a fixed device array of this module
// =====================================================================================================
#include <mutex>

#include "../../include/tf.h"

namespace tf {
namespace {

// Room for this many (row, segment) partials: 8192 x 8 bytes = 64 KiB, held by every GPU that loads the library
// until the process exits.
constexpr int kStaticPartials = 8192;
static __device__ __align__(256) float2 g_static_partials[kStaticPartials];

struct StaticScratch { void* ptr = nullptr; int sms = 0; bool ready = false; };
std::mutex g_static_mu;
StaticScratch g_static[64];

// Once per device, with that device current: the device address of the array (in host code its name is only a
// stand-in, not something a kernel can be given) and the SM count.  Allocates nothing.
cudaError_t static_scratch(StaticScratch** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(g_static_mu);
    StaticScratch& s = g_static[dev];
    if (!s.ready) {
        void* p = nullptr;
        if ((e = cudaGetSymbolAddress(&p, g_static_partials)) != cudaSuccess) return e;
        int sms = 0;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        s.ptr = p; s.sms = sms; s.ready = true;
    }
    *out = &s;
    return cudaSuccess;
}

}  // namespace
}  // namespace tf

extern "C" tf_status tf_softmax_fwd_noalloc(const void* x, void* y, int64_t rows, int64_t cols, tf_dtype dt_, void* stream) {
    using namespace tf;
    const int dt = dt_;
    if (rows < 0 || cols <= 0 || (dt != DT_F32 && dt != DT_BF16) || (rows > 0 && (!x || !y))) return TF_ERR_INVALID_ARG;
    if (rows == 0) return TF_OK;
    Args a{OP_SOFTMAX, dt, x, nullptr, nullptr, y, nullptr, nullptr, rows, cols, 0.f, nullptr};
    if (!vector_ok(a)) return TF_ERR_UNSUPPORTED;                 // needs 16-byte aligned x, y and cols * size % 16 == 0
    if (rows > kStaticPartials) return TF_ERR_UNSUPPORTED;        // more rows than the fixed scratch has partials for
    StaticScratch* sc = nullptr;
    cudaError_t e = static_scratch(&sc);
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    // about two CTAs per SM, segments of at least 4 KiB, and never more partials than the array holds
    const int64_t nvec = cols * elem_size(dt) / 16;
    int64_t splits = std::max<int64_t>(1, 2 * static_cast<int64_t>(sc->sms) / rows);
    splits = std::min<int64_t>(splits, std::max<int64_t>(1, nvec / 256));
    splits = std::min<int64_t>(splits, kStaticPartials / rows);
    Plan p;
    p.variant = V_SPLIT; p.threads = 256; p.cluster = static_cast<int>(splits);
    DeviceInfo d{};
    d.sms = sc->sms;
    if (!supports_split(p, a, d)) return TF_ERR_UNSUPPORTED;
    count_launches(2);
    e = launch_split_with_scratch(p, a, sc->ptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}
