// V_STREAM: the generic variant.  Scalar accesses and several passes over the row straight from global
// memory (the re-reads hit L2 for any row that fits there), so it runs every shape: unaligned base
// pointers, cols * sizeof(element) not a multiple of 16, and rows too long for the other variants.
// A row is owned by a warp (narrow rows) or by a whole CTA.
#include <algorithm>

#include "tf_common.cuh"

namespace tf {
namespace {

struct SArgs {
    const void* x;
    const void* p0;
    const void* p1;
    void* y;
    float* mean;
    float* rstd;
    int64_t rows, cols;
    float eps;
};

template <bool CTAWIDE, class Op>
__device__ __forceinline__ float row_reduce(float v, float* buf) {
    if constexpr (CTAWIDE) return cta_reduce<Op>(v, buf);
    else return group_reduce<Op, 32>(v);
}

template <int OP, int DT, bool CTAWIDE>
__global__ void k_stream(const SArgs a) {
    using E = Elem<DT>;
    using S = typename E::scalar;
    __shared__ float red_buf[4 * 32];
    const int width = CTAWIDE ? blockDim.x : 32;
    const int lane = CTAWIDE ? threadIdx.x : (threadIdx.x & 31);
    const int64_t gid = CTAWIDE ? blockIdx.x : static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t gstride = CTAWIDE ? gridDim.x : static_cast<int64_t>(gridDim.x) * (blockDim.x >> 5);
    const S* X = static_cast<const S*>(a.x);
    const S* P0 = static_cast<const S*>(a.p0);
    const S* P1 = static_cast<const S*>(a.p1);
    S* Y = static_cast<S*>(a.y);
    const float n = static_cast<float>(a.cols);

    int it = 0;
    for (int64_t row = gid; row < a.rows; row += gstride, ++it) {
        const S* xr = X + row * a.cols;
        S* yr = Y + row * a.cols;
        float* rb0 = red_buf + 64 * (it & 1);
        float* rb1 = rb0 + 32;
        if constexpr (OP == OP_SOFTMAX) {
            float m = kNegInf;
            for (int64_t j = lane; j < a.cols; j += width) m = fmaxf(m, E::to_float(xr[j]));
            m = row_reduce<CTAWIDE, MaxOp>(m, rb0);
            const float off = exp_offset(m);
            float s = 0.f;
            for (int64_t j = lane; j < a.cols; j += width) s += ex2_ftz(fmaf(E::to_float(xr[j]), kLog2e, off));
            s = row_reduce<CTAWIDE, SumOp>(s, rb1);
            const float inv = (s == 0.f) ? 0.f : 1.0f / s;
            for (int64_t j = lane; j < a.cols; j += width)
                yr[j] = E::from_float(ex2_ftz(fmaf(E::to_float(xr[j]), kLog2e, off)) * inv);
        } else if constexpr (OP == OP_LAYERNORM) {
            float s = 0.f;
            for (int64_t j = lane; j < a.cols; j += width) s += E::to_float(xr[j]);
            const float mean = row_reduce<CTAWIDE, SumOp>(s, rb0) / n;
            float m2 = 0.f;
            for (int64_t j = lane; j < a.cols; j += width) { const float d = E::to_float(xr[j]) - mean; m2 = fmaf(d, d, m2); }
            const float rstd = 1.0f / sqrtf(row_reduce<CTAWIDE, SumOp>(m2, rb1) / n + a.eps);
            for (int64_t j = lane; j < a.cols; j += width)
                yr[j] = E::from_float(fmaf((E::to_float(xr[j]) - mean) * rstd, E::to_float(P0[j]), E::to_float(P1[j])));
            if (lane == 0) {
                if (a.mean) a.mean[row] = mean;
                if (a.rstd) a.rstd[row] = rstd;
            }
        } else {
            float ss = 0.f;
            for (int64_t j = lane; j < a.cols; j += width) { const float v = E::to_float(xr[j]); ss = fmaf(v, v, ss); }
            const float rr = 1.0f / sqrtf(row_reduce<CTAWIDE, SumOp>(ss, rb0) / n + a.eps);
            for (int64_t j = lane; j < a.cols; j += width)
                yr[j] = E::from_float((E::to_float(xr[j]) * rr) * E::to_float(P0[j]));
            if (lane == 0 && a.rstd) a.rstd[row] = rr;
        }
    }
}

using StreamFn = void (*)(const SArgs);

template <bool W> StreamFn stream_fn(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_stream<OP_SOFTMAX, DT_F32, W>;
        case 1: return k_stream<OP_SOFTMAX, DT_BF16, W>;
        case 2: return k_stream<OP_LAYERNORM, DT_F32, W>;
        case 3: return k_stream<OP_LAYERNORM, DT_BF16, W>;
        case 4: return k_stream<OP_RMSNORM, DT_F32, W>;
        case 5: return k_stream<OP_RMSNORM, DT_BF16, W>;
    }
    return nullptr;
}

}  // namespace

bool supports_stream(const Plan& p, const Args&, const DeviceInfo&) {
    return p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 && (p.lanes == 32 || p.lanes == 0);
}

// lanes == 32: a warp per row; lanes == 0: a CTA per row.
cudaError_t launch_stream(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    const bool wide = p.lanes == 0;
    StreamFn fn = wide ? stream_fn<true>(a.op, a.dt) : stream_fn<false>(a.op, a.dt);
    if (!fn) return cudaErrorInvalidValue;
    const int64_t rows_per_cta = wide ? 1 : p.threads / 32;
    int64_t grid = (a.rows + rows_per_cta - 1) / rows_per_cta;
    if (p.persist > 0) grid = std::min<int64_t>(grid, static_cast<int64_t>(p.persist) * d.sms);
    grid = std::min<int64_t>(grid, 0x7FFFFFFF);
    SArgs k{a.x, a.p0, a.p1, a.y, a.mean, a.rstd, a.rows, a.cols, a.eps};
    note_launch(reinterpret_cast<const void*>(fn), grid, p.threads, 0, 1);
    fn<<<static_cast<unsigned>(grid), p.threads, 0, st>>>(k);
    return cudaGetLastError();
}

}  // namespace tf
