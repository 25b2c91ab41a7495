// Softmax with per-row valid lengths: row r is normalised over x[r, 0 : len[r]], y[r, len[r] :] = +0, and
// x[r, len[r] :] is never read (it may hold anything).  Against a mask stored in the data this saves the reads of
// the masked tails; the writes stay.
//
// Served by the register-resident kernels in their length mode (a lane group, a CTA or a cluster holds the row), by the
// pipeline and by the two-pass kernel's ring form for rows that fit the ring (only the live part of a row is copied), by
// the two-pass kernel's general ring form (or its direct form) for rows beyond 64 KiB, and by a scalar CTA-per-row kernel for tensors that are not
// 16-byte aligned or whose width is not a whole number of 16-byte vectors.
#include <algorithm>

#include "tf_rowreg.cuh"

namespace tf {
namespace {

using namespace rowreg;

WarpFn warp_fn_len(int dt, int l, int v, int r) {
    return dt == DT_F32 ? pick_warp<OP_SOFTMAX, DT_F32, kModeLen>(l, v, r) : pick_warp<OP_SOFTMAX, DT_BF16, kModeLen>(l, v, r);
}
CtaFn cta_fn_len(int dt, int v, bool c) {
    if (v > 4 && dt == DT_BF16) return nullptr;         // bf16 with eight vectors per thread needs 120 registers in this mode (92 plain)
    return dt == DT_F32 ? pick_cta<OP_SOFTMAX, DT_F32, kModeLen>(v, c) : pick_cta<OP_SOFTMAX, DT_BF16, kModeLen>(v, c);
}

// Any alignment, any width: a CTA per row, three scalar passes over the live part (max, sum, write), zeros behind it.
template <int DT>
__global__ void __launch_bounds__(256) k_softmax_len_scalar(const typename Elem<DT>::scalar* x, const int* len, typename Elem<DT>::scalar* y,
                                                            int64_t rows, int64_t cols) {
    using E = Elem<DT>;
    __shared__ float buf[2][32];
    const int64_t row = blockIdx.x;
    if (row >= rows) return;
    const int64_t n = min(max(static_cast<int64_t>(len[row]), int64_t{0}), cols);
    const typename E::scalar* xr = x + row * cols;
    typename E::scalar* yr = y + row * cols;
    float m = kNegInf;
    for (int64_t j = threadIdx.x; j < n; j += blockDim.x) m = fmaxf(m, E::to_float(xr[j]));
    m = cta_reduce<MaxOp>(m, buf[0]);
    float s = 0.f;
    if (m != kNegInf)
        for (int64_t j = threadIdx.x; j < n; j += blockDim.x) s += expf(E::to_float(xr[j]) - m);
    s = cta_reduce<SumOp>(s, buf[1]);
    const float inv = s > 0.f ? 1.0f / s : 0.f;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        float v = 0.f;
        if (j < n && m != kNegInf) v = expf(E::to_float(xr[j]) - m) * inv;
        yr[j] = E::from_float(v);
    }
}

}  // namespace

bool supports_softmax_len(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (a.op != OP_SOFTMAX || !a.len) return false;
    if (p.variant == V_WARP) return warp_geometry_ok(p, a) && warp_fn_len(a.dt, p.lanes, p.vpt, p.rpg) != nullptr;
    if (p.variant == V_CTA) return cta_geometry_ok(p, a, d) && cta_fn_len(a.dt, p.vpt, p.cluster > 1) != nullptr;
    if (p.variant == V_TWOPASS) return supports_twopass(p, a, d);
    if (p.variant == V_PIPE) return supports_pipe(p, a, d) && p.stages <= 8;
    return false;
}

cudaError_t launch_softmax_len(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    count_launches(1);
    if (p.variant == V_TWOPASS) return launch_twopass(p, a, d, st);
    if (p.variant == V_PIPE) return launch_pipe(p, a, d, st);
    if (p.variant == V_WARP) return launch_warp_fn(warp_fn_len(a.dt, p.lanes, p.vpt, p.rpg), p, a, d, st);
    return launch_cta_fn(cta_fn_len(a.dt, p.vpt, p.cluster > 1), p, a, d, st);
}

// Default plan, from measurements on rows of 512 B to 64 KiB: a lane group with one row in flight up to 1 KiB, the ring
// form of the two-pass kernel with the whole row in the ring for rows of 4-64 KiB (behind it, for what that form
// refuses: the length-aware pipeline for 2-byte rows, a CTA with four vectors per thread, eight for fp32 from 16 KiB
// on), the streamed two-pass kernel from there.
// (The plans that win for the plain softmax are not reused: more rows in flight per group or eight bf16 vectors per
// thread cost this mode 30-80 %.)
Plan heuristic_softmax_len(const Args& a, const DeviceInfo& d) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    Plan q;
    if (nvec < 256) {
        // rows below 4 KiB: a lane group per row, the whole row loaded at once and the part behind the length discarded
        // (65-255 vectors used to fall to a CTA per row with half its threads idle: bf16 rows of 1000 columns 154 us)
        q.variant = V_WARP; q.threads = 128; q.rpg = 1;
        if (nvec <= 8) { q.lanes = 8; q.vpt = 1; }
        else if (nvec <= 16) { q.lanes = 8; q.vpt = 2; }
        else if (nvec <= 32) { q.lanes = 16; q.vpt = 2; }
        else if (nvec <= 64) { q.lanes = 32; q.vpt = 2; }
        else if (nvec <= 128) { q.lanes = 32; q.vpt = 4; }
        else { q.lanes = 32; q.vpt = 8; }
        if (supports_softmax_len(q, a, d)) return q;
        q = Plan{};
    }
    if (nvec >= 256 && nvec <= 4096) {
        // rows of 4-64 KiB: the two-pass ring form with the whole row in the ring of one CTA copies only the live vectors of a
        // row and finds them in shared memory for the second pass.  Half-live bf16 rows of 8-64 KiB: 64 us against 73-94 us
        // for the pipeline and the two-pass direct form (and 79-85 us for the plain softmax on the same rows with the mask in
        // the data); full-length rows 82-84 us against 89-110 us.  CTAs of a sixteenth of the row's vectors for 2-byte rows
        // (four steps), an eighth for 4-byte ones.
        const int64_t per = (nvec + (a.dt == DT_BF16 ? 15 : 7)) / (a.dt == DT_BF16 ? 16 : 8);
        q = Plan{};
        q.variant = V_TWOPASS; q.chunk = 0; q.lanes = 1; q.vpt = 3; q.persist = 0; q.rpg = 1; q.cluster = 1; q.unroll = 4;
        q.threads = static_cast<int>(std::min<int64_t>(256, std::max<int64_t>(32, (per + 31) / 32 * 32)));
        const int64_t steps = (nvec + 4 * q.threads - 1) / (4 * q.threads);
        q.stages = static_cast<int>(std::max<int64_t>(2, steps));
        if (steps <= 4 && supports_softmax_len(q, a, d)) return q;
        q = Plan{};
    }
    if (nvec <= 64) {
    } else if (a.dt == DT_BF16 && nvec >= 256 && nvec <= 4096) {
        // 2-byte rows of 4-64 KiB: the pipeline copies only the live part of each row and its units skip the vectors
        // behind the length (measured 7-16 % faster than the masked plain softmax at half-live rows, where the register
        // plans below are slower than it)
        q.variant = V_PIPE; q.vpt = 8; q.rpg = 1; q.stages = 2; q.chunk = 16;
        q.lanes = 32;
        while (q.lanes < 512 && static_cast<int64_t>(q.lanes) * 8 < nvec) q.lanes *= 2;
        q.threads = std::max(256, q.lanes);
        q.persist = q.threads == 256 ? 2 : 1;
        if (supports_softmax_len(q, a, d)) return q;
        q = Plan{};
        q.variant = V_CTA; q.cluster = 1;
        q.vpt = 4;
        q.threads = std::max(64, static_cast<int>((nvec + q.vpt - 1) / q.vpt + 31) / 32 * 32);
        if (supports_softmax_len(q, a, d)) return q;
    } else if (nvec < 4096) {
        q.variant = V_CTA; q.cluster = 1;
        q.vpt = (a.dt == DT_F32 && nvec >= 1024) ? 8 : 4;
        q.threads = std::max(64, static_cast<int>((nvec + q.vpt - 1) / q.vpt + 31) / 32 * 32);
        if (supports_softmax_len(q, a, d)) return q;
    }
    if (nvec > 4096) {
        // rows beyond 64 KiB: the two-pass kernel's ring form treats every row as being as long as its length says (per-row
        // step geometry, the vector the length ends in masked where it is used, zeros behind): bf16 [4096, 131072] with
        // half-live rows 254 us against 290 us for the direct form below
        Plan g;
        g.variant = V_TWOPASS; g.threads = 512; g.chunk = 0; g.lanes = 1; g.vpt = 3; g.persist = 0; g.rpg = 1; g.cluster = 1; g.stages = 3; g.unroll = 4;
        if (supports_softmax_len(g, a, d)) return g;
    }
    Plan t;
    // (the 40-register build is the slower one in this mode: 350 against 290 us on bf16 [4096, 131072] with half-live rows)
    t.variant = V_TWOPASS; t.threads = 512; t.chunk = 49152; t.rpg = 1; t.lanes = 1; t.vpt = 3; t.stages = 0;
    return t;
}

cudaError_t launch_softmax_len_scalar(const Args& a, cudaStream_t st) {
    if (a.rows > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
    count_launches(1);
    if (a.dt == DT_F32)
        k_softmax_len_scalar<DT_F32><<<static_cast<unsigned>(a.rows), 256, 0, st>>>(static_cast<const float*>(a.x), a.len, static_cast<float*>(a.y), a.rows, a.cols);
    else
        k_softmax_len_scalar<DT_BF16><<<static_cast<unsigned>(a.rows), 256, 0, st>>>(static_cast<const uint16_t*>(a.x), a.len, static_cast<uint16_t*>(a.y), a.rows, a.cols);
    return cudaGetLastError();
}

}  // namespace tf
