// Backward passes of LayerNorm and RMSNorm from the forward pass's stored statistics.
//   xh_j = (x_j - mean) rstd  (RMSNorm: x_j rstd),  g_j = dy_j gamma_j
//   dx_j = rstd (g_j - mean_k g_k - xh_j mean_k(g_k xh_k))         (RMSNorm: no mean_k g_k term)
//   dgamma_j = sum_rows dy_j xh_j,  dbeta_j = sum_rows dy_j         (LayerNorm only)
// dx is the same row-wise reduce-then-normalise shape as the forward ops; the parameter gradients are sums over the
// ROWS, which no row-owning CTA can finish alone.  As many CTAs as are resident at once each walk a strided share of the
// rows with the row held in registers: every thread owns the same columns of every row, so it keeps its slice of gamma
// widened in registers and accumulates its slice of dgamma / dbeta in fp32 across all the rows it meets.  At the end
// every CTA writes its partial column sums to the caller's workspace and a second kernel adds the partials in a fixed
// order (deterministic) and rounds once.  x and dy are read once, dx written once.
// Rows beyond what 512 threads hold (16 KiB bf16, 32 KiB fp32) are streamed twice by one CTA per SM that keeps its
// partial column sums in shared memory (up to 200 KiB of them); unaligned tensors, odd widths and wider rows still take
// two plain kernels: scalar passes per row for dx, a thread per column for the parameter gradients.
#include <algorithm>

#include "../../include/tf.h"
#include "tf_common.cuh"

namespace tf {
namespace {

struct BArgs {
    const uint4* x;
    const uint4* gamma;
    const uint4* dy;
    const float* mean;
    const float* rstd;
    uint4* dx;
    float* part;          // [grid][LN ? 2 : 1][cols] fp32 partial column sums
    int64_t rows;
    int nvec;
    float inv_n;
};

// A CTA is cut into row groups of `gt` threads (a multiple of 32); every group owns one row per iteration, so short rows
// still fill a CTA and one barrier per iteration serves all of them.  Group-wide sums: warp shuffles, one float2 per warp
// in shared memory, one barrier, then every thread adds the partials of its own group's warps.
template <bool RMS, int DT, int VPT>
__global__ void __launch_bounds__(512) k_norm_bwd(const BArgs a, const int gt) {
    using E = Elem<DT>;
    using P = Pairs<DT>;
    constexpr int NE = E::NE, NP = P::NP;                            // the arithmetic runs on packed fp32 pairs
    __shared__ float2 red[2][16];
    pdl_wait();
    pdl_trigger();
    const int t = threadIdx.x, gid = t / gt, lg = t % gt, R = blockDim.x / gt, wg = gt / 32;
    const int warp = t >> 5, lane = t & 31;
    bool valid[VPT];
    F2 gam[VPT][NP], accg[VPT][NP], accb[RMS ? 1 : VPT][NP];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = lg + v * gt < a.nvec;
        P::unpack(valid[v] ? ld_param(a.gamma + lg + v * gt) : make_uint4(0, 0, 0, 0), gam[v]);
#pragma unroll
        for (int i = 0; i < NP; ++i) { accg[v][i] = f2(0.f); if (!RMS) accb[v][i] = f2(0.f); }
    }
    // the packed vectors of the NEXT row are requested before the current row is reduced, so that the reduction of a
    // row does not leave the memory pipe idle
    uint4 nx[VPT], nd[VPT];
    auto request = [&](int64_t row) {
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            const bool ok = valid[v] && row < a.rows;
            nx[v] = ok ? ld_stream(a.x + row * a.nvec + lg + v * gt) : make_uint4(0, 0, 0, 0);
            nd[v] = ok ? ld_stream(a.dy + row * a.nvec + lg + v * gt) : make_uint4(0, 0, 0, 0);
        }
    };
    const int64_t stride = static_cast<int64_t>(gridDim.x) * R;
    request(static_cast<int64_t>(blockIdx.x) * R + gid);
    int it = 0;
    for (int64_t row0 = static_cast<int64_t>(blockIdx.x) * R; row0 < a.rows; row0 += stride, ++it) {      // same trip count for the whole CTA
        const int64_t row = row0 + gid;
        const bool live = row < a.rows;
        const float mu = (RMS || !live) ? 0.f : __ldg(a.mean + row), rs = live ? __ldg(a.rstd + row) : 0.f;
        const F2 mu2 = f2(mu), rs2 = f2(rs);
        F2 xh[VPT][NP], g[VPT][NP], dv[VPT][NP];
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            F2 xv[NP];
            P::unpack(nx[v], xv);
            P::unpack(nd[v], dv[v]);                                     // zeros for absent columns and rows
#pragma unroll
            for (int i = 0; i < NP; ++i) xh[v][i] = (valid[v] && live) ? mul2(sub2(xv[i], mu2), rs2) : f2(0.f);
        }
        request(row + stride);
        F2 sgx2 = f2(0.f), sg2 = f2(0.f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                g[v][i] = mul2(dv[v][i], gam[v][i]);
                sgx2 = fma2(g[v][i], xh[v][i], sgx2);
                sg2 = add2(sg2, g[v][i]);
                accg[v][i] = fma2(dv[v][i], xh[v][i], accg[v][i]);
                if (!RMS) accb[v][i] = add2(accb[v][i], dv[v][i]);
            }
        }
        float sgx = group_reduce<SumOp, 32>(hsum(sgx2));
        float sg = group_reduce<SumOp, 32>(hsum(sg2));
        if (wg > 1) {
            if (lane == 0) red[it & 1][warp] = make_float2(sgx, sg);
            __syncthreads();
            sgx = 0.f; sg = 0.f;
            for (int w = 0; w < wg; ++w) { const float2 p = red[it & 1][gid * wg + w]; sgx += p.x; sg += p.y; }
        }
        const F2 mgx2 = f2(sgx * a.inv_n), mg2 = f2(RMS ? 0.f : sg * a.inv_n);
        if (live) {
            uint4* o = a.dx + row * a.nvec + lg;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                F2 d[NP];
#pragma unroll
                for (int i = 0; i < NP; ++i) d[i] = mul2(rs2, sub2(sub2(g[v][i], mg2), mul2(xh[v][i], mgx2)));
                if (valid[v]) st_stream(o + v * gt, P::pack(d));
            }
        }
    }
    // this row group's partial column sums (zeros if it met no row): part index = CTA * R + group
    float* pg = a.part + (static_cast<int64_t>(blockIdx.x) * R + gid) * (RMS ? 1 : 2) * a.nvec * NE;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        if (!valid[v]) continue;
        const int64_t c0 = static_cast<int64_t>(lg + v * gt) * NE;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            split(accg[v][i], pg[c0 + 2 * i], pg[c0 + 2 * i + 1]);
            if (!RMS) split(accb[v][i], pg[static_cast<int64_t>(a.nvec) * NE + c0 + 2 * i], pg[static_cast<int64_t>(a.nvec) * NE + c0 + 2 * i + 1]);
        }
    }
}

// Rows too long for registers: one CTA per SM keeps its partial column sums in shared memory (every thread owns the
// same columns of every row, so it updates its own entries without synchronisation) and streams each of its rows
// twice with 16-byte loads: once for the two row sums, once more (from L2) for dx and the column sums.
template <bool RMS, int DT>
__global__ void __launch_bounds__(1024) k_norm_bwd_stream(const BArgs a) {
    using E = Elem<DT>;
    constexpr int NE = E::NE, U = 2;
    extern __shared__ __align__(16) float acc[];                  // [LN ? 2 : 1][cols]
    __shared__ float buf[4][32];
    pdl_wait();
    pdl_trigger();
    const int T = blockDim.x, t = threadIdx.x;
    const int64_t cols = static_cast<int64_t>(a.nvec) * NE;
    for (int64_t c = t; c < (RMS ? 1 : 2) * cols; c += T) acc[c] = 0.f;      // own entries only: c = t + k T below as well
    __syncthreads();
    int it = 0;
    for (int64_t row = blockIdx.x; row < a.rows; row += gridDim.x, ++it) {
        const float mu = RMS ? 0.f : __ldg(a.mean + row), rs = __ldg(a.rstd + row);
        const uint4* xr = a.x + row * a.nvec;
        const uint4* dr = a.dy + row * a.nvec;
        float sgx = 0.f, sg = 0.f;
        for (int b0 = t; b0 < a.nvec; b0 += T * U) {
            uint4 rx[U], rd[U], rg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = b0 + u * T < a.nvec;
                rx[u] = ok ? ld_param(xr + b0 + u * T) : make_uint4(0, 0, 0, 0);
                rd[u] = ok ? ld_param(dr + b0 + u * T) : make_uint4(0, 0, 0, 0);
                rg[u] = ok ? ld_param(a.gamma + b0 + u * T) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float xv[NE], dv[NE], gv[NE];
                E::unpack(rx[u], xv); E::unpack(rd[u], dv); E::unpack(rg[u], gv);
                if (b0 + u * T < a.nvec) {
#pragma unroll
                    for (int i = 0; i < NE; ++i) { const float g = dv[i] * gv[i]; sgx = fmaf(g, (xv[i] - mu) * rs, sgx); sg += g; }
                }
            }
        }
        const int slot = (it & 1) * 2;
        const float mgx = cta_reduce<SumOp>(sgx, buf[slot]) * a.inv_n;
        const float mg = RMS ? 0.f : cta_reduce<SumOp>(sg, buf[slot + 1]) * a.inv_n;
        for (int b0 = t; b0 < a.nvec; b0 += T * U) {
            uint4 rx[U], rd[U], rg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool ok = b0 + u * T < a.nvec;
                rx[u] = ok ? ld_stream(xr + b0 + u * T) : make_uint4(0, 0, 0, 0);
                rd[u] = ok ? ld_stream(dr + b0 + u * T) : make_uint4(0, 0, 0, 0);
                rg[u] = ok ? ld_param(a.gamma + b0 + u * T) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (b0 + u * T >= a.nvec) continue;
                float xv[NE], dv[NE], gv[NE], d[NE];
                E::unpack(rx[u], xv); E::unpack(rd[u], dv); E::unpack(rg[u], gv);
                float* ag = acc + (b0 + u * T);                            // element i of vector k lives at [i][k]: lanes hit consecutive banks
#pragma unroll
                for (int i = 0; i < NE; ++i) {
                    const float xh = (xv[i] - mu) * rs, g = dv[i] * gv[i];
                    d[i] = rs * ((g - mg) - xh * mgx);
                    ag[i * a.nvec] = fmaf(dv[i], xh, ag[i * a.nvec]);
                    if (!RMS) ag[cols + i * a.nvec] += dv[i];
                }
                st_stream(a.dx + row * a.nvec + b0 + u * T, E::pack(d));
            }
        }
    }
    float* pg = a.part + static_cast<int64_t>(blockIdx.x) * (RMS ? 1 : 2) * cols;
    for (int b0 = t; b0 < a.nvec; b0 += T)
#pragma unroll
        for (int i = 0; i < NE; ++i) {
            pg[static_cast<int64_t>(b0) * NE + i] = acc[i * a.nvec + b0];
            if (!RMS) pg[cols + static_cast<int64_t>(b0) * NE + i] = acc[cols + i * a.nvec + b0];
        }
}

// Adds the `nparts` partial column sums and rounds once.  A CTA of 32 x 8 threads owns 32 columns: thread (c, y) adds
// parts y, y + 8, ... of column c, the eight slice sums meet in shared memory and are added in slice order -- a fixed
// order of additions whatever the launch, hence deterministic -- and 128 CTAs instead of 16 share the reading.
template <bool RMS, int DT>
__global__ void __launch_bounds__(256) k_colsum_finish(const float* __restrict__ part, typename Elem<DT>::scalar* dgamma,
                                                       typename Elem<DT>::scalar* dbeta, int nparts, int64_t cols) {
    using E = Elem<DT>;
    __shared__ float sm[2][8][32];
    pdl_wait();
    const int c = threadIdx.x & 31, y = threadIdx.x >> 5;
    const int64_t j = static_cast<int64_t>(blockIdx.x) * 32 + c;
    const int64_t stride = (RMS ? 1 : 2) * cols;
    float sg = 0.f, sb = 0.f;
    if (j < cols)
        for (int p = y; p < nparts; p += 8) {
            sg += part[p * stride + j];
            if (!RMS) sb += part[p * stride + cols + j];
        }
    sm[0][y][c] = sg;
    sm[1][y][c] = sb;
    __syncthreads();
    if (y == 0 && j < cols) {
        float tg = 0.f, tb = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) { tg += sm[0][k][c]; tb += sm[1][k][c]; }
        dgamma[j] = E::from_float(tg);
        if (!RMS) dbeta[j] = E::from_float(tb);
    }
}

// ---- any shape, any alignment ------------------------------------------------------------------------------------
template <bool RMS, int DT>
__global__ void __launch_bounds__(256) k_norm_bwd_dx_scalar(const typename Elem<DT>::scalar* x, const typename Elem<DT>::scalar* gamma,
                                                            const typename Elem<DT>::scalar* dy, const float* mean, const float* rstd,
                                                            typename Elem<DT>::scalar* dx, int64_t rows, int64_t cols) {
    using E = Elem<DT>;
    __shared__ float buf[2][32];
    const int64_t row = blockIdx.x;
    if (row >= rows) return;
    const float mu = RMS ? 0.f : mean[row], rs = rstd[row];
    const typename E::scalar* xr = x + row * cols;
    const typename E::scalar* dr = dy + row * cols;
    float sgx = 0.f, sg = 0.f;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float g = E::to_float(dr[j]) * E::to_float(gamma[j]);
        sgx = fmaf(g, (E::to_float(xr[j]) - mu) * rs, sgx);
        sg += g;
    }
    const float inv_n = 1.0f / static_cast<float>(cols);
    const float mgx = cta_reduce<SumOp>(sgx, buf[0]) * inv_n;
    const float mg = RMS ? 0.f : cta_reduce<SumOp>(sg, buf[1]) * inv_n;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float g = E::to_float(dr[j]) * E::to_float(gamma[j]), xh = (E::to_float(xr[j]) - mu) * rs;
        dx[row * cols + j] = E::from_float(rs * ((g - mg) - xh * mgx));
    }
}

template <bool RMS, int DT>
__global__ void __launch_bounds__(256) k_norm_bwd_params_scalar(const typename Elem<DT>::scalar* x, const typename Elem<DT>::scalar* dy,
                                                                const float* mean, const float* rstd, typename Elem<DT>::scalar* dgamma,
                                                                typename Elem<DT>::scalar* dbeta, int64_t rows, int64_t cols) {
    using E = Elem<DT>;
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // a thread per column: coalesced across j
    if (j >= cols) return;
    float sg = 0.f, sb = 0.f;
    for (int64_t r = 0; r < rows; ++r) {
        const float d = E::to_float(dy[r * cols + j]);
        sg = fmaf(d, (E::to_float(x[r * cols + j]) - (RMS ? 0.f : mean[r])) * rstd[r], sg);
        sb += d;
    }
    dgamma[j] = E::from_float(sg);
    if (!RMS) dbeta[j] = E::from_float(sb);
}

bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int sm_count() {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

template <class... T>
cudaError_t launch_pdl(void (*fn)(T...), int64_t grid, int threads, cudaStream_t st, T... args) {
    if (grid > 0x7FFFFFFF) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, args...);
}

// Launch geometry of the register-resident kernel: vectors per thread, threads per row group, row groups per CTA, CTAs.
struct BwdPlan { int vpt, gt, groups, grid; };

template <bool RMS, int DT>
BwdPlan bwd_plan(int64_t rows, int nvec) {
    constexpr int kMaxVpt = Elem<DT>::NE == 4 ? 4 : 2;            // 5 register arrays of VPT * NE fp32 values per thread
    BwdPlan p;
    p.vpt = 1;
    while (p.vpt < kMaxVpt && (nvec + p.vpt - 1) / p.vpt > 256) p.vpt *= 2;     // row groups of up to 256 threads while that holds the row
    p.gt = std::max(32, ((nvec + p.vpt - 1) / p.vpt + 31) / 32 * 32);
    p.groups = std::max(1, std::min(8, 256 / p.gt));                            // short rows: several per CTA
    const int threads = p.gt * p.groups;
    const void* fn = p.vpt == 1 ? reinterpret_cast<const void*>(k_norm_bwd<RMS, DT, 1>)
                   : p.vpt == 2 ? reinterpret_cast<const void*>(k_norm_bwd<RMS, DT, 2>)
                                : reinterpret_cast<const void*>(k_norm_bwd<RMS, DT, kMaxVpt>);
    // as many CTAs as are resident at once: every further CTA would only add partial column sums to write and to add up
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (rows + p.groups - 1) / p.groups;
    p.grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(want, static_cast<int64_t>(per_sm) * sm_count())));
    return p;
}

template <bool RMS, int DT>
tf_status run_bwd(const void* x, const void* gamma, const void* dy, const float* mean, const float* rstd, void* dx, void* dgamma,
                  void* dbeta, void* ws, size_t ws_bytes, int64_t rows, int64_t cols, cudaStream_t st) {
    using S = typename Elem<DT>::scalar;
    constexpr int NE = Elem<DT>::NE;
    const int64_t bytes = cols * Elem<DT>::SIZE;
    const bool aligned = al16(x) && al16(gamma) && al16(dy) && al16(dx) && bytes % 16 == 0;
    constexpr int kMaxVpt = NE == 4 ? 4 : 2;
    cudaError_t e;
    if (aligned && bytes / 16 <= 512 * kMaxVpt && cols <= 0x7FFFFFFF) {
        const int nvec = static_cast<int>(bytes / 16);
        const BwdPlan p = bwd_plan<RMS, DT>(rows, nvec);
        const int parts = p.grid * p.groups;
        const size_t need = static_cast<size_t>(parts) * (RMS ? 1 : 2) * cols * 4;
        if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 3u)) return TF_ERR_INVALID_ARG;
        BArgs a{static_cast<const uint4*>(x), static_cast<const uint4*>(gamma), static_cast<const uint4*>(dy), mean, rstd,
                static_cast<uint4*>(dx), static_cast<float*>(ws), rows, nvec, 1.0f / static_cast<float>(cols)};
        count_launches(2);
        const int threads = p.gt * p.groups;
        if (p.vpt == 1) e = launch_pdl(k_norm_bwd<RMS, DT, 1>, p.grid, threads, st, a, p.gt);
        else if (p.vpt == 2) e = launch_pdl(k_norm_bwd<RMS, DT, 2>, p.grid, threads, st, a, p.gt);
        else e = launch_pdl(k_norm_bwd<RMS, DT, kMaxVpt>, p.grid, threads, st, a, p.gt);
        if (e == cudaSuccess)
            e = launch_pdl(k_colsum_finish<RMS, DT>, (cols + 31) / 32, 256, st, static_cast<const float*>(ws), static_cast<S*>(dgamma),
                           static_cast<S*>(dbeta), parts, cols);
    } else if (aligned && cols <= 0x7FFFFFFF && static_cast<size_t>(RMS ? 1 : 2) * cols * 4 <= 200 * 1024) {
        const int nvec = static_cast<int>(bytes / 16);
        const int grid = static_cast<int>(std::min<int64_t>(rows, sm_count()));          // one CTA per SM: the accumulators fill shared memory
        const size_t smem = static_cast<size_t>(RMS ? 1 : 2) * cols * 4;
        const size_t need = static_cast<size_t>(grid) * smem;
        if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 3u)) return TF_ERR_INVALID_ARG;
        e = cudaFuncSetAttribute(k_norm_bwd_stream<RMS, DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e == cudaSuccess) {
            BArgs a{static_cast<const uint4*>(x), static_cast<const uint4*>(gamma), static_cast<const uint4*>(dy), mean, rstd,
                    static_cast<uint4*>(dx), static_cast<float*>(ws), rows, nvec, 1.0f / static_cast<float>(cols)};
            count_launches(2);
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(grid);
            cfg.blockDim = dim3(1024);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = st;
            e = cudaLaunchKernelEx(&cfg, k_norm_bwd_stream<RMS, DT>, a);
            if (e == cudaSuccess)
                e = launch_pdl(k_colsum_finish<RMS, DT>, (cols + 31) / 32, 256, st, static_cast<const float*>(ws), static_cast<S*>(dgamma),
                               static_cast<S*>(dbeta), grid, cols);
        }
    } else {
        if (rows > 0x7FFFFFFF) return TF_ERR_UNSUPPORTED;
        count_launches(2);
        k_norm_bwd_dx_scalar<RMS, DT><<<static_cast<unsigned>(rows), 256, 0, st>>>(static_cast<const S*>(x), static_cast<const S*>(gamma),
                                                                                  static_cast<const S*>(dy), mean, rstd, static_cast<S*>(dx), rows, cols);
        e = cudaGetLastError();
        if (e == cudaSuccess) {
            k_norm_bwd_params_scalar<RMS, DT><<<static_cast<unsigned>((cols + 255) / 256), 256, 0, st>>>(
                static_cast<const S*>(x), static_cast<const S*>(dy), mean, rstd, static_cast<S*>(dgamma), static_cast<S*>(dbeta), rows, cols);
            e = cudaGetLastError();
        }
    }
    if (e == cudaErrorInvalidConfiguration) return TF_ERR_UNSUPPORTED;
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}

template <bool RMS>
tf_status entry(const void* x, const void* gamma, const void* dy, const float* mean, const float* rstd, void* dx, void* dgamma,
                void* dbeta, void* ws, size_t ws_bytes, int64_t rows, int64_t cols, int dt, void* stream) {
    if (rows < 0 || cols <= 0 || (dt != DT_F32 && dt != DT_BF16)) return TF_ERR_INVALID_ARG;
    if (!gamma || !dgamma || (!RMS && !dbeta)) return TF_ERR_INVALID_ARG;
    if (rows > 0 && (!x || !dy || !dx || !rstd || (!RMS && !mean))) return TF_ERR_INVALID_ARG;
    if (rows > 0 && cols > (INT64_MAX / 8) / rows) return TF_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (rows == 0) {                                              // no rows: the parameter gradients are zero
        const size_t nb = static_cast<size_t>(cols) * elem_size(dt);
        cudaError_t e = cudaMemsetAsync(dgamma, 0, nb, st);
        if (e == cudaSuccess && !RMS) e = cudaMemsetAsync(dbeta, 0, nb, st);
        if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
        return TF_OK;
    }
    return dt == DT_F32 ? run_bwd<RMS, DT_F32>(x, gamma, dy, mean, rstd, dx, dgamma, dbeta, ws, ws_bytes, rows, cols, st)
                        : run_bwd<RMS, DT_BF16>(x, gamma, dy, mean, rstd, dx, dgamma, dbeta, ws, ws_bytes, rows, cols, st);
}

}  // namespace
}  // namespace tf

using namespace tf;

extern "C" size_t tf_norm_bwd_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows <= 0 || cols <= 0 || cols > 0x7FFFFFFF) return 0;
    // the most partial column sums any of the paths may write for this shape, whatever the element type or the op
    int64_t parts = std::min<int64_t>(rows, sm_count());                          // the streamed kernel: one CTA per SM
    if (cols % 4 == 0 && cols / 4 <= 512 * 4) {
        const BwdPlan p = bwd_plan<false, DT_F32>(rows, static_cast<int>(cols / 4)), q = bwd_plan<true, DT_F32>(rows, static_cast<int>(cols / 4));
        parts = std::max<int64_t>(parts, std::max(p.grid * p.groups, q.grid * q.groups));
    }
    if (cols % 8 == 0 && cols / 8 <= 512 * 2) {
        const BwdPlan p = bwd_plan<false, DT_BF16>(rows, static_cast<int>(cols / 8)), q = bwd_plan<true, DT_BF16>(rows, static_cast<int>(cols / 8));
        parts = std::max<int64_t>(parts, std::max(p.grid * p.groups, q.grid * q.groups));
    }
    return static_cast<size_t>(parts) * 2 * static_cast<size_t>(cols) * 4;
}

extern "C" tf_status tf_layernorm_bwd(const void* x, const void* gamma, const void* dy, const float* mean, const float* rstd, void* dx,
                                      void* dgamma, void* dbeta, void* workspace, size_t workspace_bytes, int64_t rows, int64_t cols,
                                      tf_dtype dt, void* stream) {
    return entry<false>(x, gamma, dy, mean, rstd, dx, dgamma, dbeta, workspace, workspace_bytes, rows, cols, dt, stream);
}

extern "C" tf_status tf_rmsnorm_bwd(const void* x, const void* weight, const void* dy, const float* rstd, void* dx, void* dweight,
                                    void* workspace, size_t workspace_bytes, int64_t rows, int64_t cols, tf_dtype dt, void* stream) {
    return entry<true>(x, weight, dy, nullptr, rstd, dx, dweight, nullptr, workspace, workspace_bytes, rows, cols, dt, stream);
}
