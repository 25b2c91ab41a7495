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
// Two forms of that kernel: one requests the next row (and its statistics) into registers before it reduces the current
// one; the other lets bulk copies bring the rows into a shared-memory ring, which keeps more bytes in flight than
// registers can and is what 2-byte rows of 8 KiB and more take.  Both have a specialisation without predicates for
// shapes in which no vector and no row slot is ever absent.
// Rows beyond what 512 threads hold (16 KiB bf16, 32 KiB fp32) are shared by the 2-8 CTAs of a thread-block cluster, each
// the staged form on its slice of the columns, which exchange only the two row sums (up to 65,536 columns).  Where the
// clusters cannot be placed, rows are streamed twice by one CTA per SM that keeps its partial column sums in shared
// memory (up to 200 KiB of them); unaligned tensors, odd widths and wider rows take two plain kernels: scalar passes per
// row for dx, a thread per column for the parameter gradients.
#include <cooperative_groups.h>

#include <algorithm>
#include <cstdio>
#include <vector>
#include <map>
#include <mutex>
#include <tuple>

#include "../../include/tf.h"
#include "tf_common.cuh"

namespace cg = cooperative_groups;

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

// Sum of the wg per-warp partials of a row group, the same bits in every thread of the group.  A power-of-two count is
// added as a butterfly (lane l starts from partial l mod wg; every lane walks the same tree, so all get the same bits):
// one shared-memory read and log2(wg) shuffles instead of wg reads.
__device__ __forceinline__ void group_total(const float2* part, int wg, int lane, float& a, float& b) {
    if ((wg & (wg - 1)) == 0) {
        const float2 p = part[lane & (wg - 1)];
        a = p.x; b = p.y;
        for (int o = wg >> 1; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
            b += __shfl_xor_sync(0xFFFFFFFFu, b, o);
        }
    } else {
        a = 0.f; b = 0.f;
        for (int w = 0; w < wg; ++w) { const float2 p = part[w]; a += p.x; b += p.y; }
    }
}

// A CTA is cut into row groups of `gt` threads (a multiple of 32); every group owns one row per iteration, so short rows
// still fill a CTA and one barrier per iteration serves all of them.  Group-wide sums: warp shuffles, one float2 per warp
// in shared memory, one barrier, then every thread adds the partials of its own group's warps.
// FULL: every thread's vectors exist and every row group meets a row in every iteration, so nothing needs a predicate
// or a zero fill (selects and fills were a quarter of the instructions of the general form).
template <bool RMS, int DT, int VPT, bool FULL>
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
        valid[v] = FULL || lg + v * gt < a.nvec;
        P::unpack(valid[v] ? ld_param(a.gamma + lg + v * gt) : make_uint4(0, 0, 0, 0), gam[v]);
#pragma unroll
        for (int i = 0; i < NP; ++i) { accg[v][i] = f2(0.f); if (!RMS) accb[v][i] = f2(0.f); }
    }
    // the packed vectors of the NEXT row are requested before the current row is reduced, so that the reduction of a
    // row does not leave the memory pipe idle
    uint4 nx[VPT], nd[VPT];
    float nmu = 0.f, nrs = 0.f;                                          // and its statistics: a load at the top of the iteration would stall it
    auto request = [&](int64_t row) {
        const bool in = row < a.rows;
        if (FULL) {                                                      // past the end: keep the stale registers, nobody reads them
            if (in) {
                nmu = RMS ? 0.f : __ldg(a.mean + row);
                nrs = __ldg(a.rstd + row);
#pragma unroll
                for (int v = 0; v < VPT; ++v) {
                    nx[v] = ld_stream(a.x + row * a.nvec + lg + v * gt);
                    nd[v] = ld_stream(a.dy + row * a.nvec + lg + v * gt);
                }
            }
            return;
        }
        nmu = (RMS || !in) ? 0.f : __ldg(a.mean + row);
        nrs = in ? __ldg(a.rstd + row) : 0.f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            const bool ok = valid[v] && in;
            nx[v] = ok ? ld_stream(a.x + row * a.nvec + lg + v * gt) : make_uint4(0, 0, 0, 0);
            nd[v] = ok ? ld_stream(a.dy + row * a.nvec + lg + v * gt) : make_uint4(0, 0, 0, 0);
        }
    };
    const int64_t stride = static_cast<int64_t>(gridDim.x) * R;
    request(static_cast<int64_t>(blockIdx.x) * R + gid);
    int it = 0;
    for (int64_t row0 = static_cast<int64_t>(blockIdx.x) * R; row0 < a.rows; row0 += stride, ++it) {      // same trip count for the whole CTA
        const int64_t row = row0 + gid;
        const bool live = FULL || row < a.rows;
        const float rs = nrs;
        const F2 mu2 = f2(nmu), rs2 = f2(rs);
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
            group_total(red[it & 1] + gid * wg, wg, lane, sgx, sg);
        }
        // dx = rstd g - rstd mean(g) - xh rstd mean(g xh): two fused multiply-adds per pair
        const F2 c1 = f2(-rs * (sgx * a.inv_n)), c0 = f2(RMS ? 0.f : -rs * (sg * a.inv_n));
        if (live) {
            uint4* o = a.dx + row * a.nvec + lg;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                F2 d[NP];
#pragma unroll
                for (int i = 0; i < NP; ++i) d[i] = fma2(xh[v][i], c1, fma2(g[v][i], rs2, c0));
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

// Staged form of the same kernel: the tile of R consecutive rows that the CTA's row groups take per iteration is one
// contiguous range of x and one of dy, so it arrives in a shared-memory ring stage by two bulk copies (no multicast)
// counted on the stage's mbarrier.  The bytes in flight are then the ring (64-128 KiB per CTA) and not the one row that
// registers can request ahead, which is what held the register form of the 2-byte types below the copy rate.  The
// barrier of the row reduction is also the point after which every thread has taken its vectors out of the stage, so
// thread 0 refills that stage right behind it; no producer warp, no "empty" barrier.  Waits are bounded: a CTA that
// gives up sets the status word, stops issuing copies and finishes its loop without waiting again.
constexpr int kBwdMaxStages = 8;

// The two row sums of a group of wg warps with half the shuffles of two separate reductions: after the first exchange
// the even lanes carry the first sum and the odd lanes the second, each over its lane pair, and the remaining steps keep
// that parity.  Per-warp partials meet in `red` (2 * warps floats: first and second sum of warp w at 2w and 2w + 1;
// RMSNorm has one sum, at w); after a barrier the partials of a power-of-two number of warps are added as a butterfly, so
// every thread of the group gets the same bits.
template <bool RMS>
__device__ __forceinline__ void warp_sums_store(float sgx, float sg, float* red, int warp, int lane) {
    constexpr unsigned kAll = 0xFFFFFFFFu;
    if constexpr (RMS) {
        sgx = group_reduce<SumOp, 32>(sgx);
        if (lane == 0) red[warp] = sgx;
    } else {
        const bool odd = lane & 1;
        float v = (odd ? sg : sgx) + __shfl_xor_sync(kAll, odd ? sgx : sg, 1);
#pragma unroll
        for (int o = 2; o < 32; o <<= 1) v += __shfl_xor_sync(kAll, v, o);
        if (lane < 2) red[2 * warp + lane] = v;
    }
}
template <bool RMS>
__device__ __forceinline__ void group_sums_load(float& sgx, float& sg, const float* red, int wg, int gid, int lane) {
    constexpr unsigned kAll = 0xFFFFFFFFu;
    if constexpr (RMS) {
        if ((wg & (wg - 1)) == 0) {
            sgx = red[gid * wg + (lane & (wg - 1))];
            for (int o = wg >> 1; o > 0; o >>= 1) sgx += __shfl_xor_sync(kAll, sgx, o);
        } else {
            sgx = 0.f;
            for (int w = 0; w < wg; ++w) sgx += red[gid * wg + w];
        }
        sg = 0.f;
    } else {
        const bool odd = lane & 1;
        float v;
        if ((wg & (wg - 1)) == 0) {
            v = red[2 * gid * wg + (lane & (2 * wg - 1))];
            for (int o = wg; o > 1; o >>= 1) v += __shfl_xor_sync(kAll, v, o);
        } else {
            v = 0.f;
            for (int w = 0; w < wg; ++w) v += red[2 * (gid * wg + w) + (odd ? 1 : 0)];
        }
        const float u = __shfl_xor_sync(kAll, v, 1);
        sgx = odd ? u : v;
        sg = odd ? v : u;
    }
}

template <bool RMS, int DT, int VPT, bool FULL>
__global__ void __launch_bounds__(512) k_norm_bwd_staged(const BArgs a, const int gt, const int S, int* status) {
    using P = Pairs<DT>;
    constexpr int NE = Elem<DT>::NE, NP = P::NP;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full[kBwdMaxStages];
    __shared__ float red[2][32];
    const int t = threadIdx.x, gid = t / gt, lg = t - gid * gt, R = blockDim.x / gt, wg = gt >> 5;
    const int warp = t >> 5, lane = t & 31;
    const uint32_t tile_vecs = static_cast<uint32_t>(R) * a.nvec;             // vectors of x (and of dy) per stage
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem);                    // [S][x | dy][R][nvec]
    const int64_t num_tiles = (a.rows + R - 1) / R;
    // this CTA's tiles: blockIdx.x, + gridDim.x, ...; the loop below counts them instead of comparing 64-bit row numbers
    const int n_iters = blockIdx.x < num_tiles ? static_cast<int>((num_tiles - 1 - blockIdx.x) / gridDim.x) + 1 : 0;
    if (t == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
        mbar_fence_init();
    }
    pdl_wait();
    auto issue = [&](int k, int s) {                                           // thread 0 only: this CTA's k-th tile into stage s
        const int64_t row0 = (blockIdx.x + static_cast<int64_t>(k) * gridDim.x) * R;
        const uint32_t bytes = static_cast<uint32_t>(min(static_cast<int64_t>(R), a.rows - row0)) * a.nvec * 16u;
        mbar_expect_tx(&full[s], 2u * bytes);
        bulk_g2s(ring + tile_vecs * (2 * s), a.x + row0 * a.nvec, bytes, &full[s]);
        bulk_g2s(ring + tile_vecs * (2 * s + 1), a.dy + row0 * a.nvec, bytes, &full[s]);
    };
    if (t == 0)
        for (int s = 0; s < S && s < n_iters; ++s) issue(s, s);
    bool valid[VPT];
    F2 gam[VPT][NP], accg[VPT][NP], accb[RMS ? 1 : VPT][NP];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = FULL || lg + v * gt < a.nvec;
        P::unpack(valid[v] ? ld_param(a.gamma + lg + v * gt) : make_uint4(0, 0, 0, 0), gam[v]);
#pragma unroll
        for (int i = 0; i < NP; ++i) { accg[v][i] = f2(0.f); if (!RMS) accb[v][i] = f2(0.f); }
    }
    __syncthreads();                                                           // barriers initialised
    pdl_trigger();
    bool failed = false;
    int s = 0;
    uint32_t parity = 0, stage_vecs = 0;                                       // stage s starts at vector 2 s tile_vecs of the ring
    // everything that moves with the row advances by one stride per iteration: the row number, the statistics, dx
    int64_t row = static_cast<int64_t>(blockIdx.x) * R + gid;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * R;
    const float* pmean = RMS ? nullptr : a.mean + row;
    const float* prstd = a.rstd + row;
    uint4* o = a.dx + row * a.nvec + lg;
    const int64_t ostride = stride * a.nvec;
    const uint32_t mine = static_cast<uint32_t>(gid) * a.nvec + lg;
    float nmu = 0.f, nrs = 0.f;                                                // the statistics of a row are requested one tile ahead
    if (n_iters > 0 && (FULL || row < a.rows)) { nmu = RMS ? 0.f : __ldg(pmean); nrs = __ldg(prstd); }
    for (int it = 0; it < n_iters; ++it) {                                     // same trip count for the whole CTA
        if (!failed && !mbar_wait(&full[s], parity)) {
            failed = true;
            atomicExch(status, 4);
            mbar_wait(&full[s], parity);                                       // one more bounded wait for the copies
        }
        const bool live = FULL || row < a.rows;
        const float rs = nrs;
        const F2 mu2 = f2(nmu), rs2 = f2(rs);
        prstd += stride;
        if (!RMS) pmean += stride;
        if (it + 1 < n_iters && (FULL || row + stride < a.rows)) { nmu = RMS ? 0.f : __ldg(pmean); nrs = __ldg(prstd); }
        const uint4* sx = ring + stage_vecs + mine;
        const uint4* sd = sx + tile_vecs;
        F2 xh[VPT][NP], g[VPT][NP], dv[VPT][NP];
        F2 sgx2 = f2(0.f), sg2 = f2(0.f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            const bool ok = valid[v] && live;                                  // rows past the end were not copied
            F2 xv[NP];
            P::unpack(ok ? sx[v * gt] : make_uint4(0, 0, 0, 0), xv);
            P::unpack(ok ? sd[v * gt] : make_uint4(0, 0, 0, 0), dv[v]);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                xh[v][i] = ok ? mul2(sub2(xv[i], mu2), rs2) : f2(0.f);
                g[v][i] = mul2(dv[v][i], gam[v][i]);
                sgx2 = fma2(g[v][i], xh[v][i], sgx2);
                if (!RMS) sg2 = add2(sg2, g[v][i]);
                accg[v][i] = fma2(dv[v][i], xh[v][i], accg[v][i]);
                if (!RMS) accb[v][i] = add2(accb[v][i], dv[v][i]);
            }
        }
        float sgx = hsum(sgx2), sg = RMS ? 0.f : hsum(sg2);
        warp_sums_store<RMS>(sgx, sg, red[it & 1], warp, lane);
        __syncthreads();                                                       // also: every thread has left the stage
        if (t == 0 && !failed && it + S < n_iters) issue(it + S, s);
        group_sums_load<RMS>(sgx, sg, red[it & 1], wg, gid, lane);
        // dx = rstd g - rstd mean(g) - xh rstd mean(g xh): two fused multiply-adds per pair
        const F2 c1 = f2(-rs * (sgx * a.inv_n)), c0 = f2(RMS ? 0.f : -rs * (sg * a.inv_n));
        if (live) {
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                F2 d[NP];
#pragma unroll
                for (int i = 0; i < NP; ++i) d[i] = fma2(xh[v][i], c1, fma2(g[v][i], rs2, c0));
                if (valid[v]) st_stream(o + v * gt, P::pack(d));
            }
        }
        row += stride;
        o += ostride;
        stage_vecs += 2 * tile_vecs;
        if (++s == S) { s = 0; parity ^= 1u; stage_vecs = 0; }
    }
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

// Rows too long for one CTA's registers: a thread-block cluster of `cs` CTAs shares each row.  Every CTA is the staged
// kernel above on its own slice of the columns (its slice of gamma and of the parameter-gradient accumulators in
// registers, its slice of the row in its own ring); the only thing the CTAs of a row owe each other is the pair of row
// sums, which each pushes into every peer's shared memory with an asynchronous store counted on the receiver's mbarrier.
// There is no cluster barrier inside the loop; a peer can be at most one row ahead (it needs this CTA's sums to finish
// a row), so two slot buffers suffice, and every CTA has received all pushes of its last row before it leaves.
__device__ __forceinline__ void push_sums(float* slot, uint64_t* bar, uint32_t rank, float a, float b) {
    uint32_t rslot, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rslot) : "r"(smem_u32(slot)), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_u32(bar)), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(rslot), "f"(a), "f"(b), "r"(rbar) : "memory");
}

template <bool RMS, int DT, int VPT, bool FULL>
__global__ void __launch_bounds__(512) k_norm_bwd_cluster(const BArgs a, const int cs, const int S, int* status) {
    using P = Pairs<DT>;
    constexpr int NE = Elem<DT>::NE, NP = P::NP;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full[kBwdMaxStages];
    __shared__ __align__(8) uint64_t xbar[2];                     // the sums of a row have all arrived (by row parity)
    __shared__ __align__(8) float xch[2][kMaxCluster][2];
    __shared__ float2 red[2][16];
    const int t = threadIdx.x, gt = blockDim.x, wg = gt / 32, warp = t >> 5, lane = t & 31;
    const int rank = static_cast<int>(blockIdx.x % cs);
    const int64_t cluster_id = blockIdx.x / cs, num_clusters = gridDim.x / cs;
    const int per = (a.nvec + cs - 1) / cs;                        // vectors per slice
    const int first = rank * per;
    const int len = max(0, min(per, a.nvec - first));
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem);        // [S][x | dy][per]
    cg::cluster_group cl = cg::this_cluster();
    if (t == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
        mbar_init(&xbar[0], 1);
        mbar_init(&xbar[1], 1);
        mbar_fence_init();
    }
    pdl_wait();
    auto issue = [&](int64_t row, int s) {                         // thread 0 only
        if (len == 0) return;
        const uint32_t bytes = static_cast<uint32_t>(len) * 16u;
        mbar_expect_tx(&full[s], 2u * bytes);
        bulk_g2s(ring + static_cast<size_t>(per) * (2 * s), a.x + row * a.nvec + first, bytes, &full[s]);
        bulk_g2s(ring + static_cast<size_t>(per) * (2 * s + 1), a.dy + row * a.nvec + first, bytes, &full[s]);
    };
    if (t == 0)
        for (int s = 0; s < S; ++s) {
            const int64_t row = cluster_id + static_cast<int64_t>(s) * num_clusters;
            if (row < a.rows) issue(row, s);
        }
    bool valid[VPT];
    F2 gam[VPT][NP], accg[VPT][NP], accb[RMS ? 1 : VPT][NP];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        valid[v] = FULL || t + v * gt < len;
        P::unpack(valid[v] ? ld_param(a.gamma + first + t + v * gt) : make_uint4(0, 0, 0, 0), gam[v]);
#pragma unroll
        for (int i = 0; i < NP; ++i) { accg[v][i] = f2(0.f); if (!RMS) accb[v][i] = f2(0.f); }
    }
    __syncthreads();
    cl.sync();                     // every CTA of the cluster is resident, its barriers initialised, before any remote store
    bool failed = false;
    int it = 0, s = 0;
    uint32_t parity = 0;
    float nmu = 0.f, nrs = 0.f;
    auto request_stats = [&](int64_t row) {
        if (row < a.rows) { nmu = RMS ? 0.f : __ldg(a.mean + row); nrs = __ldg(a.rstd + row); }
    };
    request_stats(cluster_id);
    for (int64_t row = cluster_id; row < a.rows; row += num_clusters, ++it) {          // same trip count for the whole cluster
        if (len > 0 && !failed && !mbar_wait(&full[s], parity)) {
            failed = true;
            atomicExch(status, 4);
            mbar_wait(&full[s], parity);                                       // one more bounded wait for the copies
        }
        const float rs = nrs;
        const F2 mu2 = f2(nmu), rs2 = f2(rs);
        request_stats(row + num_clusters);
        const uint4* sx = ring + static_cast<size_t>(per) * (2 * s) + t;
        const uint4* sd = sx + per;
        F2 xh[VPT][NP], g[VPT][NP], dv[VPT][NP];
        F2 sgx2 = f2(0.f), sg2 = f2(0.f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            F2 xv[NP];
            P::unpack(valid[v] ? sx[v * gt] : make_uint4(0, 0, 0, 0), xv);
            P::unpack(valid[v] ? sd[v * gt] : make_uint4(0, 0, 0, 0), dv[v]);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                xh[v][i] = valid[v] ? mul2(sub2(xv[i], mu2), rs2) : f2(0.f);
                g[v][i] = mul2(dv[v][i], gam[v][i]);
                sgx2 = fma2(g[v][i], xh[v][i], sgx2);
                sg2 = add2(sg2, g[v][i]);
                accg[v][i] = fma2(dv[v][i], xh[v][i], accg[v][i]);
                if (!RMS) accb[v][i] = add2(accb[v][i], dv[v][i]);
            }
        }
        float sgx = group_reduce<SumOp, 32>(hsum(sgx2));
        float sg = group_reduce<SumOp, 32>(hsum(sg2));
        const int xb = it & 1;
        if (lane == 0) red[xb][warp] = make_float2(sgx, sg);
        __syncthreads();                                                       // also: every thread has left the stage
        const int64_t next = row + static_cast<int64_t>(S) * num_clusters;
        if (t == 0 && !failed && next < a.rows) issue(next, s);
        if (wg > 1) group_total(red[xb], wg, lane, sgx, sg);                   // this CTA's sums, the same bits in every thread
        if (t == 0) mbar_expect_tx(&xbar[xb], static_cast<uint32_t>(cs) * 8u);
        if (t < cs) push_sums(&xch[xb][rank][0], &xbar[xb], static_cast<uint32_t>(t), sgx, sg);
        if (!failed && !mbar_wait(&xbar[xb], static_cast<uint32_t>(it >> 1) & 1u)) { failed = true; atomicExch(status, 4); }
        sgx = 0.f; sg = 0.f;
        for (int k = 0; k < cs; ++k) { sgx += xch[xb][k][0]; sg += xch[xb][k][1]; }     // rank order: the same bits in every CTA
        const F2 c1 = f2(-rs * (sgx * a.inv_n)), c0 = f2(RMS ? 0.f : -rs * (sg * a.inv_n));
        uint4* o = a.dx + row * a.nvec + first + t;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            F2 d[NP];
#pragma unroll
            for (int i = 0; i < NP; ++i) d[i] = fma2(xh[v][i], c1, fma2(g[v][i], rs2, c0));
            if (valid[v]) st_stream(o + v * gt, P::pack(d));
        }
        if (++s == S) { s = 0; parity ^= 1u; }
    }
    cl.sync();                     // nobody leaves while a peer (one that gave up waiting, say) may still push into its shared memory
    // this cluster's partial column sums: CTA `rank` owns columns [first, first + len) of part `cluster_id`
    float* pg = a.part + cluster_id * (RMS ? 1 : 2) * a.nvec * NE;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        if (!valid[v]) continue;
        const int64_t c0 = static_cast<int64_t>(first + t + v * gt) * NE;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            split(accg[v][i], pg[c0 + 2 * i], pg[c0 + 2 * i + 1]);
            if (!RMS) split(accb[v][i], pg[static_cast<int64_t>(a.nvec) * NE + c0 + 2 * i], pg[static_cast<int64_t>(a.nvec) * NE + c0 + 2 * i + 1]);
        }
    }
}

// Rows too long for that as well (or a device without room for the clusters): one CTA per SM keeps its partial column
// sums in shared memory (every thread owns the same columns of every row, so it updates its own entries without
// synchronisation) and streams each of its rows twice with 16-byte loads: once for the two row sums, once more (from
// L2) for dx and the column sums.
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

// Adds the `nparts` partial column sums and rounds once.  A part is one row of [dgamma | dbeta] partials (RMSNorm: the
// first alone), `width` floats; a CTA of 32 x ny threads owns 32 V consecutive positions: thread (c, y) adds parts y,
// y + ny, ... of its V positions on four independent accumulators (four reads in flight per thread: the reads, from L2,
// are what the kernel waits for -- a thread per column that walked its parts one after the other took 11-33 us on the
// training shapes, a sixth to a third of the whole call), the ny slice sums meet in shared memory and are added in slice
// order.  The order of the additions is fixed whatever the launch, hence deterministic.  V = 4 (16-byte reads; width a
// multiple of 4, so a thread's positions never straddle the two halves) is for parts wide enough to fill the GPU that
// way; ny (8, 16 or 32) follows the number of parts.
template <int V> struct FinishVec;
template <> struct FinishVec<1> {
    static __device__ __forceinline__ void add(float (&a)[1], const float* p) { a[0] += *p; }
};
template <> struct FinishVec<4> {
    static __device__ __forceinline__ void add(float (&a)[4], const float* p) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        a[0] += v.x; a[1] += v.y; a[2] += v.z; a[3] += v.w;
    }
};
template <bool RMS, int DT, int V>
__global__ void __launch_bounds__(1024) k_colsum_finish(const float* __restrict__ part, typename Elem<DT>::scalar* dgamma,
                                                        typename Elem<DT>::scalar* dbeta, int nparts, int64_t cols) {
    using E = Elem<DT>;
    __shared__ float sm[32][32 * V + 1];
    pdl_wait();
    const int c = threadIdx.x & 31, y = threadIdx.x >> 5, ny = blockDim.x >> 5;
    const int64_t width = (RMS ? 1 : 2) * cols;
    const int64_t j0 = (static_cast<int64_t>(blockIdx.x) * 32 + c) * V;
    float acc[4][V];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < V; ++v) acc[u][v] = 0.f;
    if (j0 < width) {
        const int64_t step = ny * width;
        const float* p = part + y * width + j0;
        int k = y;
        for (; k + 3 * ny < nparts; k += 4 * ny, p += 4 * step) {
            FinishVec<V>::add(acc[0], p);
            FinishVec<V>::add(acc[1], p + step);
            FinishVec<V>::add(acc[2], p + 2 * step);
            FinishVec<V>::add(acc[3], p + 3 * step);
        }
        if (k < nparts) FinishVec<V>::add(acc[0], p);
        if (k + ny < nparts) FinishVec<V>::add(acc[1], p + step);
        if (k + 2 * ny < nparts) FinishVec<V>::add(acc[2], p + 2 * step);
    }
#pragma unroll
    for (int v = 0; v < V; ++v) sm[y][c * V + v] = (acc[0][v] + acc[1][v]) + (acc[2][v] + acc[3][v]);
    __syncthreads();
    const int64_t j = static_cast<int64_t>(blockIdx.x) * 32 * V + threadIdx.x;          // one position per thread of the first 32 V
    if (threadIdx.x < 32 * V && j < width) {
        float t = 0.f;
        for (int k = 0; k < ny; ++k) t += sm[k][threadIdx.x];
        if (j < cols) dgamma[j] = E::from_float(t);
        else dbeta[j - cols] = E::from_float(t);
    }
}

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

template <bool RMS, int DT>
cudaError_t launch_finish(const void* ws, void* dgamma, void* dbeta, int nparts, int64_t cols, cudaStream_t st) {
    using S = typename Elem<DT>::scalar;
    const int64_t width = (RMS ? 1 : 2) * cols;
    const int ny = nparts >= 256 ? 32 : nparts >= 128 ? 16 : 8;
    // 16-byte reads: a workspace aligned for them, parts that keep the alignment, and two CTAs of 128 positions per SM and more
    const bool wide = (reinterpret_cast<uintptr_t>(ws) & 15u) == 0 && width % 4 == 0 && width >= static_cast<int64_t>(256) * sm_count();
    if (wide)
        return launch_pdl(k_colsum_finish<RMS, DT, 4>, (width + 127) / 128, 32 * ny, st, static_cast<const float*>(ws), static_cast<S*>(dgamma),
                          static_cast<S*>(dbeta), nparts, cols);
    return launch_pdl(k_colsum_finish<RMS, DT, 1>, (width + 31) / 32, 32 * ny, st, static_cast<const float*>(ws), static_cast<S*>(dgamma),
                      static_cast<S*>(dbeta), nparts, cols);
}

// Test and bench hook: 0 = automatic, 1 = the register form, 2 = the staged form with row groups of up to 512 threads,
// 3 = the staged form with row groups of up to 256 threads; stages 0 = automatic.
// path: 0 automatic, 1 register form, 2 / 3 / 4 staged form with row groups of up to 512 / 256 / 64 threads; stages: ring
// depth (0 automatic); cluster: 0 automatic, 1 never, 2 / 4 / 8 that many CTAs per row.
struct BwdChoice { int path, stages, cluster; };
BwdChoice g_force{0, 0, 0};                                    // the hook
thread_local const BwdChoice* t_override = nullptr;            // the tuner, while it times a candidate
std::mutex g_tuned_mu;
std::map<std::tuple<int, int, int64_t, int64_t, int>, BwdChoice> g_tuned;        // (rms, dt, rows, cols, device) -> what tf_tune_norm_bwd kept

// forced > tuned > automatic
BwdChoice current_choice(bool rms, int dt, int64_t rows, int64_t cols) {
    if (t_override) return *t_override;
    if (g_force.path || g_force.stages || g_force.cluster) return g_force;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lk(g_tuned_mu);
    const auto it = g_tuned.find(std::make_tuple(rms ? 1 : 0, dt, rows, cols, dev));
    return it == g_tuned.end() ? BwdChoice{0, 0, 0} : it->second;
}
int staged_gmax(int path) { return path == 2 ? 512 : path == 3 ? 256 : 64; }

// Launch geometry of the row-group kernels: vectors per thread, threads per row group, row groups per CTA, CTAs; for
// the staged form also the ring's stages and bytes (stages = 0: the register form).
struct BwdPlan { int vpt, gt, groups, grid, stages; size_t smem; bool full; };

template <bool RMS, int DT, int VPT> const void* bwd_fn(bool staged, bool full) {
    return staged ? (full ? reinterpret_cast<const void*>(k_norm_bwd_staged<RMS, DT, VPT, true>) : reinterpret_cast<const void*>(k_norm_bwd_staged<RMS, DT, VPT, false>))
           : full ? reinterpret_cast<const void*>(k_norm_bwd<RMS, DT, VPT, true>) : reinterpret_cast<const void*>(k_norm_bwd<RMS, DT, VPT, false>);
}

template <bool RMS, int DT>
BwdPlan bwd_plan(int64_t rows, int nvec, bool staged, int stages, int gmax = 256) {
    constexpr int kMaxVpt = Elem<DT>::NE == 4 ? 4 : 2;            // 5 register arrays of VPT * NE fp32 values per thread
    BwdPlan p{};
    p.vpt = 1;
    while (p.vpt < kMaxVpt && (nvec + p.vpt - 1) / p.vpt > gmax) p.vpt *= 2;    // row groups of up to gmax threads while that holds the row
    p.gt = std::max(32, ((nvec + p.vpt - 1) / p.vpt + 31) / 32 * 32);
    p.groups = std::max(1, std::min(8, 128 / p.gt));                            // short rows: several per CTA (CTAs of 128 threads measured best)
    const int threads = p.gt * p.groups;
    p.full = nvec == p.gt * p.vpt && rows % p.groups == 0;          // no vector and no row slot is ever absent
    const void* fn = p.vpt == 1 ? bwd_fn<RMS, DT, 1>(staged, p.full) : p.vpt == 2 ? bwd_fn<RMS, DT, 2>(staged, p.full) : bwd_fn<RMS, DT, kMaxVpt>(staged, p.full);
    if (staged) {
        // ring: the shared memory of an SM divided among the CTAs its register file holds (at most three), up to eight stages
        const size_t stage = static_cast<size_t>(2) * p.groups * nvec * 16;
        int by_regs = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&by_regs, fn, threads, 0) != cudaSuccess || by_regs < 1) by_regs = 1;
        by_regs = std::min(by_regs, 3);
        while (by_regs > 1 && (216 * 1024 / by_regs) / stage < 2) --by_regs;
        // three stages are enough (deeper rings measured a few percent slower)
        p.stages = stages > 0 ? stages : static_cast<int>(std::min<size_t>(3, (216 * 1024 / by_regs) / stage));
        p.stages = std::min(p.stages, kBwdMaxStages);
        p.smem = stage * p.stages;
        if (p.stages < 2 || p.smem > 216 * 1024 ||
            cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024) != cudaSuccess) {      // the same limit for every shape
            p.stages = 0; p.grid = 0; return p;                                         // does not fit: not available
        }
    }
    // as many CTAs as are resident at once: every further CTA would only add partial column sums to write and to add up
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, p.smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (rows + p.groups - 1) / p.groups;
    p.grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(want, static_cast<int64_t>(per_sm) * sm_count())));
    return p;
}

// Which form runs, unless the hook says otherwise: the staged one for 2-byte elements in rows of 2 KiB and more, two
// vectors per thread (measured 7-15 % faster there: a row ahead in registers is half as many bytes in flight as with
// 4-byte elements), the register form elsewhere (shorter rows and 4-byte elements: equal or faster).
template <bool RMS, int DT>
BwdPlan choose_bwd_plan_uncached(int64_t rows, int nvec, const BwdChoice& c) {
    const bool want = c.path >= 2 || (c.path == 0 && DT == DT_BF16 && nvec >= 128);
    if (want) {
        const BwdPlan p = bwd_plan<RMS, DT>(rows, nvec, true, c.stages, staged_gmax(c.path));
        if (p.stages >= 2) return p;
    }
    return bwd_plan<RMS, DT>(rows, nvec, false, 0);
}

template <bool RMS, int DT>
BwdPlan choose_bwd_plan(int64_t rows, int nvec, const BwdChoice& c) {
    // the plan of the last shape is kept (per thread): the occupancy queries cost more host time than a launch
    struct Key { int64_t rows; int nvec, path, stages, dev; };
    thread_local Key last{-1, 0, 0, 0, -1};
    thread_local BwdPlan kept{};
    int dev = 0;
    cudaGetDevice(&dev);
    if (last.rows == rows && last.nvec == nvec && last.path == c.path && last.stages == c.stages && last.dev == dev) return kept;
    last = Key{rows, nvec, c.path, c.stages, dev};
    kept = choose_bwd_plan_uncached<RMS, DT>(rows, nvec, c);
    return kept;
}

// Cluster split-row form: CTAs per row, threads, vectors per thread, ring stages, clusters resident at once.
struct ClusterPlan { int cs, threads, vpt, stages, clusters; size_t smem; bool full; };

template <bool RMS, int DT, int VPT> const void* cluster_fn(bool full) {
    return full ? reinterpret_cast<const void*>(k_norm_bwd_cluster<RMS, DT, VPT, true>) : reinterpret_cast<const void*>(k_norm_bwd_cluster<RMS, DT, VPT, false>);
}

void cluster_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, const ClusterPlan& p, int clusters, cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(static_cast<unsigned>(clusters) * p.cs);
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = p.smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;          // no programmatic early launch: persistent clusters must all be placed at once
    attr[0].val.clusterDim.x = p.cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

template <bool RMS, int DT>
ClusterPlan cluster_plan(int64_t rows, int nvec, int cs_forced, int stages) {
    constexpr int kMaxVpt = Elem<DT>::NE == 4 ? 4 : 2;
    ClusterPlan p{};
    int cs = cs_forced > 1 ? cs_forced : 2;
    // the fewest CTAs whose slices are at most 1024 vectors (2-byte elements) or 1536 (4-byte): the exchange costs about
    // as much per row whatever the slice, so large slices amortise it, up to what leaves a CTA enough registers; and
    // rather four CTAs with the largest slices than eight (clusters of eight leave SMs of a GPC unused).  Read off what
    // tf_tune_norm_bwd keeps on rows of 12-64 Ki columns.
    const int slice_cap = Elem<DT>::NE == 4 ? 1536 : 1024;
    while (cs_forced <= 1 && cs < kMaxCluster && (nvec + cs - 1) / cs > slice_cap) cs *= 2;
    if (cs_forced <= 1 && cs == 8 && (nvec + 3) / 4 <= 512 * kMaxVpt) cs = 4;
    const int per = (nvec + cs - 1) / cs;
    if (per > 512 * kMaxVpt) return p;                                                                // clusters = 0: not available
    p.cs = cs;
    p.vpt = 1;
    while (p.vpt < kMaxVpt && (per + p.vpt - 1) / p.vpt > 512) p.vpt *= 2;
    p.threads = std::max(32, ((per + p.vpt - 1) / p.vpt + 31) / 32 * 32);
    p.full = nvec % cs == 0 && per == p.threads * p.vpt;
    const size_t stage = static_cast<size_t>(2) * per * 16;
    p.stages = stages > 0 ? stages : 2;                           // two stages: what the tuner keeps for every cluster shape
    p.smem = stage * p.stages;
    if (p.stages < 2 || p.stages > kBwdMaxStages || p.smem > 216 * 1024) return p;
    const void* fn = p.vpt == 1 ? cluster_fn<RMS, DT, 1>(p.full) : p.vpt == 2 ? cluster_fn<RMS, DT, 2>(p.full) : cluster_fn<RMS, DT, kMaxVpt>(p.full);
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024) != cudaSuccess) { cudaGetLastError(); return p; }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    cluster_config(cfg, attr, p, sm_count(), nullptr);
    int fit = 0;                                                   // clusters cannot straddle GPCs: ask how many are resident at once
    if (cudaOccupancyMaxActiveClusters(&fit, fn, &cfg) != cudaSuccess) { cudaGetLastError(); return p; }
    p.clusters = static_cast<int>(std::min<int64_t>(rows, std::min(fit, sm_count())));      // the workspace is sized for one part per SM
    return p;
}

template <bool RMS, int DT>
ClusterPlan choose_cluster_plan(int64_t rows, int nvec, const BwdChoice& c) {          // the last shape's plan is kept, like the row-group plan
    struct Key { int64_t rows; int nvec, cs, stages, dev; };
    thread_local Key last{-1, 0, 0, 0, -1};
    thread_local ClusterPlan kept{};
    int dev = 0;
    cudaGetDevice(&dev);
    if (last.rows == rows && last.nvec == nvec && last.cs == c.cluster && last.stages == c.stages && last.dev == dev) return kept;
    last = Key{rows, nvec, c.cluster, c.stages, dev};
    kept = cluster_plan<RMS, DT>(rows, nvec, c.cluster, c.stages);
    return kept;
}

template <bool RMS, int DT>
cudaError_t launch_cluster(const ClusterPlan& p, const BArgs& a, int* status, cudaStream_t st) {
    constexpr int kMaxVpt = Elem<DT>::NE == 4 ? 4 : 2;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    cluster_config(cfg, attr, p, p.clusters, st);
#define TF_CL(V, F) cudaLaunchKernelEx(&cfg, k_norm_bwd_cluster<RMS, DT, V, F>, a, p.cs, p.stages, status)
    if (p.full) return p.vpt == 1 ? TF_CL(1, true) : p.vpt == 2 ? TF_CL(2, true) : TF_CL(kMaxVpt, true);
    return p.vpt == 1 ? TF_CL(1, false) : p.vpt == 2 ? TF_CL(2, false) : TF_CL(kMaxVpt, false);
#undef TF_CL
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
    // a cluster per row: rows beyond one CTA's registers (or wherever the hook asks for it)
    const BwdChoice c = current_choice(RMS, DT, rows, cols);
    ClusterPlan cp{};
    if (aligned && cols <= 0x7FFFFFFF && c.cluster != 1 && (c.cluster > 1 || bytes / 16 > 512 * kMaxVpt) &&
        bytes / 16 <= static_cast<int64_t>(kMaxCluster) * 512 * kMaxVpt)
        cp = choose_cluster_plan<RMS, DT>(rows, static_cast<int>(bytes / 16), c);
    if (cp.clusters > 0) {
        const int nvec = static_cast<int>(bytes / 16);
        const size_t need = static_cast<size_t>(cp.clusters) * (RMS ? 1 : 2) * cols * 4;
        if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 3u)) return TF_ERR_INVALID_ARG;
        int* status = device_status_word();
        if (!status) return TF_ERR_CUDA;
        BArgs a{static_cast<const uint4*>(x), static_cast<const uint4*>(gamma), static_cast<const uint4*>(dy), mean, rstd,
                static_cast<uint4*>(dx), static_cast<float*>(ws), rows, nvec, 1.0f / static_cast<float>(cols)};
        count_launches(2);
        e = launch_cluster<RMS, DT>(cp, a, status, st);
        if (e == cudaSuccess)
            e = launch_finish<RMS, DT>(ws, dgamma, dbeta, cp.clusters, cols, st);
    } else if (aligned && bytes / 16 <= 512 * kMaxVpt && cols <= 0x7FFFFFFF) {
        const int nvec = static_cast<int>(bytes / 16);
        const BwdPlan p = choose_bwd_plan<RMS, DT>(rows, nvec, c);
        const int parts = p.grid * p.groups;
        const size_t need = static_cast<size_t>(parts) * (RMS ? 1 : 2) * cols * 4;
        if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 3u)) return TF_ERR_INVALID_ARG;
        BArgs a{static_cast<const uint4*>(x), static_cast<const uint4*>(gamma), static_cast<const uint4*>(dy), mean, rstd,
                static_cast<uint4*>(dx), static_cast<float*>(ws), rows, nvec, 1.0f / static_cast<float>(cols)};
        count_launches(2);
        const int threads = p.gt * p.groups;
        if (p.stages >= 2) {
            int* status = device_status_word();
            if (!status) return TF_ERR_CUDA;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(p.grid);
            cfg.blockDim = dim3(threads);
            cfg.dynamicSmemBytes = p.smem;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (p.full) {
                if (p.vpt == 1) e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, 1, true>, a, p.gt, p.stages, status);
                else if (p.vpt == 2) e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, 2, true>, a, p.gt, p.stages, status);
                else e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, kMaxVpt, true>, a, p.gt, p.stages, status);
            } else if (p.vpt == 1) e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, 1, false>, a, p.gt, p.stages, status);
            else if (p.vpt == 2) e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, 2, false>, a, p.gt, p.stages, status);
            else e = cudaLaunchKernelEx(&cfg, k_norm_bwd_staged<RMS, DT, kMaxVpt, false>, a, p.gt, p.stages, status);
        } else if (p.full) {
            if (p.vpt == 1) e = launch_pdl(k_norm_bwd<RMS, DT, 1, true>, p.grid, threads, st, a, p.gt);
            else if (p.vpt == 2) e = launch_pdl(k_norm_bwd<RMS, DT, 2, true>, p.grid, threads, st, a, p.gt);
            else e = launch_pdl(k_norm_bwd<RMS, DT, kMaxVpt, true>, p.grid, threads, st, a, p.gt);
        } else if (p.vpt == 1) e = launch_pdl(k_norm_bwd<RMS, DT, 1, false>, p.grid, threads, st, a, p.gt);
        else if (p.vpt == 2) e = launch_pdl(k_norm_bwd<RMS, DT, 2, false>, p.grid, threads, st, a, p.gt);
        else e = launch_pdl(k_norm_bwd<RMS, DT, kMaxVpt, false>, p.grid, threads, st, a, p.gt);
        if (e == cudaSuccess)
            e = launch_finish<RMS, DT>(ws, dgamma, dbeta, parts, cols, st);
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
                e = launch_finish<RMS, DT>(ws, dgamma, dbeta, grid, cols, st);
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
    // the most partial column sums any of the paths may write for this shape, whatever the element type, the op or the
    // form (automatic, tuned or forced): every group width, and the ring depths that leave room for the most CTAs
    int64_t parts = std::min<int64_t>(rows, sm_count());                          // the streamed kernel and the clusters: at most one part per SM
    auto widest = [&](auto plan) {
        for (int stages : {2, 3, g_force.stages})
            for (int form = 0; form < 4; ++form) {
                const BwdPlan p = plan(form != 0, form == 1 ? 512 : form == 2 ? 256 : 64, stages);
                parts = std::max<int64_t>(parts, static_cast<int64_t>(p.grid) * p.groups);
            }
    };
    if (cols % 4 == 0 && cols / 4 <= 512 * 4) {
        const int nvec = static_cast<int>(cols / 4);
        widest([&](bool sg, int gmax, int st) { return bwd_plan<false, DT_F32>(rows, nvec, sg, st, sg ? gmax : 256); });
        widest([&](bool sg, int gmax, int st) { return bwd_plan<true, DT_F32>(rows, nvec, sg, st, sg ? gmax : 256); });
    }
    if (cols % 8 == 0 && cols / 8 <= 512 * 2) {
        const int nvec = static_cast<int>(cols / 8);
        widest([&](bool sg, int gmax, int st) { return bwd_plan<false, DT_BF16>(rows, nvec, sg, st, sg ? gmax : 256); });
        widest([&](bool sg, int gmax, int st) { return bwd_plan<true, DT_BF16>(rows, nvec, sg, st, sg ? gmax : 256); });
    }
    return static_cast<size_t>(parts) * 2 * static_cast<size_t>(cols) * 4;
}

extern "C" tf_status tf_norm_bwd_force(int path, int stages, int cluster) {
    if (path < 0 || path > 4 || stages < 0 || stages > kBwdMaxStages) return TF_ERR_INVALID_ARG;
    if (cluster != 0 && cluster != 1 && cluster != 2 && cluster != 4 && cluster != 8) return TF_ERR_INVALID_ARG;
    g_force = BwdChoice{path, stages, cluster};
    return TF_OK;
}

namespace tf {
void clear_norm_bwd_tuned() {
    std::lock_guard<std::mutex> lk(g_tuned_mu);
    g_tuned.clear();
}
}  // namespace tf

namespace tf {
namespace {

__global__ void k_fill_pattern(uint32_t* p, int64_t words, uint32_t seed, uint32_t base, uint32_t mask) {
    // finite values of either element type: a fixed exponent field (`base`) with hashed low bits (`mask`)
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < words; i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        uint32_t h = static_cast<uint32_t>(i) * 2654435761u + seed;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        p[i] = base | (h & mask);
    }
}
__global__ void k_fill_float(float* p, int64_t n, float v) {
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * blockDim.x) p[i] = v;
}

struct TuneScratch {
    std::vector<void*> ptrs;
    ~TuneScratch() { for (void* p : ptrs) cudaFree(p); }
    void* get(size_t bytes) {
        void* p = nullptr;
        if (cudaMalloc(&p, std::max<size_t>(bytes, 16)) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        ptrs.push_back(p);
        return p;
    }
};

thread_local int t_bwd_timed = 0;
thread_local float t_bwd_auto_us = 0.f, t_bwd_best_us = 0.f;

}  // namespace
}  // namespace tf

// The measure-and-keep loop (Algorithm 1 of the paper, as in tf_tune) over the forms of the norm backward pass: the
// automatic choice is the incumbent; every other form that can run the shape is launched (BuildRun: it must launch and
// no bounded wait may give up), timed (Profile: 3 warm-up + 5 timed batches over rotating buffers, CUDA events, median)
// and kept only if it is more than 2 % faster (Arbiter).  The winner is remembered for (op, rows, cols, type, device).
extern "C" tf_status tf_tune_norm_bwd(tf_op op_, int64_t rows, int64_t cols, tf_dtype dt_) {
    const int op = op_, dt = dt_;
    if ((op != OP_LAYERNORM && op != OP_RMSNORM) || rows <= 0 || cols <= 0 || (dt != DT_F32 && dt != DT_BF16)) return TF_ERR_INVALID_ARG;
    if (cols > 0x7FFFFFFF || cols > (INT64_MAX / 8) / rows) return TF_ERR_UNSUPPORTED;
    const bool rms = op == OP_RMSNORM;
    const int es = elem_size(dt);
    t_bwd_timed = 0; t_bwd_auto_us = 0.f; t_bwd_best_us = 0.f;
    if ((cols * es) % 16 != 0) return TF_OK;                     // only the plain kernels serve such rows: nothing to choose
    const int64_t nvec = cols * es / 16;
    const int kMaxVpt = dt == DT_F32 ? 4 : 2;
    const size_t tensor_bytes = static_cast<size_t>(rows) * cols * es;
    const int K = static_cast<int>(std::min<size_t>(16, std::max<size_t>(2, (256u << 20) / (3 * tensor_bytes) + 1)));
    TuneScratch sc;
    std::vector<void*> xs(K), dys(K), dxs(K);
    for (int k = 0; k < K; ++k) { xs[k] = sc.get(tensor_bytes); dys[k] = sc.get(tensor_bytes); dxs[k] = sc.get(tensor_bytes); if (!xs[k] || !dys[k] || !dxs[k]) return TF_ERR_NOMEM; }
    void* gamma = sc.get(static_cast<size_t>(cols) * es);
    void* dgamma = sc.get(static_cast<size_t>(cols) * es);
    void* dbeta = sc.get(static_cast<size_t>(cols) * es);
    float* mean = static_cast<float*>(sc.get(static_cast<size_t>(rows) * 4));
    float* rstd = static_cast<float*>(sc.get(static_cast<size_t>(rows) * 4));
    const size_t ws_bytes = tf_norm_bwd_workspace_bytes(rows, cols);
    void* ws = sc.get(ws_bytes);
    int* status = device_status_word();
    if (!gamma || !dgamma || !dbeta || !mean || !rstd || !ws || !status) return TF_ERR_NOMEM;
    cudaStream_t st = nullptr;
    cudaEvent_t ev[2] = {nullptr, nullptr};
    if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) return TF_ERR_CUDA;
    auto cleanup = [&]() { if (ev[0]) cudaEventDestroy(ev[0]); if (ev[1]) cudaEventDestroy(ev[1]); cudaStreamDestroy(st); t_override = nullptr; };
    if (cudaEventCreate(&ev[0]) != cudaSuccess || cudaEventCreate(&ev[1]) != cudaSuccess) { cleanup(); return TF_ERR_CUDA; }
    // values in [1, 2) (fp32) / [1, 2) in both halves (bf16): the kernels have no data-dependent control flow
    const uint32_t base = dt == DT_F32 ? 0x3F800000u : 0x3F803F80u, mask = dt == DT_F32 ? 0x007FFFFFu : 0x007F007Fu;
    for (int k = 0; k < K; ++k) {
        k_fill_pattern<<<1024, 256, 0, st>>>(static_cast<uint32_t*>(xs[k]), static_cast<int64_t>(tensor_bytes / 4), 17u * k + 1, base, mask);
        k_fill_pattern<<<1024, 256, 0, st>>>(static_cast<uint32_t*>(dys[k]), static_cast<int64_t>(tensor_bytes / 4), 31u * k + 7, base, mask);
    }
    k_fill_pattern<<<64, 256, 0, st>>>(static_cast<uint32_t*>(gamma), static_cast<int64_t>(cols) * es / 4, 5u, base, mask);
    k_fill_float<<<256, 256, 0, st>>>(mean, rows, 1.5f);
    k_fill_float<<<256, 256, 0, st>>>(rstd, rows, 2.0f);
    if (cudaStreamSynchronize(st) != cudaSuccess) { cleanup(); return TF_ERR_CUDA; }

    auto call = [&](int k) {
        return rms ? tf_rmsnorm_bwd(xs[k], gamma, dys[k], rstd, dxs[k], dgamma, ws, ws_bytes, rows, cols, dt_, st)
                   : tf_layernorm_bwd(xs[k], gamma, dys[k], mean, rstd, dxs[k], dgamma, dbeta, ws, ws_bytes, rows, cols, dt_, st);
    };
    auto profile = [&](const BwdChoice& c, float* us) -> bool {
        t_override = &c;
        bool ok = true;
        float t[5];
        for (int rep = 0; rep < 8 && ok; ++rep) {
            if (rep >= 3) cudaEventRecord(ev[0], st);
            for (int k = 0; k < K && ok; ++k) ok = call(k) == TF_OK;
            if (rep >= 3) {
                cudaEventRecord(ev[1], st);
                if (cudaEventSynchronize(ev[1]) != cudaSuccess) ok = false;
                float ms = 0.f;
                cudaEventElapsedTime(&ms, ev[0], ev[1]);
                t[rep - 3] = ms * 1000.f / K;
            }
        }
        t_override = nullptr;
        if (cudaStreamSynchronize(st) != cudaSuccess) ok = false;
        int flag = 0;                                             // a bounded wait gave up: the candidate is dropped
        if (cudaMemcpy(&flag, status, sizeof flag, cudaMemcpyDeviceToHost) != cudaSuccess) ok = false;
        if (flag != 0) { cudaMemset(status, 0, sizeof flag); ok = false; }
        if (!ok) { cudaGetLastError(); return false; }
        std::sort(t, t + 5);
        *us = t[2];
        ++t_bwd_timed;
        return true;
    };

    std::vector<BwdChoice> cands;
    if (nvec <= 512 * kMaxVpt) {                                  // one CTA can hold the row
        cands.push_back(BwdChoice{1, 0, 1});
        for (int path : {2, 3, 4})
            for (int stages : {2, 3}) cands.push_back(BwdChoice{path, stages, 1});
    }
    for (int cs : {2, 4, 8})
        if ((nvec + cs - 1) / cs <= 512 * kMaxVpt && nvec >= 512)                // clusters from 8 KiB rows on
            for (int stages : {2, 3}) cands.push_back(BwdChoice{0, stages, cs});
    const BwdChoice automatic{0, 0, 0};
    float best_us = 0.f;
    if (!profile(automatic, &best_us)) { cleanup(); return TF_ERR_CUDA; }
    t_bwd_auto_us = best_us;
    BwdChoice best = automatic;
    for (const BwdChoice& c : cands) {
        float us = 0.f;
        if (!profile(c, &us)) continue;
        if (us < 0.98f * best_us) { best = c; best_us = us; }
    }
    t_bwd_best_us = best_us;
    cleanup();
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lk(g_tuned_mu);
    g_tuned[std::make_tuple(rms ? 1 : 0, dt, rows, cols, dev)] = best;
    return TF_OK;
}

extern "C" tf_status tf_tune_norm_bwd_report(int* candidates_timed, float* automatic_us, float* best_us) {
    if (candidates_timed) *candidates_timed = t_bwd_timed;
    if (automatic_us) *automatic_us = t_bwd_auto_us;
    if (best_us) *best_us = t_bwd_best_us;
    return TF_OK;
}

extern "C" tf_status tf_norm_bwd_choice(tf_op op_, int64_t rows, int64_t cols, tf_dtype dt_, char* buf, size_t n) {
    const int op = op_, dt = dt_;
    if ((op != OP_LAYERNORM && op != OP_RMSNORM) || rows < 0 || cols <= 0 || (dt != DT_F32 && dt != DT_BF16) || !buf || n == 0) return TF_ERR_INVALID_ARG;
    const BwdChoice c = current_choice(op == OP_RMSNORM, dt, rows, cols);
    snprintf(buf, n, "path=%d,stages=%d,cluster=%d", c.path, c.stages, c.cluster);
    return TF_OK;
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
