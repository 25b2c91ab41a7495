// Batched vector-matrix product of the paper's Case Study 2:  C[m,n] = sum_k A[m,k] * B[m,n,k].
//
// B ([M, N, K], k contiguous) is read exactly once and dominates the traffic, so this is a streamed reduction bound by
// HBM (every element of B meets one multiply-add).  Viewed as M*N rows of length K, each row is dotted with the vector
// A[m,:] of its batch entry.  Measured on B200: the B stream alone runs at about 7.0 TB/s, and what holds a kernel below
// that is the traffic of the A pieces through L1/L2, one 16-byte A load for every 16-byte B load when each row fetches
// its own.  So both paths below let one A load serve several rows:
//   plain path (fp32, and bf16 when forced): a group of 4..32 lanes owns R consecutive n of one m; per step it loads
//     U vectors of A[m,:] once and the matching vectors of its R rows, accumulates in packed fp32 pairs, reduces with
//     shuffles, writes R elements of C;
//   tensor-core path (bf16): a warp owns RT tiles of 16 consecutive n and feeds m16n8k16 multiply-accumulates straight
//     from the packed words it loaded (see below).
// One contiguous block of rows per CTA, as many CTAs as there are blocks.
#include <algorithm>

#include "../../include/tf.h"
#include "tf_common.cuh"

namespace tf {
namespace {

// Lane group of LANES lanes, R rows, U vectors per row and step.  All loops have warp-uniform trip counts.
// ksplit > 1 (LANES = 32 only): that many warps of the CTA share a row group, each taking every ksplit-th step, and
// combine through shared memory -- for few, long rows, which would otherwise leave the SMs short of warps.
// KS = false compiles the split away (constant strides matter for the short rows, which issue everything at once).
template <int DT, int LANES, int R, int U, bool KS>
__global__ void __launch_bounds__(1024) k_vecmat(const uint4* __restrict__ A, const uint4* __restrict__ B,
                                                 typename Elem<DT>::scalar* __restrict__ C, int64_t N, int kvec, int tiles_per_m, int64_t tiles,
                                                 int ksplit_arg) {
    using P = Pairs<DT>;
    constexpr int NP = P::NP;
    __shared__ float part[KS ? 32 : 1][R];
    const int ksplit = KS ? ksplit_arg : 1;
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x % LANES;
    const int group = threadIdx.x / LANES, kw = group % ksplit;
    const int64_t tile = static_cast<int64_t>(blockIdx.x) * (blockDim.x / LANES / ksplit) + group / ksplit;
    const bool tile_live = tile < tiles;                          // every lane runs the loop: shuffles need the whole warp
    const int64_t m = tile_live ? tile / tiles_per_m : 0;
    const int64_t n0 = tile_live ? (tile - m * tiles_per_m) * R : 0;
    const int64_t out = m * N + n0;
    const int n_left = tile_live ? static_cast<int>(N - n0 < R ? N - n0 : R) : 0;
    const uint4* a = A + m * kvec;
    const uint4* b[R];
#pragma unroll
    for (int r = 0; r < R; ++r) b[r] = B + (out + (r < n_left ? r : 0)) * kvec;
    F2 acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = f2(0.f);
    const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll(R == 2 ? 2 : 1)                                  // measured: R = 2 gains from a second step in flight, R = 1 and 4 lose occupancy
    for (int v0 = kw * LANES * U + lane; v0 < kvec; v0 += LANES * U * ksplit) {
        uint4 bv[R][U], av[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * LANES;
            const bool ok = v < kvec;
            av[u] = ok && tile_live ? ld_param(a + v) : zero;
#pragma unroll
            for (int r = 0; r < R; ++r) bv[r][u] = ok && r < n_left ? ld_stream(b[r] + v) : zero;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            F2 y[NP];
            P::unpack(av[u], y);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                F2 x[NP];
                P::unpack(bv[r][u], x);
#pragma unroll
                for (int i = 0; i < NP; ++i) acc[r] = fma2(x[i], y[i], acc[r]);
            }
        }
    }
    float dot[R];
#pragma unroll
    for (int r = 0; r < R; ++r) dot[r] = group_reduce<SumOp, LANES>(hsum(acc[r]));
    if (!KS) {
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (r < n_left) C[out + r] = Elem<DT>::from_float(dot[r]);
        }
        return;
    }
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) part[group][r] = dot[r];
    }
    __syncthreads();
    if (kw == 0 && lane < n_left) {
        float sum = 0.f;
        for (int i = 0; i < ksplit; ++i) sum += part[group + i][lane];
        C[out + lane] = Elem<DT>::from_float(sum);
    }
}

// bf16 through the tensor cores.  Unpacking bf16 pairs and issuing fp32 multiply-adds per element costs instruction
// slots that a 7 TB/s stream does not leave; m16n8k16 multiply-accumulates take the packed pairs as they arrive.
// A warp owns RT tiles of 16 consecutive n of one batch entry.  Lane (g, t) = (lane / 4, lane % 4) loads 16-byte vectors
// of rows g and g + 8 of each tile and the matching vector of A[m,:]; since a sum over k does not care which k sits in
// which slot of the fragment, the four 32-bit words of a vector serve directly as the (k-slot 2t, 2t+8) words of two
// fragments, and the words of the A[m,:] vector, the same for every g, as the column operand: every output column holds
// the same dot product and column 0 is kept.  Products are exact in fp32; each step's four multiply-accumulates start
// from zero and the step totals are added in ordinary fp32, so the result does not lean on how the tensor core rounds
// long chains.  With few tiles, `ksplit` warps of a CTA share a tile group along k and combine through shared memory.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int WARPS, int RT>
__global__ void __launch_bounds__(WARPS * 32) k_vecmat_mma(const uint4* __restrict__ A, const uint4* __restrict__ B, uint16_t* __restrict__ C,
                                                           int64_t N, int kvec, int ksplit, int tiles_per_m, int64_t tiles) {
    constexpr int ROWS = 16 * RT;                                 // n per warp
    __shared__ float part[WARPS][ROWS];
    pdl_wait();
    pdl_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t tile = static_cast<int64_t>(blockIdx.x) * (WARPS / ksplit) + warp / ksplit;
    const int kw = warp % ksplit;
    const bool tile_live = tile < tiles;
    const int64_t m = tile_live ? tile / tiles_per_m : 0;
    const int64_t n0 = tile_live ? (tile - m * tiles_per_m) * ROWS : 0;
    const int64_t out = m * N + n0;
    const int n_left = tile_live ? static_cast<int>(N - n0 < ROWS ? N - n0 : ROWS) : 0;
    const uint4* a = A + m * kvec;
    const uint4* b[RT][2];                                        // row g + 8*h of tile q is local row 16*q + 8*h + g
#pragma unroll
    for (int q = 0; q < RT; ++q)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = 16 * q + 8 * h + g;
            b[q][h] = B + (out + (row < n_left ? row : 0)) * kvec;
        }
    const uint4 zero = make_uint4(0, 0, 0, 0);
    float acc[RT][2];
#pragma unroll
    for (int q = 0; q < RT; ++q) acc[q][0] = acc[q][1] = 0.f;
    const int steps = (kvec + 7) / 8;                             // a step is 8 vectors = 64 elements of every row
#pragma unroll 2
    for (int s = kw; s < steps; s += ksplit) {                    // trip count is the same for every lane of a warp
        uint4 r[RT][2][2], v[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int vi = s * 8 + j * 4 + t;
            const bool ok = vi < kvec;
            v[j] = ok && tile_live ? ld_param(a + vi) : zero;
#pragma unroll
            for (int q = 0; q < RT; ++q)
#pragma unroll
                for (int h = 0; h < 2; ++h) r[q][h][j] = ok && 16 * q + 8 * h + g < n_left ? ld_stream(b[q][h] + vi) : zero;
        }
#pragma unroll
        for (int q = 0; q < RT; ++q) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                mma_bf16_16816(c, r[q][0][j].x, r[q][1][j].x, r[q][0][j].y, r[q][1][j].y, v[j].x, v[j].y);
                mma_bf16_16816(c, r[q][0][j].z, r[q][1][j].z, r[q][0][j].w, r[q][1][j].w, v[j].z, v[j].w);
            }
            acc[q][0] += c[0];
            acc[q][1] += c[2];
        }
    }
    if (ksplit == 1) {
        if (t == 0) {
#pragma unroll
            for (int q = 0; q < RT; ++q)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int row = 16 * q + 8 * h + g;
                    if (row < n_left) C[out + row] = Elem<DT_BF16>::from_float(acc[q][h]);
                }
        }
        return;                                                   // uniform over the CTA: ksplit is a launch constant
    }
    if (t == 0) {
#pragma unroll
        for (int q = 0; q < RT; ++q)
#pragma unroll
            for (int h = 0; h < 2; ++h) part[warp][16 * q + 8 * h + g] = acc[q][h];
    }
    __syncthreads();
    if (kw == 0) {
        for (int row = lane; row < n_left; row += 32) {
            float sum = 0.f;
            for (int i = 0; i < ksplit; ++i) sum += part[warp + i][row];
            C[out + row] = Elem<DT_BF16>::from_float(sum);
        }
    }
}

// Long rows, staged: the register paths above read a long row 128 B at a time per warp and step, from 16 rows that
// lie kilobytes apart; here a producer lane copies 1 KiB of each of a tile's 16 rows (and of A[m,:]) per stage into a
// four-stage shared-memory ring with bulk copies (no multicast), so that memory sees long contiguous reads and the
// bytes in flight (three CTAs x 72 KiB per SM) cost no registers; four consumer warps take the stage apart.
// bf16: every warp multiplies a quarter of the chunk for all 16 rows through m16n8k16 (fragments read from shared
// memory; rows are padded by 64 B so that a quarter-warp's 16-byte reads hit distinct banks) and the four partial
// sums meet in shared memory at the end.  fp32: every warp owns four rows.  Every wait is bounded: on expiry the CTA
// sets the library's status word, stops waiting and finishes with uniform control flow.
constexpr int kTmRows = 16, kTmChunk = 1024, kTmPad = 64, kTmStages = 4;
constexpr int kTmRowStride = kTmChunk + kTmPad;
constexpr int kTmStageBytes = kTmRows * kTmRowStride + kTmChunk;
constexpr int kTmThreads = 160;                                   // four consumer warps and the producer's warp

template <int DT>
__global__ void __launch_bounds__(kTmThreads) k_vecmat_tma(const unsigned char* __restrict__ A, const unsigned char* __restrict__ B,
                                                           typename Elem<DT>::scalar* __restrict__ C, int64_t N, int64_t row_bytes,
                                                           int tiles_per_m, int* status) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t full[kTmStages], empty[kTmStages];
    __shared__ float part[4][kTmRows];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tile = blockIdx.x;
    const int64_t m = tile / tiles_per_m, n0 = (tile - m * tiles_per_m) * kTmRows;
    const int n_left = static_cast<int>(N - n0 < kTmRows ? N - n0 : kTmRows);
    const int steps = static_cast<int>((row_bytes + kTmChunk - 1) / kTmChunk);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTmStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 4); }
        mbar_fence_init();
    }
    pdl_wait();
    __syncthreads();
    pdl_trigger();
    float out0 = 0.f, out1 = 0.f;                                 // bf16: rows g and g + 8 of this warp's k quarter
    F2 acc[4] = {f2(0.f), f2(0.f), f2(0.f), f2(0.f)};              // fp32: this warp's four rows
    if (warp == 4) {
        // the producer's warp: lane 0 waits for the stage to be free and announces the bytes, then lanes 0..n_left-1 each
        // copy their row's piece and lane 16 the piece of A[m,:] (one lane issuing all 17 copies was the bottleneck)
        const unsigned char* a = A + m * row_bytes;
        const unsigned char* b = B + (m * N + n0) * row_bytes;
        int issued = 0;
        for (int s = 0; s < steps; ++s) {
            const int st = s % kTmStages;
            int ok = 1;
            if (lane == 0 && s >= kTmStages && !mbar_wait(&empty[st], static_cast<uint32_t>(s / kTmStages - 1) & 1u)) { atomicExch(status, 4); ok = 0; }
            ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
            if (!ok) break;                                           // uniform over the warp
            const int64_t off = static_cast<int64_t>(s) * kTmChunk;
            const uint32_t bytes = static_cast<uint32_t>(row_bytes - off < kTmChunk ? row_bytes - off : kTmChunk);
            unsigned char* dst = ring + st * kTmStageBytes;
            if (lane == 0) mbar_expect_tx(&full[st], bytes * static_cast<uint32_t>(n_left + 1));
            __syncwarp();
            if (lane < n_left) bulk_g2s(dst + lane * kTmRowStride, b + lane * row_bytes + off, bytes, &full[st]);
            if (lane == 16) bulk_g2s(dst + kTmRows * kTmRowStride, a + off, bytes, &full[st]);
            issued = s + 1;
        }
        // no copy may still be in flight when the CTA ends, even if the consumers gave up: poll (bounded) the barriers
        // of the last stages that were fed
        if (lane == 0)
            for (int s = issued > kTmStages ? issued - kTmStages : 0; s < issued; ++s)
                if (!mbar_wait(&full[s % kTmStages], static_cast<uint32_t>(s / kTmStages) & 1u)) { atomicExch(status, 4); break; }
    } else {
        bool failed = false;
        const int g = lane >> 2, t = lane & 3;
        for (int s = 0; s < steps; ++s) {
            const int st = s % kTmStages;
            if (!failed && !mbar_wait(&full[st], static_cast<uint32_t>(s / kTmStages) & 1u)) { failed = true; atomicExch(status, 4); }
            const int64_t off = static_cast<int64_t>(s) * kTmChunk;
            const int nv = static_cast<int>((row_bytes - off < kTmChunk ? row_bytes - off : kTmChunk) / 16);     // vectors of this chunk
            const unsigned char* src = ring + st * kTmStageBytes;
            const uint4 zero = make_uint4(0, 0, 0, 0);
            if (!failed) {
                if constexpr (DT == DT_BF16) {
                    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int vi = warp * 16 + j * 4 + t;                          // this warp's quarter of the chunk
                        const bool ok = vi < nv;
                        const uint4 r0 = ok && g < n_left ? *reinterpret_cast<const uint4*>(src + g * kTmRowStride + vi * 16) : zero;
                        const uint4 r1 = ok && g + 8 < n_left ? *reinterpret_cast<const uint4*>(src + (g + 8) * kTmRowStride + vi * 16) : zero;
                        const uint4 v = ok ? *reinterpret_cast<const uint4*>(src + kTmRows * kTmRowStride + vi * 16) : zero;
                        mma_bf16_16816(c, r0.x, r1.x, r0.y, r1.y, v.x, v.y);
                        mma_bf16_16816(c, r0.z, r1.z, r0.w, r1.w, v.z, v.w);
                    }
                    out0 += c[0];
                    out1 += c[2];
                } else {
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int vi = lane + 32 * u;
                        if (vi < nv) {
                            F2 y[2];
                            Pairs<DT_F32>::unpack(*reinterpret_cast<const uint4*>(src + kTmRows * kTmRowStride + vi * 16), y);
#pragma unroll
                            for (int r = 0; r < 4; ++r) {
                                if (warp * 4 + r < n_left) {
                                    F2 x[2];
                                    Pairs<DT_F32>::unpack(*reinterpret_cast<const uint4*>(src + (warp * 4 + r) * kTmRowStride + vi * 16), x);
                                    acc[r] = fma2(x[0], y[0], acc[r]);
                                    acc[r] = fma2(x[1], y[1], acc[r]);
                                }
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);               // also after a failure: the producer must not be left waiting
        }
        if constexpr (DT == DT_BF16) {
            if (t == 0) { part[warp][g] = out0; part[warp][g + 8] = out1; }
        } else {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float dot = group_reduce<SumOp, 32>(hsum(acc[r]));
                if (lane == 0 && warp * 4 + r < n_left) C[m * N + n0 + warp * 4 + r] = Elem<DT>::from_float(dot);
            }
        }
    }
    __syncthreads();
    if (DT == DT_BF16 && warp == 0 && lane < n_left)
        C[m * N + n0 + lane] = Elem<DT>::from_float((part[0][lane] + part[1][lane]) + (part[2][lane] + part[3][lane]));
}

// Any alignment, any K: a warp per row, scalar accesses.
template <int DT>
__global__ void __launch_bounds__(1024) k_vecmat_scalar(const typename Elem<DT>::scalar* A, const typename Elem<DT>::scalar* B,
                                                        typename Elem<DT>::scalar* C, int64_t rows, int64_t N, int64_t K) {
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const int64_t r = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const bool live = r < rows;
    const int64_t rr = live ? r : 0;
    float acc = 0.f;
    for (int64_t k = lane; k < K; k += 32) acc = fmaf(E::to_float(B[rr * K + k]), E::to_float(A[(rr / N) * K + k]), acc);
    acc = group_reduce<SumOp, 32>(acc);
    if (live && lane == 0) C[r] = E::from_float(acc);
}

bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

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

int sm_count() {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

// Warps wanted: about four waves of fully occupied SMs, so that the last, partly filled wave is a small part of the
// run (the partial-wave tail that the paper's case study removes with a tunable grid).
int64_t warps_wanted(int sms) { return 4LL * 64 * sms; }


template <int DT, int LANES, int R>
cudaError_t launch_plain_lr(int threads, int ksplit, cudaStream_t st, const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t kvec) {
    constexpr int U = R == 1 ? 4 : R == 2 ? 2 : 1;
    using S = typename Elem<DT>::scalar;
    const int64_t tiles_per_m = (N + R - 1) / R, tiles = M * tiles_per_m;
    if (tiles_per_m > 0x7FFFFFFF || kvec > 0x7FFFFFF0) return cudaErrorInvalidConfiguration;
    if (LANES < 32) ksplit = 1;
    while (ksplit > 1 && ksplit * 32 > threads) ksplit /= 2;
    const int gpc = threads / LANES / ksplit;
    if (LANES == 32 && ksplit > 1)
        return launch_pdl(k_vecmat<DT, LANES, R, U, (LANES == 32)>, (tiles + gpc - 1) / gpc, threads, st, static_cast<const uint4*>(A),
                          static_cast<const uint4*>(B), static_cast<S*>(C), N, static_cast<int>(kvec), static_cast<int>(tiles_per_m), tiles, ksplit);
    return launch_pdl(k_vecmat<DT, LANES, R, U, false>, (tiles + gpc - 1) / gpc, threads, st, static_cast<const uint4*>(A),
                      static_cast<const uint4*>(B), static_cast<S*>(C), N, static_cast<int>(kvec), static_cast<int>(tiles_per_m), tiles, 1);
}

template <int DT, int LANES>
cudaError_t launch_plain_l(int rows, int threads, int ksplit, cudaStream_t st, const void* A, const void* B, void* C, int64_t M, int64_t N,
                           int64_t kvec) {
    switch (rows) {
        case 1: return launch_plain_lr<DT, LANES, 1>(threads, ksplit, st, A, B, C, M, N, kvec);
        case 2: return launch_plain_lr<DT, LANES, 2>(threads, ksplit, st, A, B, C, M, N, kvec);
        default: return launch_plain_lr<DT, LANES, 4>(threads, ksplit, st, A, B, C, M, N, kvec);
    }
}

template <int DT>
cudaError_t launch_plain(int lanes, int rows, int ksplit, int threads, cudaStream_t st, const void* A, const void* B, void* C, int64_t M,
                         int64_t N, int64_t kvec) {
    const int sms = sm_count();
    // Measured on the K sweep: rows of up to 4 KiB run best with two rows per group sharing each A load and two
    // vectors per lane and step; longer rows with one row per group and four vectors in flight per lane.
    if (lanes == 0) lanes = kvec <= 8 ? 4 : kvec <= 16 ? 8 : kvec <= 32 ? 16 : 32;
    if (rows == 0) rows = (kvec <= 256 && N >= 2 && M * ((N + 1) / 2) * lanes / 32 >= warps_wanted(sms) / 4) ? 2 : 1;
    if (ksplit == 0) {                                            // few long rows: cut k until about one wave of warps exists
        const int64_t groups = M * ((N + rows - 1) / rows);
        const int64_t steps = kvec / (32 * (rows == 1 ? 4 : rows == 2 ? 2 : 1));
        ksplit = 1;
        while (lanes == 32 && ksplit < 8 && ksplit * 64 <= threads && groups * ksplit < 64LL * sms && steps >= 4 * ksplit) ksplit *= 2;
    }
    switch (lanes) {
        case 4: return launch_plain_l<DT, 4>(rows, threads, ksplit, st, A, B, C, M, N, kvec);
        case 8: return launch_plain_l<DT, 8>(rows, threads, ksplit, st, A, B, C, M, N, kvec);
        case 16: return launch_plain_l<DT, 16>(rows, threads, ksplit, st, A, B, C, M, N, kvec);
        default: return launch_plain_l<DT, 32>(rows, threads, ksplit, st, A, B, C, M, N, kvec);
    }
}

template <int WARPS, int RT>
cudaError_t launch_mma_wr(cudaStream_t st, const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t kvec, int ksplit) {
    const int64_t tiles_per_m = (N + 16 * RT - 1) / (16 * RT), tiles = M * tiles_per_m;
    if (tiles_per_m > 0x7FFFFFFF || kvec > 0x7FFFFFF0) return cudaErrorInvalidConfiguration;
    if (ksplit > WARPS) ksplit = WARPS;
    const int tpc = WARPS / ksplit;
    return launch_pdl(k_vecmat_mma<WARPS, RT>, (tiles + tpc - 1) / tpc, WARPS * 32, st, static_cast<const uint4*>(A),
                      static_cast<const uint4*>(B), static_cast<uint16_t*>(C), N, static_cast<int>(kvec), ksplit, static_cast<int>(tiles_per_m), tiles);
}

cudaError_t launch_mma(int rows, int ksplit, int threads, cudaStream_t st, const void* A, const void* B, void* C, int64_t M, int64_t N,
                       int64_t kvec) {
    const int sms = sm_count();
    const int64_t steps = (kvec + 7) / 8;
    if (rows == 0) rows = (steps <= 2 && N >= 32 && M * ((N + 31) / 32) >= warps_wanted(sms)) ? 32 : 16;
    if (ksplit == 0) {
        // Measured on the K sweep: from 512 elements per row on, two warps sharing a tile along k beat one (shorter
        // dependent chains of steps per warp); beyond that k is cut only until one wave of resident warps exists.
        const int64_t tiles = M * ((N + rows - 1) / rows);
        ksplit = steps >= 8 ? 2 : 1;
        while (ksplit < 8 && ksplit * 32 < threads && tiles * ksplit < 32LL * sms && steps >= 4 * ksplit) ksplit *= 2;
    }
    if (rows == 32)
        return threads <= 128 ? launch_mma_wr<4, 2>(st, A, B, C, M, N, kvec, ksplit)
             : threads <= 256 ? launch_mma_wr<8, 2>(st, A, B, C, M, N, kvec, ksplit)
                              : launch_mma_wr<16, 2>(st, A, B, C, M, N, kvec, ksplit);
    return threads <= 128 ? launch_mma_wr<4, 1>(st, A, B, C, M, N, kvec, ksplit)
         : threads <= 256 ? launch_mma_wr<8, 1>(st, A, B, C, M, N, kvec, ksplit)
                          : launch_mma_wr<16, 1>(st, A, B, C, M, N, kvec, ksplit);
}

template <int DT>
cudaError_t launch_tma(cudaStream_t st, const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t row_bytes) {
    using S = typename Elem<DT>::scalar;
    const int64_t tiles_per_m = (N + kTmRows - 1) / kTmRows, tiles = M * tiles_per_m;
    if (tiles_per_m > 0x7FFFFFFF || tiles > 0x7FFFFFFF || row_bytes / kTmChunk > 0x7FFFFF00) return cudaErrorInvalidConfiguration;
    int* status = device_status_word();
    if (!status) return cudaErrorInitializationError;
    const int smem = kTmStages * kTmStageBytes;
    cudaError_t e = cudaFuncSetAttribute(k_vecmat_tma<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(tiles));
    cfg.blockDim = dim3(kTmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_vecmat_tma<DT>, static_cast<const unsigned char*>(A), static_cast<const unsigned char*>(B),
                              static_cast<S*>(C), N, row_bytes, static_cast<int>(tiles_per_m), status);
}

}  // namespace
}  // namespace tf

using namespace tf;

extern "C" tf_status tf_bvecmat_fwd(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, tf_dtype dt_, int threads,
                                    int lanes, int rows, int ksplit, void* stream) {
    const int dt = dt_;
    if (M < 0 || N < 0 || K <= 0 || (dt != DT_F32 && dt != DT_BF16)) return TF_ERR_INVALID_ARG;
    if (M > 0 && N > 0 && (!A || !B || !C)) return TF_ERR_INVALID_ARG;
    if (threads == 0) threads = 128;
    const bool staged = lanes == 1;                               // the shared-memory staged path
    const bool tensor = dt == DT_BF16 && lanes == 0;              // any other forced `lanes` selects the plain path
    if (staged) { lanes = 0; rows = 0; ksplit = 0; }
    if (threads < 32 || threads > 1024 || threads % 32 || (lanes != 0 && lanes != 4 && lanes != 8 && lanes != 16 && lanes != 32) ||
        (ksplit != 0 && ksplit != 1 && ksplit != 2 && ksplit != 4 && ksplit != 8))
        return TF_ERR_INVALID_ARG;
    if (tensor ? (rows != 0 && rows != 16 && rows != 32) : (rows != 0 && rows != 1 && rows != 2 && rows != 4))
        return TF_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return TF_OK;
    if (N > INT64_MAX / M || K > (INT64_MAX / 8) / (M * N)) return TF_ERR_UNSUPPORTED;
    const int64_t nrows = M * N;
    const int es = elem_size(dt);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    count_launches(1);
    if (al16(A) && al16(B) && (K * es) % 16 == 0) {
        const int64_t kvec = K * es / 16;
        if (staged) e = dt == DT_F32 ? launch_tma<DT_F32>(st, A, B, C, M, N, K * es) : launch_tma<DT_BF16>(st, A, B, C, M, N, K * es);
        else if (tensor) e = launch_mma(rows, ksplit, threads, st, A, B, C, M, N, kvec);
        else if (dt == DT_F32) e = launch_plain<DT_F32>(lanes, rows, ksplit, threads, st, A, B, C, M, N, kvec);
        else e = launch_plain<DT_BF16>(lanes, rows, ksplit, threads, st, A, B, C, M, N, kvec);
    } else {
        const int64_t grid = (nrows + threads / 32 - 1) / (threads / 32);
        if (grid > 0x7FFFFFFF) return TF_ERR_UNSUPPORTED;
        if (dt == DT_F32)
            k_vecmat_scalar<DT_F32><<<static_cast<unsigned>(grid), threads, 0, st>>>(static_cast<const float*>(A), static_cast<const float*>(B), static_cast<float*>(C), nrows, N, K);
        else
            k_vecmat_scalar<DT_BF16><<<static_cast<unsigned>(grid), threads, 0, st>>>(static_cast<const uint16_t*>(A), static_cast<const uint16_t*>(B), static_cast<uint16_t*>(C), nrows, N, K);
        e = cudaGetLastError();
    }
    if (e == cudaErrorInvalidConfiguration) return TF_ERR_UNSUPPORTED;
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}
