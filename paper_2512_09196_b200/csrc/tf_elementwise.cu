// Calibration kernels: a plain device copy written in the same load/store style as the row kernels (the honest
// ceiling for "bytes in, bytes out" on this GPU at a given size), and the element-wise sine of the paper's first
// case study (a kernel whose only tuning knob is its launch geometry).
#include <algorithm>

#include "../../include/tf.h"
#include "tf_common.cuh"

namespace tf {
namespace {

// Both kernels give every CTA ONE contiguous block of threads x U vectors and launch as many CTAs as the tensor
// needs.  (Measured on B200, 512 MiB copies: this layout reaches 6.73 TB/s whatever the cache hints, while the same
// kernel as a persistent grid-stride loop over 8 CTAs per SM stays at 5.9-6.1 TB/s.)
constexpr int kEwU = 4;              // independent 16-byte accesses per thread in the copy

__global__ void __launch_bounds__(1024) k_copy(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t nvec,
                                               const unsigned char* xt, unsigned char* yt, int tail) {
    pdl_wait();
    pdl_trigger();
    const int64_t base = static_cast<int64_t>(blockIdx.x) * blockDim.x * kEwU + threadIdx.x;
    uint4 v[kEwU];
#pragma unroll
    for (int u = 0; u < kEwU; ++u)
        if (base + u * blockDim.x < nvec) v[u] = ld_stream(x + base + u * blockDim.x);
#pragma unroll
    for (int u = 0; u < kEwU; ++u)
        if (base + u * blockDim.x < nvec) st_stream(y + base + u * blockDim.x, v[u]);
    if (blockIdx.x == 0 && threadIdx.x < tail) yt[threadIdx.x] = xt[threadIdx.x];       // the last (< 16) bytes
}

__global__ void __launch_bounds__(1024) k_copy_bytes(const unsigned char* x, unsigned char* y, int64_t n) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) y[i] = x[i];
}

// sin of a 16-byte vector of bf16 whose magnitudes stay below 2^15, on packed fp32 pairs: k = round(x / pi) by the
// add-and-subtract of 1.5 * 2^23 (k's parity is then the lowest mantissa bit of the sum), r = x - k pi with pi split
// in two fp32 constants and fused multiply-adds (the rounding error is relative to r, not to x), the sign (-1)^k
// applied to r, and the odd polynomial r + r^3 (c3 + c5 r^2 + c7 r^4) on [-pi/2, pi/2] (relative error 1.3e-6,
// 1/3000 of a bf16 unit in the last place).  Evaluated in fp32 arithmetic over every bf16 value of that range the
// rounded results are the correctly rounded ones.  NaN stays NaN.
__device__ __forceinline__ uint4 sin_bf16_small(const F2 (&x)[4]) {
    const F2 inv_pi = f2(0.318309886f), magic = f2(12582912.f), neg_magic = f2(-12582912.f);
    const F2 neg_pi_hi = f2(-3.14159274f), neg_pi_lo = f2(8.74227766e-8f);      // pi = 3.14159274 - 8.74227766e-8
    const F2 c3 = f2(-0.166657895f), c5 = f2(0.00831331313f), c7 = f2(-0.00018510368f);
    F2 y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const F2 t = fma2(x[i], inv_pi, magic);
        const F2 k = add2(t, neg_magic);
        F2 r = fma2(k, neg_pi_lo, fma2(k, neg_pi_hi, x[i]));
        float t0, t1, r0, r1;
        split(t, t0, t1);
        split(r, r0, r1);
        r = f2(__uint_as_float(__float_as_uint(r0) ^ (__float_as_uint(t0) << 31)),
               __uint_as_float(__float_as_uint(r1) ^ (__float_as_uint(t1) << 31)));
        const F2 r2 = mul2(r, r);
        const F2 p = fma2(fma2(r2, c7, c5), r2, c3);
        y[i] = fma2(p, mul2(r2, r), r);
    }
    return Pairs<DT_BF16>::pack(y);
}

// y = sin(x), fp32 arithmetic, one rounding to the storage type: sinf with full range reduction (about 1 ulp of fp32)
// for fp32 tensors, for bf16 vectors that hold a magnitude of 2^15 or more (or an infinity), and in the element loop;
// the packed evaluation above for all other bf16 vectors (sinf executes 32 instructions per element against 12, which holds
// a 2-byte type at two thirds of the copy rate).  A CTA covers threads x U vectors (the "block size" knob of the
// paper's case study); the scalar tail and unaligned tensors go through the element loop at the end.
template <int DT, int U>
__global__ void __launch_bounds__(1024) k_sin(const typename Elem<DT>::scalar* x, typename Elem<DT>::scalar* y, int64_t n,
                                              int vec_ok) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    pdl_wait();
    pdl_trigger();
    const int64_t nvec = vec_ok ? n / NE : 0;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    uint4* yv = reinterpret_cast<uint4*>(y);
    const int64_t base = static_cast<int64_t>(blockIdx.x) * blockDim.x * U + threadIdx.x;
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (base + u * blockDim.x < nvec) v[u] = ld_stream(xv + base + u * blockDim.x);
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (base + u * blockDim.x < nvec) {
            if constexpr (DT == DT_BF16) {
                F2 p[4];
                Pairs<DT_BF16>::unpack(v[u], p);
                float a[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) split(p[i], a[2 * i], a[2 * i + 1]);
                float big = fmaxf(fabsf(a[0]), fabsf(a[1]));
#pragma unroll
                for (int i = 2; i < 8; ++i) big = fmaxf(big, fabsf(a[i]));
                if (big < 32768.f) {                                         // a NaN is not seen here and comes out a NaN
                    st_stream(yv + base + u * blockDim.x, sin_bf16_small(p));
                    continue;
                }
            }
            float f[NE];
            E::unpack(v[u], f);
#pragma unroll
            for (int e = 0; e < NE; ++e) f[e] = sinf(f[e]);
            st_stream(yv + base + u * blockDim.x, E::pack(f));
        }
    }
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = nvec * NE + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride)
        y[i] = E::from_float(sinf(E::to_float(x[i])));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <class... A>
cudaError_t launch_pdl(void (*fn)(A...), int grid, int threads, cudaStream_t st, A... args) {
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

int blocks_for(int64_t nvec, int threads, int u) {
    const int64_t per = static_cast<int64_t>(threads) * u;
    return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((nvec + per - 1) / per, 0x7FFFFFFF)));
}

}  // namespace
}  // namespace tf

using namespace tf;

extern "C" tf_status tf_copy(const void* x, void* y, int64_t bytes, void* stream) {
    if (bytes < 0 || (bytes > 0 && (!x || !y))) return TF_ERR_INVALID_ARG;
    if (bytes == 0) return TF_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    count_launches(1);
    if (aligned16(x) && aligned16(y)) {
        const int64_t nvec = bytes / 16;
        const int tail = static_cast<int>(bytes % 16);
        const unsigned char* xt = static_cast<const unsigned char*>(x) + nvec * 16;
        unsigned char* yt = static_cast<unsigned char*>(y) + nvec * 16;
        if (nvec > static_cast<int64_t>(0x7FFFFFFF) * 256 * kEwU) return TF_ERR_UNSUPPORTED;
        e = launch_pdl(k_copy, blocks_for(nvec, 256, kEwU), 256, st, static_cast<const uint4*>(x), static_cast<uint4*>(y), nvec, xt,
                       yt, tail);
    } else {
        const int grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((bytes + 255) / 256, 1 << 20)));
        k_copy_bytes<<<grid, 256, 0, st>>>(static_cast<const unsigned char*>(x), static_cast<unsigned char*>(y), bytes);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}

extern "C" tf_status tf_sin_fwd(const void* x, void* y, int64_t n, tf_dtype dt_, int threads, int vectors_per_thread, void* stream) {
    const int dt = dt_;
    if (n < 0 || (dt != DT_F32 && dt != DT_BF16) || (n > 0 && (!x || !y))) return TF_ERR_INVALID_ARG;
    // defaults read off the geometry sweep (256 MiB of input): 64 threads with 4 vectors per thread
    if (threads == 0) threads = 64;
    int u = vectors_per_thread == 0 ? 4 : vectors_per_thread;
    if (threads < 32 || threads > 1024 || threads % 32 || (u != 1 && u != 2 && u != 4 && u != 8)) return TF_ERR_INVALID_ARG;
    if (n == 0) return TF_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int vec_ok = aligned16(x) && aligned16(y);
    const int ne = dt == DT_F32 ? 4 : 8;
    // without the vector path the element loop does all the work: give it enough CTAs
    const int grid = vec_ok ? blocks_for(std::max<int64_t>(1, n / ne), threads, u) : blocks_for(n, threads, 8);
    count_launches(1);
    cudaError_t e = cudaErrorInvalidValue;
#define TF_SIN(U)                                                                                                               \
    if (u == U)                                                                                                                 \
        e = dt == DT_F32 ? launch_pdl(k_sin<DT_F32, U>, grid, threads, st, static_cast<const float*>(x), static_cast<float*>(y), n, vec_ok) \
                         : launch_pdl(k_sin<DT_BF16, U>, grid, threads, st, static_cast<const uint16_t*>(x), static_cast<uint16_t*>(y), n, vec_ok);
    TF_SIN(1) TF_SIN(2) TF_SIN(4) TF_SIN(8)
#undef TF_SIN
    if (e != cudaSuccess) { remember_cuda_error(e); return TF_ERR_CUDA; }
    return TF_OK;
}
