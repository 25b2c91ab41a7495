// V_RING: persistent cluster split-row variant for long rows (64 KiB .. ~1.5 MiB per row).
//
// A row is cut into `cluster` slices, one per CTA of a thread-block cluster; clusters are persistent and walk
// the rows with a fixed stride.  Each CTA owns a ring of `stages` slice buffers in shared memory that it keeps
// full with bulk asynchronous copies (cp.async.bulk global -> shared on one mbarrier per stage, no multicast:
// every CTA fetches a different slice).  Shared memory is only a prefetch buffer: a slice is read from it once,
// into registers (vpt 16-byte vectors per thread), the slice statistics are reduced across the CTA, and as soon
// as that reduction has consumed the stage thread 0 refills it with the slice of the row `stages` iterations
// ahead.  The per-slice partials (offset,sum | mean,M2 | sum of squares) are pushed into every peer's shared
// memory with asynchronous remote stores that complete a transaction count on the receiver's mbarrier (no
// cluster barrier inside the loop: a cluster-wide release would have to wait for the y stores of the previous
// row); every CTA then merges the partials in slice order, normalises its registers and writes y with 16-byte
// streaming stores.  HBM sees each element once in and once out, exponentials are evaluated
// once, and loading never waits for arithmetic.
//
// Bounded waits: an mbarrier wait that runs out of its clock budget sets TF_ERR_TIMEOUT in the status word; the
// CTA stops issuing copies and waiting but keeps taking part in every CTA and cluster barrier, so no peer hangs.
// The kernel ends with a cluster barrier (no CTA exits while a peer may still write a partial into its shared memory)
// and, after a failed wait, with one more bounded wait for each of its own copies still in flight.
#include <cooperative_groups.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <tuple>

#include "tf_rowmath.cuh"

namespace cg = cooperative_groups;

namespace tf {
namespace {

struct RArgs {
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
    int* status;
};

constexpr int kRingMaxStages = 4;
// Remote 8-byte store into CTA `rank`'s copy of `slot`, counted on that CTA's copy of `bar`.
__device__ __forceinline__ void push_partial(float* slot, uint64_t* bar, uint32_t rank, float a, float b) {
    uint32_t rslot, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rslot) : "r"(smem_u32(slot)), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_u32(bar)), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(rslot), "f"(a), "f"(b), "r"(rbar) : "memory");
}
constexpr int ring_max_threads(int vpt) { return vpt <= 4 ? 1024 : 512; }
__device__ __forceinline__ bool valid_at(int idx, int len) { return idx < len; }

// PSMEM: the CTA's slice of gamma/beta (weight) is copied into shared memory once, behind the ring, instead of being
// fetched from L1/L2 for every row: for long LayerNorm rows the parameters are twice the bytes of x on the L2-to-SM path.
template <int OP, int DT, int VPT, bool PSMEM>
__global__ void __launch_bounds__(ring_max_threads(VPT)) k_ring(const RArgs a) {
    using E = Elem<DT>;
    constexpr int NE = E::NE;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[kRingMaxStages];
    __shared__ __align__(8) uint64_t xch_bar[2];                  // partials of a row have all arrived (double-buffered by row parity)
    __shared__ float red_buf[4 * 32];
    __shared__ __align__(8) float xch[2][kMaxCluster][2];

    const int T = blockDim.x, t = threadIdx.x, cs = a.cs, S = a.nstage;
    const int rank = static_cast<int>(blockIdx.x % cs);
    const int64_t cluster_id = blockIdx.x / cs, num_clusters = gridDim.x / cs;
    const int per = (a.nvec + cs - 1) / cs;                        // vectors per slice
    const int first = rank * per;
    const int len = max(0, min(per, a.nvec - first));
    uint4* const ring = reinterpret_cast<uint4*>(dyn_smem);
    cg::cluster_group cl = cg::this_cluster();

    if (t == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full_bar[s], 1);
        mbar_init(&xch_bar[0], 1);
        mbar_init(&xch_bar[1], 1);
        mbar_fence_init();
    }
    pdl_wait();             // global reads below follow the previous kernel
    uint32_t pending = 0, phase = 0;       // thread 0: stages with a copy in flight; parity of each stage's next completion
    auto issue = [&](int64_t row, int s) {                           // thread 0 only; a slice may need several copies
        if (len == 0) return;
        pending |= 1u << s;
        const char* src = reinterpret_cast<const char*>(a.x + row * a.nvec + first);
        char* dst = reinterpret_cast<char*>(ring + static_cast<size_t>(s) * per);
        const uint32_t bytes = static_cast<uint32_t>(len) * 16u;
        mbar_expect_tx(&full_bar[s], bytes);
        for (uint32_t off = 0; off < bytes; off += 65536u) bulk_g2s(dst + off, src + off, min(65536u, bytes - off), &full_bar[s]);
    };
    if (t == 0)
        for (int s = 0; s < S; ++s) {
            const int64_t row = cluster_id + s * num_clusters;
            if (row < a.rows) issue(row, s);
        }
    __syncthreads();
    if (cs > 1) cl.sync();                 // every CTA of the cluster is resident (barriers initialised) before any remote store
    pdl_trigger();

    bool valid[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) valid[v] = (t + v * T) < len;
    const CtaRed red{red_buf};
    // A persistent CTA always owns the same columns: with few vectors per thread their parameters live in
    // registers for the whole kernel; otherwise they are fetched from L1/L2 when the normalise pass needs them.
    constexpr bool kHeld = (VPT <= 4) && OP != OP_SOFTMAX;
    HeldParams<kHeld ? VPT : 1> held;
    if constexpr (kHeld) {
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            held.g[v] = valid_at(t + v * T, len) ? ld_param(a.p0 + first + t + v * T) : make_uint4(0, 0, 0, 0);
            held.b[v] = (OP == OP_LAYERNORM && valid_at(t + v * T, len)) ? ld_param(a.p1 + first + t + v * T) : make_uint4(0, 0, 0, 0);
        }
    }
    const LazyParams lazy{a.p0, a.p1, first + t, T};
    uint4* const pg = ring + static_cast<size_t>(S) * per;        // behind the ring: gamma slice, then beta slice
    uint4* const pb = pg + per;
    if constexpr (PSMEM) {
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) {
                pg[t + v * T] = ld_param(a.p0 + first + t + v * T);
                if (OP == OP_LAYERNORM) pb[t + v * T] = ld_param(a.p1 + first + t + v * T);
            }
    }
    const OwnedSmemParams inshared{pg, pb, t, T};
    const uint4 fill = fill_vec<DT>(OP);
    auto slice_count = [&](int k) { return static_cast<float>(max(0, min(per, a.nvec - k * per))) * NE; };

    bool failed = false;
    int it = 0;
    for (int64_t row = cluster_id; row < a.rows; row += num_clusters, ++it) {
        const int s = it % S;
        if (len > 0 && !failed) {
            bool landed = mbar_wait(&full_bar[s], static_cast<uint32_t>(it / S) & 1u);
            if (!landed) {
                failed = true;
                atomicExch(a.status, 4);
                landed = mbar_wait(&full_bar[s], static_cast<uint32_t>(it / S) & 1u);      // one more bounded wait for the copy in flight
            }
            if (landed) { pending &= ~(1u << s); phase ^= 1u << s; }
        }
        const uint4* buf = ring + static_cast<size_t>(s) * per + t;
        uint4 raw[VPT], out[VPT];
#pragma unroll
        for (int v = 0; v < VPT; ++v) raw[v] = valid[v] ? buf[v * T] : fill;
        const int xb = it & 1;
        F2 w[VPT][Pairs<DT>::NP];
        bool visit[VPT];                                          // softmax visits every vector (absent ones hold -inf), the norms the ones that exist
#pragma unroll
        for (int v = 0; v < VPT; ++v) visit[v] = OP == OP_SOFTMAX || valid[v];
        const Part part = slice_stats<OP, DT, VPT>(raw, visit, red, xb * 2, slice_count(rank), w);
        // every thread passed the CTA barrier inside the reduction after its shared-memory reads: refill the stage
        const int64_t next = row + static_cast<int64_t>(S) * num_clusters;
        if (t == 0 && !failed && next < a.rows) issue(next, s);
        // A peer can be at most one row ahead of this CTA (it needs this CTA's partial to finish a row), so two
        // slot buffers suffice; every CTA receives exactly cs pushes per row, all of them before it can leave the loop.
        if (cs > 1) {
            if (t == 0) mbar_expect_tx(&xch_bar[xb], static_cast<uint32_t>(cs) * 8u);
            if (t < cs) push_partial(&xch[xb][rank][0], &xch_bar[xb], static_cast<uint32_t>(t), part.a, part.b);
            if (!mbar_wait(&xch_bar[xb], static_cast<uint32_t>(it >> 1) & 1u) && !failed) { failed = true; atomicExch(a.status, 4); }
        } else {
            if (t == 0) { xch[xb][0][0] = part.a; xch[xb][0][1] = part.b; }
            __syncthreads();
        }
        const Total tot = combine_parts<OP>(cs, rank, [&](int k) { return Part{xch[xb][k][0], xch[xb][k][1]}; }, slice_count, a.n, a.eps);
        if constexpr (kHeld) slice_finish<OP, DT, VPT, false>(visit, w, tot, held, out);
        else if constexpr (PSMEM) slice_finish<OP, DT, VPT, false>(visit, w, tot, inshared, out);
        else slice_finish<OP, DT, VPT, false>(visit, w, tot, lazy, out);
        uint4* yr = a.y + row * a.nvec + first + t;
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (valid[v]) st_stream(yr + v * T, out[v]);
        if (t == 0 && rank == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = tot.a;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = tot.b;
        }
    }
    // Nobody leaves while a peer may still push a partial into its shared memory.  Every CTA of the cluster gets here:
    // all waits above are bounded and the CTAs of a cluster walk the same rows.
    if (cs > 1) cl.sync();
    // After a wait has given up this CTA stopped consuming its ring: copies issued before that may still be in flight and
    // get one more bounded wait each before the shared memory they target is released.
    if (failed && t == 0)
        for (int s = 0; s < S; ++s)
            if (pending & (1u << s)) mbar_wait(&full_bar[s], (phase >> s) & 1u);
}

using RingFn = void (*)(const RArgs);

template <int OP, int DT> RingFn pick_ring(int vpt, bool psmem) {
    if (psmem) {                       // only where the parameters are not already held in registers
        if (OP != OP_SOFTMAX && vpt == 8) return k_ring<OP, DT, 8, (OP != OP_SOFTMAX)>;
        return nullptr;
    }
    switch (vpt) {
        case 1: return k_ring<OP, DT, 1, false>;
        case 2: return k_ring<OP, DT, 2, false>;
        case 4: return k_ring<OP, DT, 4, false>;
        case 8: return k_ring<OP, DT, 8, false>;
    }
    return nullptr;
}

RingFn ring_fn(int op, int dt, int vpt, bool psmem) {
    switch (op * 2 + dt) {
        case 0: return pick_ring<OP_SOFTMAX, DT_F32>(vpt, psmem);
        case 1: return pick_ring<OP_SOFTMAX, DT_BF16>(vpt, psmem);
        case 2: return pick_ring<OP_LAYERNORM, DT_F32>(vpt, psmem);
        case 3: return pick_ring<OP_LAYERNORM, DT_BF16>(vpt, psmem);
        case 4: return pick_ring<OP_RMSNORM, DT_F32>(vpt, psmem);
        case 5: return pick_ring<OP_RMSNORM, DT_BF16>(vpt, psmem);
    }
    return nullptr;
}

size_t ring_smem(const Plan& p, const Args& a) {
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    const int64_t per = (nvec + p.cluster - 1) / p.cluster;
    const int nparam = p.rpg == 2 ? (a.op == OP_LAYERNORM ? 2 : 1) : 0;      // rpg = 2: parameter slices in shared memory
    return static_cast<size_t>(p.stages + nparam) * per * 16;
}

}  // namespace

bool supports_ring(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (!vector_ok(a) || p.threads < 32 || p.threads % 32 || p.threads > ring_max_threads(p.vpt)) return false;
    if (p.cluster < 1 || p.cluster > kMaxCluster || p.cluster > d.max_cluster || (p.cluster & (p.cluster - 1))) return false;
    if (p.stages < 1 || p.stages > kRingMaxStages || p.persist < 1 || p.persist > 8 || (p.rpg != 1 && p.rpg != 2) || !ring_fn(a.op, a.dt, p.vpt, p.rpg == 2)) return false;
    const int64_t nvec = a.cols * elem_size(a.dt) / 16;
    if (nvec > 0x7FFFFFFF) return false;
    const int64_t per = (nvec + p.cluster - 1) / p.cluster;
    if (per > static_cast<int64_t>(p.threads) * p.vpt || per * 16 >= (1 << 20)) return false;
    return ring_smem(p, a) + 2048 <= static_cast<size_t>(d.smem_optin) / p.persist;
}

cudaError_t launch_ring(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    RingFn fn = ring_fn(a.op, a.dt, p.vpt, p.rpg == 2);
    if (!fn) return cudaErrorInvalidValue;
    cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
    if (e != cudaSuccess) return e;
    RArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows;
    k.nvec = static_cast<int>(a.cols * elem_size(a.dt) / 16);
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.cs = p.cluster; k.nstage = p.stages; k.status = a.status;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(p.threads);
    cfg.dynamicSmemBytes = ring_smem(p, a);
    cfg.stream = st;
    // No programmatic early launch here: a persistent cluster that could only be placed after the previous
    // kernel has drained would start late with a full share of rows and double the kernel's duration.
    cudaLaunchAttribute attr[1];
    int na = 0;
    if (p.cluster > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = p.cluster; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    // Persistent clusters must all be resident at once: ask how many the device can hold in this shape
    // (clusters cannot straddle GPCs, so it is usually fewer than SMs / cluster) and launch no more than that.
    int64_t clusters = std::max<int64_t>(1, static_cast<int64_t>(p.persist) * d.sms / p.cluster);
    if (p.cluster > 1) {
        static std::mutex mu;
        static std::map<std::tuple<const void*, int, int, size_t, int>, int> cache;
        const auto key = std::make_tuple(reinterpret_cast<const void*>(fn), d.ordinal, p.threads, cfg.dynamicSmemBytes, p.cluster);
        std::lock_guard<std::mutex> lk(mu);
        auto it = cache.find(key);
        if (it == cache.end()) {
            int n = 0;
            cfg.gridDim = dim3(static_cast<unsigned>(clusters * p.cluster));
            e = cudaOccupancyMaxActiveClusters(&n, fn, &cfg);
            if (e != cudaSuccess) return e;
            it = cache.emplace(key, n).first;
        }
        if (it->second < 1) return cudaErrorLaunchOutOfResources;
        clusters = std::min<int64_t>(clusters, it->second);
    }
    clusters = std::min<int64_t>(clusters, a.rows);
    cfg.gridDim = dim3(static_cast<unsigned>(clusters * p.cluster));
    note_launch(reinterpret_cast<const void*>(fn), clusters * p.cluster, p.threads, cfg.dynamicSmemBytes, p.cluster);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
