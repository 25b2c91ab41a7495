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
// Three kernels implement the plan: k_twopass (loads straight into registers), k_twopass_ring (plan field `stages` >= 2:
// asynchronous copies through per-thread rings in shared memory) and k_twopass_fit, which the launcher picks by itself
// when the ring of the plan holds the whole row (rows of 4-64 KiB per CTA): the second pass then never leaves the SM.
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
    int groups;           // row order: launch slot b works on row (b % groups) * ceil(rows / groups) + b / groups
    int64_t slots;        // groups * ceil(rows / groups)
    int stages;           // ring form: steps per thread's ring
    int64_t per_group;    // slots / groups
    int step, nfull, rag; // ring form: vectors a CTA takes per step; whole steps of a row; vectors of its ragged last step
    int policy;           // bit 0: pass A loads ask L2 to keep their lines; bit 1: pass B loads let them go
};

// MAXT / MINB: the launch bounds.  Besides the unconstrained form (1024, 0) there are (768, 2) and (512, 3), which hold
// the kernel to 40 registers so that 1536 threads are resident per SM instead of 1024-1280.
// LEN: softmax with per-row valid lengths; CACHE: the head of each row is parked in shared memory between the passes.
// Both are compile-time so that the plain build carries neither the length arithmetic nor the cache tests per vector.
template <int OP, int DT, int MAXT, int MINB, bool CL, bool LEN, bool CACHE>
__global__ void __launch_bounds__(MAXT, MINB) k_twopass(const WArgs a) {
    constexpr int NE = Elem<DT>::NE;
    __shared__ float red_buf[4 * 32];
    __shared__ float xch[CL ? 2 : 1][CL ? kMaxCluster : 1][2];   // partials of the peers, by row parity
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    uint4* const cache = reinterpret_cast<uint4*>(dyn_smem);
    pdl_wait();
    pdl_trigger();
    // pass A keeps x in L2, pass B lets it go (either hint can be switched off by the plan)
    const uint64_t keep = (a.policy & 1) ? policy_evict_last() : policy_evict_normal();
    const uint64_t last = (a.policy & 2) ? policy_evict_first() : policy_evict_normal();
    const int cs = CL ? a.cs : 1;
    const int rank = CL ? static_cast<int>(blockIdx.x % cs) : 0;
    const int64_t first_slot = CL ? blockIdx.x / cs : blockIdx.x, slot_step = CL ? gridDim.x / cs : gridDim.x;
    const int64_t per_group = a.per_group;
    const int64_t per = CL ? (a.nvec + cs - 1) / cs : a.nvec, first = rank * per;        // this CTA's slice of every row
    const int64_t seg = max(int64_t{0}, min(per, a.nvec - first));
    const int64_t cache_vecs = min(a.cache_vecs, seg);
    auto count_of = [&](int k) { return static_cast<float>(max(int64_t{0}, min(per, a.nvec - k * per)) * NE); };
    if constexpr (CL) cg::this_cluster().sync();                  // every CTA of the cluster is resident before any remote write
    int it = -1;
    for (int64_t slot = first_slot; slot < a.slots; slot += slot_step) {
        // neighbouring rows often cost alike (a causal mask grows with the row index): CTAs that run side by side take rows
        // from `groups` evenly spaced parts of the tensor, so that what is in flight between the passes is an even mix
        const int64_t row = a.groups > 1 ? (slot % a.groups) * per_group + slot / a.groups : slot;
        if (row >= a.rows) continue;                               // the same decision in every CTA of a cluster
        ++it;
        const uint4* xr = a.x + row * a.nvec + first;
        int64_t len = -1;
        if constexpr (LEN) {
            const int64_t whole = min(max(static_cast<int64_t>(__ldg(a.len + row)), int64_t{0}), a.nvec * NE);
            len = min(max(whole - first * NE, int64_t{0}), seg * NE);
        }
        const Running<OP, DT> run = stream_stats<OP, DT, LEN, CACHE>(xr, seg, keep, cache, cache_vecs, len);
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
        stream_apply<OP, DT, LEN, CACHE>(xr, a.y + row * a.nvec + first, a.p0 + first, a.p1 + first, seg, sc, last, cache, cache_vecs,
                                         run.live_slots, len);
    }
}

// ---- the ring form -------------------------------------------------------------------------------------------
// The same two passes with the loads decoupled from the arithmetic: every thread keeps a private ring of `stages`
// steps (U vectors each) in shared memory and fills it with 16-byte asynchronous copies (cp.async) `stages - 1` steps
// ahead of the step it is working on, so the bytes in flight are the ring, not what a thread's registers hold, and
// a step's arithmetic overlaps the flight of the following ones.  A slot is written and read by the same thread only,
// so no barrier guards the ring.  Pass A walks the row back to front and pass B front to back: when pass A ends, the
// ring holds the first steps of the row, which pass B takes from shared memory without touching L2 again (with a mask
// at the end of a row, as causal and padded rows have it, that head is the live part).
__device__ __forceinline__ void cp_async16(uint4* dst, const uint4* src, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait(int pending) {     // returns once at most `pending` of this thread's groups are in flight
    if (pending == 1) { asm volatile("cp.async.wait_group 1;" ::: "memory"); return; }      // two stages: the common case
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
    }
}
constexpr int kRingMaxDepth = 8;

// Work is laid out by warps: in one step a warp takes U x 32 consecutive vectors (lane l the vectors l, l + 32, ... of that
// run), so a thread's U copies, loads and stores of a step sit at fixed offsets from one pointer that advances by a
// step's worth per iteration; all counters are 32-bit.  Only the last step of a row can be ragged, and it has its own
// code: the loops over whole steps carry no predicates.
// CL: the `cs` CTAs of a thread-block cluster share a row, CTA `rank` taking the steps rank, rank + cs, ... of it (so a mask
// at the end of the row costs every CTA of the cluster the same); the partials meet between the passes through
// distributed shared memory and one cluster barrier.  A row is then in flight for 1 / cs of the time, which keeps what lies
// between the passes within L2, and each CTA's ring holds cs times as large a share of the row.
template <int OP, int DT, int U, int MAXT, int MINB, bool CL, bool LEN = false>
__global__ void __launch_bounds__(MAXT, MINB) k_twopass_ring(const WArgs a) {
    constexpr int NE = Elem<DT>::NE, CH = U * 32;                        // vectors a warp takes per step
    __shared__ float red_buf[4 * 32];
    __shared__ float xch[CL ? 2 : 1][CL ? kMaxCluster : 1][2];           // partials of the CTAs of the cluster, by row parity
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    pdl_wait();
    pdl_trigger();
    const uint64_t keep = (a.policy & 1) ? policy_evict_last() : policy_evict_normal();
    const uint64_t last = (a.policy & 2) ? policy_evict_first() : policy_evict_normal();
    const int t = threadIdx.x, S = a.stages;
    const int cs = CL ? a.cs : 1;
    const int rank = CL ? static_cast<int>(blockIdx.x % cs) : 0;
    const int nvec = static_cast<int>(a.nvec);
    const int step = a.step;                                             // vectors the CTA takes per step: warps x CH
    const int gstep = cs * step;                                         // distance in the row between two steps of this CTA
    // What a CTA needs to know about a row of `lv` vectors: whole steps of the row and vectors of its ragged last step; this
    // CTA's steps (CTA k takes the steps k, k + cs, ...; its last one is the ragged step iff that falls to it), numbered
    // 0 .. nsteps-1 from here on; pass A visits step s as its (nsteps-1-s)-th, so step 0 lives in ring slot (nsteps-1) mod S
    // (two stages, the common case, without a division).  LEN: a row is as long as its length says.
    struct Geo { int nfull, rag, nsteps, nwhole, slot0; bool has_rag; };
    auto geo_of = [&](int nfull, int rag) {
        Geo g;
        g.nfull = nfull; g.rag = rag;
        const int n = nfull + (rag ? 1 : 0);
        g.nsteps = CL ? (n > rank ? (n - rank - 1) / cs + 1 : 0) : n;
        g.has_rag = rag != 0 && (!CL || nfull % cs == rank);
        g.nwhole = g.nsteps - (g.has_rag ? 1 : 0);
        g.slot0 = g.nsteps > 0 ? (S == 2 ? ((g.nsteps - 1) & 1) : (g.nsteps - 1) % S) : 0;
        return g;
    };
    const Geo g0 = geo_of(a.nfull, a.rag);
    // elements CTA k holds of a full row (LayerNorm's merge of the CTAs' partial means)
    auto count_of = [&](int k) {
        const int n = a.nfull + (a.rag ? 1 : 0);
        const int st = CL ? (n > k ? (n - k - 1) / cs + 1 : 0) : n;
        const bool rg = a.rag != 0 && (!CL || a.nfull % cs == k);
        return static_cast<float>(((st - (rg ? 1 : 0)) * step + (rg ? a.rag : 0)) * NE);
    };
    const int toff = (t >> 5) * CH + (t & 31);                           // this thread's first vector within a step
    uint4* const myring = reinterpret_cast<uint4*>(dyn_smem) + toff;     // slot k of the ring: myring + k * step (+ u * 32)
    uint4* const ring_end = myring + S * step;
    const int64_t per_group = a.per_group;
    const uint4 fill = fill_vec<DT>(OP);
    const uint4 zero = make_uint4(0, 0, 0, 0);
    if constexpr (CL) cg::this_cluster().sync();                         // every CTA of the cluster is resident before any remote write
    const int64_t first_slot = CL ? blockIdx.x / cs : blockIdx.x, slot_step = CL ? gridDim.x / cs : gridDim.x;
    int it = -1;
    for (int64_t slot = first_slot; slot < a.slots; slot += slot_step) {
        const int64_t row = a.groups > 1 ? (slot % a.groups) * per_group + slot / a.groups : slot;
        if (row >= a.rows) continue;                                     // the same decision in every CTA of a cluster
        ++it;
        int straddle = -1, keep_el = 0;                                  // LEN: the vector the length ends in, and how much of it is live
        int lv = nvec;                                                   // LEN: live vectors of this row
        if constexpr (LEN) {
            const int len = min(max(__ldg(a.len + row), 0), nvec * NE);
            lv = (len + NE - 1) / NE;
            keep_el = len % NE;
            straddle = keep_el ? len / NE : -1;
        }
        const Geo g = LEN ? geo_of(lv / step, lv % step) : g0;
        const int64_t base = row * nvec + rank * step + toff;            // this thread's vectors of step s: base + s * gstep (+ u * 32)
        const uint4* const xr = a.x + base;
        uint4* const yr = a.y + base;
        auto issue_full = [&](const uint4* src, uint4* dst, uint64_t policy) {
#pragma unroll
            for (int u = 0; u < U; ++u) cp_async16(dst + u * 32, src + u * 32, policy);
        };
        auto issue_ragged = [&](uint4* dst, uint64_t policy) {           // vectors behind the end of the row get the fill value
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (toff + u * 32 < g.rag) cp_async16(dst + u * 32, xr + g.nwhole * gstep + u * 32, policy);
                else dst[u * 32] = fill;
            }
        };
        // ---- pass A, back to front: the k-th step visited is s = g.nsteps - 1 - k and lives in slot k mod S
        Running<OP, DT, U> run;
        {
            int k_issue = 0;
            uint4* dst_i = myring;                                       // ring slot of the step issued next
            const uint4* src_i = xr + (g.nsteps - 1) * gstep;
            auto issue_next = [&]() {
                if (k_issue < g.nsteps) {
                    if (g.has_rag && k_issue == 0) issue_ragged(dst_i, keep);
                    else issue_full(src_i, dst_i, keep);
                }
                cp_async_commit();
                ++k_issue; src_i -= gstep; dst_i += step;
                if (dst_i == ring_end) dst_i = myring;
            };
            for (int j = 0; j < S - 1; ++j) issue_next();
            const uint4* cur = myring;                                   // ring slot of the step worked on
            for (int k = 0; k < g.nsteps; ++k) {
                issue_next();
                cp_async_wait(S - 1);
                uint4 raw[U];
#pragma unroll
                for (int u = 0; u < U; ++u) raw[u] = cur[u * 32];
                cur += step;
                if (cur == ring_end) cur = myring;
                const int s = g.nsteps - 1 - k;
                if constexpr (LEN) {                                     // the vector the length ends in: its dead elements count as -inf
                    const int v0 = (rank + s * cs) * step + toff;
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (v0 + u * 32 == straddle) raw[u] = mask_tail<DT>(raw[u], keep_el);
                }
                if (g.has_rag && k == 0) {
                    bool ok[U];
                    int count = 0;
#pragma unroll
                    for (int u = 0; u < U; ++u) { ok[u] = toff + u * 32 < g.rag; count += ok[u] ? NE : 0; }
                    if (count > 0) run.template update<true>(raw, ok, count, s * U);
                } else {
                    const bool all[U] = {};
                    run.template update<false>(raw, all, U * NE, s * U);
                }
            }
        }
        Part part = merge_running<OP, DT, U>(run, CL ? fmaxf(count_of(rank), 1.f) : a.n, red_buf + 64 * (it & 1));
        if constexpr (CL) {
            cg::cluster_group cl = cg::this_cluster();
            const int xb = it & 1;
            if (t < cs) {                                                 // my partial into every CTA of the cluster
                float* dstp = cl.map_shared_rank(&xch[xb][rank][0], t);
                dstp[0] = part.a; dstp[1] = part.b;
            }
            cl.sync();                                                    // release our writes, acquire the peers'
            // the row's partial from the CTAs', in rank order (the same bits in every CTA)
            if constexpr (OP == OP_SOFTMAX) {
                float O = -kNegInf, Ssum = 0.f;
                for (int k = 0; k < cs; ++k) O = fminf(O, xch[xb][k][0]);
                for (int k = 0; k < cs; ++k) Ssum = fmaf(xch[xb][k][1], softmax_rescale(O, xch[xb][k][0]), Ssum);
                part = Part{O, Ssum};
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
        if (t == 0 && rank == 0) {
            if (OP == OP_LAYERNORM && a.mean) a.mean[row] = sc.a;
            if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = sc.b;
        }
        // ---- pass B, front to back: steps 0 .. S-1 are still in the ring; step s + S - 1 is requested while step s is
        // worked on, into the slot that step s - 1 has just left.  Softmax: from this thread's first step that holds
        // nothing but -inf on, zeros are written and x is not read again.
        const F2 ta2 = f2(sc.a), tb2 = f2(sc.b);
        const int live_steps = OP == OP_SOFTMAX ? (run.live_slots + U - 1) / U : g.nsteps;
        const int live_whole = min(live_steps, g.nwhole);
        const uint4* cur = myring + g.slot0 * step;                // ring slot of step s: one slot down per step
        const uint4* src_n = xr + S * gstep;                             // step s + S - 1 of x (s = 1 first)
        const uint4* gp = a.p0 + rank * step + toff;
        const uint4* bp = a.p1 + rank * step + toff;
        uint4* dst = yr;
        int s = 0;
        for (; s < live_whole; ++s) {
            const int sn = s + S - 1;
            if (s >= 1) {
                uint4* freed = const_cast<uint4*>(cur) + step;           // the slot step s - 1 has just left
                if (freed == ring_end) freed = myring;
                if (sn < live_steps) {
                    if (sn < g.nwhole) issue_full(src_n, freed, last);
                    else issue_ragged(freed, last);
                }
                src_n += gstep;
            }
            cp_async_commit();
            cp_async_wait(S - 1);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                uint4 raw = cur[u * 32];
                if (LEN && (rank + s * cs) * step + toff + u * 32 == straddle) raw = mask_tail<DT>(raw, keep_el);
                st_stream(dst + u * 32, apply_vec<OP, DT>(raw, gp + u * 32, bp + u * 32, ta2, tb2));
            }
            cur = (cur == myring ? ring_end : cur) - step;
            dst += gstep; gp += gstep; bp += gstep;
        }
        if (g.has_rag && s == g.nwhole && s < live_steps) {                  // the ragged step is live
            cp_async_commit();
            cp_async_wait(0);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (toff + u * 32 < g.rag) {
                    uint4 raw = cur[u * 32];
                    if (LEN && (rank + s * cs) * step + toff + u * 32 == straddle) raw = mask_tail<DT>(raw, keep_el);
                    st_stream(dst + u * 32, apply_vec<OP, DT>(raw, gp + u * 32, bp + u * 32, ta2, tb2));
                }
            }
            ++s;
        }
        for (; s < g.nwhole; ++s) {
#pragma unroll
            for (int u = 0; u < U; ++u) st_stream(yr + s * gstep + u * 32, zero);
        }
        if (g.has_rag && s == g.nwhole) {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (toff + u * 32 < g.rag) st_stream(yr + s * gstep + u * 32, zero);
        }
        cp_async_wait(0);
        if constexpr (LEN) {                                             // +0 behind the length, shared by the CTAs of the row
            uint4* const y_row = a.y + row * nvec;
            for (int i = lv + rank * static_cast<int>(blockDim.x) + t; i < nvec; i += cs * static_cast<int>(blockDim.x)) st_stream(y_row + i, zero);
        }
    }
}

// ---- the ring form for rows that fit the ring ---------------------------------------------------------------------
// When a row takes no more steps than the ring has stages (rows of 4-64 KiB with CTAs of 32-512 threads), every copy
// of the row is requested in the prologue, nothing is refilled and the second pass finds the whole row in shared
// memory: x crosses L2 once.  One row per CTA, NS steps known at compile time, so both passes are straight-line code;
// FULL: the row fills the steps exactly and no access carries a predicate.
// CL: the `cs` CTAs of a cluster share a row of up to cs x 64 KiB, CTA `rank` taking the steps rank, rank + cs, ...;
// their partials meet once, through distributed shared memory.  A CTA writes into its peers only after a cluster
// barrier that every CTA arrives at when it starts (so the peers are running), and reads what it received after a second one.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// LEN (softmax): the row is normalised over its first len[row] elements; only the live vectors are
// copied, the vector the length ends in is masked where it is used, and zeros are written behind it.
template <int OP, int DT, int U, int NS, bool FULL, bool CL, bool LEN = false>
__global__ void __launch_bounds__(1024, 1) k_twopass_fit(const WArgs a) {
    constexpr int NE = Elem<DT>::NE, CH = U * 32;
    __shared__ float red_buf[2 * 32];
    __shared__ float xch[CL ? kMaxCluster : 1][2];                       // partials of the CTAs of the cluster
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    if constexpr (CL) cluster_arrive();
    pdl_wait();
    pdl_trigger();
    const uint64_t once = (a.policy & 2) ? policy_evict_first() : policy_evict_normal();     // x is read once
    const int t = threadIdx.x;
    const int nvec = static_cast<int>(a.nvec), step = a.step;
    const int cs = CL ? a.cs : 1;
    const int rank = CL ? static_cast<int>(blockIdx.x % cs) : 0;
    const int gstep = cs * step;                                         // distance in the row between two steps of this CTA
    const int toff = (t >> 5) * CH + (t & 31);                           // this thread's first vector within a step
    const int mine = rank * step + toff;                                 // ... within the row
    const int64_t row = CL ? blockIdx.x / cs : blockIdx.x;
    const uint4* const xr = a.x + row * nvec + mine;
    uint4* const yr = a.y + row * nvec + mine;
    uint4* const myring = reinterpret_cast<uint4*>(dyn_smem) + toff;
    int lim = nvec, straddle = -1, keep = 0;                             // LEN: live vectors; the vector the length ends in and how much of it is live
    if constexpr (LEN) {
        const int len = min(max(__ldg(a.len + row), 0), nvec * NE);
        lim = (len + NE - 1) / NE;
        keep = len % NE;
        straddle = keep ? len / NE : -1;
    }
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (FULL || s * gstep + mine + u * 32 < lim) cp_async16(myring + s * step + u * 32, xr + s * gstep + u * 32, once);
        cp_async_commit();
    }
    Running<OP, DT, U> run;
    const uint4 fill = fill_vec<DT>(OP);
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        cp_async_wait(NS - 1 - s);
        const int first = s * gstep + mine;
        uint4 raw[U];
        if (FULL || (!LEN && first + (U - 1) * 32 < nvec)) {
#pragma unroll
            for (int u = 0; u < U; ++u) raw[u] = myring[s * step + u * 32];
            const bool all[U] = {};
            run.template update<false>(raw, all, U * NE, s * U);
        } else if (first < lim) {
            bool ok[U];
            int count = 0;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                ok[u] = first + u * 32 < lim;
                raw[u] = ok[u] ? myring[s * step + u * 32] : fill;
                if (LEN && first + u * 32 == straddle) raw[u] = mask_tail<DT>(raw[u], keep);
                count += ok[u] ? NE : 0;
            }
            run.template update<true>(raw, ok, count, s * U);
        }
    }
    // elements CTA k holds: its steps k, k + cs, ... clipped to the row
    auto count_of = [&](int k) {
        int c = 0;
#pragma unroll
        for (int s = 0; s < NS; ++s) c += max(0, min(step, nvec - (s * cs + k) * step));
        return static_cast<float>(c * NE);
    };
    Part part = merge_running<OP, DT, U>(run, CL ? fmaxf(count_of(rank), 1.f) : a.n, red_buf);
    if constexpr (CL) {
        cg::cluster_group cl = cg::this_cluster();
        cluster_wait();                                                   // every CTA of the cluster has started
        if (t < cs) {                                                     // my partial into every CTA of the cluster
            float* dstp = cl.map_shared_rank(&xch[rank][0], t);
            dstp[0] = part.a; dstp[1] = part.b;
        }
        cluster_arrive();
        cluster_wait();                                                   // release our writes, acquire the peers'
        // the row's partial from the CTAs', in rank order (the same bits in every CTA)
        if constexpr (OP == OP_SOFTMAX) {
            float O = -kNegInf, Ssum = 0.f;
            for (int k = 0; k < cs; ++k) O = fminf(O, xch[k][0]);
            for (int k = 0; k < cs; ++k) Ssum = fmaf(xch[k][1], softmax_rescale(O, xch[k][0]), Ssum);
            part = Part{O, Ssum};
        } else if constexpr (OP == OP_LAYERNORM) {
            float sum = 0.f, m2 = 0.f;
            for (int k = 0; k < cs; ++k) sum = fmaf(count_of(k), xch[k][0], sum);
            const float mean = fast_div(sum, a.n);
            for (int k = 0; k < cs; ++k) { const float d = xch[k][0] - mean; m2 += fmaf(count_of(k) * d, d, xch[k][1]); }
            part = Part{mean, m2};
        } else {
            float q = 0.f;
            for (int k = 0; k < cs; ++k) q += xch[k][0];
            part = Part{q, 0.f};
        }
    }
    const RowScale sc = scale_of_row<OP>(part, a.n, a.eps);
    if (t == 0 && rank == 0) {
        if (OP == OP_LAYERNORM && a.mean) a.mean[row] = sc.a;
        if (OP != OP_SOFTMAX && a.rstd) a.rstd[row] = sc.b;
    }
    const F2 ta2 = f2(sc.a), tb2 = f2(sc.b);
    const uint4* const gp = a.p0 + mine;
    const uint4* const bp = a.p1 + mine;
#pragma unroll
    for (int s = 0; s < NS; ++s) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = s * gstep + u * 32;
            if constexpr (LEN) {
                if (o + mine < lim) {
                    uint4 raw = myring[s * step + u * 32];
                    if (o + mine == straddle) raw = mask_tail<DT>(raw, keep);
                    st_stream(yr + o, apply_vec<OP, DT>(raw, gp + o, bp + o, ta2, tb2));
                } else if (o + mine < nvec) {
                    st_stream(yr + o, make_uint4(0, 0, 0, 0));
                }
            } else if (FULL || o + mine < nvec) {
                st_stream(yr + o, apply_vec<OP, DT>(myring[s * step + u * 32], gp + o, bp + o, ta2, tb2));
            }
        }
    }
}

using TwoFn = void (*)(const WArgs);

template <int NS, bool FULL, bool CL>
TwoFn fit_fn_c(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_twopass_fit<OP_SOFTMAX, DT_F32, 4, NS, FULL, CL>;
        case 1: return k_twopass_fit<OP_SOFTMAX, DT_BF16, 4, NS, FULL, CL>;
        case 2: return k_twopass_fit<OP_LAYERNORM, DT_F32, 4, NS, FULL, CL>;
        case 3: return k_twopass_fit<OP_LAYERNORM, DT_BF16, 4, NS, FULL, CL>;
        case 4: return k_twopass_fit<OP_RMSNORM, DT_F32, 4, NS, FULL, CL>;
        case 5: return k_twopass_fit<OP_RMSNORM, DT_BF16, 4, NS, FULL, CL>;
    }
    return nullptr;
}
template <int NS>
TwoFn fit_fn_b(int op, int dt, bool full, bool cl) {
    if (cl) return full ? fit_fn_c<NS, true, true>(op, dt) : fit_fn_c<NS, false, true>(op, dt);
    return full ? fit_fn_c<NS, true, false>(op, dt) : fit_fn_c<NS, false, false>(op, dt);
}
// softmax with per-row lengths (one CTA per row, or the CTAs of a cluster)
TwoFn fit_len_fn(int dt, int steps, bool cl) {
#define TF_FL(NS)                                                                                                                  \
    if (steps == NS) {                                                                                                             \
        if (cl) return dt == DT_F32 ? k_twopass_fit<OP_SOFTMAX, DT_F32, 4, NS, false, true, true> : k_twopass_fit<OP_SOFTMAX, DT_BF16, 4, NS, false, true, true>; \
        return dt == DT_F32 ? k_twopass_fit<OP_SOFTMAX, DT_F32, 4, NS, false, false, true> : k_twopass_fit<OP_SOFTMAX, DT_BF16, 4, NS, false, false, true>; \
    }
    TF_FL(1) TF_FL(2) TF_FL(3) TF_FL(4)
#undef TF_FL
    return nullptr;
}
// steps: what a CTA takes of the row (1 .. 4)
TwoFn fit_fn(int op, int dt, int steps, bool full, bool cl) {
    switch (steps) {
        case 1: return fit_fn_b<1>(op, dt, full, cl);
        case 2: return fit_fn_b<2>(op, dt, full, cl);
        case 3: return fit_fn_b<3>(op, dt, full, cl);
        case 4: return fit_fn_b<4>(op, dt, full, cl);
    }
    return nullptr;
}

template <int MAXT, int MINB, bool CL, bool CACHE>
TwoFn two_fn_c(int op, int dt, bool len) {
    if (len) {
        if (op != OP_SOFTMAX) return nullptr;
        return dt == DT_F32 ? k_twopass<OP_SOFTMAX, DT_F32, MAXT, MINB, CL, true, CACHE> : k_twopass<OP_SOFTMAX, DT_BF16, MAXT, MINB, CL, true, CACHE>;
    }
    switch (op * 2 + dt) {
        case 0: return k_twopass<OP_SOFTMAX, DT_F32, MAXT, MINB, CL, false, CACHE>;
        case 1: return k_twopass<OP_SOFTMAX, DT_BF16, MAXT, MINB, CL, false, CACHE>;
        case 2: return k_twopass<OP_LAYERNORM, DT_F32, MAXT, MINB, CL, false, CACHE>;
        case 3: return k_twopass<OP_LAYERNORM, DT_BF16, MAXT, MINB, CL, false, CACHE>;
        case 4: return k_twopass<OP_RMSNORM, DT_F32, MAXT, MINB, CL, false, CACHE>;
        case 5: return k_twopass<OP_RMSNORM, DT_BF16, MAXT, MINB, CL, false, CACHE>;
    }
    return nullptr;
}

template <int MAXT, int MINB>
TwoFn two_fn_b(int op, int dt, bool cl, bool len, bool cache) {
    if (cl) return cache ? two_fn_c<MAXT, MINB, true, true>(op, dt, len) : two_fn_c<MAXT, MINB, true, false>(op, dt, len);
    return cache ? two_fn_c<MAXT, MINB, false, true>(op, dt, len) : two_fn_c<MAXT, MINB, false, false>(op, dt, len);
}

TwoFn two_fn(int op, int dt, int threads, bool capped, bool cl, bool len, bool cache) {
    if (capped && threads <= 512) return two_fn_b<512, 3>(op, dt, cl, len, cache);
    if (capped && threads <= 768) return two_fn_b<768, 2>(op, dt, cl, len, cache);
    return two_fn_b<1024, 0>(op, dt, cl, len, cache);
}

template <int U, int MAXT, int MINB, bool CL>
TwoFn ring_fn_c(int op, int dt) {
    switch (op * 2 + dt) {
        case 0: return k_twopass_ring<OP_SOFTMAX, DT_F32, U, MAXT, MINB, CL>;
        case 1: return k_twopass_ring<OP_SOFTMAX, DT_BF16, U, MAXT, MINB, CL>;
        case 2: return k_twopass_ring<OP_LAYERNORM, DT_F32, U, MAXT, MINB, CL>;
        case 3: return k_twopass_ring<OP_LAYERNORM, DT_BF16, U, MAXT, MINB, CL>;
        case 4: return k_twopass_ring<OP_RMSNORM, DT_F32, U, MAXT, MINB, CL>;
        case 5: return k_twopass_ring<OP_RMSNORM, DT_BF16, U, MAXT, MINB, CL>;
    }
    return nullptr;
}
template <int U, int MAXT, int MINB>
TwoFn ring_fn_b(int op, int dt, bool cl) { return cl ? ring_fn_c<U, MAXT, MINB, true>(op, dt) : ring_fn_c<U, MAXT, MINB, false>(op, dt); }
// softmax with per-row lengths in the general ring form
TwoFn ring_len_fn(int dt, int threads, bool capped, bool cl) {
    if (capped && threads <= 384) {
        if (cl) return dt == DT_F32 ? k_twopass_ring<OP_SOFTMAX, DT_F32, 4, 384, 3, true, true> : k_twopass_ring<OP_SOFTMAX, DT_BF16, 4, 384, 3, true, true>;
        return dt == DT_F32 ? k_twopass_ring<OP_SOFTMAX, DT_F32, 4, 384, 3, false, true> : k_twopass_ring<OP_SOFTMAX, DT_BF16, 4, 384, 3, false, true>;
    }
    if (cl) return dt == DT_F32 ? k_twopass_ring<OP_SOFTMAX, DT_F32, 4, 1024, 1, true, true> : k_twopass_ring<OP_SOFTMAX, DT_BF16, 4, 1024, 1, true, true>;
    return dt == DT_F32 ? k_twopass_ring<OP_SOFTMAX, DT_F32, 4, 1024, 1, false, true> : k_twopass_ring<OP_SOFTMAX, DT_BF16, 4, 1024, 1, false, true>;
}
// regcap: the builds whose registers are held to what three CTAs per SM leave each thread: 56 for CTAs of up to 384
// threads, 40 for CTAs of up to 512
TwoFn ring_fn(int op, int dt, int unroll, int threads, bool capped, bool cl) {
    if (unroll == 2) return (capped && threads <= 512) ? ring_fn_b<2, 512, 3>(op, dt, cl) : ring_fn_b<2, 1024, 1>(op, dt, cl);
    if (unroll != 4) return nullptr;
    if (capped && threads <= 384) return ring_fn_b<4, 384, 3>(op, dt, cl);
    return (capped && threads <= 512) ? ring_fn_b<4, 512, 3>(op, dt, cl) : ring_fn_b<4, 1024, 1>(op, dt, cl);
}

}  // namespace

// Plan field `chunk`: bytes of each row's head kept in shared memory between the passes (0 = none); `rpg` = 2 selects
// the register-capped build (threads <= 768); `lanes`: row-order groups; `vpt`: L2 hint bits of the two passes.
bool supports_twopass(const Plan& p, const Args& a, const DeviceInfo& d) {
    if (p.cluster != 1 && p.cluster != 2 && p.cluster != 4 && p.cluster != 8) return false;
    if (p.cluster > 1 && (p.cluster > d.max_cluster || a.rows * p.cluster > 0x7FFFFFFF)) return false;
    if (p.lanes < 1 || p.lanes > 1024 || p.vpt < 0 || p.vpt > 3) return false;
    if (p.stages >= 2) {                                           // the ring form: no length mode, no separate cache
        if (p.stages > kRingMaxDepth || (p.unroll != 2 && p.unroll != 4) || p.chunk != 0) return false;
        const int64_t nvec = a.cols * elem_size(a.dt) / 16;
        if (a.len) {                                               // lengths: softmax rows that fit the ring of one CTA
            const int64_t step = static_cast<int64_t>(p.threads / 32) * p.unroll * 32;
            const bool fits = p.persist == 0 && p.rpg == 1 && ((nvec + step - 1) / step + p.cluster - 1) / p.cluster <= std::min(p.stages, 4);
            if (a.op != OP_SOFTMAX || p.lanes != 1 || p.unroll != 4 || a.rows * p.cluster > 0x7FFFFFFF) return false;
            if (!fits && p.rpg == 2 && p.threads > 384) return false;      // the general ring form: its 56-register build ends at 384 threads
        }
        if (nvec > 0x7FFFFFFF - 65536) return false;              // 32-bit vector indices inside the kernel
        return vector_ok(a) && (p.rpg == 1 || p.rpg == 2) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 &&
               (d.smem_optin == 0 || static_cast<int64_t>(p.stages) * p.threads * p.unroll * 16 + 1024 <= d.smem_optin);
    }
    if ((p.stages != 0 && p.stages != 1) || a.cols * elem_size(a.dt) / 16 < p.cluster) return false;
    return vector_ok(a) && (p.rpg == 1 || (p.rpg == 2 && p.threads <= 768)) && p.threads >= 32 && p.threads <= 1024 && p.threads % 32 == 0 && p.chunk >= 0 && p.chunk % 16 == 0 &&
           (d.smem_optin == 0 || p.chunk + 2048 <= d.smem_optin);
}

cudaError_t launch_twopass(const Plan& p, const Args& a, const DeviceInfo& d, cudaStream_t st) {
    const int cs = std::max(1, p.cluster);
    const bool ring = p.stages >= 2;
    TwoFn fn = ring ? ring_fn(a.op, a.dt, p.unroll, p.threads, p.rpg == 2, cs > 1) : two_fn(a.op, a.dt, p.threads, p.rpg == 2, cs > 1, a.len != nullptr, p.chunk > 0);
    if (!fn) return cudaErrorInvalidValue;
    const int groups = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(p.lanes, a.rows)));
    // a row that takes no more steps (per CTA of its cluster) than the ring has stages: the straight-line build
    int fit_steps = 0;
    if (ring && groups == 1 && p.persist == 0 && p.unroll == 4 && p.rpg == 1 && a.rows * cs <= 0x7FFFFFFF) {
        const int64_t nvec = a.cols * elem_size(a.dt) / 16;
        const int64_t step = static_cast<int64_t>(p.threads / 32) * p.unroll * 32;
        const int64_t steps = ((nvec + step - 1) / step + cs - 1) / cs;
        if (steps <= std::min(p.stages, 4)) {
            fit_steps = static_cast<int>(steps);
            fn = a.len ? (a.op == OP_SOFTMAX ? fit_len_fn(a.dt, fit_steps, cs > 1) : nullptr) : fit_fn(a.op, a.dt, fit_steps, steps * step * cs == nvec, cs > 1);
        }
    }
    if (ring && a.len && !fit_steps)                               // lengths in the general ring form: softmax, four vectors per step
        fn = (a.op == OP_SOFTMAX && p.unroll == 4 && groups == 1) ? ring_len_fn(a.dt, p.threads, p.rpg == 2, cs > 1) : nullptr;
    if (!fn) return cudaErrorInvalidValue;
    const int64_t slots = (a.rows + groups - 1) / groups * groups;
    int64_t grid = slots;                                          // in rows (clusters)
    if (p.persist > 0) grid = std::min<int64_t>(grid, std::max<int64_t>(1, static_cast<int64_t>(p.persist) * d.sms / cs));
    grid = std::min<int64_t>(grid, 0x7FFFFFFF / cs);
    WArgs k;
    k.x = static_cast<const uint4*>(a.x); k.p0 = static_cast<const uint4*>(a.p0); k.p1 = static_cast<const uint4*>(a.p1);
    k.y = static_cast<uint4*>(a.y); k.mean = a.mean; k.rstd = a.rstd; k.rows = a.rows; k.len = a.len;
    k.nvec = a.cols * elem_size(a.dt) / 16;
    k.n = static_cast<float>(a.cols); k.eps = a.eps;
    k.cs = cs; k.groups = groups; k.slots = slots; k.policy = p.vpt; k.per_group = slots / groups;
    k.step = (p.threads / 32) * p.unroll * 32;
    k.nfull = static_cast<int>(k.nvec / k.step);
    k.rag = static_cast<int>(k.nvec - static_cast<int64_t>(k.nfull) * k.step);
    k.cache_vecs = std::min<int64_t>((k.nvec + cs - 1) / cs, p.chunk / 16);
    k.stages = p.stages;
    const size_t smem = ring ? static_cast<size_t>(fit_steps ? fit_steps : p.stages) * p.threads * p.unroll * 16 : static_cast<size_t>(k.cache_vecs) * 16;
    if (smem > 0) {
        cudaError_t e = ensure_max_smem(reinterpret_cast<const void*>(fn), d);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = smem;
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
    note_launch(reinterpret_cast<const void*>(fn), grid * cs, p.threads, smem, cs);
    return cudaLaunchKernelEx(&cfg, fn, k);
}

}  // namespace tf
