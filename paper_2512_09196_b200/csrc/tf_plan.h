// Launch plans: which hand-written variant runs a problem and with what geometry.  Host and device.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace tf {

enum : int { DT_F32 = 0, DT_BF16 = 1 };
enum : int { OP_SOFTMAX = 0, OP_LAYERNORM = 1, OP_RMSNORM = 2, OP_COUNT = 3 };

enum Variant : int {
    V_WARP = 0,     // a group of 8/16/32 lanes holds one row in registers; several rows per warp for narrow rows
    V_CTA = 1,      // a CTA (or a cluster of CTAs) holds one row in registers; 16-byte coalesced loads
    V_TMA = 2,      // each CTA of a cluster stages its slice of the row in shared memory with bulk async copies
    V_STREAM = 3,   // generic: scalar accesses, several passes over the row, any alignment and length
    V_PIPE = 4,     // persistent CTAs: a producer thread streams row tiles into a shared-memory ring, consumer warps normalise
    V_RING = 5,     // persistent clusters: each CTA prefetches its slice of a long row into a shared-memory ring, registers hold it
    V_TWOPASS = 6,  // CTA per row, the row streamed twice with vector loads (second time from L2); any row length
    V_SPLIT = 7,    // few very long rows: a row cut into segments over many CTAs, partials merged through global scratch
    V_SROWS = 8,    // narrow LayerNorm / RMSNorm rows resident in shared memory, 1-8 lanes per row, y leaves as one bulk copy
    V_COUNT = 9
};

struct Plan {
    int variant = V_STREAM;
    int threads = 256;   // CTA size
    int lanes = 32;      // V_WARP / V_PIPE: threads per row
    int vpt = 1;         // V_WARP / V_CTA / V_PIPE: 16-byte vectors held per thread
    int rpg = 1;         // V_WARP: rows a group has in flight per iteration
    int cluster = 1;     // V_CTA / V_TMA / V_RING: CTAs sharing one row; V_SPLIT: segments per row
    int stages = 1;      // V_TMA / V_PIPE: shared-memory ring depth
    int chunk = 8192;    // V_TMA: bytes per bulk copy (one mbarrier each); V_PIPE: bytes per stage
    int persist = 0;     // 0: grid covers all rows once; k > 0: k CTAs per SM looping over rows (V_PIPE: always >= 1)
    int unroll = 4;      // V_TWOPASS with a ring (stages >= 2): 16-byte vectors per thread per ring stage (2 or 4)
};

struct Args {
    int op, dt;
    const void* x;
    const void* p0;      // gamma (LayerNorm) / weight (RMSNorm)
    const void* p1;      // beta (LayerNorm)
    void* y;
    float* mean;         // LayerNorm, nullable
    float* rstd;         // LayerNorm / RMSNorm, nullable
    int64_t rows, cols;
    float eps;
    int* status;         // device word that bounded waits set when they give up
    const void* r = nullptr;   // fused residual add: second input ...
    void* h = nullptr;         // ... and where x + r (rounded to the storage type) goes
    const int* len = nullptr;  // softmax with per-row valid lengths (elements), device memory
};

struct DeviceInfo {
    int ordinal = -1;
    int sms = 0;
    int smem_optin = 0;          // max dynamic shared memory per CTA, bytes
    int max_cluster = 8;
    int l2_bytes = 0;            // L2 cache size
};

// Geometry limits shared by the dispatcher and the kernels.
constexpr int kMaxCluster = 8;
constexpr int kMaxChunks = 32;       // bulk copies (mbarriers) per slice
constexpr int kMaxStages = 3;

// One launcher per kernel family.  `supports_*` is the host-side check that the plan's geometry can hold
// the row; `launch_*` enqueues on `stream` and returns the launch error.
bool supports_warp(const Plan&, const Args&, const DeviceInfo&);
bool supports_cta(const Plan&, const Args&, const DeviceInfo&);
bool supports_tma(const Plan&, const Args&, const DeviceInfo&);
bool supports_stream(const Plan&, const Args&, const DeviceInfo&);
bool supports_pipe(const Plan&, const Args&, const DeviceInfo&);
bool supports_ring(const Plan&, const Args&, const DeviceInfo&);
bool supports_twopass(const Plan&, const Args&, const DeviceInfo&);
bool supports_split(const Plan&, const Args&, const DeviceInfo&);
bool supports_srows(const Plan&, const Args&, const DeviceInfo&);
cudaError_t launch_warp(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_cta(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_tma(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_stream(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_pipe(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_ring(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_twopass(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_split(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_srows(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
// The split plan with caller-provided scratch (split_scratch_bytes() of device memory).
cudaError_t launch_split_with_scratch(const Plan&, const Args&, void* scratch, cudaStream_t);

// Fused residual add + norm (Args::r, Args::h set): register-resident plans only; heuristic_addnorm returns variant -1
// when none holds the row, and the caller then adds element-wise and runs the ordinary norm on h.
bool supports_addnorm(const Plan&, const Args&, const DeviceInfo&);
cudaError_t launch_addnorm(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
Plan heuristic_addnorm(const Args&, const DeviceInfo&);
cudaError_t launch_add_elementwise(const void* x, const void* r, void* h, int64_t n, int dt, cudaStream_t);

// Softmax with per-row valid lengths (Args::len set): register-resident plans and the two-pass plan; the scalar kernel
// serves what they cannot (unaligned tensors, widths that are not whole 16-byte vectors).
bool supports_softmax_len(const Plan&, const Args&, const DeviceInfo&);
cudaError_t launch_softmax_len(const Plan&, const Args&, const DeviceInfo&, cudaStream_t);
cudaError_t launch_softmax_len_scalar(const Args&, cudaStream_t);
Plan heuristic_softmax_len(const Args&, const DeviceInfo&);
size_t split_scratch_bytes(const Plan&, const Args&);

// What the launcher of a forward plan last launched on this host thread (kernel, grid, CTA size, dynamic shared memory,
// CTAs per cluster): the tuner's refinement hint reads the kernel's registers and its occupancy from these.
struct LaunchFacts { const void* fn = nullptr; int64_t grid = 0; int threads = 0; size_t dyn_smem = 0; int cluster = 1; };
void note_launch(const void* fn, int64_t grid, int threads, size_t dyn_smem, int cluster);
LaunchFacts last_launch();

// Bookkeeping shared with the C ABI layer: count kernel launches; remember the CUDA error behind a TF_ERR_CUDA.
void count_launches(int n);
void clear_norm_bwd_tuned();   // forgets what tf_tune_norm_bwd kept
int* device_status_word();     // this device's status word (bounded waits set it when they give up), or null before first use fails
void remember_cuda_error(cudaError_t e);

// Raises a kernel's dynamic shared-memory limit to the device's opt-in maximum, once per kernel and device.
cudaError_t ensure_max_smem(const void* fn, const DeviceInfo&);

inline int elem_size(int dt) { return dt == DT_F32 ? 4 : 2; }
inline bool vector_ok(const Args& a) {          // 16-byte vectors usable on every tensor
    auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return (a.cols * elem_size(a.dt)) % 16 == 0 && al(a.x) && al(a.y) && al(a.p0) && al(a.p1);
}

}  // namespace tf
