/* tf.h — C ABI of libtf.so: fused row-wise reduce-then-normalise forward kernels for NVIDIA B200
 * (sm_100a), with a measure-and-keep tuner.
 *
 * The ops are the memory-bound kernel class the TritonForge paper's loop is aimed at (Section 2 lists
 * "softmax variants" and fused operators among the hand-optimised Triton kernels it wants to automate);
 * the paper defines none of them, so each declaration below states the standard definition it computes.
 * tf_tune is that paper's Algorithm 1 in miniature: candidates are proposed, run, timed on the device
 * and kept only if the measured time improves on the best so far.
 *
 * Conventions for every *_fwd entry point
 *   Memory     All tensor pointers are DEVICE memory owned by the caller, on the current CUDA device.
 *              The library keeps no reference after the call returns.  It allocates nothing, with one
 *              exception: for a handful of very long rows (rows <= 4, >= 256 KiB each) the split-row plan takes
 *              8 bytes per row segment from the stream-ordered allocator (cudaMallocAsync / cudaFreeAsync on the
 *              caller's stream) for the duration of the call, so that calls on different streams cannot race on
 *              shared scratch.  Callers that must never allocate use tf_softmax_fwd_noalloc, or force another
 *              plan for such shapes (tf_force_plan).
 *   Layout     x and y are dense row-major [rows, cols] (row stride = cols); gamma/beta/weight are [cols];
 *              mean/rstd are [rows], always fp32.  x, y and the parameters share one element type `dt`.
 *   Alignment  Any.  A 16-byte aligned x, y and parameters with cols * sizeof(element) a multiple of 16
 *              unlock the vectorised and TMA-staged variants; anything else runs on the generic variant.
 *   Aliasing   y == x (exactly) is allowed; partial overlap is undefined.
 *   Async      Work is enqueued on `cuda_stream` (a cudaStream_t; NULL = the default stream) and the call
 *              returns without synchronising.
 *   Numerics   Arithmetic in fp32, one round-to-nearest-even conversion to the output type at the end,
 *              subnormal results kept (never flushed to zero).
 *   Errors     Return codes only; arguments are checked before any CUDA call.  rows == 0 is a no-op.
 *   Threads    Entry points may be called from several host threads.
 */
#ifndef TF_H_
#define TF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TF_OK = 0,
    TF_ERR_INVALID_ARG = 1,   /* null required pointer, rows < 0, cols <= 0, bad enum, eps negative or NaN */
    TF_ERR_UNSUPPORTED = 2,   /* size overflow, or a forced plan that cannot run this shape */
    TF_ERR_CUDA = 3,          /* a CUDA call failed: see tf_last_cuda_error() */
    TF_ERR_TIMEOUT = 4,       /* a bounded device-side wait gave up: see tf_device_status() */
    TF_ERR_NOMEM = 5          /* tf_tune could not allocate its scratch tensors */
} tf_status;

typedef enum { TF_F32 = 0, TF_BF16 = 1 } tf_dtype;
typedef enum { TF_OP_SOFTMAX = 0, TF_OP_LAYERNORM = 1, TF_OP_RMSNORM = 2 } tf_op;

/* Softmax over the last axis: y[r,j] = exp(x[r,j] - m_r) / sum_k exp(x[r,k] - m_r), m_r = max_k x[r,k].
 * No temperature.  A mask is expressed in the data: x = -inf gives exactly +0; a row that is -inf
 * throughout gives +0 everywhere (not NaN). */
tf_status tf_softmax_fwd(const void* x, void* y, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* LayerNorm: mu_r = mean_j x[r,j]; var_r = mean_j (x[r,j] - mu_r)^2 (divisor cols);
 * rstd_r = 1/sqrt(var_r + eps); y[r,j] = (x[r,j] - mu_r) * rstd_r * gamma[j] + beta[j].
 * gamma and beta are required.  mean and rstd are optional outputs (NULL to skip). */
tf_status tf_layernorm_fwd(const void* x, const void* gamma, const void* beta, void* y, float* mean, float* rstd,
                           int64_t rows, int64_t cols, float eps, tf_dtype dt, void* cuda_stream);

/* RMSNorm: rrms_r = 1/sqrt(mean_j x[r,j]^2 + eps); y[r,j] = x[r,j] * rrms_r * weight[j], rounded once.
 * weight is required; rstd (= rrms) is an optional output. */
tf_status tf_rmsnorm_fwd(const void* x, const void* weight, void* y, float* rstd, int64_t rows, int64_t cols,
                         float eps, tf_dtype dt, void* cuda_stream);

/* Softmax (same definition and conventions as tf_softmax_fwd) for callers that must not trigger a device
 * allocation: a process that handed all free device memory to its own pool at start-up (a later driver
 * allocation could fail or stall there), or a latency-critical loop in which an allocation call may
 * synchronise the device.  The paper has no counterpart; this exists for deployment.
 * It always runs the split-row plan (each row cut into segments over many CTAs, one 8-byte partial per
 * segment) with the partials in a fixed 64 KiB array inside the library (room for 8192 partials; every GPU
 * that loads the library holds it until the process exits).  It calls no cudaMalloc / cudaFree or any other
 * allocating routine.
 *   Limits   rows <= 8192; x and y 16-byte aligned and cols * sizeof(element) a multiple of 16.  Anything else
 *            returns TF_ERR_UNSUPPORTED and launches nothing.  Long rows are its purpose; short ones work
 *            but are served better by tf_softmax_fwd.
 *   Set-up   The first call on a device looks up the array's device address (with that device current).  That
 *            first use of the library on a device is also when the CUDA runtime loads the library's module
 *            onto it -- the kernels' code and this 64 KiB array occupy device memory from then on, and the
 *            runtime takes that memory itself.  So make the first call on each device early: before the
 *            process hands the remaining free memory to its pool, and before any stream capture begins.
 *            Later calls touch no allocator at all.
 *   Sharing  Every call on a device uses the same array, which keeps the previous call's partials.  Nothing in
 *            it needs clearing (each call overwrites every partial it later reads), but two calls whose
 *            kernels can overlap on the GPU (different streams without an ordering between them) race on it:
 *            order such calls yourself. */
tf_status tf_softmax_fwd_noalloc(const void* x, void* y, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* Measure-and-keep tuning for one (op, rows, cols, dt) on the current device (Algorithm 1 of the paper,
 * with the hand-written launch plans as proposals): starting from the heuristic plan as incumbent, every
 * candidate plan that can launch is run on library-owned scratch tensors, its output is checked against
 * the incumbent's at the level of the parity tolerances (two results that both meet them: 2 bf16 ulps, 2e-5 of the
 * condition scale in fp32), it is timed with CUDA events (3 warm-up batches + 5 timed regions of at least 2 ms each,
 * median; the paper's Section 3.4 protocol of 3 + 5 runs, with each run made long enough to time) on at least two
 * rotating buffer sets larger than L2, and it replaces the incumbent only if it is at least 2% faster.  A candidate
 * that cannot launch, fails that check, or whose bounded device-side wait gives up is dropped and never cached (the
 * remediation branch of Algorithm 1).  The library's own streaming copy of the same tensors is timed the same way as
 * the ceiling of the shape: tuning ends at once when the incumbent is within 2% of it, and the proposal list is cut
 * short when a proposal gets there.  After the proposals come refinement rounds: the one-parameter neighbours of the
 * best plan, the knobs named by the refinement hint first (see tf_refine_hint), a round ending at the first accepted
 * candidate ("continue") and refinement ending after a round without one ("finish"), at most 8 rounds (the paper's
 * iteration cap).  The winner is cached in memory (and in the file named by the TF_TUNE_CACHE
 * environment variable, if set) and used by later *_fwd calls with the same key.  Blocking; allocates and
 * frees its own scratch; assumes 16-byte aligned tensors. */
tf_status tf_tune(tf_op op, int64_t rows, int64_t cols, tf_dtype dt);

/* The same loop, timed on the caller's data instead of synthetic values: the contents of x (device, [rows, cols])
 * and, if given, of the parameter vectors p0 (gamma / weight) and p1 (beta) are copied into the tuner's scratch
 * tensors; the caller's tensors are only read.  Worth it when the data changes the cost, e.g. a masked softmax
 * whose -inf tails cost no exponentials.  (The paper's loop likewise profiles on the kernel's own test inputs,
 * Section 3.2.) */
tf_status tf_tune_like(tf_op op, const void* x, const void* p0, const void* p1, int64_t rows, int64_t cols, tf_dtype dt);

/* Result of the last tf_tune on this thread: number of candidates timed, median microseconds of the
 * heuristic plan and of the winner.  Any pointer may be NULL. */
tf_status tf_tune_report(int* candidates_timed, float* heuristic_us, float* best_us);

/* ---- calibration kernels --------------------------------------------------------------------------- */

/* Device copy of `bytes` bytes written in the same load/store style as the row kernels (16-byte streaming
 * accesses, four in flight per thread, one contiguous block per CTA, programmatic launch): the practical ceiling for "bytes in, bytes out" on
 * this GPU at a given size, which the bench prints beside every result.  x and y must not overlap.  Any
 * alignment (the vector path needs both 16-byte aligned). */
tf_status tf_copy(const void* x, void* y, int64_t bytes, void* cuda_stream);

/* y[i] = sin(x[i]) over n elements: the element-wise kernel of the paper's Case Study 1, whose only tuning knob is
 * its launch geometry (the paper's baseline used blocks of 4 elements; the fix was an autotune over block sizes).
 * threads per CTA (multiple of 32, <= 1024) and 16-byte vectors per thread (1, 2, 4 or 8) are that knob here -- a
 * CTA covers threads x vectors_per_thread vectors, its "block size"; 0 selects the defaults (64 threads, 4 vectors
 * per thread).
 * fp32 arithmetic with full range reduction, one rounding to the storage type (2-byte elements below 2^15 in
 * magnitude take a shorter fp32 evaluation whose rounded results are the same).  y == x is allowed. */
tf_status tf_sin_fwd(const void* x, void* y, int64_t n, tf_dtype dt, int threads, int vectors_per_thread, void* cuda_stream);

/* ---- softmax with per-row valid lengths ------------------------------------------------------------------ */

/* Row r is normalised over its first len[r] entries: y[r, j] = softmax(x[r, 0:len[r]])_j for j < len[r] and +0 for
 * j >= len[r]; the contents of x[r, j >= len[r]] are ignored (anything, NaN included; x must still be a whole
 * [rows, cols] allocation) and for 2-byte rows of 4 KiB and more and any rows of 16 KiB and more they are not read at
 * all; len[r] = 0 gives an all +0 row,
 * values outside [0, cols] are clamped.  Equal, bit for bit where the same plan runs, to tf_softmax_fwd on an x whose
 * tails hold -inf.  The paper has no counterpart (its kernels take their masks in the data).
 * x, y: [rows, cols] row-major device memory (y may alias x); len: int32 [rows], device memory; cols <= 2^31 - 1.
 * Errors and stream behaviour as tf_softmax_fwd, plus TF_ERR_INVALID_ARG for a null len.  Allocates nothing. */
tf_status tf_softmax_len_fwd(const void* x, const int32_t* len, void* y, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* ---- log-softmax forward, softmax backward ----------------------------------------------------------------- */

/* y_j = (x_j - m) - ln sum_k exp(x_k - m), m = max_k x_k, over the last axis of x [rows, cols].  Entries with x_j = -inf
 * give -inf; a row that is -inf throughout gives -inf throughout (the logarithm of the all-zero reading of softmax).
 * fp32 arithmetic, one rounding to the storage type.  y may alias x.  The paper has no counterpart. */
tf_status tf_log_softmax_fwd(const void* x, void* y, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* dx_j = y_j * (dy_j - sum_k y_k dy_k): the backward pass of softmax from its stored output y and the incoming
 * gradient dy, all [rows, cols] of one element type; fp32 arithmetic, one rounding.  dx may alias y or dy.
 * Both calls: device pointers, asynchronous on cuda_stream, allocate nothing; TF_ERR_INVALID_ARG for a null pointer
 * with rows > 0, cols <= 0 or an unknown element type; rows = 0 is a no-op.  16-byte aligned tensors whose rows are
 * whole 16-byte vectors are held in registers up to 32 KiB per row and streamed in two passes beyond; when such long rows
 * are too few to fill the device with one CTA each, the 2-8 CTAs of a thread-block cluster share a row.  Anything else
 * runs scalar passes. */
tf_status tf_softmax_bwd(const void* y, const void* dy, void* dx, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* dx_j = dy_j - exp(y_j) * sum_k dy_k: the backward pass of log-softmax from its stored output y (log-probabilities) and
 * the incoming gradient dy; with dy = -e_t it is the gradient of a cross-entropy loss, softmax(x) - e_t.  exp(-inf) = 0:
 * masked entries pass their gradient through.  fp32 arithmetic, one rounding; probabilities in the subnormal range are
 * not flushed.  Same layouts, aliasing, forms and errors as tf_softmax_bwd.  The paper has no counterpart. */
tf_status tf_log_softmax_bwd(const void* y, const void* dy, void* dx, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* ---- backward passes of the norms ------------------------------------------------------------------------- */

/* From the forward pass's inputs and its stored fp32 statistics (mean, rstd: [rows]):
 *     xh_j = (x_j - mean) rstd   (RMSNorm: x_j rstd),   g_j = dy_j gamma_j
 *     dx_j = rstd (g_j - mean_k g_k - xh_j mean_k (g_k xh_k))          (RMSNorm: without the mean_k g_k term)
 *     dgamma_j = sum over rows of dy_j xh_j,   dbeta_j = sum over rows of dy_j   (LayerNorm only)
 * fp32 arithmetic; dx, dgamma, dbeta are rounded once to the storage type; the column sums are accumulated in fp32
 * in a fixed order (deterministic).  x, dy, dx: [rows, cols]; gamma / weight, dgamma / dweight, dbeta: [cols]; dx may
 * alias x or dy.  workspace: device memory of at least tf_norm_bwd_workspace_bytes(rows, cols) bytes, 4-byte aligned,
 * used for partial column sums while the call runs (calls that may overlap on the GPU need separate workspaces); it
 * is required when the tensors are 16-byte aligned with rows of whole 16-byte vectors and up to 65,536 columns, and
 * ignored otherwise (such shapes run two plain kernels).  Rows one CTA cannot hold (more than 8,192 columns) are shared
 * by the CTAs of a thread-block cluster.  rows = 0 zeroes the parameter gradients.
 * Errors: TF_ERR_INVALID_ARG for a null pointer, cols <= 0, an unknown element type or a missing / short workspace.
 * Asynchronous on cuda_stream; allocates nothing.  The paper has no counterpart. */
size_t tf_norm_bwd_workspace_bytes(int64_t rows, int64_t cols);
tf_status tf_layernorm_bwd(const void* x, const void* gamma, const void* dy, const float* mean, const float* rstd, void* dx,
                           void* dgamma, void* dbeta, void* workspace, size_t workspace_bytes, int64_t rows, int64_t cols,
                           tf_dtype dt, void* cuda_stream);
tf_status tf_rmsnorm_bwd(const void* x, const void* weight, const void* dy, const float* rstd, void* dx, void* dweight,
                         void* workspace, size_t workspace_bytes, int64_t rows, int64_t cols, tf_dtype dt, void* cuda_stream);

/* The measure-and-keep loop of tf_tune (Algorithm 1, Sections 3.3-3.4 of the paper) over the forms of the norm backward
 * pass of `op` (TF_LAYERNORM or TF_RMSNORM) on this shape: the automatic choice is the incumbent, every other form that
 * can run the shape is launched, timed (3 warm-up + 5 timed batches on rotating buffers, CUDA events, median) and kept
 * only if more than 2 % faster; a form whose bounded waits give up is dropped.  Blocking; owns its scratch (about
 * 256 MiB or three tensors twice, whichever is more); later calls of the same op, shape and type on this device use the
 * winner (tf_clear_cache forgets it).  tf_tune_norm_bwd_report: forms timed, automatic and best time of the last call on
 * this thread.  TF_ERR_INVALID_ARG for another op, rows <= 0 or cols <= 0; TF_ERR_NOMEM without room for the scratch. */
tf_status tf_tune_norm_bwd(tf_op op, int64_t rows, int64_t cols, tf_dtype dt);
tf_status tf_tune_norm_bwd_report(int* forms_timed, float* automatic_us, float* best_us);

/* ---- fused residual add + norm ------------------------------------------------------------------------ */

/* h = x + r (fp32 add, ONE rounding to the storage type), then the LayerNorm / RMSNorm defined above applied to that
 * rounded h: bit for bit the result of an add followed by tf_layernorm_fwd / tf_rmsnorm_fwd, with x and r read once
 * and h and y written once.  The paper names fused operators as a class of its targets (Section 2) and defines none;
 * this is the residual-stream update of pre-norm transformer blocks.
 * x, r, h, y: [rows, cols] row-major, device memory, one element type; h may alias x or r, y may alias x; h and y must
 * not overlap each other.  gamma / beta / weight, mean / rstd, eps, errors and stream behaviour as for the unfused
 * calls, plus TF_ERR_INVALID_ARG for a null r or h.  Rows of up to 64 KiB on 16-byte aligned tensors run as one
 * kernel; anything else as an element-wise add followed by the unfused op (same results; what the unfused op says
 * about memory holds for that second step). */
tf_status tf_add_layernorm_fwd(const void* x, const void* r, const void* gamma, const void* beta, void* h, void* y, float* mean,
                               float* rstd, int64_t rows, int64_t cols, float eps, tf_dtype dt, void* cuda_stream);
tf_status tf_add_rmsnorm_fwd(const void* x, const void* r, const void* weight, void* h, void* y, float* rstd, int64_t rows,
                             int64_t cols, float eps, tf_dtype dt, void* cuda_stream);
/* tf_tune for the fused form of TF_OP_LAYERNORM / TF_OP_RMSNORM: measures the register-resident plans on synthetic
 * data and caches the fastest under its own key.  TF_ERR_UNSUPPORTED when no such plan holds the row (the two-kernel
 * route is then used, and there is nothing to choose); TF_ERR_INVALID_ARG for TF_OP_SOFTMAX.  Blocking. */
tf_status tf_tune_add(tf_op op, int64_t rows, int64_t cols, tf_dtype dt);

/* ---- second memory-bound workload -------------------------------------------------------------------- */

/* Batched vector-matrix product (the paper's Case Study 2, "GEMV restructuring"):
 *     C[m,n] = sum_{k<K} A[m,k] * B[m,n,k]
 * A is [M, K], B is [M, N, K] with k contiguous, C is [M, N]; all dense, device memory, one element type.
 * Products are exact in fp32, accumulation is fp32, C gets one round-to-nearest-even conversion.  B is read once:
 * the operation is bound by HBM bandwidth.  Launch geometry, every knob 0 = automatic:
 *   threads  per CTA, a multiple of 32, at most 1024;
 *   lanes    per row group on the plain path (4, 8, 16 or 32); bf16 with lanes = 0 takes the tensor-core path;
 *            lanes = 1 selects the shared-memory staged path (bulk copies into a four-stage ring; rows, ksplit ignored);
 *   rows     consecutive n that share one load of the A[m,:] pieces: 1, 2 or 4 per lane group on the plain path,
 *            16 or 32 per warp on the tensor-core path;
 *   ksplit   warps of a CTA that share a row group along k (1, 2, 4 or 8; on the plain path only with lanes = 32,
 *            and never more than threads / 32).
 * 16-byte aligned A and B with K * sizeof(element) a multiple of 16 take a vector path, anything else a scalar one.
 * Errors: TF_ERR_INVALID_ARG for a null pointer with M*N > 0, K <= 0, an unknown element type or a knob outside its
 * set; TF_ERR_UNSUPPORTED when the grid would exceed 2^31 - 1 CTAs.  Asynchronous on cuda_stream; allocates nothing;
 * A, B, C stay the caller's. */
tf_status tf_bvecmat_fwd(const void* A, const void* B, void* C, int64_t M, int64_t N, int64_t K, tf_dtype dt, int threads,
                         int lanes, int rows, int ksplit, void* cuda_stream);

const char* tf_status_string(tf_status s);

/* cudaError_t value behind the most recent TF_ERR_CUDA on the calling thread (0 if none). */
int tf_last_cuda_error(void);

/* Synchronises the current device, then returns TF_ERR_TIMEOUT if any kernel since the last call gave up
 * on a bounded wait (its output rows are then undefined), else TF_OK.  Clears the flag. */
tf_status tf_device_status(void);

/* ---- test and bench hooks ------------------------------------------------------------------------- */

/* Plans are written as "variant:key=value,..." e.g. "cta:threads=256,vpt=2", "warp:lanes=8,vpt=1,rpg=4",
 * "tma:threads=512,cluster=4,stages=1", "srows:threads=128,lanes=4,vpt=8" (LayerNorm / RMSNorm rows of up to
 * lanes x vpt 16-byte vectors, resident in shared memory), "twopass:threads=256,stages=2,u=4", "stream:threads=256".
 * tf_force_plan makes every later call of `op`
 * use that plan (NULL or "" returns to automatic choice); a forced plan that cannot run a given shape
 * makes the call return TF_ERR_UNSUPPORTED. */
tf_status tf_force_plan(tf_op op, const char* plan);

/* Writes the plan the dispatcher would use now for this problem (forced > tuned > heuristic), assuming
 * 16-byte aligned tensors if aligned != 0. */
tf_status tf_query_choice(tf_op op, int64_t rows, int64_t cols, tf_dtype dt, int aligned, char* buf, size_t n);

/* Number of candidate plans tf_tune would consider for this problem, and the index-th of them as text. */
int tf_candidate_count(tf_op op, int64_t rows, int64_t cols, tf_dtype dt);
tf_status tf_candidate(tf_op op, int64_t rows, int64_t cols, tf_dtype dt, int index, char* buf, size_t n);

/* Whether tf_log_softmax_fwd / tf_softmax_bwd share a row among the CTAs of a thread-block cluster: 0 = automatic (rows
 * beyond 32 KiB), 1 = never, 2 / 4 / 8 = that many CTAs per row wherever the slices fit.  TF_ERR_INVALID_ARG otherwise. */
tf_status tf_softmax_variants_force(int cluster);

/* Which form of the norm backward passes runs on shapes that several serve.  path: 0 = automatic, 1 = rows requested
 * into registers one row ahead, 2 / 3 / 4 = rows staged in a shared-memory ring by bulk copies with up to 512 / 256 / 64
 * threads per row.  stages = ring depth (0 = automatic, at most 8).  cluster: 0 = automatic (a thread-block cluster shares
 * a row only when one CTA cannot hold it), 1 = never, 2 / 4 / 8 = that many CTAs per row wherever the slices fit.  Ask
 * tf_norm_bwd_workspace_bytes again after changing it.  TF_ERR_INVALID_ARG outside those values.  A forced choice takes
 * precedence over a tuned one. */
tf_status tf_norm_bwd_force(int path, int stages, int cluster);

/* Writes what tf_layernorm_bwd / tf_rmsnorm_bwd (op = TF_LAYERNORM / TF_RMSNORM) would use now for this shape as
 * "path=P,stages=S,cluster=C" in the terms of tf_norm_bwd_force (forced > tuned > automatic = all zero). */
tf_status tf_norm_bwd_choice(tf_op op, int64_t rows, int64_t cols, tf_dtype dt, char* buf, size_t n);

/* The refinement hint of tf_tune (Algorithm 1's Targeted-Refinement-Hint step, rule-based here): what the library reads
 * about a plan's launch without a profiler -- registers and resident CTAs of its kernel, waves of its grid and the empty
 * share of the last one, bytes in flight per SM -- and the rule that fires on it:
 *   occupancy  (<= 25 % resident threads and > 96 registers)  try fewer vectors or rows per thread, smaller CTAs first
 *   tail       (more than 15 % of the last wave empty)        try persistent CTAs or finer units of work first
 *   inflight   (less than 40 KB in flight per SM)             try deeper rings, larger stages, more resident threads first
 *   ceiling    (within 2 % of the library's own copy of the same tensors; tf_tune only)   finish
 * tf_refine_hint launches `plan` once on zero-filled scratch tensors of this shape and writes
 * "rule=... regs=... ctas_per_sm=... occupancy=... waves=... tail=... inflight_kb=... vs_copy=... first=<plan>;<plan>;<plan>"
 * (the first neighbours the refinement would try).  tf_tune_last_hint writes the hint tf_tune computed for the heuristic
 * plan in its last run on the calling thread. */
tf_status tf_refine_hint(tf_op op, int64_t rows, int64_t cols, tf_dtype dt, const char* plan, char* buf, size_t n);
tf_status tf_tune_last_hint(char* buf, size_t n);

/* Forgets every tuned plan in memory; if the environment variable TF_TUNE_CACHE names a file, the next call reads the
 * plans stored there again. */
void tf_clear_cache(void);

/* The bounded wait that every staged kernel of this library uses, on its own: launches one small kernel on `cuda_stream`
 * that brings 16 bytes from src16 (device memory, 16-byte aligned) into shared memory with a bulk copy but arms the
 * barrier for 32, so its wait can only end by running out of `budget_cycles` SM clock cycles (1 .. 2e9; a millisecond is
 * about 2e6).  The kernel then records the timeout like any other kernel (tf_device_status() returns TF_ERR_TIMEOUT
 * once), writes 1 to *gave_up (device memory; 0 if the wait was satisfied) and returns; nothing traps or spins without a
 * bound, and the device stays usable.  The paper has no counterpart: it exercises the remediation branch of its loop,
 * where a candidate whose run fails is dropped (Algorithm 1), from the device side. */
tf_status tf_debug_wait_probe(const void* src16, int64_t budget_cycles, int* gave_up, void* cuda_stream);

/* Host-side fault injection for tf_tune: while plan_prefix is non-empty, every candidate whose plan text starts with it
 * is treated as if one of its bounded waits had given up (the status word is set from the host after its run), so the
 * tuner must drop it: never time it, never cache it.  NULL or "" switches the injection off. */
tf_status tf_debug_tune_inject_timeout(const char* plan_prefix);

/* Number of kernels this library has launched since it was loaded (all threads). */
int64_t tf_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TF_H_ */
