/*
 * cocod.h -- C boundary of the B200 CoCoD-SGD parameter engine (libcocod.so).
 *
 * The engine holds K simulated workers (the paper's N) as replicas in one GPU's HBM and runs
 * the per-round parameter path of Algorithm 1 ("CoCoD-SGD") of arxiv 1906.12043:
 *
 *     cocod_comm_begin   Step I   store x_t^i, start averaging the stored copies (side stream)
 *     cocod_local_step   Step II  one local update of every worker (compute stream), k times
 *     cocod_comm_end     line 6   x^i <- x_hat_t + (x^i - x_t^i)
 *
 * Conventions
 *   - Plain C, opaque handle, every call returns an int: 0 = COCOD_OK, negative = error.
 *     Nothing throws or aborts.  cocod_strerror() names a code.
 *   - Layout: every K x P matrix is worker-major row-major fp32 with row stride P
 *     (row i = worker i's flattened model of P parameters, the paper's d).
 *   - Ownership: the engine owns x, the momentum v, the stored copies and the average model;
 *     the caller owns gradient buffers and CUDA streams and must keep a gradient buffer valid
 *     and unmodified until the compute stream has passed the call that reads it.
 *   - "device" pointers are CUDA device pointers on the device that was current at
 *     cocod_create; "host" pointers are ordinary (preferably pinned) host memory.
 *   - Streams are passed as void* holding a cudaStream_t (NULL = the legacy default stream).
 *   - All device work is stream-ordered and asynchronous; no call blocks the host except
 *     cocod_sync, cocod_comm_wait, cocod_destroy and the transfers that name host memory.
 *   - One host thread per handle (not thread-safe).  The device that was current at
 *     cocod_create must be current for every later call on the handle.
 *   - There is no CPU fallback: without a CUDA device every call fails with COCOD_ERR_CUDA.
 */
#ifndef COCOD_H
#define COCOD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cocod_engine cocod_handle;
typedef void *cocod_stream_t; /* a cudaStream_t */

enum {
    COCOD_OK = 0,
    COCOD_ERR_INVALID = -1, /* bad argument (NULL, K < 1, P < 1, non-finite hyper-parameter, ...) */
    COCOD_ERR_OOM = -2,     /* device or pinned-host allocation failed; nothing is leaked */
    COCOD_ERR_STATE = -3,   /* call not legal now (comm_end without comm_begin, double begin) */
    COCOD_ERR_CUDA = -4,    /* a CUDA call or kernel failed; sticky, see cocod_last_cuda_error */
    COCOD_ERR_TIMEOUT = -5, /* cocod_comm_wait ran out of time; the engine is still usable */
    COCOD_ERR_TOO_LARGE = -6 /* the request exceeds a fixed capacity (see cocod_kernel_local_step_host_noalloc) */
};

/* Options for cocod_set_option. */
enum {
    /* How Step I keeps its copy of x_t^i.  COPY: a copy kernel writes the stored copies (8 B per
     * worker-parameter per round).  FLIP (default): the buffer holding x becomes the stored
     * copy and the first local step of the round writes x into the spare buffer (0 B); the
     * values are identical. */
    COCOD_OPT_SNAPSHOT = 1,
    /* Record CUDA events around every kernel and let the kernels stamp their own start and end on the GPU's
     * clock (cocod_profile_*). 0 = off (default).  Switching it on the first time allocates 256 KB on the device. */
    COCOD_OPT_PROFILE = 2,
    /* Keep a bfloat16 copy of x (K x P, same layout) current: the local-step and merge kernels
     * write bf16(x) next to x (22 B and 14 B + 4/K per worker-parameter instead of 20 and
     * 12 + 4/K).  For workloads that compute gradients from bf16 weights with an fp32 master
     * copy.  1 allocates it, 0 frees it.  Not while a communication is in flight. */
    COCOD_OPT_BF16_SHADOW = 3,
    /* 1: consecutive local-step / merge kernels walk the K x P vector in alternating directions (and the mean kernel
     * against the kernel that last wrote x), so that each starts on what its predecessor left in the L2 cache.
     * Same values bit for bit.  0 (default): every kernel walks forwards. */
    COCOD_OPT_SWEEP = 4
};
enum { COCOD_SNAPSHOT_COPY = 0, COCOD_SNAPSHOT_FLIP = 1 };

/* Kernel kinds reported by cocod_profile_get. */
enum { COCOD_KERNEL_LOCAL_STEP = 0, COCOD_KERNEL_SNAPSHOT = 1, COCOD_KERNEL_MEAN = 2, COCOD_KERNEL_MERGE = 3,
       COCOD_KERNEL_STEP_MERGE = 4 };

/* ---------------------------------------------------------------------------------------------
 * Algorithm 1, "Input" / "Initialize": K workers, model size P, learning rate gamma = lr, and
 * the optimizer constants of Section 5.1 (momentum mu, weight decay wd).  Allocates x, v, the
 * stored copies (K x P fp32 each) and the average model (P) on the current device, zero-fills
 * x and v, uses equal mini-batch sizes, the legacy default stream as compute stream, and the
 * FLIP snapshot.  *out is written only on success.
 * Errors: INVALID (out NULL, K < 1 or > 1024, P < 1, K*P*4 overflows, lr/mu/wd not finite),
 * OOM, CUDA. */
int cocod_create(cocod_handle **out, int K, int64_t P, float lr, float mu, float wd);

/* Waits for the engine's pending device work, frees everything.  NULL is a no-op. */
int cocod_destroy(cocod_handle *h);

/* Algorithm 1, Step II body, one iteration tau for every worker, with the optimizer of the
 * paper's experiments (Section 5.1; PyTorch SGD form, v starts at 0):
 *     d = g + wd * x ;  v = mu * v + d ;  x = x - lr * v
 * (mu = wd = 0 is Algorithm 1's x <- x - gamma G literally.)  grads: device, K x P, borrowed.
 * Asynchronous on the compute stream.  Legal with or without a communication in flight. */
int cocod_local_step(cocod_handle *h, const float *grads);

/* Same update with the gradients in HOST memory (K x P): the engine stages them to the device
 * in chunks on an internal copy stream, overlapping the copies with the update kernel.  The
 * host buffer must stay valid until cocod_sync (or a later blocking call) returns. */
int cocod_local_step_host(cocod_handle *h, const float *host_grads);

/* Algorithm 1, Step I: store x_t^i and start computing the weighted mean of the stored copies
 * x_hat_t = sum_i (M_i / sum_j M_j) x_t^i, concurrently with Step II: the mean kernel runs on
 * `side`, ordered after the compute stream's work so far.  side == compute stream is allowed
 * (then it simply runs in order).  Errors: STATE if a communication is already in flight. */
int cocod_comm_begin(cocod_handle *h, cocod_stream_t side);

/* Algorithm 1, line 6: once the mean is complete (stream-ordered wait, the host does not
 * block), x^i <- x_hat_t + (x^i - x_t^i) for every worker.  Errors: STATE without a begin. */
int cocod_comm_end(cocod_handle *h);

/* A fusion variant of the round: the LAST iteration of Step II of a round and line 6 in one call and one pass over the
 * data.  Equal, bit for bit, to cocod_local_step(h, grads) followed by cocod_comm_end(h): the stepped model
 * x' = x - lr v never goes to memory and line 6, x^i <- x_hat_t + (x' - x_t^i), is applied to it at once, so a round
 * of k steps moves 20 (k - 1) + 24 + 4/K bytes per worker-parameter (plus the mean kernel's) instead of
 * 20 k + 12 + 4/K.  The call waits (stream-ordered, not on the host) for the mean started by cocod_comm_begin, so with
 * k = 1 nothing is left for the averaging to overlap with; with k >= 2 it still overlaps the first k - 1 steps.
 * grads: device, K x P, borrowed.  Shapes the fused kernel does not take (P not a multiple of 8, misaligned gradient
 * pointer) run the two kernels one after the other.  Errors: STATE without a begin (and, on a sharded engine, before
 * cocod_comm_exchanged). */
int cocod_local_step_end(cocod_handle *h, const float *grads);

/* ---------------------------------------------------------------------------------------------
 * The two sequential schemes the paper compares against (Section 2 and Section 4.2, time-speedup
 * equations of S-SGD and Local-SGD), as calls on the same engine and kernels, so that the cost of
 * NOT decoupling can be measured on identical code.
 *
 * Local-SGD: after k local steps every worker's model is replaced by the weighted mean of all
 * models, sequentially: x^i <- sum_j (M_j / sum M) x^j.  On the compute stream, no side stream.
 * Equals cocod_comm_begin + cocod_comm_end with no step in between.  STATE while a communication
 * is in flight. */
int cocod_local_sgd_average(cocod_handle *h);

/* S-SGD: one synchronous step: the K workers' gradients are averaged (same weights), and every
 * worker applies the same averaged gradient: g_bar = sum_j (M_j / sum M) g^j, then the local update
 * with g_bar.  grads: device, K x P, borrowed.  On the compute stream.  STATE while a communication
 * is in flight (the average-model buffer is used for g_bar; cocod_get_mean is invalid afterwards). */
int cocod_ssgd_step(cocod_handle *h, const float *grads);

/* ---------------------------------------------------------------------------------------------
 * Additions the five calls above need around them (initial point, results, schedule).      */

/* Stream for local steps, stored copies and merges (borrowed).  Not while a communication is
 * in flight (STATE). */
int cocod_set_stream(cocod_handle *h, cocod_stream_t compute);

/* Algorithm 1, Initialize (x_i^0 = x_hat_0 for every worker): broadcast P values to all K workers.  on_host selects what
 * kind of pointer x0 is.  Stream-ordered on the compute stream (host sources are copied
 * synchronously first).  Not while a communication is in flight (STATE). */
int cocod_set_params(cocod_handle *h, const float *x0, int on_host);

/* Set / get all K x P models, the momentum, and the last average model (P values).  The get
 * calls with on_host = 1 block until the data is in `out`; with on_host = 0 they are ordered on
 * the compute stream.  set_* are not legal while a communication is in flight (STATE). */
int cocod_set_params_all(cocod_handle *h, const float *x, int on_host);
int cocod_set_momentum(cocod_handle *h, const float *v, int on_host);
int cocod_get_params(cocod_handle *h, float *out, int on_host);
int cocod_get_momentum(cocod_handle *h, float *out, int on_host);
int cocod_get_mean(cocod_handle *h, float *out, int on_host);

/* Device pointer of the bf16 shadow (K x P bfloat16), valid until the option is switched off or
 * the handle is destroyed.  STATE if the option is off.  Reads must be ordered after the
 * compute stream's work. */
int cocod_get_bf16_shadow(cocod_handle *h, void **out);

/* The paper changes gamma during a run (warm-up, decay at epoch 81; Section 5.1). */
int cocod_set_lr(cocod_handle *h, float lr);

/* Mini-batch sizes M_1..M_K of Algorithm 1 (sampling in proportion to the workers' data, Section 3.2): the mean
 * uses weights M_i / sum_j M_j.  M: host, K positive finite values; NULL = all equal. */
int cocod_set_batch_sizes(cocod_handle *h, const double *M);

int cocod_set_option(cocod_handle *h, int option, int value);

/* Block the host until all of the engine's device work is done.  Returns the sticky error. */
int cocod_sync(cocod_handle *h);

/* Poll (no device-side waiting) until the mean started by comm_begin is complete or
 * timeout_ms has passed: OK, TIMEOUT, or STATE if nothing is in flight. */
int cocod_comm_wait(cocod_handle *h, int timeout_ms);

/* Number of local steps taken so far (the paper's iteration counter t). */
int64_t cocod_step_count(const cocod_handle *h);

/* The cudaError_t of the first failed CUDA call on this handle (0 if none). */
int cocod_last_cuda_error(const cocod_handle *h);

const char *cocod_strerror(int code);

/* ---------------------------------------------------------------------------------------------
 * Profiling (COCOD_OPT_PROFILE = 1): the engine brackets each of its kernels with CUDA events.
 * cocod_profile_count syncs the device and returns how many records exist (at most 16384 since
 * the last reset); cocod_profile_get returns record i: the kernel kind and its start/end in
 * milliseconds relative to the first record's start.  Used to report per-kernel bandwidth and
 * how much of the mean kernel's lifetime overlaps local steps. */
int cocod_profile_reset(cocod_handle *h);
int cocod_profile_count(cocod_handle *h);
int cocod_profile_get(cocod_handle *h, int i, int *kind, float *start_ms, float *end_ms);

/* The same record's lifetime as the kernel itself saw it: the earliest start and the latest end of its
 * thread blocks in nanoseconds of the GPU's own clock (one clock for all streams, so the lifetimes of the
 * mean kernel on the side stream and of the local steps on the compute stream can be intersected exactly:
 * the overlap Algorithm 1 asks for between Step I and Step II).  Valid after cocod_profile_count (STATE
 * before it).  Both are 0 for a record whose kernel takes no stamps (the scalar fall-back kernels, the
 * stored-copy kernel, the gather kernel). */
int cocod_profile_get_device_ns(cocod_handle *h, int i, uint64_t *start_ns, uint64_t *end_ns);

/* Number of kernels this handle has launched since creation (all kinds). */
int64_t cocod_launch_count(const cocod_handle *h);

/* ---------------------------------------------------------------------------------------------
 * Workers spread over several GPUs, one process per GPU (the paper's own layout, Section 5.1: one
 * worker per GPU, models averaged with an all-reduce).  Each process holds a contiguous block of
 * the K_global workers in an engine of its own; Step II and line 6 stay local, only Step I's
 * weighted mean x_hat_t = sum_i (M_i / sum_j M_j) x_t^i spans the GPUs.  Every process makes the
 * same sequence of calls.  Two ways to complete the mean, both queued on the side stream:
 *
 *   all-reduce   cocod_comm_begin leaves this GPU's PARTIAL sum (its workers' terms, already
 *                carrying the global weights) in the average buffer; the caller sums that buffer
 *                over the processes in place (an all-reduce of P floats queued on the side stream,
 *                e.g. NCCL), then calls cocod_comm_exchanged.
 *   gather       after cocod_ipc_attach every GPU can address every GPU's buffers.  The caller
 *                queues a barrier over the processes on the side stream (all stored copies exist),
 *                calls cocod_comm_gather -- ONE kernel that reads the K_global stored copies of this
 *                GPU's share of the columns straight from the GPUs holding them, sums them in
 *                worker order (the same order as the single-GPU mean, so the result does not depend
 *                on how the workers are spread) and stores the finished columns into every GPU's
 *                average buffer -- queues a second barrier (all columns have arrived everywhere)
 *                and calls cocod_comm_exchanged.
 *
 * cocod_comm_end is refused (STATE) until cocod_comm_exchanged has been called in that round.
 * cocod_local_sgd_average and cocod_ssgd_step are not available on a sharded engine (STATE). */

/* Declare this engine's K workers to be workers first .. first + K - 1 of K_global.  M_global:
 * host, K_global positive finite mini-batch sizes of ALL workers, or NULL for equal sizes (this
 * replaces cocod_set_batch_sizes on a sharded engine).  K_global = 0 returns the engine to the
 * unsharded behaviour.  Errors: INVALID (range outside 0..K_global, K_global > 1024, bad M),
 * STATE while a communication is in flight or peers are attached. */
int cocod_set_shard(cocod_handle *h, int K_global, int first, const double *M_global);

/* Device pointer of the average buffer (P floats, engine-owned, valid until cocod_destroy): the
 * operand of the caller's all-reduce. */
int cocod_mean_buffer(cocod_handle *h, float **out);

/* The caller has queued, on the side stream given to cocod_comm_begin, everything that completes
 * the average buffer; the engine marks that point of the side stream as "mean complete".
 * Errors: STATE unless a communication of a sharded engine is in flight and not yet marked. */
int cocod_comm_exchanged(cocod_handle *h);

/* Addresses for the gather form.  cocod_ipc_export writes COCOD_IPC_EXPORT_BYTES bytes (host)
 * describing this engine's buffers (inter-process memory handles of x, the stored copies and the
 * average buffer, plus K, first, K_global and P for cross-checking).  The caller collects the
 * blobs of all G processes in rank order (any host transport) and passes them to cocod_ipc_attach
 * together with its own rank; the engine opens the other processes' buffers (they must be on GPUs
 * with peer access to this one, or on this one) and builds its address tables.  Engines of the
 * calling process itself are addressed directly, without a handle (if they sit on other GPUs, the
 * caller has enabled peer access between the devices).  The blobs must
 * tile 0..K_global with equal P and K_global (INVALID otherwise; CUDA if a handle cannot be
 * opened).  G is at most 64.  cocod_ipc_detach closes them again (also done by cocod_destroy);
 * every process must detach before any process destroys its engine.  Requires cocod_set_shard
 * first.  Not while a communication is in flight (STATE). */
#define COCOD_IPC_EXPORT_BYTES 256
int cocod_ipc_export(cocod_handle *h, void *out);
int cocod_ipc_attach(cocod_handle *h, int G, int rank, const void *blobs);
int cocod_ipc_detach(cocod_handle *h);

/* Gather form of Step I's mean (see above): queue the gather kernel on the side stream.  STATE
 * unless peers are attached and a communication is in flight whose mean has not been started. */
int cocod_comm_gather(cocod_handle *h);

/* The gather kernel on caller-owned buffers (no handle): rows = device array of K device pointers
 * (row i = worker i's P stored values, in any allocation this GPU can address), outs = device
 * array of G device pointers to P-float average buffers; columns [col_lo, col_hi) are averaged
 * (weights w: device, K floats, or NULL for 1/K) and written to every outs[q].  vec = 1, 4 or 8 is the
 * number of columns per access: the caller vouches that every row and output pointer is aligned
 * to 4 * vec bytes, and col_lo, col_hi must be multiples of vec (INVALID otherwise; 8 is used for
 * K <= 4 only, larger K take the 4-column path). */
int cocod_kernel_mean_gather(const float *const *rows, int K, int64_t col_lo, int64_t col_hi, const float *w,
                             float *const *outs, int G, int vec, cocod_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * The four kernels on caller-owned device buffers (no handle, no state): the same code the
 * engine launches, exposed for per-kernel measurement and tests.  All pointers: device, fp32.
 *   local_step: n = number of elements; x_out may equal x_in (in place).
 *   mean:       w = K device weights, or NULL for the plain mean.
 *   merge:      x (K x P) updated in place from snap (K x P) and mean (P).              */
int cocod_kernel_local_step(const float *x_in, float *x_out, float *v, const float *g, int64_t n,
                            float lr, float mu, float wd, cocod_stream_t stream);
int cocod_kernel_snapshot(const float *x, float *snap, int64_t n, cocod_stream_t stream);
int cocod_kernel_mean(const float *snap, int K, int64_t P, const float *w, float *mean,
                      cocod_stream_t stream);
int cocod_kernel_merge(float *x, const float *snap, const float *mean, int K, int64_t P,
                       cocod_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * (No counterpart in the paper: a deployment convenience.)
 *
 * Local step with the gradients in HOST memory for callers that must not allocate device
 * memory: code running under a framework whose caching allocator already owns the whole GPU (a
 * raw cudaMalloc then fails or fights the pool), and latency-critical loops that cannot accept
 * the device-wide synchronisation an allocation may imply.  Unlike cocod_local_step_host, which
 * cudaMallocs its staging buffers on first use, this call stages the gradients through a fixed
 * array that is part of the library image, and it calls no allocation routine of any kind.
 *
 *   x_in, x_out, v : device, n fp32 each (caller-owned; x_out may equal x_in)
 *   host_grads     : host, n fp32 (pinned memory keeps the copy asynchronous)
 *   n              : at most COCOD_NOALLOC_MAX_ELEMS; larger requests are rejected with
 *                    COCOD_ERR_TOO_LARGE before anything is launched (split the vector instead)
 * Same arithmetic as cocod_kernel_local_step.  Work is queued on `stream`: one host-to-device copy
 * into the staging array, then the update kernel.
 *
 * The staging array (COCOD_NOALLOC_MAX_ELEMS * 4 bytes = 16 MiB) is held by every GPU that loads
 * the library until the process exits.  All calls on a device share it and it keeps the previous
 * call's bytes; each call overwrites the part it uses, so nothing needs clearing, but two calls
 * whose GPU work can overlap (different streams without ordering between them) race on it:
 * order them yourself.
 * The first call on each device looks up the array's device address (once per device, with that
 * device current); make that first call outside any stream capture. */
#define COCOD_NOALLOC_MAX_ELEMS (4 * 1024 * 1024)
int cocod_kernel_local_step_host_noalloc(const float *x_in, float *x_out, float *v, const float *host_grads,
                                         int64_t n, float lr, float mu, float wd, cocod_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* COCOD_H */
