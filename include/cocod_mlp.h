/*
 * cocod_mlp.h -- per-worker mini-batch stochastic gradients for the end-to-end configuration
 * (part of libcocod.so).
 *
 * Algorithm 1 of arxiv 1906.12043, Step II: every worker i forms the stochastic gradient G_tau^i of
 * its current model as the mean of the per-sample gradients over its mini-batch of M_i samples.
 * Here f is the softmax cross-entropy
 * of a 3-layer ReLU MLP (d_in -> d_hidden -> d_hidden -> d_out) and all K workers' gradients are
 * computed in one batched pass: the contractions run on the sm_100a tensor cores (tcgen05.mma,
 * bf16 operands, fp32 accumulation in TMEM, TMA-staged operands), everything else in small fused
 * CUDA-core kernels.
 *
 * Precision (what the workload fixes: bf16 weights with an fp32 master copy):
 *   parameters read by forward/backward : the bf16 shadow of the fp32 master copy (all six tensors)
 *   hidden activations h1, h2           : rounded to bf16 after ReLU
 *   dz3 = (softmax - onehot) / batch    : rounded to bf16; dz2, dz1 = bf16(dh * (h > 0))
 *   every sum / product                 : fp32 accumulation; logits, softmax and loss in fp32
 *   gradients                           : fp32, written in the flat parameter order
 *
 * Flat parameter order per worker: W1 [d_hidden][d_in], b1, W2 [d_hidden][d_hidden], b2,
 * W3 [d_out][d_hidden], b3, then zero padding up to a multiple of 64 elements (the padded count
 * is what cocod_mlp_param_count returns and what the engine must be created with: padding
 * parameters and their gradients are always 0, so they never change any result).
 *
 * Same conventions as cocod.h: int return codes (COCOD_*), device pointers on the device current
 * at create, one host thread per handle, asynchronous on the given stream.
 */
#ifndef COCOD_MLP_H
#define COCOD_MLP_H

#include <stdint.h>

#include "cocod.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cocod_mlp cocod_mlp_handle;

/* Allocate the scratch buffers (hidden activations and their gradients) for K workers.  Restrictions: batch == 128, d_in % 8 == 0, d_hidden % 128 == 0, 1 <= d_out <= 16.
 * Errors: INVALID, OOM, CUDA (also when the driver lacks the tensor-map encoder). */
int cocod_mlp_create(cocod_mlp_handle **out, int K, int batch, int d_in, int d_hidden, int d_out);
int cocod_mlp_destroy(cocod_mlp_handle *h);

/* Padded parameters per worker (multiple of 64) and the unpadded count. */
int64_t cocod_mlp_param_count(const cocod_mlp_handle *h);
int64_t cocod_mlp_param_count_unpadded(const cocod_mlp_handle *h);

/* One mini-batch gradient for every worker.
 *   params_bf16 : device, K x P bfloat16 (P = padded count): the engine's bf16 shadow
 *                 (cocod_get_bf16_shadow)
 *   x           : device, K x batch x d_in bfloat16, the workers' mini-batches
 *   labels      : device, K x batch int32 in [0, d_out)
 *   grads       : device, K x P fp32, written completely (padding = 0); feed it to cocod_local_step
 *   loss        : device, K fp32: mean cross-entropy of each worker's mini-batch
 * Asynchronous on `stream`.  A kernel-side wait that runs out of time is reported by the next
 * cocod_mlp_check as COCOD_ERR_TIMEOUT. */
int cocod_mlp_grad(cocod_mlp_handle *h, const void *params_bf16, const void *x, const int32_t *labels,
                   float *grads, float *loss, cocod_stream_t stream);

/* The same gradient pass fused with the engine's local step (Algorithm 1, Step II: gradient and
 * update of one iteration in one call).  `engine` must have been created with
 * K = the handle's K and P = cocod_mlp_param_count, with COCOD_OPT_BF16_SHADOW on (STATE otherwise):
 * the gradients are computed from its bf16 copy of x.  For the two weight matrices W1 and W2
 * (99.4 % of the parameters) one persistent, warp-specialised kernel walks over the 128 x 128 tiles of
 * W2 and then of W1: it forms a tile's weight gradient on the tensor cores (two accumulators in tensor
 * memory, so the next tile's product forms meanwhile) and applies d = g + wd x; v = mu v + d;
 * x = x - lr v to that tile at once: the gradient tile never leaves the SM, x, v and the bf16 copy are
 * read and written once.  The remaining tensors (biases, W3) take the same update inside the kernels
 * that produce their gradients, so no gradient is ever written to memory.  Results are bit-identical
 * to cocod_mlp_grad followed by cocod_local_step.  Runs on the engine's compute stream; counts as
 * one local step.
 *   x, labels, loss: as for cocod_mlp_grad. */
int cocod_mlp_grad_step(cocod_mlp_handle *h, cocod_handle *engine, const void *x, const int32_t *labels,
                        float *loss);

/* Measurement.  COCOD_MLP_OPT_PROFILE = 1: every later call of cocod_mlp_grad / cocod_mlp_grad_step that is not
 * being captured into a CUDA graph records a CUDA-event pair around the whole pass (first kernel to last) and, for
 * both calls, a second pair around the persistent kernel that forms the weight gradients of W1 and W2 (and, in
 * cocod_mlp_grad_step, updates them; it is then launched as an ordinary, not a programmatic, dependent, so that the
 * events bracket it alone).  At most 4096 calls are recorded.
 * Setting the option (to either value) synchronises the device and discards the records.
 * cocod_mlp_profile_get synchronises the device and returns the number of recorded calls and the average
 * milliseconds of the pass and of the update kernel (0 when no call recorded one).
 * COCOD_MLP_OPT_PROFILE = 2: no events and no change to how anything is launched; the update kernel alone stamps the
 * earliest start (after its wait for the predecessor) and the latest end of its thread blocks on the GPU's own clock,
 * so that its duration INSIDE the chain, with the programmatic overlap at both ends, can be read
 * (cocod_mlp_profile_get_device: number of stamped launches and their average milliseconds; also filled with
 * value 1).  The first non-zero setting allocates 64 KB on the device.
 * COCOD_MLP_OPT_CHAIN = 1 (default) / 0: how the part of a gradient pass before the weight gradients (both hidden
 * layers forward, the output layer, the hidden deltas) is launched: as ONE kernel in which the d_hidden / 128 thread
 * blocks of a worker each own 128 columns of every hidden quantity and hand their tiles to one another through
 * counters in global memory (every wait bounded; at most one block per SM per launch, all resident together, more
 * workers than fit are split over several launches), or as one kernel per layer.  Both give the same bits. */
enum { COCOD_MLP_OPT_PROFILE = 1, COCOD_MLP_OPT_CHAIN = 2 };
int cocod_mlp_set_option(cocod_mlp_handle *h, int option, int value);
int cocod_mlp_profile_get(cocod_mlp_handle *h, int *calls, float *pass_ms, float *update_ms);
int cocod_mlp_profile_get_device(cocod_mlp_handle *h, int *calls, float *update_ms);

/* Synchronise `stream` and report whether any kernel of this handle gave up a wait. */
int cocod_mlp_check(cocod_mlp_handle *h, cocod_stream_t stream);

/* Number of kernels launched by this handle so far. */
int64_t cocod_mlp_launch_count(const cocod_mlp_handle *h);

/* The tensor-core building block on its own (tests, measurement):
 *   C_w[m][n] = sum_k A_w(m, k) * B_w(n, k)   for w in [0, batch_count)
 * A, B: device bfloat16.  With a_rows_contiguous = 0, A is stored [M][K] (reduction index
 * contiguous, row stride lda); with 1 it is stored [K][M] (row index contiguous, row stride lda).
 * Likewise B: [N][K] or [K][N] with ldb.  No operand is copied or transposed.  lda, ldb and the
 * worker strides are in elements and must be multiples of 8; bases 16-byte aligned.
 * C: device fp32 [M][N], row stride ldc.  Blocks until the result is complete. */
int cocod_gemm_bf16(const void *A, const void *B, float *C, int M, int N, int K, int batch_count,
                    int a_rows_contiguous, int b_rows_contiguous, int64_t lda, int64_t ldb, int64_t ldc,
                    int64_t stride_a, int64_t stride_b, int64_t stride_c, cocod_stream_t stream);

/* Self-test of the kernels' bounded waits (failure detection without a GPU fault): launches one
 * tile whose operand copies are deliberately never issued, so the thread that issues the tensor-core
 * instructions waits on a barrier nothing will flip.  After wait_ms (1..2000) the kernel gives up,
 * records the fact, releases its tensor memory and returns; the call then returns COCOD_ERR_TIMEOUT
 * and the CUDA context stays usable.  (COCOD_OK would mean the wait did not run out.) */
int cocod_gemm_wait_selftest(int wait_ms, cocod_stream_t stream);

/* The same self-test for the persistent gradient + update kernel of cocod_mlp_grad_step: one CTA
 * with three tiles whose copies are never issued.  The thread that issues the tensor-core
 * instructions gives up after wait_ms, the other roles see that and walk through their remaining
 * tiles without touching memory (every barrier still sees all of its threads), tensor memory is
 * released, COCOD_ERR_TIMEOUT is returned and the context stays usable. */
int cocod_gemm_update_wait_selftest(int wait_ms, cocod_stream_t stream);

/* The same for the chain kernel (the part of the gradient pass before the weight gradients as one kernel whose CTAs wait
 * for one another's tiles at counters in global memory): a small model of its own is run with a switch that keeps every
 * CTA from reporting its first tile, so the wait for the worker's first hidden layer runs out after `wait_ms`
 * (1 .. 2000); every CTA gives up, lets its copies land, frees its tensor memory and returns.  Returns COCOD_ERR_TIMEOUT
 * (the expected outcome), COCOD_OK if nothing timed out, or a set-up error.  The context stays usable. */
int cocod_mlp_chain_wait_selftest(int wait_ms, cocod_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* COCOD_MLP_H */
