// Batched bf16 GEMM for sm_100a on the 5th-generation tensor cores:
//
//     D_w[m][n] = sum_k A_w(m, k) * B_w(n, k)        for every worker w (blockIdx.z)
//
// Each operand may be stored "K-major" (the reduction index k is the contiguous one: A is [M][K],
// B is [N][K]) or "MN-major" (m resp. n is contiguous: A is [K][M], B is [K][N]); the tensor cores
// read both forms from shared memory, so no operand is ever transposed in memory.  One CTA
// computes one 128 x 128 tile of one worker:
//   * operands are staged by TMA (cp.async.bulk.tensor, 128-byte swizzle; every CTA fetches its own tiles) into a
//     shared-memory ring of up to 6 stages (32 KB each) guarded by mbarriers;
//   * one elected thread issues tcgen05.mma (kind::f16, bf16 inputs, fp32 accumulation) on
//     shared-memory descriptors; the 128 x 128 fp32 accumulator lives in TMEM (128 columns);
//   * all four warps read the accumulator back with tcgen05.ld (32 lanes x 32 columns at a time)
//     and run a fused epilogue: bias + ReLU or ReLU-mask (optionally with the column sums of the
//     tile, written out or applied to a bias vector as its local step) leaving as bf16 through
//     staged TMA bulk stores, or an fp32 store that goes through swizzled shared memory and TMA
//     bulk stores (full 128-byte lines).  (The weight-gradient GEMM that applies the momentum
//     update to its own tile is a kernel of its own: cocod_gemm_update_sm100.cuh.)
// Out-of-range rows / reduction columns are zero-filled by TMA, so M, N, K need not be
// multiples of the tile; stores are predicated.
//
// Every wait is bounded in time: if a barrier does not flip within about two seconds the kernel
// records a code in *error_flag, drains its own copies, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cocod_kernels.cuh"

namespace cocod {
namespace gemm {

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 6, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TMEM_COLS = 128;
constexpr int NEXT_N = 16;             // width of the optional second contraction (the output layer's classes, padded)
constexpr int MAX_STAGES = STAGES;
// ring (at least two stages: the fp32 epilogue stages a whole 128 x 128 tile = 64 KB there) + alignment
// slack + a tail holding the barriers (256 B), the bias tile (512 B)
__host__ __device__ constexpr int ring_stages(int stages) { return stages < 2 ? 2 : stages; }
// ... and, behind them, room for a slice of the output layer's weights (16 classes x 128 columns fp32, 8 KB)
constexpr int TAIL_BYTES = 1024 + 16 * BN * 4;
__host__ __device__ constexpr int smem_bytes(int stages) { return ring_stages(stages) * STAGE_BYTES + 1024 + TAIL_BYTES; }
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

enum Epilogue {
    EPI_F32 = 0,        // c[m][n] = acc                         (fp32, row stride ldc; TMA store if map_c_ok)
    EPI_BIAS_RELU = 1,  // o[m][n] = bf16(max(acc + bias[n], 0))          (o = the bf16 matrix map_c describes: boxes of
    EPI_MASK = 2        // o[m][n] = bf16(acc * (mask[m][n] > 0));         64 columns x 128 rows, 128-byte swizzle)
                        // optionally colsum[n] = sum_m o[m][n] (M <= 128)
};

// Where a kernel that has just produced a gradient element applies the local step itself (fused gradient +
// update call): pointers to the worker-major K x P state, already offset to the tensor's first element.
// x_in == nullptr: no update, the gradient is written out instead.
struct StepTarget {
    const float *x_in;
    float *x_out;
    float *v;
    __nv_bfloat16 *shadow;             // may be nullptr
    long long worker_stride;           // P
    float lr, mu, wd;
};
// d = fma(wd, x, g); v = fma(mu, v, d); x = fma(-lr, v, x); shadow = bf16(x)   (the engine's arithmetic)
__device__ __forceinline__ void step_element(const StepTarget &t, long long idx, float g)
{
    const float x = t.x_in[idx];
    const float d = __fmaf_rn(t.wd, x, g);
    const float vn = __fmaf_rn(t.mu, t.v[idx], d);
    t.v[idx] = vn;
    const float xn = __fmaf_rn(-t.lr, vn, x);
    t.x_out[idx] = xn;
    if (t.shadow != nullptr) t.shadow[idx] = __float2bfloat16_rn(xn);
}

// The same for up to N elements at once: all loads first, so that their round trips overlap.
template <int N>
__device__ __forceinline__ void step_elements(const StepTarget &t, const long long (&idx)[N], const float (&g)[N], int n)
{
    float x[N], v[N];
#pragma unroll
    for (int i = 0; i < N; ++i)
        if (i < n) {
            x[i] = t.x_in[idx[i]];
            v[i] = t.v[idx[i]];
        }
#pragma unroll
    for (int i = 0; i < N; ++i)
        if (i < n) {
            const float d = __fmaf_rn(t.wd, x[i], g[i]);
            const float vn = __fmaf_rn(t.mu, v[i], d);
            t.v[idx[i]] = vn;
            const float xn = __fmaf_rn(-t.lr, vn, x[i]);
            t.x_out[idx[i]] = xn;
            if (t.shadow != nullptr) t.shadow[idx[i]] = __float2bfloat16_rn(xn);
        }
}

struct Params {
    int M, N, K;                       // per-worker problem
    float *c;                          // EPI_F32
    long long c_worker_stride;         // elements
    int ldc;
    int map_c_ok;                      // EPI_F32: map_c describes c, use TMA stores
    const __nv_bfloat16 *bias;         // [N]
    long long bias_worker_stride;
    const __nv_bfloat16 *mask;         // [M][N], row stride N
    long long mask_worker_stride;
    float *colsum;                     // EPI_MASK, optional: [N] column sums of the bf16 output (needs M <= 128)
    long long colsum_worker_stride;
    StepTarget colsum_step;            // ... or (x_in != nullptr) the local step of that [N] tensor, the sums as gradient
    // EPI_BIAS_RELU, optional (logit_part != nullptr; needs M <= 128 and 128 threads): this tile's contribution to the
    // next (narrow) layer, part[w][tile_n][m][c] = sum_{n in tile} o[m][n] * w_next[c][n] for c < next_out <= 16, taken
    // from the bf16 values o the tile stores; rows of 16 floats.  Summed over tile_n by whoever reads it.  It is a second,
    // small contraction on the tensor cores: A = the staged output tile (it sits in shared memory in exactly the
    // operand layout), B = the 16 x 128 slice of w_next fetched through map_n, accumulator = 16 more TMEM columns.
    float *logit_part;
    const __nv_bfloat16 *b_next;       // [next_out] per worker: added by the CTAs of tile_n == 0
    long long b_next_worker_stride;
    int next_out;
    int stages;                        // shared-memory ring depth, 1 .. MAX_STAGES
    int *error_flag;
    unsigned long long wait_ns;        // time limit of every barrier wait (0 = WAIT_LIMIT_NS)
    int debug_no_loads;                // self-test: the producer issues nothing, so the waits run out
    int b_keep;                        // 1: operand B (weights the next kernels of the chain read again) is fetched with the
                                       //    L2 evict-last priority
#ifdef COCOD_GEMM_TRACE
    unsigned long long *trace;         // tuning builds only: 8 timestamps per CTA
#endif
};
#ifdef COCOD_GEMM_TRACE
#define COCOD_TRACE(i) do { if (p.trace && (threadIdx.x & 31) == 0) p.trace[((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 8 + (i)] = now_ns(); } while (0)
#else
#define COCOD_TRACE(i) do { } while (0)
#endif

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long now_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Wait for a barrier phase, giving up after WAIT_LIMIT_NS or when another role has aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort,
                                          unsigned long long limit_ns)
{
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = now_ns();
    for (unsigned it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort) return false;
            if (now_ns() - t0 > limit_ns) return false;
        }
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
// L2 eviction priorities for bulk copies: data that is read or written once and not needed again soon leaves first,
// data the next kernels of the chain come back to (the bf16 copy of the weights) leaves last.
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z,
                                            uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
                 "[%0], [%1, {%3, %4, %5}], [%2], %6;"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int x, int y, int z, uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], [%1], %5;"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void tma_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute may
// become resident while its predecessor in the stream still runs; it must not touch anything the
// predecessor (or, transitively, anything before it) writes until pdl_wait() has returned, which
// happens once the predecessor grid has completed and its writes are visible.
// pdl_launch_dependents() lets the successor's CTAs be scheduled as soon as every CTA of this grid has
// called it (or exited): call it only after this CTA holds all the resources it will ever take
// (shared memory, TMEM), so that a waiting successor can never hold something a CTA of this grid
// still needs.  Both are no-ops for kernels launched without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on an mbarrier once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (version 1 = sm_100, 128-byte swizzle), for tiles laid out by TMA:
//  * K-major tile: rows (m or n) of 128 bytes = 64 bf16 along k; 8-row groups are 1024 bytes apart
//    (stride byte offset); the leading byte offset is unused.  One MMA (k = 16) advances 32 bytes.
//  * MN-major tile: rows are k, each 128 bytes = 64 bf16 along m (or n); 8-row groups (8 values of
//    k) are 1024 bytes apart (stride byte offset), and the second block of 64 m/n values lives one
//    whole 64-row block later (leading byte offset = 64 * 128 bytes).  One MMA (k = 16) advances two
//    8-row groups = 2048 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, bool mn_major)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);                              // start address, 16-byte units
    d |= (uint64_t)(mn_major ? (BK * 128) >> 4 : 1) << 16;               // leading byte offset
    d |= (uint64_t)(1024 >> 4) << 32;                                     // stride byte offset = 1024 B
    d |= (uint64_t)1 << 46;                                               // descriptor version
    d |= (uint64_t)2 << 61;                                               // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, M = 128, N = 128, operand majors as given.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn, int n = BN)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// ------------------------------------------------------------------------------------------ kernel
// Tensor maps: a K-major operand is {k (contiguous), rows, workers} with box {64, 128, 1}; an
// MN-major operand is {m or n (contiguous), k, workers} with box {64, 64, 1} (two boxes per tile).
// map_c (EPI_F32 only): {n (contiguous), m, workers} fp32 with box {32, 128, 1}, 128-byte swizzle.
// map_n (EPI_BIAS_RELU with logit_part): the next layer's weights {n (contiguous), classes, workers} bf16, box {64, 16, 1}
// (classes beyond the matrix are zero-filled).
// NT threads per CTA: 128 (every thread drains one accumulator row; 256 would let two threads share a row).
template <int EPI, bool A_MN, bool B_MN, int NT>
__global__ void __launch_bounds__(NT)
gemm_bf16(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
          const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_n, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    if (threadIdx.x == 0) COCOD_TRACE(0);
    const int stages = p.stages;
    uint8_t *tail = smem + ring_stages(stages) * STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + MAX_STAGES), accum = smem_u32(bars + 2 * MAX_STAGES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 5);
    volatile int *abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *never = abort + 1;          // stays 0: used by waits that must not be cut short
    float *sbias = reinterpret_cast<float *>(tail + 256);
    uint8_t *swn = tail + 1024;                  // the next layer's weight slice: two k-blocks of 16 rows x 128 bytes
    const uint32_t wn_full = smem_u32(bars + 2 * MAX_STAGES + 1), wn_done = smem_u32(bars + 2 * MAX_STAGES + 2);
    const bool with_next = (EPI == EPI_BIAS_RELU) && (NT == 128) && (p.logit_part != nullptr);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM, wk = blockIdx.z;
    const int nkb = (p.K + BK - 1) / BK;
    const uint32_t smem_base = smem_u32(smem);
    const unsigned long long limit = p.wait_ns ? p.wait_ns : WAIT_LIMIT_NS;

    // One k-block's operand tiles into stage s (producer thread only).
    auto issue_loads = [&](int kb, int s) {
        const uint32_t bar = full0 + 8 * s;
        mbar_expect_tx(bar, STAGE_BYTES);
        const uint32_t dst_a = smem_base + s * STAGE_BYTES, dst_b = dst_a + A_BYTES;
        if (A_MN) {
            tma_load_3d(dst_a, &map_a, bar, m0, kb * BK, wk);
            tma_load_3d(dst_a + BK * 128, &map_a, bar, m0 + 64, kb * BK, wk);
        } else {
            tma_load_3d(dst_a, &map_a, bar, kb * BK, m0, wk);
        }
        if (p.b_keep) {
            const uint64_t pl = l2_policy_evict_last();
            if (B_MN) {
                tma_load_3d(dst_b, &map_b, bar, n0, kb * BK, wk, pl);
                tma_load_3d(dst_b + BK * 128, &map_b, bar, n0 + 64, kb * BK, wk, pl);
            } else {
                tma_load_3d(dst_b, &map_b, bar, kb * BK, n0, wk, pl);
            }
        } else if (B_MN) {
            tma_load_3d(dst_b, &map_b, bar, n0, kb * BK, wk);
            tma_load_3d(dst_b + BK * 128, &map_b, bar, n0 + 64, kb * BK, wk);
        } else {
            tma_load_3d(dst_b, &map_b, bar, kb * BK, n0, wk);
        }
    };

    int armed = 0;
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        if (EPI == EPI_BIAS_RELU || EPI == EPI_MASK || (EPI == EPI_F32 && p.map_c_ok))
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        mbar_init(wn_full, 1);
        mbar_init(wn_done, 1);
        abort[0] = 0;
        abort[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
        pdl_wait();                   // everything above overlapped the previous kernel's tail
        // the first ring of copies starts now, under the rest of the set-up
        if (!p.debug_no_loads)
            for (; armed < nkb && armed < stages; ++armed) issue_loads(armed, armed);
        if (with_next && !p.debug_no_loads) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_n) : "memory");
            mbar_expect_tx(wn_full, 2 * NEXT_N * 128);
            tma_load_3d(smem_u32(swn), &map_n, wn_full, n0, 0, wk);
            tma_load_3d(smem_u32(swn) + NEXT_N * 128, &map_n, wn_full, n0 + 64, 0, wk);
        }
    }
    if (threadIdx.x == 0) COCOD_TRACE(6);
    __syncwarp();
    const uint32_t tmem_cols = with_next ? 2 * TMEM_COLS : TMEM_COLS;      // (a power of two)
    if (warp == 0) {                  // warp-collective TMEM allocation
        tmem_alloc(smem_u32(tmem_slot), tmem_cols);
        tmem_relinquish();
    }
    if (threadIdx.x == 0) COCOD_TRACE(7);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) COCOD_TRACE(1);
    pdl_launch_dependents();          // this CTA holds its shared memory and TMEM: the next kernel may set up
    pdl_wait();                       // (thread 0 has passed it already) before any thread reads global memory

    int failed = 0;
    constexpr int NCH = (NT == 256) ? 2 : 4;       // 32-column chunks drained by one thread
    const int row = (warp & 3) * 32 + lane;        // accumulator row = TMEM lane (a warp reaches lanes 32 (w % 4) ..)
    const int cbase = (warp >> 2) * NCH;           // first chunk of this thread
    const int m = m0 + row;
    uint4 maskv[NCH * 4];             // EPI_MASK: this thread's mask values, fetched while the MMAs run
    if (warp == 0 && lane == 0) {
        // ---- producer: the remaining k-blocks, each as soon as its stage is free again
        for (int kb = armed; kb < nkb && !p.debug_no_loads; ++kb) {
            const int s = kb % stages;
            if (!mbar_wait(empty0 + 8 * s, ((kb / stages) - 1) & 1, abort, limit)) { failed = 1; break; }
            issue_loads(kb, s);
            armed = kb + 1;
        }
        if (failed) {                 // let copies that were already issued land before leaving
            abort[0] = 1;
            for (int kb = (armed > stages ? armed - stages : 0); kb < armed; ++kb)
                mbar_wait(full0 + 8 * (kb % stages), (kb / stages) & 1, never, limit);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        constexpr uint32_t idesc = instr_desc(A_MN, B_MN);
        constexpr uint32_t a_step = A_MN ? 2048u : (uint32_t)(UMMA_K * 2), b_step = B_MN ? 2048u : (uint32_t)(UMMA_K * 2);
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % stages;
            if (!mbar_wait(full0 + 8 * s, (kb / stages) & 1, abort, limit)) { failed = 2; break; }
            if (kb == 0) COCOD_TRACE(2);
            if (kb == nkb - 1) COCOD_TRACE(3);
            tc_fence_after();
            const uint32_t a_addr = smem_base + s * STAGE_BYTES, b_addr = a_addr + A_BYTES;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
                const uint64_t ad = smem_desc(a_addr + k * a_step, A_MN);
                const uint64_t bd = smem_desc(b_addr + k * b_step, B_MN);
                umma_bf16(tmem_base, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(empty0 + 8 * s);      // frees the stage once these MMAs have read it
        }
        if (!failed) umma_commit(accum);      // accumulator complete
        else abort[0] = 1;
    } else if (warp >= 2) {
        // ---- idle warps fetch what the epilogue needs besides the accumulator
        if (EPI == EPI_BIAS_RELU) {
            const __nv_bfloat16 *bias = p.bias + (long long)wk * p.bias_worker_stride;
            for (int i = threadIdx.x - 64; i < BN; i += NT - 64) sbias[i] = (n0 + i < p.N) ? __bfloat162float(bias[n0 + i]) : 0.0f;
        }
    }
    auto load_mask = [&]() {
        const int nm = n0 + cbase * 32;
        const __nv_bfloat16 *mrow = p.mask + (long long)wk * p.mask_worker_stride + (long long)m * p.N + nm;
        const bool vec = (m < p.M) && (nm + NCH * 32 <= p.N) && ((reinterpret_cast<uintptr_t>(mrow) & 15u) == 0);
#pragma unroll
        for (int q = 0; q < NCH * 4; ++q) {
            if (vec) {
                maskv[q] = *reinterpret_cast<const uint4 *>(mrow + q * 8);
            } else {
                __align__(16) __nv_bfloat16 t[8];
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    t[e] = (m < p.M && nm + q * 8 + e < p.N) ? mrow[q * 8 + e] : __float2bfloat16_rn(0.0f);
                maskv[q] = *reinterpret_cast<const uint4 *>(t);
            }
        }
    };
    // Only the two warps without a role prefetch under the main loop: in the warps of the producer and of
    // the MMA issuer the other 31 lanes' loads interleave with the elected lane's loop and slowed the main
    // loop by 40 % (8.2 vs 5.8 us for 16 reduction blocks); those two warps fetch their rows afterwards.
    if (EPI == EPI_MASK && warp >= 2) load_mask();
    __syncwarp();

    if (EPI == EPI_MASK && warp < 2) load_mask();
    // ---- epilogue: every thread owns one accumulator row (TMEM lane) of the tile
    bool ok = mbar_wait(accum, 0, abort, limit + limit / 2);

    ok = __all_sync(0xffffffffu, ok);
    if (__syncthreads_and(ok ? 1 : 0)) {          // (also makes sbias visible)
        if (threadIdx.x == 0) COCOD_TRACE(4);
        tc_fence_after();
        const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + cbase * 32;
        uint32_t r[NCH][32];                       // this thread's part of the accumulator row
#pragma unroll
        for (int cc = 0; cc < NCH; ++cc) tmem_ld32(trow + cc * 32, r[cc]);
        tmem_ld_wait();
        if (EPI == EPI_F32) {
            if (p.map_c_ok) {
                // stage the fp32 tile in the (now idle) ring as 128 x 32 sub-tiles with the 128-byte swizzle
                // (16-byte piece j of row r sits at piece j ^ (r & 7)); each sub-tile is handed to the store
                // engine as soon as the 128 threads sharing it have written it
                const int group = warp >> 2;
                const bool leader = (threadIdx.x & 127) == 0;
#pragma unroll
                for (int cc = 0; cc < NCH; ++cc) {
                    const int c = cbase + cc;
                    uint8_t *tile = smem + c * (BM * 128);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4 *>(tile + row * 128 + ((j ^ (row & 7)) << 4)) =
                            make_uint4(r[cc][4 * j], r[cc][4 * j + 1], r[cc][4 * j + 2], r[cc][4 * j + 3]);
                    fence_async_smem();
                    asm volatile("bar.sync %0, 128;" ::"r"(group + 1) : "memory");
                    if (leader && n0 + c * 32 < p.N) {
                        tma_store_3d(&map_c, smem_base + c * (BM * 128), n0 + c * 32, m0, wk);
                        tma_store_commit();
                    }
                }
                if (leader) tma_store_wait_read<0>();      // shared memory must outlive the reads
            } else if (m < p.M) {
                float *dst = p.c + (long long)wk * p.c_worker_stride + (long long)m * p.ldc + n0;
#pragma unroll
                for (int cc = 0; cc < NCH; ++cc)
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + (cbase + cc) * 32 + j < p.N) dst[(cbase + cc) * 32 + j] = __uint_as_float(r[cc][j]);
            }
        } else {
#pragma unroll
            for (int cc = 0; cc < NCH; ++cc) {
                const int c = cbase + cc;
                __align__(16) __nv_bfloat16 outv[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float a = __uint_as_float(r[cc][j]);
                    if (EPI == EPI_BIAS_RELU) {
                        a = fmaxf(a + sbias[c * 32 + j], 0.0f);
                    } else {
                        const __nv_bfloat16 *mk = reinterpret_cast<const __nv_bfloat16 *>(&maskv[cc * 4 + (j >> 3)]);
                        a = (__bfloat162float(mk[j & 7]) > 0.0f) ? a : 0.0f;
                    }
                    outv[j] = __float2bfloat16_rn(a);
                }
                // stage the bf16 row in the (now idle) ring in the TMA swizzle: 64-column boxes of 128-byte rows,
                // 16-byte piece j of row r at piece j ^ (r & 7)
                {
                    const uint4 *src = reinterpret_cast<const uint4 *>(outv);
                    uint8_t *box = smem + (c >> 1) * (BM * 128) + row * 128;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4 *>(box + ((((c & 1) * 4 + j) ^ (row & 7)) << 4)) = src[j];
                }
            }
            // the tile leaves through two bulk stores (whole 128-byte lines; rows and columns beyond the
            // matrix are clipped by the tensor map)
            fence_async_smem();
            __syncthreads();
            if (threadIdx.x == 0) {
#pragma unroll
                for (int b = 0; b < BN / 64; ++b)
                    if (n0 + b * 64 < p.N) tma_store_3d(&map_c, smem_base + b * (BM * 128), n0 + b * 64, m0, wk);
                tma_store_commit();
            }
            if (with_next) {
                // the staged tile (two 64-column boxes in the 128-byte swizzle) is the A operand as it stands
                if (threadIdx.x == 0) {
                    if (mbar_wait(wn_full, 0, abort, limit)) {
                        tc_fence_after();
                        constexpr uint32_t idesc_n = instr_desc(false, false, NEXT_N);
#pragma unroll
                        for (int b = 0; b < BN / 64; ++b)
#pragma unroll
                            for (int k = 0; k < BK / UMMA_K; ++k)
                                umma_bf16(tmem_base + TMEM_COLS, smem_desc(smem_base + b * (BM * 128) + k * (UMMA_K * 2), false),
                                          smem_desc(smem_u32(swn) + b * (NEXT_N * 128) + k * (UMMA_K * 2), false), idesc_n,
                                          (b > 0 || k > 0) ? 1u : 0u);
                        umma_commit(wn_done);
                    } else {
                        abort[0] = 1;
                        if (p.error_flag != nullptr) atomicExch(p.error_flag, 5);
                    }
                }
                __syncwarp();
                if (mbar_wait(wn_done, 0, abort, limit)) {
                    tc_fence_after();
                    uint32_t q[NEXT_N];
                    tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + TMEM_COLS, q);
                    tmem_ld_wait();
                    if (m < p.M) {
                        float o[NEXT_N];
#pragma unroll
                        for (int c = 0; c < NEXT_N; ++c) o[c] = __uint_as_float(q[c]);
                        if (blockIdx.x == 0) {   // the next layer's bias enters here, in the kernel BEFORE the one that may update it
                            const __nv_bfloat16 *bn = p.b_next + (long long)wk * p.b_next_worker_stride;
#pragma unroll
                            for (int c = 0; c < NEXT_N; ++c) if (c < p.next_out) o[c] += __bfloat162float(bn[c]);
                        }
                        float4 *dst = reinterpret_cast<float4 *>(p.logit_part + (((long long)wk * gridDim.x + blockIdx.x) * BM + row) * NEXT_N);
#pragma unroll
                        for (int c = 0; c < NEXT_N / 4; ++c) dst[c] = make_float4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                    }
                } else if (p.error_flag != nullptr) {
                    atomicExch(p.error_flag, 6);
                }
            }
            if (EPI == EPI_MASK && (p.colsum != nullptr || p.colsum_step.x_in != nullptr)) {
                // the whole batch is in this tile: thread t adds column t of the staged tile over the rows, in row order
                const int t = threadIdx.x;
                if (t < BN && n0 + t < p.N) {
                    const int rows = (p.M - m0 < BM) ? (p.M - m0) : BM;
                    const uint8_t *colp = smem + (t >> 6) * (BM * 128) + (t & 7) * 2;
                    const int piece = (t & 63) >> 3;
                    float acc = 0.0f;
                    for (int rr = 0; rr < rows; ++rr)
                        acc += __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(colp + rr * 128 + ((piece ^ (rr & 7)) << 4)));
                    if (p.colsum_step.x_in != nullptr) step_element(p.colsum_step, (long long)wk * p.colsum_step.worker_stride + n0 + t, acc);
                    else p.colsum[(long long)wk * p.colsum_worker_stride + n0 + t] = acc;
                }
            }
            if (threadIdx.x == 0) tma_store_wait_read<0>();      // shared memory must outlive the reads
        }
    } else if (threadIdx.x == 0 && p.error_flag != nullptr) {
        atomicExch(p.error_flag, 1);
    }
    if (failed && p.error_flag != nullptr) atomicExch(p.error_flag, 1 + failed);

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) COCOD_TRACE(5);
    if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
}

}  // namespace gemm
}  // namespace cocod
