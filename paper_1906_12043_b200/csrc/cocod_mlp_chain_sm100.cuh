// The gradient chain of the 3-layer ReLU MLP up to the hidden-layer deltas, as ONE kernel (Algorithm 1, Step II: the
// per-worker mini-batch gradient):
//
//     h1 = relu(x W1^T + b1) -> h2 = relu(h1 W2^T + b2) -> logits, softmax, loss, dz3 -> dz2 = (dz3 W3) * (h2 > 0),
//     dW3, db3, db2 -> dz1 = (dz2 W2) * (h1 > 0), db1
//
// The d_h / 128 CTAs (blockIdx.x) of a worker (blockIdx.z) each own columns 128 r .. 128 r + 127 of every hidden quantity:
// one 128 x 128 tile per layer, the batch of 128 being the tile's height.  A layer's reduction runs over ALL columns of
// the layer before it, which the worker's other CTAs have just stored (to global memory, i.e. L2, through bulk stores):
// between two layers the worker's CTAs meet at a counter in global memory (one atomic add per CTA when its tile is
// complete; whoever needs the others' tiles waits, with a time limit, until the counter has reached their number).  ALL
// CTAs OF THE GRID MUST BE RESIDENT AT THE SAME TIME: the host launches at most one CTA per SM (a cooperative launch) and
// splits the workers over several launches otherwise.  (Thread-block clusters with their hardware barrier would lift
// that condition, but a cluster of 8 fits only 15 times on this 148-SM part: the sixteenth worker would run alone in a
// second wave.)  Against one kernel per layer this removes three launches with their set-up, tail and launch latency,
// and lets every layer's weights (which depend on nothing in the chain) arrive under the previous layer's epilogue: the
// producer refills the operand ring with the NEXT layer's weight blocks as stages come free and adds the activation
// blocks once the counter says they are stored.
//
// Roles in a CTA of 320 threads: warps 0..7 are the workers (epilogues, output layer), warp 8 (one lane) issues the TMA
// loads, warp 9 (one lane) issues tcgen05.mma.  Shared memory: a 5-stage operand ring (32 KB per stage), one 128 x 128
// bf16 tile buffer in the TMA / UMMA swizzle (h1, then h2, then dz2 in place of h2, then dz1), dz3, biases, the output
// layer's partial sums, barriers.
// TMEM: two 128-column accumulators and 16 columns for the partial logits.
//
// The arithmetic, operation for operation, is that of the per-layer kernels (gemm_bf16 epilogues and head_backward), so
// both routes give the same bits.  Every wait is bounded; a role that gives up sets the CTA's abort flag and the error
// flag in global memory, which every waiting CTA polls.
#pragma once
#include "cocod_gemm_sm100.cuh"

namespace cocod {
namespace gemm {

constexpr int CH_THREADS = 320;
constexpr int CH_STAGES = 5;
constexpr int CH_OFF_TILE = CH_STAGES * STAGE_BYTES;
constexpr int CH_OFF_WN = CH_OFF_TILE + BM * BN * 2;
constexpr int CH_OFF_DZ = CH_OFF_WN + 2 * NEXT_N * 128;
constexpr int CH_OFF_BIAS = CH_OFF_DZ + BM * NEXT_N * 4;
constexpr int CH_OFF_ROWLOSS = CH_OFF_BIAS + 2 * BN * 4;
constexpr int CH_OFF_RED = CH_OFF_ROWLOSS + BM * 4;             // partial sums of the output layer: [2][16][128] + [2][128] floats
constexpr int CH_OFF_BARS = CH_OFF_RED + (2 * 16 + 2) * BN * 4;
constexpr int CH_SMEM = CH_OFF_BARS + 256 + 1024;  // + alignment slack
static_assert(CH_SMEM <= 227 * 1024, "shared memory of the chain kernel");

struct ChainParams {
    int d_in, d_h, d_out;
    long long P, P_raw, oW3, ob1, ob2, ob3;
    const __nv_bfloat16 *params;       // bf16 copy of the K x P state
    const int32_t *labels;             // [K][128]
    float *loss;                       // [K]
    float *grads;                      // K x P fp32 (used when step.x_in == nullptr): dW3, db1, db2, db3, padding
    StepTarget step;                   // x_in != nullptr: those tensors take their local step here instead
    float *logit_part;                 // scratch [K][tiles][128][16]: every tile's partial logits
    int *sync;                         // [K][4] counters, all zero between launches (the last CTA of a worker clears them)
    int w0;                            // first worker of this launch (blockIdx.z counts from it)
    int *error_flag;
    unsigned long long wait_ns;        // time limit of every wait (0 = WAIT_LIMIT_NS)
    int debug_no_arrive;               // self-test: no CTA reports its first tile, so the wait for the worker's h1 runs out
};

#ifdef COCOD_CHAIN_TRACE
__device__ unsigned long long g_chain_trace[1024 * 16];
#define CH_TRACE(i) do { if (threadIdx.x == 0) g_chain_trace[(blockIdx.z * gridDim.x + blockIdx.x) * 16 + (i)] = now_ns(); } while (0)
#else
#define CH_TRACE(i) do { } while (0)
#endif

// One arrival at a counter in global memory: everything this thread has written (or has seen complete) before is
// visible to whoever reads the counter with ld.acquire afterwards.
__device__ __forceinline__ void count_arrive(int *counter)
{
    __threadfence();
    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(counter) : "memory");
}
// Wait until the counter has reached `target`; gives up after limit_ns, or when this CTA or any CTA of the grid has
// recorded a failure.
__device__ __forceinline__ bool count_wait(const int *counter, int target, volatile int *abort, const int *error_flag,
                                           unsigned long long limit_ns)
{
    const unsigned long long t0 = now_ns();
    for (unsigned it = 0;; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (v >= target) return true;
        if ((it & 31u) == 31u) {
            if (*abort) return false;
            if (error_flag != nullptr && *reinterpret_cast<const volatile int *>(error_flag) != 0) return false;
            if (now_ns() - t0 > limit_ns) return false;
        }
    }
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// grid = (d_h / 128, 1, workers of this launch) with at most one CTA per SM, all resident together; block = CH_THREADS;
// dynamic shared memory = CH_SMEM.
// Maps: k_x {d_in, 128, K}, k_w1 {d_in, d_h, K}, k_h1 {d_h, 128, K}, k_w2 {d_h, d_h, K} (boxes 64 x 128: reduction index
// contiguous); k_w3 {d_h, d_out, K} (box 64 x 16); k_dz2 like k_h1; mn_w2 {d_h, d_h, K} (box 64 x 64: W2 read with its
// column index contiguous); st_dz1 {d_h, 128, K} (box 64 x 128).
template <int DOUT>
__global__ void __launch_bounds__(CH_THREADS, 1)
mlp_chain(const __grid_constant__ CUtensorMap k_x, const __grid_constant__ CUtensorMap k_w1,
          const __grid_constant__ CUtensorMap k_h1, const __grid_constant__ CUtensorMap k_w2,
          const __grid_constant__ CUtensorMap k_w3, const __grid_constant__ CUtensorMap k_dz2,
          const __grid_constant__ CUtensorMap mn_w2, const __grid_constant__ CUtensorMap st_dz1, const ChainParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    CH_TRACE(0);
    uint8_t *T = smem + CH_OFF_TILE;
    uint8_t *swn = smem + CH_OFF_WN;
    float *sdz = reinterpret_cast<float *>(smem + CH_OFF_DZ);
    float *sbias = reinterpret_cast<float *>(smem + CH_OFF_BIAS);          // [0..127] b1, [128..255] b2 of this tile
    float *srowloss = reinterpret_cast<float *>(smem + CH_OFF_ROWLOSS);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + CH_OFF_BARS);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + CH_STAGES), accum0 = smem_u32(bars + 2 * CH_STAGES);
    const uint32_t wn_full = smem_u32(bars + 2 * CH_STAGES + 3), wn_done = smem_u32(bars + 2 * CH_STAGES + 4);
    const uint32_t staged = smem_u32(bars + 2 * CH_STAGES + 5);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * CH_STAGES + 6);
    volatile int *abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *never = abort + 1;
    float *red = reinterpret_cast<float *>(smem + CH_OFF_RED);             // [2][16][128]
    float *redsum = red + 2 * 16 * BN;                                      // [2][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = blockIdx.x, tiles = gridDim.x, w = p.w0 + blockIdx.z;
    const int n0 = rank * BN;
    const int nkb1 = (p.d_in + BK - 1) / BK, nkb2 = p.d_h / BK;
    const uint32_t smem_base = smem_u32(smem), T_addr = smem_u32(T);
    const unsigned long long limit = p.wait_ns ? p.wait_ns : WAIT_LIMIT_NS;
    int *cnt = p.sync + 4 * w;         // [0] h1 stored, [1] partial logits written, [2] dz2 stored, [3] CTAs that are through
    constexpr uint32_t TMEM_ALLOC = 512;

    if (threadIdx.x == 0) {
        for (int s = 0; s < CH_STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int i = 0; i < 3; ++i) mbar_init(accum0 + 8 * i, 1);
        mbar_init(wn_full, 1);
        mbar_init(wn_done, 1);
        mbar_init(staged, 256);
        abort[0] = 0;
        abort[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 8 && lane == 0) {
        const CUtensorMap *maps[8] = {&k_x, &k_w1, &k_h1, &k_w2, &k_w3, &k_dz2, &mn_w2, &st_dz1};
        for (int i = 0; i < 8; ++i) asm volatile("prefetch.tensormap [%0];" ::"l"(maps[i]) : "memory");
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_ALLOC);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();
    CH_TRACE(1);

    int failed = 0;
    // global number g of an operand block -> its ring stage and the parity of its use
    auto stage_of = [](int g) { return g % CH_STAGES; };
    auto wait_free = [&](int g) -> bool {          // producer: the stage of block g has been read by the MMAs of block g - STAGES
        const int use = g / CH_STAGES;
        return use == 0 || mbar_wait(empty0 + 8 * stage_of(g), (use - 1) & 1, abort, limit);
    };

    if (warp == 8) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int g = 0, issued = 0;
            const uint64_t keep = l2_policy_evict_last();       // the weights come back in the backward pass and next step
            // the output layer's weight slice of this tile (two boxes of 64 columns x 16 classes)
            mbar_expect_tx(wn_full, 2 * NEXT_N * 128);
            tma_load_3d(smem_u32(swn), &k_w3, wn_full, n0, 0, w);
            tma_load_3d(smem_u32(swn) + NEXT_N * 128, &k_w3, wn_full, n0 + 64, 0, w);
            // layer 1: x (all CTAs of the worker read the same rows) and this tile's rows of W1
            for (int kb = 0; kb < nkb1 && !failed; ++kb, ++g) {
                if (!wait_free(g)) { failed = 1; break; }
                const uint32_t bar = full0 + 8 * stage_of(g), dst = smem_base + stage_of(g) * STAGE_BYTES;
                mbar_expect_tx(bar, STAGE_BYTES);
                tma_load_3d(dst, &k_x, bar, kb * BK, 0, w);
                tma_load_3d(dst + A_BYTES, &k_w1, bar, kb * BK, n0, w, keep);
                issued = g + 1;
            }
            // One later layer: its first weight blocks as stages come free, then (once the worker's CTAs have stored the
            // activations: counter `which`) the activation blocks of those stages, then the rest block by block.
            auto layer = [&](const CUtensorMap *act, const CUtensorMap *wgt, bool wgt_mn, int which) {
                auto load_w = [&](uint32_t dst, uint32_t bar, int kb) {
                    if (wgt_mn) {
                        tma_load_3d(dst + A_BYTES, wgt, bar, n0, kb * BK, w, keep);
                        tma_load_3d(dst + A_BYTES + BK * 128, wgt, bar, n0 + 64, kb * BK, w, keep);
                    } else {
                        tma_load_3d(dst + A_BYTES, wgt, bar, kb * BK, n0, w, keep);
                    }
                };
                const int pre = nkb2 < CH_STAGES ? nkb2 : CH_STAGES;
                int armed = 0;
                for (int i = 0; i < pre && !failed; ++i) {
                    if (!wait_free(g + i)) { failed = 1; break; }
                    const uint32_t bar = full0 + 8 * stage_of(g + i);
                    mbar_expect_tx(bar, STAGE_BYTES);
                    load_w(smem_base + stage_of(g + i) * STAGE_BYTES, bar, i);
                    armed = i + 1;
                }
                // (if the wait runs out the activation halves of the armed stages are still asked for, whatever they hold, so
                //  that every copy in flight completes a barrier this thread can wait for before the CTA leaves)
                if (!failed && !count_wait(cnt + which, tiles, abort, p.error_flag, limit)) failed = 5;
                fence_async_all();
                for (int i = 0; i < armed; ++i) {
                    tma_load_3d(smem_base + stage_of(g + i) * STAGE_BYTES, act, full0 + 8 * stage_of(g + i), i * BK, 0, w);
                    issued = g + i + 1;
                }
                for (int kb = armed; kb < nkb2 && !failed; ++kb) {
                    if (!wait_free(g + kb)) { failed = 1; break; }
                    const uint32_t bar = full0 + 8 * stage_of(g + kb), dst = smem_base + stage_of(g + kb) * STAGE_BYTES;
                    mbar_expect_tx(bar, STAGE_BYTES);
                    tma_load_3d(dst, act, bar, kb * BK, 0, w);
                    load_w(dst, bar, kb);
                    issued = g + kb + 1;
                }
                g += nkb2;
            };
            layer(&k_h1, &k_w2, false, 0);
            if (!failed) layer(&k_dz2, &mn_w2, true, 2);
            if (failed) {             // let the complete blocks that were issued land before leaving
                abort[0] = 1;
                for (int o = (issued > CH_STAGES ? issued - CH_STAGES : 0); o < issued; ++o)
                    mbar_wait(full0 + 8 * stage_of(o), (o / CH_STAGES) & 1, never, limit);
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int g = 0;
            auto contraction = [&](int nkb, uint32_t acc, bool b_mn, uint32_t done_bar) {
                const uint32_t idesc = b_mn ? instr_desc(false, true) : instr_desc(false, false);
                const uint32_t b_step = b_mn ? 2048u : (uint32_t)(UMMA_K * 2);
                for (int kb = 0; kb < nkb; ++kb, ++g) {
                    if (failed) continue;
                    const int s = stage_of(g);
                    if (!mbar_wait(full0 + 8 * s, (g / CH_STAGES) & 1, abort, limit)) { failed = 2; continue; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * STAGE_BYTES, b_addr = a_addr + A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_bf16(acc, smem_desc(a_addr + k * (UMMA_K * 2), false), smem_desc(b_addr + k * b_step, b_mn), idesc,
                                  (kb > 0 || k > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                }
                if (!failed) umma_commit(done_bar);
                else abort[0] = 1;
            };
            contraction(nkb1, tmem_base, false, accum0);
            contraction(nkb2, tmem_base + TMEM_COLS, false, accum0 + 8);
            // the tile's partial logits: A = the staged h2 tile (two 64-column boxes in the operand layout as they stand),
            // B = the 16 x 128 slice of W3
            if (!failed && mbar_wait(staged, 0, abort, limit) && mbar_wait(wn_full, 0, abort, limit)) {
                tc_fence_after();
                constexpr uint32_t idesc_n = instr_desc(false, false, NEXT_N);
#pragma unroll
                for (int b = 0; b < BN / 64; ++b)
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_bf16(tmem_base + 2 * TMEM_COLS, smem_desc(T_addr + b * (BM * 128) + k * (UMMA_K * 2), false),
                                  smem_desc(smem_u32(swn) + b * (NEXT_N * 128) + k * (UMMA_K * 2), false), idesc_n,
                                  (b > 0 || k > 0) ? 1u : 0u);
                umma_commit(wn_done);
            } else if (!failed) {
                failed = 3;
                abort[0] = 1;
            }
            // (the first accumulator was drained long before the first block of this layer can arrive: its activations
            //  exist only after every CTA of the worker has finished the output layer)
            contraction(nkb2, tmem_base, true, accum0 + 16);
        }
    } else {
        // ------------------------------------------------------------------ workers
        const int row = (warp & 3) * 32 + lane;          // accumulator row = TMEM lane = sample
        const int hf = warp >> 2;                        // which 64-column box of the tile this thread drains
        const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + hf * 64;
        uint8_t *my_row = T + hf * (BM * 128) + row * 128;
        const int tid = threadIdx.x;                     // 0 .. 255
        const int j = tid & (BN - 1), sh = tid >> 7;     // output-layer phase: column of the tile; which half of the samples
        // biases of this tile; this sample's label
        {
            const __nv_bfloat16 *b = p.params + (long long)w * p.P + (tid < BN ? p.ob1 : p.ob2) + n0 + (tid & (BN - 1));
            sbias[tid] = __bfloat162float(*b);
        }
        const int y = (tid < BM) ? p.labels[(long long)w * BM + tid] : 0;
        asm volatile("bar.sync 1, 256;" ::: "memory");

        // drain one accumulator into the tile buffer as bf16 through f(value, column within this thread's 64)
        auto drain = [&](uint32_t acc_off, auto f) {
            uint32_t r[2][32];
            tmem_ld32(trow + acc_off, r[0]);
            tmem_ld32(trow + acc_off + 32, r[1]);
            tmem_ld_wait();
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                __align__(16) __nv_bfloat16 outv[32];
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) outv[jj] = f(__uint_as_float(r[cc][jj]), cc * 32 + jj);
                const uint4 *src = reinterpret_cast<const uint4 *>(outv);
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    *reinterpret_cast<uint4 *>(my_row + (((cc * 4 + jj) ^ (row & 7)) << 4)) = src[jj];
            }
        };

        // ---- layer 1
        unsigned long long on1 = 0ull;                   // (h1 > 0) of this thread's 64 columns: the mask of the last phase
        bool ok = mbar_wait(accum0, 0, abort, limit);
        ok = __all_sync(0xffffffffu, ok);
        CH_TRACE(2);
        tc_fence_after();
        if (ok) {
            drain(0, [&](float a, int jj) {
                const __nv_bfloat16 o = __float2bfloat16_rn(fmaxf(a + sbias[hf * 64 + jj], 0.0f));
                if (__bfloat162float(o) > 0.0f) on1 |= 1ull << jj;
                return o;
            });
        }
        tc_fence_before();
        fence_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0 && ok) {
            tma_store_3d(&k_h1, T_addr, n0, 0, w);
            tma_store_3d(&k_h1, T_addr + BM * 128, n0 + 64, 0, w);
            tma_store_commit();
            tma_store_wait_all();                        // complete, not only read: the other CTAs load it next
            fence_async_all();
            if (!p.debug_no_arrive) count_arrive(cnt + 0);
        }
        CH_TRACE(3);

        // ---- layer 2 and the tile's partial logits
        bool ok2 = mbar_wait(accum0 + 8, 0, abort, limit);
        ok2 = __all_sync(0xffffffffu, ok2);
        CH_TRACE(5);
        tc_fence_after();
        if (tid == 0) tma_store_wait_read<0>();          // (the tile buffer: already free, see above)
        if (ok2) {
            drain(TMEM_COLS, [&](float a, int jj) { return __float2bfloat16_rn(fmaxf(a + sbias[BN + hf * 64 + jj], 0.0f)); });
        }
        tc_fence_before();
        fence_async_smem();
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(staged) : "memory");
        // this thread's column of the output layer's weights (read before anybody may update them)
        float w3[DOUT];
#pragma unroll
        for (int c = 0; c < DOUT; ++c)
            w3[c] = (c < p.d_out) ? __bfloat162float(p.params[(long long)w * p.P + p.oW3 + (long long)c * p.d_h + n0 + j]) : 0.0f;
        bool ok3 = ok2 && mbar_wait(wn_done, 0, abort, limit);
        ok3 = __all_sync(0xffffffffu, ok3);
        CH_TRACE(6);
        tc_fence_after();
        if (hf == 0) {
            uint32_t q[NEXT_N];
            float o[NEXT_N];
            if (ok3) {
                tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + 2 * TMEM_COLS, q);
                tmem_ld_wait();
            }
#pragma unroll
            for (int c = 0; c < NEXT_N; ++c) o[c] = ok3 ? __uint_as_float(q[c]) : 0.0f;
            if (rank == 0) {                             // the output layer's bias enters with the first tile
                const __nv_bfloat16 *bn = p.params + (long long)w * p.P + p.ob3;
#pragma unroll
                for (int c = 0; c < NEXT_N; ++c) if (c < p.d_out) o[c] += __bfloat162float(bn[c]);
            }
            float4 *dst = reinterpret_cast<float4 *>(p.logit_part + (((long long)w * tiles + rank) * BM + row) * NEXT_N);
#pragma unroll
            for (int c = 0; c < NEXT_N / 4; ++c) dst[c] = make_float4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
        }
        tc_fence_before();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        bool ok5 = true;
        if (tid == 0) {
            if (ok3) count_arrive(cnt + 1);
            ok5 = ok3 && count_wait(cnt + 1, tiles, abort, p.error_flag, limit);
            if (!ok5) abort[0] = 1;
        }
        CH_TRACE(7);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        ok5 = (abort[0] == 0);
        CH_TRACE(8);

        // ---- output layer: logits (tiles in order), softmax, row loss, dz3 of sample tid
        constexpr int C4 = (DOUT + 3) / 4;
        if (tid < BM && ok5) {
            float z[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) z[c] = 0.0f;
            const float4 *pp = reinterpret_cast<const float4 *>(p.logit_part + (((long long)w * tiles) * BM + tid) * NEXT_N);
            constexpr int TB = 4;
            for (int t0 = 0; t0 < tiles; t0 += TB) {
                float4 v[TB][C4];
#pragma unroll
                for (int u = 0; u < TB; ++u)
#pragma unroll
                    for (int q = 0; q < C4; ++q)
                        v[u][q] = (t0 + u < tiles) ? __ldcg(pp + (long long)(t0 + u) * (BM * NEXT_N / 4) + q) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
                for (int u = 0; u < TB; ++u) {
                    if (t0 + u < tiles) {
#pragma unroll
                        for (int q = 0; q < C4; ++q) {
                            z[4 * q] += v[u][q].x; z[4 * q + 1] += v[u][q].y; z[4 * q + 2] += v[u][q].z; z[4 * q + 3] += v[u][q].w;
                        }
                    }
                }
            }
            float zmax = -INFINITY;
#pragma unroll
            for (int c = 0; c < 16; ++c) if (c < p.d_out) zmax = fmaxf(zmax, z[c]);
            float e[16], ssum = 0.0f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                e[c] = (c < p.d_out) ? expf(z[c] - zmax) : 0.0f;
                ssum += e[c];
            }
            float py = 0.0f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float pc = e[c] / ssum;
                if (c == y) py = pc;
                const float d = (c < p.d_out) ? (pc - (c == y ? 1.0f : 0.0f)) / (float)BM : 0.0f;
                sdz[tid * 16 + c] = __bfloat162float(__float2bfloat16_rn(d));
            }
            srowloss[tid] = -logf(py);
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        CH_TRACE(9);

        // ---- dz2 = (dz3 W3) * (h2 > 0) in place of h2, dW3 and db2 of this tile's columns.  Thread (column j, half sh) walks
        //      the samples b = 4 i + 2 sh + e, e = 0, 1: four interleaved partial sums per column, added as ((S0 + S1) + S2) + S3
        {
            float acc3[2][DOUT], csum[2] = {0.0f, 0.0f};
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
                for (int c = 0; c < DOUT; ++c) acc3[e][c] = 0.0f;
            uint8_t *col = T + (j >> 6) * (BM * 128) + (j & 7) * 2;
            const int piece = (j & 63) >> 3;
            if (ok5) {
                for (int i = 0; i < BM / 4; ++i) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int b = 4 * i + 2 * sh + e;
                        __nv_bfloat16 *cell = reinterpret_cast<__nv_bfloat16 *>(col + b * 128 + ((piece ^ (b & 7)) << 4));
                        const float h = __bfloat162float(*cell);
                        float a = 0.0f;
                        const float4 *d4 = reinterpret_cast<const float4 *>(sdz + b * 16);
#pragma unroll
                        for (int c4 = 0; c4 < C4; ++c4) {
                            const float4 dd = d4[c4];
                            const float d[4] = {dd.x, dd.y, dd.z, dd.w};
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                if (4 * c4 + u < DOUT) {
                                    a = fmaf(d[u], w3[4 * c4 + u], a);
                                    acc3[e][4 * c4 + u] = fmaf(d[u], h, acc3[e][4 * c4 + u]);
                                }
                            }
                        }
                        const __nv_bfloat16 v = __float2bfloat16_rn(h > 0.0f ? a : 0.0f);
                        *cell = v;
                        csum[e] += __bfloat162float(v);
                    }
                }
            }
            fence_async_smem();
            CH_TRACE(10);
            if (sh == 1) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
#pragma unroll
                    for (int c = 0; c < DOUT; ++c) red[(e * 16 + c) * BN + j] = acc3[e][c];
                    redsum[e * BN + j] = csum[e];
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (tid == 0 && ok5) {
                tma_store_3d(&k_dz2, T_addr, n0, 0, w);
                tma_store_3d(&k_dz2, T_addr + BM * 128, n0 + 64, 0, w);
                tma_store_commit();
                tma_store_wait_all();
                fence_async_all();
                count_arrive(cnt + 2);
            }
            CH_TRACE(11);
            if (sh == 0 && ok5) {
                // dW3 (one element per class) and db2 of column j: gradient written out, or the local step of those elements
                long long idx[DOUT + 1];
                float g[DOUT + 1];
#pragma unroll
                for (int c = 0; c < DOUT; ++c) {
                    float s = 0.0f;
                    s += acc3[0][c]; s += acc3[1][c]; s += red[c * BN + j]; s += red[(16 + c) * BN + j];
                    g[c + 1] = s;
                    idx[c + 1] = (long long)w * p.P + p.oW3 + (long long)c * p.d_h + n0 + j;
                }
                {
                    float s = 0.0f;
                    s += csum[0]; s += csum[1]; s += redsum[j]; s += redsum[BN + j];
                    g[0] = s;
                    idx[0] = (long long)w * p.P + p.ob2 + n0 + j;
                }
                if (p.step.x_in != nullptr) {
                    step_elements<DOUT + 1>(p.step, idx, g, p.d_out + 1);
                } else {
#pragma unroll
                    for (int c = 0; c < DOUT + 1; ++c) if (c < p.d_out + 1) p.grads[idx[c]] = g[c];
                }
            }
            // per-worker scalars, by the warps of the second half: db3 in the first CTA, loss and padding in the last
            if (sh == 1 && rank == 0 && ok5) {
                for (int c = warp - 4; c < p.d_out; c += 4) {
                    float s = 0.0f;
                    for (int b = lane; b < BM; b += 32) s += sdz[b * 16 + c];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if (lane == 0) {
                        if (p.step.x_in != nullptr) step_element(p.step, (long long)w * p.P + p.ob3 + c, s);
                        else p.grads[(long long)w * p.P + p.ob3 + c] = s;
                    }
                }
            }
            if (sh == 1 && rank == tiles - 1 && ok5) {
                if (warp == 4) {
                    float t[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) t[i] = srowloss[lane + 32 * i];
                    float s = (t[0] + t[1]) + (t[2] + t[3]);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if (lane == 0) p.loss[w] = s / (float)BM;
                } else {
                    for (long long i = p.P_raw + (tid - 160); i < p.P; i += 96) {
                        if (p.step.x_in != nullptr) step_element(p.step, (long long)w * p.P + i, 0.0f);
                        else p.grads[(long long)w * p.P + i] = 0.0f;
                    }
                }
            }
        }

        // ---- layer 2 backwards: dz1 = (dz2 W2) * (h1 > 0), db1 = its column sums
        bool ok4 = ok5 && mbar_wait(accum0 + 16, 0, abort, limit);
        ok4 = __all_sync(0xffffffffu, ok4);
        CH_TRACE(13);
        tc_fence_after();
        if (ok4) {
            drain(0, [&](float a, int jj) { return __float2bfloat16_rn(((on1 >> jj) & 1ull) ? a : 0.0f); });
        }
        tc_fence_before();
        fence_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0 && ok4) {
            tma_store_3d(&st_dz1, T_addr, n0, 0, w);
            tma_store_3d(&st_dz1, T_addr + BM * 128, n0 + 64, 0, w);
            tma_store_commit();
        }
        if (tid < BN && ok4) {
            // the whole batch is in this tile: thread t adds column t of the staged tile over the rows, in row order
            const uint8_t *colp = T + (tid >> 6) * (BM * 128) + (tid & 7) * 2;
            const int piece = (tid & 63) >> 3;
            float acc = 0.0f;
            for (int rr = 0; rr < BM; ++rr)
                acc += __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(colp + rr * 128 + ((piece ^ (rr & 7)) << 4)));
            const long long idx = (long long)w * p.P + p.ob1 + n0 + tid;
            if (p.step.x_in != nullptr) step_element(p.step, idx, acc);
            else p.grads[idx] = acc;
        }
        if (tid == 0) {
            tma_store_wait_read<0>();
            // the worker's last CTA to get here clears the counters for the next launch: everybody is past all waits
            if (ok4) {
                int before;
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(before) : "l"(cnt + 3) : "memory");
                if (before == tiles - 1) {
                    cnt[0] = 0; cnt[1] = 0; cnt[2] = 0; cnt[3] = 0;
                }
            }
        }
        CH_TRACE(14);
        if (!(ok && ok2 && ok3 && ok4)) failed = 4;
    }
    if (failed && p.error_flag != nullptr) atomicExch(p.error_flag, 20 + failed);
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem_base, TMEM_ALLOC);
}

}  // namespace gemm
}  // namespace cocod
