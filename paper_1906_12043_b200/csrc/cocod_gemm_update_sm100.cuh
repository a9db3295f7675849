// Weight-gradient GEMM fused with the momentum-SGD update (Algorithm 1, Step II: gradient and update of
// one iteration), as ONE persistent, warp-specialised kernel over the tiles of up to two weight matrices.
//
//   g = A^T-view x B-view   (bf16 operands read with their row index contiguous, fp32 accumulation in TMEM)
//   d = fma(wd, x, g) ; v = fma(mu, v, d) ; x = fma(-lr, v, x) ; shadow = bf16(x)
//
// Why persistent: the update moves 18 B per parameter through an SM that holds one 128 x 128 tile at a
// time (x and v: 128 KB of shared memory).  As one CTA per tile, the tile's loads, its arithmetic and its
// store drain follow one another and the SM's share of HBM idles between tiles.  Here one CTA per SM walks
// over its tiles with three roles that run ahead of one another:
//
//   warp 0 (one lane)   producer: TMA loads of the operand blocks (2-stage ring) and of the x / v chunks
//                       (four 32-column chunks, each re-armed as soon as its stores have read it)
//   warp 1 (one lane)   MMA issuer: tcgen05.mma into one of TWO accumulators in TMEM, so the next tile's
//                       product is formed while the current tile is being updated
//   warps 2..9          update: TMEM -> registers, x and v updated in place in shared memory (TMA swizzle),
//                       bulk stores chunk by chunk (x, v and the staged bf16 copy of x)
//
// so that the loads of tile t + 1 run under the update and the store drain of tile t.  The same kernel also serves the
// gradient call that writes the weight gradients out (store_only): the update warps then stage the product itself, in
// the x / v buffers alternately from tile to tile, and store it through x_out.  All waits are
// bounded (the kernel reports a timeout through error_flag, lets issued copies land, frees TMEM, returns).
//
// Every x / v chunk buffer and its two barriers belong to ONE update group for the whole kernel.  That matters: an
// mbarrier wait knows only the parity of the phase it waits for, so a waiter that could get two uses ahead of a
// barrier would pass at once on stale data.  (A variant with the operands in a single stage and a ring of five
// chunk slots handed from group to group -- one more chunk of x and v in flight per SM -- had exactly that fault
// until each slot got three "landed" barriers used in turn; it was then correct and 3 us per step SLOWER, because
// the tensor-core thread had to fetch its two operand blocks one after the other: bytes in flight are not what
// bounds this kernel.)
#pragma once
#include "cocod_gemm_sm100.cuh"

namespace cocod {
namespace gemm {

struct UpdateProblem {
    CUtensorMap a, b;                  // operands [K][M] and [K][N] per worker (row index contiguous), bf16
    CUtensorMap x_in, x_out, v;        // fp32 [M][N] per worker, boxes of 32 columns x 128 rows, 128-byte swizzle
    CUtensorMap shadow;                // bf16 copy of x, boxes of 64 columns x 128 rows, 128-byte swizzle
    int has_shadow;
    int M, N;
    int tiles_m, tiles_n, tiles;       // tiles = workers * tiles_m * tiles_n (0: problem absent)
};

struct UpdateParams {
    int K;                             // reduction length, at most 2 * BK (one operand block per ring stage)
    float lr, mu, wd;
    int *error_flag;
    unsigned long long wait_ns;        // time limit of every barrier wait (0 = WAIT_LIMIT_NS)
    int debug_no_loads;                // self-test: the producer issues nothing, so the waits run out
    int store_only;                    // 1: no update -- the product itself (the weight gradient) is written through x_out;
                                       //    x_in, v and shadow of the problems are unused, nothing but the operands is loaded
    unsigned long long *stamp;         // measurement (nullptr = off): [0] earliest start, [1] latest end of the CTAs, in ns
                                       // of the GPU's clock, taken after the wait for the predecessor and at the very end
};

constexpr int UPD_THREADS = 320;       // producer warp, MMA warp, 8 update warps
constexpr int UPD_RING = 2 * STAGE_BYTES;                       // two operand blocks
constexpr int UPD_XV = 2 * BM * BN * 4;                         // x and v of one tile
constexpr int UPD_SHADOW = BM * BN * 2;                         // staging of the bf16 copy of one tile
constexpr int UPD_SMEM = UPD_RING + UPD_XV + UPD_SHADOW + 1024 + 1024;      // + alignment slack + barriers

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// grid = min(tiles of both problems, number of SMs); block = UPD_THREADS; dynamic shared memory = UPD_SMEM.
__global__ void __launch_bounds__(UPD_THREADS, 1)
gemm_update_persistent(const __grid_constant__ UpdateProblem p0, const __grid_constant__ UpdateProblem p1,
                       const UpdateParams q)
{
    extern __shared__ uint8_t upd_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(upd_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xs = smem + UPD_RING, *vs = xs + BM * BN * 4;
    uint8_t *ss = vs + BM * BN * 4;           // bf16 staging: 64-column box b at b * 16 KB
    uint64_t *bars = reinterpret_cast<uint64_t *>(ss + UPD_SHADOW);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 3), accf0 = smem_u32(bars + 6), acce0 = smem_u32(bars + 8);
    const uint32_t xvf0 = smem_u32(bars + 10), xve0 = smem_u32(bars + 14);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 18);
    // Operand ring: two stages of one reduction block each (one tile's operands) -- three in store_only mode, where the
    // staging area of the bf16 copy is free: the first block of the next tile is then fetched while this tile's second
    // block is still being multiplied.  Block number o = tile index * nkb + kb sits in stage o % n_stages.
    const int n_stages = q.store_only ? 3 : 2;
    auto stage_addr = [&](int st) { return st < 2 ? smem_u32(smem) + st * STAGE_BYTES : smem_u32(ss); };
    volatile int *abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *never = abort + 1;          // stays 0: used by waits that must not be cut short

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (q.K + BK - 1) / BK;      // 1 or 2
    const int total = p0.tiles + p1.tiles;
    const uint32_t smem_base = smem_u32(smem);
    const unsigned long long limit = q.wait_ns ? q.wait_ns : WAIT_LIMIT_NS;

    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p0.a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p0.b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p0.x_in) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&p0.v) : "memory");
        for (int s = 0; s < 3; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(accf0 + 8 * s, 1);
            mbar_init(acce0 + 8 * s, 8);      // one arrival per update warp
        }
        for (int c = 0; c < 4; ++c) {
            mbar_init(xvf0 + 8 * c, 1);
            mbar_init(xve0 + 8 * c, 1);
        }
        abort[0] = 0;
        abort[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {                  // warp-collective TMEM allocation: two accumulators of 128 columns
        tmem_alloc(smem_u32(tmem_slot), 2 * TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();
    pdl_wait();
    if (q.stamp != nullptr && threadIdx.x == 0) atomicMin(q.stamp, now_ns());

    // tile t of the whole list -> problem, worker, tile origin
    auto decode = [&](int t, const UpdateProblem *&P, int &wk, int &m0, int &n0) {
        P = (t < p0.tiles) ? &p0 : &p1;
        if (t >= p0.tiles) t -= p0.tiles;
        const int per = P->tiles_m * P->tiles_n;
        wk = t / per;
        const int rem = t - wk * per;
        m0 = (rem / P->tiles_n) * BM;
        n0 = (rem % P->tiles_n) * BN;
    };

    int failed = 0;
    if (warp == 0 && lane == 0) {
        // ---- producer
        int i = 0, issued_ops = 0, issued_xv = 0;      // operand blocks / tiles whose x-v copies have been issued
        for (int t = blockIdx.x; t < total && !failed && !q.debug_no_loads; t += gridDim.x, ++i) {
            const UpdateProblem *P; int wk, m0, n0;
            decode(t, P, wk, m0, n0);
            for (int kb = 0; kb < nkb; ++kb) {
                const int o = i * nkb + kb, st = o % n_stages, use = o / n_stages;
                if (use > 0 && !mbar_wait(empty0 + 8 * st, (use - 1) & 1, abort, limit)) { failed = 1; break; }
                const uint32_t bar = full0 + 8 * st;
                mbar_expect_tx(bar, STAGE_BYTES);
                const uint32_t dst_a = stage_addr(st), dst_b = dst_a + A_BYTES;
                tma_load_3d(dst_a, &P->a, bar, m0, kb * BK, wk);
                tma_load_3d(dst_a + BK * 128, &P->a, bar, m0 + 64, kb * BK, wk);
                tma_load_3d(dst_b, &P->b, bar, n0, kb * BK, wk);
                tma_load_3d(dst_b + BK * 128, &P->b, bar, n0 + 64, kb * BK, wk);
                issued_ops = o + 1;
            }
            if (failed) break;
            for (int cq = 0; cq < 4 && !q.store_only; ++cq) {
                const int c = ((cq & 1) << 1) | (cq >> 1);      // 0, 2, 1, 3: each group's first chunk first
                if (i > 0 && !mbar_wait(xve0 + 8 * c, (i - 1) & 1, abort, limit)) { failed = 1; break; }
                const uint32_t bar = xvf0 + 8 * c;
                mbar_expect_tx(bar, 2 * BM * 128);
                tma_load_3d(smem_u32(xs) + c * (BM * 128), &P->x_in, bar, n0 + c * 32, m0, wk);
                tma_load_3d(smem_u32(vs) + c * (BM * 128), &P->v, bar, n0 + c * 32, m0, wk);
            }
            if (!failed) issued_xv = i + 1;
        }
        if (failed) {                 // let the copies of the last issued tile land before leaving
            abort[0] = 1;
            for (int o = (issued_ops > n_stages ? issued_ops - n_stages : 0); o < issued_ops; ++o)
                mbar_wait(full0 + 8 * (o % n_stages), (o / n_stages) & 1, never, limit);
            if (issued_xv > 0)
                for (int c = 0; c < 4; ++c) mbar_wait(xvf0 + 8 * c, (issued_xv - 1) & 1, never, limit);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        constexpr uint32_t idesc = instr_desc(true, true);
        int i = 0;
        for (int t = blockIdx.x; t < total && !failed; t += gridDim.x, ++i) {
            const int a = i & 1, u = i >> 1;
            if (u > 0 && !mbar_wait(acce0 + 8 * a, (u - 1) & 1, abort, limit)) { failed = 2; break; }
            tc_fence_after();
            for (int kb = 0; kb < nkb; ++kb) {
                const int o = i * nkb + kb, st = o % n_stages, use = o / n_stages;
                if (!mbar_wait(full0 + 8 * st, use & 1, abort, limit)) { failed = 2; break; }
                tc_fence_after();
                const uint32_t a_addr = stage_addr(st), b_addr = a_addr + A_BYTES;
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k)
                    umma_bf16(tmem_base + a * TMEM_COLS, smem_desc(a_addr + k * 2048u, true), smem_desc(b_addr + k * 2048u, true),
                              idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(empty0 + 8 * st);     // frees the stage once these MMAs have read it
            }
            if (failed) break;
            umma_commit(accf0 + 8 * a);           // accumulator complete
        }
        if (failed) abort[0] = 1;
    } else if (warp >= 2) {
        // ---- update warps: group 0 (warps 2..5) owns chunks 0 and 1, group 1 (warps 6..9) chunks 2 and 3;
        //      a warp reaches the TMEM lanes 32 (warp % 4) .. + 31
        const int group = (warp - 2) >> 2, quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const bool leader = (warp == 2 + 4 * group) && lane == 0;
        int i = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++i) {
            const UpdateProblem *P; int wk, m0, n0;
            decode(t, P, wk, m0, n0);
            const int a = i & 1, u = i >> 1;
            // (a thread that has given up keeps walking the tiles without touching anything, so that every
            //  named barrier below still sees all of its 128 threads)
            bool ok = !failed && mbar_wait(accf0 + 8 * a, u & 1, abort, limit);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            uint2 held[8];            // bf16 copy of the first chunk: staged together with the second one (see below)
            // store_only: tile i stages in the x buffers, tile i + 1 in the v buffers.  A thread that writes tile i + 1 has
            // passed the named barriers of tile i, which the leader joined only after the stores of tile i - 1 (the last
            // user of the same buffers) had read them (its wait at the end of tile i - 1, below).
            uint8_t *xb = (q.store_only && (i & 1)) ? vs : xs;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                const int c = group * 2 + cc;
                uint32_t r[32];
                if (ok) {
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + a * TMEM_COLS + c * 32, r);
                    tmem_ld_wait();
                }
                if (cc == 1) {        // this warp has read all it needs of the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acce0 + 8 * a);
                }
                if (!q.store_only) {
                    ok = ok && mbar_wait(xvf0 + 8 * c, i & 1, abort, limit);      // this chunk's x and v
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (ok && q.store_only) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4 *>(xb + c * (BM * 128) + row * 128 + ((j ^ (row & 7)) << 4)) =
                            make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                } else if (ok) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int off = c * (BM * 128) + row * 128 + ((j ^ (row & 7)) << 4);
                        float4 xx = *reinterpret_cast<float4 *>(xs + off), vv = *reinterpret_cast<float4 *>(vs + off);
                        const float4 gg = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                      __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                        sgd_update(xx, vv, gg, q.lr, q.mu, q.wd);
                        *reinterpret_cast<float4 *>(xs + off) = xx;
                        *reinterpret_cast<float4 *>(vs + off) = vv;
                        // The staging of the bf16 copy is still being read by the previous tile's store while the
                        // first chunk is updated (its buffers came back early): hold these values in registers
                        // and stage them with the second chunk, whose buffers come back after that store.
                        const uint2 pk = make_uint2(pack_bf16x2(xx.x, xx.y), pack_bf16x2(xx.z, xx.w));
                        if (cc == 0) {
                            held[j] = pk;
                        } else if (P->has_shadow) {
                            uint8_t *srow = ss + group * (BM * 128) + row * 128;
                            const int n1 = 32 + 4 * j, n0c = 4 * j;       // columns within the group's 64-column box
                            *reinterpret_cast<uint2 *>(srow + ((((n1 & 63) >> 3) ^ (row & 7)) << 4) + ((n1 >> 2) & 1) * 8) = pk;
                            *reinterpret_cast<uint2 *>(srow + ((((n0c & 63) >> 3) ^ (row & 7)) << 4) + ((n0c >> 2) & 1) * 8) = held[j];
                        }
                    }
                }
                fence_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(group + 1) : "memory");
                if (leader) {
                    if (ok && n0 + c * 32 < P->N) {
                        tma_store_3d(&P->x_out, smem_u32(xb) + c * (BM * 128), n0 + c * 32, m0, wk);
                        if (!q.store_only) tma_store_3d(&P->v, smem_u32(vs) + c * (BM * 128), n0 + c * 32, m0, wk);
                    }
                    // the group's 64-column box of the bf16 copy is complete after its second chunk
                    // (evict-last: the 59 MB of bf16 weights are what the next step's forward and backward GEMMs read; x and v,
                    //  ten times as much, pass through L2 with the normal priority.  Evict-first on the x / v loads cost 8 us.)
                    if (ok && cc == 1 && !q.store_only && P->has_shadow && n0 + group * 64 < P->N)
                        tma_store_3d(&P->shadow, smem_u32(ss) + group * (BM * 128), n0 + group * 64, m0, wk, l2_policy_evict_last());
                    tma_store_commit();
                }
            }
            if (leader) {
                if (q.store_only) {
                    tma_store_wait_read<0>();
                } else {              // a chunk's buffers go back to the producer once its stores have read them
                    tma_store_wait_read<1>();
                    mbar_arrive(xve0 + 8 * (group * 2));
                    tma_store_wait_read<0>();
                    mbar_arrive(xve0 + 8 * (group * 2 + 1));
                }
            }
            if (!ok && !failed) {
                failed = 3;
                abort[0] = 1;
            }
        }
        if (leader) tma_store_wait_read<0>();      // shared memory must outlive the reads of the last stores
    }
    if (failed && q.error_flag != nullptr) atomicExch(q.error_flag, 10 + failed);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * TMEM_COLS);
    if (q.stamp != nullptr && threadIdx.x == 0) atomicMax(q.stamp + 1, now_ns());
}

}  // namespace gemm
}  // namespace cocod
