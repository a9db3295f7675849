// Device kernels of the CoCoD-SGD parameter path (Algorithm 1 of arxiv 1906.12043) for sm_100a.
//
// All four are HBM-bandwidth-bound streaming kernels (0.2-0.3 flop per byte): the design
// goal is full-width coalesced 128-bit accesses, enough independent loads in flight per SM to
// cover HBM latency, and no byte moved twice.  K x P matrices are worker-major row-major fp32
// with row stride P.
//
// Arithmetic order is fixed (and mirrored by the test oracle's fp32 mode, so results can be
// compared bit for bit):
//   local step : d = fma(wd, x, g) ; v = fma(mu, v, d) ; x = fma(-lr, v, x)
//   mean       : rows are taken in blocks of 8 consecutive workers; a block is summed as a balanced
//                pairwise tree ((t0+t1)+(t2+t3))+((t4+t5)+(t6+t7)) (absent rows are skipped, not
//                added as zeros), block sums are accumulated in block order; t_i = snap_i and
//                mean = s * (1/K) for equal weights, t_i = w_i * snap_i and mean = s otherwise.
//                (Rounding error grows with log2(8) + K/8 additions instead of K.)
//   merge      : x = mean + (x - snap)
//   step+merge : the local step's three operations, then the merge's two, on the stepped x (same values as the two
//                kernels one after the other)
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace cocod {

// (Non-template kernels are `static`: this header is included by both translation units of the library.)
constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------ loads / stores
// Stored copies are read exactly once per kernel: stream them (evict-first).
__device__ __forceinline__ float4 ld_stream(const float4 *p)
{
    return __ldcs(p);
}
__device__ __forceinline__ float4 ld_plain(const float4 *p) { return *p; }
__device__ __forceinline__ void st_plain(float4 *p, float4 v) { *p = v; }

// 256-bit global accesses (sm_100): one instruction per 8 floats, 32-byte aligned.
struct f32x8 { float a[8]; };
__device__ __forceinline__ f32x8 ld256(const float *p)
{
    f32x8 r;
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.a[0]), "=f"(r.a[1]), "=f"(r.a[2]), "=f"(r.a[3]), "=f"(r.a[4]), "=f"(r.a[5]),
                   "=f"(r.a[6]), "=f"(r.a[7]) : "l"(p));
    return r;
}
__device__ __forceinline__ f32x8 ld256_stream(const float *p)
{
    f32x8 r;
    asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.a[0]), "=f"(r.a[1]), "=f"(r.a[2]), "=f"(r.a[3]), "=f"(r.a[4]), "=f"(r.a[5]),
                   "=f"(r.a[6]), "=f"(r.a[7]) : "l"(p));
    return r;
}
__device__ __forceinline__ void st256(float *p, const f32x8 &r)
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(r.a[0]), "f"(r.a[1]), "f"(r.a[2]), "f"(r.a[3]), "f"(r.a[4]), "f"(r.a[5]),
                    "f"(r.a[6]), "f"(r.a[7]) : "memory");
}

// bfloat16 shadow of the parameters (round to nearest even), packed stores.
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);      // .x = a (low half), .y = b
    return *reinterpret_cast<const uint32_t *>(&h);
}
// The bf16 copy is what the gradient kernels of the next local step read (twice: forward and backward), a tenth of the
// bytes that stream past it in between: it is stored with the L2 evict-last priority.
__device__ __forceinline__ uint64_t l2_keep_policy()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void st_shadow4(__nv_bfloat16 *p, const float4 &x)
{
    asm volatile("st.global.L2::cache_hint.v2.b32 [%0], {%1, %2}, %3;"
                 :: "l"(p), "r"(pack_bf16x2(x.x, x.y)), "r"(pack_bf16x2(x.z, x.w)), "l"(l2_keep_policy()) : "memory");
}
__device__ __forceinline__ void st_shadow8(__nv_bfloat16 *p, const f32x8 &o)
{
    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;"
                 :: "l"(p), "r"(pack_bf16x2(o.a[0], o.a[1])), "r"(pack_bf16x2(o.a[2], o.a[3])),
                    "r"(pack_bf16x2(o.a[4], o.a[5])), "r"(pack_bf16x2(o.a[6], o.a[7])), "l"(l2_keep_policy()) : "memory");
}

__device__ __forceinline__ void sgd_update(float4 &x, float4 &v, const float4 &g, float lr, float mu, float wd)
{
    float d;
    d = __fmaf_rn(wd, x.x, g.x); v.x = __fmaf_rn(mu, v.x, d); x.x = __fmaf_rn(-lr, v.x, x.x);
    d = __fmaf_rn(wd, x.y, g.y); v.y = __fmaf_rn(mu, v.y, d); x.y = __fmaf_rn(-lr, v.y, x.y);
    d = __fmaf_rn(wd, x.z, g.z); v.z = __fmaf_rn(mu, v.z, d); x.z = __fmaf_rn(-lr, v.z, x.z);
    d = __fmaf_rn(wd, x.w, g.w); v.w = __fmaf_rn(mu, v.w, d); x.w = __fmaf_rn(-lr, v.w, x.w);
}

// ------------------------------------------------------------------------------------------ device-side time stamps
// Profiling only (stamp == nullptr otherwise): stamp[0] = earliest start, stamp[1] = latest end of the kernel's CTAs
// on the GPU's own nanosecond clock, which all streams share -- so the lifetimes of kernels on different streams can
// be intersected.  Only the first and the last 2048 CTAs of a grid take part (they contain the first CTA to start
// and the last to finish), which keeps the same-address atomics to a few thousand per launch.
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void stamp_begin(unsigned long long *stamp)
{
    if (stamp != nullptr && threadIdx.x == 0) {
        const unsigned long long lin = (unsigned long long)blockIdx.y * gridDim.x + blockIdx.x;
        if (lin < 2048ull) atomicMin(stamp, global_ns());
    }
}
__device__ __forceinline__ void stamp_end(unsigned long long *stamp)
{
    if (stamp != nullptr && threadIdx.x == 0) {
        const unsigned long long lin = (unsigned long long)blockIdx.y * gridDim.x + blockIdx.x;
        if (lin + 2048ull >= (unsigned long long)gridDim.x * gridDim.y) atomicMax(stamp + 1, global_ns());
    }
}

// ------------------------------------------------------------------------------------------ local step (Step II)
// One CTA owns a contiguous tile of THREADS * UNROLL float4 of the flat K*P vector: all
// 3 * UNROLL loads of a thread are issued before the first use.  x_in may equal x_out.
// Measured on B200 (K*P = 187 M, back-to-back launches): 1024 threads x 1 float4 (a CTA sweeps
// 16 KB of each stream in one go) sustains 7.02 TB/s, 256 x 4 sustains 6.84 TB/s; streaming
// (evict-first) hints on g made no difference, so plain loads are used.
// SHADOW: also write bf16(x) to `shadow` (22 B instead of 20 B per worker-parameter).
template <int THREADS, int UNROLL, bool SHADOW>
__global__ void __launch_bounds__(THREADS)
local_step_vec4(const float4 *x_in, float4 *x_out, float4 *v, const float4 *__restrict__ g,
                int64_t nvec, float lr, float mu, float wd, __nv_bfloat16 *__restrict__ shadow,
                unsigned long long *stamp, int backwards)
{
    stamp_begin(stamp);
    // backwards: the grid walks the vector from its end, so that a kernel that follows one that walked forwards starts
    // on what that one left in L2
    const unsigned blk = backwards ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
    const int64_t base = (int64_t)blk * (THREADS * UNROLL) + threadIdx.x;
    float4 xr[UNROLL], vr[UNROLL], gr[UNROLL];
    if (base + (int64_t)(UNROLL - 1) * THREADS < nvec) {       // full tile: no predicates
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t i = base + (int64_t)u * THREADS;
            gr[u] = ld_plain(g + i);
            xr[u] = ld_plain(x_in + i);
            vr[u] = ld_plain(v + i);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t i = base + (int64_t)u * THREADS;
            sgd_update(xr[u], vr[u], gr[u], lr, mu, wd);
            st_plain(v + i, vr[u]);
            st_plain(x_out + i, xr[u]);
            if (SHADOW) st_shadow4(shadow + 4 * i, xr[u]);
        }
    } else {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t i = base + (int64_t)u * THREADS;
            if (i < nvec) {
                float4 xx = ld_plain(x_in + i), vv = ld_plain(v + i), gg = ld_plain(g + i);
                sgd_update(xx, vv, gg, lr, mu, wd);
                st_plain(v + i, vv);
                st_plain(x_out + i, xx);
                if (SHADOW) st_shadow4(shadow + 4 * i, xx);
            }
        }
    }
    stamp_end(stamp);
}

// Scalar path: misaligned pointers and the n mod 4 tail.  Elements [first, first + count).
static __global__ void __launch_bounds__(kThreads)
local_step_scalar(const float *x_in, float *x_out, float *v, const float *__restrict__ g,
                  int64_t first, int64_t count, float lr, float mu, float wd, __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += stride) {
        const int64_t e = first + j;
        const float d = __fmaf_rn(wd, x_in[e], g[e]);
        const float vn = __fmaf_rn(mu, v[e], d);
        v[e] = vn;
        const float xn = __fmaf_rn(-lr, vn, x_in[e]);
        x_out[e] = xn;
        if (shadow != nullptr) shadow[e] = __float2bfloat16_rn(xn);
    }
}

// ------------------------------------------------------------------------------------------ stored copy (Step I)
template <int UNROLL>
__global__ void __launch_bounds__(kThreads)
snapshot_vec4(const float4 *__restrict__ x, float4 *__restrict__ snap, int64_t nvec)
{
    const int64_t base = (int64_t)blockIdx.x * (kThreads * UNROLL) + threadIdx.x;
    float4 r[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
        const int64_t i = base + (int64_t)u * kThreads;
        if (i < nvec) r[u] = ld_plain(x + i);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
        const int64_t i = base + (int64_t)u * kThreads;
        if (i < nvec) st_plain(snap + i, r[u]);
    }
}

static __global__ void __launch_bounds__(kThreads)
snapshot_scalar(const float *__restrict__ x, float *__restrict__ snap, int64_t first, int64_t count)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += stride)
        snap[first + j] = x[first + j];
}

// ------------------------------------------------------------------------------------------ average model (Step I)
// Balanced pairwise sum of the first cnt (1..8) entries of t[], skipping absent entries.
__device__ __forceinline__ float tree8(const float (&t)[8], int cnt)
{
    float a[4], b[2];
#pragma unroll
    for (int j = 0; j < 4; ++j) a[j] = (2 * j + 1 < cnt) ? __fadd_rn(t[2 * j], t[2 * j + 1]) : t[2 * j];
    const int c1 = (cnt + 1) >> 1;
#pragma unroll
    for (int j = 0; j < 2; ++j) b[j] = (2 * j + 1 < c1) ? __fadd_rn(a[2 * j], a[2 * j + 1]) : a[2 * j];
    const int c2 = (c1 + 1) >> 1;
    return (c2 > 1) ? __fadd_rn(b[0], b[1]) : b[0];
}
__device__ __forceinline__ float tree8_full(const float (&t)[8])
{
    return __fadd_rn(__fadd_rn(__fadd_rn(t[0], t[1]), __fadd_rn(t[2], t[3])),
                     __fadd_rn(__fadd_rn(t[4], t[5]), __fadd_rn(t[6], t[7])));
}

// Sum over the K rows of the NV columns held by one thread.  Rows are taken in blocks of 8 (all loads
// of a block in flight together); full blocks run without predicates, the last partial block with.
// CAP < 8 is for few workers (K <= CAP): a single partial block with only CAP loads per thread.
// load(i, v) fills v[0..NV) with the thread's values of row i.
template <int NV, int CAP, typename Load>
__device__ __forceinline__ void mean_rows(float (&s)[NV], int K, const float *__restrict__ w, float inv_k, Load load)
{
    int i0 = 0;
    if (CAP == 8) {
        for (; i0 + 8 <= K; i0 += 8) {
            float r[8][NV];
#pragma unroll
            for (int j = 0; j < 8; ++j) load(i0 + j, r[j]);
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                float t[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) t[j] = (w != nullptr) ? __fmul_rn(__ldg(w + i0 + j), r[j][q]) : r[j][q];
                const float blk = tree8_full(t);
                s[q] = (i0 == 0) ? blk : __fadd_rn(s[q], blk);
            }
        }
    }
    if (i0 < K) {
        const int cnt = K - i0;                    // 1 .. CAP (CAP == 8: at most 7)
        float r[CAP][NV];
#pragma unroll
        for (int j = 0; j < CAP; ++j)
            if (j < cnt) load(i0 + j, r[j]);
#pragma unroll
        for (int q = 0; q < NV; ++q) {
            float t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                t[j] = 0.0f;
                if (j < CAP && j < cnt) t[j] = (w != nullptr) ? __fmul_rn(__ldg(w + i0 + j), r[j < CAP ? j : 0][q]) : r[j < CAP ? j : 0][q];
            }
            const float blk = tree8(t, cnt);
            s[q] = (i0 == 0) ? blk : __fadd_rn(s[q], blk);
        }
    }
    if (w == nullptr) {
#pragma unroll
        for (int q = 0; q < NV; ++q) s[q] = __fmul_rn(s[q], inv_k);
    }
}

// One thread owns one float4 of columns.  Needs P mod 4 == 0 and 16-byte aligned bases.
static __global__ void __launch_bounds__(kThreads)
mean_vec4(const float4 *__restrict__ snap, int K, int64_t pvec, const float *__restrict__ w,
          float4 *__restrict__ mean, float inv_k, unsigned long long *stamp, int backwards)
{
    stamp_begin(stamp);
    const unsigned blk = backwards ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
    const int64_t c = (int64_t)blk * kThreads + threadIdx.x;
    if (c >= pvec) return;
    const float4 *col = snap + c;
    float s[4];
    mean_rows<4, 8>(s, K, w, inv_k, [&](int i, float (&v)[4]) {
        const float4 t = ld_stream(col + (int64_t)i * pvec);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    });
    mean[c] = make_float4(s[0], s[1], s[2], s[3]);
    stamp_end(stamp);
}

// Few workers (K <= CAP <= 4): a float4 per row would leave too few bytes in flight per thread, so
// one thread owns 8 columns (256-bit loads).  P mod 8 == 0, 32-byte aligned bases.
template <int CAP>
__global__ void __launch_bounds__(kThreads)
mean_vec8(const float *__restrict__ snap, int K, int64_t P, const float *__restrict__ w,
          float *__restrict__ mean, float inv_k, unsigned long long *stamp)
{
    stamp_begin(stamp);
    const int64_t c = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 8;
    if (c >= P) return;
    float s[8];
    mean_rows<8, CAP>(s, K, w, inv_k, [&](int i, float (&v)[8]) {
        const f32x8 t = ld256_stream(snap + (int64_t)i * P + c);
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = t.a[q];
    });
    f32x8 o;
#pragma unroll
    for (int q = 0; q < 8; ++q) o.a[q] = s[q];
    st256(mean + c, o);
    stamp_end(stamp);
}

// Any P / alignment: one thread per column.
static __global__ void __launch_bounds__(kThreads)
mean_scalar(const float *__restrict__ snap, int K, int64_t P, const float *__restrict__ w,
            float *__restrict__ mean, float inv_k)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    float s[1];
    mean_rows<1, 8>(s, K, w, inv_k, [&](int i, float (&v)[1]) { v[0] = snap[(int64_t)i * P + p]; });
    mean[p] = s[0];
}

// ------------------------------------------------------------------------------------------ average model over GPUs
// Workers spread over several GPUs: row i of the stored copies is wherever rows[i] points (this GPU's
// memory or a peer's, read over NVLink with ordinary loads), and the finished columns go to every
// GPU's average buffer outs[0..G) with ordinary stores.  Each GPU runs this over its own share of the
// columns [c_lo, c_hi), so every remote value crosses the link once.  Rows are summed in worker order
// by the same mean_rows as above: the result is bit-identical to the single-GPU mean however the
// workers are spread.  No waiting inside the kernel: the callers order it after "all stored copies
// exist" and order the merges after "all GPUs' kernels are done" on the stream.
static __global__ void __launch_bounds__(kThreads)
mean_gather_vec4(const float4 *const *__restrict__ rows, int K, int64_t c_lo, int64_t c_hi,
                 const float *__restrict__ w, float4 *const *__restrict__ outs, int G, float inv_k)
{
    // the row addresses once per CTA into shared memory (dynamic, K pointers): the 8 loads of a block of
    // rows then depend on nothing but a shared-memory read
    extern __shared__ const float4 *gather_rows[];
    for (int i = threadIdx.x; i < K; i += kThreads) gather_rows[i] = rows[i];
    __syncthreads();
    const int64_t c = c_lo + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= c_hi) return;
    float s[4];
    mean_rows<4, 8>(s, K, w, inv_k, [&](int i, float (&v)[4]) {
        const float4 t = __ldcs(gather_rows[i] + c);       // each value is read once
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    });
    const float4 o = make_float4(s[0], s[1], s[2], s[3]);
    for (int q = 0; q < G; ++q) outs[q][c] = o;
}

// Few workers (K <= CAP <= 4): 8 columns per thread with 256-bit accesses, as in mean_vec8.  32-byte aligned rows
// and outputs, c_lo and c_hi in units of 8 columns.
template <int CAP>
__global__ void __launch_bounds__(kThreads)
mean_gather_vec8(const float *const *__restrict__ rows, int K, int64_t c_lo, int64_t c_hi,
                 const float *__restrict__ w, float *const *__restrict__ outs, int G, float inv_k)
{
    const int64_t c = c_lo + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= c_hi) return;
    float s[8];
    mean_rows<8, CAP>(s, K, w, inv_k, [&](int i, float (&v)[8]) {
        const f32x8 t = ld256_stream(rows[i] + c * 8);
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = t.a[q];
    });
    f32x8 o;
#pragma unroll
    for (int q = 0; q < 8; ++q) o.a[q] = s[q];
    for (int q = 0; q < G; ++q) st256(outs[q] + c * 8, o);
}

static __global__ void __launch_bounds__(kThreads)
mean_gather_scalar(const float *const *__restrict__ rows, int K, int64_t p_lo, int64_t p_hi,
                   const float *__restrict__ w, float *const *__restrict__ outs, int G, float inv_k)
{
    const int64_t p = p_lo + (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= p_hi) return;
    float s[1];
    mean_rows<1, 8>(s, K, w, inv_k, [&](int i, float (&v)[1]) { v[0] = __ldcg(rows[i] + p); });
    for (int q = 0; q < G; ++q) outs[q][p] = s[0];
}

// ------------------------------------------------------------------------------------------ merge (line 6)
// Same column ownership: the average is read once per column (4/K B per worker-parameter) and
// reused for all K rows; RC rows (2 * RC loads) in flight per thread.  x may alias snap (a
// merge with no local step in between): every element is read before it is written.
template <int RC>
__global__ void __launch_bounds__(kThreads)
merge_vec4(float4 *x, const float4 *snap, const float4 *__restrict__ mean, int K, int64_t pvec,
           __nv_bfloat16 *__restrict__ shadow, unsigned long long *stamp)
{
    stamp_begin(stamp);
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= pvec) return;
    const float4 m = mean[c];
    for (int i0 = 0; i0 < K; i0 += RC) {
        float4 xr[RC], sr[RC];
#pragma unroll
        for (int j = 0; j < RC; ++j)
            if (i0 + j < K) {
                const int64_t e = (int64_t)(i0 + j) * pvec + c;
                xr[j] = ld_plain(x + e);
                sr[j] = ld_stream(snap + e);
            }
#pragma unroll
        for (int j = 0; j < RC; ++j)
            if (i0 + j < K) {
                const int64_t e = (int64_t)(i0 + j) * pvec + c;
                float4 o;
                o.x = __fadd_rn(m.x, __fsub_rn(xr[j].x, sr[j].x));
                o.y = __fadd_rn(m.y, __fsub_rn(xr[j].y, sr[j].y));
                o.z = __fadd_rn(m.z, __fsub_rn(xr[j].z, sr[j].z));
                o.w = __fadd_rn(m.w, __fsub_rn(xr[j].w, sr[j].w));
                st_plain(x + e, o);
                if (shadow != nullptr) st_shadow4(shadow + 4 * e, o);
            }
    }
    stamp_end(stamp);
}

// Widest path (P mod 8 == 0, 32-byte aligned bases): one thread owns 8 columns (256-bit accesses,
// a warp sweeps 1 KB of a row), blockIdx.y picks a group of RC rows, so consecutive CTAs stream
// along rows.  Sustains 6.80 TB/s on B200 where the float4 / all-rows-per-thread shape above
// sustains 6.48 TB/s.  x may alias snap.
template <int RC>
__global__ void __launch_bounds__(kThreads)
merge_vec8(float *x, const float *snap, const float *__restrict__ mean, int K, int64_t P,
           __nv_bfloat16 *__restrict__ shadow, unsigned long long *stamp, int backwards)
{
    stamp_begin(stamp);
    const unsigned bx = backwards ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
    const unsigned by = backwards ? gridDim.y - 1u - blockIdx.y : blockIdx.y;
    const int64_t c = ((int64_t)bx * kThreads + threadIdx.x) * 8;
    if (c >= P) return;
    const f32x8 m = ld256(mean + c);
    const int i0 = by * RC;
    f32x8 xr[RC], sr[RC];
#pragma unroll
    for (int j = 0; j < RC; ++j)
        if (i0 + j < K) {
            const int64_t e = (int64_t)(i0 + j) * P + c;
            xr[j] = ld256(x + e);
            sr[j] = ld256_stream(snap + e);
        }
#pragma unroll
    for (int j = 0; j < RC; ++j)
        if (i0 + j < K) {
            const int64_t e = (int64_t)(i0 + j) * P + c;
            f32x8 o;
#pragma unroll
            for (int q = 0; q < 8; ++q) o.a[q] = __fadd_rn(m.a[q], __fsub_rn(xr[j].a[q], sr[j].a[q]));
            st256(x + e, o);
            if (shadow != nullptr) st_shadow8(shadow + e, o);
        }
    stamp_end(stamp);
}

// Last local step of a round and line 6 in ONE pass (a fusion variant of the round; same values bit for bit as the
// local step followed by the merge): d = fma(wd, x, g) ; v = fma(mu, v, d) ; x' = fma(-lr, v, x) ; x = mean + (x' - snap).
// x' never goes to memory, the merge's re-read of x disappears: 24 + 4/K bytes per worker-parameter where the two
// kernels move 20 + 12 + 4/K.  Same shape as merge_vec8: a thread owns 8 columns and RC rows, blockIdx.y picks the row
// group.  x_in may alias snap (a round of one local step under the buffer flip) and x_in may equal x_out: every
// element is read before it is written, by the same thread.
template <int RC>
__global__ void __launch_bounds__(kThreads)
step_merge_vec8(const float *x_in, float *x_out, float *v, const float *__restrict__ g, const float *snap,
                const float *__restrict__ mean, int K, int64_t P, float lr, float mu, float wd,
                __nv_bfloat16 *__restrict__ shadow, unsigned long long *stamp, int backwards)
{
    stamp_begin(stamp);
    const unsigned bx = backwards ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
    const unsigned by = backwards ? gridDim.y - 1u - blockIdx.y : blockIdx.y;
    const int64_t c = ((int64_t)bx * kThreads + threadIdx.x) * 8;
    if (c >= P) return;
    const f32x8 m = ld256(mean + c);
    const int i0 = by * RC;
    f32x8 xr[RC], vr[RC], gr[RC], sr[RC];
#pragma unroll
    for (int j = 0; j < RC; ++j)
        if (i0 + j < K) {
            const int64_t e = (int64_t)(i0 + j) * P + c;
            gr[j] = ld256(g + e);
            xr[j] = ld256(x_in + e);
            vr[j] = ld256(v + e);
            sr[j] = ld256_stream(snap + e);
        }
#pragma unroll
    for (int j = 0; j < RC; ++j)
        if (i0 + j < K) {
            const int64_t e = (int64_t)(i0 + j) * P + c;
            f32x8 o, vn;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float d = __fmaf_rn(wd, xr[j].a[q], gr[j].a[q]);
                vn.a[q] = __fmaf_rn(mu, vr[j].a[q], d);
                const float xs = __fmaf_rn(-lr, vn.a[q], xr[j].a[q]);
                o.a[q] = __fadd_rn(m.a[q], __fsub_rn(xs, sr[j].a[q]));
            }
            st256(v + e, vn);
            st256(x_out + e, o);
            if (shadow != nullptr) st_shadow8(shadow + e, o);
        }
    stamp_end(stamp);
}

static __global__ void __launch_bounds__(kThreads)
merge_scalar(float *x, const float *snap, const float *__restrict__ mean, int K, int64_t P,
             __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    const float m = mean[p];
    for (int i = 0; i < K; ++i) {
        const int64_t e = (int64_t)i * P + p;
        const float o = __fadd_rn(m, __fsub_rn(x[e], snap[e]));
        x[e] = o;
        if (shadow != nullptr) shadow[e] = __float2bfloat16_rn(o);
    }
}

// Local step of every worker with ONE gradient vector shared by all (S-SGD: the averaged gradient):
// grid (blocks over P / 4, K); gbar is read K times but stays in L2.  Same arithmetic as the local step.
static __global__ void __launch_bounds__(kThreads)
local_step_shared_grad_vec4(const float4 *x_in, float4 *x_out, float4 *v, const float4 *__restrict__ gbar,
                            int64_t pvec, float lr, float mu, float wd, __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= pvec) return;
    const int64_t e = (int64_t)blockIdx.y * pvec + c;
    float4 xx = x_in[e], vv = v[e];
    const float4 gg = gbar[c];
    sgd_update(xx, vv, gg, lr, mu, wd);
    v[e] = vv;
    x_out[e] = xx;
    if (shadow != nullptr) st_shadow4(shadow + 4 * e, xx);
}
static __global__ void __launch_bounds__(kThreads)
local_step_shared_grad_scalar(const float *x_in, float *x_out, float *v, const float *__restrict__ gbar, int64_t P,
                              float lr, float mu, float wd, __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    const int64_t e = (int64_t)blockIdx.y * P + p;
    const float d = __fmaf_rn(wd, x_in[e], gbar[p]);
    const float vn = __fmaf_rn(mu, v[e], d);
    v[e] = vn;
    const float xn = __fmaf_rn(-lr, vn, x_in[e]);
    x_out[e] = xn;
    if (shadow != nullptr) shadow[e] = __float2bfloat16_rn(xn);
}

// Broadcast P values to K rows (Algorithm 1, Initialize: x_i^0 = x_hat_0 for every worker).
static __global__ void __launch_bounds__(kThreads)
broadcast_rows(const float *__restrict__ x0, float *__restrict__ x, int K, int64_t P)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    const float a = x0[p];
    for (int i = 0; i < K; ++i) x[(int64_t)i * P + p] = a;
}

// shadow[e] = bf16(x[e]) for a whole buffer (after the parameters were set from outside).
static __global__ void __launch_bounds__(kThreads)
shadow_refresh(const float *__restrict__ x, __nv_bfloat16 *__restrict__ shadow, int64_t n)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride)
        shadow[e] = __float2bfloat16_rn(x[e]);
}

}  // namespace cocod
