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
//   mean       : uniform  s = snap_0 ; s = s + snap_i (i = 1..K-1) ; mean = s * (1/K)
//                weighted s = w_0 * snap_0 ; s = fma(w_i, snap_i, s)
//   merge      : x = mean + (x - snap)
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace cocod {

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
__device__ __forceinline__ void st_shadow4(__nv_bfloat16 *p, const float4 &x)
{
    *reinterpret_cast<uint2 *>(p) = make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
}

__device__ __forceinline__ void sgd_update(float4 &x, float4 &v, const float4 &g, float lr, float mu, float wd)
{
    float d;
    d = __fmaf_rn(wd, x.x, g.x); v.x = __fmaf_rn(mu, v.x, d); x.x = __fmaf_rn(-lr, v.x, x.x);
    d = __fmaf_rn(wd, x.y, g.y); v.y = __fmaf_rn(mu, v.y, d); x.y = __fmaf_rn(-lr, v.y, x.y);
    d = __fmaf_rn(wd, x.z, g.z); v.z = __fmaf_rn(mu, v.z, d); x.z = __fmaf_rn(-lr, v.z, x.z);
    d = __fmaf_rn(wd, x.w, g.w); v.w = __fmaf_rn(mu, v.w, d); x.w = __fmaf_rn(-lr, v.w, x.w);
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
                int64_t nvec, float lr, float mu, float wd, __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t base = (int64_t)blockIdx.x * (THREADS * UNROLL) + threadIdx.x;
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
}

// Scalar path: misaligned pointers and the n mod 4 tail.  Elements [first, first + count).
__global__ void __launch_bounds__(kThreads)
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

__global__ void __launch_bounds__(kThreads)
snapshot_scalar(const float *__restrict__ x, float *__restrict__ snap, int64_t first, int64_t count)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += stride)
        snap[first + j] = x[first + j];
}

// ------------------------------------------------------------------------------------------ average model (Step I)
// One thread owns one float4 of columns and walks the K rows in order, RC row loads in flight
// at a time (RC * 16 B per thread).  Needs P mod 4 == 0 and 16-byte aligned bases.
template <int RC>
__global__ void __launch_bounds__(kThreads)
mean_vec4(const float4 *__restrict__ snap, int K, int64_t pvec, const float *__restrict__ w,
          float4 *__restrict__ mean, float inv_k)
{
    const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (c >= pvec) return;
    const float4 *col = snap + c;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i0 = 0; i0 < K; i0 += RC) {
        float4 r[RC];
#pragma unroll
        for (int j = 0; j < RC; ++j)
            if (i0 + j < K) r[j] = ld_stream(col + (int64_t)(i0 + j) * pvec);
#pragma unroll
        for (int j = 0; j < RC; ++j) {
            const int i = i0 + j;
            if (i < K) {
                if (w != nullptr) {
                    const float wi = __ldg(w + i);
                    if (i == 0) {
                        s.x = __fmul_rn(wi, r[j].x); s.y = __fmul_rn(wi, r[j].y);
                        s.z = __fmul_rn(wi, r[j].z); s.w = __fmul_rn(wi, r[j].w);
                    } else {
                        s.x = __fmaf_rn(wi, r[j].x, s.x); s.y = __fmaf_rn(wi, r[j].y, s.y);
                        s.z = __fmaf_rn(wi, r[j].z, s.z); s.w = __fmaf_rn(wi, r[j].w, s.w);
                    }
                } else {
                    if (i == 0) s = r[j];
                    else {
                        s.x = __fadd_rn(s.x, r[j].x); s.y = __fadd_rn(s.y, r[j].y);
                        s.z = __fadd_rn(s.z, r[j].z); s.w = __fadd_rn(s.w, r[j].w);
                    }
                }
            }
        }
    }
    if (w == nullptr) {
        s.x = __fmul_rn(s.x, inv_k); s.y = __fmul_rn(s.y, inv_k);
        s.z = __fmul_rn(s.z, inv_k); s.w = __fmul_rn(s.w, inv_k);
    }
    mean[c] = s;
}

// Few workers (K <= 4): a float4 per row would leave too few bytes in flight per thread, so
// one thread owns 8 columns (256-bit loads).  Same row order.  P mod 8 == 0, 32-byte aligned.
template <int RC>
__global__ void __launch_bounds__(kThreads)
mean_vec8(const float *__restrict__ snap, int K, int64_t P, const float *__restrict__ w,
          float *__restrict__ mean, float inv_k)
{
    const int64_t c = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 8;
    if (c >= P) return;
    f32x8 s;
    for (int i0 = 0; i0 < K; i0 += RC) {
        f32x8 r[RC];
#pragma unroll
        for (int j = 0; j < RC; ++j)
            if (i0 + j < K) r[j] = ld256_stream(snap + (int64_t)(i0 + j) * P + c);
#pragma unroll
        for (int j = 0; j < RC; ++j) {
            const int i = i0 + j;
            if (i < K) {
                if (w != nullptr) {
                    const float wi = __ldg(w + i);
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        s.a[q] = (i == 0) ? __fmul_rn(wi, r[j].a[q]) : __fmaf_rn(wi, r[j].a[q], s.a[q]);
                } else {
#pragma unroll
                    for (int q = 0; q < 8; ++q) s.a[q] = (i == 0) ? r[j].a[q] : __fadd_rn(s.a[q], r[j].a[q]);
                }
            }
        }
    }
    if (w == nullptr) {
#pragma unroll
        for (int q = 0; q < 8; ++q) s.a[q] = __fmul_rn(s.a[q], inv_k);
    }
    st256(mean + c, s);
}

// Any P / alignment: one thread per column, same row order.
__global__ void __launch_bounds__(kThreads)
mean_scalar(const float *__restrict__ snap, int K, int64_t P, const float *__restrict__ w,
            float *__restrict__ mean, float inv_k)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    float s;
    if (w != nullptr) {
        s = __fmul_rn(__ldg(w), snap[p]);
        for (int i = 1; i < K; ++i) s = __fmaf_rn(__ldg(w + i), snap[(int64_t)i * P + p], s);
    } else {
        s = snap[p];
        for (int i = 1; i < K; ++i) s = __fadd_rn(s, snap[(int64_t)i * P + p]);
        s = __fmul_rn(s, inv_k);
    }
    mean[p] = s;
}

// ------------------------------------------------------------------------------------------ merge (line 6)
// Same column ownership: the average is read once per column (4/K B per worker-parameter) and
// reused for all K rows; RC rows (2 * RC loads) in flight per thread.  x may alias snap (a
// merge with no local step in between): every element is read before it is written.
template <int RC>
__global__ void __launch_bounds__(kThreads)
merge_vec4(float4 *x, const float4 *snap, const float4 *__restrict__ mean, int K, int64_t pvec,
           __nv_bfloat16 *__restrict__ shadow)
{
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
}

// Widest path (P mod 8 == 0, 32-byte aligned bases): one thread owns 8 columns (256-bit accesses,
// a warp sweeps 1 KB of a row), blockIdx.y picks a group of RC rows, so consecutive CTAs stream
// along rows.  Sustains 6.80 TB/s on B200 where the float4 / all-rows-per-thread shape above
// sustains 6.48 TB/s.  x may alias snap.
template <int RC>
__global__ void __launch_bounds__(kThreads)
merge_vec8(float *x, const float *snap, const float *__restrict__ mean, int K, int64_t P,
           __nv_bfloat16 *__restrict__ shadow)
{
    const int64_t c = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * 8;
    if (c >= P) return;
    const f32x8 m = ld256(mean + c);
    const int i0 = blockIdx.y * RC;
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
            if (shadow != nullptr)
                *reinterpret_cast<uint4 *>(shadow + e) =
                    make_uint4(pack_bf16x2(o.a[0], o.a[1]), pack_bf16x2(o.a[2], o.a[3]),
                               pack_bf16x2(o.a[4], o.a[5]), pack_bf16x2(o.a[6], o.a[7]));
        }
}

__global__ void __launch_bounds__(kThreads)
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

// Broadcast P values to K rows ("Initialize: x_i^0 = x_hat_0").
__global__ void __launch_bounds__(kThreads)
broadcast_rows(const float *__restrict__ x0, float *__restrict__ x, int K, int64_t P)
{
    const int64_t p = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (p >= P) return;
    const float a = x0[p];
    for (int i = 0; i < K; ++i) x[(int64_t)i * P + p] = a;
}

// shadow[e] = bf16(x[e]) for a whole buffer (after the parameters were set from outside).
__global__ void __launch_bounds__(kThreads)
shadow_refresh(const float *__restrict__ x, __nv_bfloat16 *__restrict__ shadow, int64_t n)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride)
        shadow[e] = __float2bfloat16_rn(x[e]);
}

}  // namespace cocod
