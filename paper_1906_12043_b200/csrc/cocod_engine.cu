// libcocod.so: host side of the CoCoD-SGD parameter engine -- state machine, stream/event
// plumbing and kernel launches behind the C boundary declared in include/cocod.h.
//
// One round of Algorithm 1 (arxiv 1906.12043) maps to
//   comm_begin : [compute] stored copy (copy kernel, or buffer flip) -> ev_snap
//                [side]    wait ev_snap -> mean kernel -> ev_mean
//   local_step : [compute] fused momentum-SGD kernel over the flat K*P vector, k times
//   comm_end   : [compute] wait ev_mean -> merge kernel
// Ordering is by stream events only; no kernel spins on another and the host never blocks
// inside a round.
#include "cocod.h"
#include "cocod_internal.h"
#include "cocod_kernels.cuh"

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

#include <unistd.h>

namespace {

constexpr int kMaxWorkers = 1024;
constexpr int kMaxRanks = 64;
constexpr int kMaxProfile = 16384;
constexpr int64_t kHostChunk = int64_t(1) << 24;   // elements per staged host->device chunk (64 MiB)
constexpr int kHostSlots = 2;

enum State { IDLE = 0, IN_FLIGHT = 1 };

struct ProfileRec {
    int kind;
    cudaEvent_t a, b;
};

// Where the kernel launched inside the current profiling bracket leaves its device-side time stamps
// (nullptr outside a bracket, for the stateless entry points, and while profiling is off).
thread_local unsigned long long *g_stamp = nullptr;
// Experiment: direction in which the next streaming kernel walks its data (see COCOD_OPT_SWEEP).
thread_local int g_backwards = 0;

}  // namespace

struct cocod_engine {
    int K = 0;
    int64_t P = 0, n = 0;
    float lr = 0, mu = 0, wd = 0;
    int device = 0;
    // buf[cur] holds x; buf[1 - cur] holds the stored copies (or is spare between rounds)
    float *buf[2] = {nullptr, nullptr};
    int cur = 0;
    float *v = nullptr, *mean = nullptr, *w = nullptr;
    __nv_bfloat16 *shadow = nullptr;    // optional bf16 copy of x, kept current by every kernel that writes x
    bool weighted = false;
    const float *snap = nullptr;       // where this round's stored copies live
    bool pending_flip = false;          // FLIP mode: x still lives in the stored-copy buffer
    bool mean_valid = false;
    bool mean_captured = false;         // the last averaging was recorded into a CUDA graph, not executed
    int state = IDLE;
    int snapshot_mode = COCOD_SNAPSHOT_FLIP;
    cudaStream_t compute = nullptr, side = nullptr, copy = nullptr;
    cudaEvent_t ev_snap = nullptr, ev_mean = nullptr, ev_tmp = nullptr;
    // workers spread over several GPUs (K_global == 0: this engine holds all workers)
    int K_global = 0, first = 0;
    float *wg = nullptr;                // weights of all K_global workers (device), when batch sizes differ
    bool mean_started = false;          // this round's kernel that fills the average buffer has been queued
    bool exchanged = false;             // ... and the caller has marked the buffer complete
    int G = 0, rank = 0;                // attached peers (G == 0: none)
    void *opened[kMaxRanks][3] = {};    // peer buffers opened through inter-process handles (to be closed)
    const float **rows_tab[2] = {nullptr, nullptr};   // device: row pointers of all K_global workers in buf[0] / buf[1]
    float **outs_tab = nullptr;         // device: every GPU's average buffer
    // staging for host gradients
    float *stage[kHostSlots] = {nullptr, nullptr};
    cudaEvent_t ev_copied[kHostSlots] = {nullptr, nullptr}, ev_consumed[kHostSlots] = {nullptr, nullptr};
    bool slot_used[kHostSlots] = {false, false};
    bool host_ready = false;            // copy stream, staging buffers and their events all exist
    // bookkeeping
    int64_t steps = 0, launches = 0;
    int cuda_error = 0;
    bool sweep = false;                 // COCOD_OPT_SWEEP: consecutive streaming kernels walk in alternating directions
    int dir = 0;                        // direction of the last kernel on the compute stream
    bool profile = false;
    std::vector<ProfileRec> prof;
    unsigned long long *stamps = nullptr;       // device: kMaxProfile x {earliest start, latest end} in ns of the GPU's clock
    std::vector<unsigned long long> stamps_host; // copy taken by cocod_profile_count
};

namespace {

inline bool fail(cocod_engine *h, cudaError_t e)
{
    if (e == cudaSuccess) return false;
    if (h && h->cuda_error == 0) h->cuda_error = (int)e;
    return true;
}
#define CK(h, call) do { if (fail((h), (call))) return COCOD_ERR_CUDA; } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

inline unsigned grid_for(int64_t items, int per_block)
{
    return (unsigned)((items + per_block - 1) / per_block);
}

// ---------------------------------------------------------------- launchers (shared with the stateless entry points)
cudaError_t launch_local_step(const float *x_in, float *x_out, float *v, const float *g, int64_t n,
                              float lr, float mu, float wd, __nv_bfloat16 *shadow, cudaStream_t s, int *n_launch)
{
    using namespace cocod;
    if (n <= 0) return cudaSuccess;
    constexpr int THREADS = 1024, UNROLL = 1;
    int64_t done = 0;
    if (aligned16(x_in) && aligned16(x_out) && aligned16(v) && aligned16(g) && n >= 4 &&
        (shadow == nullptr || (reinterpret_cast<uintptr_t>(shadow) & 7u) == 0)) {
        const int64_t nvec = n / 4;
        const unsigned grid = grid_for(nvec, THREADS * UNROLL);
        if (shadow != nullptr)
            local_step_vec4<THREADS, UNROLL, true><<<grid, THREADS, 0, s>>>(
                reinterpret_cast<const float4 *>(x_in), reinterpret_cast<float4 *>(x_out),
                reinterpret_cast<float4 *>(v), reinterpret_cast<const float4 *>(g), nvec, lr, mu, wd, shadow, g_stamp, g_backwards);
        else
            local_step_vec4<THREADS, UNROLL, false><<<grid, THREADS, 0, s>>>(
                reinterpret_cast<const float4 *>(x_in), reinterpret_cast<float4 *>(x_out),
                reinterpret_cast<float4 *>(v), reinterpret_cast<const float4 *>(g), nvec, lr, mu, wd, nullptr, g_stamp, g_backwards);
        done = nvec * 4;
        if (n_launch) ++*n_launch;
    }
    if (done < n) {
        const int64_t rest = n - done;
        const unsigned grid = (unsigned)std::min<int64_t>((rest + kThreads - 1) / kThreads, 148 * 8);
        local_step_scalar<<<grid, kThreads, 0, s>>>(x_in, x_out, v, g, done, rest, lr, mu, wd, shadow);
        if (n_launch) ++*n_launch;
    }
    return cudaGetLastError();
}

cudaError_t launch_snapshot(const float *x, float *snap, int64_t n, cudaStream_t s, int *n_launch)
{
    using namespace cocod;
    if (n <= 0) return cudaSuccess;
    constexpr int UNROLL = 4;
    int64_t done = 0;
    if (aligned16(x) && aligned16(snap) && n >= 4) {
        const int64_t nvec = n / 4;
        snapshot_vec4<UNROLL><<<grid_for(nvec, kThreads * UNROLL), kThreads, 0, s>>>(
            reinterpret_cast<const float4 *>(x), reinterpret_cast<float4 *>(snap), nvec);
        done = nvec * 4;
        if (n_launch) ++*n_launch;
    }
    if (done < n) {
        const int64_t rest = n - done;
        const unsigned grid = (unsigned)std::min<int64_t>((rest + kThreads - 1) / kThreads, 148 * 8);
        snapshot_scalar<<<grid, kThreads, 0, s>>>(x, snap, done, rest);
        if (n_launch) ++*n_launch;
    }
    return cudaGetLastError();
}

// inv_k: factor of the unweighted sum (1/K; 1/K_global for a partial sum over this GPU's workers)
cudaError_t launch_mean(const float *snap, int K, int64_t P, const float *w, float *mean, float inv_k,
                        cudaStream_t s, int *n_launch)
{
    using namespace cocod;
    if (K <= 4 && (P % 8) == 0 && aligned32(snap) && aligned32(mean)) {
        const unsigned grid = grid_for(P / 8, kThreads);
        if (K <= 2) mean_vec8<2><<<grid, kThreads, 0, s>>>(snap, K, P, w, mean, inv_k, g_stamp);
        else mean_vec8<4><<<grid, kThreads, 0, s>>>(snap, K, P, w, mean, inv_k, g_stamp);
    } else if ((P % 4) == 0 && aligned16(snap) && aligned16(mean)) {
        const int64_t pvec = P / 4;
        mean_vec4<<<grid_for(pvec, kThreads), kThreads, 0, s>>>(
            reinterpret_cast<const float4 *>(snap), K, pvec, w, reinterpret_cast<float4 *>(mean), inv_k, g_stamp, g_backwards);
    } else {
        mean_scalar<<<grid_for(P, kThreads), kThreads, 0, s>>>(snap, K, P, w, mean, inv_k);
    }
    if (n_launch) ++*n_launch;
    return cudaGetLastError();
}

// Average of columns [lo, hi) over rows held in separate allocations, written to G buffers.  vec (1, 4 or 8):
// the caller vouches that all row and output pointers are 4 * vec-byte aligned and lo, hi are multiples of vec.
cudaError_t launch_mean_gather(const float *const *rows, int K, int64_t lo, int64_t hi, const float *w,
                               float *const *outs, int G, float inv_k, int vec, cudaStream_t s, int *n_launch)
{
    using namespace cocod;
    if (hi <= lo) return cudaSuccess;
    if (vec == 8 && K <= 4) {           // few workers: 256-bit accesses keep enough bytes in flight
        const int64_t c_lo = lo / 8, c_hi = hi / 8;
        const unsigned grid = grid_for(c_hi - c_lo, kThreads);
        if (K <= 2) mean_gather_vec8<2><<<grid, kThreads, 0, s>>>(rows, K, c_lo, c_hi, w, outs, G, inv_k);
        else mean_gather_vec8<4><<<grid, kThreads, 0, s>>>(rows, K, c_lo, c_hi, w, outs, G, inv_k);
    } else if (vec >= 4) {
        const int64_t c_lo = lo / 4, c_hi = hi / 4;
        mean_gather_vec4<<<grid_for(c_hi - c_lo, kThreads), kThreads, (size_t)K * sizeof(float4 *), s>>>(
            reinterpret_cast<const float4 *const *>(rows), K, c_lo, c_hi, w,
            reinterpret_cast<float4 *const *>(outs), G, inv_k);
    } else {
        mean_gather_scalar<<<grid_for(hi - lo, kThreads), kThreads, 0, s>>>(rows, K, lo, hi, w, outs, G, inv_k);
    }
    if (n_launch) ++*n_launch;
    return cudaGetLastError();
}

cudaError_t launch_merge(float *x, const float *snap, const float *mean, int K, int64_t P,
                         __nv_bfloat16 *shadow, cudaStream_t s, int *n_launch)
{
    using namespace cocod;
    if ((P % 8) == 0 && aligned32(x) && aligned32(snap) && aligned32(mean) && K <= 8 * 65535 &&
        (shadow == nullptr || aligned16(shadow))) {
        // rows per thread: as many as K allows up to 8 (registers scale with it)
        const unsigned gx = grid_for(P / 8, kThreads);
        if (K >= 8) merge_vec8<8><<<dim3(gx, (unsigned)((K + 7) / 8)), kThreads, 0, s>>>(x, snap, mean, K, P, shadow, g_stamp, g_backwards);
        else if (K >= 4) merge_vec8<4><<<dim3(gx, (unsigned)((K + 3) / 4)), kThreads, 0, s>>>(x, snap, mean, K, P, shadow, g_stamp, g_backwards);
        else if (K >= 2) merge_vec8<2><<<dim3(gx, (unsigned)((K + 1) / 2)), kThreads, 0, s>>>(x, snap, mean, K, P, shadow, g_stamp, g_backwards);
        else merge_vec8<1><<<dim3(gx, 1), kThreads, 0, s>>>(x, snap, mean, K, P, shadow, g_stamp, g_backwards);
    } else if ((P % 4) == 0 && aligned16(x) && aligned16(snap) && aligned16(mean) &&
               (shadow == nullptr || (reinterpret_cast<uintptr_t>(shadow) & 7u) == 0)) {
        const int64_t pvec = P / 4;
        merge_vec4<4><<<grid_for(pvec, kThreads), kThreads, 0, s>>>(
            reinterpret_cast<float4 *>(x), reinterpret_cast<const float4 *>(snap),
            reinterpret_cast<const float4 *>(mean), K, pvec, shadow, g_stamp);
    } else {
        merge_scalar<<<grid_for(P, kThreads), kThreads, 0, s>>>(x, snap, mean, K, P, shadow);
    }
    if (n_launch) ++*n_launch;
    return cudaGetLastError();
}

// The fused last step + merge needs 8 columns per thread everywhere: returns false (nothing launched) when P or an
// alignment does not allow it; the caller then runs the local step and the merge one after the other (same values).
bool launch_step_merge(const float *x_in, float *x_out, float *v, const float *g, const float *snap, const float *mean,
                       int K, int64_t P, float lr, float mu, float wd, __nv_bfloat16 *shadow, cudaStream_t s,
                       cudaError_t *err)
{
    using namespace cocod;
    *err = cudaSuccess;
    if ((P % 8) != 0 || !aligned32(x_in) || !aligned32(x_out) || !aligned32(v) || !aligned32(g) || !aligned32(snap) ||
        !aligned32(mean) || K > 4 * 65535 || (shadow != nullptr && !aligned16(shadow)))
        return false;
    const unsigned gx = grid_for(P / 8, kThreads);
    if (K >= 4)                       // (four rows per thread: 0.673 ms on the ResNet18-sized workload, two rows: 0.698 ms)
        step_merge_vec8<4><<<dim3(gx, (unsigned)((K + 3) / 4)), kThreads, 0, s>>>(x_in, x_out, v, g, snap, mean, K, P, lr, mu, wd,
                                                                                shadow, g_stamp, g_backwards);
    else if (K >= 2)
        step_merge_vec8<2><<<dim3(gx, (unsigned)((K + 1) / 2)), kThreads, 0, s>>>(x_in, x_out, v, g, snap, mean, K, P, lr, mu, wd,
                                                                                shadow, g_stamp, g_backwards);
    else
        step_merge_vec8<1><<<dim3(gx, 1), kThreads, 0, s>>>(x_in, x_out, v, g, snap, mean, K, P, lr, mu, wd, shadow, g_stamp,
                                                          g_backwards);
    *err = cudaGetLastError();
    return true;
}

// ---------------------------------------------------------------- profiling brackets
struct Bracket {
    cocod_engine *h;
    cudaStream_t s;
    int kind;
    cudaEvent_t a = nullptr, b = nullptr;
    bool on = false;
    Bracket(cocod_engine *h_, cudaStream_t s_, int kind_) : h(h_), s(s_), kind(kind_)
    {
        if (!h->profile || (int)h->prof.size() >= kMaxProfile) return;
        if (cudaEventCreate(&a) != cudaSuccess) { a = nullptr; return; }
        if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); a = b = nullptr; return; }
        on = true;
        if (h->stamps) g_stamp = h->stamps + 2 * h->prof.size();      // this record's slot
        cudaEventRecord(a, s);
    }
    void cancel()                       // nothing was launched inside this bracket: keep no record
    {
        g_stamp = nullptr;
        if (!on) return;
        cudaEventDestroy(a);
        cudaEventDestroy(b);
        on = false;
    }
    ~Bracket()
    {
        g_stamp = nullptr;
        if (!on) return;
        cudaEventRecord(b, s);
        h->prof.push_back({kind, a, b});
    }
};

// start = all ones (atomicMin), end = 0 (atomicMax); the engine is idle when this is called
cudaError_t stamps_reset(cocod_engine *h)
{
    if (!h->stamps) return cudaSuccess;
    std::vector<unsigned long long> init(2 * (size_t)kMaxProfile);
    for (size_t i = 0; i < init.size(); i += 2) { init[i] = ~0ull; init[i + 1] = 0ull; }
    return cudaMemcpy(h->stamps, init.data(), init.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice);
}

void profile_clear(cocod_engine *h)
{
    for (auto &r : h->prof) {
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    h->prof.clear();
    h->stamps_host.clear();
    stamps_reset(h);
}

int check_live(const cocod_engine *h)
{
    if (!h) return COCOD_ERR_INVALID;
    if (h->cuda_error) return COCOD_ERR_CUDA;
    return COCOD_OK;
}

// Weights and scale of Step I's kernel: the whole mean, or this GPU's part of it with the global weights.
inline const float *mean_weights(const cocod_engine *h)
{
    if (h->K_global > 0) return h->wg ? h->wg + h->first : nullptr;
    return h->weighted ? h->w : nullptr;
}
inline float mean_scale(const cocod_engine *h)
{
    return 1.0f / (float)(h->K_global > 0 ? h->K_global : h->K);
}

void detach_peers(cocod_engine *h)
{
    for (int q = 0; q < kMaxRanks; ++q)
        for (int b = 0; b < 3; ++b)
            if (h->opened[q][b]) { cudaIpcCloseMemHandle(h->opened[q][b]); h->opened[q][b] = nullptr; }
    for (int b = 0; b < 2; ++b)
        if (h->rows_tab[b]) { cudaFree((void *)h->rows_tab[b]); h->rows_tab[b] = nullptr; }
    if (h->outs_tab) { cudaFree((void *)h->outs_tab); h->outs_tab = nullptr; }
    h->G = 0;
    h->rank = 0;
    cudaGetLastError();
}

void free_all(cocod_engine *h)
{
    profile_clear(h);
    if (h->stamps) { cudaFree(h->stamps); h->stamps = nullptr; }
    detach_peers(h);
    if (h->wg) cudaFree(h->wg);
    for (int i = 0; i < 2; ++i) if (h->buf[i]) cudaFree(h->buf[i]);
    if (h->v) cudaFree(h->v);
    if (h->mean) cudaFree(h->mean);
    if (h->w) cudaFree(h->w);
    if (h->shadow) cudaFree(h->shadow);
    for (int i = 0; i < kHostSlots; ++i) {
        if (h->stage[i]) cudaFree(h->stage[i]);
        if (h->ev_copied[i]) cudaEventDestroy(h->ev_copied[i]);
        if (h->ev_consumed[i]) cudaEventDestroy(h->ev_consumed[i]);
    }
    if (h->ev_snap) cudaEventDestroy(h->ev_snap);
    if (h->ev_mean) cudaEventDestroy(h->ev_mean);
    if (h->ev_tmp) cudaEventDestroy(h->ev_tmp);
    if (h->copy) cudaStreamDestroy(h->copy);
    delete h;
}

// copy `bytes` into a device buffer from host or device memory, ordered on the compute stream
int copy_in(cocod_engine *h, float *dst, const float *src, size_t bytes, int on_host)
{
    if (on_host) {
        CK(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, h->compute));
        CK(h, cudaStreamSynchronize(h->compute));
    } else {
        CK(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, h->compute));
    }
    return COCOD_OK;
}

int copy_out(cocod_engine *h, float *dst, const float *src, size_t bytes, int on_host)
{
    if (on_host) {
        CK(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, h->compute));
        CK(h, cudaStreamSynchronize(h->compute));
    } else {
        CK(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, h->compute));
    }
    return COCOD_OK;
}

// Recompute the bf16 shadow from x (after x was set from outside).
int refresh_shadow(cocod_engine *h)
{
    if (!h->shadow) return COCOD_OK;
    const unsigned grid = (unsigned)std::min<int64_t>((h->n + cocod::kThreads - 1) / cocod::kThreads, 148 * 16);
    cocod::shadow_refresh<<<grid, cocod::kThreads, 0, h->compute>>>(h->buf[h->cur], h->shadow, h->n);
    CK(h, cudaGetLastError());
    ++h->launches;
    return COCOD_OK;
}

// One local step over elements [off, off + len) with gradients at g (already offset).
int step_range(cocod_engine *h, const float *g, int64_t off, int64_t len)
{
    const float *x_in = h->buf[h->cur] + off;
    float *x_out = (h->pending_flip ? h->buf[1 - h->cur] : h->buf[h->cur]) + off;
    int nl = 0;
    {
        Bracket br(h, h->compute, COCOD_KERNEL_LOCAL_STEP);
        if (h->sweep && off == 0) h->dir ^= 1;
        g_backwards = h->sweep ? h->dir : 0;
        const cudaError_t e = launch_local_step(x_in, x_out, h->v + off, g, len, h->lr, h->mu, h->wd,
                                                h->shadow ? h->shadow + off : nullptr, h->compute, &nl);
        g_backwards = 0;
        CK(h, e);
    }
    h->launches += nl;
    return COCOD_OK;
}

// The side stream's work so far completes the average buffer.
int mark_mean_complete(cocod_engine *h)
{
    CK(h, cudaEventRecord(h->ev_mean, h->side));
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CK(h, cudaStreamIsCapturing(h->side, &cap));
    h->mean_captured = (cap != cudaStreamCaptureStatusNone);      // a captured event cannot be waited on later
    h->mean_valid = true;
    return COCOD_OK;
}

void finish_step(cocod_engine *h)
{
    if (h->pending_flip) {      // x now lives in the other buffer; the old one stays as stored copy
        h->cur = 1 - h->cur;
        h->pending_flip = false;
    }
    ++h->steps;
}

}  // namespace

extern "C" {

int cocod_create(cocod_handle **out, int K, int64_t P, float lr, float mu, float wd)
{
    if (!out || K < 1 || K > kMaxWorkers || P < 1) return COCOD_ERR_INVALID;
    if (!std::isfinite(lr) || !std::isfinite(mu) || !std::isfinite(wd)) return COCOD_ERR_INVALID;
    if (P > (INT64_MAX / 4) / K) return COCOD_ERR_INVALID;
    cocod_engine *h = new (std::nothrow) cocod_engine();
    if (!h) return COCOD_ERR_OOM;
    h->K = K; h->P = P; h->n = (int64_t)K * P;
    h->lr = lr; h->mu = mu; h->wd = wd;
    if (cudaGetDevice(&h->device) != cudaSuccess) { cudaGetLastError(); delete h; return COCOD_ERR_CUDA; }
    const size_t bytes = (size_t)h->n * sizeof(float);
    cudaError_t e = cudaSuccess;
    auto alloc = [&](float **p, size_t b) { if (e == cudaSuccess) e = cudaMalloc((void **)p, b); };
    alloc(&h->buf[0], bytes);
    alloc(&h->buf[1], bytes);
    alloc(&h->v, bytes);
    alloc(&h->mean, (size_t)P * sizeof(float));
    alloc(&h->w, (size_t)K * sizeof(float));
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_snap, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_mean, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_tmp, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->buf[0], 0, bytes, h->compute);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->v, 0, bytes, h->compute);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->mean, 0, (size_t)P * sizeof(float), h->compute);
    if (e != cudaSuccess) {
        const int rc = (e == cudaErrorMemoryAllocation) ? COCOD_ERR_OOM : COCOD_ERR_CUDA;
        cudaGetLastError();
        free_all(h);
        return rc;
    }
    *out = h;
    return COCOD_OK;
}

int cocod_destroy(cocod_handle *h)
{
    if (!h) return COCOD_OK;
    cudaStreamSynchronize(h->compute);
    if (!h->mean_captured) cudaEventSynchronize(h->ev_mean);      // last work on the borrowed side stream
    if (h->copy) cudaStreamSynchronize(h->copy);
    cudaGetLastError();
    const int rc = h->cuda_error ? COCOD_ERR_CUDA : COCOD_OK;
    free_all(h);
    return rc;
}

int cocod_local_step(cocod_handle *h, const float *grads)
{
    if (int rc = check_live(h)) return rc;
    if (!grads) return COCOD_ERR_INVALID;
    if (int rc = step_range(h, grads, 0, h->n)) return rc;
    finish_step(h);
    return COCOD_OK;
}

int cocod_local_step_host(cocod_handle *h, const float *host_grads)
{
    if (int rc = check_live(h)) return rc;
    if (!host_grads) return COCOD_ERR_INVALID;
    if (!h->host_ready) {           // first use: all or nothing, so a failed attempt can be retried
        const int64_t cap = std::min<int64_t>(kHostChunk, h->n);
        cudaError_t e = h->copy ? cudaSuccess : cudaStreamCreateWithFlags(&h->copy, cudaStreamNonBlocking);
        for (int i = 0; i < kHostSlots && e == cudaSuccess; ++i) {
            if (!h->stage[i]) e = cudaMalloc((void **)&h->stage[i], (size_t)cap * sizeof(float));
            if (e == cudaSuccess && !h->ev_copied[i]) e = cudaEventCreateWithFlags(&h->ev_copied[i], cudaEventDisableTiming);
            if (e == cudaSuccess && !h->ev_consumed[i]) e = cudaEventCreateWithFlags(&h->ev_consumed[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) {
            cudaGetLastError();
            for (int i = 0; i < kHostSlots; ++i)
                if (h->stage[i]) { cudaFree(h->stage[i]); h->stage[i] = nullptr; }
            return e == cudaErrorMemoryAllocation ? COCOD_ERR_OOM : COCOD_ERR_CUDA;
        }
        h->host_ready = true;
    }
    int slot = 0;
    for (int64_t off = 0; off < h->n; off += kHostChunk, slot = (slot + 1) % kHostSlots) {
        const int64_t len = std::min<int64_t>(kHostChunk, h->n - off);
        if (h->slot_used[slot]) CK(h, cudaStreamWaitEvent(h->copy, h->ev_consumed[slot], 0));
        CK(h, cudaMemcpyAsync(h->stage[slot], host_grads + off, (size_t)len * sizeof(float),
                              cudaMemcpyHostToDevice, h->copy));
        CK(h, cudaEventRecord(h->ev_copied[slot], h->copy));
        CK(h, cudaStreamWaitEvent(h->compute, h->ev_copied[slot], 0));
        if (int rc = step_range(h, h->stage[slot], off, len)) return rc;
        CK(h, cudaEventRecord(h->ev_consumed[slot], h->compute));
        h->slot_used[slot] = true;
    }
    finish_step(h);
    return COCOD_OK;
}

int cocod_comm_begin(cocod_handle *h, cocod_stream_t side)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    h->side = (cudaStream_t)side;
    if (h->snapshot_mode == COCOD_SNAPSHOT_FLIP) {
        h->snap = h->buf[h->cur];
        h->pending_flip = true;
    } else {
        float *dst = h->buf[1 - h->cur];
        int nl = 0;
        {
            Bracket br(h, h->compute, COCOD_KERNEL_SNAPSHOT);
            CK(h, launch_snapshot(h->buf[h->cur], dst, h->n, h->compute, &nl));
        }
        h->launches += nl;
        h->snap = dst;
        h->pending_flip = false;
    }
    if (h->side != h->compute) {
        CK(h, cudaEventRecord(h->ev_snap, h->compute));
        CK(h, cudaStreamWaitEvent(h->side, h->ev_snap, 0));
    }
    h->mean_started = false;
    h->exchanged = false;
    if (h->G > 0) {                 // gather form: the caller queues a barrier, then cocod_comm_gather
        h->mean_valid = false;
        h->state = IN_FLIGHT;
        return COCOD_OK;
    }
    int nl = 0;
    {
        Bracket br(h, h->side, COCOD_KERNEL_MEAN);
        g_backwards = h->sweep ? (h->dir ^ 1) : 0;       // against the kernel that last wrote x
        const cudaError_t e = launch_mean(h->snap, h->K, h->P, mean_weights(h), h->mean, mean_scale(h), h->side, &nl);
        g_backwards = 0;
        CK(h, e);
    }
    h->launches += nl;
    h->mean_started = true;
    h->state = IN_FLIGHT;
    if (h->K_global > 0) {          // partial sum: complete only after the caller's all-reduce
        h->mean_valid = false;
        return COCOD_OK;
    }
    return mark_mean_complete(h);
}

int cocod_comm_gather(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IN_FLIGHT || h->G == 0 || h->mean_started) return COCOD_ERR_STATE;
    // this GPU's share of the columns, in units of 8, 4 or 1 columns as the rows' alignment allows
    const int vec = (h->P % 8) == 0 ? 8 : (h->P % 4) == 0 ? 4 : 1;
    const int64_t units = h->P / vec;
    const int64_t base = units / h->G, rem = units % h->G;
    const int64_t lo = h->rank * base + std::min<int64_t>(h->rank, rem);
    const int64_t hi = lo + base + (h->rank < rem ? 1 : 0);
    const int b = (h->snap == h->buf[0]) ? 0 : 1;
    int nl = 0;
    {
        Bracket br(h, h->side, COCOD_KERNEL_MEAN);
        CK(h, launch_mean_gather(h->rows_tab[b], h->K_global, lo * vec, hi * vec, h->wg, h->outs_tab, h->G,
                                 mean_scale(h), vec, h->side, &nl));
    }
    h->launches += nl;
    h->mean_started = true;
    return COCOD_OK;
}

int cocod_comm_exchanged(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IN_FLIGHT || h->K_global == 0 || !h->mean_started || h->exchanged) return COCOD_ERR_STATE;
    h->exchanged = true;
    return mark_mean_complete(h);
}

int cocod_comm_end(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IN_FLIGHT) return COCOD_ERR_STATE;
    if (h->K_global > 0 && !h->exchanged) return COCOD_ERR_STATE;      // the mean over the GPUs is not complete
    if (h->side != h->compute) CK(h, cudaStreamWaitEvent(h->compute, h->ev_mean, 0));
    int nl = 0;
    {
        Bracket br(h, h->compute, COCOD_KERNEL_MERGE);
        // with no local step since comm_begin (FLIP) x still aliases the stored copies
        if (h->sweep) h->dir ^= 1;
        g_backwards = h->sweep ? h->dir : 0;
        const cudaError_t e = launch_merge(h->buf[h->cur], h->snap, h->mean, h->K, h->P, h->shadow, h->compute, &nl);
        g_backwards = 0;
        CK(h, e);
    }
    h->launches += nl;
    h->pending_flip = false;
    h->snap = nullptr;
    h->state = IDLE;
    return COCOD_OK;
}

int cocod_local_step_end(cocod_handle *h, const float *grads)
{
    if (int rc = check_live(h)) return rc;
    if (!grads) return COCOD_ERR_INVALID;
    if (h->state != IN_FLIGHT) return COCOD_ERR_STATE;
    if (h->K_global > 0 && !h->exchanged) return COCOD_ERR_STATE;      // the mean over the GPUs is not complete
    if (h->side != h->compute) CK(h, cudaStreamWaitEvent(h->compute, h->ev_mean, 0));
    const float *x_in = h->buf[h->cur];
    float *x_out = h->pending_flip ? h->buf[1 - h->cur] : h->buf[h->cur];
    bool fused = false;
    {
        Bracket br(h, h->compute, COCOD_KERNEL_STEP_MERGE);
        if (h->sweep) h->dir ^= 1;
        g_backwards = h->sweep ? h->dir : 0;
        cudaError_t e = cudaSuccess;
        fused = launch_step_merge(x_in, x_out, h->v, grads, h->snap, h->mean, h->K, h->P, h->lr, h->mu, h->wd, h->shadow,
                                  h->compute, &e);
        g_backwards = 0;
        if (!fused) br.cancel();
        CK(h, e);
    }
    if (!fused) {                    // shapes the fused kernel does not take: the two kernels, one after the other
        if (int rc = cocod_local_step(h, grads)) return rc;
        return cocod_comm_end(h);
    }
    ++h->launches;
    finish_step(h);
    h->pending_flip = false;
    h->snap = nullptr;
    h->state = IDLE;
    return COCOD_OK;
}

int cocod_local_sgd_average(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE || h->K_global > 0) return COCOD_ERR_STATE;
    int nl = 0;
    {
        Bracket br(h, h->compute, COCOD_KERNEL_MEAN);
        CK(h, launch_mean(h->buf[h->cur], h->K, h->P, h->weighted ? h->w : nullptr, h->mean, 1.0f / (float)h->K,
                          h->compute, &nl));
    }
    // after the sequential mean nothing from the side stream is pending for this value
    CK(h, cudaEventRecord(h->ev_mean, h->compute));
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CK(h, cudaStreamIsCapturing(h->compute, &cap));
    h->mean_captured = (cap != cudaStreamCaptureStatusNone);
    h->side = h->compute;
    h->mean_valid = true;
    cocod::broadcast_rows<<<grid_for(h->P, cocod::kThreads), cocod::kThreads, 0, h->compute>>>(
        h->mean, h->buf[h->cur], h->K, h->P);
    CK(h, cudaGetLastError());
    h->launches += nl + 1;
    return refresh_shadow(h);
}

int cocod_ssgd_step(cocod_handle *h, const float *grads)
{
    if (int rc = check_live(h)) return rc;
    if (!grads) return COCOD_ERR_INVALID;
    if (h->state != IDLE || h->K_global > 0) return COCOD_ERR_STATE;   // the average buffer holds the averaged gradient
    using namespace cocod;
    int nl = 0;
    {
        Bracket br(h, h->compute, COCOD_KERNEL_MEAN);
        CK(h, launch_mean(grads, h->K, h->P, h->weighted ? h->w : nullptr, h->mean, 1.0f / (float)h->K, h->compute,
                          &nl));
    }
    h->mean_valid = false;                              // it is a gradient now, not an average model
    float *x = h->buf[h->cur];
    {
        Bracket br(h, h->compute, COCOD_KERNEL_LOCAL_STEP);
        if ((h->P % 4) == 0 && (h->shadow == nullptr || (reinterpret_cast<uintptr_t>(h->shadow) & 7u) == 0)) {
            const int64_t pvec = h->P / 4;
            local_step_shared_grad_vec4<<<dim3(grid_for(pvec, kThreads), (unsigned)h->K), kThreads, 0, h->compute>>>(
                reinterpret_cast<const float4 *>(x), reinterpret_cast<float4 *>(x), reinterpret_cast<float4 *>(h->v),
                reinterpret_cast<const float4 *>(h->mean), pvec, h->lr, h->mu, h->wd, h->shadow);
        } else {
            local_step_shared_grad_scalar<<<dim3(grid_for(h->P, kThreads), (unsigned)h->K), kThreads, 0, h->compute>>>(
                x, x, h->v, h->mean, h->P, h->lr, h->mu, h->wd, h->shadow);
        }
        CK(h, cudaGetLastError());
    }
    h->launches += nl + 1;
    ++h->steps;
    return COCOD_OK;
}

int cocod_set_stream(cocod_handle *h, cocod_stream_t compute)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    cudaStream_t s = (cudaStream_t)compute;
    if (s != h->compute) {      // later work on the new stream stays ordered after earlier work
        CK(h, cudaEventRecord(h->ev_tmp, h->compute));
        CK(h, cudaStreamWaitEvent(s, h->ev_tmp, 0));
        h->compute = s;
    }
    return COCOD_OK;
}

int cocod_set_params(cocod_handle *h, const float *x0, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!x0) return COCOD_ERR_INVALID;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    const float *src = x0;
    if (on_host) {      // stage through the (idle) average-model buffer
        if (int rc = copy_in(h, h->mean, x0, (size_t)h->P * sizeof(float), 1)) return rc;
        src = h->mean;
        h->mean_valid = false;
    }
    cocod::broadcast_rows<<<grid_for(h->P, cocod::kThreads), cocod::kThreads, 0, h->compute>>>(
        src, h->buf[h->cur], h->K, h->P);
    CK(h, cudaGetLastError());
    ++h->launches;
    return refresh_shadow(h);
}

int cocod_set_params_all(cocod_handle *h, const float *x, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!x) return COCOD_ERR_INVALID;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    if (int rc = copy_in(h, h->buf[h->cur], x, (size_t)h->n * sizeof(float), on_host)) return rc;
    return refresh_shadow(h);
}

int cocod_set_momentum(cocod_handle *h, const float *v, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!v) return COCOD_ERR_INVALID;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    return copy_in(h, h->v, v, (size_t)h->n * sizeof(float), on_host);
}

int cocod_get_params(cocod_handle *h, float *out, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    return copy_out(h, out, h->buf[h->cur], (size_t)h->n * sizeof(float), on_host);
}

int cocod_get_momentum(cocod_handle *h, float *out, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    return copy_out(h, out, h->v, (size_t)h->n * sizeof(float), on_host);
}

int cocod_get_mean(cocod_handle *h, float *out, int on_host)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    if (!h->mean_valid) return COCOD_ERR_STATE;
    if (h->side != h->compute) CK(h, cudaStreamWaitEvent(h->compute, h->ev_mean, 0));
    return copy_out(h, out, h->mean, (size_t)h->P * sizeof(float), on_host);
}

int cocod_set_lr(cocod_handle *h, float lr)
{
    if (int rc = check_live(h)) return rc;
    if (!std::isfinite(lr)) return COCOD_ERR_INVALID;
    h->lr = lr;
    return COCOD_OK;
}

int cocod_set_batch_sizes(cocod_handle *h, const double *M)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE || h->K_global > 0) return COCOD_ERR_STATE;      // sharded: cocod_set_shard carries them
    if (!M) { h->weighted = false; return COCOD_OK; }
    double sum = 0.0;
    for (int i = 0; i < h->K; ++i) {
        if (!(M[i] > 0.0) || !std::isfinite(M[i])) return COCOD_ERR_INVALID;
        sum += M[i];
    }
    float w[kMaxWorkers];
    for (int i = 0; i < h->K; ++i) w[i] = (float)(M[i] / sum);
    CK(h, cudaMemcpyAsync(h->w, w, (size_t)h->K * sizeof(float), cudaMemcpyHostToDevice, h->compute));
    CK(h, cudaStreamSynchronize(h->compute));      // w[] is a stack buffer
    h->weighted = true;
    return COCOD_OK;
}

int cocod_set_option(cocod_handle *h, int option, int value)
{
    if (int rc = check_live(h)) return rc;
    switch (option) {
    case COCOD_OPT_SNAPSHOT:
        if (value != COCOD_SNAPSHOT_COPY && value != COCOD_SNAPSHOT_FLIP) return COCOD_ERR_INVALID;
        if (h->state != IDLE) return COCOD_ERR_STATE;
        h->snapshot_mode = value;
        return COCOD_OK;
    case COCOD_OPT_SWEEP:
        h->sweep = value != 0;
        h->dir = 0;
        return COCOD_OK;
    case COCOD_OPT_PROFILE:
        if (value && !h->stamps) {      // device-side time stamps: 256 KB, kept until the handle is destroyed
            if (cudaMalloc((void **)&h->stamps, 2 * (size_t)kMaxProfile * sizeof(unsigned long long)) != cudaSuccess) {
                cudaGetLastError();
                h->stamps = nullptr;
                return COCOD_ERR_OOM;
            }
            CK(h, cudaDeviceSynchronize());
            CK(h, stamps_reset(h));
        }
        h->profile = value != 0;
        return COCOD_OK;
    case COCOD_OPT_BF16_SHADOW:
        if (h->state != IDLE) return COCOD_ERR_STATE;
        if (value && !h->shadow) {
            cudaError_t e = cudaMalloc((void **)&h->shadow, (size_t)h->n * sizeof(__nv_bfloat16));
            if (e != cudaSuccess) { cudaGetLastError(); h->shadow = nullptr; return COCOD_ERR_OOM; }
            return refresh_shadow(h);
        }
        if (!value && h->shadow) {
            CK(h, cudaStreamSynchronize(h->compute));
            cudaFree(h->shadow);
            h->shadow = nullptr;
        }
        return COCOD_OK;
    default:
        return COCOD_ERR_INVALID;
    }
}

int cocod_sync(cocod_handle *h)
{
    if (!h) return COCOD_ERR_INVALID;
    fail(h, cudaStreamSynchronize(h->compute));
    if (!h->mean_captured) fail(h, cudaEventSynchronize(h->ev_mean));      // side-stream work (no-op if never recorded)
    if (h->copy) fail(h, cudaStreamSynchronize(h->copy));
    return h->cuda_error ? COCOD_ERR_CUDA : COCOD_OK;
}

int cocod_comm_wait(cocod_handle *h, int timeout_ms)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IN_FLIGHT || (h->K_global > 0 && !h->exchanged)) return COCOD_ERR_STATE;
    const auto t0 = std::chrono::steady_clock::now();
    for (;;) {
        cudaError_t e = cudaEventQuery(h->ev_mean);
        if (e == cudaSuccess) return COCOD_OK;
        if (e != cudaErrorNotReady) { fail(h, e); return COCOD_ERR_CUDA; }
        cudaGetLastError();
        const auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(
                            std::chrono::steady_clock::now() - t0).count();
        if (ms >= timeout_ms) return COCOD_ERR_TIMEOUT;
        std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}

int cocod_get_bf16_shadow(cocod_handle *h, void **out)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    if (!h->shadow) return COCOD_ERR_STATE;
    *out = h->shadow;
    return COCOD_OK;
}

int64_t cocod_step_count(const cocod_handle *h) { return h ? h->steps : -1; }

int cocod_last_cuda_error(const cocod_handle *h) { return h ? h->cuda_error : 0; }

int64_t cocod_launch_count(const cocod_handle *h) { return h ? h->launches : -1; }

const char *cocod_strerror(int code)
{
    switch (code) {
    case COCOD_OK: return "ok";
    case COCOD_ERR_INVALID: return "invalid argument";
    case COCOD_ERR_OOM: return "out of memory";
    case COCOD_ERR_STATE: return "call not legal in the engine's current state";
    case COCOD_ERR_CUDA: return "CUDA error";
    case COCOD_ERR_TIMEOUT: return "timed out";
    case COCOD_ERR_TOO_LARGE: return "request exceeds the fixed capacity of this entry point";
    default: return "unknown error code";
    }
}

int cocod_profile_reset(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (int rc = cocod_sync(h)) return rc;
    profile_clear(h);
    return COCOD_OK;
}

int cocod_profile_count(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (int rc = cocod_sync(h)) return rc;
    if (h->stamps && !h->prof.empty()) {
        h->stamps_host.resize(2 * h->prof.size());
        CK(h, cudaMemcpy(h->stamps_host.data(), h->stamps, h->stamps_host.size() * sizeof(unsigned long long),
                         cudaMemcpyDeviceToHost));
    }
    return (int)h->prof.size();
}

int cocod_profile_get_device_ns(cocod_handle *h, int i, uint64_t *start_ns, uint64_t *end_ns)
{
    if (int rc = check_live(h)) return rc;
    if (i < 0 || i >= (int)h->prof.size() || !start_ns || !end_ns) return COCOD_ERR_INVALID;
    if (2 * (size_t)i + 1 >= h->stamps_host.size()) return COCOD_ERR_STATE;      // cocod_profile_count first
    const unsigned long long a = h->stamps_host[2 * i], b = h->stamps_host[2 * i + 1];
    const bool have = (a != ~0ull) && (b != 0ull);
    *start_ns = have ? (uint64_t)a : 0;
    *end_ns = have ? (uint64_t)b : 0;
    return COCOD_OK;
}

int cocod_profile_get(cocod_handle *h, int i, int *kind, float *start_ms, float *end_ms)
{
    if (int rc = check_live(h)) return rc;
    if (i < 0 || i >= (int)h->prof.size() || !kind || !start_ms || !end_ms) return COCOD_ERR_INVALID;
    const ProfileRec &r = h->prof[i];
    *kind = r.kind;
    CK(h, cudaEventElapsedTime(start_ms, h->prof[0].a, r.a));
    CK(h, cudaEventElapsedTime(end_ms, h->prof[0].a, r.b));
    return COCOD_OK;
}

// ------------------------------------------------------------------ workers spread over several GPUs
int cocod_set_shard(cocod_handle *h, int K_global, int first, const double *M_global)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE || h->G > 0) return COCOD_ERR_STATE;
    if (K_global == 0) {
        h->K_global = 0; h->first = 0;
        if (h->wg) { CK(h, cudaStreamSynchronize(h->compute)); cudaFree(h->wg); h->wg = nullptr; }
        return COCOD_OK;
    }
    if (K_global < h->K || K_global > kMaxWorkers || first < 0 || first > K_global - h->K) return COCOD_ERR_INVALID;
    float *wg = nullptr;
    if (M_global) {
        double sum = 0.0;
        for (int i = 0; i < K_global; ++i) {
            if (!(M_global[i] > 0.0) || !std::isfinite(M_global[i])) return COCOD_ERR_INVALID;
            sum += M_global[i];
        }
        float w[kMaxWorkers];
        for (int i = 0; i < K_global; ++i) w[i] = (float)(M_global[i] / sum);
        if (cudaMalloc((void **)&wg, (size_t)K_global * sizeof(float)) != cudaSuccess) {
            cudaGetLastError();
            return COCOD_ERR_OOM;
        }
        cudaError_t e = cudaMemcpyAsync(wg, w, (size_t)K_global * sizeof(float), cudaMemcpyHostToDevice, h->compute);
        if (e == cudaSuccess) e = cudaStreamSynchronize(h->compute);      // w[] is a stack buffer
        if (e != cudaSuccess) { cudaFree(wg); fail(h, e); return COCOD_ERR_CUDA; }
    }
    if (h->wg) { CK(h, cudaStreamSynchronize(h->compute)); cudaFree(h->wg); }
    h->wg = wg;
    h->K_global = K_global;
    h->first = first;
    return COCOD_OK;
}

int cocod_mean_buffer(cocod_handle *h, float **out)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    *out = h->mean;
    return COCOD_OK;
}

namespace {
// What one process tells the others about its engine (COCOD_IPC_EXPORT_BYTES bytes on the wire).
struct IpcBlob {
    uint32_t magic;
    int32_t K, first, K_global, cur, pid;
    int64_t P;
    uint64_t ptr[3];                    // buf[0], buf[1], average buffer: usable as they are inside process `pid`
    cudaIpcMemHandle_t mem[3];          // the same three for other processes
};
static_assert(sizeof(IpcBlob) <= COCOD_IPC_EXPORT_BYTES, "export blob too large");
constexpr uint32_t kIpcMagic = 0xC0C0D5D1u;
}  // namespace

int cocod_ipc_export(cocod_handle *h, void *out)
{
    if (int rc = check_live(h)) return rc;
    if (!out) return COCOD_ERR_INVALID;
    if (h->K_global == 0) return COCOD_ERR_STATE;
    IpcBlob b{};
    b.magic = kIpcMagic;
    b.K = h->K; b.first = h->first; b.K_global = h->K_global; b.cur = h->cur; b.pid = (int32_t)getpid();
    b.P = h->P;
    float *ptrs[3] = {h->buf[0], h->buf[1], h->mean};
    for (int i = 0; i < 3; ++i) {
        b.ptr[i] = (uint64_t)reinterpret_cast<uintptr_t>(ptrs[i]);
        CK(h, cudaIpcGetMemHandle(&b.mem[i], ptrs[i]));
    }
    std::memset(out, 0, COCOD_IPC_EXPORT_BYTES);
    std::memcpy(out, &b, sizeof(b));
    return COCOD_OK;
}

int cocod_ipc_attach(cocod_handle *h, int G, int rank, const void *blobs)
{
    if (int rc = check_live(h)) return rc;
    if (!blobs || G < 1 || G > kMaxRanks || rank < 0 || rank >= G) return COCOD_ERR_INVALID;
    if (h->state != IDLE || h->K_global == 0 || h->G > 0) return COCOD_ERR_STATE;
    std::vector<IpcBlob> all((size_t)G);
    int next = 0;
    for (int q = 0; q < G; ++q) {
        std::memcpy(&all[q], (const unsigned char *)blobs + (size_t)q * COCOD_IPC_EXPORT_BYTES, sizeof(IpcBlob));
        const IpcBlob &b = all[q];
        if (b.magic != kIpcMagic || b.P != h->P || b.K_global != h->K_global || b.K < 1 || b.first != next ||
            b.cur != h->cur)
            return COCOD_ERR_INVALID;
        next += b.K;
    }
    if (next != h->K_global || all[rank].K != h->K || all[rank].first != h->first ||
        all[rank].ptr[0] != (uint64_t)reinterpret_cast<uintptr_t>(h->buf[0]) || all[rank].pid != (int32_t)getpid())
        return COCOD_ERR_INVALID;
    // addresses of every process's three buffers as seen from here
    std::vector<float *> base((size_t)G * 3, nullptr);
    for (int q = 0; q < G; ++q)
        for (int i = 0; i < 3; ++i) {
            if (all[q].pid == (int32_t)getpid()) {      // same process (also this engine itself): same address space
                base[(size_t)q * 3 + i] = reinterpret_cast<float *>((uintptr_t)all[q].ptr[i]);
                continue;
            }
            void *p = nullptr;
            cudaError_t e = cudaIpcOpenMemHandle(&p, all[q].mem[i], cudaIpcMemLazyEnablePeerAccess);
            if (e != cudaSuccess) { fail(h, e); cudaGetLastError(); detach_peers(h); return COCOD_ERR_CUDA; }
            h->opened[q][i] = p;
            base[(size_t)q * 3 + i] = static_cast<float *>(p);
        }
    std::vector<const float *> rows[2];
    std::vector<float *> outs((size_t)G);
    for (int b = 0; b < 2; ++b) rows[b].resize((size_t)h->K_global);
    for (int q = 0; q < G; ++q) {
        for (int r = 0; r < all[q].K; ++r)
            for (int b = 0; b < 2; ++b) rows[b][(size_t)all[q].first + r] = base[(size_t)q * 3 + b] + (int64_t)r * h->P;
        outs[q] = base[(size_t)q * 3 + 2];
    }
    cudaError_t e = cudaSuccess;
    for (int b = 0; b < 2 && e == cudaSuccess; ++b) {
        e = cudaMalloc((void **)&h->rows_tab[b], (size_t)h->K_global * sizeof(float *));
        if (e == cudaSuccess)
            e = cudaMemcpy((void *)h->rows_tab[b], rows[b].data(), (size_t)h->K_global * sizeof(float *),
                           cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMalloc((void **)&h->outs_tab, (size_t)G * sizeof(float *));
    if (e == cudaSuccess) e = cudaMemcpy((void *)h->outs_tab, outs.data(), (size_t)G * sizeof(float *), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        const bool oom = (e == cudaErrorMemoryAllocation);
        cudaGetLastError();
        detach_peers(h);
        if (oom) return COCOD_ERR_OOM;
        fail(h, e);
        return COCOD_ERR_CUDA;
    }
    h->G = G;
    h->rank = rank;
    return COCOD_OK;
}

int cocod_ipc_detach(cocod_handle *h)
{
    if (int rc = check_live(h)) return rc;
    if (h->state != IDLE) return COCOD_ERR_STATE;
    // peers may still be reading this GPU's buffers only until their own side streams are done; what
    // this engine itself queued must be done before its mappings go away
    CK(h, cudaStreamSynchronize(h->compute));
    if (!h->mean_captured) CK(h, cudaEventSynchronize(h->ev_mean));
    detach_peers(h);
    return COCOD_OK;
}

int cocod_kernel_mean_gather(const float *const *rows, int K, int64_t col_lo, int64_t col_hi, const float *w,
                             float *const *outs, int G, int vec, cocod_stream_t stream)
{
    if (!rows || !outs || K < 1 || G < 1 || col_lo < 0 || col_hi < col_lo) return COCOD_ERR_INVALID;
    if (vec != 1 && vec != 4 && vec != 8) return COCOD_ERR_INVALID;
    if ((col_lo % vec) || (col_hi % vec)) return COCOD_ERR_INVALID;
    return launch_mean_gather(rows, K, col_lo, col_hi, w, outs, G, 1.0f / (float)K, vec, (cudaStream_t)stream,
                              nullptr) == cudaSuccess ? COCOD_OK : COCOD_ERR_CUDA;
}

// ------------------------------------------------------------------ stateless kernel entry points
int cocod_kernel_local_step(const float *x_in, float *x_out, float *v, const float *g, int64_t n,
                            float lr, float mu, float wd, cocod_stream_t stream)
{
    if (!x_in || !x_out || !v || !g || n < 0) return COCOD_ERR_INVALID;
    return launch_local_step(x_in, x_out, v, g, n, lr, mu, wd, nullptr, (cudaStream_t)stream, nullptr) == cudaSuccess
               ? COCOD_OK : COCOD_ERR_CUDA;
}

int cocod_kernel_snapshot(const float *x, float *snap, int64_t n, cocod_stream_t stream)
{
    if (!x || !snap || n < 0) return COCOD_ERR_INVALID;
    return launch_snapshot(x, snap, n, (cudaStream_t)stream, nullptr) == cudaSuccess ? COCOD_OK : COCOD_ERR_CUDA;
}

int cocod_kernel_mean(const float *snap, int K, int64_t P, const float *w, float *mean, cocod_stream_t stream)
{
    if (!snap || !mean || K < 1 || P < 1) return COCOD_ERR_INVALID;
    return launch_mean(snap, K, P, w, mean, 1.0f / (float)K, (cudaStream_t)stream, nullptr) == cudaSuccess
               ? COCOD_OK : COCOD_ERR_CUDA;
}

int cocod_kernel_merge(float *x, const float *snap, const float *mean, int K, int64_t P, cocod_stream_t stream)
{
    if (!x || !snap || !mean || K < 1 || P < 1) return COCOD_ERR_INVALID;
    return launch_merge(x, snap, mean, K, P, nullptr, (cudaStream_t)stream, nullptr) == cudaSuccess ? COCOD_OK
                                                                                                     : COCOD_ERR_CUDA;
}

}  // extern "C"

// ------------------------------------------------------------------ internal interface (cocod_internal.h)
int cocod_internal_plan_step(cocod_handle *h, cocod_step_plan *plan)
{
    if (int rc = check_live(h)) return rc;
    if (!plan) return COCOD_ERR_INVALID;
    plan->x_in = h->buf[h->cur];
    plan->x_out = h->pending_flip ? h->buf[1 - h->cur] : h->buf[h->cur];
    plan->v = h->v;
    plan->shadow = h->shadow;
    plan->lr = h->lr; plan->mu = h->mu; plan->wd = h->wd;
    plan->K = h->K; plan->P = h->P;
    plan->compute = h->compute;
    return COCOD_OK;
}

int cocod_internal_finish_step(cocod_handle *h, int kernels_launched)
{
    if (int rc = check_live(h)) return rc;
    h->launches += kernels_launched;
    finish_step(h);
    return COCOD_OK;
}

// ------------------------------------------------------------------ allocation-free host-gradient step
// Staging for cocod_kernel_local_step_host_noalloc.  In host code the name below is only a
// stand-in for the symbol, not a device address: the address is looked up once per device.
static __device__ __align__(256) float g_noalloc_stage[COCOD_NOALLOC_MAX_ELEMS];

namespace {
constexpr int kMaxDevices = 64;
float *g_noalloc_ptr[kMaxDevices] = {nullptr};
}  // namespace

extern "C" int cocod_kernel_local_step_host_noalloc(const float *x_in, float *x_out, float *v,
                                                    const float *host_grads, int64_t n, float lr, float mu,
                                                    float wd, cocod_stream_t stream)
{
    if (!x_in || !x_out || !v || !host_grads || n < 0) return COCOD_ERR_INVALID;
    if (n > (int64_t)COCOD_NOALLOC_MAX_ELEMS) return COCOD_ERR_TOO_LARGE;
    if (n == 0) return COCOD_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return COCOD_ERR_CUDA;
    if (g_noalloc_ptr[dev] == nullptr) {       // set-up, once per device, that device being current
        float *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_noalloc_stage) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return COCOD_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
    }
    float *stage = g_noalloc_ptr[dev];
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(stage, host_grads, (size_t)n * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess) {
        cudaGetLastError();
        return COCOD_ERR_CUDA;
    }
    return launch_local_step(x_in, x_out, v, stage, n, lr, mu, wd, nullptr, s, nullptr) == cudaSuccess
               ? COCOD_OK : COCOD_ERR_CUDA;
}
