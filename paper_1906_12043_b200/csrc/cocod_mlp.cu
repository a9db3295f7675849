// Per-worker mini-batch gradients of the 3-layer ReLU MLP (the stochastic gradient of Algorithm 1,
// Step II), batched over the K workers.  Declared in include/cocod_mlp.h.
//
// Data flow of one call (every matrix exists once per worker; no matrix is ever transposed in
// memory: the tensor cores read an operand either with the reduction index contiguous or with the
// row index contiguous):
//
//   h1 = bf16(relu(x  W1^T + b1))     GEMM 128 x d_h x d_in   A = x, B = W1            epilogue bias+ReLU
//   h2 = bf16(relu(h1 W2^T + b2))     GEMM 128 x d_h x d_h    A = h1, B = W2           epilogue bias+ReLU
//   logits = h2 W3^T + b3 (per-tile partial sums from the epilogue of the GEMM above) ;
//   loss ; dz3 = bf16((softmax - onehot)/batch)                                       CUDA cores
//   dz2 = bf16((dz3 W3) * (h2 > 0)) ; dW3 = dz3^T h2 ; db3, db2 = column sums           CUDA cores
//   dz1 = bf16((dz2 W2) * (h1 > 0))   GEMM 128 x d_h x d_h    A = dz2, B = W2 read [k][n]  epilogue mask,
//   db1 = column sums of dz1                                   (same epilogue: the batch is one tile)
//   dW2 = dz2^T h1                    GEMM d_h x d_h x 128    A = dz2 read [k][m], B = h1 read [k][n]   one persistent kernel over
//   dW1 = dz1^T x                     GEMM d_h x d_in x 128   A = dz1 read [k][m], B = x  read [k][n]   the tiles of both: fp32
//                                                                                      out, or the local step applied in place
#include "cocod_mlp.h"
#include "cocod_gemm_sm100.cuh"
#include "cocod_gemm_update_sm100.cuh"
#include "cocod_mlp_chain_sm100.cuh"
#include "cocod_internal.h"

#include <algorithm>
#include <cstdio>
#include <new>
#include <utility>
#include <vector>

namespace {

using bf16 = __nv_bfloat16;
using namespace cocod::gemm;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encoder()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// 3-D maps over a batched row-major matrix: dims {cols (contiguous), rows, workers}.  `box_rows` is
// 128 for a K-major operand tile, 64 for an MN-major one; a box is 64 bf16 columns wide (128 bytes,
// the swizzle span).
bool make_map(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t workers, uint64_t ld,
              uint64_t worker_stride, uint32_t box_rows)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    const cuuint64_t dims[3] = {cols, rows, workers};
    const cuuint64_t strides[2] = {ld * sizeof(bf16), worker_stride * sizeof(bf16)};
    const cuuint32_t box[3] = {64, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool map_k(CUtensorMap *m, const void *base, uint64_t k, uint64_t rows, uint64_t workers, uint64_t ld, uint64_t ws)
{
    return make_map(m, base, k, rows, workers, ld, ws, 128);
}
inline bool map_mn(CUtensorMap *m, const void *base, uint64_t mn, uint64_t k, uint64_t workers, uint64_t ld, uint64_t ws)
{
    return make_map(m, base, mn, k, workers, ld, ws, 64);
}
// fp32 output map for the TMA-store epilogue: box = 32 columns (128 bytes) x 128 rows.
bool map_out(CUtensorMap *m, float *base, uint64_t cols, uint64_t rows, uint64_t workers, uint64_t ld,
             uint64_t worker_stride)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || (ld % 4) || (worker_stride % 4)) return false;
    const cuuint64_t dims[3] = {cols, rows, workers};
    const cuuint64_t strides[2] = {ld * sizeof(float), worker_stride * sizeof(float)};
    const cuuint32_t box[3] = {32, 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Facts that belong to a device (function attributes set, SM count, scratch of the stand-alone GEMM call) are
// cached per device, indexed by the current device: one process may drive engines on several GPUs.
constexpr int MAX_DEVICES = 64;
inline int current_device()
{
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= MAX_DEVICES) return -1;
    return d;
}

// Launch with the programmatic-serialization attribute: the kernel may become resident (and run the
// part of its prologue that precedes pdl_wait()) while the previous kernel in the stream drains.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                             Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <int EPI, bool A_MN, bool B_MN>
cudaError_t launch_gemm(const CUtensorMap &a, const CUtensorMap &b, const CUtensorMap &c, const Params &p, int workers,
                        cudaStream_t s, bool pdl = false, const CUtensorMap *next = nullptr)
{
    constexpr int NT = 128;
    const int need = smem_bytes(p.stages);
    static int configured[MAX_DEVICES] = {};      // per instantiation and per device
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (configured[dev] < need) {
        const int cap = smem_bytes(MAX_STAGES);
        if (need > cap) return cudaErrorInvalidValue;
        cudaError_t e = cudaFuncSetAttribute(gemm_bf16<EPI, A_MN, B_MN, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap);
        if (e != cudaSuccess) return e;
        configured[dev] = cap;
    }
    const dim3 grid((p.N + BN - 1) / BN, (p.M + BM - 1) / BM, workers);
    if (p.logit_part != nullptr && next == nullptr) return cudaErrorInvalidValue;
    return launch_dependent(pdl, gemm_bf16<EPI, A_MN, B_MN, NT>, grid, dim3(NT), (size_t)need, s, a, b, c, next ? *next : c, p);
}

// The persistent gradient + update kernel over the tiles of up to two weight matrices.
cudaError_t launch_update(const UpdateProblem &p0, const UpdateProblem &p1, const UpdateParams &q, cudaStream_t s, bool pdl)
{
    static int sm_count[MAX_DEVICES] = {};        // 0 = this device has not been set up yet
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_update_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, UPD_SMEM);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int total = p0.tiles + p1.tiles;
    if (total <= 0) return cudaSuccess;
    return launch_dependent(pdl, gemm_update_persistent, dim3(std::min(total, sm_count[dev])), dim3(UPD_THREADS), (size_t)UPD_SMEM, s,
                            p0, p1, q);
}

// The gradient chain up to dz1 as one kernel: d_h / 128 CTAs per worker that wait for one another, so all CTAs of a
// launch must be resident together: at most one CTA per SM per launch (a cooperative launch), the workers split over
// several launches when there are more.
template <int DOUT>
cudaError_t launch_chain(const CUtensorMap &k_x, const CUtensorMap &k_w1, const CUtensorMap &k_h1, const CUtensorMap &k_w2,
                         const CUtensorMap &k_w3, const CUtensorMap &k_dz2, const CUtensorMap &mn_w2, const CUtensorMap &st_dz1,
                         ChainParams p, int tiles, int workers, cudaStream_t s, bool pdl, int *launches)
{
    static int sm_count[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(mlp_chain<DOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, CH_SMEM);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int per_launch = sm_count[dev] / tiles;
    if (per_launch < 1) return cudaErrorInvalidConfiguration;
    for (int w0 = 0; w0 < workers; w0 += per_launch) {
        const int n = std::min(per_launch, workers - w0);
        p.w0 = w0;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(tiles, 1, n); cfg.blockDim = dim3(CH_THREADS); cfg.dynamicSmemBytes = CH_SMEM; cfg.stream = s;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeCooperative;
        at[0].val.cooperative = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = pdl ? 2 : 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, mlp_chain<DOUT>, k_x, k_w1, k_h1, k_w2, k_w3, k_dz2, mn_w2, st_dz1, p);
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    return cudaSuccess;
}

inline int stages_for(int k) { return std::max(1, std::min(MAX_STAGES, (k + BK - 1) / BK)); }

// ------------------------------------------------------------------------------------------ small kernels
// warps per CTA of head_backward (measured inside the gradient chain: 2 warps 20.3 us, 4 warps 14.3 us,
// 8 warps 15.9 us; about 8 us of it is fixed cost, not the loop over the samples)
constexpr int HEAD_NW = 4;
// The output layer and everything downstream of it that runs on CUDA cores.  The second hidden layer's GEMM leaves, per
// 128-column tile t, the partial logits part[w][t][b][c] = sum_{j in tile} h2[b][j] W3[c][j] (+ b3[c] in tile 0: in the fused
// call the extra CTA below UPDATES b3, so no CTA of this kernel may read it); every CTA here first finishes
// them for all samples of its worker (thread b: z[c] = sum_t part[t][b][c] in tile order, softmax, row loss
// -log softmax[label], dz3[b][c] = bf16((softmax - onehot) / batch), kept in shared memory), then, for its 32 hidden
// units j and all samples:
//   dz2[b][j] = bf16((sum_c dz3[b][c] W3[c][j]) * (h2[b][j] > 0)),  db2[j] = sum_b dz2[b][j],
//   dW3[c][j] = sum_b dz3[b][c] h2[b][j];
// one extra CTA per worker writes db3[c] = sum_b dz3[b][c], loss[w] = mean_b row loss and the zero padding of
// the gradient.  Fixed summation orders (deterministic).  grid (d_h / 32 + 1, K).  (Recomputing the 128 softmaxes in
// each of a worker's 33 CTAs costs about a microsecond and saves a kernel of 8.5 us that did nothing else.)
template <int DOUT, int NW>
__global__ void __launch_bounds__(32 * NW)
head_backward(const bf16 *__restrict__ h2, const bf16 *params, const float *__restrict__ part, int n_tiles,
              const int *__restrict__ labels, bf16 *__restrict__ dz2, float *__restrict__ grads,
              float *__restrict__ loss, long long P, long long P_raw, long long oW3, long long ob2, long long ob3,
              int B, int d_h, int d_out, const StepTarget step)
{
    // step.x_in != nullptr: instead of writing dW3, db2, db3 (and the zero padding) to `grads`, apply the local
    // step to those parameters here (indices are flat positions in the K x P state).  Every CTA reads and
    // updates only its own columns of W3, so the update cannot disturb another CTA's reads.
    // NW warps per CTA; warp wp owns samples wp, wp + NW, ...; DOUT bounds the class loops (>= d_out)
    static_assert(NW >= 2, "the scalar CTA uses two warps");
    constexpr int C4 = (DOUT + 3) / 4;
    __shared__ __align__(16) float sdz[128 * 16];
    __shared__ float srowloss[128];
    __shared__ float red[NW][16][33];
    __shared__ float colsum[NW][33];
    const int w = blockIdx.y, j0 = blockIdx.x * 32, lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int j = j0 + lane;
    const bool scalar_cta = (blockIdx.x == gridDim.x - 1);
    pdl_launch_dependents();
    pdl_wait();
    // first batch of this thread's h2 values: in flight while the logits are finished
    float hreg[16];
    if (!scalar_cta) {
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int b = wp + NW * q;
            hreg[q] = (b < B) ? __bfloat162float(h2[((long long)w * B + b) * d_h + j]) : 0.0f;
        }
    }
    // the logits, softmax, row loss and dz3 of sample b (B <= 128)
    for (int b = threadIdx.x; b < B; b += 32 * NW) {
        float z[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) z[c] = 0.0f;          // (b3 is already inside the first tile's partial sums)
        // tiles in order, four at a time with all their loads in flight (only the float4s that hold classes < DOUT;
        // eight at a time took 186 registers and was slower)
        const float4 *pp = reinterpret_cast<const float4 *>(part + (((long long)w * n_tiles) * 128 + b) * 16);
        constexpr int TB = 4;
        for (int t0 = 0; t0 < n_tiles; t0 += TB) {
            float4 v[TB][C4];
#pragma unroll
            for (int u = 0; u < TB; ++u)
#pragma unroll
                for (int q = 0; q < C4; ++q)
                    v[u][q] = (t0 + u < n_tiles) ? __ldcg(pp + (long long)(t0 + u) * (128 * 16 / 4) + q) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
            for (int u = 0; u < TB; ++u) {
                if (t0 + u < n_tiles) {
#pragma unroll
                    for (int q = 0; q < C4; ++q) {
                        z[4 * q] += v[u][q].x; z[4 * q + 1] += v[u][q].y; z[4 * q + 2] += v[u][q].z; z[4 * q + 3] += v[u][q].w;
                    }
                }
            }
        }
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < 16; ++c) if (c < d_out) zmax = fmaxf(zmax, z[c]);
        float e[16], ssum = 0.0f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            e[c] = (c < d_out) ? expf(z[c] - zmax) : 0.0f;
            ssum += e[c];
        }
        const int y = labels[(long long)w * B + b];
        float py = 0.0f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            const float pc = e[c] / ssum;
            if (c == y) py = pc;
            const float d = (c < d_out) ? (pc - (c == y ? 1.0f : 0.0f)) / (float)B : 0.0f;
            sdz[b * 16 + c] = __bfloat162float(__float2bfloat16_rn(d));
        }
        srowloss[b] = -logf(py);
    }
    if (scalar_cta) {
        // The extra CTA of every worker: the per-worker scalars db3[c] = sum_b dz3[b][c], loss = mean_b rowloss and
        // the zero padding of the gradient, each by one warp (lane-strided partial sums, then a fixed shuffle tree).
        // As an epilogue of one of the column CTAs this made that CTA the straggler of the kernel (2.3 us).
        __syncthreads();
        if (wp == 0) {
            for (int c = 0; c < d_out; ++c) {
                float s = 0.0f;
                for (int b = lane; b < B; b += 32) s += sdz[b * 16 + c];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) {
                    if (step.x_in != nullptr) step_element(step, (long long)w * P + ob3 + c, s);
                    else grads[(long long)w * P + ob3 + c] = s;
                }
            }
        } else if (wp == 1) {
            float t[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (lane + 32 * i < B) t[i] = srowloss[lane + 32 * i];
            float s = (t[0] + t[1]) + (t[2] + t[3]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) loss[w] = s / (float)B;
        }
        for (long long i = P_raw + threadIdx.x; i < P; i += 32 * NW) {
            if (step.x_in != nullptr) step_element(step, (long long)w * P + i, 0.0f);
            else grads[(long long)w * P + i] = 0.0f;
        }
        return;
    }
    // (requesting this column of W3 before the logits are finished gained 1 us in the eager chain and lost 1.4 us in a
    //  replayed graph)
    float w3[4 * C4], acc3[4 * C4];
#pragma unroll
    for (int c = 0; c < 4 * C4; ++c) {
        w3[c] = (c < d_out) ? __bfloat162float(params[(long long)w * P + oW3 + (long long)c * d_h + j]) : 0.0f;
        acc3[c] = 0.0f;
    }
    __syncthreads();
    float csum = 0.0f;
    for (int q0 = 0; q0 * NW < B; q0 += 16) {
        if (q0 > 0) {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int b = wp + NW * (q0 + q);
                hreg[q] = (b < B) ? __bfloat162float(h2[((long long)w * B + b) * d_h + j]) : 0.0f;
            }
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int b = wp + NW * (q0 + q);
            if (b < B) {
                const float h = hreg[q];
                float a = 0.0f;
                const float4 *d4 = reinterpret_cast<const float4 *>(sdz + b * 16);
#pragma unroll
                for (int c4 = 0; c4 < C4; ++c4) {
                    const float4 dd = d4[c4];
                    const float d[4] = {dd.x, dd.y, dd.z, dd.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (4 * c4 + e < DOUT) {
                            a = fmaf(d[e], w3[4 * c4 + e], a);
                            acc3[4 * c4 + e] = fmaf(d[e], h, acc3[4 * c4 + e]);
                        }
                    }
                }
                const bf16 v = __float2bfloat16_rn(h > 0.0f ? a : 0.0f);
                dz2[((long long)w * B + b) * d_h + j] = v;
                csum += __bfloat162float(v);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < 16; ++c) red[wp][c][lane] = (c < DOUT) ? acc3[c < DOUT ? c : 0] : 0.0f;
    colsum[wp][lane] = csum;
    __syncthreads();
    for (int i = threadIdx.x; i < 16 * 32; i += 32 * NW) {
        const int c = i >> 5, l = i & 31;
        if (c < d_out) {
            float s = 0.0f;
#pragma unroll
            for (int q = 0; q < NW; ++q) s += red[q][c][l];
            const long long idx = (long long)w * P + oW3 + (long long)c * d_h + j0 + l;
            if (step.x_in != nullptr) step_element(step, idx, s);
            else grads[idx] = s;
        }
    }
    if (threadIdx.x < 32) {
        float s = 0.0f;
#pragma unroll
        for (int q = 0; q < NW; ++q) s += colsum[q][threadIdx.x];
        const long long idx = (long long)w * P + ob2 + j0 + threadIdx.x;
        if (step.x_in != nullptr) step_element(step, idx, s);
        else grads[idx] = s;
    }
}

}  // namespace

struct cocod_mlp {
    int K, B, d_in, d_h, d_out;
    long long P, P_raw, oW1, ob1, oW2, ob2, oW3, ob3;
    bf16 *h1 = nullptr, *h2 = nullptr, *dz2 = nullptr, *dz1 = nullptr;
    float *logit_part = nullptr;        // [K][d_h / 128][128][16]: per-tile partial logits left by the second layer's GEMM
    int *error_flag = nullptr;
    // maps over scratch (fixed addresses): reduction-contiguous (k) and row-contiguous (mn) views
    CUtensorMap k_h1, k_dz2, mn_dz2, mn_h1, mn_dz1;
    CUtensorMap st_h2, st_dz1;          // store views (64 columns x 128 rows) of outputs that are not read that way
    long long launches = 0;
    int *chain_sync = nullptr;          // [K][4] counters of the chain kernel (zero between launches)
    int chain = 1;                      // COCOD_MLP_OPT_CHAIN: the four kernels before the weight gradients as one cluster kernel
    // COCOD_MLP_OPT_PROFILE: CUDA events around every gradient pass and around its gradient + update kernel
    int profile = 0;                    // 0 off, 1 events (+ stamps), 2 stamps only
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_pass, prof_update;
    unsigned long long *stamps = nullptr;     // device: kMaxStamps x {earliest start, latest end} of the update kernel's CTAs
    int n_stamps = 0;
};

namespace {

constexpr int kMaxStamps = 4096;

void mlp_profile_clear(cocod_mlp *h)
{
    h->n_stamps = 0;
    if (h->stamps) {                   // start = all ones (atomicMin), end = 0 (atomicMax); the device is idle here
        std::vector<unsigned long long> init(2 * (size_t)kMaxStamps);
        for (size_t i = 0; i < init.size(); i += 2) { init[i] = ~0ull; init[i + 1] = 0ull; }
        cudaMemcpy(h->stamps, init.data(), init.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice);
    }
    for (auto *list : {&h->prof_pass, &h->prof_update}) {
        for (auto &pr : *list) {
            cudaEventDestroy(pr.first);
            cudaEventDestroy(pr.second);
        }
        list->clear();
    }
}

// An event pair whose first event is recorded now; the caller records the second one.
bool mlp_profile_open(cocod_mlp *h, std::vector<std::pair<cudaEvent_t, cudaEvent_t>> &list, cudaStream_t s)
{
    if (h->profile != 1 || list.size() >= 4096) return false;
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaEventCreate(&a) != cudaSuccess) { cudaGetLastError(); return false; }
    if (cudaEventCreate(&b) != cudaSuccess) { cudaGetLastError(); cudaEventDestroy(a); return false; }
    cudaEventRecord(a, s);
    list.emplace_back(a, b);
    return true;
}

void mlp_free(cocod_mlp *h)
{
    mlp_profile_clear(h);
    void *ptrs[] = {h->h1, h->h2, h->dz2, h->dz1, h->logit_part, h->error_flag, h->stamps, h->chain_sync};
    for (void *p : ptrs) if (p) cudaFree(p);
    delete h;
}

}  // namespace

extern "C" {

int cocod_mlp_create(cocod_mlp_handle **out, int K, int batch, int d_in, int d_hidden, int d_out)
{
    if (!out || K < 1 || K > 1024 || batch != 128 || d_in < 8 || d_in % 8 || d_hidden < 128 || d_hidden % 128 ||
        d_out < 1 || d_out > 16)
        return COCOD_ERR_INVALID;
    if (!get_encoder()) return COCOD_ERR_CUDA;
    cocod_mlp *h = new (std::nothrow) cocod_mlp();
    if (!h) return COCOD_ERR_OOM;
    h->K = K; h->B = batch; h->d_in = d_in; h->d_h = d_hidden; h->d_out = d_out;
    h->oW1 = 0;
    h->ob1 = h->oW1 + (long long)d_hidden * d_in;
    h->oW2 = h->ob1 + d_hidden;
    h->ob2 = h->oW2 + (long long)d_hidden * d_hidden;
    h->oW3 = h->ob2 + d_hidden;
    h->ob3 = h->oW3 + (long long)d_out * d_hidden;
    h->P_raw = h->ob3 + d_out;
    h->P = (h->P_raw + 63) / 64 * 64;
    const size_t act = (size_t)K * batch * d_hidden * sizeof(bf16);
    cudaError_t e = cudaSuccess;
    auto alloc = [&](void **p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
    alloc((void **)&h->h1, act);
    alloc((void **)&h->h2, act);
    alloc((void **)&h->dz2, act);
    alloc((void **)&h->dz1, act);
    alloc((void **)&h->logit_part, (size_t)K * (d_hidden / 128) * 128 * 16 * sizeof(float));
    alloc((void **)&h->error_flag, sizeof(int));
    alloc((void **)&h->chain_sync, (size_t)K * 4 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->error_flag, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->chain_sync, 0, (size_t)K * 4 * sizeof(int));
    if (e != cudaSuccess) {
        cudaGetLastError();
        mlp_free(h);
        return e == cudaErrorMemoryAllocation ? COCOD_ERR_OOM : COCOD_ERR_CUDA;
    }
    const uint64_t uK = K, uB = batch, uh = d_hidden;
    // activations are [B][d_h] per worker: as a reduction-contiguous operand the reduction runs over
    // d_h; as a row-contiguous operand the reduction runs over the batch.
    bool ok = map_k(&h->k_h1, h->h1, uh, uB, uK, uh, uB * uh) && map_k(&h->k_dz2, h->dz2, uh, uB, uK, uh, uB * uh) &&
              map_mn(&h->mn_dz2, h->dz2, uh, uB, uK, uh, uB * uh) && map_mn(&h->mn_h1, h->h1, uh, uB, uK, uh, uB * uh) &&
              map_mn(&h->mn_dz1, h->dz1, uh, uB, uK, uh, uB * uh) && map_k(&h->st_h2, h->h2, uh, uB, uK, uh, uB * uh) &&
              map_k(&h->st_dz1, h->dz1, uh, uB, uK, uh, uB * uh);
    if (!ok) {
        mlp_free(h);
        return COCOD_ERR_CUDA;
    }
    *out = h;
    return COCOD_OK;
}

int cocod_mlp_destroy(cocod_mlp_handle *h)
{
    if (!h) return COCOD_OK;
    cudaDeviceSynchronize();
    mlp_free(h);
    return COCOD_OK;
}

int64_t cocod_mlp_param_count(const cocod_mlp_handle *h) { return h ? h->P : -1; }
int64_t cocod_mlp_param_count_unpadded(const cocod_mlp_handle *h) { return h ? h->P_raw : -1; }
int64_t cocod_mlp_launch_count(const cocod_mlp_handle *h) { return h ? h->launches : -1; }

}  // extern "C"

namespace {

// The whole gradient pass.  One persistent kernel (gemm_update_persistent: the tiles of W2, then of W1, two
// accumulators in tensor memory) forms the weight gradients dW1, dW2: with fused == nullptr it writes them to
// `grads`; otherwise it applies the engine's local step tile by tile (x, v and the bf16 copy of x are updated in
// place, nothing is written to `grads`).
int run_grad(cocod_mlp *h, const bf16 *prm, const bf16 *xin, const int32_t *labels, float *grads, float *loss,
             cudaStream_t s, const cocod_step_plan *fused)
{
    const int K = h->K, B = h->B, d_in = h->d_in, d_h = h->d_h, d_out = h->d_out;
    const long long P = h->P;
    const uint64_t uK = K, uB = B, uh = d_h, ui = d_in, uP = P;
    // maps over caller memory
    CUtensorMap k_x, mn_x, k_w1, k_w2, mn_w2, k_w3, c_w1{}, c_w2{};
    if (!make_map(&k_w3, prm + h->oW3, uh, (uint64_t)d_out, uK, uh, uP, NEXT_N) ||
        !map_k(&k_x, xin, ui, uB, uK, ui, uB * ui) || !map_mn(&mn_x, xin, ui, uB, uK, ui, uB * ui) ||
        !map_k(&k_w1, prm + h->oW1, ui, uh, uK, ui, uP) || !map_k(&k_w2, prm + h->oW2, uh, uh, uK, uh, uP) ||
        !map_mn(&mn_w2, prm + h->oW2, uh, uh, uK, uh, uP))
        return COCOD_ERR_CUDA;
    struct StateMaps { CUtensorMap x_in, x_out, v, shadow; } s_w1{}, s_w2{};      // views of W1 and W2 in the engine's state
    if (fused) {
        float *xi = const_cast<float *>(fused->x_in);
        bf16 *sh = fused->shadow;
        bool ok = map_out(&s_w2.x_in, xi + h->oW2, uh, uh, uK, uh, uP) && map_out(&s_w2.x_out, fused->x_out + h->oW2, uh, uh, uK, uh, uP) &&
                  map_out(&s_w2.v, fused->v + h->oW2, uh, uh, uK, uh, uP) &&
                  map_out(&s_w1.x_in, xi + h->oW1, ui, uh, uK, ui, uP) && map_out(&s_w1.x_out, fused->x_out + h->oW1, ui, uh, uK, ui, uP) &&
                  map_out(&s_w1.v, fused->v + h->oW1, ui, uh, uK, ui, uP);
        if (ok && sh) ok = map_k(&s_w2.shadow, sh + h->oW2, uh, uh, uK, uh, uP) && map_k(&s_w1.shadow, sh + h->oW1, ui, uh, uK, ui, uP);
        if (!ok) return COCOD_ERR_CUDA;
    } else if (!map_out(&c_w1, grads + h->oW1, ui, uh, uK, ui, uP) || !map_out(&c_w2, grads + h->oW2, uh, uh, uK, uh, uP)) {
        return COCOD_ERR_CUDA;
    }
#define LAUNCH_OK() do { if (cudaGetLastError() != cudaSuccess) return COCOD_ERR_CUDA; ++h->launches; } while (0)
#define GEMM_OK(call) do { if ((call) != cudaSuccess) return COCOD_ERR_CUDA; ++h->launches; } while (0)
    // Each kernel of the chain may set up while its predecessor drains (programmatic dependent launch): 11 % off
    // the eager chain.  Under stream capture only the two forward GEMMs keep these edges: measured edge by edge in a
    // replayed graph, they gain 1.1 and 0.8 us there, while the edges into the two output-layer kernels and into the
    // backward GEMMs cost 1.5 - 2.7 us each.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) return COCOD_ERR_CUDA;
    const bool pdl = (capturing == cudaStreamCaptureStatusNone);
    const bool pdl_fwd = true;
    // profiling (never while capturing): events around the whole pass and around the gradient + update kernel
    const bool prof_pass = (capturing == cudaStreamCaptureStatusNone) && mlp_profile_open(h, h->prof_pass, s);
    // fused call: the small tensors (biases, W3, padding) take their local step inside the kernels that produce
    // their gradients; otherwise those kernels write the gradients out
    StepTarget small{};
    if (fused) {
        small.x_in = fused->x_in; small.x_out = fused->x_out; small.v = fused->v; small.shadow = fused->shadow;
        small.worker_stride = P; small.lr = fused->lr; small.mu = fused->mu; small.wd = fused->wd;
    }
    const bool chain = h->chain != 0;
    if (chain) {
        ChainParams c{};
        c.d_in = d_in; c.d_h = d_h; c.d_out = d_out;
        c.P = P; c.P_raw = h->P_raw; c.oW3 = h->oW3; c.ob1 = h->ob1; c.ob2 = h->ob2; c.ob3 = h->ob3;
        c.params = prm; c.labels = labels; c.loss = loss; c.grads = grads; c.step = small; c.error_flag = h->error_flag;
        c.logit_part = h->logit_part; c.sync = h->chain_sync;
        int n = 0;
        const cudaError_t e = (d_out == 10 ? launch_chain<10> : launch_chain<16>)(k_x, k_w1, h->k_h1, k_w2, k_w3, h->k_dz2, mn_w2,
                                                                                 h->st_dz1, c, d_h / 128, K, s, pdl_fwd, &n);
        h->launches += n;
        if (e != cudaSuccess) { fprintf(stderr, "chain launch: %s\n", cudaGetErrorString(e)); return COCOD_ERR_CUDA; }
    }
    Params p{};
    p.b_keep = 1;                      // the weights: read again by the backward pass and, rewritten in place, by the next step
    p.error_flag = h->error_flag;
    // h1 = relu(x W1^T + b1)
    p.M = B; p.N = d_h; p.K = d_in; p.stages = stages_for(d_in);
    p.bias = prm + h->ob1; p.bias_worker_stride = P;
    if (!chain) GEMM_OK((launch_gemm<EPI_BIAS_RELU, false, false>(k_x, k_w1, h->k_h1, p, K, s, pdl_fwd)));
    // h2 = relu(h1 W2^T + b2), and per 128-column tile the partial logits h2 W3^T of that tile
    p.K = d_h; p.stages = stages_for(d_h); p.bias = prm + h->ob2;
    p.logit_part = h->logit_part; p.b_next = prm + h->ob3; p.b_next_worker_stride = P; p.next_out = d_out;
    if (!chain) GEMM_OK((launch_gemm<EPI_BIAS_RELU, false, false>(h->k_h1, k_w2, h->st_h2, p, K, s, pdl_fwd, &k_w3)));
    // logits, loss, dz3; then dz2, dW3, db3, db2
    if (!chain)
        GEMM_OK(launch_dependent(pdl, d_out == 10 ? head_backward<10, HEAD_NW> : head_backward<16, HEAD_NW>, dim3(d_h / 32 + 1, K),
                                 dim3(32 * HEAD_NW), 0, s, h->h2, prm, (const float *)h->logit_part, d_h / 128, labels,
                                 h->dz2, grads, loss, P, h->P_raw, h->oW3, h->ob2, h->ob3, B, d_h, d_out, small));
    // dz1 = (dz2 W2) * (h1 > 0): B operand is W2 itself, read with n contiguous
    Params q{};
    q.b_keep = 1;
    q.error_flag = h->error_flag;
    q.M = B; q.N = d_h; q.K = d_h; q.stages = stages_for(d_h);
    q.mask = h->h1; q.mask_worker_stride = (long long)B * d_h;
    // db1 = column sums of dz1, from the same epilogue
    if (!fused) {
        q.colsum = grads + h->ob1; q.colsum_worker_stride = P;
    } else {                                                      // ... applied to b1 on the spot
        q.colsum_step = small;
        q.colsum_step.x_in += h->ob1; q.colsum_step.x_out += h->ob1; q.colsum_step.v += h->ob1;
        if (q.colsum_step.shadow) q.colsum_step.shadow += h->ob1;
    }
    // One persistent kernel walks the tiles of W2 and then of W1 (the batch of 128 is its whole reduction: two operand
    // blocks): in the fused call it applies the local step to each tile as soon as its product is formed, in the gradient
    // call it writes the product out.
    static_assert(2 * BK == 128, "the update kernel holds the whole reduction in its two-stage ring");
    if (!chain) GEMM_OK((launch_gemm<EPI_MASK, false, true>(h->k_dz2, mn_w2, h->st_dz1, q, K, s, pdl)));
    {
        UpdateProblem u2{}, u1{};
        u2.a = h->mn_dz2; u2.b = h->mn_h1;
        u2.M = d_h; u2.N = d_h; u2.tiles_m = (d_h + BM - 1) / BM; u2.tiles_n = (d_h + BN - 1) / BN;
        u2.tiles = K * u2.tiles_m * u2.tiles_n;
        u1.a = h->mn_dz1; u1.b = mn_x;
        u1.M = d_h; u1.N = d_in; u1.tiles_m = (d_h + BM - 1) / BM; u1.tiles_n = (d_in + BN - 1) / BN;
        u1.tiles = K * u1.tiles_m * u1.tiles_n;
        UpdateParams uq{};
        uq.K = B; uq.error_flag = h->error_flag;
        if (fused) {
            u2.x_in = s_w2.x_in; u2.x_out = s_w2.x_out; u2.v = s_w2.v; u2.shadow = s_w2.shadow; u2.has_shadow = fused->shadow != nullptr;
            u1.x_in = s_w1.x_in; u1.x_out = s_w1.x_out; u1.v = s_w1.v; u1.shadow = s_w1.shadow; u1.has_shadow = fused->shadow != nullptr;
            uq.lr = fused->lr; uq.mu = fused->mu; uq.wd = fused->wd;
        } else {                      // the gradient tensors take the place of x_out; nothing else is touched
            u2.x_out = c_w2; u1.x_out = c_w1;
            u2.x_in = u2.v = c_w2; u1.x_in = u1.v = c_w1;      // (valid maps; never used)
            uq.store_only = 1;
        }
        const bool prof_upd = (capturing == cudaStreamCaptureStatusNone) && mlp_profile_open(h, h->prof_update, s);
        if (h->profile != 0 && h->stamps && capturing == cudaStreamCaptureStatusNone && h->n_stamps < kMaxStamps)
            uq.stamp = h->stamps + 2 * (size_t)(h->n_stamps++);
        GEMM_OK(launch_update(u2, u1, uq, s, pdl && !prof_upd));
        if (prof_upd) cudaEventRecord(h->prof_update.back().second, s);
    }
#undef LAUNCH_OK
#undef GEMM_OK
    if (prof_pass) cudaEventRecord(h->prof_pass.back().second, s);
    return COCOD_OK;
}

// Device scratch of one self-test call: allocated on the current device, released (after the device has gone
// idle: the destructor runs only after the call has synchronised its stream or failed) when the call returns.
struct SelftestScratch {
    void *ptrs[4] = {nullptr, nullptr, nullptr, nullptr};
    int n = 0;
    void *alloc(size_t bytes)
    {
        void *p = nullptr;
        if (n >= 4 || cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        ptrs[n++] = p;
        return p;
    }
    ~SelftestScratch()
    {
        if (n > 0) cudaDeviceSynchronize();
        for (int i = 0; i < n; ++i) cudaFree(ptrs[i]);
    }
};

}  // namespace

extern "C" {

int cocod_mlp_grad(cocod_mlp_handle *h, const void *params_bf16, const void *x, const int32_t *labels, float *grads,
                   float *loss, cocod_stream_t stream)
{
    if (!h || !params_bf16 || !x || !labels || !grads || !loss) return COCOD_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(params_bf16) & 15u) || (reinterpret_cast<uintptr_t>(x) & 15u) ||
        (reinterpret_cast<uintptr_t>(grads) & 15u))
        return COCOD_ERR_INVALID;
    return run_grad(h, static_cast<const bf16 *>(params_bf16), static_cast<const bf16 *>(x), labels, grads, loss,
                    (cudaStream_t)stream, nullptr);
}

int cocod_mlp_grad_step(cocod_mlp_handle *h, cocod_handle *engine, const void *x, const int32_t *labels, float *loss)
{
    if (!h || !engine || !x || !labels || !loss) return COCOD_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(x) & 15u) return COCOD_ERR_INVALID;
    cocod_step_plan plan{};
    if (int rc = cocod_internal_plan_step(engine, &plan)) return rc;
    if (plan.K != h->K || plan.P != h->P) return COCOD_ERR_INVALID;
    if (!plan.shadow) return COCOD_ERR_STATE;            // the gradients are computed from the bf16 copy of x
    // no gradient buffer: every tensor takes its local step inside the kernel that produces its gradient
    if (int rc = run_grad(h, plan.shadow, static_cast<const bf16 *>(x), labels, nullptr, loss, plan.compute, &plan))
        return rc;
    return cocod_internal_finish_step(engine, 0);
}

#ifdef COCOD_CHAIN_TRACE
int cocod_debug_chain_trace(unsigned long long *out, int n)
{
    return cudaMemcpyFromSymbol(out, cocod::gemm::g_chain_trace, (size_t)n * sizeof(unsigned long long)) == cudaSuccess ? 0 : 1;
}
#endif

int cocod_mlp_set_option(cocod_mlp_handle *h, int option, int value)
{
    if (!h) return COCOD_ERR_INVALID;
    if (option == COCOD_MLP_OPT_CHAIN) {
        if (value != 0 && value != 1) return COCOD_ERR_INVALID;
        h->chain = value;
        return COCOD_OK;
    }
    if (option != COCOD_MLP_OPT_PROFILE) return COCOD_ERR_INVALID;
    if (value < 0 || value > 2) return COCOD_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) return COCOD_ERR_CUDA;
    if (value != 0 && !h->stamps &&
        cudaMalloc((void **)&h->stamps, 2 * (size_t)kMaxStamps * sizeof(unsigned long long)) != cudaSuccess) {
        cudaGetLastError();
        h->stamps = nullptr;
        return COCOD_ERR_OOM;
    }
    mlp_profile_clear(h);
    h->profile = value;
    return COCOD_OK;
}

int cocod_mlp_profile_get(cocod_mlp_handle *h, int *calls, float *pass_ms, float *update_ms)
{
    if (!h || !calls || !pass_ms || !update_ms) return COCOD_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) return COCOD_ERR_CUDA;
    auto average = [](const std::vector<std::pair<cudaEvent_t, cudaEvent_t>> &list, float *out) {
        double sum = 0.0;
        for (const auto &pr : list) {
            float ms = 0.0f;
            if (cudaEventElapsedTime(&ms, pr.first, pr.second) != cudaSuccess) return false;
            sum += ms;
        }
        *out = list.empty() ? 0.0f : (float)(sum / (double)list.size());
        return true;
    };
    if (!average(h->prof_pass, pass_ms) || !average(h->prof_update, update_ms)) { cudaGetLastError(); return COCOD_ERR_CUDA; }
    *calls = (int)h->prof_pass.size();
    return COCOD_OK;
}

int cocod_mlp_profile_get_device(cocod_mlp_handle *h, int *calls, float *update_ms)
{
    if (!h || !calls || !update_ms) return COCOD_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) return COCOD_ERR_CUDA;
    *calls = 0;
    *update_ms = 0.0f;
    if (!h->stamps || h->n_stamps == 0) return COCOD_OK;
    std::vector<unsigned long long> st(2 * (size_t)h->n_stamps);
    if (cudaMemcpy(st.data(), h->stamps, st.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return COCOD_ERR_CUDA;
    }
    double sum = 0.0;
    int n = 0;
    for (int i = 0; i < h->n_stamps; ++i)
        if (st[2 * i] != ~0ull && st[2 * i + 1] > st[2 * i]) { sum += (double)(st[2 * i + 1] - st[2 * i]); ++n; }
    *calls = n;
    *update_ms = n ? (float)(sum / n * 1e-6) : 0.0f;
    return COCOD_OK;
}

int cocod_mlp_check(cocod_mlp_handle *h, cocod_stream_t stream)
{
    if (!h) return COCOD_ERR_INVALID;
    int flag = 0;
    if (cudaMemcpyAsync(&flag, h->error_flag, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return COCOD_ERR_CUDA;
    // a chain kernel that gave up leaves its counters as they were: clear them once nothing of this handle runs any more
    if (flag && (cudaDeviceSynchronize() != cudaSuccess ||
                 cudaMemset(h->chain_sync, 0, (size_t)h->K * 4 * sizeof(int)) != cudaSuccess))
        return COCOD_ERR_CUDA;
    return flag ? COCOD_ERR_TIMEOUT : COCOD_OK;
}

int cocod_gemm_bf16(const void *A, const void *B, float *C, int M, int N, int Kd, int batch_count, int a_rows_contiguous,
                    int b_rows_contiguous, int64_t lda, int64_t ldb, int64_t ldc, int64_t stride_a, int64_t stride_b,
                    int64_t stride_c, cocod_stream_t stream)
{
    if (!A || !B || !C || M < 1 || N < 1 || Kd < 1 || batch_count < 1 || batch_count > 65535) return COCOD_ERR_INVALID;
    const int64_t a_cols = a_rows_contiguous ? M : Kd, a_rows = a_rows_contiguous ? Kd : M;
    const int64_t b_cols = b_rows_contiguous ? N : Kd, b_rows = b_rows_contiguous ? Kd : N;
    if ((lda % 8) || (ldb % 8) || (stride_a % 8) || (stride_b % 8) || lda < a_cols || ldb < b_cols || ldc < N)
        return COCOD_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(A) & 15u) || (reinterpret_cast<uintptr_t>(B) & 15u)) return COCOD_ERR_INVALID;
    CUtensorMap ma, mb, mc{};
    const uint64_t sa = batch_count > 1 ? (uint64_t)stride_a : (uint64_t)a_rows * lda;
    const uint64_t sb = batch_count > 1 ? (uint64_t)stride_b : (uint64_t)b_rows * ldb;
    const uint64_t sc = batch_count > 1 ? (uint64_t)stride_c : (uint64_t)M * ldc;
    if (!make_map(&ma, A, a_cols, a_rows, batch_count, lda, sa, a_rows_contiguous ? 64 : 128) ||
        !make_map(&mb, B, b_cols, b_rows, batch_count, ldb, sb, b_rows_contiguous ? 64 : 128))
        return COCOD_ERR_CUDA;
    // the kernel's timeout flag: 4 bytes per device that ever makes this call, kept until the process exits
    static int *flags[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return COCOD_ERR_CUDA;
    if (!flags[dev]) {
        if (cudaMalloc((void **)&flags[dev], sizeof(int)) != cudaSuccess) { cudaGetLastError(); return COCOD_ERR_OOM; }
        cudaMemset(flags[dev], 0, sizeof(int));
    }
    int *flag = flags[dev];
    Params p{};
    p.M = M; p.N = N; p.K = Kd; p.stages = stages_for(Kd);
    p.c = C; p.c_worker_stride = (long long)sc; p.ldc = (int)ldc;
    p.map_c_ok = map_out(&mc, C, N, M, batch_count, ldc, sc) ? 1 : 0;      // else: plain predicated stores
    p.error_flag = flag;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (a_rows_contiguous && b_rows_contiguous) e = launch_gemm<EPI_F32, true, true>(ma, mb, mc, p, batch_count, s);
    else if (a_rows_contiguous) e = launch_gemm<EPI_F32, true, false>(ma, mb, mc, p, batch_count, s);
    else if (b_rows_contiguous) e = launch_gemm<EPI_F32, false, true>(ma, mb, mc, p, batch_count, s);
    else e = launch_gemm<EPI_F32, false, false>(ma, mb, mc, p, batch_count, s);
    if (e != cudaSuccess) return COCOD_ERR_CUDA;
    int f = 0;
    if (cudaMemcpyAsync(&f, flag, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    if (f) {
        cudaMemset(flag, 0, sizeof(int));
        return COCOD_ERR_TIMEOUT;
    }
    return COCOD_OK;
}

// Self-test of the bounded waits: one tile whose operand copies are never issued.
int cocod_gemm_wait_selftest(int wait_ms, cocod_stream_t stream)
{
    if (wait_ms < 1 || wait_ms > 2000) return COCOD_ERR_INVALID;
    // scratch of this call only (on the current device), freed before returning
    SelftestScratch sc;
    bf16 *buf = static_cast<bf16 *>(sc.alloc(128 * 64 * sizeof(bf16)));
    int *flag = static_cast<int *>(sc.alloc(sizeof(int)));
    if (!buf || !flag) return COCOD_ERR_OOM;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(buf, 0, 128 * 64 * sizeof(bf16), s) != cudaSuccess ||
        cudaMemsetAsync(flag, 0, sizeof(int), s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    CUtensorMap m, none{};
    if (!map_k(&m, buf, 64, 128, 1, 64, 128 * 64)) return COCOD_ERR_CUDA;
    Params p{};
    p.M = 128; p.N = 128; p.K = 64; p.stages = 1;
    p.c = nullptr; p.map_c_ok = 0;
    p.error_flag = flag;
    p.wait_ns = (unsigned long long)wait_ms * 1000000ull;
    p.debug_no_loads = 1;
    if (launch_gemm<EPI_F32, false, false>(m, m, none, p, 1, s) != cudaSuccess) return COCOD_ERR_CUDA;
    int f = 0;
    if (cudaMemcpyAsync(&f, flag, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    return f ? COCOD_ERR_TIMEOUT : COCOD_OK;
}

int cocod_gemm_update_wait_selftest(int wait_ms, cocod_stream_t stream)
{
    if (wait_ms < 1 || wait_ms > 2000) return COCOD_ERR_INVALID;
    SelftestScratch sc;                       // scratch of this call only, freed before returning
    bf16 *ops = static_cast<bf16 *>(sc.alloc(128 * 128 * sizeof(bf16)));
    float *state = static_cast<float *>(sc.alloc(128 * 128 * sizeof(float)));
    int *flag = static_cast<int *>(sc.alloc(sizeof(int)));
    if (!ops || !state || !flag) return COCOD_ERR_OOM;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(flag, 0, sizeof(int), s) != cudaSuccess) return COCOD_ERR_CUDA;
    // three tiles for one CTA: nothing is ever copied, so the maps only have to exist
    UpdateProblem u{}, none{};
    if (!map_mn(&u.a, ops, 128, 128, 1, 128, 128 * 128) || !map_mn(&u.b, ops, 128, 128, 1, 128, 128 * 128) ||
        !map_out(&u.x_in, state, 128, 128, 1, 128, 128 * 128) || !map_out(&u.x_out, state, 128, 128, 1, 128, 128 * 128) ||
        !map_out(&u.v, state, 128, 128, 1, 128, 128 * 128))
        return COCOD_ERR_CUDA;
    u.has_shadow = 0; u.M = 128; u.N = 128; u.tiles_m = 1; u.tiles_n = 1; u.tiles = 3;
    UpdateParams q{};
    q.K = 128; q.lr = 0.1f; q.mu = 0.9f; q.wd = 0.0f; q.error_flag = flag;
    q.wait_ns = (unsigned long long)wait_ms * 1000000ull;
    q.debug_no_loads = 1;
    if (cudaFuncSetAttribute(gemm_update_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, UPD_SMEM) != cudaSuccess)
        return COCOD_ERR_CUDA;
    if (launch_dependent(false, gemm_update_persistent, dim3(1), dim3(UPD_THREADS), (size_t)UPD_SMEM, s, u, none, q) != cudaSuccess)
        return COCOD_ERR_CUDA;
    int f = 0;
    if (cudaMemcpyAsync(&f, flag, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    return f ? COCOD_ERR_TIMEOUT : COCOD_OK;
}

int cocod_mlp_chain_wait_selftest(int wait_ms, cocod_stream_t stream)
{
    if (wait_ms < 1 || wait_ms > 2000) return COCOD_ERR_INVALID;
    // a small model of its own: 2 workers x 2 tiles, all inputs zero
    cocod_mlp_handle *h = nullptr;
    if (int rc = cocod_mlp_create(&h, 2, 128, 64, 256, 10)) return rc;
    struct Guard { cocod_mlp_handle *h; ~Guard() { cocod_mlp_destroy(h); } } guard{h};
    SelftestScratch sc;
    const size_t n_state = (size_t)h->K * h->P;
    bf16 *prm = static_cast<bf16 *>(sc.alloc(n_state * sizeof(bf16)));
    bf16 *x = static_cast<bf16 *>(sc.alloc((size_t)h->K * 128 * 64 * sizeof(bf16)));
    int32_t *labels = static_cast<int32_t *>(sc.alloc((size_t)h->K * 128 * sizeof(int32_t)));
    float *out = static_cast<float *>(sc.alloc((n_state + h->K) * sizeof(float)));
    if (!prm || !x || !labels || !out) return COCOD_ERR_OOM;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(prm, 0, n_state * sizeof(bf16), s) != cudaSuccess ||
        cudaMemsetAsync(x, 0, (size_t)h->K * 128 * 64 * sizeof(bf16), s) != cudaSuccess ||
        cudaMemsetAsync(labels, 0, (size_t)h->K * 128 * sizeof(int32_t), s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    const uint64_t uK = h->K, uB = 128, uh = h->d_h, ui = h->d_in, uP = h->P;
    CUtensorMap k_x, k_w1, k_w2, mn_w2, k_w3;
    if (!make_map(&k_w3, prm + h->oW3, uh, 10, uK, uh, uP, NEXT_N) || !map_k(&k_x, x, ui, uB, uK, ui, uB * ui) ||
        !map_k(&k_w1, prm + h->oW1, ui, uh, uK, ui, uP) || !map_k(&k_w2, prm + h->oW2, uh, uh, uK, uh, uP) ||
        !map_mn(&mn_w2, prm + h->oW2, uh, uh, uK, uh, uP))
        return COCOD_ERR_CUDA;
    ChainParams c{};
    c.d_in = h->d_in; c.d_h = h->d_h; c.d_out = h->d_out;
    c.P = h->P; c.P_raw = h->P_raw; c.oW3 = h->oW3; c.ob1 = h->ob1; c.ob2 = h->ob2; c.ob3 = h->ob3;
    c.params = prm; c.labels = labels; c.loss = out + n_state; c.grads = out; c.error_flag = h->error_flag;
    c.logit_part = h->logit_part; c.sync = h->chain_sync;
    c.wait_ns = (unsigned long long)wait_ms * 1000000ull;
    c.debug_no_arrive = 1;
    int n = 0;
    if (launch_chain<10>(k_x, k_w1, h->k_h1, k_w2, k_w3, h->k_dz2, mn_w2, h->st_dz1, c, h->d_h / 128, h->K, s, false, &n) != cudaSuccess)
        return COCOD_ERR_CUDA;
    int f = 0;
    if (cudaMemcpyAsync(&f, h->error_flag, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return COCOD_ERR_CUDA;
    return f ? COCOD_ERR_TIMEOUT : COCOD_OK;
}

}  // extern "C"
