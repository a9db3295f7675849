// Per-worker mini-batch gradients of the 3-layer ReLU MLP (Algorithm 1, Step II: "compute a
// mini-batch stochastic gradient"), batched over the K workers.  Declared in include/cocod_mlp.h.
//
// Data flow of one call (every matrix below exists once per worker; "T" = stored transposed so
// that each tensor-core contraction sees both operands with the reduction index contiguous):
//
//   xT  = transpose(x)                                    w2T = transpose(W2)
//   h1, h1T  = bf16(relu(x  W1^T + b1))        GEMM 128 x d_h x d_in    epilogue bias+ReLU
//   h2       = bf16(relu(h1 W2^T + b2))        GEMM 128 x d_h x d_h     epilogue bias+ReLU
//   logits = h2 W3^T + b3 ; loss ; dz3 = bf16((softmax - onehot)/batch)        CUDA cores
//   dW3 = dz3^T h2 ; db3 = colsum dz3                                           CUDA cores
//   dz2, dz2T = bf16((dz3 W3) * (h2 > 0)) ; db2 = colsum dz2                    CUDA cores
//   dz1T     = bf16((dz2 W2) * (h1 > 0))       GEMM 128 x d_h x d_h (B = w2T)  epilogue mask
//   db1 = rowsum dz1T                                                           CUDA cores
//   dW2 = dz2T h1T^T                           GEMM d_h x d_h x 128            epilogue fp32
//   dW1 = dz1T xT^T                            GEMM d_h x d_in x 128           epilogue fp32
#include "cocod_mlp.h"
#include "cocod_gemm_sm100.cuh"

#include <cstdio>
#include <new>

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

// 3-D map over a batched K-major bf16 matrix: dims {cols (contiguous), rows, workers}; one box is
// a 64-column x 128-row tile of one worker, stored with the 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t workers, uint64_t ld,
              uint64_t worker_stride)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    const cuuint64_t dims[3] = {cols, rows, workers};
    const cuuint64_t strides[2] = {ld * sizeof(bf16), worker_stride * sizeof(bf16)};
    const cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)BM, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int EPI>
cudaError_t launch_gemm(const CUtensorMap &a, const CUtensorMap &b, const Params &p, int workers, cudaStream_t s)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tn_bf16<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const dim3 grid((p.N + BN - 1) / BN, (p.M + BM - 1) / BM, workers);
    gemm_tn_bf16<EPI><<<grid, 128, SMEM_BYTES, s>>>(a, b, p);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ small kernels
// out[w][c][r] = in[w][r][c]; 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256)
transpose_bf16(const bf16 *__restrict__ in, bf16 *__restrict__ out, int R, int C, long long in_ld,
               long long in_worker_stride, long long out_worker_stride)
{
    __shared__ bf16 tile[32][33];
    const bf16 *src = in + (long long)blockIdx.z * in_worker_stride;
    bf16 *dst = out + (long long)blockIdx.z * out_worker_stride;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        if (r < R && c < C) tile[i][tx] = src[(long long)r * in_ld + c];
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;
        if (r < R && c < C) dst[(long long)c * R + r] = tile[tx][i];
    }
}

// One warp per (worker, sample): logits = h2 W3^T + b3 (fp32), row loss, dz3 = bf16((softmax - onehot)/batch)
// kept as fp32 values in dz3[w][b][16].
__global__ void __launch_bounds__(256)
head_logits(const bf16 *__restrict__ h2, const bf16 *__restrict__ params, long long P, long long oW3, long long ob3,
            const int *__restrict__ labels, float *__restrict__ dz3, float *__restrict__ rowloss, int B, int d_h,
            int d_out)
{
    const int gw = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int w = gw / B, b = gw % B;
    const bf16 *hrow = h2 + ((long long)w * B + b) * d_h;
    const bf16 *W3 = params + (long long)w * P + oW3;
    float acc[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) acc[c] = 0.0f;
    for (int j = lane; j < d_h; j += 32) {
        const float h = __bfloat162float(hrow[j]);
#pragma unroll
        for (int c = 0; c < 16; ++c)
            if (c < d_out) acc[c] = fmaf(h, __bfloat162float(W3[(long long)c * d_h + j]), acc[c]);
    }
#pragma unroll
    for (int c = 0; c < 16; ++c)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
    if (lane == 0) {
        const bf16 *b3 = params + (long long)w * P + ob3;
        float z[16], zmax = -INFINITY;
        for (int c = 0; c < d_out; ++c) {
            z[c] = acc[c] + __bfloat162float(b3[c]);
            zmax = fmaxf(zmax, z[c]);
        }
        float s = 0.0f;
        for (int c = 0; c < d_out; ++c) {
            z[c] = expf(z[c] - zmax);
            s += z[c];
        }
        const int y = labels[(long long)w * B + b];
        const float inv = 1.0f / s, invB = 1.0f / (float)B;
        float lz = 0.0f;
        for (int c = 0; c < 16; ++c) {
            float d = 0.0f;
            if (c < d_out) {
                const float pc = z[c] * inv;
                if (c == y) lz = pc;
                d = __bfloat162float(__float2bfloat16_rn((pc - (c == y ? 1.0f : 0.0f)) * invB));
            }
            dz3[((long long)w * B + b) * 16 + c] = d;
        }
        rowloss[(long long)w * B + b] = -logf(lz);
    }
}

// dW3[c][j] = sum_b dz3[b][c] h2[b][j]; db3[c] = sum_b dz3[b][c]; loss[w] = mean_b rowloss; the
// gradient's zero padding.  grid (d_h / 256, K).
__global__ void __launch_bounds__(256)
head_dw3(const bf16 *__restrict__ h2, const float *__restrict__ dz3, const float *__restrict__ rowloss,
         float *__restrict__ grads, float *__restrict__ loss, long long P, long long P_raw, long long oW3,
         long long ob3, int B, int d_h, int d_out)
{
    __shared__ float sdz[128 * 16];
    const int w = blockIdx.y, j = blockIdx.x * 256 + threadIdx.x;
    for (int i = threadIdx.x; i < B * 16; i += 256) sdz[i] = dz3[(long long)w * B * 16 + i];
    __syncthreads();
    float acc[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) acc[c] = 0.0f;
    if (j < d_h) {
        const bf16 *col = h2 + (long long)w * B * d_h + j;
        for (int b = 0; b < B; ++b) {
            const float h = __bfloat162float(col[(long long)b * d_h]);
#pragma unroll
            for (int c = 0; c < 16; ++c) acc[c] = fmaf(sdz[b * 16 + c], h, acc[c]);
        }
        float *g = grads + (long long)w * P + oW3;
#pragma unroll
        for (int c = 0; c < 16; ++c)
            if (c < d_out) g[(long long)c * d_h + j] = acc[c];
    }
    if (blockIdx.x == 0) {
        if (threadIdx.x < d_out) {
            float s = 0.0f;
            for (int b = 0; b < B; ++b) s += sdz[b * 16 + threadIdx.x];
            grads[(long long)w * P + ob3 + threadIdx.x] = s;
        }
        if (threadIdx.x == 32) {
            float s = 0.0f;
            for (int b = 0; b < B; ++b) s += rowloss[(long long)w * B + b];
            loss[w] = s / (float)B;
        }
        for (long long i = P_raw + threadIdx.x; i < P; i += 256) grads[(long long)w * P + i] = 0.0f;
    }
}

// dz2[b][j] = bf16((sum_c dz3[b][c] W3[c][j]) * (h2[b][j] > 0)); also dz2T[j][b] and db2[j] = sum_b dz2[b][j].
// One CTA = 32 columns j x all 128 samples.  grid (d_h / 32, K).
__global__ void __launch_bounds__(256)
head_dz2(const bf16 *__restrict__ h2, const bf16 *__restrict__ params, const float *__restrict__ dz3,
         bf16 *__restrict__ dz2, bf16 *__restrict__ dz2T, float *__restrict__ grads, long long P, long long oW3,
         long long ob2, int B, int d_h, int d_out)
{
    __shared__ float sdz[128 * 16];
    __shared__ bf16 tile[32][128 + 8];
    const int w = blockIdx.y, j0 = blockIdx.x * 32, lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < B * 16; i += 256) sdz[i] = dz3[(long long)w * B * 16 + i];
    const int j = j0 + lane;
    float w3[16];
#pragma unroll
    for (int c = 0; c < 16; ++c)
        w3[c] = (c < d_out) ? __bfloat162float(params[(long long)w * P + oW3 + (long long)c * d_h + j]) : 0.0f;
    __syncthreads();
    for (int b = wp; b < B; b += 8) {
        float a = 0.0f;
#pragma unroll
        for (int c = 0; c < 16; ++c) a = fmaf(sdz[b * 16 + c], w3[c], a);
        const long long e = ((long long)w * B + b) * d_h + j;
        const bf16 v = __float2bfloat16_rn(__bfloat162float(h2[e]) > 0.0f ? a : 0.0f);
        dz2[e] = v;
        tile[lane][b] = v;
    }
    __syncthreads();
    // transposed rows: 32 rows x 128 samples, 16 bytes per thread
    for (int i = threadIdx.x; i < 32 * (B / 8); i += 256) {
        const int r = i / (B / 8), q = i % (B / 8);
        *reinterpret_cast<uint4 *>(dz2T + ((long long)w * d_h + j0 + r) * B + q * 8) =
            *reinterpret_cast<const uint4 *>(&tile[r][q * 8]);
    }
    if (threadIdx.x < 32) {
        float s = 0.0f;
        for (int b = 0; b < B; ++b) s += __bfloat162float(tile[threadIdx.x][b]);
        grads[(long long)w * P + ob2 + j0 + threadIdx.x] = s;
    }
}

// db1[j] = sum_b dz1T[j][b]: one warp per row, fixed summation order.
__global__ void __launch_bounds__(256)
rowsum_bf16(const bf16 *__restrict__ dzT, float *__restrict__ grads, long long P, long long ob, int B, int d_h)
{
    const int w = blockIdx.y, j = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (j >= d_h) return;
    const bf16 *row = dzT + ((long long)w * d_h + j) * B;
    float s = 0.0f;
    for (int b = lane; b < B; b += 32) s += __bfloat162float(row[b]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) grads[(long long)w * P + ob + j] = s;
}

}  // namespace

struct cocod_mlp {
    int K, B, d_in, d_h, d_out;
    long long P, P_raw, oW1, ob1, oW2, ob2, oW3, ob3;
    bf16 *xT = nullptr, *h1 = nullptr, *h1T = nullptr, *h2 = nullptr, *dz2 = nullptr, *dz2T = nullptr,
         *dz1T = nullptr, *w2T = nullptr;
    float *dz3 = nullptr, *rowloss = nullptr;
    int *error_flag = nullptr;
    CUtensorMap m_h1, m_dz2, m_w2T, m_dz2T, m_h1T, m_dz1T, m_xT;      // maps over scratch (fixed addresses)
    long long launches = 0;
};

namespace {

void mlp_free(cocod_mlp *h)
{
    void *ptrs[] = {h->xT, h->h1, h->h1T, h->h2, h->dz2, h->dz2T, h->dz1T, h->w2T, h->dz3, h->rowloss, h->error_flag};
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
    alloc((void **)&h->xT, (size_t)K * batch * d_in * sizeof(bf16));
    alloc((void **)&h->h1, act);
    alloc((void **)&h->h1T, act);
    alloc((void **)&h->h2, act);
    alloc((void **)&h->dz2, act);
    alloc((void **)&h->dz2T, act);
    alloc((void **)&h->dz1T, act);
    alloc((void **)&h->w2T, (size_t)K * d_hidden * d_hidden * sizeof(bf16));
    alloc((void **)&h->dz3, (size_t)K * batch * 16 * sizeof(float));
    alloc((void **)&h->rowloss, (size_t)K * batch * sizeof(float));
    alloc((void **)&h->error_flag, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(h->error_flag, 0, sizeof(int));
    if (e != cudaSuccess) {
        cudaGetLastError();
        mlp_free(h);
        return e == cudaErrorMemoryAllocation ? COCOD_ERR_OOM : COCOD_ERR_CUDA;
    }
    const uint64_t uK = K, uB = batch, uh = d_hidden, ui = d_in;
    bool ok = make_map(&h->m_h1, h->h1, uh, uB, uK, uh, uB * uh)           // [B][d_h]
              && make_map(&h->m_dz2, h->dz2, uh, uB, uK, uh, uB * uh)      // [B][d_h]
              && make_map(&h->m_w2T, h->w2T, uh, uh, uK, uh, uh * uh)      // [d_h in][d_h out]
              && make_map(&h->m_dz2T, h->dz2T, uB, uh, uK, uB, uh * uB)    // [d_h][B]
              && make_map(&h->m_h1T, h->h1T, uB, uh, uK, uB, uh * uB)      // [d_h][B]
              && make_map(&h->m_dz1T, h->dz1T, uB, uh, uK, uB, uh * uB)    // [d_h][B]
              && make_map(&h->m_xT, h->xT, uB, ui, uK, uB, ui * uB);       // [d_in][B]
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

int cocod_mlp_grad(cocod_mlp_handle *h, const void *params_bf16, const void *x, const int32_t *labels, float *grads,
                   float *loss, cocod_stream_t stream)
{
    if (!h || !params_bf16 || !x || !labels || !grads || !loss) return COCOD_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(params_bf16) & 15u) || (reinterpret_cast<uintptr_t>(x) & 15u))
        return COCOD_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    const bf16 *prm = static_cast<const bf16 *>(params_bf16);
    const bf16 *xin = static_cast<const bf16 *>(x);
    const int K = h->K, B = h->B, d_in = h->d_in, d_h = h->d_h, d_out = h->d_out;
    const long long P = h->P;
    // maps over caller memory: x [B][d_in], W1 [d_h][d_in], W2 [d_h][d_h]
    CUtensorMap m_x, m_w1, m_w2;
    if (!make_map(&m_x, xin, d_in, B, K, d_in, (uint64_t)B * d_in) ||
        !make_map(&m_w1, prm + h->oW1, d_in, d_h, K, d_in, P) ||
        !make_map(&m_w2, prm + h->oW2, d_h, d_h, K, d_h, P))
        return COCOD_ERR_CUDA;
#define LAUNCH_OK() do { if (cudaGetLastError() != cudaSuccess) return COCOD_ERR_CUDA; ++h->launches; } while (0)
    // transposed copies: xT [d_in][B], w2T [d_h in][d_h out]
    transpose_bf16<<<dim3((d_in + 31) / 32, (B + 31) / 32, K), 256, 0, s>>>(xin, h->xT, B, d_in, d_in,
                                                                            (long long)B * d_in, (long long)B * d_in);
    LAUNCH_OK();
    transpose_bf16<<<dim3(d_h / 32, d_h / 32, K), 256, 0, s>>>(prm + h->oW2, h->w2T, d_h, d_h, d_h, P,
                                                               (long long)d_h * d_h);
    LAUNCH_OK();
    Params p{};
    p.error_flag = h->error_flag;
    // h1 = relu(x W1^T + b1)
    p.M = B; p.N = d_h; p.K = d_in;
    p.o = h->h1; p.oT = h->h1T; p.o_worker_stride = (long long)B * d_h;
    p.bias = prm + h->ob1; p.bias_worker_stride = P;
    if (launch_gemm<EPI_BIAS_RELU>(m_x, m_w1, p, K, s) != cudaSuccess) return COCOD_ERR_CUDA;
    ++h->launches;
    // h2 = relu(h1 W2^T + b2)
    p.K = d_h; p.o = h->h2; p.oT = nullptr; p.bias = prm + h->ob2;
    if (launch_gemm<EPI_BIAS_RELU>(h->m_h1, m_w2, p, K, s) != cudaSuccess) return COCOD_ERR_CUDA;
    ++h->launches;
    // output layer, loss, dz3, dW3, db3, dz2, db2
    head_logits<<<K * B / 8, 256, 0, s>>>(h->h2, prm, P, h->oW3, h->ob3, labels, h->dz3, h->rowloss, B, d_h, d_out);
    LAUNCH_OK();
    head_dw3<<<dim3((d_h + 255) / 256, K), 256, 0, s>>>(h->h2, h->dz3, h->rowloss, grads, loss, P, h->P_raw, h->oW3,
                                                        h->ob3, B, d_h, d_out);
    LAUNCH_OK();
    head_dz2<<<dim3(d_h / 32, K), 256, 0, s>>>(h->h2, prm, h->dz3, h->dz2, h->dz2T, grads, P, h->oW3, h->ob2, B, d_h,
                                               d_out);
    LAUNCH_OK();
    // dz1T = ((dz2 W2) * (h1 > 0))^T
    Params q{};
    q.error_flag = h->error_flag;
    q.M = B; q.N = d_h; q.K = d_h;
    q.o = nullptr; q.oT = h->dz1T; q.o_worker_stride = (long long)B * d_h;
    q.mask = h->h1; q.mask_worker_stride = (long long)B * d_h;
    if (launch_gemm<EPI_MASK>(h->m_dz2, h->m_w2T, q, K, s) != cudaSuccess) return COCOD_ERR_CUDA;
    ++h->launches;
    rowsum_bf16<<<dim3((d_h + 7) / 8, K), 256, 0, s>>>(h->dz1T, grads, P, h->ob1, B, d_h);
    LAUNCH_OK();
    // dW2 = dz2T h1T^T, dW1 = dz1T xT^T
    Params r{};
    r.error_flag = h->error_flag;
    r.M = d_h; r.N = d_h; r.K = B;
    r.c = grads + h->oW2; r.c_worker_stride = P; r.ldc = d_h;
    if (launch_gemm<EPI_F32>(h->m_dz2T, h->m_h1T, r, K, s) != cudaSuccess) return COCOD_ERR_CUDA;
    ++h->launches;
    r.N = d_in; r.c = grads + h->oW1; r.ldc = d_in;
    if (launch_gemm<EPI_F32>(h->m_dz1T, h->m_xT, r, K, s) != cudaSuccess) return COCOD_ERR_CUDA;
    ++h->launches;
#undef LAUNCH_OK
    return COCOD_OK;
}

int cocod_mlp_check(cocod_mlp_handle *h, cocod_stream_t stream)
{
    if (!h) return COCOD_ERR_INVALID;
    int flag = 0;
    if (cudaMemcpyAsync(&flag, h->error_flag, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return COCOD_ERR_CUDA;
    return flag ? COCOD_ERR_TIMEOUT : COCOD_OK;
}

int cocod_gemm_tn_bf16(const void *A, const void *B, float *C, int M, int N, int Kd, int batch_count, int64_t lda,
                       int64_t ldb, int64_t ldc, int64_t stride_a, int64_t stride_b, int64_t stride_c,
                       cocod_stream_t stream)
{
    if (!A || !B || !C || M < 1 || N < 1 || Kd < 1 || batch_count < 1 || batch_count > 65535) return COCOD_ERR_INVALID;
    if ((lda % 8) || (ldb % 8) || (stride_a % 8) || (stride_b % 8) || lda < Kd || ldb < Kd || ldc < N)
        return COCOD_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(A) & 15u) || (reinterpret_cast<uintptr_t>(B) & 15u)) return COCOD_ERR_INVALID;
    CUtensorMap ma, mb;
    const uint64_t sa = batch_count > 1 ? (uint64_t)stride_a : (uint64_t)M * lda;
    const uint64_t sb = batch_count > 1 ? (uint64_t)stride_b : (uint64_t)N * ldb;
    if (!make_map(&ma, A, Kd, M, batch_count, lda, sa) || !make_map(&mb, B, Kd, N, batch_count, ldb, sb))
        return COCOD_ERR_CUDA;
    static int *flag = nullptr;
    if (!flag) {
        if (cudaMalloc((void **)&flag, sizeof(int)) != cudaSuccess) return COCOD_ERR_OOM;
        cudaMemset(flag, 0, sizeof(int));
    }
    Params p{};
    p.M = M; p.N = N; p.K = Kd;
    p.c = C; p.c_worker_stride = stride_c; p.ldc = (int)ldc;
    p.error_flag = flag;
    if (launch_gemm<EPI_F32>(ma, mb, p, batch_count, (cudaStream_t)stream) != cudaSuccess) return COCOD_ERR_CUDA;
    int f = 0;
    if (cudaMemcpyAsync(&f, flag, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return COCOD_ERR_CUDA;
    if (f) {
        cudaMemset(flag, 0, sizeof(int));
        return COCOD_ERR_TIMEOUT;
    }
    return COCOD_OK;
}

}  // extern "C"
