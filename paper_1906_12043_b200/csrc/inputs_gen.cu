// libcocod_inputs.so: device build of the seeded synthetic-input generator.
//
// This is NOT part of the CoCoD-SGD path: it only fills buffers with the Gaussian inputs the
// method consumes (initial point, per-(worker, step) gradients, MLP minibatches).  It repeats,
// operation for operation, the recipe of paper_1906_12043_b200/inputs.py: a 64-bit mixer per
// element, then Box-Muller whose ln and cos are fixed polynomials evaluated only with IEEE
// double add / multiply / divide / sqrt (round-to-nearest intrinsics, never contracted into
// fused multiply-adds), so host and device return identical bits.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

__device__ __forceinline__ double mul(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ double add(double a, double b) { return __dadd_rn(a, b); }

struct Coef {
    double ln[11];    // 1/(2n+1), n = 10..0
    double sn[8];     // (-1)^n/(2n+1)!, n = 7..0
    double cs[9];     // (-1)^n/(2n)!,   n = 8..0
};

__device__ double std_normal(unsigned long long h, const Coef &C)
{
    const unsigned long long a = (h >> 32) + 1ULL;       // 1 .. 2^32
    const unsigned int b = (unsigned int)(h & 0xFFFFFFFFULL);
    // ln(a / 2^32): a = f * 2^E, f in [0.5, 1)
    int E = 64 - __clzll((long long)a);
    double f = mul((double)a, __longlong_as_double((long long)(1023 - E) << 52));
    if (f < 0.7071067811865476) { f = mul(f, 2.0); E -= 1; }
    const double s = __ddiv_rn(add(f, -1.0), add(f, 1.0));
    const double s2 = mul(s, s);
    double p = C.ln[0];
#pragma unroll
    for (int i = 1; i < 11; ++i) p = add(mul(p, s2), C.ln[i]);
    const double ln_f = mul(mul(2.0, s), p);
    const double ln_u1 = add(mul((double)(E - 32), 0.6931471805599453), ln_f);
    const double r = __dsqrt_rn(mul(-2.0, ln_u1));
    // cos(2 pi b / 2^32): octant o, remainder rem / 2^29 of an octant
    const int o = (int)(b >> 29);
    int rem = (int)(b & ((1u << 29) - 1u));
    if (o & 1) rem = (1 << 29) - rem;
    const double y = mul(mul((double)rem, 1.0 / 536870912.0), 0.7853981633974483);
    const double y2 = mul(y, y);
    double c;
    if (o == 1 || o == 2 || o == 5 || o == 6) {
        double q = C.sn[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) q = add(mul(q, y2), C.sn[i]);
        c = mul(q, y);
    } else {
        double q = C.cs[0];
#pragma unroll
        for (int i = 1; i < 9; ++i) q = add(mul(q, y2), C.cs[i]);
        c = q;
    }
    if (o >= 2 && o <= 5) c = -c;
    return mul(r, c);
}

template <typename T> __device__ __forceinline__ T narrow(float v);
template <> __device__ __forceinline__ float narrow<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 narrow<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256)
gaussian_kernel(T *out, unsigned long long key, long long p0, long long n, double sigma, Coef C)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride) {
        const unsigned long long p = (unsigned long long)(p0 + j);
        const unsigned long long h = mix64(key + (p + 1ULL) * 0x9E3779B97F4A7C15ULL);
        out[j] = narrow<T>(__double2float_rn(mul(sigma, std_normal(h, C))));
    }
}

Coef make_coef()
{
    // the same doubles inputs.py builds: 1.0 / (2n+1) and (+-1.0) / n! with n! accumulated in double
    Coef C;
    double fact[18];
    fact[0] = 1.0;
    for (int i = 1; i < 18; ++i) fact[i] = fact[i - 1] * (double)i;
    for (int k = 0; k < 11; ++k) { int n = 10 - k; C.ln[k] = 1.0 / (double)(2 * n + 1); }
    for (int k = 0; k < 8; ++k) { int n = 7 - k; C.sn[k] = ((n & 1) ? -1.0 : 1.0) / fact[2 * n + 1]; }
    for (int k = 0; k < 9; ++k) { int n = 8 - k; C.cs[k] = ((n & 1) ? -1.0 : 1.0) / fact[2 * n]; }
    return C;
}

template <typename T>
int run(void *out, uint64_t key, int64_t p0, int64_t n, double sigma, void *stream)
{
    if (n <= 0) return 0;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    gaussian_kernel<T><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
        (T *)out, key, p0, n, sigma, make_coef());
    return (int)cudaGetLastError();
}

}  // namespace

extern "C" {

// Fill out[0..n) (device) with float32(sigma * Z(key, p0 + j)).  Returns a cudaError_t.
int cocod_inputs_gaussian_f32(void *out, uint64_t key, int64_t p0, int64_t n, double sigma, void *stream)
{
    return run<float>(out, key, p0, n, sigma, stream);
}

// Same values rounded once more to bfloat16 (round to nearest even).
int cocod_inputs_gaussian_bf16(void *out, uint64_t key, int64_t p0, int64_t n, double sigma, void *stream)
{
    return run<__nv_bfloat16>(out, key, p0, n, sigma, stream);
}

}  // extern "C"
