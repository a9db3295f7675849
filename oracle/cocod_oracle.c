/*
 * CPU oracle for the CoCoD-SGD parameter engine -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, sequential restatement of Algorithm 1 of the paper ("CoCoD-SGD") with the
 * optimizer its experiments use (Section 5.1, "Hyper-parameters": momentum 0.9 and weight
 * decay under PyTorch's SGD).  Only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it; the CUDA library never does and shares no code with it.
 *
 * Notation follows the paper: K workers (the paper's N), P parameters per worker (the
 * paper's d), period k (local steps per round), gamma = lr.  All matrices are worker-major
 * row-major K x P with row stride P: row i is worker i's flattened model x^i.
 *
 * Three numeric modes, one function each:
 *   *_ref    the parity target.  State is STORED in fp32 (the workloads say "fp32 params,
 *            fp32 momentum"); every stored value is evaluated in fp64 from the fp32 operands
 *            and rounded once.
 *   *_f64    state stored in fp64 as well (used by the pins; shows what fp32 storage costs).
 *   *_mirror pure fp32 arithmetic in exactly the operation order written here, with a fused
 *            multiply-add wherever "a*b + c" is written (fmaf is correctly rounded on every
 *            IEEE machine).  A device kernel that performs the same fp32 operations in the
 *            same order must agree bit for bit, so any differing element is an indexing or
 *            race bug rather than rounding.
 *
 * Every pin that ties these functions to something other than themselves lives in
 * tests/test_oracle_pins.py; no function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;

/* Number of host threads the loops below use (they are embarrassingly parallel over the
 * parameter index; the arithmetic per element does not depend on the thread count). */
void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int oracle_get_threads(void) { return g_threads; }

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ Step II: local update
 * Algorithm 1, Step II body: x_{tau+1}^i = x_tau^i - gamma * G_tau^i, generalised to the
 * optimizer of Section 5.1 (momentum mu, coupled L2 weight decay wd, PyTorch SGD form):
 *     d = g + wd * x ;  v = mu * v + d ;  x = x - lr * v          (v starts at 0)
 * With mu = 0 and wd = 0 this is Algorithm 1's update literally.
 */
void oracle_local_step_ref(int K, int64_t P, float *x, float *v, const float *g,
                           float lr, float mu, float wd)
{
    const int64_t n = (int64_t)K * P;
    const double dlr = lr, dmu = mu, dwd = wd;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double d = (double)g[e] + dwd * (double)x[e];
        float vn = (float)(dmu * (double)v[e] + d);
        v[e] = vn;
        x[e] = (float)((double)x[e] - dlr * (double)vn);
    }
}

void oracle_local_step_f64(int K, int64_t P, double *x, double *v, const double *g,
                           double lr, double mu, double wd)
{
    const int64_t n = (int64_t)K * P;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double d = g[e] + wd * x[e];
        v[e] = mu * v[e] + d;
        x[e] = x[e] - lr * v[e];
    }
}

void oracle_local_step_mirror(int K, int64_t P, float *x, float *v, const float *g,
                              float lr, float mu, float wd)
{
    const int64_t n = (int64_t)K * P;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        float d = fmaf(wd, x[e], g[e]);
        float vn = fmaf(mu, v[e], d);
        v[e] = vn;
        x[e] = fmaf(-lr, vn, x[e]);
    }
}

/* ------------------------------------------------------------------ Step I: store x_t^i
 * Algorithm 1, Step I: every worker keeps a copy of its model x_t^i as it is at iteration t. */
void oracle_snapshot_f32(int K, int64_t P, const float *x, float *snap)
{
    memcpy(snap, x, (size_t)K * (size_t)P * sizeof(float));
}

void oracle_snapshot_f64(int K, int64_t P, const double *x, double *snap)
{
    memcpy(snap, x, (size_t)K * (size_t)P * sizeof(double));
}

/* ------------------------------------------------------------------ Step I: average model
 * Algorithm 1, Step I: x_hat_t = sum_i (M_i / sum_j M_j) x_t^i, taken over the stored copies.
 * M == NULL means equal mini-batch sizes (the homogeneous setting), i.e. the plain mean. */
void oracle_mean_ref(int K, int64_t P, const float *snap, const double *M, float *mean)
{
    double Msum = 0.0;
    if (M) for (int i = 0; i < K; ++i) Msum += M[i];
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        double s = 0.0;
        if (M) {
            for (int i = 0; i < K; ++i) s += (M[i] / Msum) * (double)snap[(int64_t)i * P + p];
        } else {
            for (int i = 0; i < K; ++i) s += (double)snap[(int64_t)i * P + p];
            s /= (double)K;
        }
        mean[p] = (float)s;
    }
}

void oracle_mean_f64(int K, int64_t P, const double *snap, const double *M, double *mean)
{
    double Msum = 0.0;
    if (M) for (int i = 0; i < K; ++i) Msum += M[i];
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        double s = 0.0;
        if (M) {
            for (int i = 0; i < K; ++i) s += (M[i] / Msum) * snap[(int64_t)i * P + p];
        } else {
            for (int i = 0; i < K; ++i) s += snap[(int64_t)i * P + p];
            s /= (double)K;
        }
        mean[p] = s;
    }
}

/* fp32 order of the mirror mode.  Algorithm 1 fixes no summation order for the mean, so the mirror
 * takes the order of the device kernels: workers are taken in blocks of 8 consecutive rows; a block
 * is summed as a balanced pairwise tree ((t0+t1)+(t2+t3))+((t4+t5)+(t6+t7)) in which absent rows are
 * skipped (not added as zeros); block sums are accumulated in block order.  Equal batch sizes:
 * t_i = snap_i and mean = s * (1.0f / K).  Otherwise t_i = w_i * snap_i with
 * w_i = (float)(M_i / sum_j M_j) rounded once from fp64, and mean = s. */
static float tree8_f32(const float *t, int cnt)
{
    float a[4], b[2];
    for (int j = 0; j < 4; ++j) a[j] = (2 * j + 1 < cnt) ? t[2 * j] + t[2 * j + 1] : t[2 * j];
    const int c1 = (cnt + 1) / 2;
    for (int j = 0; j < 2; ++j) b[j] = (2 * j + 1 < c1) ? a[2 * j] + a[2 * j + 1] : a[2 * j];
    const int c2 = (c1 + 1) / 2;
    return (c2 > 1) ? b[0] + b[1] : b[0];
}

void oracle_mean_mirror(int K, int64_t P, const float *snap, const double *M, float *mean)
{
    float w[1024];
    double Msum = 0.0;
    if (M) {
        for (int i = 0; i < K; ++i) Msum += M[i];
        for (int i = 0; i < K && i < 1024; ++i) w[i] = (float)(M[i] / Msum);
    }
    const float invK = 1.0f / (float)K;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        float s = 0.0f;
        for (int i0 = 0; i0 < K; i0 += 8) {
            float t[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            const int cnt = (K - i0 < 8) ? (K - i0) : 8;
            for (int j = 0; j < cnt; ++j) {
                const float v = snap[(int64_t)(i0 + j) * P + p];
                t[j] = M ? w[i0 + j] * v : v;
            }
            const float blk = tree8_f32(t, cnt);
            s = (i0 == 0) ? blk : s + blk;
        }
        mean[p] = M ? s : s * invK;
    }
}

/* ------------------------------------------------------------------ merge
 * Algorithm 1, line 6: x_{t+k}^i = x_hat_t + (x_{t+k}^i - x_t^i): the local drift since the
 * stored copy is taken first, then added to the average. */
void oracle_merge_ref(int K, int64_t P, float *x, const float *snap, const float *mean)
{
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        const double m = (double)mean[p];
        for (int i = 0; i < K; ++i) {
            const int64_t e = (int64_t)i * P + p;
            x[e] = (float)(m + ((double)x[e] - (double)snap[e]));
        }
    }
}

void oracle_merge_f64(int K, int64_t P, double *x, const double *snap, const double *mean)
{
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        for (int i = 0; i < K; ++i) {
            const int64_t e = (int64_t)i * P + p;
            x[e] = mean[p] + (x[e] - snap[e]);
        }
    }
}

void oracle_merge_mirror(int K, int64_t P, float *x, const float *snap, const float *mean)
{
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t p = 0; p < P; ++p) {
        const float m = mean[p];
        for (int i = 0; i < K; ++i) {
            const int64_t e = (int64_t)i * P + p;
            const float drift = x[e] - snap[e];
            x[e] = m + drift;
        }
    }
}
