// Small coefficient-side kernels around the step kernels: forecasts of the principal
// coefficients by predictors other than the EMA (Sec. 5.3, Fig. 4(b)), singular values from the
// calibration spectrum (Eq. 7) and the left factors of Eq. 8.  All of it is N x k work -- a few
// per cent of the bytes a step moves.
#include "internal.cuh"

namespace svdc {

namespace {

constexpr int kMaxOrder = 7;

struct ForecastArgs {
    const float *hist[kMaxOrder + 1];   // block 0's coefficient arrays, newest first
    float w[kMaxOrder + 1];             // weight of each
    size_t hist_stride;                 // bytes between blocks in every history array
    char *out;                          // block 0's forecast buffer: fp32 | hi | lo
    size_t out_stride;
    size_t hi_off, lo_off;
    int64_t n;                          // N * k
    int order, split;
};

// out = sum_j w_j hist_j, and (bf16 mode) its split pair for the tensor-core cached step
__global__ void __launch_bounds__(256) forecast_kernel(const ForecastArgs a) {
    const int b = blockIdx.y;
    float *o32 = reinterpret_cast<float *>(a.out + (size_t)b * a.out_stride);
    __nv_bfloat16 *ohi = reinterpret_cast<__nv_bfloat16 *>(a.out + (size_t)b * a.out_stride + a.hi_off);
    __nv_bfloat16 *olo = reinterpret_cast<__nv_bfloat16 *>(a.out + (size_t)b * a.out_stride + a.lo_off);
    for (int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; e < a.n; e += (int64_t)gridDim.x * blockDim.x * 4) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j <= a.order; ++j) {
            const float4 h = *reinterpret_cast<const float4 *>(
                reinterpret_cast<const char *>(a.hist[j]) + (size_t)b * a.hist_stride + (size_t)e * 4);
            acc.x = fmaf(a.w[j], h.x, acc.x); acc.y = fmaf(a.w[j], h.y, acc.y);
            acc.z = fmaf(a.w[j], h.z, acc.z); acc.w = fmaf(a.w[j], h.w, acc.w);
        }
        *reinterpret_cast<float4 *>(o32 + e) = acc;
        if (a.split) {
            __nv_bfloat16 hi[4], lo[4];
            split_bf16(acc.x, hi[0], lo[0]); split_bf16(acc.y, hi[1], lo[1]);
            split_bf16(acc.z, hi[2], lo[2]); split_bf16(acc.w, hi[3], lo[3]);
            *reinterpret_cast<uint2 *>(ohi + e) = *reinterpret_cast<const uint2 *>(hi);
            *reinterpret_cast<uint2 *>(olo + e) = *reinterpret_cast<const uint2 *>(lo);
        }
    }
}

__global__ void sigma_kernel(const double *lambda, int k, double *sigma) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < k) sigma[i] = lambda[i] > 0.0 ? sqrt(lambda[i]) : 0.0;
}

__global__ void __launch_bounds__(256) left_factors_kernel(const float *C, const double *sigma, int64_t n, int k, float *U) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        const double s = sigma[e % k];
        U[e] = s > 0.0 ? (float)((double)C[e] / s) : 0.0f;
    }
}

// similarity (Fig. 1(b)) of the columns j of two D x k bases (one CTA per column, fixed reduction order)
__global__ void __launch_bounds__(256) column_cosines_kernel(const float *A, const float *B, int D, int k, double *out) {
    __shared__ double part[256];
    const int j = blockIdx.x;
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int d = threadIdx.x; d < D; d += 256) {
        const double a = (double)A[(size_t)d * k + j], b = (double)B[(size_t)d * k + j];
        ab += a * b; aa += a * a; bb += b * b;
    }
    double r[3] = {ab, aa, bb};
    for (int q = 0; q < 3; ++q) {
        part[threadIdx.x] = r[q];
        __syncthreads();
        for (int sft = 128; sft > 0; sft >>= 1) {
            if ((int)threadIdx.x < sft) part[threadIdx.x] += part[threadIdx.x + sft];
            __syncthreads();
        }
        r[q] = part[0];
        __syncthreads();
    }
    if (threadIdx.x == 0) {   // cosine similarity (in magnitude: singular vectors are sign-free) x magnitude similarity
        const double na = sqrt(r[1]), nb = sqrt(r[2]);
        out[j] = (na > 0.0 && nb > 0.0) ? fabs(r[0]) / (na * nb) * (na < nb ? na / nb : nb / na) : 0.0;
    }
}

}  // namespace

int column_cosines_launch(const float *A, const float *B, int D, int k, double *out, cudaStream_t s) {
    column_cosines_kernel<<<k, 256, 0, s>>>(A, B, D, k, out);
    count_launch();
    return check_last_launch();
}

ForecastLayout forecast_layout(int64_t N, int k) {
    ForecastLayout L;
    L.f32 = 0;
    L.hi = align_up((size_t)N * k * 4, kAlign);
    L.lo = L.hi + align_up((size_t)N * k * 2, kAlign);
    L.total = L.lo + align_up((size_t)N * k * 2, kAlign);
    return L;
}

// Weights of the history (newest first) for a cached step u = s / interval intervals past the
// newest full step.  Backward differences D^i = sum_j (-1)^j binom(i, j) c_{n-j}; the forecast is
// sum_i g_i(u) D^i with g_i = u^i / i! (Taylor form) or u (u+1) ... (u+i-1) / i! (Newton's
// backward-difference formula), so w_j = (-1)^j sum_{i >= j} g_i(u) binom(i, j).
int forecast_weights(int predictor, int order, double u, double *w) {
    if (order < 0 || order > kMaxOrder) return SVDCACHE_ERR_INVALID_ARG;
    if (predictor != SVDCACHE_PREDICT_TAYLOR && predictor != SVDCACHE_PREDICT_NEWTON) return SVDCACHE_ERR_INVALID_ARG;
    double g[kMaxOrder + 1];
    g[0] = 1.0;
    for (int i = 1; i <= order; ++i)
        g[i] = g[i - 1] * (predictor == SVDCACHE_PREDICT_TAYLOR ? u : u + (double)(i - 1)) / (double)i;
    for (int j = 0; j <= order; ++j) {
        double acc = 0.0, binom = 1.0;               // binom(i, j), starting at i = j
        for (int i = j; i <= order; ++i) {
            acc += g[i] * binom;
            binom = binom * (double)(i + 1) / (double)(i + 1 - j);
        }
        w[j] = (j & 1) ? -acc : acc;
    }
    return SVDCACHE_OK;
}

int forecast_launch(const float *const *hist, size_t hist_stride, const double *w, int order, int64_t N, int k,
                    int dtype, int nblocks, void *out, size_t out_stride, cudaStream_t s) {
    ForecastArgs a{};
    for (int j = 0; j <= order; ++j) { a.hist[j] = hist[j]; a.w[j] = (float)w[j]; }
    const ForecastLayout L = forecast_layout(N, k);
    a.hist_stride = hist_stride; a.out = (char *)out; a.out_stride = out_stride;
    a.hi_off = L.hi; a.lo_off = L.lo;
    a.n = N * k; a.order = order; a.split = dtype == SVDCACHE_BF16;
    int64_t gx = (a.n / 4 + 255) / 256;
    if (gx > 2048) gx = 2048;
    if (gx < 1) gx = 1;
    forecast_kernel<<<dim3((unsigned)gx, (unsigned)nblocks), 256, 0, s>>>(a);
    count_launch();
    return check_last_launch();
}

int sigma_launch(const double *lambda, int k, double *sigma, cudaStream_t s) {
    sigma_kernel<<<(k + 127) / 128, 128, 0, s>>>(lambda, k, sigma);
    count_launch();
    return check_last_launch();
}

int left_factors_launch(const float *C, const double *sigma, int64_t N, int k, float *U, cudaStream_t s) {
    const int64_t n = N * k;
    int64_t gx = (n + 255) / 256;
    if (gx > 4096) gx = 4096;
    left_factors_kernel<<<(unsigned)gx, 256, 0, s>>>(C, sigma, n, k, U);
    count_launch();
    return check_last_launch();
}

}  // namespace svdc
