// The extern "C" surface: argument validation, layout queries, dispatch to the kernels.
#include <atomic>
#include <cstdio>
#include <cmath>
#include <cstring>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "internal.cuh"

namespace svdc {

static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_path{0};
static std::atomic<int> g_last_path{0};
static thread_local char g_cuda_error[256] = "";

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int record_cuda(cudaError_t e) {
    if (e == cudaSuccess) return SVDCACHE_OK;
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return SVDCACHE_ERR_CUDA;
}

int check_last_launch() { return record_cuda(cudaGetLastError()); }

// An NVTX range around an entry point (costs nothing unless a profiler is attached): the kernels
// of a call show up under its name in a timeline.
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_shape(int64_t N, int D, int k, int dtype) {
    if (dtype != SVDCACHE_F32 && dtype != SVDCACHE_BF16) return SVDCACHE_ERR_INVALID_ARG;
    if (N < 1 || D < 8 || D > 16384 || (D % 8) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    if (k < 8 || k > 256 || (k % 8) != 0 || k > D) return SVDCACHE_ERR_BAD_SHAPE;
    return SVDCACHE_OK;
}

static int check_pitch(int64_t ld, int D, int dtype) {
    if (ld < D) return SVDCACHE_ERR_BAD_SHAPE;
    if (((size_t)ld * elem_bytes(dtype)) % 16 != 0) return SVDCACHE_ERR_BAD_ALIGN;
    return SVDCACHE_OK;
}

static int dispatch(const StepArgs &a_in, bool full, cudaStream_t s) {
    StepArgs a = a_in;
    const int want = g_path.load();
    const bool can_umma = umma_supported(a, full);
    if (want == 2 && !can_umma) return SVDCACHE_ERR_BAD_SHAPE;
    const bool use_umma = (want == 2) || (want == 0 && can_umma);
    g_last_path.store(use_umma ? 2 : 1);
    if (use_umma) return full ? umma_full_step(a, s) : umma_cached_step(a, s);
    return full ? simt_full_step(a, s) : simt_cached_step(a, s);
}

__global__ void state_reset_kernel(StateHeader *h, int64_t N, int D, int k, int dtype) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        h->magic = kStateMagic;
        h->dtype = dtype;
        h->N = N;
        h->D = D;
        h->k = k;
        h->full_steps = 0;
        h->status = SVDCACHE_OK;
        h->done = 0;
        h->pad = 0;
        h->exits = 0;
    }
}

}  // namespace svdc

using namespace svdc;

extern "C" {

const char *svdcache_status_string(int status) {
    switch (status) {
        case SVDCACHE_OK: return "ok";
        case SVDCACHE_ERR_INVALID_ARG: return "invalid argument";
        case SVDCACHE_ERR_BAD_SHAPE: return "shape outside the supported limits";
        case SVDCACHE_ERR_BAD_ALIGN: return "pointer or pitch not 16-byte aligned";
        case SVDCACHE_ERR_STATE: return "cached step on a state that has seen no full step";
        case SVDCACHE_ERR_WORKSPACE: return "workspace or buffer too small";
        case SVDCACHE_ERR_TIMEOUT: return "a bounded in-kernel wait ran out";
        case SVDCACHE_ERR_CUDA: return "CUDA call failed";
        case SVDCACHE_ERR_NOT_CONVERGED: return "eigen-solver did not converge";
        case SVDCACHE_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library carries built in";
        default: return "unknown status";
    }
}

const char *svdcache_last_cuda_error(void) { return g_cuda_error; }

uint64_t svdcache_kernel_launches(void) { return g_launches.load(); }
int svdcache_set_path(int path) {
    if (path < 0 || path > 2) return SVDCACHE_ERR_INVALID_ARG;
    return g_path.exchange(path);
}
int svdcache_last_path(void) { return g_last_path.load(); }

int svdcache_selftest_wait_timeout(void *state, int64_t limit_cycles, void *stream) {
    if (!state) return SVDCACHE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(state) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if (limit_cycles < 1 || limit_cycles > 200000000LL) return SVDCACHE_ERR_INVALID_ARG;   // at most ~0.1 s
    return umma_wait_selftest(state, (long long)limit_cycles, (cudaStream_t)stream);
}

/* ----------------------------------------------------------------- calibration --- */

int svdcache_calibrate_workspace_bytes(int D, int k, size_t *bytes) {
    if (!bytes) return SVDCACHE_ERR_INVALID_ARG;
    int rc = check_shape(1, D, k, SVDCACHE_F32);
    if (rc) return rc;
    *bytes = calib_workspace_bytes(D, k);
    return SVDCACHE_OK;
}

static int check_ws(int D, int k, void *ws, size_t bytes) {
    int rc = check_shape(1, D, k, SVDCACHE_F32);
    if (rc) return rc;
    if (!ws) return SVDCACHE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if (bytes < calib_workspace_bytes(D, k)) return SVDCACHE_ERR_WORKSPACE;
    return SVDCACHE_OK;
}

int svdcache_calibrate_begin(int D, int k, void *ws, size_t bytes, void *stream) {
    int rc = check_ws(D, k, ws, bytes);
    if (rc) return rc;
    return calib_begin(D, k, ws, (cudaStream_t)stream);
}

int svdcache_calibrate_accumulate(const void *F, int64_t M, int D, int64_t ld, int dtype, void *ws,
                                  size_t bytes, void *stream) {
    NvtxRange range("svdcache_calibrate_accumulate");
    if (dtype != SVDCACHE_F32 && dtype != SVDCACHE_BF16) return SVDCACHE_ERR_INVALID_ARG;
    if (M < 0 || D < 8 || D > 16384 || (D % 8) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    if (!ws) return SVDCACHE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if (bytes < calib_workspace_bytes(D, 8)) return SVDCACHE_ERR_WORKSPACE;
    if (M == 0) return SVDCACHE_OK;
    if (!F) return SVDCACHE_ERR_INVALID_ARG;
    int rc = check_pitch(ld, D, dtype);
    if (rc) return rc;
    if (!aligned16(F)) return SVDCACHE_ERR_BAD_ALIGN;
    return calib_accumulate(F, M, D, ld, dtype, ws, (cudaStream_t)stream);
}

int svdcache_calibrate_finish(int D, int k, float *Vk, double *lambda, double *trace, double *info,
                              void *ws, size_t bytes, void *stream) {
    NvtxRange range("svdcache_calibrate_finish");
    int rc = check_ws(D, k, ws, bytes);
    if (rc) return rc;
    if (!Vk) return SVDCACHE_ERR_INVALID_ARG;
    if (!aligned16(Vk)) return SVDCACHE_ERR_BAD_ALIGN;
    return calib_finish(D, k, Vk, lambda, trace, info, ws, (cudaStream_t)stream);
}

int svdcache_calibrate(const void *Fstack, int64_t M, int D, int64_t ld, int dtype, int k, float *Vk,
                       double *lambda, double *trace, double *info, void *ws, size_t bytes,
                       void *stream) {
    if (M < 1) return SVDCACHE_ERR_BAD_SHAPE;
    int rc = svdcache_calibrate_begin(D, k, ws, bytes, stream);
    if (rc) return rc;
    rc = svdcache_calibrate_accumulate(Fstack, M, D, ld, dtype, ws, bytes, stream);
    if (rc) return rc;
    return svdcache_calibrate_finish(D, k, Vk, lambda, trace, info, ws, bytes, stream);
}

int svdcache_calibrate_gram_region(int D, size_t *offset, size_t *bytes) {
    if (!offset || !bytes) return SVDCACHE_ERR_INVALID_ARG;
    if (D < 8 || D > 16384 || (D % 8) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    *offset = calib_gram_offset();
    *bytes = (size_t)D * D * sizeof(double);
    return SVDCACHE_OK;
}

int svdcache_basis_similarity(const float *VkA, const double *lambdaA, const float *VkB, const double *lambdaB, int D,
                              int k, double *column_cos, double *out, void *stream) {
    if (!VkA || !VkB || !lambdaA || !lambdaB || !column_cos || !out) return SVDCACHE_ERR_INVALID_ARG;
    if (D < 1 || k < 1 || k > D || k > 16384) return SVDCACHE_ERR_BAD_SHAPE;
    int rc = column_cosines_launch(VkA, VkB, D, k, column_cos, (cudaStream_t)stream);
    if (rc) return rc;
    // the spectra are k numbers each: their statistic is formed on the host
    std::vector<double> la(k), lb(k), cs(k);
    rc = record_cuda(cudaMemcpyAsync(la.data(), lambdaA, k * sizeof(double), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (!rc) rc = record_cuda(cudaMemcpyAsync(lb.data(), lambdaB, k * sizeof(double), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (!rc) rc = record_cuda(cudaMemcpyAsync(cs.data(), column_cos, k * sizeof(double), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (!rc) rc = record_cuda(cudaStreamSynchronize((cudaStream_t)stream));
    if (rc) return rc;
    double ab = 0.0, aa = 0.0, bb = 0.0, mean = 0.0;
    for (int i = 0; i < k; ++i) {
        const double sa = la[i] > 0.0 ? std::sqrt(la[i]) : 0.0, sb = lb[i] > 0.0 ? std::sqrt(lb[i]) : 0.0;
        ab += sa * sb; aa += sa * sa; bb += sb * sb;
        mean += cs[i];
    }
    const double na = std::sqrt(aa), nb = std::sqrt(bb);
    out[0] = (na > 0.0 && nb > 0.0) ? (ab / (na * nb)) * (na < nb ? na / nb : nb / na) : 0.0;
    out[1] = mean / k;
    return SVDCACHE_OK;
}

int svdcache_rank_for_energy(const double *lambda, int n, double trace, double tau, int *k_out) {
    if (!lambda || !k_out || n < 1 || !(trace > 0.0) || !(tau >= 0.0) || !(tau <= 1.0))
        return SVDCACHE_ERR_INVALID_ARG;
    double acc = 0.0;
    *k_out = n;
    for (int i = 0; i < n; ++i) {
        acc += lambda[i];
        if (acc / trace >= tau) { *k_out = i + 1; break; }
    }
    return SVDCACHE_OK;
}

/* ------------------------------------------------------------------------ basis --- */

int svdcache_basis_bytes(int D, int k, int dtype, size_t *bytes) {
    if (!bytes) return SVDCACHE_ERR_INVALID_ARG;
    int rc = check_shape(1, D, k, dtype);
    if (rc) return rc;
    *bytes = basis_layout(D, k, dtype).total;
    return SVDCACHE_OK;
}

int svdcache_basis_layout(int D, int k, int dtype, size_t *v32, size_t *vt32, size_t *v16, size_t *vt16) {
    int rc = check_shape(1, D, k, dtype);
    if (rc) return rc;
    const BasisLayout L = basis_layout(D, k, dtype);
    if (v32) *v32 = L.v_f32;
    if (vt32) *vt32 = L.vt_f32;
    if (v16) *v16 = (dtype == SVDCACHE_BF16) ? L.v_bf16 : 0;
    if (vt16) *vt16 = (dtype == SVDCACHE_BF16) ? L.vt_bf16 : 0;
    return SVDCACHE_OK;
}

int svdcache_basis_prepare(const float *Vk, int D, int k, int dtype, void *basis, size_t bytes, void *stream) {
    int rc = check_shape(1, D, k, dtype);
    if (rc) return rc;
    if (!Vk || !basis) return SVDCACHE_ERR_INVALID_ARG;
    if (!aligned16(Vk) || (reinterpret_cast<uintptr_t>(basis) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if (bytes < basis_layout(D, k, dtype).total) return SVDCACHE_ERR_WORKSPACE;
    return basis_prepare(Vk, D, k, dtype, basis, (cudaStream_t)stream);
}

/* ------------------------------------------------------------------------ state --- */

int svdcache_state_bytes(int64_t N, int D, int k, int dtype, size_t *bytes) {
    if (!bytes) return SVDCACHE_ERR_INVALID_ARG;
    int rc = check_shape(N, D, k, dtype);
    if (rc) return rc;
    *bytes = state_layout(N, D, k, dtype).total;
    return SVDCACHE_OK;
}

int svdcache_state_layout(int64_t N, int D, int k, int dtype, size_t *chat_offset, size_t *r_offset) {
    int rc = check_shape(N, D, k, dtype);
    if (rc) return rc;
    const StateLayout L = state_layout(N, D, k, dtype);
    if (chat_offset) *chat_offset = L.chat;
    if (r_offset) *r_offset = L.r;
    return SVDCACHE_OK;
}

int svdcache_state_reset(void *state, int64_t N, int D, int k, int dtype, void *stream) {
    int rc = check_shape(N, D, k, dtype);
    if (rc) return rc;
    if (!state) return SVDCACHE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(state) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    state_reset_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((StateHeader *)state, N, D, k, dtype);
    count_launch();
    return check_last_launch();
}

int svdcache_state_query(const void *state, void *stream, int64_t *full_steps, int *status) {
    if (!state) return SVDCACHE_ERR_INVALID_ARG;
    StateHeader h;
    int rc = record_cuda(cudaMemcpyAsync(&h, state, sizeof(h), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (rc) return rc;
    rc = record_cuda(cudaStreamSynchronize((cudaStream_t)stream));
    if (rc) return rc;
    if (h.magic != kStateMagic) return SVDCACHE_ERR_STATE;
    if (full_steps) *full_steps = (int64_t)h.full_steps;
    if (status) *status = h.status;
    return SVDCACHE_OK;
}

/* ------------------------------------------------------------------------ steps --- */

static int check_step(const StepArgs &a, bool full) {
    int rc = check_shape(a.N, a.D, a.k, a.dtype);
    if (rc) return rc;
    if (a.nblocks < 1) return SVDCACHE_ERR_BAD_SHAPE;
    if (!a.basis || !a.state || (full ? !a.F : !a.Fhat)) return SVDCACHE_ERR_INVALID_ARG;
    rc = check_pitch(a.ld, a.D, a.dtype);
    if (rc) return rc;
    if (!aligned16(full ? a.F : (const void *)a.Fhat)) return SVDCACHE_ERR_BAD_ALIGN;
    if ((reinterpret_cast<uintptr_t>(a.basis) & 255u) || (reinterpret_cast<uintptr_t>(a.state) & 255u))
        return SVDCACHE_ERR_BAD_ALIGN;
    if (a.C_out && !aligned16(a.C_out)) return SVDCACHE_ERR_BAD_ALIGN;
    if (full && !(a.beta >= 0.0f && a.beta <= 1.0f)) return SVDCACHE_ERR_INVALID_ARG;
    if (a.nblocks > 1) {
        const size_t strides[5] = {a.F_stride, a.Fhat_stride, a.basis_stride, a.state_stride, a.C_stride};
        for (size_t st : strides)
            if (st % 256 != 0) return SVDCACHE_ERR_BAD_ALIGN;
        if (a.basis_stride < basis_layout(a.D, a.k, a.dtype).total) return SVDCACHE_ERR_BAD_SHAPE;
        if (a.state_stride < state_layout(a.N, a.D, a.k, a.dtype).total) return SVDCACHE_ERR_BAD_SHAPE;
        const size_t need = ((size_t)(a.N - 1) * a.ld + a.D) * elem_bytes(a.dtype);
        if ((full ? a.F_stride : a.Fhat_stride) < need) return SVDCACHE_ERR_BAD_SHAPE;
        if (a.C_out && a.C_stride < (size_t)a.N * a.k * 4) return SVDCACHE_ERR_BAD_SHAPE;
    }
    return SVDCACHE_OK;
}

int svdcache_full_step_batched(int nblocks, const void *F, int64_t ld, size_t F_stride, const void *basis,
                               size_t basis_stride, void *state, size_t state_stride, float *C_out,
                               size_t C_stride, int64_t N, int D, int k, int dtype, float beta,
                               void *stream) {
    NvtxRange range("svdcache_full_step_batched");
    StepArgs a{};
    a.F = F; a.ld = ld; a.F_stride = F_stride; a.basis = basis; a.basis_stride = basis_stride;
    a.state = state; a.state_stride = state_stride; a.C_out = C_out; a.C_stride = C_stride;
    a.N = N; a.D = D; a.k = k; a.dtype = dtype; a.beta = beta; a.nblocks = nblocks;
    int rc = check_step(a, true);
    if (rc) return rc;
    return dispatch(a, true, (cudaStream_t)stream);
}

int svdcache_cached_step_batched(int nblocks, const void *state, size_t state_stride, const void *basis,
                                 size_t basis_stride, void *Fhat, int64_t ld, size_t Fhat_stride,
                                 int64_t N, int D, int k, int dtype, int steps_since_full, void *stream) {
    NvtxRange range("svdcache_cached_step_batched");
    (void)steps_since_full;  // the EMA forecast does not depend on it
    StepArgs a{};
    a.Fhat = Fhat; a.ld = ld; a.Fhat_stride = Fhat_stride; a.basis = basis; a.basis_stride = basis_stride;
    a.state = const_cast<void *>(state); a.state_stride = state_stride;
    a.N = N; a.D = D; a.k = k; a.dtype = dtype; a.nblocks = nblocks;
    int rc = check_step(a, false);
    if (rc) return rc;
    return dispatch(a, false, (cudaStream_t)stream);
}

int svdcache_full_step_residual_ema_batched(int nblocks, const void *F, int64_t ld, size_t F_stride,
                                            const void *basis, size_t basis_stride, void *state,
                                            size_t state_stride, float *C_out, size_t C_stride, int64_t N,
                                            int D, int k, int dtype, float beta, float beta_r, void *stream) {
    NvtxRange range("svdcache_full_step_residual_ema_batched");
    if (!(beta_r >= 0.0f && beta_r <= 1.0f)) return SVDCACHE_ERR_INVALID_ARG;
    StepArgs a{};
    a.F = F; a.ld = ld; a.F_stride = F_stride; a.basis = basis; a.basis_stride = basis_stride;
    a.state = state; a.state_stride = state_stride; a.C_out = C_out; a.C_stride = C_stride;
    a.N = N; a.D = D; a.k = k; a.dtype = dtype; a.beta = beta; a.beta_r = beta_r; a.nblocks = nblocks;
    int rc = check_step(a, true);
    if (rc) return rc;
    return dispatch(a, true, (cudaStream_t)stream);
}

int svdcache_forecast_weights(int predictor, int order, int steps_since_full, int interval, double *w) {
    if (!w || interval < 1 || steps_since_full < 0) return SVDCACHE_ERR_INVALID_ARG;
    return forecast_weights(predictor, order, (double)steps_since_full / (double)interval, w);
}

int svdcache_forecast_bytes(int64_t N, int k, size_t *bytes) {
    if (!bytes) return SVDCACHE_ERR_INVALID_ARG;
    if (N < 1 || k < 8 || k > 256 || (k % 8) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    *bytes = forecast_layout(N, k).total;
    return SVDCACHE_OK;
}

int svdcache_cached_step_forecast_batched(int nblocks, const void *state, size_t state_stride, const void *basis,
                                          size_t basis_stride, void *Fhat, int64_t ld, size_t Fhat_stride,
                                          int64_t N, int D, int k, int dtype, const float *const *C_hist,
                                          size_t C_stride, int predictor, int order, int steps_since_full,
                                          int interval, void *forecast, size_t forecast_stride, void *stream) {
    NvtxRange range("svdcache_cached_step_forecast_batched");
    StepArgs a{};
    a.Fhat = Fhat; a.ld = ld; a.Fhat_stride = Fhat_stride; a.basis = basis; a.basis_stride = basis_stride;
    a.state = const_cast<void *>(state); a.state_stride = state_stride;
    a.N = N; a.D = D; a.k = k; a.dtype = dtype; a.nblocks = nblocks;
    int rc = check_step(a, false);
    if (rc) return rc;
    if (predictor == SVDCACHE_PREDICT_EMA) return dispatch(a, false, (cudaStream_t)stream);   // the state's own forecast
    if (!C_hist || !forecast || interval < 1 || steps_since_full < 0) return SVDCACHE_ERR_INVALID_ARG;
    double w[8];
    rc = forecast_weights(predictor, order, (double)steps_since_full / (double)interval, w);
    if (rc) return rc;
    for (int j = 0; j <= order; ++j) {
        if (!C_hist[j]) return SVDCACHE_ERR_INVALID_ARG;
        if (!aligned16(C_hist[j])) return SVDCACHE_ERR_BAD_ALIGN;
    }
    if ((reinterpret_cast<uintptr_t>(forecast) & 255u) != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if (nblocks > 1) {
        if (C_stride % 256 != 0 || forecast_stride % 256 != 0) return SVDCACHE_ERR_BAD_ALIGN;
        if (C_stride < (size_t)N * k * 4 || forecast_stride < forecast_layout(N, k).total) return SVDCACHE_ERR_BAD_SHAPE;
    }
    rc = forecast_launch(C_hist, C_stride, w, order, N, k, dtype, nblocks, forecast, forecast_stride, (cudaStream_t)stream);
    if (rc) return rc;
    a.coef = forecast;
    a.coef_stride = forecast_stride;
    return dispatch(a, false, (cudaStream_t)stream);
}

int svdcache_singular_values(const double *lambda, int k, double *sigma, void *stream) {
    if (!lambda || !sigma) return SVDCACHE_ERR_INVALID_ARG;
    if (k < 1 || k > 16384) return SVDCACHE_ERR_BAD_SHAPE;
    return sigma_launch(lambda, k, sigma, (cudaStream_t)stream);
}

int svdcache_left_factors(const float *C, const double *sigma, int64_t N, int k, float *U, void *stream) {
    if (!C || !sigma || !U) return SVDCACHE_ERR_INVALID_ARG;
    if (N < 1 || k < 1 || k > 16384) return SVDCACHE_ERR_BAD_SHAPE;
    return left_factors_launch(C, sigma, N, k, U, (cudaStream_t)stream);
}

/* Blocks of different rank in one call: consecutive blocks of equal rank form one batched launch. */
int svdcache_full_step_ranked_batched(int nblocks, const void *F, int64_t ld, size_t F_stride, const void *basis,
                                      size_t basis_stride, void *state, size_t state_stride, float *C_out,
                                      size_t C_stride, int64_t N, int D, const int *k_per_block, int dtype,
                                      float beta, void *stream) {
    if (!k_per_block || nblocks < 1) return SVDCACHE_ERR_INVALID_ARG;
    for (int b0 = 0; b0 < nblocks;) {
        int b1 = b0 + 1;
        while (b1 < nblocks && k_per_block[b1] == k_per_block[b0]) ++b1;
        const int rc = svdcache_full_step_batched(
            b1 - b0, (const char *)F + (size_t)b0 * F_stride, ld, F_stride, (const char *)basis + (size_t)b0 * basis_stride,
            basis_stride, (char *)state + (size_t)b0 * state_stride, state_stride,
            C_out ? reinterpret_cast<float *>((char *)C_out + (size_t)b0 * C_stride) : nullptr, C_stride, N, D,
            k_per_block[b0], dtype, beta, stream);
        if (rc) return rc;
        b0 = b1;
    }
    return SVDCACHE_OK;
}

int svdcache_cached_step_ranked_batched(int nblocks, const void *state, size_t state_stride, const void *basis,
                                        size_t basis_stride, void *Fhat, int64_t ld, size_t Fhat_stride, int64_t N,
                                        int D, const int *k_per_block, int dtype, int steps_since_full, void *stream) {
    if (!k_per_block || nblocks < 1) return SVDCACHE_ERR_INVALID_ARG;
    for (int b0 = 0; b0 < nblocks;) {
        int b1 = b0 + 1;
        while (b1 < nblocks && k_per_block[b1] == k_per_block[b0]) ++b1;
        const int rc = svdcache_cached_step_batched(
            b1 - b0, (const char *)state + (size_t)b0 * state_stride, state_stride,
            (const char *)basis + (size_t)b0 * basis_stride, basis_stride, (char *)Fhat + (size_t)b0 * Fhat_stride, ld,
            Fhat_stride, N, D, k_per_block[b0], dtype, steps_since_full, stream);
        if (rc) return rc;
        b0 = b1;
    }
    return SVDCACHE_OK;
}

int svdcache_full_step(const void *F, int64_t ld, const void *basis, void *state, float *C_out, int64_t N,
                       int D, int k, int dtype, float beta, void *stream) {
    return svdcache_full_step_batched(1, F, ld, 0, basis, 0, state, 0, C_out, 0, N, D, k, dtype, beta, stream);
}

int svdcache_cached_step(const void *state, const void *basis, void *Fhat, int64_t ld, int64_t N, int D,
                         int k, int dtype, int steps_since_full, void *stream) {
    return svdcache_cached_step_batched(1, state, 0, basis, 0, Fhat, ld, 0, N, D, k, dtype, steps_since_full,
                                        stream);
}

}  // extern "C"
