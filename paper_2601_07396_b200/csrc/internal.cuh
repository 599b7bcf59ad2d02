// Shared declarations of the CUDA library: buffer headers, layouts, launch bookkeeping.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/svdcache.h"

namespace svdc {

constexpr uint32_t kBasisMagic = 0x53564342u;  // "SVCB"
constexpr uint32_t kStateMagic = 0x53564353u;  // "SVCS"
constexpr size_t kHeaderBytes = 256;
constexpr size_t kAlign = 256;

struct BasisHeader {   // first 256 bytes of a basis buffer
    uint32_t magic;
    int32_t D, k, dtype;
};

struct StateHeader {   // first 256 bytes of a state buffer
    uint32_t magic;
    int32_t dtype;
    int64_t N;
    int32_t D, k;
    uint32_t full_steps;   // full steps seen since the last reset
    int32_t status;        // sticky device status word (SVDCACHE_OK or an error code)
    uint32_t done;         // CUDA-core full step: CTAs of this block that have finished
    uint32_t pad;          // which wait ran out first: site << 16 | CTA (diagnosis)
    // tcgen05 full step, in block 0's header: CTAs of the launch that have left the kernel (the
    // last one counts the step in every block's header)
    uint32_t exits;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_bytes(int dtype) { return dtype == SVDCACHE_BF16 ? 2 : 4; }

struct BasisLayout {
    size_t v_f32, vt_f32, v_bf16, vt_bf16, total;
};
inline BasisLayout basis_layout(int D, int k, int dtype) {
    BasisLayout L;
    const size_t f = align_up((size_t)D * k * 4, kAlign), h = align_up((size_t)D * k * 2, kAlign);
    L.v_f32 = kHeaderBytes;
    L.vt_f32 = L.v_f32 + f;
    L.v_bf16 = L.vt_f32 + f;
    L.vt_bf16 = L.v_bf16 + (dtype == SVDCACHE_BF16 ? h : 0);
    L.total = L.vt_bf16 + (dtype == SVDCACHE_BF16 ? h : 0);
    return L;
}

// header | Chat fp32 [N x k] | (bf16 only) Chat as a split-bf16 pair: hi [N x k], lo [N x k] | R [N x D].
// hi = bf16(x), lo = bf16(x - hi).  The pair of Chat is the tensor-core operand of the cached
// step, written by the full step next to Chat so that the cached step reads it as it is.
struct StateLayout {
    size_t chat, op_hi, op_lo, r, total;
};
inline StateLayout state_layout(int64_t N, int D, int k, int dtype) {
    StateLayout L;
    const bool bf = dtype == SVDCACHE_BF16;
    const size_t op = bf ? align_up((size_t)N * k * 2, kAlign) : 0;
    L.chat = kHeaderBytes;
    L.op_hi = L.chat + align_up((size_t)N * k * 4, kAlign);
    L.op_lo = L.op_hi + op;
    L.r = L.op_lo + op;
    L.total = L.r + align_up((size_t)N * D * elem_bytes(dtype), kAlign);
    return L;
}

// split of an fp32 value into the bf16 pair (hi, lo) described above
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// Arguments shared by the step kernels of every family.  Pointers are block 0's; block b
// adds b * stride bytes.
struct StepArgs {
    const void *F;          // full step input / unused in the cached step
    void *Fhat;             // cached step output
    const void *basis;
    void *state;
    float *C_out;
    size_t F_stride, Fhat_stride, basis_stride, state_stride, C_stride;
    int64_t ld;             // pitch of F / Fhat in elements
    int64_t N;
    int D, k, dtype, nblocks;
    float beta;
    float beta_r;           // full step: EMA weight of the stored residual (0 = the residual is replaced, Sec. 3.5)
    const void *coef;       // cached step: forecast buffer (fp32 | hi | lo, forecast_layout) to take the
    size_t coef_stride;     //   coefficients from instead of the state's Chat; null = the state's own
};

// launch bookkeeping (api.cu)
void count_launch(int n = 1);
int record_cuda(cudaError_t e);    // returns SVDCACHE_OK or SVDCACHE_ERR_CUDA, remembers text
int check_last_launch();

// CUDA-core family (step_simt.cu)
int simt_full_step(const StepArgs &a, cudaStream_t s);
int simt_cached_step(const StepArgs &a, cudaStream_t s);

// tcgen05 family (step_umma.cu)
bool umma_supported(const StepArgs &a, bool full);
int umma_full_step(const StepArgs &a, cudaStream_t s);
int umma_cached_step(const StepArgs &a, cudaStream_t s);
int umma_wait_selftest(void *state, long long limit_cycles, cudaStream_t s);

// forecasts and coefficient-side helpers (forecast.cu)
struct ForecastLayout {
    size_t f32, hi, lo, total;
};
ForecastLayout forecast_layout(int64_t N, int k);
int forecast_weights(int predictor, int order, double u, double *w);
int forecast_launch(const float *const *hist, size_t hist_stride, const double *w, int order, int64_t N, int k,
                    int dtype, int nblocks, void *out, size_t out_stride, cudaStream_t s);
int sigma_launch(const double *lambda, int k, double *sigma, cudaStream_t s);
int left_factors_launch(const float *C, const double *sigma, int64_t N, int k, float *U, cudaStream_t s);
int column_cosines_launch(const float *A, const float *B, int D, int k, double *out, cudaStream_t s);

// basis (basis.cu)
int basis_prepare(const float *Vk, int D, int k, int dtype, void *basis, cudaStream_t s);

// calibration (calibrate.cu)
size_t calib_workspace_bytes(int D, int k);
size_t calib_gram_offset();
int calib_begin(int D, int k, void *ws, cudaStream_t s);
int calib_accumulate(const void *F, int64_t M, int D, int64_t ld, int dtype, void *ws, cudaStream_t s);
int calib_finish(int D, int k, float *Vk, double *lambda, double *trace, double *info, void *ws,
                 cudaStream_t s);

}  // namespace svdc
