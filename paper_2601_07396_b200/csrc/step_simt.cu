// CUDA-core family of the step kernels.
//
// This is the fp32-I/O path (fp64 accumulation: the residual is ~5 % of the feature's
// norm, so the coefficients must be good to ~1e-7 for R to meet a 1e-5 relative bound)
// and the fall-back for bf16 shapes outside what the tcgen05 kernels take.  One CTA owns
// a tile of ROWS feature rows: the rows sit in shared memory, the coefficients are
// reduced over D by one thread per (row, component), then every thread owns feature
// columns and applies C V_k^T from the transposed basis copy with coalesced loads.
#include "internal.cuh"

namespace svdc {
namespace {

template <typename T> __device__ __forceinline__ float ld_as_float(const T *p);
template <> __device__ __forceinline__ float ld_as_float<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_as_float<__nv_bfloat16>(const __nv_bfloat16 *p) {
    return __bfloat162float(*p);
}
template <typename T, typename A> __device__ __forceinline__ T from_acc(A x);
template <> __device__ __forceinline__ float from_acc<float, double>(double x) { return (float)x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_acc<__nv_bfloat16, float>(float x) {
    return __float2bfloat16_rn(x);
}

constexpr int kThreads = 256;

// Full step: Eq. 8-9 (C = F V_k), Eq. 10 (R = F - C V_k^T), Eq. 11 (EMA of C).
template <typename T, typename BT, typename Acc, int kRows>
__global__ void __launch_bounds__(kThreads)
simt_full_kernel(StepArgs a, size_t v_off, size_t vt_off, StateLayout SL) {
    const size_t chat_off = SL.chat, r_off = SL.r;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int D = a.D, k = a.k;
    float *Fs = reinterpret_cast<float *>(smem_raw);                        // kRows x D
    Acc *Cs = reinterpret_cast<Acc *>(smem_raw + (size_t)kRows * D * 4);    // kRows x k

    const int b = blockIdx.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const T *F = reinterpret_cast<const T *>((const char *)a.F + (size_t)b * a.F_stride);
    const char *basis = (const char *)a.basis + (size_t)b * a.basis_stride;
    char *state = (char *)a.state + (size_t)b * a.state_stride;
    const BT *V = reinterpret_cast<const BT *>(basis + v_off);
    const BT *Vt = reinterpret_cast<const BT *>(basis + vt_off);
    StateHeader *hdr = reinterpret_cast<StateHeader *>(state);
    float *Chat = reinterpret_cast<float *>(state + chat_off);
    T *R = reinterpret_cast<T *>(state + r_off);
    float *C_out = a.C_out ? reinterpret_cast<float *>((char *)a.C_out + (size_t)b * a.C_stride) : nullptr;

    const bool first = (*(volatile uint32_t *)&hdr->full_steps) == 0;

    for (int idx = threadIdx.x; idx < kRows * D; idx += kThreads) {
        const int r = idx / D, d = idx - r * D;
        const int64_t n = row0 + r;
        Fs[idx] = (n < a.N) ? ld_as_float(F + n * a.ld + d) : 0.0f;
    }
    __syncthreads();

    const float beta = a.beta, omb = 1.0f - a.beta;
    for (int idx = threadIdx.x; idx < kRows * k; idx += kThreads) {
        const int r = idx / k, j = idx - r * k;
        const float *f = Fs + (size_t)r * D;
        Acc acc = 0;
        for (int d = 0; d < D; ++d) acc += (Acc)f[d] * (Acc)ld_as_float(V + (size_t)d * k + j);
        Cs[idx] = acc;
        const int64_t n = row0 + r;
        if (n < a.N) {
            const float c = (float)acc;
            if (C_out) C_out[n * k + j] = c;
            float *ch = Chat + n * k + j;
            const float ema = first ? c : fmaf(beta, *ch, omb * c);
            *ch = ema;
            if (SL.op_lo != SL.op_hi) {   // bf16 mode: the cached step's tensor-core operand
                __nv_bfloat16 hi, lo;
                split_bf16(ema, hi, lo);
                reinterpret_cast<__nv_bfloat16 *>(state + SL.op_hi)[n * k + j] = hi;
                reinterpret_cast<__nv_bfloat16 *>(state + SL.op_lo)[n * k + j] = lo;
            }
        }
    }
    __syncthreads();

    for (int d = threadIdx.x; d < D; d += kThreads) {
        Acc acc[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) acc[r] = 0;
        for (int j = 0; j < k; ++j) {
            const Acc v = (Acc)ld_as_float(Vt + (size_t)j * D + d);
#pragma unroll
            for (int r = 0; r < kRows; ++r) acc[r] += Cs[r * k + j] * v;
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const int64_t n = row0 + r;
            if (n < a.N) {
                Acc res = (Acc)Fs[(size_t)r * D + d] - acc[r];
                // ablation (Sec. 4.5): the stored residual as an EMA of the residuals
                if (a.beta_r > 0.0f && !first) res = (Acc)a.beta_r * (Acc)ld_as_float(R + n * D + d) + (Acc)(1.0f - a.beta_r) * res;
                R[n * D + d] = from_acc<T, Acc>(res);
            }
        }
    }

    // the last CTA of this block's grid row counts the full step
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t prev = atomicAdd(&hdr->done, 1u);
        if (prev == gridDim.x - 1) {
            hdr->done = 0;
            hdr->full_steps = hdr->full_steps + 1;
        }
    }
}

// Cached step (Sec. 3.5): Fhat = Chat V_k^T + R.
template <typename T, typename BT, typename Acc, int kRows>
__global__ void __launch_bounds__(kThreads)
simt_cached_kernel(StepArgs a, size_t vt_off, size_t chat_off, size_t r_off) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int D = a.D, k = a.k;
    Acc *Cs = reinterpret_cast<Acc *>(smem_raw);    // kRows x k

    const int b = blockIdx.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const char *basis = (const char *)a.basis + (size_t)b * a.basis_stride;
    char *state = (char *)a.state + (size_t)b * a.state_stride;
    const BT *Vt = reinterpret_cast<const BT *>(basis + vt_off);
    StateHeader *hdr = reinterpret_cast<StateHeader *>(state);
    // the coefficients come from the state's EMA, or from a forecast buffer (its fp32 part first)
    const float *Chat = a.coef ? reinterpret_cast<const float *>((const char *)a.coef + (size_t)b * a.coef_stride)
                               : reinterpret_cast<const float *>(state + chat_off);
    const T *R = reinterpret_cast<const T *>(state + r_off);
    T *Fhat = reinterpret_cast<T *>((char *)a.Fhat + (size_t)b * a.Fhat_stride);

    if ((*(volatile uint32_t *)&hdr->full_steps) == 0) {
        if (threadIdx.x == 0 && blockIdx.x == 0) hdr->status = SVDCACHE_ERR_STATE;
        return;
    }
    for (int idx = threadIdx.x; idx < kRows * k; idx += kThreads) {
        const int64_t n = row0 + idx / k;
        Cs[idx] = (n < a.N) ? (Acc)Chat[n * k + (idx % k)] : (Acc)0;
    }
    __syncthreads();
    for (int d = threadIdx.x; d < D; d += kThreads) {
        Acc acc[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) acc[r] = 0;
        for (int j = 0; j < k; ++j) {
            const Acc v = (Acc)ld_as_float(Vt + (size_t)j * D + d);
#pragma unroll
            for (int r = 0; r < kRows; ++r) acc[r] += Cs[r * k + j] * v;
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const int64_t n = row0 + r;
            if (n < a.N) Fhat[n * a.ld + d] = from_acc<T, Acc>(acc[r] + (Acc)ld_as_float(R + n * D + d));
        }
    }
}

template <typename T, typename BT, typename Acc, int kRows>
int launch_full(const StepArgs &a, size_t v_off, size_t vt_off, cudaStream_t s) {
    const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
    const size_t smem = (size_t)kRows * a.D * 4 + (size_t)kRows * a.k * sizeof(Acc);
    auto kern = simt_full_kernel<T, BT, Acc, kRows>;
    int rc = record_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (rc) return rc;
    dim3 grid((unsigned)((a.N + kRows - 1) / kRows), (unsigned)a.nblocks);
    kern<<<grid, kThreads, smem, s>>>(a, v_off, vt_off, SL);
    count_launch();
    return check_last_launch();
}

template <typename T, typename BT, typename Acc, int kRows>
int launch_cached(const StepArgs &a, size_t vt_off, cudaStream_t s) {
    const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
    const size_t smem = (size_t)kRows * a.k * sizeof(Acc);
    dim3 grid((unsigned)((a.N + kRows - 1) / kRows), (unsigned)a.nblocks);
    simt_cached_kernel<T, BT, Acc, kRows><<<grid, kThreads, smem, s>>>(a, vt_off, SL.chat, SL.r);
    count_launch();
    return check_last_launch();
}

}  // namespace

int simt_full_step(const StepArgs &a, cudaStream_t s) {
    const BasisLayout BL = basis_layout(a.D, a.k, a.dtype);
    const bool wide = a.D > 4096;   // fewer rows per CTA so that the row tile still fits in shared memory
    if (a.dtype == SVDCACHE_F32)
        return wide ? launch_full<float, float, double, 2>(a, BL.v_f32, BL.vt_f32, s)
                    : launch_full<float, float, double, 8>(a, BL.v_f32, BL.vt_f32, s);
    return wide ? launch_full<__nv_bfloat16, __nv_bfloat16, float, 2>(a, BL.v_bf16, BL.vt_bf16, s)
                : launch_full<__nv_bfloat16, __nv_bfloat16, float, 8>(a, BL.v_bf16, BL.vt_bf16, s);
}

int simt_cached_step(const StepArgs &a, cudaStream_t s) {
    const BasisLayout BL = basis_layout(a.D, a.k, a.dtype);
    if (a.dtype == SVDCACHE_F32) return launch_cached<float, float, double, 8>(a, BL.vt_f32, s);
    return launch_cached<__nv_bfloat16, __nv_bfloat16, float, 8>(a, BL.vt_bf16, s);
}

}  // namespace svdc
