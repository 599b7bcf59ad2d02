// Basis buffer of Eq. 7 in the layouts the step kernels read: V_k and its transpose, in
// fp32 and (for bf16 I/O) rounded to bf16.
#include "internal.cuh"

namespace svdc {
namespace {

__global__ void basis_prepare_kernel(const float *__restrict__ Vk, int D, int k, int dtype, char *basis,
                                     BasisLayout L) {
    const int64_t total = (int64_t)D * k;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        BasisHeader *h = reinterpret_cast<BasisHeader *>(basis);
        h->magic = kBasisMagic;
        h->D = D;
        h->k = k;
        h->dtype = dtype;
    }
    float *v32 = reinterpret_cast<float *>(basis + L.v_f32);
    float *vt32 = reinterpret_cast<float *>(basis + L.vt_f32);
    __nv_bfloat16 *v16 = reinterpret_cast<__nv_bfloat16 *>(basis + L.v_bf16);
    __nv_bfloat16 *vt16 = reinterpret_cast<__nv_bfloat16 *>(basis + L.vt_bf16);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int d = (int)(i / k), j = (int)(i - (int64_t)d * k);
        const float v = Vk[i];
        v32[i] = v;
        vt32[(size_t)j * D + d] = v;
        if (dtype == SVDCACHE_BF16) {
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            v16[i] = h;
            vt16[(size_t)j * D + d] = h;
        }
    }
}

}  // namespace

int basis_prepare(const float *Vk, int D, int k, int dtype, void *basis, cudaStream_t s) {
    const BasisLayout L = basis_layout(D, k, dtype);
    const int64_t total = (int64_t)D * k;
    const int threads = 256;
    const int blocks = (int)((total + threads - 1) / threads < 1184 ? (total + threads - 1) / threads : 1184);
    basis_prepare_kernel<<<blocks, threads, 0, s>>>(Vk, D, k, dtype, (char *)basis, L);
    count_launch();
    return check_last_launch();
}

}  // namespace svdc
