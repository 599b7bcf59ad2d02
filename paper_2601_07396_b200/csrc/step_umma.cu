// tcgen05 family of the step kernels (placeholder until the tensor-core path lands).
#include "internal.cuh"

namespace svdc {

bool umma_supported(const StepArgs &, bool) { return false; }
int umma_full_step(const StepArgs &, cudaStream_t) { return SVDCACHE_ERR_BAD_SHAPE; }
int umma_cached_step(const StepArgs &, cudaStream_t) { return SVDCACHE_ERR_BAD_SHAPE; }

bool umma_gram_supported(int64_t, int, int64_t, int) { return false; }
size_t umma_gram_scratch_bytes(int) { return 0; }
int umma_gram_accumulate(const void *, int64_t, int, int64_t, double *, void *, size_t, cudaStream_t) {
    return SVDCACHE_ERR_BAD_SHAPE;
}

}  // namespace svdc
