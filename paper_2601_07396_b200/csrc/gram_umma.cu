// Gram matrix of the calibration stack on the tensor cores (Sec. 3.2 Eq. 4, Sec. 3.3):
//     G += F^T F,   F an M x D stack of bf16 feature rows, G the D x D fp64 accumulator.
//
// Both operands of the product are F itself with the reduction index (the stack row) as
// the strided dimension, so they are "MN-major" for the tensor core: a shared-memory row is
// one stack row's 64 consecutive columns (128 bytes, 128-byte swizzle, written by TMA),
// eight such rows form a K group of 1 KB, and the 64-column blocks of a tile sit 8 KB apart.
// bf16 products are exact in fp32; the fp32 TMEM accumulator only ever covers a chunk of
// kChunkRows stack rows, after which the epilogue warps add it into the fp64 G (the eigen-
// gap at k of the spectra met here is ~1e-6 of the leading eigenvalue: an fp32 sum over the
// whole stack would not resolve it).  Two accumulators alternate, so the flush of one chunk
// overlaps the MMAs of the next.
//
// One CTA owns one 128 x 256 tile of G's upper block triangle for the whole call, and walks
// its chunks in order: no atomics, a fixed summation order, bit-reproducible results.  When
// there are a few more tiles than SMs (D = 3072: 156 tiles, 148 SMs), the surplus tiles are
// not left to a nearly empty second wave: each is cut along the stack rows into segments,
// one per CTA, that sum into private fp64 partial tiles, and a small kernel adds those to G
// in segment order afterwards.
// Warp roles (192 threads): 0 = TMA producer, 1 = MMA issuer (+ TMEM owner), 2..5 = flush.
#include "internal.cuh"
#include "umma.cuh"

namespace svdc {

using namespace sm100;

namespace {

constexpr int kGThreads = 192;
constexpr int kGTileI = 128;          // rows of G per tile (MMA M)
constexpr int kGTileJ = 256;          // columns of G per tile (MMA N, at most)
constexpr int kGBlk = 64;             // columns of F per shared-memory block (128 bytes)
constexpr int kGStageRows = 64;       // stack rows per pipeline stage
constexpr uint32_t kGBlkBytes = kGStageRows * 128u;                                   // 8 KB
constexpr uint32_t kGStageBytes = (kGTileI / kGBlk + kGTileJ / kGBlk) * kGBlkBytes;   // 48 KB
constexpr int kGStages = 4;
constexpr int kChunkRows = 2048;      // stack rows summed in fp32 before the fp64 flush
constexpr uint32_t kGBarBytes = 8 * (2 * kGStages + 4 + 2);

struct GramParams {
    int64_t M;
    int D;
    int tiles_j;          // 256-column tiles per row of tiles
    int ntiles;
    int whole;            // tiles [0, whole) are summed over the whole stack by one CTA each, into G
    int nseg;             // each tile of [whole, ntiles) is cut into nseg row segments (units after the whole tiles)
    int units;            // whole + (ntiles - whole) * nseg
    double *partials;     // one dense 128 x 256 fp64 tile per segment unit
    double *G;
    int *status;          // device word that receives SVDCACHE_ERR_TIMEOUT if a bounded wait runs out
};

// tile t of the upper block triangle -> (ti, tj): tiles of row ti start at the first tj whose
// columns reach the diagonal
__device__ __forceinline__ void decode_tile(const GramParams &p, int t, int &ti, int &tj) {
    ti = 0;
    for (;; ++ti) {
        const int first = (ti * kGTileI) / kGTileJ;
        const int n = p.tiles_j - first;
        if (t < n) { tj = first + t; return; }
        t -= n;
    }
}

struct GramUnit {
    int tile, st_lo, st_hi;   // tile, stage range [st_lo, st_hi) of the stack
    double *out;              // partial tile, or nullptr: the tile of G itself
    int store_first;          // 1: the first chunk overwrites (partial tiles start undefined)
};
__device__ __forceinline__ GramUnit decode_gram_unit(const GramParams &p, int u, int nstages_total) {
    GramUnit x;
    if (u < p.whole) {
        x.tile = u; x.st_lo = 0; x.st_hi = nstages_total; x.out = nullptr; x.store_first = 0;
    } else {
        const int idx = u - p.whole, seg = idx % p.nseg;
        x.tile = p.whole + idx / p.nseg;
        x.st_lo = (int)(((int64_t)seg * nstages_total) / p.nseg);
        x.st_hi = (int)(((int64_t)(seg + 1) * nstages_total) / p.nseg);
        x.out = p.partials + (size_t)idx * (kGTileI * kGTileJ);
        x.store_first = 1;
    }
    return x;
}

// MN-major operand descriptor, 128-byte swizzle: 64-element blocks along M/N are `lbo` bytes
// apart, groups of eight K rows 1 KB apart
__device__ __forceinline__ uint64_t smem_desc_mnmajor(uint32_t saddr, uint32_t lbo) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
__host__ __device__ constexpr uint32_t idesc_bf16_mnmajor(int M, int N) {
    return idesc_bf16(M, N) | (1u << 15) | (1u << 16);
}

__global__ void __launch_bounds__(kGThreads, 1)
umma_gram_kernel(const __grid_constant__ CUtensorMap tm_f, const GramParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + kGStages * kGStageBytes;
    const uint32_t full = bars, empty = full + 8 * kGStages, acc_full = empty + 8 * kGStages, acc_empty = acc_full + 16;
    const uint32_t tmem_slot_a = acc_empty + 16, abort_a = tmem_slot_a + 8;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen + (tmem_slot_a - base));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + (abort_a - base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kGStages; ++s) { mbar_init(full + 8 * s, 1); mbar_init(empty + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 128); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_f);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot_a, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int nstages_total = (int)((p.M + kGStageRows - 1) / kGStageRows);
    constexpr int kChunkStages = kChunkRows / kGStageRows;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const GramUnit gu = decode_gram_unit(p, u, nstages_total);
                int ti, tj;
                decode_tile(p, gu.tile, ti, tj);
                const int i0 = ti * kGTileI, j0 = tj * kGTileJ;
                const int nj = min(kGTileJ, p.D - j0) / kGBlk;
                for (int st = gu.st_lo; st < gu.st_hi; ++st, ++it) {
                    const uint32_t s = it % kGStages, ph = (it / kGStages) & 1u;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag, 1)) goto done;
                    const uint32_t dst = base + s * kGStageBytes;
                    mbar_arrive_expect_tx(full + 8 * s, (2 + nj) * kGBlkBytes);
                    for (int b = 0; b < 2; ++b)
                        tma_load_3d(dst + b * kGBlkBytes, &tm_f, full + 8 * s, i0 + b * kGBlk, st * kGStageRows, 0);
                    for (int b = 0; b < nj; ++b)
                        tma_load_3d(dst + (2 + b) * kGBlkBytes, &tm_f, full + 8 * s, j0 + b * kGBlk, st * kGStageRows, 0);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, ic = 0;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const GramUnit gu = decode_gram_unit(p, u, nstages_total);
                int ti, tj;
                decode_tile(p, gu.tile, ti, tj);
                const int nj = min(kGTileJ, p.D - tj * kGTileJ) / kGBlk;
                const uint32_t idesc = idesc_bf16_mnmajor(kGTileI, nj * kGBlk);
                for (int st0 = gu.st_lo; st0 < gu.st_hi; st0 += kChunkStages, ++ic) {
                    const uint32_t buf = ic & 1u;
                    if (!mbar_wait(acc_empty + 8 * buf, ((ic >> 1) & 1u) ^ 1u, abort_flag, 2)) goto done;
                    tc_fence_after();
                    const int st1 = min(st0 + kChunkStages, gu.st_hi);
                    for (int st = st0; st < st1; ++st, ++it) {
                        const uint32_t s = it % kGStages, ph = (it / kGStages) & 1u;
                        if (!mbar_wait(full + 8 * s, ph, abort_flag, 3)) goto done;
                        tc_fence_after();
                        const uint32_t a = base + s * kGStageBytes;
                        const uint64_t ad = smem_desc_mnmajor(a, kGBlkBytes), bd = smem_desc_mnmajor(a + 2 * kGBlkBytes, kGBlkBytes);
#pragma unroll
                        for (int ks = 0; ks < kGStageRows / 16; ++ks)   // 16 stack rows = two K groups = 2 KB
                            mma_bf16_ss(tmem_base + buf * kGTileJ, ad + ks * 128, bd + ks * 128, idesc,
                                        (st > st0 || ks > 0) ? 1u : 0u);
                        mma_commit(empty + 8 * s);
                    }
                    mma_commit(acc_full + 8 * buf);
                }
            }
        }
    } else {
        // flush: G[i0 + row][j0 ...] += accumulator row (thread = TMEM lane = tile row)
        const int q = warp & 3, row = q * 32 + lane;
        uint32_t ic = 0;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
            const GramUnit gu = decode_gram_unit(p, u, nstages_total);
            int ti, tj;
            decode_tile(p, gu.tile, ti, tj);
            const int i0 = ti * kGTileI, j0 = tj * kGTileJ;
            const int ncols = min(kGTileJ, p.D - j0);
            double *grow = gu.out ? gu.out + (size_t)row * kGTileJ : p.G + (size_t)(i0 + row) * p.D + j0;
            for (int st0 = gu.st_lo; st0 < gu.st_hi; st0 += kChunkStages, ++ic) {
                const bool overwrite = gu.store_first && st0 == gu.st_lo;
                const uint32_t buf = ic & 1u;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(acc_full + 8 * buf, (ic >> 1) & 1u, abort_flag, 4))) goto done;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kGTileJ;
                for (int c0 = 0; c0 < ncols; c0 += 32) {
                    uint32_t acc[32];
                    tmem_ld_32x32(taddr + c0, acc);
                    double2 g[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        g[i] = overwrite ? make_double2(0.0, 0.0) : *reinterpret_cast<const double2 *>(grow + c0 + 2 * i);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        g[i].x += (double)__uint_as_float(acc[2 * i]);
                        g[i].y += (double)__uint_as_float(acc[2 * i + 1]);
                        *reinterpret_cast<double2 *>(grow + c0 + 2 * i) = g[i];
                    }
                }
                tc_fence_before();
                mbar_arrive(acc_empty + 8 * buf);
            }
        }
    }

done:
    if (*abort_flag && (threadIdx.x & 31) == 0) atomicExch(p.status, SVDCACHE_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// G tile += its partial tiles, in segment order (one thread per element)
__global__ void gram_reduce_kernel(GramParams p) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;           // element within a tile
    const int x = blockIdx.y;                                      // which split tile
    if (e >= kGTileI * kGTileJ) return;
    int ti, tj;
    decode_tile(p, p.whole + x, ti, tj);
    const int r = e / kGTileJ, c = e % kGTileJ;
    const int j = tj * kGTileJ + c;
    if (j >= p.D) return;
    const int nstages_total = (int)((p.M + kGStageRows - 1) / kGStageRows);
    double acc = 0.0;
    for (int s = 0; s < p.nseg; ++s) {
        const GramUnit gu = decode_gram_unit(p, p.whole + x * p.nseg + s, nstages_total);
        if (gu.st_hi > gu.st_lo)   // a short stack leaves some segments empty: their partial tiles were never written
            acc += p.partials[((size_t)x * p.nseg + s) * (kGTileI * kGTileJ) + e];
    }
    p.G[(size_t)(ti * kGTileI + r) * p.D + j] += acc;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn gram_encode_fn() {
    static EncodeTiledFn fn = [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(ptr);
        return (EncodeTiledFn) nullptr;
    }();
    return fn;
}

constexpr int kNominalSMs = 148;   // the split of surplus tiles is sized for this many CTAs

int gram_tiles(int D, int *tiles_j) {
    const int ti_n = D / kGTileI, tj_n = (D + kGTileJ - 1) / kGTileJ;
    int n = 0;
    for (int ti = 0; ti < ti_n; ++ti) n += tj_n - (ti * kGTileI) / kGTileJ;
    *tiles_j = tj_n;
    return n;
}

}  // namespace

// The tensor path takes bf16 stacks whose width is a multiple of 128, in calls of at least
// one chunk of rows; everything else goes through the fp64 CUDA-core GEMM.
bool umma_gram_supported(int64_t M, int D, int64_t ld, int dtype) {
    if (dtype != SVDCACHE_BF16) return false;
    if (D < 256 || (D % kGTileI) != 0) return false;
    if (M < kChunkRows || M > 0x7FFFFFFFLL) return false;
    if (((size_t)ld * 2) % 16 != 0) return false;
    return gram_encode_fn() != nullptr;
}

// surplus tiles (beyond one per SM) and the segments each is cut into; 0 / 1 when the split does not apply
static void gram_split(int ntiles, int *surplus, int *nseg) {
    *surplus = 0; *nseg = 1;
    const int e = ntiles - kNominalSMs;
    if (e > 0 && e <= kNominalSMs / 2) { *surplus = e; *nseg = kNominalSMs / e; }
}

// bytes of the partial tiles (depends on D only)
size_t umma_gram_scratch_bytes(int D) {
    if (D < 256 || (D % kGTileI) != 0) return 0;
    int tj, surplus, nseg;
    const int ntiles = gram_tiles(D, &tj);
    gram_split(ntiles, &surplus, &nseg);
    return (size_t)surplus * nseg * kGTileI * kGTileJ * sizeof(double);
}

int umma_gram_accumulate(const void *F, int64_t M, int D, int64_t ld, double *G, double *scratch, int *status,
                         cudaStream_t s) {
    EncodeTiledFn fn = gram_encode_fn();
    if (!fn) return SVDCACHE_ERR_CUDA;
    CUtensorMap tm;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)M, 1};
    const cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)ld * 2 * (cuuint64_t)M};
    const cuuint32_t box[3] = {kGBlk, kGStageRows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(F), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SVDCACHE_ERR_CUDA;
    GramParams p{};
    p.M = M; p.D = D; p.G = G; p.status = status;
    p.ntiles = gram_tiles(D, &p.tiles_j);
    int sms = 0, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = kNominalSMs;
    int surplus = 0, nseg = 1;
    if (sms == kNominalSMs && scratch) gram_split(p.ntiles, &surplus, &nseg);
    p.whole = p.ntiles - surplus;
    p.nseg = nseg;
    p.units = p.whole + surplus * nseg;
    p.partials = scratch;
    const size_t smem = 1024 + (size_t)kGStages * kGStageBytes + kGBarBytes + 64;
    {   // kept per device by the runtime: set on every call
        int rc = record_cuda(cudaFuncSetAttribute(umma_gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (rc) return rc;
    }
    const int grid = p.units < sms ? p.units : sms;
    umma_gram_kernel<<<grid, kGThreads, smem, s>>>(tm, p);
    count_launch();
    if (surplus > 0) {
        gram_reduce_kernel<<<dim3((kGTileI * kGTileJ + 255) / 256, surplus), 256, 0, s>>>(p);
        count_launch();
    }
    return check_last_launch();
}

}  // namespace svdc
