// tcgen05 family of the step kernels (bf16 I/O): warp-specialised, persistent, TMA-fed.
//
// Both kernels stream 128-row x 64-column tiles of the big operand (R or F) through a
// ring of shared-memory slots (16 KB each, 128-byte swizzled, written by TMA).  The tensor
// cores produce the product C V_k^T into TMEM; the epilogue warps read it back, combine it
// with the staged tile in place and hand the tile to a TMA store.  Every global access on
// the streaming path is a TMA bulk copy: under a saturated memory system an ordinary load
// takes microseconds, so nothing on the critical path waits for one.  The 128 x k
// coefficient tile is the A operand, a split-bf16 pair (hi + lo) so that the product keeps
// ~16 mantissa bits.
#include <cstdio>
#include <mutex>

#include "internal.cuh"
#include "umma.cuh"

namespace svdc {

using namespace sm100;

namespace {

constexpr int kThreadsUmma = 320;
constexpr int kTileRows = 128;      // MMA M
constexpr int kTileCols = 64;       // columns of D per stage (MMA N in the reconstruct GEMM)
constexpr int kTileBytes = kTileRows * kTileCols * 2;   // 16 KB
constexpr int kAccStages = 4;       // TMEM accumulator ring (64 fp32 columns each)
constexpr int kMaxStages = 12;
constexpr int kMaxVSlots = 2;
constexpr int kMaxABufs = 2;

struct UmmaParams {
    int64_t N;
    int D, k, nblocks;
    int row_tiles, chunks_total, dsplit, chunks_per_slice, units;
    int kb_elems, kb_bytes, nkb;         // K-block of the rank dimension: min(k, 64) elements
    int stages, a_bufs;
    uint32_t a_half_bytes, a_bytes, v_bytes, stage_bytes;
    int gc, acc_stages, acc_cols, v_slots;   // cached step: chunks per MMA group, TMEM ring, basis ring
    uint32_t vslice_bytes;
    char *state;
    size_t state_stride, chat_off, ophi_off, oplo_off;
    float *C_out;
    size_t C_stride;
    float beta;
};

struct SmemLayout {
    uint32_t a, stages, bars;   // byte offsets from the 1024-aligned base
};

// barrier slots (8 bytes each) after the tiles
struct Bars {
    uint32_t full, empty, acc_full, acc_empty, a_full, a_empty, c_full, c_done, v_full, v_empty, tmem_slot, abort_flag;
};

__device__ __forceinline__ Bars bars_at(uint32_t base) {
    Bars b;
    b.full = base;
    b.empty = b.full + 8 * kMaxStages;
    b.acc_full = b.empty + 8 * kMaxStages;
    b.acc_empty = b.acc_full + 8 * kAccStages;
    b.a_full = b.acc_empty + 8 * kAccStages;
    b.a_empty = b.a_full + 8 * kMaxABufs;
    b.c_full = b.a_empty + 8 * kMaxABufs;
    b.c_done = b.c_full + 8;
    b.v_full = b.c_done + 8;
    b.v_empty = b.v_full + 8 * kMaxVSlots;
    b.tmem_slot = b.v_empty + 8 * kMaxVSlots;
    b.abort_flag = b.tmem_slot + 8;
    return b;
}
constexpr uint32_t kBarBytes = 8 * (2 * kMaxStages + 2 * kAccStages + 2 * kMaxABufs + 2 * kMaxVSlots + 4);

__device__ __forceinline__ StateHeader *header_of(const UmmaParams &p, int b) {
    return reinterpret_cast<StateHeader *>(p.state + (size_t)b * p.state_stride);
}

struct Unit {
    int b, rt, c0, c1;
};
__device__ __forceinline__ Unit decode_unit(const UmmaParams &p, int u) {
    Unit x;
    const int per_block = p.row_tiles * p.dsplit;
    x.b = u / per_block;
    const int rem = u - x.b * per_block;
    x.rt = rem / p.dsplit;
    const int ds = rem - x.rt * p.dsplit;
    x.c0 = ds * p.chunks_per_slice;
    x.c1 = min(x.c0 + p.chunks_per_slice, p.chunks_total);
    return x;
}

__device__ __forceinline__ void record_timeout(const UmmaParams &p) {
    atomicExch(&header_of(p, 0)->status, SVDCACHE_ERR_TIMEOUT);
}

// 8 bf16 (one 16-byte chunk) combined with 8 fp32 accumulator values: out = sign*acc + tile
template <bool SUBTRACT>
__device__ __forceinline__ uint4 combine_chunk(uint4 t, const uint32_t *acc) {
    uint32_t w[4] = {t.x, t.y, t.z, t.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        const float a0 = __uint_as_float(acc[2 * i]), a1 = __uint_as_float(acc[2 * i + 1]);
        const float r0 = SUBTRACT ? (lo - a0) : (lo + a0);
        const float r1 = SUBTRACT ? (hi - a1) : (hi + a1);
        const __nv_bfloat162 pk = __floats2bfloat162_rn(r0, r1);
        o[i] = *reinterpret_cast<const uint32_t *>(&pk);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t x, uint32_t y) {
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}

// Write 4 consecutive coefficients (columns j0..j0+3 of tile row `row`) into the A operand:
// a K-major, swizzled tile made of K-blocks of kb_elems columns, stored twice -- the bf16
// rounding of each value ("hi") and the bf16 rounding of what that rounding lost ("lo").
// hi + lo carries ~16 mantissa bits, so the product with V_k is good to ~1e-5 relative.
__device__ __forceinline__ void store_a4(uint32_t a_base, const UmmaParams &p, int row, int j0, float4 v) {
    const int kb = j0 / p.kb_elems, jj = j0 - kb * p.kb_elems;
    const uint32_t chunk = (uint32_t)jj >> 3, within = ((uint32_t)jj & 7u) * 2u;
    const uint32_t addr = a_base + (uint32_t)kb * (kTileRows * p.kb_bytes) + (uint32_t)row * p.kb_bytes +
                          swizzled_chunk((uint32_t)row, chunk, (uint32_t)p.kb_bytes) * 16u + within;
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(v.x, v.y), h23 = __floats2bfloat162_rn(v.z, v.w);
    const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(v.x - f01.x, v.y - f01.y);
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(v.z - f23.x, v.w - f23.y);
    sts64(addr, *reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
    sts64(addr + p.a_half_bytes, *reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
}

// issue the 2 * k/16 MMAs of one 128 x 64 output tile: D = (A_hi + A_lo)[128 x k] * B[64 x k]^T
__device__ __forceinline__ void issue_reconstruct_mmas(const UmmaParams &p, uint32_t d_tmem, uint32_t a_base,
                                                       uint32_t v_base) {
    const uint32_t idesc = idesc_bf16(kTileRows, kTileCols);
    const int ksteps = p.kb_elems / 16;
    bool acc = false;
    for (int part = 0; part < 2; ++part) {
        for (int kb = 0; kb < p.nkb; ++kb) {
            const uint32_t a_kb = a_base + (uint32_t)part * p.a_half_bytes + (uint32_t)kb * (kTileRows * p.kb_bytes);
            const uint32_t v_kb = v_base + (uint32_t)kb * (kTileCols * p.kb_bytes);
            for (int ks = 0; ks < ksteps; ++ks) {
                mma_bf16_ss(d_tmem, smem_desc_kmajor(a_kb + ks * 32, p.kb_bytes),
                            smem_desc_kmajor(v_kb + ks * 32, p.kb_bytes), idesc, acc ? 1u : 0u);
                acc = true;
            }
        }
    }
}

// ======================================================================================
// Cached step (Sec. 3.5):  Fhat = Chat V_k^T + R
//
// A unit is one 128-row tile of one block (times a column range when the launch is too
// small to occupy the GPU otherwise).  Its A operand -- the split-bf16 copy of Chat that the
// full step left in the state -- arrives by TMA.  The columns are walked in groups of
// `gc` 64-column chunks: one basis slice (gc*64 x k) per group feeds MMAs of N = gc*64
// (few, wide instructions: a dependent MMA costs ~200 cycles whatever its N), while the R
// tiles of the group's chunks stream through their own ring and meet the accumulator in
// the epilogue.
//
// Warp roles (320 threads): 0 = TMA producer, 1 = MMA issuer (+ TMEM owner), 2..9 = two
// epilogue groups of four warps (TMEM lane quarter = warp % 4; group g takes the chunks
// whose running index is g modulo 2).  Each epilogue warp owns a 32-row slab of the chunk
// from the TMEM read to its own TMA store, so the eight warps never meet at a barrier.
// ======================================================================================
constexpr int kThreadsCached = 320;
constexpr int kSlabRows = 32;                              // rows one epilogue warp stores
constexpr uint32_t kSlabBytes = kSlabRows * kTileCols * 2; // 4 KB

__global__ void __launch_bounds__(kThreadsCached, 1)
umma_cached_kernel(const __grid_constant__ CUtensorMap tm_r, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_ahi, const __grid_constant__ CUtensorMap tm_alo,
                   const __grid_constant__ CUtensorMap tm_out, const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_base0 = base;
    const uint32_t v_base0 = a_base0 + (uint32_t)p.a_bufs * p.a_bytes;
    const uint32_t stage0 = v_base0 + (uint32_t)p.v_slots * p.vslice_bytes;
    const Bars bar = bars_at(stage0 + (uint32_t)p.stages * kTileBytes);
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen_base + (bar.abort_flag - base));
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen_base + (bar.tmem_slot - base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tmem_cols = 512;

    if (threadIdx.x == 0) {
        // R slot: free again once the four slab stores have read it.  Accumulator: four
        // arrivals (one per lane quarter) for each of the gc chunks of a group.
        for (int s = 0; s < p.stages; ++s) { mbar_init(bar.full + 8 * s, 1); mbar_init(bar.empty + 8 * s, 4); }
        for (int s = 0; s < p.acc_stages; ++s) { mbar_init(bar.acc_full + 8 * s, 1); mbar_init(bar.acc_empty + 8 * s, 4 * p.gc); }
        for (int s = 0; s < p.a_bufs; ++s) { mbar_init(bar.a_full + 8 * s, 1); mbar_init(bar.a_empty + 8 * s, 1); }
        for (int s = 0; s < p.v_slots; ++s) { mbar_init(bar.v_full + 8 * s, 1); mbar_init(bar.v_empty + 8 * s, 1); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_r);
        prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_ahi);
        prefetch_tensormap(&tm_alo);
        prefetch_tensormap(&tm_out);
    }
    if (warp == 1) {
        tmem_alloc(bar.tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer ---
        if (lane == 0) {
            uint32_t it = 0, ig = 0, ui = 0, ua = 0;   // chunks, groups, units started; A tiles requested
            int u_a = blockIdx.x;                      // unit cursor of the A-tile requests (runs ahead)
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit un = decode_unit(p, u);
                if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) {
                    if (un.rt == 0 && un.c0 == 0) header_of(p, un.b)->status = SVDCACHE_ERR_STATE;
                    continue;
                }
                // request the A tiles of this unit and of the next a_bufs - 1 live units
                while (ua < ui + (uint32_t)p.a_bufs && u_a < p.units) {
                    const Unit ux = decode_unit(p, u_a);
                    u_a += gridDim.x;
                    if (*(volatile uint32_t *)&header_of(p, ux.b)->full_steps == 0) continue;
                    const uint32_t ab = ua % p.a_bufs;
                    if (!mbar_wait(bar.a_empty + 8 * ab, ((ua / p.a_bufs) & 1u) ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    const uint32_t dst = a_base0 + ab * p.a_bytes;
                    mbar_arrive_expect_tx(bar.a_full + 8 * ab, p.a_bytes);
                    for (int kb = 0; kb < p.nkb; ++kb) {
                        tma_load_3d(dst + kb * (kTileRows * p.kb_bytes), &tm_ahi, bar.a_full + 8 * ab,
                                    kb * p.kb_elems, ux.rt * kTileRows, ux.b);
                        tma_load_3d(dst + p.a_half_bytes + kb * (kTileRows * p.kb_bytes), &tm_alo, bar.a_full + 8 * ab,
                                    kb * p.kb_elems, ux.rt * kTileRows, ux.b);
                    }
                    ++ua;
                }
                ++ui;
                for (int cg = un.c0; cg < un.c1; cg += p.gc, ++ig) {
                    const uint32_t vs = ig % p.v_slots;
                    if (!mbar_wait(bar.v_empty + 8 * vs, ((ig / p.v_slots) & 1u) ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    const uint32_t vdst = v_base0 + vs * p.vslice_bytes;
                    mbar_arrive_expect_tx(bar.v_full + 8 * vs, p.vslice_bytes);
                    for (int kb = 0; kb < p.nkb; ++kb)
                        tma_load_3d(vdst + kb * (p.gc * kTileCols * p.kb_bytes), &tm_v, bar.v_full + 8 * vs,
                                    kb * p.kb_elems, cg * kTileCols, un.b);
                    const int ce = min(cg + p.gc, un.c1);
                    for (int c = cg; c < ce; ++c, ++it) {
                        const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                        if (!mbar_wait(bar.empty + 8 * s, ph ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                        mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes);
                        tma_load_3d(stage0 + s * kTileBytes, &tm_r, bar.full + 8 * s, c * kTileCols, un.rt * kTileRows, un.b);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer ---
        if (lane == 0) {
            uint32_t ig = 0, ui = 0;
            const int ksteps = p.kb_elems / 16;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit un = decode_unit(p, u);
                if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) continue;
                const uint32_t ab = ui % p.a_bufs;
                if (!mbar_wait(bar.a_full + 8 * ab, (ui / p.a_bufs) & 1u, abort_flag)) { record_timeout(p); goto done; }
                const uint64_t a_desc0 = smem_desc_kmajor(a_base0 + ab * p.a_bytes, p.kb_bytes);
                for (int cg = un.c0; cg < un.c1; cg += p.gc, ++ig) {
                    const uint32_t vs = ig % p.v_slots, as = ig % p.acc_stages;
                    const int nsub = min(p.gc, un.c1 - cg);
                    if (!mbar_wait(bar.v_full + 8 * vs, (ig / p.v_slots) & 1u, abort_flag)) { record_timeout(p); goto done; }
                    if (!mbar_wait(bar.acc_empty + 8 * as, ((ig / p.acc_stages) & 1u) ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    tc_fence_after();
                    const uint32_t idesc = idesc_bf16(kTileRows, nsub * kTileCols);
                    const uint32_t d_tmem = tmem_base + as * p.acc_cols;
                    const uint64_t v_desc0 = smem_desc_kmajor(v_base0 + vs * p.vslice_bytes, p.kb_bytes);
                    uint32_t acc = 0;
                    for (int part = 0; part < 2; ++part)
                        for (int kb = 0; kb < p.nkb; ++kb) {
                            // descriptors address in 16-byte units: add byte offsets >> 4
                            const uint64_t a_kb = a_desc0 + ((part * p.a_half_bytes + kb * (kTileRows * p.kb_bytes)) >> 4);
                            const uint64_t v_kb = v_desc0 + ((kb * (p.gc * kTileCols * p.kb_bytes)) >> 4);
                            for (int ks = 0; ks < ksteps; ++ks) {
                                mma_bf16_ss(d_tmem, a_kb + 2 * ks, v_kb + 2 * ks, idesc, acc);
                                acc = 1;
                            }
                        }
                    mma_commit(bar.v_empty + 8 * vs);
                    mma_commit(bar.acc_full + 8 * as);
                }
                mma_commit(bar.a_empty + 8 * ab);
                ++ui;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue ---
        const int q = warp & 3, row = q * kSlabRows + lane;
        const uint32_t grp = (uint32_t)(warp - 2) >> 2;
        uint32_t it = 0, ig = 0;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
            const Unit un = decode_unit(p, u);
            if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) continue;
            const int slab_row0 = un.rt * kTileRows + q * kSlabRows;
            const bool slab_live = (int64_t)slab_row0 < p.N;
            for (int cg = un.c0; cg < un.c1; cg += p.gc, ++ig) {
                const uint32_t as = ig % p.acc_stages, aph = (ig / p.acc_stages) & 1u;
                const int nsub = min(p.gc, un.c1 - cg);
                for (int j = 0; j < nsub; ++j, ++it) {
                    if ((it & 1u) != grp) continue;
                    const int c = cg + j;
                    const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                    bool ok = mbar_wait(bar.acc_full + 8 * as, aph, abort_flag);
                    ok = ok && mbar_wait(bar.full + 8 * s, ph, abort_flag);
                    if (!__all_sync(0xFFFFFFFFu, ok)) { record_timeout(p); goto done; }
                    tc_fence_after();
                    const uint32_t tile = stage0 + s * kTileBytes + (uint32_t)row * 128u;
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + as * p.acc_cols + j * kTileCols;
                    uint32_t acc0[32], acc1[32];
                    tmem_ld_32x32(taddr, acc0);
                    tmem_ld_32x32(taddr + 32, acc1);
                    uint4 t[8];
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) t[cc] = lds128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    // this quarter's share of the group's accumulator is in registers; the last
                    // chunk of a short group also arrives for the chunks the group does not have
                    if (lane == 0) mbar_arrive_n(bar.acc_empty + 8 * as, j == nsub - 1 ? 1u + (uint32_t)(p.gc - nsub) : 1u);
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc)
                        sts128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u,
                               combine_chunk<false>(t[cc], cc < 4 ? acc0 + cc * 8 : acc1 + (cc - 4) * 8));
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (slab_live)
                            tma_store_3d(&tm_out, stage0 + s * kTileBytes + (uint32_t)q * kSlabBytes, c * kTileCols,
                                         slab_row0, un.b);
                        tma_store_commit();
                        tma_store_wait_read<0>();
                        mbar_arrive(bar.empty + 8 * s);
                    }
                    __syncwarp();
                }
            }
        }
        if (lane == 0) tma_store_wait<0>();
    }

done:
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ======================================================================================
// Full step (Eq. 8 - Eq. 11):  C = F V_k,  Chat <- EMA(C),  R = F - C V_k^T
//
// A unit is one 128-row tile of one block.  Pass 1 streams the tile's F in 64-column
// slices and accumulates C (128 x k, fp32) in TMEM: A = F slice, B = matching slice of
// V_k^T.  The C warps then read C from TMEM, apply the EMA to the state, and write C as a
// split-bf16 A operand.  Pass 2 streams the same F slices again (in reverse order, so the
// most recently touched ones come first and are still in L2) with slices of V_k, forms
// C V_k^T per slice in TMEM, and the epilogue stores R = F - C V_k^T through TMA.
// ======================================================================================
constexpr uint32_t kAcc1Col = kAccStages * kTileCols;   // C accumulator sits after the pass-2 ring

__global__ void __launch_bounds__(kThreadsUmma, 1)
umma_full_kernel(const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_vt,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_rout,
                 const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_base0 = base;
    const uint32_t stage0 = a_base0 + p.a_bytes;
    const Bars bar = bars_at(stage0 + (uint32_t)p.stages * p.stage_bytes);
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen_base + (bar.abort_flag - base));
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen_base + (bar.tmem_slot - base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tmem_cols = 512;
    const int CT = p.chunks_total;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(bar.full + 8 * s, 1); mbar_init(bar.empty + 8 * s, 2); }
        for (int s = 0; s < kAccStages; ++s) { mbar_init(bar.acc_full + 8 * s, 1); mbar_init(bar.acc_empty + 8 * s, 128); }
        mbar_init(bar.a_full, 128);
        mbar_init(bar.c_full, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_f);
        prefetch_tensormap(&tm_vt);
        prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_rout);
    }
    if (warp == 1) {
        tmem_alloc(bar.tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer ---
        if (lane == 0) {
            uint32_t it = 0;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit un = decode_unit(p, u);
                for (int c = 0; c < CT; ++c, ++it) {            // pass 1: F slice + V^T slice
                    const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                    if (!mbar_wait(bar.empty + 8 * s, ph ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    const uint32_t slot = stage0 + s * p.stage_bytes;
                    mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes + (uint32_t)p.k * 128u);
                    tma_load_3d(slot, &tm_f, bar.full + 8 * s, c * kTileCols, un.rt * kTileRows, un.b);
                    tma_load_3d(slot + kTileBytes, &tm_vt, bar.full + 8 * s, c * kTileCols, 0, un.b);
                }
                for (int c2 = 0; c2 < CT; ++c2, ++it) {         // pass 2: F slice again + V slice
                    const int c = CT - 1 - c2;
                    const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                    if (!mbar_wait(bar.empty + 8 * s, ph ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    const uint32_t slot = stage0 + s * p.stage_bytes;
                    mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes + p.v_bytes);
                    tma_load_3d(slot, &tm_f, bar.full + 8 * s, c * kTileCols, un.rt * kTileRows, un.b);
                    for (int kb = 0; kb < p.nkb; ++kb)
                        tma_load_3d(slot + kTileBytes + kb * (kTileCols * p.kb_bytes), &tm_v, bar.full + 8 * s,
                                    kb * p.kb_elems, c * kTileCols, un.b);
                }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer ---
        if (lane == 0) {
            uint32_t it = 0, ia = 0, ui = 0;
            const uint32_t idesc1 = idesc_bf16(kTileRows, p.k);
            for (int u = blockIdx.x; u < p.units; u += gridDim.x, ++ui) {
                for (int c = 0; c < CT; ++c, ++it) {            // pass 1: C += F_slice * (V^T slice)^T
                    const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                    if (!mbar_wait(bar.full + 8 * s, ph, abort_flag)) { record_timeout(p); goto done; }
                    tc_fence_after();
                    const uint32_t slot = stage0 + s * p.stage_bytes;
#pragma unroll
                    for (int ks = 0; ks < kTileCols / 16; ++ks)
                        mma_bf16_ss(tmem_base + kAcc1Col, smem_desc_kmajor(slot + ks * 32, 128),
                                    smem_desc_kmajor(slot + kTileBytes + ks * 32, 128), idesc1,
                                    (c | ks) != 0 ? 1u : 0u);
                    mma_commit(bar.empty + 8 * s);
                    mbar_arrive(bar.empty + 8 * s);   // the F slice is not stored in pass 1: second arrival
                }
                mma_commit(bar.c_full);
                if (!mbar_wait(bar.a_full, ui & 1u, abort_flag)) { record_timeout(p); goto done; }
                tc_fence_after();
                for (int c2 = 0; c2 < CT; ++c2, ++it, ++ia) {   // pass 2: acc = C * (V slice)^T
                    const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                    const uint32_t as = ia % kAccStages, aph = (ia / kAccStages) & 1u;
                    if (!mbar_wait(bar.full + 8 * s, ph, abort_flag)) { record_timeout(p); goto done; }
                    if (!mbar_wait(bar.acc_empty + 8 * as, aph ^ 1u, abort_flag)) { record_timeout(p); goto done; }
                    tc_fence_after();
                    issue_reconstruct_mmas(p, tmem_base + as * kTileCols, a_base0,
                                           stage0 + s * p.stage_bytes + kTileBytes);
                    mma_commit(bar.empty + 8 * s);
                    mma_commit(bar.acc_full + 8 * as);
                }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------- epilogue: R = F - C V_k^T, TMA store ---
        const int q = warp & 3, row = q * 32 + lane;
        const bool leader = (warp == 2 && lane == 0);
        uint32_t it = 0, ia = 0;
        int prev_stage = -1;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
            const Unit un = decode_unit(p, u);
            it += CT;   // pass 1 stages are consumed by the MMA warp alone
            for (int c2 = 0; c2 < CT; ++c2, ++it, ++ia) {
                const int c = CT - 1 - c2;
                const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                const uint32_t as = ia % kAccStages, aph = (ia / kAccStages) & 1u;
                bool ok = mbar_wait(bar.acc_full + 8 * as, aph, abort_flag);
                ok = ok && mbar_wait(bar.full + 8 * s, ph, abort_flag);
                if (ok) {
                    tc_fence_after();
                    const uint32_t tile = stage0 + s * p.stage_bytes + (uint32_t)row * 128u;
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + as * kTileCols;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t acc[32];
                        tmem_ld_32x32(taddr + half * 32, acc);
                        tmem_wait_ld();
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            const uint32_t addr = tile + (((uint32_t)(half * 4 + cc)) ^ ((uint32_t)row & 7u)) * 16u;
                            sts128(addr, combine_chunk<true>(lds128(addr), acc + cc * 8));
                        }
                    }
                    tc_fence_before();
                    mbar_arrive(bar.acc_empty + 8 * as);
                    fence_proxy_async();
                } else {
                    record_timeout(p);
                }
                named_barrier_sync(1, 128);
                if (leader && ok) {
                    tma_store_3d(&tm_rout, stage0 + s * p.stage_bytes, c * kTileCols, un.rt * kTileRows, un.b);
                    tma_store_commit();
                    // A stage goes back to the producer once its store has read it.  Inside a
                    // unit that is checked one tile late; the unit's last tile is released at
                    // once, because the next unit's pass 1 needs the whole ring to get going.
                    if (c2 == CT - 1) {
                        tma_store_wait_read<0>();
                        if (prev_stage >= 0) mbar_arrive(bar.empty + 8 * prev_stage);
                        mbar_arrive(bar.empty + 8 * s);
                        prev_stage = -1;
                    } else {
                        if (prev_stage >= 0) {
                            tma_store_wait_read<1>();
                            mbar_arrive(bar.empty + 8 * prev_stage);
                        }
                        prev_stage = (int)s;
                    }
                }
            }
        }
        if (leader) {
            tma_store_wait_read<0>();
            if (prev_stage >= 0) mbar_arrive(bar.empty + 8 * prev_stage);
            tma_store_wait<0>();
        }
    } else {
        // --------------------------- C warps: TMEM -> EMA on the state -> split-bf16 A operand ---
        const int q = warp & 3, row = q * 32 + lane;
        const float beta = p.beta, omb = 1.0f - p.beta;
        uint32_t ui = 0;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x, ++ui) {
            const Unit un = decode_unit(p, u);
            StateHeader *hdr = header_of(p, un.b);
            const bool first = *(volatile uint32_t *)&hdr->full_steps == 0;
            if (!mbar_wait(bar.c_full, ui & 1u, abort_flag)) { record_timeout(p); goto done; }
            tc_fence_after();
            const int64_t n = (int64_t)un.rt * kTileRows + row;
            float *chat = reinterpret_cast<float *>(p.state + (size_t)un.b * p.state_stride + p.chat_off) + n * p.k;
            float *cout = p.C_out ? reinterpret_cast<float *>((char *)p.C_out + (size_t)un.b * p.C_stride) + n * p.k
                                  : nullptr;
            char *st_b = p.state + (size_t)un.b * p.state_stride;
            __nv_bfloat16 *ophi = reinterpret_cast<__nv_bfloat16 *>(st_b + p.ophi_off) + n * p.k;
            __nv_bfloat16 *oplo = reinterpret_cast<__nv_bfloat16 *>(st_b + p.oplo_off) + n * p.k;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + kAcc1Col;
            for (int g = 0; g * 32 < p.k; ++g) {
                uint32_t acc[32];
                tmem_ld_32x32(taddr + g * 32, acc);
                tmem_wait_ld();
#pragma unroll
                for (int j4 = 0; j4 < 8; ++j4) {
                    const int j = g * 32 + j4 * 4;
                    if (j < p.k) {
                        const float4 cv = make_float4(__uint_as_float(acc[j4 * 4]), __uint_as_float(acc[j4 * 4 + 1]),
                                                      __uint_as_float(acc[j4 * 4 + 2]), __uint_as_float(acc[j4 * 4 + 3]));
                        if (n < p.N) {
                            float4 ch = cv;
                            if (!first) {
                                const float4 pv = *reinterpret_cast<const float4 *>(chat + j);
                                ch.x = fmaf(beta, pv.x, omb * cv.x);
                                ch.y = fmaf(beta, pv.y, omb * cv.y);
                                ch.z = fmaf(beta, pv.z, omb * cv.z);
                                ch.w = fmaf(beta, pv.w, omb * cv.w);
                            }
                            *reinterpret_cast<float4 *>(chat + j) = ch;
                            if (cout) *reinterpret_cast<float4 *>(cout + j) = cv;
                            __nv_bfloat16 h[4], l[4];
                            split_bf16(ch.x, h[0], l[0]);
                            split_bf16(ch.y, h[1], l[1]);
                            split_bf16(ch.z, h[2], l[2]);
                            split_bf16(ch.w, h[3], l[3]);
                            *reinterpret_cast<uint2 *>(ophi + j) = *reinterpret_cast<const uint2 *>(h);
                            *reinterpret_cast<uint2 *>(oplo + j) = *reinterpret_cast<const uint2 *>(l);
                        }
                        store_a4(a_base0, p, row, j, cv);
                    }
                }
            }
            tc_fence_before();
            fence_proxy_async();
            mbar_arrive(bar.a_full);
            // count this unit; the last unit of a block to get here counts the full step
            if (warp == 6 && lane == 0) {
                const uint32_t prev = atomicAdd(&hdr->done, 1u);
                if (prev == (uint32_t)p.row_tiles - 1u) {
                    hdr->done = 0;
                    hdr->full_steps = hdr->full_steps + 1;
                }
            }
        }
    }

done:
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ------------------------------------------------------------------------- host side ---

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// bf16 tensor (inner, rows, blocks) with byte pitches; box (box_inner, box_rows, 1)
int make_map(CUtensorMap *m, const void *base, uint64_t inner, uint64_t rows, uint64_t blocks, uint64_t row_pitch,
             uint64_t block_pitch, uint32_t box_inner, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SVDCACHE_ERR_CUDA;
    const cuuint64_t dims[3] = {inner, rows, blocks};
    if (blocks <= 1 || block_pitch == 0) block_pitch = row_pitch * rows;
    block_pitch = (block_pitch + 15) / 16 * 16;
    const cuuint64_t strides[2] = {row_pitch, block_pitch};
    const cuuint32_t box[3] = {box_inner, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const uint32_t inner_bytes = box_inner * 2;
    const CUtensorMapSwizzle sw = inner_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : inner_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                      : CU_TENSOR_MAP_SWIZZLE_32B;
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDCACHE_OK : SVDCACHE_ERR_CUDA;
}

int num_sms() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

constexpr size_t kSmemBudget = 227 * 1024;

bool fill_params(const StepArgs &a, UmmaParams &p, int want_a_bufs) {
    p.N = a.N; p.D = a.D; p.k = a.k; p.nblocks = a.nblocks;
    p.row_tiles = (int)((a.N + kTileRows - 1) / kTileRows);
    p.chunks_total = (a.D + kTileCols - 1) / kTileCols;
    p.kb_elems = a.k < 64 ? a.k : 64;
    p.kb_bytes = p.kb_elems * 2;
    p.nkb = a.k / p.kb_elems;
    p.a_half_bytes = (uint32_t)kTileRows * a.k * 2;
    p.a_bytes = 2 * p.a_half_bytes;
    p.v_bytes = (uint32_t)kTileCols * a.k * 2;
    p.stage_bytes = kTileBytes + ((p.v_bytes + 1023u) & ~1023u);
    const size_t avail = kSmemBudget - 1024 /*alignment*/ - kBarBytes - 64;
    p.a_bufs = (want_a_bufs == 2 && 2 * (size_t)p.a_bytes + 4 * (size_t)p.stage_bytes <= avail) ? 2 : 1;
    if ((size_t)p.a_bufs * p.a_bytes + 2 * (size_t)p.stage_bytes > avail) return false;
    p.stages = (int)((avail - (size_t)p.a_bufs * p.a_bytes) / p.stage_bytes);
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    p.state = (char *)a.state;
    p.state_stride = a.state_stride;
    {
        const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
        p.chat_off = SL.chat; p.ophi_off = SL.op_hi; p.oplo_off = SL.op_lo;
    }
    p.C_out = a.C_out;
    p.C_stride = a.C_stride;
    p.beta = a.beta;
    return true;
}

// Cached step: shared memory = A tile(s) | basis-slice ring | R ring | barriers.
bool fill_cached(const StepArgs &a, UmmaParams &p) {
    if (!fill_params(a, p, 1)) return false;
    p.gc = 16384 / (kTileCols * a.k);            // basis slice (gc * 64 x k bf16) of at most 32 KB
    if (p.gc > 4) p.gc = 4;                      // MMA N = gc * 64 <= 256
    if (p.gc < 1) p.gc = 1;
    p.acc_cols = p.gc * kTileCols;
    p.acc_stages = 512 / p.acc_cols < kAccStages ? 512 / p.acc_cols : kAccStages;
    p.vslice_bytes = (uint32_t)p.gc * kTileCols * a.k * 2;
    p.v_slots = kMaxVSlots;
    const size_t avail = kSmemBudget - 1024 /*alignment*/ - kBarBytes - 64;
    const size_t fixed = (size_t)p.v_slots * p.vslice_bytes;
    p.a_bufs = (2 * (size_t)p.a_bytes + fixed + 6 * (size_t)kTileBytes <= avail) ? 2 : 1;
    if ((size_t)p.a_bufs * p.a_bytes + fixed + 2 * (size_t)kTileBytes > avail) return false;
    p.stages = (int)((avail - (size_t)p.a_bufs * p.a_bytes - fixed) / kTileBytes);
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    return true;
}
size_t smem_bytes_cached(const UmmaParams &p) {
    return 1024 + (size_t)p.a_bufs * p.a_bytes + (size_t)p.v_slots * p.vslice_bytes + (size_t)p.stages * kTileBytes +
           kBarBytes + 64;
}

size_t smem_bytes(const UmmaParams &p) {
    return 1024 + (size_t)p.a_bufs * p.a_bytes + (size_t)p.stages * p.stage_bytes + kBarBytes + 64;
}

bool shape_ok(const StepArgs &a) {
    if (a.dtype != SVDCACHE_BF16) return false;
    if (!(a.k == 16 || a.k == 32 || (a.k % 64) == 0)) return false;
    if (a.D < 64 || a.N < 1 || a.N > 0x7FFFFFFFLL) return false;
    return encode_fn() != nullptr;
}

}  // namespace

bool umma_supported(const StepArgs &a, bool full) {
    if (!shape_ok(a)) return false;
    UmmaParams p;
    return full ? fill_params(a, p, 1) : fill_cached(a, p);
}

int umma_cached_step(const StepArgs &a, cudaStream_t s) {
    UmmaParams p{};
    if (!fill_cached(a, p)) return SVDCACHE_ERR_BAD_SHAPE;
    // Split D across CTAs only when there are too few row tiles to occupy the GPU: pick the
    // split (in whole MMA groups) that minimises the chunks the busiest CTA has to stream.
    const int tiles = p.row_tiles * a.nblocks;
    const int groups_total = (p.chunks_total + p.gc - 1) / p.gc;
    int best_load = 1 << 30;
    p.dsplit = 1;
    p.chunks_per_slice = p.chunks_total;
    for (int ds = 1; ds <= groups_total && ds <= 16; ++ds) {
        const int gps = (groups_total + ds - 1) / ds;            // groups per slice
        const int eff = (groups_total + gps - 1) / gps;          // slices that result
        const int rounds = (tiles * eff + num_sms() - 1) / num_sms();
        if (rounds * gps < best_load) { best_load = rounds * gps; p.dsplit = eff; p.chunks_per_slice = gps * p.gc; }
    }
    p.units = tiles * p.dsplit;

    const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
    const BasisLayout BL = basis_layout(a.D, a.k, a.dtype);
    CUtensorMap tm_r, tm_v, tm_ahi, tm_alo, tm_out;
    int rc = make_map(&tm_r, (const char *)a.state + SL.r, a.D, a.N, a.nblocks, (uint64_t)a.D * 2, a.state_stride,
                      kTileCols, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_v, (const char *)a.basis + BL.v_bf16, a.k, a.D, a.nblocks, (uint64_t)a.k * 2, a.basis_stride,
                  p.kb_elems, p.gc * kTileCols);
    if (rc) return rc;
    rc = make_map(&tm_ahi, (const char *)a.state + SL.op_hi, a.k, a.N, a.nblocks, (uint64_t)a.k * 2, a.state_stride,
                  p.kb_elems, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_alo, (const char *)a.state + SL.op_lo, a.k, a.N, a.nblocks, (uint64_t)a.k * 2, a.state_stride,
                  p.kb_elems, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_out, a.Fhat, a.D, a.N, a.nblocks, (uint64_t)a.ld * 2, a.Fhat_stride, kTileCols, kSlabRows);
    if (rc) return rc;

    const size_t smem = smem_bytes_cached(p);
    static bool attr_set = false;
    if (!attr_set) {
        rc = record_cuda(cudaFuncSetAttribute(umma_cached_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kSmemBudget));
        if (rc) return rc;
        attr_set = true;
    }
    const int grid = p.units < num_sms() ? p.units : num_sms();
    umma_cached_kernel<<<grid, kThreadsCached, smem, s>>>(tm_r, tm_v, tm_ahi, tm_alo, tm_out, p);
    count_launch();
    return check_last_launch();
}

int umma_full_step(const StepArgs &a, cudaStream_t s) {
    UmmaParams p{};
    if (!fill_params(a, p, 1)) return SVDCACHE_ERR_BAD_SHAPE;
    p.dsplit = 1;
    p.chunks_per_slice = p.chunks_total;
    p.units = p.row_tiles * a.nblocks;

    const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
    const BasisLayout BL = basis_layout(a.D, a.k, a.dtype);
    CUtensorMap tm_f, tm_vt, tm_v, tm_rout;
    int rc = make_map(&tm_f, a.F, a.D, a.N, a.nblocks, (uint64_t)a.ld * 2, a.F_stride, kTileCols, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_vt, (const char *)a.basis + BL.vt_bf16, a.D, a.k, a.nblocks, (uint64_t)a.D * 2,
                  a.basis_stride, kTileCols, a.k);
    if (rc) return rc;
    rc = make_map(&tm_v, (const char *)a.basis + BL.v_bf16, a.k, a.D, a.nblocks, (uint64_t)a.k * 2, a.basis_stride,
                  p.kb_elems, kTileCols);
    if (rc) return rc;
    rc = make_map(&tm_rout, (char *)a.state + SL.r, a.D, a.N, a.nblocks, (uint64_t)a.D * 2, a.state_stride,
                  kTileCols, kTileRows);
    if (rc) return rc;

    const size_t smem = smem_bytes(p);
    static bool attr_set = false;
    if (!attr_set) {
        rc = record_cuda(cudaFuncSetAttribute(umma_full_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kSmemBudget));
        if (rc) return rc;
        attr_set = true;
    }
    const int grid = p.units < num_sms() ? p.units : num_sms();
    umma_full_kernel<<<grid, kThreadsUmma, smem, s>>>(tm_f, tm_vt, tm_v, tm_rout, p);
    count_launch();
    return check_last_launch();
}

bool umma_gram_supported(int64_t, int, int64_t, int) { return false; }
size_t umma_gram_scratch_bytes(int) { return 0; }
int umma_gram_accumulate(const void *, int64_t, int, int64_t, double *, void *, size_t, cudaStream_t) {
    return SVDCACHE_ERR_BAD_SHAPE;
}

}  // namespace svdc
