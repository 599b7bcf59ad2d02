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
#include <cstdlib>
#include <mutex>

#include "internal.cuh"
#include "umma.cuh"

namespace svdc {

using namespace sm100;

#ifdef SVDC_TRACE
__device__ unsigned long long g_trace[148 * 16 * 8];
#endif

namespace {

constexpr int kTileRows = 128;      // MMA M
constexpr int kTileCols = 64;       // columns of D per stage (MMA N in the reconstruct GEMM)
constexpr int kTileBytes = kTileRows * kTileCols * 2;   // 16 KB
constexpr int kAccStages = 4;       // TMEM accumulator ring (64 fp32 columns each)
constexpr int kMaxStages = 12;
constexpr int kMaxVSlots = 4;
constexpr int kMaxABufs = 2;

struct UmmaParams {
    int64_t N;
    int D, k, nblocks;
    int row_tiles, chunks_total, dsplit, chunks_per_slice, units;
    int kb_elems, kb_bytes, nkb;         // K-block of the rank dimension: min(k, 64) elements
    int stages, a_bufs;
    uint32_t a_half_bytes, a_bytes;
    int gc, acc_stages, acc_cols, v_slots;   // chunks per MMA group, TMEM ring, basis ring
    int acc_stride;                          // TMEM columns per stage of the accumulator ring
    int acc_base;                            // cached step: first TMEM column of the accumulator ring (operand buffers before it)
    uint32_t vslice_bytes;
    uint32_t a_region_bytes, chat_stage_off; // full step: A operand (+ Chat staging when it is not in place)
    char *state;
    size_t state_stride, chat_off, ophi_off, oplo_off;
    float *C_out;
    size_t C_stride;
    float beta;
    float beta_r;          // full step: EMA weight of the stored residual (0: the residual is replaced)
    size_t r_off;          // offset of R in a block's state
    int r_slots;           // full step with residual EMA: slots of the ring the old R streams through
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

// A wait ran out: make the status sticky and leave a diagnosis in block 0's state header --
// `pad` = (site of the first wait of the first CTA to give up) << 16 | that CTA, and, for
// each warp of that CTA that got here, four words at byte 64 + 16 * warp: its own view of
// the site and three progress counters of its role.
__device__ __forceinline__ void record_timeout(const UmmaParams &p, volatile int *abort_flag, uint32_t c0 = 0,
                                               uint32_t c1 = 0, uint32_t c2 = 0) {
    StateHeader *h = header_of(p, 0);
    atomicExch(&h->status, SVDCACHE_ERR_TIMEOUT);
    const uint32_t mine = ((uint32_t)*abort_flag << 16) | (blockIdx.x & 0xFFFFu);
    atomicCAS(&h->pad, 0u, mine);
    if ((*(volatile uint32_t *)&h->pad & 0xFFFFu) == (blockIdx.x & 0xFFFFu) && (threadIdx.x & 31u) == 0u) {
        uint32_t *w = reinterpret_cast<uint32_t *>(h) + 16 + 4 * (threadIdx.x >> 5);
        w[0] = mine; w[1] = c0; w[2] = c1; w[3] = c2;
    }
}

// Every CTA of a full-step launch reports here when it has nothing left to do; the last one
// counts the step in every block's header.  No CTA reads full_steps after its own report, so
// the first-step test of the EMA (Eq. 11) sees one value for the whole launch, whatever the
// order in which the warps of a CTA and the CTAs of the grid get to their tiles.
__device__ __forceinline__ void report_exit_and_count_step(const UmmaParams &p) {
    StateHeader *h0 = header_of(p, 0);
    __threadfence();
    const uint32_t prev = atomicAdd(&h0->exits, 1u);
    if (prev == gridDim.x - 1u) {
        __threadfence();
        for (int b = 0; b < p.nblocks; ++b) {
            StateHeader *h = header_of(p, b);
            h->full_steps = h->full_steps + 1;
        }
        h0->exits = 0;
    }
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

// The same for the residual EMA of the ablation (Sec. 4.5): out = beta_r * old + (1 - beta_r) * (tile - acc),
// formed in fp32 and rounded once
__device__ __forceinline__ uint4 combine_chunk_ema(uint4 t, const uint32_t *acc, uint4 old, float beta_r) {
    const uint32_t w[4] = {t.x, t.y, t.z, t.w}, ow[4] = {old.x, old.y, old.z, old.w};
    uint32_t o[4];
    const float omb = 1.0f - beta_r;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        const float olo = __uint_as_float(ow[i] << 16), ohi = __uint_as_float(ow[i] & 0xFFFF0000u);
        const float r0 = lo - __uint_as_float(acc[2 * i]), r1 = hi - __uint_as_float(acc[2 * i + 1]);
        const __nv_bfloat162 pk = __floats2bfloat162_rn(fmaf(beta_r, olo, omb * r0), fmaf(beta_r, ohi, omb * r1));
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
// Position in a ring of n slots -- slot index and phase parity -- advanced without dividing:
// the roles below are serial instruction chains, and a division by a run-time ring size
// costs each of them ~100 cycles per chunk.
struct RingPos {
    uint32_t idx = 0, ph = 0;
    __device__ __forceinline__ void step(uint32_t n) { if (++idx == n) { idx = 0; ph ^= 1u; } }
    __device__ __forceinline__ void skip(uint32_t k, uint32_t n) { const uint32_t t = idx + k; idx = t % n; ph ^= (t / n) & 1u; }
};

// Every epilogue warp waits for every accumulator of the ring, in order, and arrives on its
// "empty" barrier once per group -- after reading its last chunk of the group, or at once if
// the group holds none of its chunks.  A waiter that skipped a phase of an mbarrier could
// take the completion of the phase before it for the one it wants (parities alias), and one
// that does not gate the reuse could fall two phases behind; waiting on every phase and
// gating each reuse rules both out.  Returns the index (within the group) of the last chunk
// that belongs to epilogue group `grp`, or -1: chunk j of the group has running index
// it0 + j and belongs to group (it0 + j) & 1.
__device__ __forceinline__ int last_own_chunk(uint32_t it0, int nsub, uint32_t grp) {
    int last = nsub - 1;
    if (((it0 + (uint32_t)last) & 1u) != grp) --last;
    return last;   // -1 when nsub == 1 and the only chunk is the other group's
}

// ======================================================================================
// Cached step (Sec. 3.5):  Fhat = Chat V_k^T + R
//
// A unit is one 128-row tile of one block (times a column range when the launch is too
// small to occupy the GPU otherwise).  Its A operand is the split-bf16 copy of Chat that the
// full step left in the state (or a forecast of it).  The columns are walked in groups of
// `gc` 64-column chunks: one basis slice (gc*64 x k) per group feeds MMAs of N = gc*64
// (few, wide instructions: an MMA of M = 128, K = 16 costs ~105 cycles up to N = 128), while the
// R tiles of the group's chunks stream through their own ring and meet the accumulator in
// the epilogue.
//
// Where the operand lives:
//   k <= 64   two shared-memory buffers (32 KB each at k = 64), filled by TMA one unit ahead;
//   k >= 128  tensor memory (kTmemA).  The tile's 2 * nkb pieces (hi and lo words of every 64-wide K
//     block, 16 KB each) travel through the R ring like any chunk, one unit ahead of their use;
//     the epilogue warps move them into TMEM (128 bytes of a row = 32 columns, two bf16 each) and
//     the MMAs take their A operand from there.  TMEM columns: a_bufs * k of operand (two buffers
//     at k = 128, one above), then the accumulator ring.  All of shared memory goes to the rings.
//
// Warp roles (320 threads): 0 = TMA producer (lane 0: R tiles and basis slices -- and the operand
// pieces when they go through the ring --, lane 1: operand tiles for the shared-memory buffers),
// 1 = MMA issuer (+ TMEM owner), 2..9 = two epilogue groups of four warps (TMEM lane quarter =
// warp % 4; group g takes the chunks whose running index is g modulo 2).  Each epilogue warp owns a
// 32-row slab of the chunk from the TMEM read to its own TMA store, so the eight warps never meet
// at a barrier.
// ======================================================================================
constexpr int kThreadsCached = 320;
constexpr int kSlabRows = 32;                              // rows one epilogue warp stores
constexpr uint32_t kSlabBytes = kSlabRows * kTileCols * 2; // 4 KB

template <bool kTmemA>
__global__ void __launch_bounds__(kThreadsCached, 1)
umma_cached_kernel(const __grid_constant__ CUtensorMap tm_r, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_ahi, const __grid_constant__ CUtensorMap tm_alo,
                   const __grid_constant__ CUtensorMap tm_out, const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_base0 = base;
    const uint32_t v_base0 = a_base0 + (kTmemA ? 0u : (uint32_t)p.a_bufs * p.a_bytes);
    const uint32_t stage0 = v_base0 + (uint32_t)p.v_slots * p.vslice_bytes;
    const Bars bar = bars_at(stage0 + (uint32_t)p.stages * kTileBytes);
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen_base + (bar.abort_flag - base));
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen_base + (bar.tmem_slot - base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    SVDC_TRACE_DECL
    const uint32_t tmem_cols = 512;
    // kTmemA (k >= 128): the operand tile travels through the R ring as 2 * nkb ordinary chunks
    // (hi and lo part of every 64-wide K block) and the epilogue warps copy it into tensor memory
    const int n_a_chunks = 2 * p.nkb;
    // units this CTA works on: those of blocks that have seen a full step
    auto next_live = [&](int u) {
        while (u < p.units && *(volatile uint32_t *)&header_of(p, decode_unit(p, u).b)->full_steps == 0) u += (int)gridDim.x;
        return u;
    };
    // the operand of the next unit is requested, and copied, right before the R chunks of this group
    // of the current one: the first with two operand buffers, the last with one (its MMAs, the last
    // readers of the buffer, have their basis slice requested by then)
    auto insert_group = [&](const Unit &un) { return p.a_bufs > 1 ? 0 : (un.c1 - un.c0 + p.gc - 1) / p.gc - 1; };

    if (threadIdx.x == 0) {
        // R slot: free again once the four slab stores have read it.  Accumulator: one arrival
        // from each of the eight epilogue warps per group (see group_share below).
        for (int s = 0; s < p.stages; ++s) { mbar_init(bar.full + 8 * s, 1); mbar_init(bar.empty + 8 * s, 4); }
        for (int s = 0; s < p.acc_stages; ++s) { mbar_init(bar.acc_full + 8 * s, 1); mbar_init(bar.acc_empty + 8 * s, 8); }
        for (int s = 0; s < p.a_bufs; ++s) {   // operand in TMEM: four warps announce each of its chunks
            mbar_init(bar.a_full + 8 * s, kTmemA ? 4u * (uint32_t)n_a_chunks : 1u);
            mbar_init(bar.a_empty + 8 * s, 1);
        }
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
        // Operand in shared memory (k <= 64, two buffers): the A tile of live unit number ua (of unit
        // ux) is requested on a lane of its own, one unit ahead of the MMAs, and never holds up the R
        // and basis streams (+4 % on the FLUX shape).
        auto request_a = [&](const Unit &ux, uint32_t ua) {
            const uint32_t ab = ua % p.a_bufs;
            SVDC_TRACE_MARK(p0);
            if (!mbar_wait(bar.a_empty + 8 * ab, ((ua / p.a_bufs) & 1u) ^ 1u, abort_flag, 1)) return false;
            SVDC_TRACE_ADD(0, p0);
            const uint32_t dst = a_base0 + ab * p.a_bytes;
            mbar_arrive_expect_tx(bar.a_full + 8 * ab, p.a_bytes);
            for (int kb = 0; kb < p.nkb; ++kb) {
                tma_load_3d(dst + kb * (kTileRows * p.kb_bytes), &tm_ahi, bar.a_full + 8 * ab,
                            kb * p.kb_elems, ux.rt * kTileRows, ux.b);
                tma_load_3d(dst + p.a_half_bytes + kb * (kTileRows * p.kb_bytes), &tm_alo, bar.a_full + 8 * ab,
                            kb * p.kb_elems, ux.rt * kTileRows, ux.b);
            }
            return true;
        };
        if constexpr (kTmemA) {
            if (lane == 0) {
                RingPos fr, vr;                        // next ring slot, next basis slot
                auto mark_dead = [&](int u0, int u1) {   // blocks without a full step: report once per block
                    for (int u = u0; u < u1 && u < p.units; u += (int)gridDim.x) {
                        const Unit x = decode_unit(p, u);
                        if (x.rt == 0 && x.c0 == 0 && *(volatile uint32_t *)&header_of(p, x.b)->full_steps == 0)
                            header_of(p, x.b)->status = SVDCACHE_ERR_STATE;
                    }
                };
                auto request_a_chunks = [&](const Unit &ux) {   // hi K block 0, lo K block 0, hi K block 1, ...
                    for (int i = 0; i < n_a_chunks; ++i) {
                        const uint32_t s = fr.idx;
                        SVDC_TRACE_MARK(p0);
                        if (!mbar_wait(bar.empty + 8 * s, fr.ph ^ 1u, abort_flag, 1)) return false;
                        SVDC_TRACE_ADD(0, p0);
                        fr.step((uint32_t)p.stages);
                        mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes);
                        tma_load_3d(stage0 + s * kTileBytes, (i & 1) ? &tm_alo : &tm_ahi, bar.full + 8 * s,
                                    (i >> 1) * p.kb_elems, ux.rt * kTileRows, ux.b);
                    }
                    return true;
                };
                int u = next_live((int)blockIdx.x);
                mark_dead((int)blockIdx.x, u);
                if (u < p.units && !request_a_chunks(decode_unit(p, u))) { record_timeout(p, abort_flag); goto done; }
                while (u < p.units) {
                    const Unit un = decode_unit(p, u);
                    const int u_next = next_live(u + (int)gridDim.x);
                    mark_dead(u + (int)gridDim.x, u_next);
                    const int g_ins = insert_group(un);
                    int g = 0;
                    for (int cg = un.c0; cg < un.c1; cg += p.gc, ++g) {
                        const uint32_t vs = vr.idx;
                        SVDC_TRACE_MARK(p1);
                        if (!mbar_wait(bar.v_empty + 8 * vs, vr.ph ^ 1u, abort_flag, 2)) { record_timeout(p, abort_flag); goto done; }
                        SVDC_TRACE_ADD(1, p1);
                        vr.step((uint32_t)p.v_slots);
                        const uint32_t vdst = v_base0 + vs * p.vslice_bytes;
                        mbar_arrive_expect_tx(bar.v_full + 8 * vs, p.vslice_bytes);
                        for (int kb = 0; kb < p.nkb; ++kb)
                            tma_load_3d(vdst + kb * (p.gc * kTileCols * p.kb_bytes), &tm_v, bar.v_full + 8 * vs,
                                        kb * p.kb_elems, cg * kTileCols, un.b);
                        if (g == g_ins && u_next < p.units && !request_a_chunks(decode_unit(p, u_next))) {
                            record_timeout(p, abort_flag);
                            goto done;
                        }
                        const int ce = min(cg + p.gc, un.c1);
                        for (int c = cg; c < ce; ++c) {
                            const uint32_t s = fr.idx;
                            SVDC_TRACE_MARK(p2);
                            if (!mbar_wait(bar.empty + 8 * s, fr.ph ^ 1u, abort_flag, 3)) { record_timeout(p, abort_flag); goto done; }
                            SVDC_TRACE_ADD(2, p2);
                            fr.step((uint32_t)p.stages);
                            mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes);
                            tma_load_3d(stage0 + s * kTileBytes, &tm_r, bar.full + 8 * s, c * kTileCols, un.rt * kTileRows, un.b);
                        }
                    }
                    u = u_next;
                }
            }
        } else
        if (lane == 0) {
            RingPos fr, vr;                            // next R slot, next basis slot
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit un = decode_unit(p, u);
                if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) {
                    if (un.rt == 0 && un.c0 == 0) header_of(p, un.b)->status = SVDCACHE_ERR_STATE;
                    continue;
                }
                for (int cg = un.c0; cg < un.c1; cg += p.gc) {
                    const uint32_t vs = vr.idx;
                    SVDC_TRACE_MARK(p1);
                    if (!mbar_wait(bar.v_empty + 8 * vs, vr.ph ^ 1u, abort_flag, 2)) { record_timeout(p, abort_flag); goto done; }
                    vr.step((uint32_t)p.v_slots);
                    SVDC_TRACE_ADD(1, p1);
                    const uint32_t vdst = v_base0 + vs * p.vslice_bytes;
                    mbar_arrive_expect_tx(bar.v_full + 8 * vs, p.vslice_bytes);
                    for (int kb = 0; kb < p.nkb; ++kb)
                        tma_load_3d(vdst + kb * (p.gc * kTileCols * p.kb_bytes), &tm_v, bar.v_full + 8 * vs,
                                    kb * p.kb_elems, cg * kTileCols, un.b);
                    const int ce = min(cg + p.gc, un.c1);
                    for (int c = cg; c < ce; ++c) {
                        const uint32_t s = fr.idx;
                        SVDC_TRACE_MARK(p2);
                        if (!mbar_wait(bar.empty + 8 * s, fr.ph ^ 1u, abort_flag, 3)) { record_timeout(p, abort_flag); goto done; }
                        fr.step((uint32_t)p.stages);
                        SVDC_TRACE_ADD(2, p2);
                        mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes);
                        tma_load_3d(stage0 + s * kTileBytes, &tm_r, bar.full + 8 * s, c * kTileCols, un.rt * kTileRows, un.b);
                    }
                }
            }
        } else if (lane == 1) {
            uint32_t ua = 0;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit ux = decode_unit(p, u);
                if (*(volatile uint32_t *)&header_of(p, ux.b)->full_steps == 0) continue;
                if (!request_a(ux, ua)) { record_timeout(p, abort_flag); goto done; }
                ++ua;
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer ---
        if (lane == 0) {
            uint32_t ui = 0;
            RingPos vr, ar;   // basis slot, accumulator stage of the next group
            const int ksteps = p.kb_elems / 16;
            for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
                const Unit un = decode_unit(p, u);
                if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) continue;
                const uint32_t ab = ui % p.a_bufs;
                SVDC_TRACE_MARK(m0);
                if (!mbar_wait(bar.a_full + 8 * ab, (ui / p.a_bufs) & 1u, abort_flag, 4)) { record_timeout(p, abort_flag); goto done; }
                SVDC_TRACE_ADD(0, m0);
                if constexpr (kTmemA) tc_fence_after();   // the operand was written by tcgen05.st of other threads
                const uint64_t a_desc0 = smem_desc_kmajor(a_base0 + ab * p.a_bytes, p.kb_bytes);
                for (int cg = un.c0; cg < un.c1; cg += p.gc) {
                    const uint32_t vs = vr.idx, as = ar.idx;
                    const int nsub = min(p.gc, un.c1 - cg);
                    SVDC_TRACE_MARK(m1);
                    if (!mbar_wait(bar.v_full + 8 * vs, vr.ph, abort_flag, 5)) { record_timeout(p, abort_flag); goto done; }
                    SVDC_TRACE_ADD(1, m1);
                    SVDC_TRACE_MARK(m2);
                    if (!mbar_wait(bar.acc_empty + 8 * as, ar.ph ^ 1u, abort_flag, 6)) { record_timeout(p, abort_flag); goto done; }
                    vr.step((uint32_t)p.v_slots);
                    ar.step((uint32_t)p.acc_stages);
                    SVDC_TRACE_ADD(2, m2);
                    tc_fence_after();
                    SVDC_TRACE_MARK(m3);
                    const uint32_t idesc = idesc_bf16(kTileRows, nsub * kTileCols);
                    const uint32_t d_tmem = tmem_base + (uint32_t)p.acc_base + as * p.acc_stride;
                    const uint64_t v_desc0 = smem_desc_kmajor(v_base0 + vs * p.vslice_bytes, p.kb_bytes);
                    if constexpr (kTmemA) {
                        // operand buffer ab: k/2 columns of hi words, then k/2 of lo words (two bf16 per
                        // 32-bit column); one K step of 16 is 8 columns
                        const uint32_t a_t = tmem_base + ab * (uint32_t)p.k;
                        uint32_t acc = 0;
                        for (int part = 0; part < 2; ++part)
                            for (int kb = 0; kb < p.nkb; ++kb) {
                                const uint64_t v_kb = v_desc0 + ((kb * (p.gc * kTileCols * p.kb_bytes)) >> 4);
                                for (int ks = 0; ks < ksteps; ++ks) {
                                    mma_bf16_ts(d_tmem, a_t + (uint32_t)(part * (p.k >> 1) + kb * 32 + ks * 8), v_kb + 2 * ks, idesc, acc);
                                    acc = 1;
                                }
                            }
                    } else {
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
                    }
                    mma_commit(bar.v_empty + 8 * vs);
                    mma_commit(bar.acc_full + 8 * as);
                    SVDC_TRACE_ADD(3, m3);
                }
                mma_commit(bar.a_empty + 8 * ab);
                ++ui;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue ---
        const int q = warp & 3, row = q * kSlabRows + lane;
        const uint32_t grp = (uint32_t)(warp - 2) >> 2;
        uint32_t it = 0, ua = 0;   // chunks taken from the ring, live units begun
        RingPos fr, ar;   // R slot of chunk `it`, accumulator stage of the next group
        // kTmemA: the operand chunks of live unit number `n` leave the ring for TMEM buffer n % a_bufs.
        // Every warp waits for the buffer's release (the MMAs of its last user have completed), each
        // in its turn, so no phase of that barrier goes unseen; a chunk is taken by the group its
        // running index selects, like an R chunk, and each of the four warps moves the 32 rows of its
        // TMEM lane quarter: 128 bytes of a row are 32 columns.
        auto copy_operand = [&](uint32_t n) {
            const uint32_t ab = n % (uint32_t)p.a_bufs;
            SVDC_TRACE_MARK(e4);
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.a_empty + 8 * ab, ((n / (uint32_t)p.a_bufs) & 1u) ^ 1u, abort_flag, 11)))
                return false;
            SVDC_TRACE_ADD(4, e4);
            tc_fence_after();
            for (int i = 0; i < n_a_chunks; ++i, ++it, fr.step((uint32_t)p.stages)) {
                if ((it & 1u) != grp) continue;
                const uint32_t s = fr.idx;
                SVDC_TRACE_MARK(e5);
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.full + 8 * s, fr.ph, abort_flag, 12))) return false;
                SVDC_TRACE_ADD(5, e5);
                const uint32_t tile = stage0 + s * kTileBytes + (uint32_t)row * 128u;
                uint32_t w[32];
#pragma unroll
                for (int cc = 0; cc < 8; ++cc) {
                    const uint4 t = lds128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u);
                    w[4 * cc] = t.x; w[4 * cc + 1] = t.y; w[4 * cc + 2] = t.z; w[4 * cc + 3] = t.w;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.empty + 8 * s);
                tmem_st_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * (uint32_t)p.k +
                                  (uint32_t)((i & 1) * (p.k >> 1) + (i >> 1) * 32), w);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.a_full + 8 * ab);
            }
            return true;
        };
        if constexpr (kTmemA) {
            if (next_live((int)blockIdx.x) < p.units && !copy_operand(0)) { record_timeout(p, abort_flag); goto done; }
        }
        for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
            const Unit un = decode_unit(p, u);
            if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) continue;
            const int slab_row0 = un.rt * kTileRows + q * kSlabRows;
            const bool slab_live = (int64_t)slab_row0 < p.N;
            const bool more = kTmemA && next_live(u + (int)gridDim.x) < p.units;
            const int g_ins = insert_group(un);
            ++ua;
            for (int cg = un.c0, g = 0; cg < un.c1; cg += p.gc, ++g) {
                if constexpr (kTmemA) {
                    if (g == g_ins && more && !copy_operand(ua)) { record_timeout(p, abort_flag); goto done; }
                }
                const uint32_t as = ar.idx, aph = ar.ph;
                ar.step((uint32_t)p.acc_stages);
                const int nsub = min(p.gc, un.c1 - cg);
                const int last_own = last_own_chunk(it, nsub, grp);
                SVDC_TRACE_MARK(e0);
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.acc_full + 8 * as, aph, abort_flag, 7))) { record_timeout(p, abort_flag); goto done; }
                SVDC_TRACE_ADD(0, e0);
                if (last_own < 0 && lane == 0) mbar_arrive(bar.acc_empty + 8 * as);
                for (int j = 0; j < nsub; ++j, ++it, fr.step((uint32_t)p.stages)) {
                    if ((it & 1u) != grp) continue;
                    const int c = cg + j;
                    const uint32_t s = fr.idx, ph = fr.ph;
                    SVDC_TRACE_MARK(e1);
                    if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.full + 8 * s, ph, abort_flag, 8))) { record_timeout(p, abort_flag); goto done; }
                    SVDC_TRACE_ADD(1, e1);
                    SVDC_TRACE_MARK(e2);
                    tc_fence_after();
                    const uint32_t tile = stage0 + s * kTileBytes + (uint32_t)row * 128u;
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)p.acc_base + as * p.acc_stride + j * kTileCols;
                    uint32_t acc0[32], acc1[32];
                    tmem_ld_32x32(taddr, acc0);
                    tmem_ld_32x32(taddr + 32, acc1);
                    uint4 t[8];
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) t[cc] = lds128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0 && j == last_own) mbar_arrive(bar.acc_empty + 8 * as);   // this warp is done with the group
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
                    SVDC_TRACE_ADD(2, e2);
                    SVDC_TRACE_COUNT(3);
                }
            }
        }
        if (lane == 0) tma_store_wait<0>();
    }

done:
    SVDC_TRACE_FLUSH(g_trace);
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
// A unit is one 128-row tile of one block.
//   Pass 1 streams the tile's F in 64-column chunks and accumulates C (128 x k, fp32) in
//     TMEM: A = F chunk, B = matching columns of V_k^T.
//   The C job reads C from TMEM, applies the EMA against the previous Chat, writes Chat, its
//     split-bf16 copy for the cached step and C_out, and leaves C itself as a split-bf16 A
//     operand: from k = 64 on in tensor memory, over the columns of C (kTmemA: both epilogue
//     groups share the job, the previous Chat comes through registers, and all of shared memory
//     goes to the rings); below that in a shared-memory region that also stages the previous
//     Chat by TMA (warps 6..9 alone).
//   Pass 2 streams the same F chunks again, last group first (the most recently read ones
//     are the likeliest to sit in L2), with V_k slices of gc*64 rows: C V_k^T per group in
//     TMEM, and the epilogue stores R = F - C V_k^T through TMA.
// TMEM holds C in columns [0, k) and the pass-2 accumulator ring after it, so pass 1 of the
// next unit runs while the epilogue still drains this one.  The producer requests each basis
// slice one group ahead of the F chunks that go with it.
//
// Warp roles (352 threads): 0 = TMA producer of the F chunks, 10 = TMA producer of the basis
// slices, 1 = MMA issuer (+ TMEM owner), 2..5 and 6..9 = the two epilogue groups of pass 2,
// which first do the C job (pass 2 cannot start before the operand is written, so the two
// jobs never overlap).
// ======================================================================================
constexpr int kThreadsFull = 352;
constexpr int kFullVWarp = 10;   // second TMA producer (basis slices); warps 2..9 are the epilogue
constexpr uint32_t kBlk32Bytes = kTileRows * 128u;   // 16 KB: 128 rows x 32 fp32 (or x 64 bf16)

__device__ __forceinline__ void load_row32(uint32_t row_addr, uint32_t row, uint32_t row_bytes, int ncols, float (&v)[32]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i * 4 < ncols) {
            const uint4 t = lds128(row_addr + swizzled_chunk(row, (uint32_t)i, row_bytes) * 16u);
            v[4 * i] = __uint_as_float(t.x); v[4 * i + 1] = __uint_as_float(t.y);
            v[4 * i + 2] = __uint_as_float(t.z); v[4 * i + 3] = __uint_as_float(t.w);
        }
    }
}

// hi/lo bf16 of 8 consecutive values -> one 16-byte chunk each
__device__ __forceinline__ void pack_split8(const float *v, uint4 &hi, uint4 &lo) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        const float2 hf = __bfloat1622float2(hh);
        const __nv_bfloat162 ll = __floats2bfloat162_rn(v[2 * i] - hf.x, v[2 * i + 1] - hf.y);
        h[i] = *reinterpret_cast<const uint32_t *>(&hh);
        l[i] = *reinterpret_cast<const uint32_t *>(&ll);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// 32-byte stores: a thread of the C job owns a whole row, so every store instruction touches 32
// different lines -- the fewer and wider they are, the less time the job spends in the
// load-store unit
__device__ __forceinline__ void stg256(float *dst, const float *v) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "f"(v[0]), "f"(v[1]), "f"(v[2]),
                 "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}
__device__ __forceinline__ void stg256(void *dst, uint4 a, uint4 b) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(a.x), "r"(a.y), "r"(a.z),
                 "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
}

template <bool kTmemA, bool kResEma>
__global__ void __launch_bounds__(kThreadsFull, 1)
umma_full_kernel(const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_vt,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_rout,
                 const __grid_constant__ CUtensorMap tm_chat, const __grid_constant__ CUtensorMap tm_rold,
                 const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_base = base;                                     // A operand (and, for k >= 64, staged Chat)
    const uint32_t chat_base = a_base + p.chat_stage_off;             // == a_base when k >= 64
    const uint32_t v_base0 = a_base + p.a_region_bytes;
    const uint32_t stage0 = v_base0 + (uint32_t)p.v_slots * p.vslice_bytes;
    // residual EMA (kResEma): the stored R streams through r_slots slots after the F ring, whose
    // barriers are entries stages .. stages + r_slots - 1 of the ring's barrier arrays
    const uint32_t rold0 = stage0 + (uint32_t)p.stages * kTileBytes;
    const int r_slots = kResEma ? p.r_slots : 0;
    const Bars bar = bars_at(rold0 + (uint32_t)r_slots * kTileBytes);
    // barriers beyond the ring ones: c_full (C accumulated), a_full (A operand written),
    // p2_done (pass-2 MMAs of the unit finished: the A region may be restaged), chat_full
    // (previous Chat staged)
    const uint32_t chat_full = bar.a_full + 8, p2_done = bar.c_done;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen_base + (bar.abort_flag - base));
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen_base + (bar.tmem_slot - base));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    SVDC_TRACE_DECL
    const uint32_t tmem_cols = 512;
    const int CT = p.chunks_total;
    const int cid = (int)blockIdx.x, nctas = (int)gridDim.x;
    const int G = (CT + p.gc - 1) / p.gc;               // column groups per pass
    const uint32_t a_part = p.k >= 64 ? kBlk32Bytes : p.a_half_bytes;   // hi -> lo distance
    // From k = 64 on the A operand of pass 2 lives in tensor memory, over C itself, and both
    // epilogue groups share the C job; below that it is staged in shared memory.
    // (Each variant is an instantiation of its own: compiled together, the two C jobs spill.)
    constexpr bool c_split = kTmemA;
    const uint32_t a_kb = 2u * kBlk32Bytes;                             // K-block distance (k >= 64)

    if (threadIdx.x == 0) {
        // F slot: free again after five arrivals -- pass 1: the MMAs' commit plus four from the
        // MMA thread; pass 2: the four slab stores plus the MMA thread's "seen" (see there)
        for (int s = 0; s < p.stages; ++s) { mbar_init(bar.full + 8 * s, 1); mbar_init(bar.empty + 8 * s, 5); }
        // old-R slot: free again once the four warps of the chunk's epilogue group have read it
        for (int s = p.stages; s < p.stages + r_slots; ++s) { mbar_init(bar.full + 8 * s, 1); mbar_init(bar.empty + 8 * s, 4); }
        for (int s = 0; s < p.acc_stages; ++s) { mbar_init(bar.acc_full + 8 * s, 1); mbar_init(bar.acc_empty + 8 * s, 8); }
        for (int s = 0; s < p.v_slots; ++s) { mbar_init(bar.v_full + 8 * s, 1); mbar_init(bar.v_empty + 8 * s, 1); }
        mbar_init(bar.a_full, c_split ? 256 : 128);
        mbar_init(chat_full, 1);
        mbar_init(bar.c_full, 1);
        mbar_init(p2_done, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_f);
        prefetch_tensormap(&tm_vt);
        prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_rout);
        prefetch_tensormap(&tm_chat);
        if constexpr (kResEma) prefetch_tensormap(&tm_rold);
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
        // ---------------------------------------------------- TMA producer: F chunks ---
        // Two request streams feed the tensor cores: F chunks (ring of p.stages slots) and basis
        // slices (ring of p.v_slots slots), both in (unit, pass, group) order.  Neither may hold
        // the other up -- a blocked F ring must not delay the next basis slice, and the other way
        // round -- so each stream has a thread of its own (this one, and warp 10), each a plain
        // loop of wait / expect / copy: a single thread polling both rings spent ~1200 cycles per
        // chunk on its own serial instruction chain and was the bottleneck of the kernel.
        if (lane == 0) {
            const uint64_t pol_keep = policy_evict_last(), pol_drop = policy_evict_first();
            uint32_t it = 0, s = 0, ph = 0;   // F chunks requested so far; ring slot and phase of the next one
            for (int u = cid; u < p.units; u += nctas) {
                const Unit un = decode_unit(p, u);
                for (int pass = 0; pass < 2; ++pass)
                    for (int g = 0; g < G; ++g) {
                        const int cg = (pass == 0 ? g : G - 1 - g) * p.gc;
                        const int nsub = min(p.gc, CT - cg);
                        for (int j = 0; j < nsub; ++j, ++it) {
                            if (!mbar_wait(bar.empty + 8 * s, ph ^ 1u, abort_flag, 100)) {
                                record_timeout(p, abort_flag, it, (uint32_t)(pass * 100 + g));
                                goto done;
                            }
                            mbar_arrive_expect_tx(bar.full + 8 * s, kTileBytes);
                            tma_load_3d_hint(stage0 + s * kTileBytes, &tm_f, bar.full + 8 * s, (cg + j) * kTileCols,
                                             un.rt * kTileRows, un.b, pass == 0 ? pol_keep : pol_drop);
                            if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
                        }
                    }
            }
        }
        if constexpr (kResEma) {
            // Third request stream (residual EMA of the ablation, Sec. 4.5): the chunks of the stored R,
            // in the order pass 2 meets them.  A block's first full step blends nothing and asks for none.
            if (lane == 1) {
                RingPos rr;
                uint32_t ir = 0;
                for (int u = cid; u < p.units; u += nctas) {
                    const Unit un = decode_unit(p, u);
                    if (*(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0) continue;
                    for (int g = 0; g < G; ++g) {
                        const int cg = (G - 1 - g) * p.gc;
                        const int nsub = min(p.gc, CT - cg);
                        for (int j = 0; j < nsub; ++j, ++ir) {
                            const uint32_t sl = (uint32_t)p.stages + rr.idx;
                            if (!mbar_wait(bar.empty + 8 * sl, rr.ph ^ 1u, abort_flag, 102)) {
                                record_timeout(p, abort_flag, ir, (uint32_t)g);
                                goto done;
                            }
                            mbar_arrive_expect_tx(bar.full + 8 * sl, kTileBytes);
                            tma_load_3d(rold0 + rr.idx * kTileBytes, &tm_rold, bar.full + 8 * sl, (cg + j) * kTileCols,
                                        un.rt * kTileRows, un.b);
                            rr.step((uint32_t)r_slots);
                        }
                    }
                }
            }
        }
    } else if (warp == kFullVWarp) {
        // ------------------------------------------------ TMA producer: basis slices ---
        if (lane == 0) {
            uint32_t iv = 0, vs = 0, vph = 0;
            for (int u = cid; u < p.units; u += nctas) {
                const Unit un = decode_unit(p, u);
                for (int pass = 0; pass < 2; ++pass)
                    for (int g = 0; g < G; ++g, ++iv) {
                        const int cg = (pass == 0 ? g : G - 1 - g) * p.gc;
                        if (!mbar_wait(bar.v_empty + 8 * vs, vph ^ 1u, abort_flag, 101)) {
                            record_timeout(p, abort_flag, iv, (uint32_t)(pass * 100 + g));
                            goto done;
                        }
                        const uint32_t vdst = v_base0 + vs * p.vslice_bytes;
                        mbar_arrive_expect_tx(bar.v_full + 8 * vs, p.vslice_bytes);
                        if (pass == 0) {   // V_k^T columns of each chunk: gc boxes of k rows x 64
                            for (int j = 0; j < p.gc; ++j)
                                tma_load_3d(vdst + j * (p.k * 128), &tm_vt, bar.v_full + 8 * vs, (cg + j) * kTileCols, 0, un.b);
                        } else {           // V_k rows of the group: one box of gc*64 rows per K block
                            for (int kb = 0; kb < p.nkb; ++kb)
                                tma_load_3d(vdst + kb * (p.gc * kTileCols * p.kb_bytes), &tm_v, bar.v_full + 8 * vs,
                                            kb * p.kb_elems, cg * kTileCols, un.b);
                        }
                        if (++vs == (uint32_t)p.v_slots) { vs = 0; vph ^= 1u; }
                    }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer ---
        if (lane == 0) {
            uint32_t it = 0, iv = 0, ig = 0, ui = 0;   // F chunks, basis slices, pass-2 groups, units
            RingPos fr, vr, ar;                        // ring positions of chunk `it`, slice `iv`, group `ig`
            const uint32_t idesc1 = idesc_bf16(kTileRows, p.k);
            const int ksteps = p.kb_elems / 16;
            const uint64_t a_desc0 = smem_desc_kmajor(a_base, p.kb_bytes);
            for (int u = cid; u < p.units; u += nctas, ++ui) {
                // C of the previous unit has been read out of TMEM: a_full(ui - 1) was awaited below
                for (int g = 0; g < G; ++g, ++iv) {                 // pass 1: C_a += F_chunk (V^T chunk)^T
                    const int cg = g * p.gc, ce = min(cg + p.gc, CT);
                    const uint32_t vs = vr.idx;
                    SVDC_TRACE_MARK(t0);
                    if (!mbar_wait(bar.v_full + 8 * vs, vr.ph, abort_flag, 9)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                    SVDC_TRACE_ADD(0, t0);
                    vr.step((uint32_t)p.v_slots);
                    for (int c = cg; c < ce; ++c, ++it, fr.step((uint32_t)p.stages)) {
                        const uint32_t s = fr.idx, ph = fr.ph;
                        SVDC_TRACE_MARK(t1);
                        if (!mbar_wait(bar.full + 8 * s, ph, abort_flag, 10)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                        SVDC_TRACE_ADD(1, t1);
                        tc_fence_after();
                        SVDC_TRACE_MARK(t2);
                        const uint64_t fd = smem_desc_kmajor(stage0 + s * kTileBytes, 128);
                        const uint64_t vd = smem_desc_kmajor(v_base0 + vs * p.vslice_bytes + (c - cg) * (p.k * 128), 128);
#pragma unroll
                        for (int ks = 0; ks < kTileCols / 16; ++ks)
                            mma_bf16_ss(tmem_base, fd + 2 * ks, vd + 2 * ks, idesc1, (c != 0 || ks != 0) ? 1u : 0u);
                        mma_commit(bar.empty + 8 * s);
                        mbar_arrive_n(bar.empty + 8 * s, 4);   // pass 1 has no slab stores: the other four arrivals
                        SVDC_TRACE_ADD(2, t2);
                    }
                    mma_commit(bar.v_empty + 8 * vs);
                }
                mma_commit(bar.c_full);
                SVDC_TRACE_MARK(t3);
                if (!mbar_wait(bar.a_full, ui & 1u, abort_flag, 11)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                SVDC_TRACE_ADD(3, t3);
                tc_fence_after();
                for (int g = 0; g < G; ++g, ++iv, ++ig) {           // pass 2: acc = C (V slice)^T
                    const int cg = (G - 1 - g) * p.gc;
                    const int nsub = min(p.gc, CT - cg);
                    const uint32_t vs = vr.idx, as = ar.idx;
                    SVDC_TRACE_MARK(t4);
                    if (!mbar_wait(bar.v_full + 8 * vs, vr.ph, abort_flag, 12)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                    SVDC_TRACE_ADD(4, t4);
                    SVDC_TRACE_MARK(t5);
                    if (!mbar_wait(bar.acc_empty + 8 * as, ar.ph ^ 1u, abort_flag, 13)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                    SVDC_TRACE_ADD(5, t5);
                    vr.step((uint32_t)p.v_slots);
                    ar.step((uint32_t)p.acc_stages);
                    tc_fence_after();
                    SVDC_TRACE_MARK(t6);
                    const uint32_t idesc = idesc_bf16(kTileRows, nsub * kTileCols);
                    const uint32_t d_tmem = tmem_base + p.k + as * p.acc_cols;
                    const uint64_t v_desc0 = smem_desc_kmajor(v_base0 + vs * p.vslice_bytes, p.kb_bytes);
                    uint32_t acc = 0;
                    for (int part = 0; part < 2; ++part)
                        for (int kb = 0; kb < p.nkb; ++kb) {
                            const uint64_t ad = a_desc0 + ((part * a_part + kb * a_kb) >> 4);
                            const uint64_t vd = v_desc0 + ((kb * (p.gc * kTileCols * p.kb_bytes)) >> 4);
                            for (int ks = 0; ks < ksteps; ++ks) {
                                if constexpr (c_split)   // operand in TMEM: 64-column block kb, half ks / 2, hi or lo words, K step
                                    mma_bf16_ts(d_tmem, tmem_base + (uint32_t)(kb * 64 + (ks >> 1) * 32 + part * 16 + (ks & 1) * 8),
                                                vd + 2 * ks, idesc, acc);
                                else
                                    mma_bf16_ss(d_tmem, ad + 2 * ks, vd + 2 * ks, idesc, acc);
                                acc = 1;
                            }
                        }
                    mma_commit(bar.v_empty + 8 * vs);
                    mma_commit(bar.acc_full + 8 * as);
                    SVDC_TRACE_ADD(6, t6);
                    // The MMAs of pass 2 do not read F, but this thread still has to see every phase of
                    // a ring slot's barrier (or its wait for the slot's next pass-1 chunk could be
                    // satisfied by the phase before a skipped one), and the slot must not be reused
                    // before it has: it waits for the group's chunks here, after the MMAs are on their
                    // way, and its arrival is one of the five that free the slot.
                    for (int j = 0; j < nsub; ++j, ++it, fr.step((uint32_t)p.stages)) {
                        if (!mbar_wait(bar.full + 8 * fr.idx, fr.ph, abort_flag, 19)) { record_timeout(p, abort_flag, it, iv, ig); goto done; }
                        mbar_arrive(bar.empty + 8 * fr.idx);
                    }
                }
                mma_commit(p2_done);
            }
        }
    } else {
        // --------------- epilogue (R = F - C V_k^T, TMA store) and, for warps 6..9, the C job ---
        const int q = warp & 3, row = q * kSlabRows + lane;
        const uint32_t grp = (uint32_t)(warp - 2) >> 2;
        const bool c_warp = grp == 1;
        const bool issuer = (warp == 6 && lane == 0);
        const float beta = p.beta, omb = 1.0f - p.beta;
        const uint32_t chat_row_bytes = p.k >= 32 ? 128u : (uint32_t)p.k * 4u;
        const int nblk = (p.k + 31) / 32;
        uint32_t it = 0, ig = 0, ui = 0, nchat = 0;   // F chunks, pass-2 groups, units, Chat tiles consumed
        RingPos fr, ar, ro;                           // ring positions of chunk `it`, group `ig`, old-R chunk
        int prev_slot = -1;                           // slot whose slab store may still be reading
        const bool defer_release = p.stages >= 4;
        // R is not read again by this step: its lines are the first to go, which leaves more of L2 to
        // the F tiles waiting for their second pass
        const uint64_t pol_store = policy_evict_first();

        auto request_chat = [&](const Unit &x) {   // previous Chat of unit x -> staging, by TMA
            mbar_arrive_expect_tx(chat_full, (uint32_t)kTileRows * p.k * 4u);
            for (int b = 0; b < nblk; ++b)
                tma_load_3d(chat_base + b * kBlk32Bytes, &tm_chat, chat_full, b * 32, x.rt * kTileRows, x.b);
        };
        if (issuer && cid < p.units && !c_split) {
            const Unit x = decode_unit(p, cid);
            if (*(volatile uint32_t *)&header_of(p, x.b)->full_steps != 0) request_chat(x);
        }
        for (int u = cid; u < p.units; u += nctas, ++ui) {
            const Unit un = decode_unit(p, u);
            if constexpr (c_split) {
                // ---- C job, operand in tensor memory (k >= 64): both epilogue groups take part.  Of
                // every 64-column block of C, a thread of warps 6..9 owns the lower 32 columns of its
                // row and a thread of warps 2..5 the upper 32: it reads them from TMEM, applies the EMA
                // against the previous Chat (prefetched into registers while pass 1 ran), and writes the
                // split-bf16 pair back over the very columns it has read -- 16 columns of hi words,
                // then 16 of lo words (two bf16 per 32-bit column) -- which is where the MMAs of pass 2
                // take their A operand from.  No staging, no shared memory, nobody else's columns.
                StateHeader *hdr = header_of(p, un.b);
                const bool first = *(volatile uint32_t *)&hdr->full_steps == 0;
                const int h = c_warp ? 0 : 1;
                const int64_t n = (int64_t)un.rt * kTileRows + row;
                const bool row_live = n < p.N;
                char *st_b = p.state + (size_t)un.b * p.state_stride;
                float *chat_g = reinterpret_cast<float *>(st_b + p.chat_off) + n * p.k + h * 32;
                float *cout_g = p.C_out ? reinterpret_cast<float *>((char *)p.C_out + (size_t)un.b * p.C_stride) + n * p.k + h * 32
                                        : nullptr;
                __nv_bfloat16 *ohi = reinterpret_cast<__nv_bfloat16 *>(st_b + p.ophi_off) + n * p.k + h * 32;
                __nv_bfloat16 *olo = reinterpret_cast<__nv_bfloat16 *>(st_b + p.oplo_off) + n * p.k + h * 32;
                auto load_prev = [&](int kb, float (&pv)[32]) {
                    if (!first && row_live) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 t = *reinterpret_cast<const float4 *>(chat_g + kb * 64 + 4 * i);
                            pv[4 * i] = t.x; pv[4 * i + 1] = t.y; pv[4 * i + 2] = t.z; pv[4 * i + 3] = t.w;
                        }
                    }
                };
                float prev0[32];   // previous Chat of the first K block: on its way while pass 1 runs
                load_prev(0, prev0);
                SVDC_TRACE_MARK(c1);
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.c_full, ui & 1u, abort_flag, 15))) { record_timeout(p, abort_flag, it, ig, ui); goto done; }
                SVDC_TRACE_ADD(1, c1);
                tc_fence_after();
                SVDC_TRACE_MARK(c2);
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 32);
                auto k_block = [&](int kb, float (&pv)[32]) {
                    uint32_t w[32];
                    tmem_ld_32x32(taddr + kb * 64, w);
                    tmem_wait_ld();
                    float cs[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) cs[i] = __uint_as_float(w[i]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {   // hi words of columns 8i..8i+7 -> w[4i..], lo words -> w[16+4i..]
                        uint4 hi, lo;
                        pack_split8(cs + 8 * i, hi, lo);
                        w[4 * i] = hi.x; w[4 * i + 1] = hi.y; w[4 * i + 2] = hi.z; w[4 * i + 3] = hi.w;
                        w[16 + 4 * i] = lo.x; w[16 + 4 * i + 1] = lo.y; w[16 + 4 * i + 2] = lo.z; w[16 + 4 * i + 3] = lo.w;
                    }
                    tmem_st_32x32(taddr + kb * 64, w);
                    if (kb == p.nkb - 1) {   // the operand is what pass 2 waits for: announce it before the stores below
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive(bar.a_full);
                        SVDC_TRACE_ADD(2, c2);
                    }
                    if (row_live) {
                        if (!first) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) pv[i] = fmaf(beta, pv[i], omb * cs[i]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) pv[i] = cs[i];
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            stg256(chat_g + kb * 64 + 8 * i, pv + 8 * i);
                            if (cout_g) stg256(cout_g + kb * 64 + 8 * i, cs + 8 * i);
                        }
#pragma unroll
                        for (int i = 0; i < 2; ++i) {   // the state keeps the split of the new Chat
                            uint4 hi0, lo0, hi1, lo1;
                            pack_split8(pv + 16 * i, hi0, lo0);
                            pack_split8(pv + 16 * i + 8, hi1, lo1);
                            stg256(ohi + kb * 64 + 16 * i, hi0, hi1);
                            stg256(olo + kb * 64 + 16 * i, lo0, lo1);
                        }
                    }
                };
                for (int kb = 0; kb < p.nkb; ++kb) {
                    // wider ranks: the previous Chat of the later blocks is fetched as it is needed -- the
                    // operand does not wait for it, only this thread's own stores do
                    if (kb > 0) load_prev(kb, prev0);
                    k_block(kb, prev0);
                }
            } else if (c_warp) {   // (discarded statement of the if constexpr above when the operand is in TMEM)
                // ---- C job: TMEM -> EMA -> Chat, split-bf16 A operand (+ the state's operand copy)
                StateHeader *hdr = header_of(p, un.b);
                const bool first = *(volatile uint32_t *)&hdr->full_steps == 0;
                bool ok = true;
                SVDC_TRACE_MARK(c0);
                if (!first) { ok = mbar_wait(chat_full, nchat & 1u, abort_flag, 14); ++nchat; }
                SVDC_TRACE_ADD(0, c0);
                SVDC_TRACE_MARK(c1);
                ok = ok && mbar_wait(bar.c_full, ui & 1u, abort_flag, 15);
                if (!__all_sync(0xFFFFFFFFu, ok)) { record_timeout(p, abort_flag, it, ig, ui); goto done; }
                SVDC_TRACE_ADD(1, c1);
                tc_fence_after();
                SVDC_TRACE_MARK(c2);
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
                const int64_t n = (int64_t)un.rt * kTileRows + row;
                const bool row_live = n < p.N;
                char *st_b = p.state + (size_t)un.b * p.state_stride;
                float *chat_g = reinterpret_cast<float *>(st_b + p.chat_off) + n * p.k;
                float *cout_g = p.C_out ? reinterpret_cast<float *>((char *)p.C_out + (size_t)un.b * p.C_stride) + n * p.k
                                        : nullptr;
                const int nkb64 = p.k >= 64 ? p.nkb : 1;
                for (int kb = 0; kb < nkb64; ++kb) {
                    // staged previous Chat of this row: the block holding columns kb*64 .. +31 (A) and
                    // the one holding +32 .. +63 (B).  For k >= 64 they are exactly where this row's
                    // hi and lo operand rows go, so B is read before anything is written.
                    const uint32_t stA = chat_base + (uint32_t)(2 * kb) * kBlk32Bytes + (uint32_t)row * chat_row_bytes;
                    const uint32_t stB = stA + kBlk32Bytes;
                    const uint32_t hi_row = a_base + (uint32_t)kb * a_kb + (uint32_t)row * p.kb_bytes;
                    const uint32_t lo_row = hi_row + a_part;
                    const int halves = p.k >= 64 ? 2 : 1;
                    float prevB[32];
                    if (!first && halves == 2) load_row32(stB, (uint32_t)row, chat_row_bytes, 32, prevB);
                    for (int h = 0; h < halves; ++h) {
                        const int col0 = kb * 64 + h * 32;
                        const int ncols = p.k - col0 < 32 ? p.k - col0 : 32;
                        float cs[32];
                        {
                            uint32_t tmp[32];
                            tmem_ld_32x32(taddr + col0, tmp);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) cs[i] = __uint_as_float(tmp[i]);
                        }
                        float ch[32];
                        if (first) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) ch[i] = cs[i];
                        } else {
                            if (h == 0) load_row32(stA, (uint32_t)row, chat_row_bytes, ncols, ch);
                            else {
#pragma unroll
                                for (int i = 0; i < 32; ++i) ch[i] = prevB[i];
                            }
#pragma unroll
                            for (int i = 0; i < 32; ++i) ch[i] = fmaf(beta, ch[i], omb * cs[i]);
                        }
                        // split-bf16 operand of C (not of Chat) for pass 2 ...
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (i * 8 < ncols) {
                                uint4 hi, lo;
                                pack_split8(cs + 8 * i, hi, lo);
                                const uint32_t chunk = swizzled_chunk((uint32_t)row, (uint32_t)(h * 4 + i), (uint32_t)p.kb_bytes) * 16u;
                                sts128(hi_row + chunk, hi);
                                sts128(lo_row + chunk, lo);
                            }
                        }
                        if (row_live) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (i * 4 < ncols) {
                                    *reinterpret_cast<float4 *>(chat_g + col0 + 4 * i) =
                                        make_float4(ch[4 * i], ch[4 * i + 1], ch[4 * i + 2], ch[4 * i + 3]);
                                    if (cout_g)
                                        *reinterpret_cast<float4 *>(cout_g + col0 + 4 * i) =
                                            make_float4(cs[4 * i], cs[4 * i + 1], cs[4 * i + 2], cs[4 * i + 3]);
                                }
                            }
                            // ... while the state keeps the split of the new Chat
                            __nv_bfloat16 *ohi = reinterpret_cast<__nv_bfloat16 *>(st_b + p.ophi_off) + n * p.k + col0;
                            __nv_bfloat16 *olo = reinterpret_cast<__nv_bfloat16 *>(st_b + p.oplo_off) + n * p.k + col0;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (i * 8 < ncols) {
                                    uint4 hi, lo;
                                    pack_split8(ch + 8 * i, hi, lo);
                                    *reinterpret_cast<uint4 *>(ohi + 8 * i) = hi;
                                    *reinterpret_cast<uint4 *>(olo + 8 * i) = lo;
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                fence_proxy_async();
                mbar_arrive(bar.a_full);
                SVDC_TRACE_ADD(2, c2);
            }
            // ---- epilogue duty for this group's chunks of pass 2
            const bool first_unit = kResEma && *(volatile uint32_t *)&header_of(p, un.b)->full_steps == 0;
            const bool blend = kResEma && !first_unit;   // every pass-2 chunk of this unit has an old-R chunk in the ring
            const int slab_row0 = un.rt * kTileRows + q * kSlabRows;
            const bool slab_live = (int64_t)slab_row0 < p.N;
            it += CT;   // pass-1 slots are consumed by the MMA warp alone
            fr.skip((uint32_t)CT, (uint32_t)p.stages);
            for (int g = 0; g < G; ++g, ++ig) {
                const int cg = (G - 1 - g) * p.gc;
                const int nsub = min(p.gc, CT - cg);
                const uint32_t as = ar.idx, aph = ar.ph;
                ar.step((uint32_t)p.acc_stages);
                const int last_own = last_own_chunk(it, nsub, grp);
                SVDC_TRACE_MARK(e3);
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.acc_full + 8 * as, aph, abort_flag, 16))) { record_timeout(p, abort_flag, it, ig, ui); goto done; }
                SVDC_TRACE_ADD(3, e3);
                if (last_own < 0 && lane == 0) mbar_arrive(bar.acc_empty + 8 * as);
                for (int j = 0; j < nsub; ++j, ++it, fr.step((uint32_t)p.stages), (blend ? ro.step((uint32_t)r_slots) : (void)0)) {
                    if ((it & 1u) != grp) continue;
                    const int c = cg + j;
                    const uint32_t s = fr.idx, ph = fr.ph;
                    // residual EMA (ablation): this row's 64 columns of the stored R, from the old-R ring (rows
                    // past N and columns past D arrive as zeros and are never stored)
                    uint4 r_old[kResEma ? 8 : 1];
                    if constexpr (kResEma) {
                        if (blend) {
                            const uint32_t sl = (uint32_t)p.stages + ro.idx;
                            if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.full + 8 * sl, ro.ph, abort_flag, 20))) { record_timeout(p, abort_flag, it, ig, ui); goto done; }
                            const uint32_t otile = rold0 + ro.idx * kTileBytes + (uint32_t)row * 128u;
#pragma unroll
                            for (int cc = 0; cc < 8; ++cc) r_old[cc] = lds128(otile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u);
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar.empty + 8 * sl);
                        }
                    }
                    SVDC_TRACE_MARK(e4);
                    if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar.full + 8 * s, ph, abort_flag, 17))) { record_timeout(p, abort_flag, it, ig, ui); goto done; }
                    SVDC_TRACE_ADD(4, e4);
                    tc_fence_after();
                    SVDC_TRACE_MARK(e5);
                    const uint32_t tile = stage0 + s * kTileBytes + (uint32_t)row * 128u;
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + p.k + as * p.acc_cols + j * kTileCols;
                    uint32_t acc0[32], acc1[32];
                    tmem_ld_32x32(taddr, acc0);
                    tmem_ld_32x32(taddr + 32, acc1);
                    uint4 t[8];
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) t[cc] = lds128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0 && j == last_own) mbar_arrive(bar.acc_empty + 8 * as);   // this warp is done with the group
#pragma unroll
                    for (int cc = 0; cc < 8; ++cc) {
                        const uint32_t *ac = cc < 4 ? acc0 + cc * 8 : acc1 + (cc - 4) * 8;
                        uint4 o;
                        if constexpr (kResEma) o = blend ? combine_chunk_ema(t[cc], ac, r_old[cc], p.beta_r) : combine_chunk<true>(t[cc], ac);
                        else o = combine_chunk<true>(t[cc], ac);
                        sts128(tile + (((uint32_t)cc) ^ ((uint32_t)row & 7u)) * 16u, o);
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (slab_live)
                            tma_store_3d_hint(&tm_rout, stage0 + s * kTileBytes + (uint32_t)q * kSlabBytes, c * kTileCols,
                                              slab_row0, un.b, pol_store);
                        tma_store_commit();
                        // the slot goes back once its store has read it: checked one chunk late, so
                        // the warp does not sit out the store it has just issued
                        if (!defer_release) {   // a ring this short cannot lend a slot per warp
                            tma_store_wait_read<0>();
                            mbar_arrive(bar.empty + 8 * s);
                        } else {
                            if (prev_slot >= 0) {
                                tma_store_wait_read<1>();
                                mbar_arrive(bar.empty + 8 * prev_slot);
                            }
                            prev_slot = (int)s;
                        }
                    }
                    __syncwarp();
                    SVDC_TRACE_ADD(5, e5);
                    SVDC_TRACE_COUNT(6);
                }
            }
            if (lane == 0 && prev_slot >= 0) {   // last chunk of the unit: release at once
                tma_store_wait_read<0>();
                mbar_arrive(bar.empty + 8 * prev_slot);
                prev_slot = -1;
            }
            // Every accumulator of this unit has been read, so its pass-2 MMAs are complete and
            // the A region is free: stage the next unit's previous Chat there.
            if (issuer) {
                const int un_next = u + nctas;
                const bool ok = mbar_wait(p2_done, ui & 1u, abort_flag, 18);
                if (ok && un_next < p.units && !c_split) {
                    const Unit x = decode_unit(p, un_next);
                    if (*(volatile uint32_t *)&header_of(p, x.b)->full_steps != 0) request_chat(x);
                }
            }
            __syncwarp();
        }
        if (lane == 0) tma_store_wait<0>();
    }

done:
    SVDC_TRACE_FLUSH(g_trace);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0) report_exit_and_count_step(p);
}

// One CTA that waits, with the bounded wait of the step kernels, for an mbarrier phase nobody
// will ever complete: the wait must give up after `limit` cycles, the kernel must record the
// time-out in the state header exactly as the step kernels do, and return.
__global__ void __launch_bounds__(64, 1) wait_selftest_kernel(const UmmaParams p, long long limit) {
    __shared__ __align__(8) unsigned long long bar_mem;
    __shared__ int abort_mem;
    const uint32_t bar = smem_u32(&bar_mem);
    volatile int *abort_flag = &abort_mem;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_mem = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (!__all_sync(0xFFFFFFFFu, mbar_wait(bar, 0u, abort_flag, 99, limit)))
        record_timeout(p, abort_flag, (uint32_t)(threadIdx.x >> 5), 0u, 0u);
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

// bf16 (or fp32: elem = 4) tensor (inner, rows, blocks) with byte pitches; box (box_inner, box_rows, 1)
int make_map(CUtensorMap *m, const void *base, uint64_t inner, uint64_t rows, uint64_t blocks, uint64_t row_pitch,
             uint64_t block_pitch, uint32_t box_inner, uint32_t box_rows, uint32_t elem = 2) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SVDCACHE_ERR_CUDA;
    const cuuint64_t dims[3] = {inner, rows, blocks};
    if (blocks <= 1 || block_pitch == 0) block_pitch = row_pitch * rows;
    block_pitch = (block_pitch + 15) / 16 * 16;
    const cuuint64_t strides[2] = {row_pitch, block_pitch};
    const cuuint32_t box[3] = {box_inner, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const uint32_t inner_bytes = box_inner * elem;
    const CUtensorMapSwizzle sw = inner_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : inner_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                      : CU_TENSOR_MAP_SWIZZLE_32B;
    const CUresult r = fn(m, elem == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDCACHE_OK : SVDCACHE_ERR_CUDA;
}

// SMs of the current device (asked every time: a process may drive several devices)
int num_sms() {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize is kept per device: set on every call (cheap)
template <typename K> int allow_big_smem(K kern, size_t bytes) {
    return record_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
}

constexpr size_t kSmemBudget = 227 * 1024;

bool fill_params(const StepArgs &a, UmmaParams &p) {
    p.N = a.N; p.D = a.D; p.k = a.k; p.nblocks = a.nblocks;
    p.row_tiles = (int)((a.N + kTileRows - 1) / kTileRows);
    p.chunks_total = (a.D + kTileCols - 1) / kTileCols;
    p.kb_elems = a.k < 64 ? a.k : 64;            // K block of the rank dimension: one swizzled row
    p.kb_bytes = p.kb_elems * 2;
    p.nkb = a.k / p.kb_elems;
    p.a_half_bytes = (uint32_t)kTileRows * a.k * 2;
    p.a_bytes = 2 * p.a_half_bytes;
    p.state = (char *)a.state;
    p.state_stride = a.state_stride;
    {
        const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
        p.chat_off = SL.chat; p.ophi_off = SL.op_hi; p.oplo_off = SL.op_lo;
    }
    p.C_out = a.C_out;
    p.C_stride = a.C_stride;
    p.beta = a.beta;
    p.beta_r = a.beta_r;
    p.r_off = state_layout(a.N, a.D, a.k, a.dtype).r;
    return true;
}

void fill_groups(const StepArgs &a, UmmaParams &p) {
    p.gc = 16384 / (kTileCols * a.k);            // basis slice (gc * 64 x k bf16) of at most 32 KB
    if (p.gc > 4) p.gc = 4;                      // MMA N = gc * 64 <= 256
    if (p.gc < 1) p.gc = 1;
    p.acc_cols = p.gc * kTileCols;
    p.acc_stages = 512 / p.acc_cols < kAccStages ? 512 / p.acc_cols : kAccStages;
    p.vslice_bytes = (uint32_t)p.gc * kTileCols * a.k * 2;
    p.v_slots = 2;
}

// Full step: shared memory = A operand region (+ Chat staging when k < 64) | basis ring | F ring | barriers.
bool fill_full(const StepArgs &a, UmmaParams &p) {
    if (!fill_params(a, p)) return false;
    fill_groups(a, p);
    const bool a_tmem = a.k >= 64;
    // With the operand in TMEM the basis slices may outgrow the 32 KB of fill_groups: wider groups
    // mean fewer, wider MMAs in pass 2 (N = 192 costs ~144 cycles, two of N = 128 ~230) and fewer
    // hand-overs per unit -- as wide as TMEM and, below, shared memory allow (measured: k = 128
    // +4 %, k = 256 +44 % over slices of 32 KB).
    if (a_tmem) p.gc = 4;
    // TMEM: C in columns [0, k), then the pass-2 ring; at least two ring stages
    while (p.gc > 1 && a.k + 2 * p.gc * kTileCols > 512) --p.gc;
    // shared memory: two basis slices and at least six F slots
    while (a_tmem && p.gc > 1 && 2 * (size_t)p.gc * kTileCols * a.k * 2 + 6 * (size_t)kTileBytes > kSmemBudget - 2048 - kBarBytes) --p.gc;
    p.acc_cols = p.gc * kTileCols;
    p.acc_stages = (512 - a.k) / p.acc_cols < kAccStages ? (512 - a.k) / p.acc_cols : kAccStages;
    p.vslice_bytes = (uint32_t)p.gc * kTileCols * a.k * 2;
    // From k = 64 on the A operand lives in tensor memory (the kernel's c_split) and the previous
    // Chat comes through registers: no A region at all, and the shared memory goes to the rings --
    // a third basis slot first (a slice arrives 2000-3000 cycles after its request under load, a
    // group of MMAs lasts ~1000), a fourth if it costs no F slot.  Below k = 64 the operand and
    // the staged Chat share a region of shared memory.
    p.chat_stage_off = a_tmem ? 0u : p.a_bytes;
    p.a_region_bytes = a_tmem ? 0u : p.a_bytes + (uint32_t)kTileRows * a.k * 4u;
    p.a_region_bytes = (p.a_region_bytes + 1023u) & ~1023u;
    const size_t avail = kSmemBudget - 1024 /*alignment*/ - kBarBytes - 64;
    auto stages_for = [&](int v_slots) {
        const size_t fixed = (size_t)p.a_region_bytes + (size_t)v_slots * p.vslice_bytes;
        if (fixed + 2 * (size_t)kTileBytes > avail) return 0;
        int st = (int)((avail - fixed) / kTileBytes);
        if (st > kMaxStages) st = kMaxStages;
        return st & ~1;   // even: a slot then always serves the same epilogue group (chunk parity)
    };
    p.v_slots = 2;
    if (a_tmem && stages_for(3) >= 8) p.v_slots = 3;
    if (a_tmem && p.v_slots == 3 && stages_for(4) == stages_for(3)) p.v_slots = 4;
    p.stages = stages_for(p.v_slots);
    if (p.stages < 2) return false;
    p.a_bufs = 1;
    p.r_slots = 0;
    if (a.beta_r > 0.0f) {
        // residual EMA: the old R is a third stream, as many bytes as F -- it takes up to four slots,
        // from the F ring (down to six slots) and, before that, from the basis ring (down to two)
        auto room = [&]() { return (int)((avail - (size_t)p.a_region_bytes - (size_t)p.v_slots * p.vslice_bytes) / kTileBytes); };
        while (p.v_slots > 2 && room() < 6 + 4) --p.v_slots;
        const int slots = room() < kMaxStages ? room() : kMaxStages;
        p.r_slots = slots - 6 < 4 ? slots - 6 : 4;
        if (p.r_slots < 2) { p.r_slots = 2; }
        p.stages = (slots - p.r_slots) & ~1;
        if (p.stages < 2) return false;
    }
    return true;
}
size_t smem_bytes_full(const UmmaParams &p) {
    return 1024 + (size_t)p.a_region_bytes + (size_t)p.v_slots * p.vslice_bytes + (size_t)(p.stages + p.r_slots) * kTileBytes +
           kBarBytes + 64;
}

// From k = 128 on the cached step keeps its operand in tensor memory (the kernel's kTmemA): one tile
// of the split pair would take 64 KB of shared memory and more, which left room for a single
// buffer -- a bubble at every unit boundary -- and a short R ring (measured at k = 128 / 256 on FLUX
// rows: 0.75 / 0.38 of the copy bandwidth with the operand in shared memory, 0.83-0.91 / 0.64 so).
// TMEM bounds the rank: k columns of operand and two accumulators.
bool cached_operand_in_tmem(int k) { return k >= 128 && k + 2 * kTileCols <= 512; }

bool fill_cached(const StepArgs &a, UmmaParams &p) {
    if (!fill_params(a, p)) return false;
    fill_groups(a, p);
    const size_t avail = kSmemBudget - 1024 /*alignment*/ - kBarBytes - 64;
    if (cached_operand_in_tmem(a.k)) {
        // TMEM: operand buffers of k columns first (two while two accumulators still fit behind
        // them), then the accumulator ring.  Groups of two chunks while they fit: N = 128 is the
        // narrowest MMA that costs no more than a narrower one.
        p.gc = a.k + 2 * 2 * kTileCols <= 512 ? 2 : 1;
        p.acc_cols = p.gc * kTileCols;
        p.acc_stride = p.acc_cols;
        p.a_bufs = 2 * a.k + 2 * p.acc_cols <= 512 ? 2 : 1;
        p.acc_base = p.a_bufs * a.k;
        p.acc_stages = (512 - p.acc_base) / p.acc_stride < kAccStages ? (512 - p.acc_base) / p.acc_stride : kAccStages;
        p.vslice_bytes = (uint32_t)p.gc * kTileCols * a.k * 2;
        auto stages_for = [&](int v_slots) {
            const size_t fixed = (size_t)v_slots * p.vslice_bytes;
            if (fixed + 4 * (size_t)kTileBytes > avail) return 0;
            int st = (int)((avail - fixed) / kTileBytes);
            if (st > kMaxStages) st = kMaxStages;
            return st & ~1;   // even: a slot then always serves the same epilogue group (chunk parity)
        };
        p.v_slots = stages_for(3) >= 8 ? 3 : 2;
        p.stages = stages_for(p.v_slots);
        return p.stages >= 4 && p.acc_stages >= 2;
    }
    // operand in shared memory, two buffers (k <= 64)
    p.acc_base = 0;
    p.acc_stride = p.acc_cols;
    const size_t fixed = (size_t)p.v_slots * p.vslice_bytes;
    p.a_bufs = 2;
    if (2 * (size_t)p.a_bytes + fixed + 6 * (size_t)kTileBytes > avail) return false;
    p.stages = (int)((avail - 2 * (size_t)p.a_bytes - fixed) / kTileBytes);
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    p.stages &= ~1;   // even: a slot then always serves the same epilogue group (chunk parity)
    return true;
}
size_t smem_bytes_cached(const UmmaParams &p) {
    const size_t a_smem = cached_operand_in_tmem(p.k) ? 0 : (size_t)p.a_bufs * p.a_bytes;
    return 1024 + a_smem + (size_t)p.v_slots * p.vslice_bytes + (size_t)p.stages * kTileBytes + kBarBytes + 64;
}

bool shape_ok(const StepArgs &a) {
    if (a.dtype != SVDCACHE_BF16) return false;
    if (!(a.k == 16 || a.k == 32 || (a.k % 64) == 0)) return false;
    if (a.D < 64 || a.N < 1 || a.N > 0x7FFFFFFFLL) return false;
    return encode_fn() != nullptr;
}

}  // namespace

#ifdef SVDC_TRACE
}  // namespace svdc
extern "C" __attribute__((visibility("default"))) int svdcache_trace_dump(unsigned long long *host) {
    return (int)cudaMemcpyFromSymbol(host, svdc::g_trace, sizeof(svdc::g_trace));
}
namespace svdc {
#endif

bool umma_supported(const StepArgs &a, bool full) {
    if (!shape_ok(a)) return false;
    UmmaParams p;
    return full ? fill_full(a, p) : fill_cached(a, p);
}

int umma_cached_step(const StepArgs &a, cudaStream_t s) {
    UmmaParams p{};
    if (!fill_cached(a, p)) return SVDCACHE_ERR_BAD_SHAPE;
    // Units: a row tile, or a column range of it (in whole MMA groups).  The split is the one that
    // minimises what the busiest CTA has to stream, in chunks of R + Fhat traffic (32 KB) -- and,
    // among splits within a few per cent of that, the finest one the operand buffers allow: CTAs that
    // work on neighbouring column ranges of the same rows at the same time read and write whole
    // DRAM pages together (measured on the FLUX shape: 6.3 TB/s with single-group units, 5.7 with
    // whole tiles).  Every unit fetches its own copy of the tile's operand; with the operand in
    // tensor memory that is nkb chunks' worth of traffic per unit, which the count includes.
    const int sms = num_sms();
    const int tiles = p.row_tiles * a.nblocks;
    const int groups_total = (p.chunks_total + p.gc - 1) / p.gc;
    const bool a_tmem = cached_operand_in_tmem(a.k);
    const int unit_cost = a_tmem ? p.nkb : 0;
    auto load_of = [&](int ds, int *eff_out, int *gps_out) {
        const int gps = (groups_total + ds - 1) / ds;            // groups per slice
        const int eff = (groups_total + gps - 1) / gps;          // slices that result
        const int rounds = (tiles * eff + sms - 1) / sms;
        *eff_out = eff; *gps_out = gps;
        return rounds * (gps * p.gc + unit_cost);
    };
    int best_load = 1 << 30;
    p.dsplit = 1;
    p.chunks_per_slice = p.chunks_total;
    for (int ds = 1; ds <= groups_total && ds <= 16; ++ds) {
        int eff, gps;
        const int load = load_of(ds, &eff, &gps);
        if (load < best_load) { best_load = load; p.dsplit = eff; p.chunks_per_slice = gps * p.gc; }
    }
    if (p.a_bufs > 1)
        for (int ds = 1; ds <= groups_total && ds <= 16; ++ds) {
            int eff, gps;
            const int slack = a_tmem ? 20 : 50;   // within 5 % (operand in tensor memory: measured at k = 128), else 2 %
            if (load_of(ds, &eff, &gps) * slack <= best_load * (slack + 1) && eff > p.dsplit) { p.dsplit = eff; p.chunks_per_slice = gps * p.gc; }
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
    // the operand: the split pair of the state's Chat, or that of a forecast buffer
    const ForecastLayout FL = forecast_layout(a.N, a.k);
    const char *op_hi = a.coef ? (const char *)a.coef + FL.hi : (const char *)a.state + SL.op_hi;
    const char *op_lo = a.coef ? (const char *)a.coef + FL.lo : (const char *)a.state + SL.op_lo;
    const size_t op_stride = a.coef ? a.coef_stride : a.state_stride;
    rc = make_map(&tm_ahi, op_hi, a.k, a.N, a.nblocks, (uint64_t)a.k * 2, op_stride, p.kb_elems, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_alo, op_lo, a.k, a.N, a.nblocks, (uint64_t)a.k * 2, op_stride, p.kb_elems, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_out, a.Fhat, a.D, a.N, a.nblocks, (uint64_t)a.ld * 2, a.Fhat_stride, kTileCols, kSlabRows);
    if (rc) return rc;

    const size_t smem = smem_bytes_cached(p);
    const int grid = p.units < sms ? p.units : sms;
    if (a_tmem) {
        rc = allow_big_smem(umma_cached_kernel<true>, kSmemBudget);
        if (rc) return rc;
        umma_cached_kernel<true><<<grid, kThreadsCached, smem, s>>>(tm_r, tm_v, tm_ahi, tm_alo, tm_out, p);
    } else {
        rc = allow_big_smem(umma_cached_kernel<false>, kSmemBudget);
        if (rc) return rc;
        umma_cached_kernel<false><<<grid, kThreadsCached, smem, s>>>(tm_r, tm_v, tm_ahi, tm_alo, tm_out, p);
    }
    count_launch();
    return check_last_launch();
}

int umma_wait_selftest(void *state, long long limit_cycles, cudaStream_t s) {
    UmmaParams p{};
    p.state = (char *)state;
    p.nblocks = 1;
    wait_selftest_kernel<<<1, 64, 0, s>>>(p, limit_cycles);
    count_launch();
    return check_last_launch();
}

int umma_full_step(const StepArgs &a, cudaStream_t s) {
    UmmaParams p{};
    if (!fill_full(a, p)) return SVDCACHE_ERR_BAD_SHAPE;
    p.dsplit = 1;
    p.chunks_per_slice = p.chunks_total;
    p.units = p.row_tiles * a.nblocks;

    const StateLayout SL = state_layout(a.N, a.D, a.k, a.dtype);
    const BasisLayout BL = basis_layout(a.D, a.k, a.dtype);
    CUtensorMap tm_f, tm_vt, tm_v, tm_rout, tm_chat, tm_rold;
    int rc = make_map(&tm_f, a.F, a.D, a.N, a.nblocks, (uint64_t)a.ld * 2, a.F_stride, kTileCols, kTileRows);
    if (rc) return rc;
    rc = make_map(&tm_vt, (const char *)a.basis + BL.vt_bf16, a.D, a.k, a.nblocks, (uint64_t)a.D * 2,
                  a.basis_stride, kTileCols, a.k);
    if (rc) return rc;
    rc = make_map(&tm_v, (const char *)a.basis + BL.v_bf16, a.k, a.D, a.nblocks, (uint64_t)a.k * 2, a.basis_stride,
                  p.kb_elems, p.gc * kTileCols);
    if (rc) return rc;
    rc = make_map(&tm_rout, (char *)a.state + SL.r, a.D, a.N, a.nblocks, (uint64_t)a.D * 2, a.state_stride,
                  kTileCols, kSlabRows);
    if (rc) return rc;
    rc = make_map(&tm_chat, (char *)a.state + SL.chat, a.k, a.N, a.nblocks, (uint64_t)a.k * 4, a.state_stride,
                  a.k < 32 ? a.k : 32, kTileRows, 4);
    if (rc) return rc;
    // the stored R as whole chunks, for the residual EMA's third stream (unused otherwise)
    rc = make_map(&tm_rold, (const char *)a.state + SL.r, a.D, a.N, a.nblocks, (uint64_t)a.D * 2, a.state_stride,
                  kTileCols, kTileRows);
    if (rc) return rc;

    const size_t smem = smem_bytes_full(p);
    const int sms = num_sms();
    const int grid = p.units < sms ? p.units : sms;
    auto launch = [&](auto kern) {
        const int rc_attr = allow_big_smem(kern, kSmemBudget);
        if (rc_attr) return rc_attr;
        kern<<<grid, kThreadsFull, smem, s>>>(tm_f, tm_vt, tm_v, tm_rout, tm_chat, tm_rold, p);
        return (int)SVDCACHE_OK;
    };
    // operand in tensor memory from k = 64 on (fill_full has sized the rings for it); the residual EMA
    // of the ablation is an instantiation of its own (a third TMA stream and ring for the old R)
    const bool ema = a.beta_r > 0.0f;
    if (a.k >= 64) rc = ema ? launch(umma_full_kernel<true, true>) : launch(umma_full_kernel<true, false>);
    else rc = ema ? launch(umma_full_kernel<false, true>) : launch(umma_full_kernel<false, false>);
    if (rc) return rc;
    count_launch();
    return check_last_launch();
}

}  // namespace svdc
