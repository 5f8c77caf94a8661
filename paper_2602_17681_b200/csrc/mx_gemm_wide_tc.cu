// Block-scaled GEMM on CTA pairs with 256 x 256 output tiles:  out[M x N] = g dq(Qa) dq(Qw)^T + c.
//
// The 256 x 192 pair kernel pulls 31 KB per SM from L2 for every 412 tensor-pipe cycles; a 256 x 256 tile needs 35 KB
// per 550, 14 % fewer bytes per flop.  But two 256-column accumulators would fill all 512 tensor-memory columns and leave
// none for the scale factors, which the block-scaled MMA reads from tensor memory.  So a tile is accumulated as two
// independent halves of 128 columns (two N = 128 MMAs per K step) in THREE rotating 128-column buffers, with the scale
// buffers in the remaining 128 columns.  Half h (tile t has halves 2t and 2t + 1) lives in buffer h mod 3: when a tile
// starts, its first half's buffer was drained a whole tile ago and its second half's buffer is the one the epilogue
// empties FIRST -- into registers, handing it back at once.  Until that has happened the MMA warp issues first halves
// only, running up to four K slabs ahead, and catches the second half up on the same shared-memory stages afterwards:
// the tensor pipe does not idle at a tile boundary (measured before this: about 3000 cycles per tile, a fifth of the
// main loop at K = 4096, spent waiting for the commit -> epilogue -> tcgen05.ld -> remote arrive chain).
// Each CTA keeps rows [64 r, 64 r + 64) and [128 + 64 r, 128 + 64 r + 64) of the weight tile (r = its rank), so that an
// N = 128 pair MMA finds half of its columns in each CTA for either half of the tile.
//
//   warp 0    code producer (both CTAs): per 128-byte K slab three tiled loads, its 128 rows of activation codes and its
//             two 64-row pieces of the weight tile; bytes of both CTAs are counted on the leader's "full" barrier
//   warp 3    scale producer (both CTAs): per slab the scale tiles of its 128 activation rows and of all 256 weight rows
//   warp 2    leader: tcgen05.cp of the scale tiles into one of SF_BUFS tensor-memory buffers (a ring of its own, not
//             tied to the code stages), once the MMAs that last read that buffer are done; its commit is the second
//             arrival on the code stage's "full" barrier, so the MMA warp waits once per slab (a wait costs the issuing
//             thread about 100 cycles even when it succeeds at once, a commit 55: with two waits per slab the thread
//             needed 620 cycles per slab for 576 cycles of tensor-pipe work)
//   warp 1    leader: MMA issue as described; one commit per slab frees its stage once BOTH halves have used it
//   warps 4-7 epilogue (both CTAs): per half, four tcgen05.ld into registers, buffer handed back, then + c, swizzled
//             staging, TMA store; the tile's 256 values of c are fetched into shared memory before the wait
// Tail: the tiles of the last, partly filled wave are cut into column slices of 128 or 64 (as many as fit the CTA pairs),
// each a work item of its own that uses one accumulator half; every output element still sums its K slabs in the same
// order, so the result does not depend on the cut.
// Formats: MXFP4 (kind::mxf4), MXFP8 / MXINT4 bytes (kind::mxf8f6f4) and NVFP4 (kind::mxf4nvf4: blocks of 16, E4M3
// scales, result multiplied by the product of the two tensor scales).  Every wait is bounded.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

template <int FMT, int STAGES_>
struct MxGemmWideCfg {
    static constexpr int BLOCK_M = 128, BLOCK_N = 256, HALF_N = 128, PIECE_N = 64, NB_RT = 2;
    static constexpr int SF_KT = FMT == FMT_FP4 ? 2 : FMT == FMT_NVFP4 ? 4 : 1;   // scale tiles (128 rows x 4 scales) per 128-byte K slab
    static constexpr int A_BYTES = BLOCK_M * 128, B_BYTES = HALF_N * 128, STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SFA_BYTES = SF_KT * 512, SFB_BYTES = NB_RT * SF_KT * 512, SF_SLOT_BYTES = SFA_BYTES + SFB_BYTES;
    static constexpr int STAGES = STAGES_;
    static constexpr int STG_BUFS = 2;                                            // 4 KB staging buffers per epilogue warp
    static constexpr int SF_SLOTS = FMT == FMT_NVFP4 ? 4 : 8;
    static constexpr int STAGING_BYTES = 4 * STG_BUFS * 4096;
    static constexpr int CVEC_BYTES = 4 * BLOCK_N * 4;                            // each epilogue warp's copy of the tile's c[n]
    static constexpr int BAR_BYTES = 1024;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + SF_SLOTS * SF_SLOT_BYTES + STAGING_BYTES + CVEC_BYTES + BAR_BYTES;
    static constexpr int ACC_COLS = 384;                                          // three rotating 128-column accumulators
    static constexpr int SF_COLS = SF_KT * 4 * (1 + NB_RT);                       // tensor-memory columns of one slab's scales
    static constexpr int SF_BUFS = (512 - ACC_COLS) / SF_COLS > 5 ? 5 : (512 - ACC_COLS) / SF_COLS;
    static constexpr int TMEM_COLS = 512;
    static_assert(SF_BUFS >= 2 && ACC_COLS + SF_BUFS * SF_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(STAGE_BYTES % 1024 == 0 && SF_SLOT_BYTES % 512 == 0, "operand tiles must stay 1024-byte aligned");
    static constexpr int MAX_AHEAD = (STAGES < SF_BUFS ? STAGES : SF_BUFS) - 1;   // slabs the first half may run ahead of the second
    static_assert(MAX_AHEAD >= 1, "the first half must be able to run ahead");
    // the scale copier's commit is the second arrival on a stage's "full" barrier: it must not reach a stage before the
    // phase of the slab that used the stage last has completed, which holds while the scale ring is no longer than the code ring
    static_assert(SF_BUFS <= STAGES, "scale ring longer than the code ring");
    static_assert(2 * STAGES + 2 * SF_SLOTS + SF_BUFS + 7 <= 120, "barrier area");
};

struct MxGemmWideParams {
    const float* c;
    const float* ga; const float* gw;      // NVFP4: the operands' tensor scales (device memory); null otherwise
    int M, N, num_kb, m_tiles, n_tiles;
    int full_items;      // work items [0, full_items) are whole 256 x 256 tiles; the rest are column slices of the remaining tiles
    int num_items;
    int slices;          // slices per cut tile: 1 (no cut), 2 (128 columns each) or 4 (64 columns each)
    uint32_t* status;
};

constexpr int kWideThreads = 8 * 32;

// Work item -> row tile, first column, width (256, 128 or 64).
__device__ __forceinline__ void wide_decode(const MxGemmWideParams& p, int item, int& m_tile, int& n0, int& width) {
    if (item < p.full_items) {
        m_tile = item % p.m_tiles; n0 = (item / p.m_tiles) * 256; width = 256;
    } else {
        const int r = item - p.full_items, tile = p.full_items + r / p.slices, slice = r % p.slices;
        width = 256 / p.slices;
        m_tile = tile % p.m_tiles; n0 = (tile / p.m_tiles) * 256 + slice * width;
    }
}

template <int FMT, int STAGES_>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kWideThreads, 1)
mx_gemm_wide_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                       const __grid_constant__ CUtensorMap tm_b32, const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfb,
                       const __grid_constant__ CUtensorMap tm_out, const MxGemmWideParams p) {
    using Cfg = MxGemmWideCfg<FMT, STAGES_>;
    constexpr int STAGES = Cfg::STAGES, SF_SLOTS = Cfg::SF_SLOTS, SF_BUFS = Cfg::SF_BUFS, STG_BUFS = Cfg::STG_BUFS;
    extern __shared__ uint8_t smem_raw[];
    // the dynamic shared-memory window starts at the same offset in both CTAs: every address below is valid in the peer too
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sf_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t staging_base = sf_base + SF_SLOTS * Cfg::SF_SLOT_BYTES;
    const uint32_t cvec_base = staging_base + Cfg::STAGING_BYTES;
    const uint32_t bar_base = cvec_base + Cfg::CVEC_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                     // leader: both CTAs' code bytes landed AND the slab's scales copied
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };         // each CTA: the slab's MMAs are done
    constexpr int kSf0 = 2 * STAGES;
    auto sf_full_bar = [&](int g) { return bar_base + 8u * (kSf0 + g); };         // leader: both CTAs' scale bytes landed
    auto sf_empty_bar = [&](int g) { return bar_base + 8u * (kSf0 + SF_SLOTS + g); };   // each CTA: slot copied to tensor memory
    constexpr int kSft0 = kSf0 + 2 * SF_SLOTS;
    constexpr int kAcc0 = kSft0 + SF_BUFS;
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (kAcc0 + b); };     // each CTA: the half in accumulator buffer b is complete
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (kAcc0 + 3 + b); };   // leader: buffer b has been read out (8 warps)
    const uint32_t tmem_slot = bar_base + 8u * (kAcc0 + 6);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const bool leader = rank == 0;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_a); prefetch_tmap(&tm_b); prefetch_tmap(&tm_b32); prefetch_tmap(&tm_sfa); prefetch_tmap(&tm_sfb); prefetch_tmap(&tm_out);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // full: code bytes + scale copy
        for (int g = 0; g < SF_SLOTS; ++g) { mbar_init(sf_full_bar(g), 1); mbar_init(sf_empty_bar(g), 1); }
        for (int b = 0; b < 3; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 8); }   // 4 epilogue warps x 2 CTAs
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS); tmem_relinquish_pair(); }
    tc_fence_before();
    cluster_sync_all();                                 // both CTAs' barriers and tensor memory exist from here on
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    grid_dependency_wait();            // set-up above may have overlapped the previous kernel; its results are needed from here on
    grid_launch_dependents();          // the kernel after this one may set itself up on SMs this one has left
    const int num_tiles = p.num_items;                  // work items: whole tiles, then the slices of the last wave's tiles
    const int pair = (int)cluster_id_x(), num_pairs = (int)num_clusters_x();
    constexpr uint16_t kBoth = 3, kLeader = 1;
    int tiles_mine = 0;
    for (int tile = pair; tile < num_tiles; tile += num_pairs) ++tiles_mine;
    const long long slabs_mine = (long long)tiles_mine * p.num_kb;

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ code producer (both CTAs)
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int m_tile, n0, width;
                wide_decode(p, tile, m_tile, n0, width);
                const int m0 = m_tile * 256 + (int)rank * Cfg::BLOCK_M;
                // bytes per CTA and slab: its rows of A and its share (a quarter of the item's columns, twice for a whole tile)
                const uint32_t cta_bytes = (uint32_t)(Cfg::A_BYTES + (width >> 1) * 128);
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    if (leader) mbar_expect_tx(full_bar(s), 2 * cta_bytes);
                    const uint32_t bar = mapa_shared(full_bar(s), 0), st = smem_base + s * Cfg::STAGE_BYTES;
                    tma_load_2d_pair(st, &tm_a, kb * 128, m0, bar);
                    if (width == 64) {
                        tma_load_2d_pair(st + Cfg::A_BYTES, &tm_b32, kb * 128, n0 + (int)rank * 32, bar);
                    } else {
                        tma_load_2d_pair(st + Cfg::A_BYTES, &tm_b, kb * 128, n0 + (int)rank * Cfg::PIECE_N, bar);
                        if (width == 256)
                            tma_load_2d_pair(st + Cfg::A_BYTES + Cfg::B_BYTES / 2, &tm_b, kb * 128, n0 + Cfg::HALF_N + (int)rank * Cfg::PIECE_N, bar);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp_idx == 3) {
        // ------------------------------------------------------------------ scale producer (both CTAs)
        if (lane == 0) {
            uint32_t g = 0, gph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int m_tile, n0, width;
                wide_decode(p, tile, m_tile, n0, width);
                const int m_rt = (m_tile * 256 + (int)rank * Cfg::BLOCK_M) >> 7, n_rt = n0 >> 7;   // a slice's scales sit in the first of the two weight row tiles
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(sf_empty_bar(g), gph ^ 1u, p.status))) break;
                    if (leader) mbar_expect_tx(sf_full_bar(g), 2 * Cfg::SF_SLOT_BYTES);
                    const uint32_t bar = mapa_shared(sf_full_bar(g), 0), slot = sf_base + g * Cfg::SF_SLOT_BYTES;
                    // coordinates: (word in tile, scale k-tile, 128-row tile); tiles outside the buffer read as zero
                    tma_load_3d_pair(slot, &tm_sfa, 0, kb * Cfg::SF_KT, m_rt, bar);
                    tma_load_3d_pair(slot + Cfg::SFA_BYTES, &tm_sfb, 0, kb * Cfg::SF_KT, n_rt, bar);
                    if (++g == SF_SLOTS) { g = 0; gph ^= 1u; }
                }
            }
        }
    } else if (warp_idx == 2) {
        // ------------------------------------------------------------------ scale copies (leader CTA only)
        // Slab i's scales go to tensor-memory buffer i % SF_BUFS, which the MMAs of slab i - SF_BUFS read last; those are
        // done when the "empty" barrier of THAT slab's code stage completes the phase that slab belongs to.  The warp
        // waits for the slabs in order, so it observes every phase of every stage's barrier.
        if (leader) {
            const bool issuer = elect_one();
            const uint32_t sf_t0 = tmem_base + Cfg::ACC_COLS;
            uint32_t g = 0, gph = 0, j = 0, jslab = 0 /* counts up to SF_BUFS, then stays */, es = 0, eph = 0, cs = 0 /* the slab's code stage */;
            for (long long i = 0; i < slabs_mine; ++i) {
                mbar_wait_or_flag(sf_full_bar(g), gph, p.status);
                if (jslab >= (uint32_t)SF_BUFS) {
                    mbar_wait_or_flag(empty_bar(es), eph, p.status);
                    if (++es == (uint32_t)STAGES) { es = 0; eph ^= 1u; }
                } else {
                    ++jslab;
                }
                tc_fence_after();
                if (issuer) {
                    const uint32_t sfa_t = sf_t0 + j * Cfg::SF_COLS, sfb_t = sfa_t + Cfg::SF_KT * 4;
                    const uint32_t sf_lo = desc_lo(sf_base + g * Cfg::SF_SLOT_BYTES), sfb_lo = sf_lo + (Cfg::SFA_BYTES >> 4);
#pragma unroll
                    for (int kt = 0; kt < Cfg::SF_KT; ++kt) {
                        tc_cp_scale_pair_lean(sfa_t + kt * 4, sf_lo + kt * 32);
#pragma unroll
                        for (int r = 0; r < Cfg::NB_RT; ++r)
                            tc_cp_scale_pair_lean(sfb_t + kt * Cfg::NB_RT * 4 + r * 4, sfb_lo + (r * Cfg::SF_KT + kt) * 32);
                    }
                    tc_commit_pair(full_bar(cs), kLeader);        // second arrival on the stage's barrier: the scales are in tensor memory ...
                    tc_commit_pair(sf_empty_bar(g), kBoth);       // ... and both CTAs' slots have been read
                }
                __syncwarp();
                if (++g == (uint32_t)SF_SLOTS) { g = 0; gph ^= 1u; }
                if (++j == (uint32_t)SF_BUFS) j = 0;
                if (++cs == (uint32_t)STAGES) cs = 0;
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue (leader CTA only)
        if (leader) {                                    // whole warp, one elected lane issues
            const bool issuer = elect_one();
            constexpr uint32_t kIdescMx = make_idesc_block_scaled(2 * Cfg::BLOCK_M, Cfg::HALF_N, FMT == FMT_FP8 ? 0u : 1u);
            constexpr uint32_t kIdesc = FMT == FMT_NVFP4 ? (kIdescMx & ~(1u << 23)) : kIdescMx;     // NVFP4: E4M3 scales
            constexpr uint32_t kIdesc64 = (kIdesc & ~(0x3Fu << 17)) | ((64u >> 3) << 17);           // the same with N = 64
            const uint32_t a_lo0 = desc_lo(smem_base), sf_t0 = tmem_base + Cfg::ACC_COLS;
            // The four MMAs of one half on one stage, each 32 bytes of K per row.  Whole tile: half 0 = columns [0, 128),
            // half 1 = [128, 256), second weight piece and second scale row tile.  Slice: half 0 only, N = 128 or 64, and
            // `sfb_off` = the slice's first row inside its scale row tile, in units of 32 rows (0 or 2).
            auto issue_half = [&](uint32_t half, uint32_t stage, uint32_t sfbuf, uint32_t d_tmem, uint32_t first_accum, uint32_t idesc_n,
                                  uint32_t sfb_off) {
                const uint32_t a_lo = a_lo0 + stage * (Cfg::STAGE_BYTES >> 4);
                const uint32_t b_lo = a_lo + (Cfg::A_BYTES >> 4) + half * (Cfg::B_BYTES >> 5);
                const uint32_t sfa_t = sf_t0 + sfbuf * Cfg::SF_COLS, sfb_t = sfa_t + Cfg::SF_KT * 4 + half * 4 + sfb_off;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int kt = FMT == FMT_FP4 ? (q >> 1) : FMT == FMT_NVFP4 ? q : 0;
                    const uint32_t sf_id = FMT == FMT_FP4 ? (uint32_t)(q & 1) * 2u : FMT == FMT_NVFP4 ? 0u : (uint32_t)q;
                    const uint32_t idesc = idesc_n | (sf_id << 4) | (sf_id << 29);
                    const uint32_t accum = q == 0 ? first_accum : 1u;
                    if (FMT == FMT_FP4) mma_mxf4_pair_lean(d_tmem, a_lo + 2 * q, b_lo + 2 * q, idesc, sfa_t + kt * 4, sfb_t + kt * Cfg::NB_RT * 4, accum);
                    else if (FMT == FMT_NVFP4) mma_nvf4_pair_lean(d_tmem, a_lo + 2 * q, b_lo + 2 * q, idesc, sfa_t + kt * 4, sfb_t + kt * Cfg::NB_RT * 4, accum);
                    else mma_mxf8_pair_lean(d_tmem, a_lo + 2 * q, b_lo + 2 * q, idesc, sfa_t + kt * 4, sfb_t + kt * Cfg::NB_RT * 4, accum);
                }
            };
            // cursors of the first half (x: waits for data) and of the second half (y: follows on stages x has seen)
            uint32_t sx = 0, sphx = 0, jx = 0, sy = 0, jy = 0, tile_count = 0;
            for (int tile = pair; tile < num_tiles; tile += num_pairs, ++tile_count) {
                const uint32_t h0 = 2u * tile_count, h1 = h0 + 1u;
                const uint32_t b0 = h0 % 3u, b1 = h1 % 3u, u0 = h0 / 3u, u1 = h1 / 3u;
                const uint32_t d0 = tmem_base + b0 * 128u, d1 = tmem_base + b1 * 128u;
                int m_tile, n0, width;
                wide_decode(p, tile, m_tile, n0, width);
                mbar_wait_or_flag(tempty_bar(b0), (u0 & 1u) ^ 1u, p.status);       // drained a tile ago: passes at once
                tc_fence_after();
                if (width != 256) {
                    // a slice: one half, N = 128 or 64; the item's second half-slot stays empty but keeps its place in the
                    // rotation (its buffer's barriers see every phase)
                    const uint32_t idesc_n = width == 64 ? kIdesc64 : kIdesc, sfb_off = (uint32_t)(n0 & 127) >> 5;
                    for (int kb = 0; kb < p.num_kb; ++kb) {
                        mbar_wait_or_flag(full_bar(sx), sphx, p.status);
                        tc_fence_after();
                        if (issuer) {
                            issue_half(0u, sx, jx, d0, (uint32_t)(kb != 0), idesc_n, sfb_off);
                            tc_commit_pair(empty_bar(sx), kBoth);
                            if (kb == p.num_kb - 1) tc_commit_pair(tfull_bar(b0), kBoth);
                        }
                        __syncwarp();
                        if (++sx == (uint32_t)STAGES) { sx = 0; sphx ^= 1u; }
                        if (++jx == (uint32_t)SF_BUFS) jx = 0;
                    }
                    sy = sx; jy = jx;
                    mbar_wait_or_flag(tempty_bar(b1), (u1 & 1u) ^ 1u, p.status);
                    if (issuer) tc_commit_pair(tfull_bar(b1), kBoth);
                    __syncwarp();
                    continue;
                }
                bool y_free = false;
                int kx = 0, ky = 0;
                while (ky < p.num_kb) {
                    if (!y_free) {
                        y_free = __any_sync(0xffffffffu, mbar_try_wait(tempty_bar(b1), (u1 & 1u) ^ 1u));
                        if (!y_free && (kx == p.num_kb || kx - ky >= Cfg::MAX_AHEAD)) {    // nothing left to run ahead with
                            mbar_wait_or_flag(tempty_bar(b1), (u1 & 1u) ^ 1u, p.status);
                            y_free = true;
                        }
                        if (y_free) tc_fence_after();
                    }
                    if (y_free && ky < kx) {
                        // catch up: the second half on a stage the first half has already used; frees the stage
                        if (issuer) {
                            issue_half(1u, sy, jy, d1, (uint32_t)(ky != 0), kIdesc, 0u);
                            tc_commit_pair(empty_bar(sy), kBoth);
                            if (ky == p.num_kb - 1) tc_commit_pair(tfull_bar(b1), kBoth);
                        }
                        __syncwarp();
                        if (++sy == (uint32_t)STAGES) sy = 0;
                        if (++jy == (uint32_t)SF_BUFS) jy = 0;
                        ++ky;
                    } else {
                        // next slab: first half, and the second half with it when that has caught up
                        mbar_wait_or_flag(full_bar(sx), sphx, p.status);
                        tc_fence_after();
                        const bool both = y_free;                                  // then ky == kx
                        if (issuer) {
                            issue_half(0u, sx, jx, d0, (uint32_t)(kx != 0), kIdesc, 0u);
                            if (kx == p.num_kb - 1) tc_commit_pair(tfull_bar(b0), kBoth);
                            if (both) {
                                issue_half(1u, sx, jx, d1, (uint32_t)(kx != 0), kIdesc, 0u);
                                tc_commit_pair(empty_bar(sx), kBoth);              // frees the code stage in both CTAs; the scale copier watches it too
                                if (kx == p.num_kb - 1) tc_commit_pair(tfull_bar(b1), kBoth);
                            }
                        }
                        __syncwarp();
                        if (++sx == (uint32_t)STAGES) { sx = 0; sphx ^= 1u; }
                        if (++jx == (uint32_t)SF_BUFS) jx = 0;
                        ++kx;
                        if (both) { sy = sx; jy = jx; ++ky; }
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 4..7, both CTAs)
        const int q = warp_idx & 3;                     // tensor-memory lane quarter this warp may read
        const uint32_t stg0 = staging_base + (uint32_t)(warp_idx - 4) * STG_BUFS * 4096u;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t cvec = cvec_base + (uint32_t)(warp_idx - 4) * (Cfg::BLOCK_N * 4);
        float out_scale = 1.0f;
        if (FMT == FMT_NVFP4) out_scale = __ldg(p.ga) * __ldg(p.gw);
        uint32_t tile_count = 0, stg_it = 0;
        int tile_n0 = 0;
        bool ok = true;
        // one 32 x 32 piece of the result: + c, into the swizzled staging buffer, out through the copy engine
        auto store_chunk = [&](const uint32_t (&r)[32], int row0, int col0) {
            const uint32_t stg = stg0 + (stg_it % STG_BUFS) * 4096u;
            ++stg_it;
            if (lane == 0) bulk_wait_read<STG_BUFS - 1>();       // the store that last used this buffer has read it
            __syncwarp();
            const uint32_t cv_addr = cvec + (uint32_t)(col0 - tile_n0) * 4u;
#pragma unroll
            for (int t = 0; t < 8; ++t) {                        // 128-byte swizzle: chunk t of row `lane` -> t ^ (lane & 7)
                float cv[4];                                     // every lane reads the same address: a broadcast
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(cv[0]), "=f"(cv[1]), "=f"(cv[2]), "=f"(cv[3]) : "r"(cv_addr + 16u * t));
                float4 v;
                if (FMT == FMT_NVFP4) {
                    v = make_float4(fmaf(__uint_as_float(r[4 * t]), out_scale, cv[0]), fmaf(__uint_as_float(r[4 * t + 1]), out_scale, cv[1]),
                                    fmaf(__uint_as_float(r[4 * t + 2]), out_scale, cv[2]), fmaf(__uint_as_float(r[4 * t + 3]), out_scale, cv[3]));
                } else {
                    v = make_float4(__uint_as_float(r[4 * t]) + cv[0], __uint_as_float(r[4 * t + 1]) + cv[1],
                                    __uint_as_float(r[4 * t + 2]) + cv[2], __uint_as_float(r[4 * t + 3]) + cv[3]);
                }
                const uint32_t dst = stg + (uint32_t)lane * 128u + (uint32_t)((t ^ (lane & 7)) * 16);
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && col0 < p.N && row0 < p.M) {
                tma_store_2d(&tm_out, stg, col0, row0);
                bulk_commit();
            }
        };
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tile_count) {
            int m_tile, n0, width;
            wide_decode(p, tile, m_tile, n0, width);
            const int m0 = m_tile * 256 + (int)rank * Cfg::BLOCK_M;
            // the tile's 256 values of c into this warp's shared-memory copy, fetched while the MMAs still run (a lane
            // brings eight of them); the previous tile's last reads of the copy lie before the __syncwarp of its last chunk
            tile_n0 = n0;
            {
                float4 c0 = make_float4(0.f, 0.f, 0.f, 0.f), c1 = c0;
                const int cn = n0 + lane * 8;
                if (p.c != nullptr) {
                    if (cn + 8 <= p.N) {
                        c0 = __ldg(reinterpret_cast<const float4*>(p.c + cn));
                        c1 = __ldg(reinterpret_cast<const float4*>(p.c + cn) + 1);
                    } else {
                        float t[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) t[i] = cn + i < p.N ? p.c[cn + i] : 0.f;
                        c0 = make_float4(t[0], t[1], t[2], t[3]); c1 = make_float4(t[4], t[5], t[6], t[7]);
                    }
                }
                const uint32_t dst = cvec + (uint32_t)lane * 32u;
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(c0.x), "f"(c0.y), "f"(c0.z), "f"(c0.w) : "memory");
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 16u), "f"(c1.x), "f"(c1.y), "f"(c1.z), "f"(c1.w) : "memory");
                __syncwarp();
            }
            const int row0 = m0 + q * 32;
#pragma unroll 1
            for (uint32_t half = 0; half < 2 && ok; ++half) {
                const uint32_t h = 2u * tile_count + half, b = h % 3u, u = h / 3u;
                ok = mbar_wait(tfull_bar(b), u & 1u, p.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                // the whole half into registers, and the buffer back to the MMA warp at once (a slice: its 128 or 64 columns
                // as the first half, nothing as the second)
                const int cols = width == 256 ? 128 : (half == 0 ? width : 0);
                uint32_t r0[32], r1[32], r2[32], r3[32];
                const uint32_t t0 = lane_base + b * 128u;
                if (cols >= 64) { tc_ld_32x32b_x32(t0, r0); tc_ld_32x32b_x32(t0 + 32u, r1); }
                if (cols == 128) { tc_ld_32x32b_x32(t0 + 64u, r2); tc_ld_32x32b_x32(t0 + 96u, r3); }
                tc_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (leader) mbar_arrive(tempty_bar(b));
                    else mbar_arrive_cluster(mapa_shared(tempty_bar(b), 0));
                }
                const int c0 = n0 + (int)half * 128;
                if (cols >= 64) { store_chunk(r0, row0, c0); store_chunk(r1, row0, c0 + 32); }
                if (cols == 128) { store_chunk(r2, row0, c0 + 64); store_chunk(r3, row0, c0 + 96); }
            }
        }
        if (lane == 0) bulk_wait<0>();
    }
    // teardown: if any wait gave up, let copies still in flight land before shared memory goes away
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    cluster_sync_all();             // the leader's MMAs read the peer's shared memory and write its tensor memory
    if (warp_idx == 1) tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
}

// ----------------------------------------------------------------------------------------------------
bool mx_gemm_wide_tc_supported(const MxGemmArgs& a) {
    if (a.fmt == FMT_FP4 || a.fmt == FMT_NVFP4) { if (a.K % 256 != 0) return false; }
    else if (a.fmt == FMT_FP8) { if (a.K % 128 != 0) return false; }
    else return false;
    if (a.M <= 128) return false;                      // one CTA covers 128 rows: a pair would idle its second half
    if (a.M > (1ll << 30) || a.N > (1ll << 30) || a.K > (1ll << 30)) return false;
    return a.K > 0;
}

template <int FMT, int STAGES>
static cudaError_t launch_wide_variant(const MxGemmArgs& a, cudaStream_t st) {
    using Cfg = MxGemmWideCfg<FMT, STAGES>;
    const int64_t k_bytes = a.fmt == FMT_FP8 ? a.K : a.K / 2;
    const uint64_t kt_total = a.fmt == FMT_NVFP4 ? (uint64_t)nvfp4_sf_k_tiles(a.K) : (uint64_t)sf_k_tiles(a.K);
    CUtensorMap tm_a, tm_b, tm_b32, tm_sfa, tm_sfb, tm_out;
    if (!make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)k_bytes, (uint64_t)a.M, (uint64_t)k_bytes, 128, Cfg::BLOCK_M) ||
        !make_tensor_map_2d(&tm_b, a.w_codes, 0, (uint64_t)k_bytes, (uint64_t)a.N, (uint64_t)k_bytes, 128, Cfg::PIECE_N) ||
        !make_tensor_map_2d(&tm_b32, a.w_codes, 0, (uint64_t)k_bytes, (uint64_t)a.N, (uint64_t)k_bytes, 128, 32) ||
        !make_tensor_map_scale_tiles(&tm_sfa, a.a_scales, kt_total, (uint64_t)((a.M + 127) / 128), Cfg::SF_KT, 1) ||
        !make_tensor_map_scale_tiles(&tm_sfb, a.w_scales, kt_total, (uint64_t)((a.N + 127) / 128), Cfg::SF_KT, Cfg::NB_RT) ||
        !make_tensor_map_2d(&tm_out, a.out, 2, (uint64_t)a.N, (uint64_t)a.M, (uint64_t)a.ldo * 4, 32, 32))
        return cudaErrorInvalidValue;
    MxGemmWideParams p;
    p.c = a.c; p.ga = a.a_tensor_scale; p.gw = a.w_tensor_scale;
    p.M = (int)a.M; p.N = (int)a.N; p.num_kb = (int)(k_bytes / 128);
    p.m_tiles = (int)((a.M + 255) / 256);
    p.n_tiles = (int)((a.N + Cfg::BLOCK_N - 1) / Cfg::BLOCK_N);
    p.status = a.status;
    auto kern = mx_gemm_wide_tc_kernel<FMT, STAGES>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int pairs = resident_cta_pairs((const void*)kern, kWideThreads, Cfg::SMEM_BYTES);
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    // the last, partly filled wave (or the only one) is cut into as many column slices as the CTA pairs can take at once
    const int64_t rem = tiles % pairs;
    p.slices = rem == 0 ? 1 : 4 * rem <= pairs ? 4 : 2 * rem <= pairs ? 2 : 1;
    if ((a.flags >> 12) & 1u) p.slices = 1;            // tuning: bit 12 of flags leaves the last wave uncut
    p.full_items = p.slices == 1 ? (int)tiles : (int)(tiles - rem);
    p.num_items = p.slices == 1 ? (int)tiles : (int)(tiles - rem + rem * p.slices);
    const unsigned grid = 2u * (unsigned)(p.num_items < pairs ? p.num_items : pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kWideThreads); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_b32, tm_sfa, tm_sfb, tm_out, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mx_gemm_wide_tc(const MxGemmArgs& a, cudaStream_t st) {
    if (a.fmt == FMT_FP4) return launch_wide_variant<FMT_FP4, 5>(a, st);
    if (a.fmt == FMT_NVFP4) return launch_wide_variant<FMT_NVFP4, 5>(a, st);
    return launch_wide_variant<FMT_FP8, 5>(a, st);
}

}  // namespace latmix
