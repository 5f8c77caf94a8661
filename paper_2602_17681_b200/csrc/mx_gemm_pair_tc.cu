// Block-scaled MX GEMM on CTA pairs (tcgen05 cta_group::2):  out[M x N] = dq(Qa) dq(Qw)^T + c.
//
// What bounds this product on B200 (measured with back-to-back issue probes and by timing the kernel with parts
// of its work left out):
//   * the tensor pipe needs N/2 + 7 cycles for a 128-row x N x 64 MXFP4 MMA (103 cycles at N = 192), the same in
//     pair mode; but ONE thread issues every MMA, it is an in-order machine that spends several cycles per
//     instruction, and a tcgen05.commit is seen by a waiting thread about 450 cycles after the work it tracks
//     ends -- a loop that rebuilds descriptors, copies scales and chains commits cannot keep the pipe fed;
//   * in this kernel all SMs together pull about 16 TB/s from L2 (the copy engine itself delivers 20-30 TB/s when one
//     thread per SM issues 16-32 KB boxes; each TMA instruction costs its issuing thread about 86 cycles), and the result's
//     235 MB on their way out slow the loads down further: bytes per SM per MMA cycle matter as much as DRAM.
// Hence two CTAs of a cluster share one 256 x BLOCK_N output tile: each loads its own 128 rows of activation
// codes but only HALF of the weight rows (28 KB instead of 40 KB per 128-byte K slab), and the issue work is spread:
//
//   warp 0    code producer (both CTAs): per K slab two tiled TMA loads into one of five stages -- the code tiles
//             of A and of this CTA's half of B.  Bytes of both CTAs are counted on the LEADER's "full" barrier.
//   warp 3    scale producer (both CTAs): per K slab two 3-D tiled loads into one of eight small slots -- the scale
//             tiles of its 128 rows of A and of ALL columns of B (each CTA's tensor core scales its rows against
//             every column).  Scales are 10 % of the bytes, so this ring runs well ahead of the code ring.
//   warp 2    leader: tcgen05.cp.cta_group::2 of the scale tiles into the tensor-memory scale buffer that belongs
//             to the stage (five stages, five buffers), as soon as the stage's previous MMAs are done; its
//             tcgen05.commit is the second arrival on the stage's "full" barrier (the first comes with the code
//             bytes).  That commit hop runs beside the TMA latency of the code tiles, not after it.
//   warp 1    leader: per K slab one wait, four tcgen05.mma.cta_group::2 .block_scale, one commit.  The loop is
//             unrolled over the stages and every operand is computed once, before the loop.
//   warps 4-7 epilogue (both CTAs): the tile's c[n] fetched into shared memory before the wait; the accumulator read in
//             two batches of three tcgen05.ld issued together (one at a time they made the epilogue the slowest part:
//             a load takes about 2000 cycles while MMAs run); + c, swizzled staging, TMA store; one arrival per warp on
//             the leader's "accumulator empty" barrier (remote for the peer) after the last batch has been read.
// Every wait is bounded; whatever happens, all threads of both CTAs meet at a cluster barrier before tensor
// memory is released and the CTAs exit, so neither CTA can touch a peer that has already gone.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

template <int FMT, int BLOCK_N_>
struct MxGemmPairCfg {
    static constexpr int BLOCK_M = 128;                            // rows per CTA; the pair covers 256
    static constexpr int BLOCK_N = BLOCK_N_, HALF_N = BLOCK_N_ / 2;
    static constexpr int NUM_ACC = 2, STG_BUFS = 2;
    static constexpr int SF_KT = FMT == FMT_FP4 ? 2 : 1;           // scale k-tiles (4 blocks each) per 128-byte K slab
    static constexpr int N_LOWBIT = BLOCK_N & -BLOCK_N;
    static constexpr int MAX_ROW_OFFSET = N_LOWBIT >= 128 ? 0 : 128 - N_LOWBIT;
    static constexpr int NB_RT = (MAX_ROW_OFFSET + BLOCK_N + 127) / 128;   // 128-row weight scale tiles a tile can touch
    static constexpr int A_BYTES = BLOCK_M * 128, B_BYTES = HALF_N * 128;
    static constexpr int SFA_BYTES = SF_KT * 512, SFB_BYTES = NB_RT * SF_KT * 512;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SF_SLOT_BYTES = SFA_BYTES + SFB_BYTES;
    static constexpr int STAGES = 5;                               // code ring; the issue loops are unrolled over it
    static constexpr int SF_SLOTS = 8;                             // scale ring in shared memory
    static constexpr int STAGING_BYTES = 4 * STG_BUFS * 4096;      // per epilogue warp: 32 rows x 128 bytes
    static constexpr int CVEC_BYTES = 4 * BLOCK_N * 4;              // each epilogue warp's copy of the tile's c[n]
    static constexpr int BAR_BYTES = 1024;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + SF_SLOTS * SF_SLOT_BYTES + STAGING_BYTES + CVEC_BYTES + BAR_BYTES;
    static constexpr int ACC_COLS = NUM_ACC * BLOCK_N;
    static constexpr int SF_COLS = SF_KT * 4 + SF_KT * NB_RT * 4;  // tensor-memory columns of one K slab's scales
    static constexpr int TMEM_COLS = 512;
    static_assert(ACC_COLS + STAGES * SF_COLS <= TMEM_COLS, "tensor memory budget: one scale buffer per stage");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(STAGE_BYTES % 1024 == 0 && SF_SLOT_BYTES % 512 == 0, "operand tiles must stay 1024-byte aligned");
    // scale-factor column offsets handed to the MMA must be even (an odd one raised a misaligned-address fault):
    // tiles start at multiples of 64 rows
    static_assert(BLOCK_N % 64 == 0 && BLOCK_N <= 256 && HALF_N % 8 == 0, "tile shape");
};

struct MxGemmPairParams {
    const float* c;
    int M, N, num_kb, m_tiles /* of 256 rows */, n_tiles;
    uint32_t* status;
};

constexpr int kPairThreads = 8 * 32;

template <int FMT, int BLOCK_N>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
mx_gemm_pair_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                       const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfb,
                       const __grid_constant__ CUtensorMap tm_out, const MxGemmPairParams p) {
    using Cfg = MxGemmPairCfg<FMT, BLOCK_N>;
    constexpr int STAGES = Cfg::STAGES, NUM_ACC = Cfg::NUM_ACC, STG_BUFS = Cfg::STG_BUFS;
    extern __shared__ uint8_t smem_raw[];
    // the dynamic shared-memory window starts at the same offset in both CTAs, so every address below is the
    // same offset in the peer: the MMA's descriptors and the multicast commits rely on that
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sf_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t staging_base = sf_base + Cfg::SF_SLOTS * Cfg::SF_SLOT_BYTES;
    const uint32_t cvec_base = staging_base + Cfg::STAGING_BYTES;
    const uint32_t bar_base = cvec_base + Cfg::CVEC_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };      // leader: both CTAs' code bytes landed AND scales copied
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };           // each CTA: stage may be refilled
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + NUM_ACC + a); };
    constexpr int kSfBar0 = 2 * STAGES + 2 * NUM_ACC;
    auto sf_full_bar = [&](int g) { return bar_base + 8u * (kSfBar0 + g); };        // leader: both CTAs' scale bytes landed
    auto sf_empty_bar = [&](int g) { return bar_base + 8u * (kSfBar0 + Cfg::SF_SLOTS + g); };   // each CTA: slot may be refilled
    const uint32_t tmem_slot = bar_base + 8u * (kSfBar0 + 2 * Cfg::SF_SLOTS);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const bool leader = rank == 0;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_a); prefetch_tmap(&tm_b); prefetch_tmap(&tm_sfa); prefetch_tmap(&tm_sfb); prefetch_tmap(&tm_out);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }   // producer's expect_tx + copier's commit
        for (int g = 0; g < Cfg::SF_SLOTS; ++g) { mbar_init(sf_full_bar(g), 1); mbar_init(sf_empty_bar(g), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }   // 4 epilogue warps x 2 CTAs
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS); tmem_relinquish_pair(); }
    tc_fence_before();
    cluster_sync_all();                                 // both CTAs' barriers and tensor memory exist from here on
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    grid_dependency_wait();            // set-up above may have overlapped the previous kernel; its results are needed from here on
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int pair = (int)cluster_id_x(), num_pairs = (int)num_clusters_x();
    constexpr uint16_t kBoth = 3, kLeader = 1;

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ code producer (both CTAs)
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                const int m0 = (tile % p.m_tiles) * 256 + (int)rank * Cfg::BLOCK_M, n0 = (tile / p.m_tiles) * BLOCK_N;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    if (leader) mbar_expect_tx(full_bar(s), 2 * Cfg::STAGE_BYTES);
                    const uint32_t bar = mapa_shared(full_bar(s), 0), st = smem_base + s * Cfg::STAGE_BYTES;
                    tma_load_2d_pair(st, &tm_a, kb * 128, m0, bar);
                    tma_load_2d_pair(st + Cfg::A_BYTES, &tm_b, kb * 128, n0 + (int)rank * Cfg::HALF_N, bar);
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
                const int m_rt = ((tile % p.m_tiles) * 256 + (int)rank * Cfg::BLOCK_M) >> 7, n_rt = ((tile / p.m_tiles) * BLOCK_N) >> 7;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(sf_empty_bar(g), gph ^ 1u, p.status))) break;
                    if (leader) mbar_expect_tx(sf_full_bar(g), 2 * Cfg::SF_SLOT_BYTES);
                    const uint32_t bar = mapa_shared(sf_full_bar(g), 0), slot = sf_base + g * Cfg::SF_SLOT_BYTES;
                    // coordinates: (word in tile, scale k-tile, 128-row tile); tiles outside the buffer read as zero
                    tma_load_3d_pair(slot, &tm_sfa, 0, kb * Cfg::SF_KT, m_rt, bar);
                    tma_load_3d_pair(slot + Cfg::SFA_BYTES, &tm_sfb, 0, kb * Cfg::SF_KT, n_rt, bar);
                    if (++g == Cfg::SF_SLOTS) { g = 0; gph ^= 1u; }
                }
            }
        }
    } else if (warp_idx == 2) {
        // ------------------------------------------------------------------ scale copies (leader CTA only)
        // The whole warp runs the loop so that addresses and counters stay warp-uniform (the tcgen05 instructions
        // take uniform operands); one elected lane issues.
        if (leader) {
            const bool issuer = elect_one();
            const uint32_t sf_lo0 = desc_lo(sf_base), sf_t0 = tmem_base + Cfg::ACC_COLS;
            int tiles_mine = 0;
            for (int tile = pair; tile < num_tiles; tile += num_pairs) ++tiles_mine;
            long long left = (long long)tiles_mine * p.num_kb;
            uint32_t g = 0, gph = 0, sf_lo = sf_lo0, round_ph = 0;
            while (left > 0) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s) {                   // s is a constant in each unrolled copy
                    mbar_wait_or_flag(sf_full_bar(g), gph, p.status);
                    mbar_wait_or_flag(empty_bar(s), round_ph ^ 1u, p.status);   // the stage's previous MMAs have read its scale buffer
                    tc_fence_after();
                    if (issuer) {
                    const uint32_t sfa_t = sf_t0 + s * Cfg::SF_COLS, sfb_t = sfa_t + Cfg::SF_KT * 4;
                    const uint32_t sfb_lo = sf_lo + (Cfg::SFA_BYTES >> 4);
#pragma unroll
                    for (int kt = 0; kt < Cfg::SF_KT; ++kt) {
                        tc_cp_scale_pair_lean(sfa_t + kt * 4, sf_lo + kt * 32);
#pragma unroll
                        for (int r = 0; r < Cfg::NB_RT; ++r)
                            tc_cp_scale_pair_lean(sfb_t + kt * Cfg::NB_RT * 4 + r * 4, sfb_lo + (r * Cfg::SF_KT + kt) * 32);
                    }
                    tc_commit_pair(full_bar(s), kLeader);         // second arrival: the scales are in tensor memory ...
                    tc_commit_pair(sf_empty_bar(g), kBoth);       // ... and both CTAs' slots have been read
                    }
                    __syncwarp();
                    if (++g == Cfg::SF_SLOTS) { g = 0; gph ^= 1u; sf_lo = sf_lo0; } else sf_lo += Cfg::SF_SLOT_BYTES >> 4;
                    if (--left == 0) break;
                }
                round_ph ^= 1u;
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue (leader CTA only)
        if (leader) {                                    // whole warp, one elected lane issues (see the scale-copy warp)
            const bool issuer = elect_one();
            constexpr uint32_t kIdesc = make_idesc_block_scaled(2 * Cfg::BLOCK_M, BLOCK_N, FMT == FMT_FP4 ? 1u : 0u);
            constexpr uint32_t kId2 = kIdesc | (2u << 4) | (2u << 29);
            // every operand of every MMA of a round, computed once
            uint32_t a_lo[STAGES][4], b_lo[STAGES][4], sfa_t[STAGES][Cfg::SF_KT], sfb_t[STAGES][Cfg::SF_KT], full_addr[STAGES], empty_addr[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                full_addr[s] = full_bar(s); empty_addr[s] = empty_bar(s);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a_lo[s][j] = desc_lo(smem_base) + s * (Cfg::STAGE_BYTES >> 4) + 2 * j;
                    b_lo[s][j] = a_lo[s][j] + (Cfg::A_BYTES >> 4);
                }
#pragma unroll
                for (int kt = 0; kt < Cfg::SF_KT; ++kt) {
                    sfa_t[s][kt] = tmem_base + Cfg::ACC_COLS + s * Cfg::SF_COLS + kt * 4;
                    sfb_t[s][kt] = tmem_base + Cfg::ACC_COLS + s * Cfg::SF_COLS + Cfg::SF_KT * 4 + kt * Cfg::NB_RT * 4;
                }
            }
            uint32_t round_ph = 0, tile_count = 0, d_tmem = 0, sfb_col = 0, acc = 0;
            int tile = pair, kb = 0;
            bool more = tile < num_tiles;
            while (more) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s) {                   // s is a constant in each unrolled copy
                    if (kb == 0) {
                        acc = tile_count & 1u;
                        mbar_wait_or_flag(tempty_bar(acc), ((tile_count >> 1) & 1u) ^ 1u, p.status);
                        d_tmem = tmem_base + acc * BLOCK_N;
                        sfb_col = (uint32_t)(((tile / p.m_tiles) * BLOCK_N) & 127) >> 5;
                    }
                    mbar_wait_or_flag(full_addr[s], round_ph, p.status);
                    tc_fence_after();
                    if (issuer) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {     // four MMAs, each 32 bytes of K per row
                        const int kt = FMT == FMT_FP4 ? (j >> 1) : 0;
                        const uint32_t idesc = FMT == FMT_FP4 ? ((j & 1) ? kId2 : kIdesc) : (kIdesc | ((uint32_t)j << 4) | ((uint32_t)j << 29));
                        const uint32_t accum = j == 0 ? (uint32_t)(kb != 0) : 1u;
                        if (FMT == FMT_FP4) mma_mxf4_pair_lean(d_tmem, a_lo[s][j], b_lo[s][j], idesc, sfa_t[s][kt], sfb_t[s][kt] + sfb_col, accum);
                        else mma_mxf8_pair_lean(d_tmem, a_lo[s][j], b_lo[s][j], idesc, sfa_t[s][kt], sfb_t[s][kt] + sfb_col, accum);
                    }
                    tc_commit_pair(empty_addr[s], kBoth);          // frees the stage and its scale buffer, in both CTAs
                    }
                    __syncwarp();
                    if (++kb == p.num_kb) {
                        if (issuer) tc_commit_pair(tfull_bar(acc), kBoth);
                        __syncwarp();
                        kb = 0; ++tile_count; tile += num_pairs;
                        if (tile >= num_tiles) { more = false; break; }
                    }
                }
                round_ph ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 4..7, both CTAs)
        const int q = warp_idx & 3;                     // tensor-memory lane quarter this warp may read
        const uint32_t stg0 = staging_base + (uint32_t)(warp_idx - 4) * STG_BUFS * 4096u;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t cvec = cvec_base + (uint32_t)(warp_idx - 4) * (BLOCK_N * 4);
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
                const float4 v = make_float4(__uint_as_float(r[4 * t]) + cv[0], __uint_as_float(r[4 * t + 1]) + cv[1],
                                             __uint_as_float(r[4 * t + 2]) + cv[2], __uint_as_float(r[4 * t + 3]) + cv[3]);
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
            const int m0 = (tile % p.m_tiles) * 256 + (int)rank * Cfg::BLOCK_M, n0 = (tile / p.m_tiles) * BLOCK_N;
            const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
            // the tile's values of c into this warp's shared-memory copy while the MMAs still run (a lane brings eight of them);
            // the previous tile's last reads of the copy lie before the __syncwarp of its last chunk
            tile_n0 = n0;
            if (lane * 8 < BLOCK_N) {
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
            }
            __syncwarp();
            ok = mbar_wait(tfull_bar(acc), acc_ph, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            // The accumulator leaves in batches of three 32-column loads issued together: a tcgen05.ld takes far longer
            // while MMAs run (about 2000 cycles against 100 on an idle pipe) but several overlap.  After the last batch the
            // buffer goes back to the MMA warp, before this warp's stores.
            const int row0 = m0 + q * 32;
            const uint32_t t0 = lane_base + acc * BLOCK_N;
            constexpr int kBatches = BLOCK_N / 96;
            static_assert(BLOCK_N % 96 == 0, "the epilogue reads the accumulator in batches of 96 columns");
#pragma unroll 1
            for (int bt = 0; bt < kBatches; ++bt) {
                uint32_t r0[32], r1[32], r2[32];
                tc_ld_32x32b_x32(t0 + bt * 96u, r0); tc_ld_32x32b_x32(t0 + bt * 96u + 32u, r1); tc_ld_32x32b_x32(t0 + bt * 96u + 64u, r2);
                tc_wait_ld();
                if (bt == kBatches - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {                              // this warp has drained its quarter of the accumulator
                        if (leader) mbar_arrive(tempty_bar(acc));
                        else mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
                    }
                }
                const int c0 = n0 + bt * 96;
                store_chunk(r0, row0, c0); store_chunk(r1, row0, c0 + 32); store_chunk(r2, row0, c0 + 64);
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
bool mx_gemm_pair_tc_supported(const MxGemmArgs& a) {
    if (a.fmt == FMT_FP4) { if (a.K % 256 != 0) return false; }
    else if (a.fmt == FMT_FP8) { if (a.K % 128 != 0) return false; }
    else return false;
    if (a.M <= 128) return false;                      // one CTA covers 128 rows: a pair would idle its second half
    if (a.M > (1ll << 30) || a.N > (1ll << 30) || a.K > (1ll << 30)) return false;
    return a.K > 0;
}

template <int FMT, int BLOCK_N>
static cudaError_t launch_pair_variant(const MxGemmArgs& a, cudaStream_t st) {
    using Cfg = MxGemmPairCfg<FMT, BLOCK_N>;
    const int64_t k_bytes = a.fmt == FMT_FP4 ? a.K / 2 : a.K;
    const uint64_t kt_total = (uint64_t)sf_k_tiles(a.K);
    CUtensorMap tm_a, tm_b, tm_sfa, tm_sfb, tm_out;
    if (!make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)k_bytes, (uint64_t)a.M, (uint64_t)k_bytes, 128, Cfg::BLOCK_M) ||
        !make_tensor_map_2d(&tm_b, a.w_codes, 0, (uint64_t)k_bytes, (uint64_t)a.N, (uint64_t)k_bytes, 128, Cfg::HALF_N) ||
        !make_tensor_map_scale_tiles(&tm_sfa, a.a_scales, kt_total, (uint64_t)((a.M + 127) / 128), Cfg::SF_KT, 1) ||
        !make_tensor_map_scale_tiles(&tm_sfb, a.w_scales, kt_total, (uint64_t)((a.N + 127) / 128), Cfg::SF_KT, Cfg::NB_RT) ||
        !make_tensor_map_2d(&tm_out, a.out, 2, (uint64_t)a.N, (uint64_t)a.M, (uint64_t)a.ldo * 4, 32, 32))
        return cudaErrorInvalidValue;
    MxGemmPairParams p;
    p.c = a.c;
    p.M = (int)a.M; p.N = (int)a.N; p.num_kb = (int)(k_bytes / 128);
    p.m_tiles = (int)((a.M + 255) / 256);
    p.n_tiles = (int)((a.N + BLOCK_N - 1) / BLOCK_N);
    p.status = a.status;
    auto kern = mx_gemm_pair_tc_kernel<FMT, BLOCK_N>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int pairs = resident_cta_pairs((const void*)kern, kPairThreads, Cfg::SMEM_BYTES);
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    const unsigned grid = 2u * (unsigned)(tiles < pairs ? tiles : pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kPairThreads); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_sfa, tm_sfb, tm_out, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mx_gemm_pair_tc(const MxGemmArgs& a, cudaStream_t st) {
    return a.fmt == FMT_FP4 ? launch_pair_variant<FMT_FP4, 192>(a, st) : launch_pair_variant<FMT_FP8, 192>(a, st);
}

}  // namespace latmix
