// Block-scaled MX GEMM on the 5th-generation tensor cores:  out[M x N] = dq(Qa) dq(Qw)^T + c.
//
// Both operands are K-major code matrices (MXFP4: two E2M1 codes per byte; MXFP8: one E4M3 byte) with one
// E8M0 scale per 32 elements in the 128-row x 4-block tile layout.  One persistent CTA per SM walks over
// 128 x BLOCK_N output tiles:
//   warp 0    producer: TMA loads of the code tiles (128-byte swizzle) and bulk copies of the scale tiles
//   warp 1    tcgen05.cp of the scales into tensor memory, then tcgen05.mma kind::mxf4 / kind::mxf8f6f4
//             .block_scale with the fp32 accumulator in tensor memory (NUM_ACC accumulators, so the epilogue
//             of one tile overlaps the main loop of the next)
//   warps 2-5 epilogue: tcgen05.ld, + c[n], swizzled staging in shared memory, TMA store of 32 x 32 boxes
// Products of element values and power-of-two scales are exact; accumulation is the tensor core's fp32.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

template <int FMT, int BLOCK_N_, int NUM_ACC_, int STG_BUFS_>
struct MxGemmCfg {
    static constexpr int BLOCK_M = 128, BLOCK_N = BLOCK_N_, NUM_ACC = NUM_ACC_, STG_BUFS = STG_BUFS_;
    static constexpr int SF_KT = FMT == FMT_FP4 ? 2 : 1;          // scale k-tiles (4 blocks each) per 128-byte K slab
    // 128-row scale tiles a B tile can touch: a tile starts at a multiple of BLOCK_N, i.e. at most
    // 128 - gcd(BLOCK_N, 128) rows into a scale tile
    static constexpr int N_LOWBIT = BLOCK_N & -BLOCK_N;
    static constexpr int MAX_ROW_OFFSET = N_LOWBIT >= 128 ? 0 : 128 - N_LOWBIT;
    static constexpr int NB_RT = (MAX_ROW_OFFSET + BLOCK_N + 127) / 128;
    static constexpr int A_BYTES = BLOCK_M * 128, B_BYTES = BLOCK_N * 128;
    static constexpr int SFA_BYTES = SF_KT * 512, SFB_BYTES = NB_RT * SF_KT * 512;
    static constexpr int STAGE_BYTES = (A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES + 1023) / 1024 * 1024;
    static constexpr int STAGING_BYTES = 4 * STG_BUFS * 4096;     // per epilogue warp: 32 rows x 128 bytes
    static constexpr int BAR_BYTES = 1024;
    static constexpr int SMEM_LIMIT = 227 * 1024;
    static constexpr int STAGES_RAW = (SMEM_LIMIT - 1024 - BAR_BYTES - STAGING_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES;
    static constexpr int ACC_COLS = NUM_ACC * BLOCK_N;
    static constexpr int SF_COLS = SF_KT * 4 + SF_KT * NB_RT * 4;  // per buffer; two buffers alternate by k-slab
    static constexpr int TMEM_COLS = 512;
    static_assert(ACC_COLS + 2 * SF_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert(STAGES >= 2, "shared memory budget");
    // A tile's first scale column inside a 128-row scale tile is (n0 % 128) / 32; the block-scaled MMA takes
    // only even column offsets there (an odd one raised a misaligned-address fault), so n0 must be a multiple of 64.
    static_assert(BLOCK_N % 64 == 0 && BLOCK_N <= 256, "tile shape");
};

struct MxGemmParams {
    const uint8_t* a_scales; const uint8_t* w_scales; const float* c;
    int M, N, num_kb, sf_kt_total, m_tiles, n_tiles, n_rt_total;
    uint32_t* status; uint32_t flags;
};

template <int FMT, int BLOCK_N, int NUM_ACC, int STG_BUFS>
__global__ void __launch_bounds__(192, 1)
mx_gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_out, const MxGemmParams p) {
    using Cfg = MxGemmCfg<FMT, BLOCK_N, NUM_ACC, STG_BUFS>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base + STAGES * Cfg::STAGE_BYTES;
    const uint32_t bar_base = staging_base + Cfg::STAGING_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + NUM_ACC + a); };
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 2 * NUM_ACC);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));   // generic pointer to the aligned base

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_a); prefetch_tmap(&tm_b); prefetch_tmap(&tm_out);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc(tmem_slot, Cfg::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    const int num_tiles = p.m_tiles * p.n_tiles;

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_tile = tile % p.m_tiles, n_tile = tile / p.m_tiles;
                const int m0 = m_tile * Cfg::BLOCK_M, n0 = n_tile * BLOCK_N, rt0 = n0 >> 7;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    // failure-path test: the first CTA never arms and never loads the second K slab of its first tile, so
                    // the waits that depend on it run out while nothing of that slab is in flight
                    if ((p.flags & LATMIX_FLAG_TEST_DROP_LOAD) && tile == 0 && kb == 1) continue;
                    const uint32_t st = smem_base + s * Cfg::STAGE_BYTES;
                    int valid_rt = 0;
#pragma unroll
                    for (int r = 0; r < Cfg::NB_RT; ++r) valid_rt += (rt0 + r < p.n_rt_total);
                    mbar_expect_tx(full_bar(s), Cfg::A_BYTES + Cfg::B_BYTES + Cfg::SFA_BYTES + valid_rt * Cfg::SF_KT * 512);
                    tma_load_2d(st, &tm_a, kb * 128, m0, full_bar(s));
                    tma_load_2d(st + Cfg::A_BYTES, &tm_b, kb * 128, n0, full_bar(s));
                    bulk_load(st + Cfg::A_BYTES + Cfg::B_BYTES,
                              p.a_scales + ((size_t)m_tile * p.sf_kt_total + (size_t)kb * Cfg::SF_KT) * 512, Cfg::SFA_BYTES, full_bar(s));
#pragma unroll
                    for (int r = 0; r < Cfg::NB_RT; ++r)
                        if (rt0 + r < p.n_rt_total)
                            bulk_load(st + Cfg::A_BYTES + Cfg::B_BYTES + Cfg::SFA_BYTES + r * Cfg::SF_KT * 512,
                                      p.w_scales + ((size_t)(rt0 + r) * p.sf_kt_total + (size_t)kb * Cfg::SF_KT) * 512,
                                      Cfg::SF_KT * 512, full_bar(s));
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            constexpr uint32_t kIdesc = make_idesc_block_scaled(Cfg::BLOCK_M, BLOCK_N, FMT == FMT_FP4 ? 1u : 0u);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_count) {
                const int n0 = (tile / p.m_tiles) * BLOCK_N;
                const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
                if (!(ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, p.status))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(full_bar(s), ph, p.status))) break;
                    tc_fence_after();
                    const uint32_t st = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sfa_s = st + Cfg::A_BYTES + Cfg::B_BYTES, sfb_s = sfa_s + Cfg::SFA_BYTES;
                    const uint32_t sfa_t = tmem_base + Cfg::ACC_COLS + (it & 1u) * Cfg::SF_COLS;
                    const uint32_t sfb_t = sfa_t + Cfg::SF_KT * 4;
#pragma unroll
                    for (int kt = 0; kt < Cfg::SF_KT; ++kt) {
                        tc_cp_32x128b_warpx4(sfa_t + kt * 4, make_smem_desc(sfa_s + kt * 512, 0, 128, kSwizzleNone));
#pragma unroll
                        for (int r = 0; r < Cfg::NB_RT; ++r)
                            tc_cp_32x128b_warpx4(sfb_t + kt * Cfg::NB_RT * 4 + r * 4,
                                                 make_smem_desc(sfb_s + (r * Cfg::SF_KT + kt) * 512, 0, 128, kSwizzleNone));
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {     // four MMAs, each 32 bytes of K per row
                        const uint64_t a_desc = make_smem_desc(st + j * 32, 0, 1024, kSwizzle128B);
                        const uint64_t b_desc = make_smem_desc(st + Cfg::A_BYTES + j * 32, 0, 1024, kSwizzle128B);
                        const int kt = FMT == FMT_FP4 ? (j >> 1) : 0;
                        const uint32_t sf_id = FMT == FMT_FP4 ? (uint32_t)(j & 1) * 2u : (uint32_t)j;
                        const uint32_t idesc = idesc_with_sf_ids(kIdesc, sf_id, sf_id);
                        const uint32_t sfa = sfa_t + kt * 4;
                        const uint32_t sfb = sfb_t + kt * Cfg::NB_RT * 4 + ((n0 & 127) >> 5);
                        if (FMT == FMT_FP4) mma_mxf4(d_tmem, a_desc, b_desc, idesc, sfa, sfb, (kb | j) != 0);
                        else mma_mxf8(d_tmem, a_desc, b_desc, idesc, sfa, sfb, (kb | j) != 0);
                    }
                    tc_commit(empty_bar(s));
                }
                if (ok) tc_commit(tfull_bar(acc));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp_idx & 3;                     // tensor-memory lane quarter this warp may read
        const uint32_t stg0 = staging_base + (uint32_t)(warp_idx - 2) * STG_BUFS * 4096u;
        uint32_t tile_count = 0, stg_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_count) {
            const int m0 = (tile % p.m_tiles) * Cfg::BLOCK_M, n0 = (tile / p.m_tiles) * BLOCK_N;
            const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
            ok = mbar_wait(tfull_bar(acc), acc_ph, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int chunk = 0; chunk < BLOCK_N / 32; ++chunk, ++stg_it) {
                uint32_t r[32];
                tc_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BLOCK_N + chunk * 32, r);
                tc_wait_ld();
                const int col0 = n0 + chunk * 32;
                const uint32_t stg = stg0 + (stg_it % STG_BUFS) * 4096u;
                if (lane == 0) bulk_wait_read<STG_BUFS - 1>();   // the store that last used this buffer has read it
                __syncwarp();
                float cv[32];
                if (p.c != nullptr && col0 + 32 <= p.N) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 t = __ldg(reinterpret_cast<const float4*>(p.c + col0) + j);
                        cv[4 * j] = t.x; cv[4 * j + 1] = t.y; cv[4 * j + 2] = t.z; cv[4 * j + 3] = t.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) cv[i] = (p.c != nullptr && col0 + i < p.N) ? p.c[col0 + i] : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {                     // 128-byte swizzle: chunk j of row `lane` -> j ^ (lane & 7)
                    const float4 v = make_float4(__uint_as_float(r[4 * j]) + cv[4 * j], __uint_as_float(r[4 * j + 1]) + cv[4 * j + 1],
                                                 __uint_as_float(r[4 * j + 2]) + cv[4 * j + 2], __uint_as_float(r[4 * j + 3]) + cv[4 * j + 3]);
                    const uint32_t dst = stg + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) * 16);
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && col0 < p.N && m0 + q * 32 < p.M) {
                    tma_store_2d(&tm_out, stg, col0, m0 + q * 32);
                    bulk_commit();
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(acc));
        }
        if (lane == 0) bulk_wait<0>();
    }
    // teardown: if any wait gave up, let copies still in flight land before shared memory goes away
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

// ----------------------------------------------------------------------------------------------------
bool mx_gemm_tc_supported(const MxGemmArgs& a) {
    if (a.fmt == FMT_FP4) { if (a.K % 256 != 0) return false; }
    else if (a.fmt == FMT_FP8) { if (a.K % 128 != 0) return false; }
    else return false;
    if (a.M > (1ll << 30) || a.N > (1ll << 30) || a.K > (1ll << 30)) return false;
    return a.K > 0;
}

template <int FMT, int BLOCK_N, int NUM_ACC, int STG_BUFS>
static cudaError_t launch_variant(const MxGemmArgs& a, cudaStream_t st) {
    using Cfg = MxGemmCfg<FMT, BLOCK_N, NUM_ACC, STG_BUFS>;
    const int64_t k_bytes = a.fmt == FMT_FP4 ? a.K / 2 : a.K;
    CUtensorMap tm_a, tm_b, tm_out;
    if (!make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)k_bytes, (uint64_t)a.M, (uint64_t)k_bytes, 128, Cfg::BLOCK_M) ||
        !make_tensor_map_2d(&tm_b, a.w_codes, 0, (uint64_t)k_bytes, (uint64_t)a.N, (uint64_t)k_bytes, 128, BLOCK_N) ||
        !make_tensor_map_2d(&tm_out, a.out, 2, (uint64_t)a.N, (uint64_t)a.M, (uint64_t)a.ldo * 4, 32, 32))
        return cudaErrorInvalidValue;
    MxGemmParams p;
    p.a_scales = a.a_scales; p.w_scales = a.w_scales; p.c = a.c;
    p.M = (int)a.M; p.N = (int)a.N; p.num_kb = (int)(k_bytes / 128);
    p.sf_kt_total = (int)sf_k_tiles(a.K);
    p.m_tiles = (int)((a.M + Cfg::BLOCK_M - 1) / Cfg::BLOCK_M);
    p.n_tiles = (int)((a.N + BLOCK_N - 1) / BLOCK_N);
    p.n_rt_total = (int)((a.N + 127) / 128);
    p.status = a.status; p.flags = a.flags;
    auto kern = mx_gemm_tc_kernel<FMT, BLOCK_N, NUM_ACC, STG_BUFS>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    kern<<<grid, 192, Cfg::SMEM_BYTES, st>>>(tm_a, tm_b, tm_out, p);
    count_launch();
    return cudaGetLastError();
}

template <int FMT>
static cudaError_t launch_fmt(const MxGemmArgs& a, cudaStream_t st) {
    const uint32_t variant = (a.flags >> 8) & 0xFu;     // tuning override: 1 = 128x128 (2 acc), 2 = 128x192 (2 acc), 3 = 128x256 (1 acc)
    if (variant == 1) return launch_variant<FMT, 128, 2, 2>(a, st);
    if (variant == 3) return launch_variant<FMT, 256, 1, 1>(a, st);
    if (variant == 2) return launch_variant<FMT, 192, 2, 2>(a, st);
    // One row tile only (decode and small batches): the weights are streamed once whatever the tile width, so take
    // narrow tiles to spread them over more SMs.
    if (a.M <= 128) return launch_variant<FMT, 128, 2, 2>(a, st);
    return launch_variant<FMT, 192, 2, 2>(a, st);
}

cudaError_t launch_mx_gemm_tc(const MxGemmArgs& a, cudaStream_t st) {
    return a.fmt == FMT_FP4 ? launch_fmt<FMT_FP4>(a, st) : launch_fmt<FMT_FP8>(a, st);
}

}  // namespace latmix
