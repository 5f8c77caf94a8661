// MXINT8 product on the tensor cores:  out[M x N] = dq(Qa) dq(Qw)^T + c.
//
// There is no block-scaled tcgen05 kind for 8-bit integers.  An MXINT8 element is k 2^(E-6) with |k| <= 127: seven
// significant bits times a power of two, which bf16 (eight significant bits, the exponent range of fp32, subnormals
// included) represents exactly.  So both operands are expanded to bf16 in scratch memory (exactly), and the product is
// a plain bf16 x bf16 -> fp32 contraction: products are exact, accumulation is the tensor core's fp32, just as on the
// block-scaled path.  The GEMM uses CTA pairs (tcgen05.mma.cta_group::2 kind::f16, 256 x 256 tiles, two 64-deep K
// slabs per stage, 2 x 256 TMEM columns) and the fp32 TMA-store epilogue of the block-scaled kernels.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

// ---- expansion: int8 codes + E8M0 scales (128-row x 4-block tile layout) -> bf16 ---------------------------------
// A warp walks along a row, 512 codes per step: a lane = 16 codes (one 16-byte load, two 16-byte stores), two lanes =
// one MX block.  Rows are dealt out to the warps; nothing in the loop multiplies or divides addresses.
__global__ void __launch_bounds__(256) mxint8_to_bf16_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                                             int64_t rows, int64_t K, __nv_bfloat16* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t kt = sf_k_tiles(K);
    // scale byte of this lane's block: block index lane / 2 within the step; four blocks per 512-byte tile
    const int sf_lane = (lane >> 3) * 512 + ((lane >> 1) & 3);
    for (int64_t row = warp0; row < rows; row += n_warps) {
        const uint8_t* pc = codes + row * K + lane * 16;
        const uint8_t* ps = scales + ((row >> 7) * kt) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + sf_lane;
        uint4* po = reinterpret_cast<uint4*>(out + row * K + lane * 16);
        constexpr int UNROLL = 4;                             // 64 bytes per lane in flight
        for (int64_t k = lane * 16; k - lane * 16 < K; k += UNROLL * 512, pc += UNROLL * 512, ps += UNROLL * 4 * 512, po += UNROLL * 64) {
            uint4 raw[UNROLL];
            uint32_t sb[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const bool active = k + u * 512 < K;
                raw[u] = active ? __ldg(reinterpret_cast<const uint4*>(pc + u * 512)) : make_uint4(0u, 0u, 0u, 0u);
                sb[u] = active ? __ldg(ps + u * 4 * 512) : 0u;
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (k + u * 512 >= K) break;
                uint4 lo, hi;
                int8x16_to_bf16(raw[u], int8_mult(sb[u]), lo, hi);
                po[u * 64] = lo;
                po[u * 64 + 1] = hi;
            }
        }
    }
}

namespace i8g {
constexpr int BLOCK_M = 128, BLOCK_N = 256, HALF_N = 128, SLAB_K = 64, SLABS = 2;
constexpr int A_BYTES = BLOCK_M * 128, B_BYTES = HALF_N * 128;             // one slab of each operand
constexpr int B_OFFSET = SLABS * A_BYTES;
constexpr int STAGE_BYTES = SLABS * (A_BYTES + B_BYTES);                   // 64 KiB
constexpr int STAGES = 3, NUM_ACC = 2, STG_BUFS = 2;
constexpr int STAGING_BYTES = 4 * STG_BUFS * 4096;
constexpr int BAR_BYTES = 1024;
constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES;
constexpr int TMEM_COLS = 512, THREADS = 6 * 32;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
}  // namespace i8g

struct Bf16GemmPairParams {
    const float* c;
    int M, N, num_kb, m_tiles /* of 256 rows */, n_tiles;
    uint32_t* status;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(i8g::THREADS, 1)
bf16_gemm_pair_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                         const __grid_constant__ CUtensorMap tm_out, const Bf16GemmPairParams p) {
    using namespace i8g;
    extern __shared__ uint8_t smem_raw[];
    // same shared-memory offsets in both CTAs: the MMA's descriptors and the multicast commits rely on that
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base + STAGES * STAGE_BYTES;
    const uint32_t bar_base = staging_base + STAGING_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                   // leader: both CTAs' bytes landed
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };       // each CTA: stage may be refilled
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + NUM_ACC + a); };   // leader: 4 warps x 2 CTAs
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 2 * NUM_ACC);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_a); prefetch_tmap(&tm_b); prefetch_tmap(&tm_out);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int pair = (int)cluster_id_x(), num_pairs = (int)num_clusters_x();
    constexpr uint16_t kBoth = 3;

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                const int row0 = (tile % p.m_tiles) * 256 + (int)rank * BLOCK_M, wrow0 = (tile / p.m_tiles) * BLOCK_N + (int)rank * HALF_N;
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    if (leader) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
                    const uint32_t bar = mapa_shared(full_bar(s), 0), st = smem_base + s * STAGE_BYTES;
#pragma unroll
                    for (int h = 0; h < SLABS; ++h) {               // slabs past the end of K read as zero
                        const int k0 = (kb * SLABS + h) * SLAB_K;
                        tma_load_2d_pair(st + h * A_BYTES, &tm_a, k0, row0, bar);
                        tma_load_2d_pair(st + B_OFFSET + h * B_BYTES, &tm_b, k0, wrow0, bar);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue (leader CTA only)
        // whole warp, one elected lane issues; unrolled over the stages, operands precomputed, one wait and one commit per stage
        if (leader) {
            const bool issuer = elect_one();
            constexpr uint32_t kIdesc = make_idesc_bf16(2 * BLOCK_M, BLOCK_N, 0, 0);      // both operands K-major
            constexpr int MMAS = SLABS * 4;                          // K = 16 per instruction
            uint32_t a_lo[STAGES][MMAS], b_lo[STAGES][MMAS], full_addr[STAGES], empty_addr[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                full_addr[s] = full_bar(s); empty_addr[s] = empty_bar(s);
#pragma unroll
                for (int j = 0; j < MMAS; ++j) {                     // 32 bytes further along each 128-byte row per instruction
                    a_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + (j >> 2) * A_BYTES + (j & 3) * 32);
                    b_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + B_OFFSET + (j >> 2) * B_BYTES + (j & 3) * 32);
                }
            }
            uint32_t round_ph = 0, tile_count = 0, d_tmem = 0, acc = 0;
            int tile = pair, kb = 0;
            bool more = tile < num_tiles;
            while (more) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s) {                   // s is a constant in each unrolled copy
                    if (kb == 0) {
                        acc = tile_count & 1u;
                        mbar_wait_or_flag(tempty_bar(acc), ((tile_count >> 1) & 1u) ^ 1u, p.status);
                        d_tmem = tmem_base + acc * BLOCK_N;
                    }
                    mbar_wait_or_flag(full_addr[s], round_ph, p.status);
                    tc_fence_after();
                    if (issuer) {
#pragma unroll
                        for (int j = 0; j < MMAS; ++j)
                            mma_bf16_pair_lean(d_tmem, a_lo[s][j], b_lo[s][j], kIdesc, j == 0 ? (uint32_t)(kb != 0) : 1u);
                        tc_commit_pair(empty_addr[s], kBoth);
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
        // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int q = warp_idx & 3;                     // tensor-memory lane quarter this warp may read
        const uint32_t stg0 = staging_base + (uint32_t)(warp_idx - 2) * STG_BUFS * 4096u;
        uint32_t tile_count = 0, stg_it = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tile_count) {
            const int m0 = (tile % p.m_tiles) * 256 + (int)rank * BLOCK_M, n0 = (tile / p.m_tiles) * BLOCK_N;
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
            __syncwarp();
            if (lane == 0) {                                      // this warp has drained its quarter of the accumulator
                if (leader) mbar_arrive(tempty_bar(acc));
                else mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
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
    if (warp_idx == 1) tmem_dealloc_pair(tmem_base, TMEM_COLS);
}


// ----------------------------------------------------------------------------------------------------
size_t mxint8_gemm_tc_scratch_bytes(int64_t M, int64_t K, int64_t N) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    return up((size_t)M * (size_t)K * 2) + up((size_t)N * (size_t)K * 2);
}

bool mxint8_gemm_tc_supported(const MxGemmArgs& a) {
    return a.fmt == FMT_INT8 && a.K > 0 && a.K % 32 == 0 && a.M > 0 && a.N > 0 && a.M < (1ll << 30) && a.N < (1ll << 30) &&
           a.K < (1ll << 30);
}

// `scratch` holds mxint8_gemm_tc_scratch_bytes(M, K, N) bytes, 256-byte aligned.
cudaError_t launch_mxint8_gemm_tc(const MxGemmArgs& a, void* scratch, cudaStream_t st) {
    using namespace i8g;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    __nv_bfloat16* a16 = static_cast<__nv_bfloat16*>(scratch);
    __nv_bfloat16* w16 = reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(scratch) + up((size_t)a.M * (size_t)a.K * 2));
    const int sms = sm_count();
    auto blocks = [&](int64_t rows) {                       // a warp per row at a time, at most 8 CTAs of 8 warps per SM
        const int64_t want = (rows + 7) / 8;
        return (unsigned)(want < (int64_t)sms * 8 ? (want > 0 ? want : 1) : (int64_t)sms * 8);
    };
    mxint8_to_bf16_kernel<<<blocks(a.M), 256, 0, st>>>(a.a_codes, a.a_scales, a.M, a.K, a16);
    mxint8_to_bf16_kernel<<<blocks(a.N), 256, 0, st>>>(a.w_codes, a.w_scales, a.N, a.K, w16);
    count_launch(2);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    CUtensorMap tm_a, tm_b, tm_out;
    if (!make_tensor_map_2d(&tm_a, a16, 1, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K * 2, SLAB_K, BLOCK_M) ||
        !make_tensor_map_2d(&tm_b, w16, 1, (uint64_t)a.K, (uint64_t)a.N, (uint64_t)a.K * 2, SLAB_K, HALF_N) ||
        !make_tensor_map_2d(&tm_out, a.out, 2, (uint64_t)a.N, (uint64_t)a.M, (uint64_t)a.ldo * 4, 32, 32))
        return cudaErrorInvalidValue;
    Bf16GemmPairParams p;
    p.c = a.c;
    p.M = (int)a.M; p.N = (int)a.N;
    p.num_kb = (int)((a.K + SLABS * SLAB_K - 1) / (SLABS * SLAB_K));
    p.m_tiles = (int)((a.M + 255) / 256);
    p.n_tiles = (int)((a.N + BLOCK_N - 1) / BLOCK_N);
    p.status = a.status;
    e = set_max_dynamic_smem((const void*)bf16_gemm_pair_tc_kernel, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int pairs = resident_cta_pairs((const void*)bf16_gemm_pair_tc_kernel, THREADS, SMEM_BYTES);
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    const unsigned grid = 2u * (unsigned)(tiles < pairs ? tiles : pairs);
    bf16_gemm_pair_tc_kernel<<<grid, THREADS, SMEM_BYTES, st>>>(tm_a, tm_b, tm_out, p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace latmix
