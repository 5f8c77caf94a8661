// Fused online affine transform + MX quantisation on the tensor cores:  codes, scales = Q(X A + 1 b^T).
//
// X (M x K, bf16, row-major) is the K-major A operand; the transform matrix A (K x K, bf16, row-major,
// element [k][j]) is consumed as it is stored, as an MN-major B operand, so no transposed copy is needed.
// One persistent CTA per SM walks over 128 x 256 tiles of Y = X A:
//   warp 0    producer: TMA loads (128-byte swizzle) of a 128 x 64 slab of X and four 64 x 64 boxes of A
//   warp 1    tcgen05.mma kind::f16 (bf16 x bf16 -> fp32) into one of two 256-column accumulators in
//             tensor memory, so the quantising epilogue of a tile overlaps the products of the next
//   warps 2-5 epilogue: with the 32x32b tensor-memory load one thread owns one row and 32 consecutive
//             columns, i.e. exactly one MX block: add b, block maximum, E8M0 exponent, exact power-of-two
//             scaling, round-to-nearest-even conversion, packed store -- no cross-lane traffic.
// The fp32 accumulator is quantised directly (Y never exists in memory unless a dump is requested).
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace tq {
constexpr int BLOCK_M = 128, BLOCK_N = 256, BLOCK_K = 64;       // BLOCK_K bf16 = 128 bytes = one swizzle row
constexpr int A_BYTES = BLOCK_M * 128;                          // X slab
constexpr int B_BOX_BYTES = BLOCK_K * 128;                      // one 64(k) x 64(n) box of the transform matrix
constexpr int B_BYTES = (BLOCK_N / 64) * B_BOX_BYTES;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;                  // 48 KiB
constexpr int STAGES = 4;
constexpr int NUM_ACC = 2;
constexpr int BAR_BYTES = 1024;
constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + BAR_BYTES;
constexpr int TMEM_COLS = 512;
}  // namespace tq

struct TransformQuantParams {
    const float* b;
    uint8_t* codes; uint8_t* scales; float* Y_dump;
    int M, K, num_kb, m_tiles, n_tiles, sf_layout, sf_kt_total;
    uint32_t* status; uint32_t flags;
};

template <int FMT>
__global__ void __launch_bounds__(192, 1)
transform_quant_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_a,
                          const TransformQuantParams p) {
    using namespace tq;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + NUM_ACC + a); };
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 2 * NUM_ACC);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_a);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    const int num_tiles = p.m_tiles * p.n_tiles;

    if (warp_idx == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile / p.n_tiles) * BLOCK_M, n0 = (tile % p.n_tiles) * BLOCK_N;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    mbar_expect_tx(full_bar(s), STAGE_BYTES);
                    tma_load_2d(st, &tm_x, kb * BLOCK_K, m0, full_bar(s));
#pragma unroll
                    for (int j = 0; j < BLOCK_N / 64; ++j)      // box: 64 columns (n) x 64 rows (k) of the transform matrix
                        tma_load_2d(st + A_BYTES + j * B_BOX_BYTES, &tm_a, n0 + j * 64, kb * BLOCK_K, full_bar(s));
                }
            }
        }
    } else if (warp_idx == 1) {
        if (lane == 0) {
            constexpr uint32_t kIdesc = make_idesc_bf16(BLOCK_M, BLOCK_N, 0, 1);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_count) {
                const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
                if (!(ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, p.status))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(full_bar(s), ph, p.status))) break;
                    tc_fence_after();
                    const uint32_t st = smem_base + s * STAGE_BYTES;
#pragma unroll
                    for (int j = 0; j < BLOCK_K / 16; ++j) {   // K = 16 per instruction
                        // X slab, K-major: 32 bytes further along each 128-byte row
                        const uint64_t a_desc = make_smem_desc(st + j * 32, 0, 1024, kSwizzle128B);
                        // transform matrix, MN-major: 16 k-rows (2 groups of 8 rows = 2 x 1024 bytes) further down;
                        // leading offset = distance between 64-column boxes, stride offset = 8-row group pitch
                        const uint64_t b_desc = make_smem_desc(st + A_BYTES + j * 2048, B_BOX_BYTES, 1024, kSwizzle128B);
                        mma_bf16(d_tmem, a_desc, b_desc, kIdesc, (kb | j) != 0);
                    }
                    tc_commit(empty_bar(s));
                }
                if (ok) tc_commit(tfull_bar(acc));
            }
        }
    } else {
        const int q = warp_idx & 3;
        constexpr int kRMax = FormatTraits<FMT>::kRMax;
        uint32_t tile_count = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_count) {
            const int m0 = (tile / p.n_tiles) * BLOCK_M, n0 = (tile % p.n_tiles) * BLOCK_N;
            const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
            ok = mbar_wait(tfull_bar(acc), acc_ph, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int64_t row = m0 + q * 32 + lane;
            const bool row_ok = row < p.M;
            uint32_t sf_word = 0;
#pragma unroll 1
            for (int chunk = 0; chunk < BLOCK_N / 32; ++chunk) {
                uint32_t r[32];
                tc_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BLOCK_N + chunk * 32, r);
                tc_wait_ld();
                const int col0 = n0 + chunk * 32;
                const bool blk_ok = row_ok && col0 < p.K;        // K is a multiple of 32: whole blocks only
                float v[32];
                float amax = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p.b != nullptr && col0 < p.K) bb = __ldg(reinterpret_cast<const float4*>(p.b + col0) + j);
                    v[4 * j] = __uint_as_float(r[4 * j]) + bb.x;
                    v[4 * j + 1] = __uint_as_float(r[4 * j + 1]) + bb.y;
                    v[4 * j + 2] = __uint_as_float(r[4 * j + 2]) + bb.z;
                    v[4 * j + 3] = __uint_as_float(r[4 * j + 3]) + bb.w;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(v[i]));
                if (p.Y_dump != nullptr && blk_ok) {
                    float4* d = reinterpret_cast<float4*>(p.Y_dump + row * p.K + col0);
#pragma unroll
                    for (int j = 0; j < 8; ++j) d[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                }
                if ((p.flags & LATMIX_FLAG_CHECK_FINITE) && blk_ok && !isfinite(amax)) atomicOr(p.status, 1u << LATMIX_ERR_NONFINITE);
                const uint32_t sb = scale_byte_from_amax(amax, kRMax);
                const float2 f = inv_scale_factors(sb);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = (v[i] * f.x) * f.y;
                if (blk_ok) {
                    if (FMT == FMT_FP4) {
                        uint4 w = make_uint4(pack8_fp4(v), pack8_fp4(v + 8), pack8_fp4(v + 16), pack8_fp4(v + 24));
                        *reinterpret_cast<uint4*>(p.codes + row * (p.K >> 1) + (col0 >> 1)) = w;
                    } else {
                        uint2 w0, w1, w2, w3;
                        w0 = pack8_bytes<FMT>(v); w1 = pack8_bytes<FMT>(v + 8); w2 = pack8_bytes<FMT>(v + 16); w3 = pack8_bytes<FMT>(v + 24);
                        uint4* d = reinterpret_cast<uint4*>(p.codes + row * (int64_t)p.K + col0);
                        d[0] = make_uint4(w0.x, w0.y, w1.x, w1.y);
                        d[1] = make_uint4(w2.x, w2.y, w3.x, w3.y);
                    }
                    const int64_t kb = col0 >> 5;
                    if (p.sf_layout == LATMIX_SF_LINEAR) {
                        p.scales[row * (p.K >> 5) + kb] = (uint8_t)sb;
                    } else {
                        // four consecutive blocks of a row share one aligned 32-bit word of the tile layout
                        sf_word |= sb << (8 * (chunk & 3));
                        if ((chunk & 3) == 3 || col0 + 32 >= p.K)
                            *reinterpret_cast<uint32_t*>(p.scales + sf_tcgen05_offset(row, kb & ~3ll, p.sf_kt_total)) = sf_word;
                    }
                }
                if ((chunk & 3) == 3) sf_word = 0;
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(acc));
        }
    }
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) tmem_dealloc(tmem_base, tq::TMEM_COLS);
}

bool transform_quant_tc_supported(const TransformQuantArgs& a) {
    return a.K > 0 && a.K % 32 == 0 && a.M > 0 && a.M < (1ll << 30) && a.K < (1ll << 30);
}

cudaError_t launch_transform_quant_tc(const TransformQuantArgs& a, cudaStream_t st) {
    using namespace tq;
    CUtensorMap tm_x, tm_a;
    if (!make_tensor_map_2d(&tm_x, a.X, 1, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K * 2, BLOCK_K, BLOCK_M) ||
        !make_tensor_map_2d(&tm_a, a.A, 1, (uint64_t)a.K, (uint64_t)a.K, (uint64_t)a.K * 2, 64, BLOCK_K))
        return cudaErrorInvalidValue;
    TransformQuantParams p;
    p.b = a.b; p.codes = a.codes; p.scales = a.scales; p.Y_dump = a.Y_dump;
    p.M = (int)a.M; p.K = (int)a.K;
    p.num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);
    p.m_tiles = (int)((a.M + BLOCK_M - 1) / BLOCK_M);
    p.n_tiles = (int)((a.K + BLOCK_N - 1) / BLOCK_N);
    p.sf_layout = a.sf_layout; p.sf_kt_total = (int)sf_k_tiles(a.K);
    p.status = a.status; p.flags = a.flags;
    const int sms = sm_count();
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
#define LATMIX_TQ(FMT)                                                                                                 \
    do {                                                                                                               \
        auto kern = transform_quant_tc_kernel<FMT>;                                                                    \
        cudaError_t e = set_max_dynamic_smem((const void*)kern, SMEM_BYTES);           \
        if (e != cudaSuccess) return e;                                                                                \
        kern<<<grid, 192, SMEM_BYTES, st>>>(tm_x, tm_a, p);                                                            \
    } while (0)
    if (a.fmt == FMT_FP4) LATMIX_TQ(FMT_FP4);
    else if (a.fmt == FMT_FP8) LATMIX_TQ(FMT_FP8);
    else if (a.fmt == FMT_INT4) LATMIX_TQ(FMT_INT4);
    else LATMIX_TQ(FMT_INT8);
#undef LATMIX_TQ
    count_launch();
    return cudaGetLastError();
}

}  // namespace latmix
