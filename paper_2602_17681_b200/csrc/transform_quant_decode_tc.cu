// Fused affine transform + MX quantisation for a handful of rows on the tensor cores (M <= 64, K <= 16384):
//   codes, scales = Q(X A + 1 b^T).
//
// With so few rows the call is bound by reading the K x K matrix once.  As in the small-batch GEMM the operands swap roles:
// the MMA's 128 rows are 128 COLUMNS of A (read as stored: an MN-major operand), its N side the 16 or 64 (zero-filled) rows of X,
// so that a ring stage carries 32 KB of A and 4 (16) KB of X in two tiled bulk copies of 8 KB each per 64-deep slab.  K / 128 tiles
// alone would reach too few SMs, hence a cluster of four CTAs shares a tile, each with a quarter of the summation index.
// 4096 x 4096 (33.7 MB, ncu): 11.1 us, of which 6 us are fixed (a 512 x 512 call takes 6.2 us) and the rest streams at the
// DRAM rate; the tiled pair kernel needs 24 us, a CUDA-core-fed mma.sync kernel (one CTA per 32 columns) needed 18 us.
//   warp 0    producer: per stage two 64-deep slabs = four 64 x 64 boxes of A and two 64 x 16 boxes of X
//   warp 1    tcgen05.mma kind::f16 (bf16 x bf16 -> fp32), eight per stage, into a 128-lane x 16-column accumulator
//   warps 2-5 epilogue: tcgen05.ld (a thread = one column k of the result, the rows m along its registers); all-to-all through
//             distributed shared memory: the partial sums of a quarter of the rows go to each CTA of the cluster; cluster barrier;
//             every CTA adds the four partial sums of its rows in rank order, then b, and quantises them: the 32 lanes of
//             a warp are the 32 columns of one MX block.
// Every wait is bounded; all CTAs of a cluster reach the cluster barrier whatever happens.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace tqd2 {
constexpr int BLOCK_K = 128;                       // columns of A (rows of the MMA) per tile
constexpr int SPLIT = 4;                           // CTAs per tile = parts of the summation index
constexpr int SLAB_J = 64;                         // summation indices per slab (128 bytes of X per row)
constexpr int A_BOX_BYTES = SLAB_J * 128;          // 64 rows (j) x 64 columns (k) bf16
constexpr int A_BYTES = 2 * A_BOX_BYTES;
constexpr int SLABS = 2;
constexpr int BAR_BYTES = 256;
constexpr int MAX_K = 16384;                       // tiles x 4 CTAs beyond one wave simply queue (31 us at 8192, 83 us at 14336)
template <int ROWS_>                               // rows of X (N of the MMA): 16 or 64
struct Cfg {
    static constexpr int ROWS = ROWS_;
    static constexpr int X_BYTES = ROWS * 128;
    static constexpr int SLAB_BYTES = A_BYTES + X_BYTES;
    static constexpr int STAGE_BYTES = SLABS * SLAB_BYTES;
    static constexpr int ROWS_PER_RANK = ROWS / SPLIT;                        // rows each CTA of the cluster finishes
    static constexpr int SLOT_BYTES = SPLIT * ROWS_PER_RANK * BLOCK_K * 4;    // partial sums [sender rank][row of mine][k] fp32
    static constexpr int STAGES_RAW = (227 * 1024 - 1024 - SLOT_BYTES - BAR_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 6 ? 6 : STAGES_RAW;
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + SLOT_BYTES + BAR_BYTES;
    static constexpr int TMEM_COLS = ROWS < 32 ? 32 : ROWS;
    static_assert(SLAB_BYTES % 1024 == 0 && STAGES >= 3 && SMEM_BYTES <= 227 * 1024, "shared memory layout");
    static_assert(ROWS % 16 == 0 && ROWS <= 64 && ROWS % SPLIT == 0, "MMA shape; every CTA of the cluster finishes the same number of rows");
};
}  // namespace tqd2

struct TransformQuantDecodeParams {
    const float* b;
    uint8_t* codes; uint8_t* scales; float* Y_dump;
    int M, K, slice;          // slice = summation indices per CTA, a multiple of 64
    int sf_layout;
    uint32_t* status; uint32_t flags;
};

__device__ __forceinline__ void st_shared_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

template <int FMT, int ROWS>
__global__ void __cluster_dims__(tqd2::SPLIT, 1, 1) __launch_bounds__(192, 1)
transform_quant_decode_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_x,
                                 const TransformQuantDecodeParams p) {
    using namespace tqd2;
    using C = Cfg<ROWS>;
    constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, SLAB_BYTES = C::SLAB_BYTES, X_BYTES = C::X_BYTES;
    constexpr int SLOT_BYTES = C::SLOT_BYTES, ROWS_PER_RANK = C::ROWS_PER_RANK, TMEM_COLS = C::TMEM_COLS;
    extern __shared__ uint8_t smem_raw[];
    // same offsets in every CTA of the cluster: the partial sums below are written to the peers at this CTA's own offsets
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t slots_base = smem_base + STAGES * STAGE_BYTES;
    const uint32_t bar_base = slots_base + SLOT_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * STAGES);
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 1);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const float* slots = reinterpret_cast<const float*>(smem_gen + (slots_base - smem_base));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int k0 = (int)cluster_id_x() * BLOCK_K;                 // first column of A of this tile
    const int j_begin = (int)rank * p.slice;
    const int slabs = j_begin >= p.K ? 0 : (min(p.K, j_begin + p.slice) - j_begin + SLAB_J - 1) / SLAB_J;
    const int stages = (slabs + SLABS - 1) / SLABS;

    if (warp_idx == 0 && lane == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    grid_launch_dependents();          // the product kernel that follows may set itself up while this one runs

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < stages && ok; ++it) {
                const int s = it % STAGES;
                if (!(ok = mbar_wait(empty_bar(s), ((it / STAGES) & 1u) ^ 1u, p.status))) break;
                const int n = min(SLABS, slabs - it * SLABS);
                mbar_expect_tx(full_bar(s), (uint32_t)n * (A_BYTES + X_BYTES));
                for (int h = 0; h < n; ++h) {                     // rows of A past K, columns of A and X past K, rows of X past M: zeros
                    const int j0 = j_begin + (it * SLABS + h) * SLAB_J;
                    const uint32_t st = smem_base + s * STAGE_BYTES + h * SLAB_BYTES;
                    tma_load_2d(st, &tm_a, k0, j0, full_bar(s));
                    tma_load_2d(st + A_BOX_BYTES, &tm_a, k0 + 64, j0, full_bar(s));
                    tma_load_2d(st + A_BYTES, &tm_x, j0, 0, full_bar(s));
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0 && stages > 0) {
            // the MMA's "A" operand: 128 columns of A, MN-major (two 64-column boxes, box pitch in the descriptor's leading
            // offset); its "B" operand: the 16 rows of X, K-major
            constexpr uint32_t kIdesc = make_idesc_bf16(BLOCK_K, ROWS, 1, 0);
            bool ok = true;
            for (int it = 0; it < stages && ok; ++it) {
                const int s = it % STAGES;
                if (!(ok = mbar_wait(full_bar(s), (it / STAGES) & 1u, p.status))) break;
                tc_fence_after();
                const int n = min(SLABS, slabs - it * SLABS);
                for (int h = 0; h < n; ++h) {
                    const uint32_t st = smem_base + s * STAGE_BYTES + h * SLAB_BYTES;
#pragma unroll
                    for (int jj = 0; jj < SLAB_J / 16; ++jj) {     // K = 16 per instruction
                        const uint32_t a_lo = desc_lo(st + jj * 2048) | ((uint32_t)(A_BOX_BYTES >> 4) << 16);
                        const uint32_t b_lo = desc_lo(st + A_BYTES + jj * 32);
                        mma_bf16_lean(tmem_base, a_lo, b_lo, kIdesc, (uint32_t)((it | h | jj) != 0));
                    }
                }
                tc_commit(empty_bar(s));
            }
            tc_commit(tfull_bar);                                  // also when a wait gave up: the epilogue must not hang
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp_idx & 3;                                // tensor-memory lane quarter this warp may read
        const int kl = q * 32 + lane;                              // this thread's column within the tile
        if (stages > 0) {
            mbar_wait(tfull_bar, 0u, p.status);
            tc_fence_after();
        }
#pragma unroll
        for (int chunk = 0; chunk < (ROWS + 31) / 32; ++chunk) {
            uint32_t r[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = 0u;
            if (stages > 0) {       // with 16 rows, columns 16..31 of the allocation are not part of the accumulator
                tc_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + chunk * 32, r);
                tc_wait_ld();
            }
            // partial sum of row m into the slot [this rank][m % ROWS_PER_RANK] of CTA m / ROWS_PER_RANK: a warp writes 32 consecutive k
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int m = chunk * 32 + i;
                if (m < ROWS) {
                    const uint32_t dst = mapa_shared(slots_base, (uint32_t)(m / ROWS_PER_RANK)) + rank * (uint32_t)(ROWS_PER_RANK * BLOCK_K * 4) +
                                         (uint32_t)((m % ROWS_PER_RANK) * BLOCK_K * 4) + (uint32_t)kl * 4u;
                    st_shared_cluster_f32(dst, __uint_as_float(r[i]));
                }
            }
        }
    }
    tc_fence_before();
    cluster_sync_all();                                            // every CTA holds the four partial sums of its rows
    if (warp_idx == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    if (warp_idx < 2) return;
    // warps 2..5: a thread = column k, a warp = one MX block of each of this CTA's rows
    const int q = warp_idx & 3, kl = q * 32 + lane, k = k0 + kl;
    if (k0 + q * 32 >= p.K) return;                                // whole blocks only: K is a multiple of 32
    const float bk = p.b != nullptr ? p.b[k] : 0.f;
    for (int i = 0; i < ROWS_PER_RANK; ++i) {
        const int m = (int)rank * ROWS_PER_RANK + i;
        if (m >= p.M) break;
        float y = 0.f;
#pragma unroll
        for (int rk = 0; rk < SPLIT; ++rk) y += slots[(rk * ROWS_PER_RANK + i) * BLOCK_K + kl];
        y += bk;
        if (p.Y_dump != nullptr) p.Y_dump[(size_t)m * p.K + k] = y;
        float amax = fabsf(y);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if ((p.flags & LATMIX_FLAG_CHECK_FINITE) && __any_sync(0xffffffffu, !isfinite(y)) && lane == 0) atomicOr(p.status, 1u << LATMIX_ERR_NONFINITE);
        const uint32_t sb = scale_byte_from_amax(amax, FormatTraits<FMT>::kRMax);
        const float2 f = inv_scale_factors(sb);
        float v[8] = {(y * f.x) * f.y, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (FMT == FMT_FP4) {
            const uint32_t code = pack8_fp4(v) & 0xFu;
            const uint32_t next = __shfl_down_sync(0xffffffffu, code, 1);
            if ((lane & 1) == 0) p.codes[(size_t)m * (p.K >> 1) + (k >> 1)] = (uint8_t)(code | (next << 4));
        } else {
            p.codes[(size_t)m * p.K + k] = (uint8_t)(pack8_bytes<FMT>(v).x & 0xFFu);
        }
        if (lane == 0) {
            const int64_t kb = k >> 5;
            const size_t off = p.sf_layout == LATMIX_SF_LINEAR ? (size_t)m * (p.K >> 5) + kb : sf_tcgen05_offset(m, kb, sf_k_tiles(p.K));
            p.scales[off] = (uint8_t)sb;
        }
    }
}

bool transform_quant_decode_tc_supported(const TransformQuantArgs& a) {
    // tensor maps want row pitches that are multiples of 16 bytes (K is a multiple of 32)
    return a.M > 0 && a.M <= 64 && a.K > 0 && a.K % 32 == 0 && a.K <= tqd2::MAX_K;
}

template <int ROWS>
static cudaError_t launch_decode_rows(const TransformQuantArgs& a, cudaStream_t st) {
    using namespace tqd2;
    constexpr int SMEM_BYTES = Cfg<ROWS>::SMEM_BYTES;
    CUtensorMap tm_a, tm_x;
    if (!make_tensor_map_2d(&tm_a, a.A, 1, (uint64_t)a.K, (uint64_t)a.K, (uint64_t)a.K * 2, 64, SLAB_J) ||
        !make_tensor_map_2d(&tm_x, a.X, 1, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K * 2, SLAB_J, ROWS))
        return cudaErrorInvalidValue;
    TransformQuantDecodeParams p;
    p.b = a.b; p.codes = a.codes; p.scales = a.scales; p.Y_dump = a.Y_dump;
    p.M = (int)a.M; p.K = (int)a.K;
    p.slice = (int)(((a.K + SPLIT - 1) / SPLIT + SLAB_J - 1) / SLAB_J * SLAB_J);
    p.sf_layout = a.sf_layout; p.status = a.status; p.flags = a.flags;
    const void* kern = a.fmt == FMT_FP4 ? (const void*)transform_quant_decode_tc_kernel<FMT_FP4, ROWS>
                     : a.fmt == FMT_FP8 ? (const void*)transform_quant_decode_tc_kernel<FMT_FP8, ROWS>
                     : a.fmt == FMT_INT4 ? (const void*)transform_quant_decode_tc_kernel<FMT_INT4, ROWS>
                                         : (const void*)transform_quant_decode_tc_kernel<FMT_INT8, ROWS>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const unsigned tiles = (unsigned)((a.K + BLOCK_K - 1) / BLOCK_K);
    void* args[] = {(void*)&tm_a, (void*)&tm_x, (void*)&p};
    e = cudaLaunchKernel(kern, dim3(tiles * SPLIT), dim3(192), args, SMEM_BYTES, st);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_transform_quant_decode_tc(const TransformQuantArgs& a, cudaStream_t st) {
    return a.M <= 16 ? launch_decode_rows<16>(a, st) : launch_decode_rows<64>(a, st);
}

}  // namespace latmix
