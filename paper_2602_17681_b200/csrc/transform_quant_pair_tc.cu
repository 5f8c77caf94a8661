// Fused online affine transform + MX quantisation on CTA pairs:  codes, scales = Q(X A + 1 b^T).
//
// Same product and the same quantising epilogue as transform_quant_tc.cu, but two CTAs of a cluster share one
// 256 x 256 tile of Y = X A (tcgen05.mma.cta_group::2): each CTA loads its own 128 rows of X and only HALF of
// the columns of the transform matrix, 32 KB instead of 48 KB per 64-deep K slab.  A stage holds TWO such slabs
// (eight MMAs): the issuing thread spends a few hundred cycles per stage on its wait, commit and loop, which four
// 135-cycle MMAs do not hide but eight do.  The single-CTA kernel is bound
// by what the SMs can pull from L2 (1.6 GB per call at the 4096 x 4096 size, about 16 TB/s for all SMs together);
// pairs cut that by a third.
//
// Tail: T tiles on P resident pairs leave the last wave partly empty (256 tiles on 74 pairs: 3.46 waves).  When the
// remainder r = T mod P satisfies 2 r <= P, the last r tiles are cut into two 256 x 128 halves each, so the last
// wave takes half as long.
//
//   warp 0    producer (both CTAs): TMA loads (128-byte swizzle) of a 128 x 64 slab of X and of this CTA's
//             64-column boxes of A; bytes of both CTAs are counted on the LEADER's "full" barrier.
//   warp 1    leader: tcgen05.mma.cta_group::2 kind::f16 into one of two 256-column accumulators per CTA; the loop
//             is unrolled over the stages, every operand precomputed, one wait and one commit per stage.
//   warps 2-5 epilogue (both CTAs): one thread owns one row and 32 consecutive columns = one MX block: add b,
//             block maximum, E8M0 exponent, exact power-of-two scaling, round-to-nearest-even conversion, store.
// Every wait is bounded; all threads of both CTAs meet at a cluster barrier before tensor memory is released.
//
// The same kernel, instantiated with FOLD = true, is the offline fold + weight quantisation
// W~^T[n][k] = sum_j W[j][n] A_inv[k][j]  (Eq. "fold_kqv_1", row form, transposed so that the MX blocks run along k):
// rows are the N output columns of W, read as they are stored (W is j-major: an MN-major A operand), and the fp32
// A_inv is consumed as three bf16 matrices hi + mid + lo (24 significant bits, K-major B operands), three MMAs per
// K = 16 step into the same accumulator: bf16 weights times each term are exact products, so the result has fp32
// accuracy.  One 64-deep slab of j per stage (twelve MMAs).  In its general form (launch_fold_product) the left operand may
// itself be three bf16 terms stacked along the summation index, whose reduction coordinate on the right-hand terms wraps
// (all nine products: the two-sided fold, the back-mapping product of the transformation MSE), the right operand may be a
// single exact term, and the quantiser may be switched off (fp32 product only).
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace tqp {
constexpr int BLOCK_M = 128;                                    // rows per CTA; the pair covers 256
constexpr int BLOCK_N = 256, SLAB_K = 64;                       // SLAB_K bf16 = 128 bytes = one swizzle row
constexpr int SLABS = 2, BLOCK_K = SLABS * SLAB_K;              // K per stage
constexpr int A_BYTES = BLOCK_M * 128;                          // one X slab
constexpr int B_BOX_BYTES = SLAB_K * 128;                       // one 64(k) x 64(n) box of the transform matrix
constexpr int B_BOXES = BLOCK_N / 2 / 64;                       // boxes per CTA and slab for a full-width tile
constexpr int B_OFFSET = SLABS * A_BYTES;                       // stage layout: X slabs, then the boxes slab by slab
constexpr int STAGE_BYTES = SLABS * (A_BYTES + B_BOXES * B_BOX_BYTES);    // 64 KiB
constexpr int STAGES = 3;
constexpr int NUM_ACC = 2;
constexpr int BAR_BYTES = 1024;
constexpr int CODE_STAGING_BYTES = 4 * 32 * BLOCK_N;            // per epilogue warp: 32 rows x up to 256 code bytes (8-bit formats)
constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + BAR_BYTES + CODE_STAGING_BYTES;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
constexpr int TMEM_COLS = 512;
constexpr int THREADS = 6 * 32;
}  // namespace tqp

// fold mode: one slab per stage = W boxes (2 x 8 KiB) + three 16 KiB tiles of the A_inv terms
namespace tqp {
constexpr int FOLD_TERMS = 3;
constexpr int FOLD_A_BYTES = 2 * B_BOX_BYTES;                   // this CTA's 128 rows of W^T: two 64(n) x 64(j) boxes
constexpr int FOLD_T_BYTES = 128 * 128;                         // 128 rows (k) x 64 (j) of one term
static_assert(FOLD_A_BYTES + FOLD_TERMS * FOLD_T_BYTES == STAGE_BYTES, "both modes use the same stage size");
}  // namespace tqp

struct TransformQuantPairParams {
    // fold mode: the right-hand operand is the sum of `num_terms` (1 or 3) bf16 matrices stacked `term_rows` rows apart;
    // its reduction coordinate is j mod `wrap` (the left-hand operand may be three stacked terms of its own, in which
    // case the reduction runs three times over the same columns of the right-hand one)
    int term_rows, num_terms, wrap;
    const float* b;
    uint8_t* codes; uint8_t* scales; float* Y_dump;
    int M, K, num_kb, m_tiles /* of 256 rows */, n_tiles /* of 256 columns */;
    int full_items;      // work items [0, full_items) are whole tiles, the rest are half-width tiles (two per tile)
    int num_items;
    int sf_layout, sf_kt_total;
    uint32_t* status; uint32_t flags;
};

// Work item -> first row of the pair's tile, first column, width (256 or 128).
__device__ __forceinline__ void tqp_decode(const TransformQuantPairParams& p, int item, int& m0, int& n0, int& bn) {
    int tile, half = 0;
    if (item < p.full_items) { tile = item; bn = tqp::BLOCK_N; }
    else { const int h = item - p.full_items; tile = p.full_items + (h >> 1); half = h & 1; bn = tqp::BLOCK_N / 2; }
    m0 = (tile / p.n_tiles) * 256;
    n0 = (tile % p.n_tiles) * tqp::BLOCK_N + half * (tqp::BLOCK_N / 2);
}

template <int FMT, bool FOLD>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(tqp::THREADS, 1)
transform_quant_pair_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_a,
                               const TransformQuantPairParams p) {
    using namespace tqp;
    extern __shared__ uint8_t smem_raw[];
    // same shared-memory offsets in both CTAs: the MMA's descriptors and the multicast commits rely on that
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };                   // leader: both CTAs' bytes landed
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };       // each CTA: stage may be refilled
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + NUM_ACC + a); };   // leader: 4 warps x 2 CTAs
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 2 * NUM_ACC);
    const uint32_t code_staging_base = bar_base + BAR_BYTES;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_a);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    grid_launch_dependents();          // a product kernel launched for it may set itself up on SMs this kernel has left
    grid_dependency_wait();            // and this one may have been set up while its predecessor still ran: its results (the
                                       // activations) are read, and its operands (the codes of the step before) overwritten, from here on
    const int pair = (int)cluster_id_x(), num_pairs = (int)num_clusters_x();
    constexpr uint16_t kBoth = 3;

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int item = pair; item < p.num_items && ok; item += num_pairs) {
                int m0, n0, bn;
                tqp_decode(p, item, m0, n0, bn);
                const int row0 = m0 + (int)rank * BLOCK_M, col0 = n0 + (int)rank * (bn >> 1), boxes = bn >> 7;
                int jt = 0;                                          // fold mode: reduction coordinate of the right-hand terms
                for (int kb = 0; kb < p.num_kb; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    const uint32_t bar = mapa_shared(full_bar(s), 0), st = smem_base + s * STAGE_BYTES;
                    if constexpr (FOLD) {
                        // tm_x: W, box = 64 columns (n) x 64 rows (j); tm_a: the three terms stacked, box = 64 (j) x 128 rows (k).
                        // A half-width tile uses only the first 64 rows of each term tile; the box is loaded whole.
                        if (leader) mbar_expect_tx(full_bar(s), 2 * (FOLD_A_BYTES + p.num_terms * FOLD_T_BYTES));
                        tma_load_2d_pair(st, &tm_x, row0, kb * SLAB_K, bar);
                        tma_load_2d_pair(st + B_BOX_BYTES, &tm_x, row0 + 64, kb * SLAB_K, bar);
#pragma unroll
                        for (int t = 0; t < FOLD_TERMS; ++t)
                            if (t < p.num_terms)
                                tma_load_2d_pair(st + FOLD_A_BYTES + t * FOLD_T_BYTES, &tm_a, jt, t * p.term_rows + col0, bar);
                        jt += SLAB_K;
                        if (jt >= p.wrap) jt = 0;
                        if (++s == STAGES) { s = 0; ph ^= 1u; }
                        continue;
                    }
                    if (leader) mbar_expect_tx(full_bar(s), 2 * SLABS * (A_BYTES + boxes * B_BOX_BYTES));
#pragma unroll
                    for (int h = 0; h < SLABS; ++h) {               // slabs past the end of K read as zero
                        const int k0 = kb * BLOCK_K + h * SLAB_K;
                        const uint32_t bx = st + B_OFFSET + h * B_BOXES * B_BOX_BYTES;
                        tma_load_2d_pair(st + h * A_BYTES, &tm_x, k0, row0, bar);
                        // box: 64 columns (n) x 64 rows (k) of the transform matrix
                        tma_load_2d_pair(bx, &tm_a, col0, k0, bar);
                        if (boxes == 2) tma_load_2d_pair(bx + B_BOX_BYTES, &tm_a, col0 + 64, k0, bar);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue (leader CTA only)
        // Whole warp, one elected lane issues, so that operands stay warp-uniform; the loop is unrolled over the
        // stages and every descriptor word is computed once.
        if (leader) {
            const bool issuer = elect_one();
            // transform: X K-major, A MN-major; fold: W^T MN-major, A_inv terms K-major
            constexpr uint32_t kIdescFull = make_idesc_bf16(2 * BLOCK_M, BLOCK_N, FOLD ? 1 : 0, FOLD ? 0 : 1);
            constexpr uint32_t kIdescHalf = make_idesc_bf16(2 * BLOCK_M, BLOCK_N / 2, FOLD ? 1 : 0, FOLD ? 0 : 1);
            constexpr int MMAS = FOLD ? 4 * FOLD_TERMS : SLABS * 4;   // K = 16 per instruction
            uint32_t a_lo[STAGES][MMAS], b_lo[STAGES][MMAS], full_addr[STAGES], empty_addr[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                full_addr[s] = full_bar(s); empty_addr[s] = empty_bar(s);
#pragma unroll
                for (int j = 0; j < MMAS; ++j) {
                    if constexpr (FOLD) {
                        const int jj = j / FOLD_TERMS, t = j % FOLD_TERMS;    // K step, term
                        // W^T, MN-major: 16 j-rows = 2 x 1024 bytes further down per step; leading offset = box pitch
                        a_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + jj * 2048) | ((uint32_t)(B_BOX_BYTES >> 4) << 16);
                        // term tile, K-major: 32 bytes further along each 128-byte row per step
                        b_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + FOLD_A_BYTES + t * FOLD_T_BYTES + jj * 32);
                        continue;
                    }
                    const int h = j >> 2, jj = j & 3;
                    // X slab, K-major: 32 bytes further along each 128-byte row
                    a_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + h * A_BYTES + jj * 32);
                    // transform matrix, MN-major: 16 k-rows = 2 groups of 8 rows = 2 x 1024 bytes further down; leading
                    // offset = distance between the 64-column boxes, stride offset = 8-row group pitch
                    b_lo[s][j] = desc_lo(smem_base + s * STAGE_BYTES + B_OFFSET + h * B_BOXES * B_BOX_BYTES + jj * 2048) |
                                 ((uint32_t)(B_BOX_BYTES >> 4) << 16);
                }
            }
            uint32_t round_ph = 0, item_count = 0, d_tmem = 0, idesc = kIdescFull, acc = 0;
            int item = pair, kb = 0;
            bool more = item < p.num_items;
            while (more) {
#pragma unroll
                for (int s = 0; s < STAGES; ++s) {                   // s is a constant in each unrolled copy
                    if (kb == 0) {
                        acc = item_count & 1u;
                        mbar_wait_or_flag(tempty_bar(acc), ((item_count >> 1) & 1u) ^ 1u, p.status);
                        d_tmem = tmem_base + acc * BLOCK_N;
                        idesc = item < p.full_items ? kIdescFull : kIdescHalf;
                    }
                    mbar_wait_or_flag(full_addr[s], round_ph, p.status);
                    tc_fence_after();
                    if (issuer) {
#pragma unroll
                        for (int j = 0; j < MMAS; ++j) {
                            if (FOLD && (j % FOLD_TERMS) >= p.num_terms) continue;      // absent terms (j = 0 is term 0)
                            mma_bf16_pair_lean(d_tmem, a_lo[s][j], b_lo[s][j], idesc, j == 0 ? (uint32_t)(kb != 0) : 1u);
                        }
                        tc_commit_pair(empty_addr[s], kBoth);
                    }
                    __syncwarp();
                    if (++kb == p.num_kb) {
                        if (issuer) tc_commit_pair(tfull_bar(acc), kBoth);
                        __syncwarp();
                        kb = 0; ++item_count; item += num_pairs;
                        if (item >= p.num_items) { more = false; break; }
                    }
                }
                round_ph ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ quantising epilogue (warps 2..5, both CTAs)
        const int q = warp_idx & 3;                                  // tensor-memory lane quarter this warp may read
        constexpr int kRMax = FormatTraits<FMT == FMT_NVFP4 ? FMT_FP4 : FMT>::kRMax;
        // The codes of a tile go out through shared memory: a thread owns one row (32 values per chunk, i.e. 16 or 32 code
        // bytes), so stored directly a warp's instruction would touch 32 rows with 16 bytes each.  Staged (16-byte pieces,
        // piece index XOR row to keep the banks apart), a warp then writes whole rows: 8 or 16 lanes per row, 128 or 256
        // contiguous bytes.
        constexpr bool kPacked = FMT == FMT_FP4 || FMT == FMT_NVFP4;          // two codes per byte
        constexpr int kPiecesPerChunk = kPacked ? 1 : 2;                      // 16-byte pieces of codes per thread and chunk
        constexpr int kRowBytes = kPacked ? BLOCK_N / 2 : BLOCK_N;            // staging row pitch
        const uint32_t stg = code_staging_base + (uint32_t)(warp_idx - 2) * (32 * BLOCK_N);
        auto stage_piece = [&](int piece, const uint4& w) {
            const uint32_t dst = stg + (uint32_t)lane * kRowBytes + (uint32_t)(((piece & ~7) | ((piece ^ lane) & 7)) * 16);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
        };
        float nv_g = 1.0f;                                           // NVFP4: the tensor scale, from the scale buffer's trailer
        if (FMT == FMT_NVFP4 && p.codes != nullptr) nv_g = *nvfp4_tensor_scale_ptr(p.scales, p.M, p.K, p.sf_layout);
        uint32_t item_count = 0;
        bool ok = true;
        for (int item = pair; item < p.num_items && ok; item += num_pairs, ++item_count) {
            int m0, n0, bn;
            tqp_decode(p, item, m0, n0, bn);
            const uint32_t acc = item_count % NUM_ACC, acc_ph = (item_count / NUM_ACC) & 1u;
            ok = mbar_wait(tfull_bar(acc), acc_ph, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int64_t row = m0 + (int)rank * BLOCK_M + q * 32 + lane;
            const bool row_ok = row < p.M;
            uint32_t sf_word = 0;
#pragma unroll 1
            for (int chunk = 0; chunk < (bn >> 5); ++chunk) {
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
                if (p.codes == nullptr) continue;                // product only: the dump above is the result
                if (FMT == FMT_NVFP4) {
                    // two blocks of 16 per thread; their scale bytes are neighbours in both layouts
                    uint2 w0, w1;
                    const uint32_t s0 = nvfp4_quantize_block(v, nv_g, w0), s1 = nvfp4_quantize_block(v + 16, nv_g, w1);
                    if (blk_ok) {
                        stage_piece(chunk, make_uint4(w0.x, w0.y, w1.x, w1.y));
                        const int64_t kblk = col0 >> 4;
                        const size_t off = p.sf_layout == LATMIX_SF_LINEAR ? (size_t)(row * (p.K >> 4) + kblk)
                                                                           : sf_tcgen05_offset(row, kblk, p.sf_kt_total);
                        *reinterpret_cast<uint16_t*>(p.scales + off) = (uint16_t)(s0 | (s1 << 8));
                    }
                    continue;
                }
                const uint32_t sb = scale_byte_from_amax(amax, kRMax);
                const float2 f = inv_scale_factors(sb);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = (v[i] * f.x) * f.y;
                if (blk_ok) {
                    if (FMT == FMT_FP4 || FMT == FMT_NVFP4) {
                        stage_piece(chunk, make_uint4(pack8_fp4(v), pack8_fp4(v + 8), pack8_fp4(v + 16), pack8_fp4(v + 24)));
                    } else {
                        uint2 w0, w1, w2, w3;
                        w0 = pack8_bytes<FMT>(v); w1 = pack8_bytes<FMT>(v + 8); w2 = pack8_bytes<FMT>(v + 16); w3 = pack8_bytes<FMT>(v + 24);
                        stage_piece(2 * chunk, make_uint4(w0.x, w0.y, w1.x, w1.y));
                        stage_piece(2 * chunk + 1, make_uint4(w2.x, w2.y, w3.x, w3.y));
                    }
                    const int64_t kblk = col0 >> 5;
                    if (p.sf_layout == LATMIX_SF_LINEAR) {
                        p.scales[row * (p.K >> 5) + kblk] = (uint8_t)sb;
                    } else {
                        // four consecutive blocks of a row share one aligned 32-bit word of the tile layout
                        sf_word |= sb << (8 * (chunk & 3));
                        if ((chunk & 3) == 3 || col0 + 32 >= p.K)
                            *reinterpret_cast<uint32_t*>(p.scales + sf_tcgen05_offset(row, kblk & ~3ll, p.sf_kt_total)) = sf_word;
                    }
                }
                if ((chunk & 3) == 3) sf_word = 0;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {                                      // this warp has drained its quarter of the accumulator
                if (leader) mbar_arrive(tempty_bar(acc));
                else mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
            }
            if (p.codes != nullptr) {
                // the staged codes, whole rows at a time: `lanes_per_row` lanes write one row's 16-byte pieces side by side
                const int pieces = (bn >> 5) * kPiecesPerChunk;                  // per row in this item: 4, 8 or 16
                const int rows_per_it = 32 / pieces, piece = lane % pieces;
                const int64_t row_base = m0 + (int)rank * BLOCK_M + q * 32;
                const int64_t row_pitch = kPacked ? (int64_t)(p.K >> 1) : (int64_t)p.K, col_byte0 = kPacked ? (n0 >> 1) : n0;
                for (int r0 = 0; r0 < 32; r0 += rows_per_it) {
                    const int r = r0 + lane / pieces;
                    const uint32_t src = stg + (uint32_t)r * kRowBytes + (uint32_t)(((piece & ~7) | ((piece ^ r) & 7)) * 16);
                    uint4 w;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(src));
                    // a piece = 32 elements (4-bit) or 16 (8-bit); K is a multiple of 32, so a piece is inside the matrix or outside it
                    const int64_t elem0 = n0 + (int64_t)piece * (kPacked ? 32 : 16);
                    if (row_base + r < p.M && elem0 < p.K)
                        *reinterpret_cast<uint4*>(p.codes + (row_base + r) * row_pitch + col_byte0 + piece * 16) = w;
                }
                __syncwarp();                                     // the buffer is rewritten by the next item's first chunk
            }
        }
    }
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    cluster_sync_all();             // the leader's MMAs read the peer's shared memory and write its tensor memory
    if (warp_idx == 1) tmem_dealloc_pair(tmem_base, tqp::TMEM_COLS);
}

bool transform_quant_pair_tc_supported(const TransformQuantArgs& a) {
    // With 128 rows or fewer the second CTA of a pair multiplies zero rows, but each CTA still streams only its half of
    // the transform matrix's columns, which is what bounds small batches.
    return a.K > 0 && a.K % 32 == 0 && a.M > 0 && a.M < (1ll << 30) && a.K < (1ll << 30);
}

cudaError_t launch_transform_quant_pair_tc(const TransformQuantArgs& a, cudaStream_t st) {
    using namespace tqp;
    CUtensorMap tm_x, tm_a;
    if (!make_tensor_map_2d(&tm_x, a.X, 1, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K * 2, SLAB_K, BLOCK_M) ||
        !make_tensor_map_2d(&tm_a, a.A, 1, (uint64_t)a.K, (uint64_t)a.K, (uint64_t)a.K * 2, 64, SLAB_K))
        return cudaErrorInvalidValue;
    TransformQuantPairParams p;
    p.b = a.b; p.codes = a.codes; p.scales = a.scales; p.Y_dump = a.Y_dump;
    p.M = (int)a.M; p.K = (int)a.K;
    p.num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);
    p.m_tiles = (int)((a.M + 255) / 256);
    p.n_tiles = (int)((a.K + BLOCK_N - 1) / BLOCK_N);
    p.sf_layout = a.sf_layout; p.sf_kt_total = (int)(a.fmt == FMT_NVFP4 ? nvfp4_sf_k_tiles(a.K) : sf_k_tiles(a.K));
    p.status = a.status; p.flags = a.flags;
    p.term_rows = 0; p.num_terms = 0; p.wrap = 1;
    const void* kern = a.fmt == FMT_FP4 ? (const void*)transform_quant_pair_tc_kernel<FMT_FP4, false>
                     : a.fmt == FMT_FP8 ? (const void*)transform_quant_pair_tc_kernel<FMT_FP8, false>
                     : a.fmt == FMT_INT4 ? (const void*)transform_quant_pair_tc_kernel<FMT_INT4, false>
                     : a.fmt == FMT_NVFP4 ? (const void*)transform_quant_pair_tc_kernel<FMT_NVFP4, false>
                                        : (const void*)transform_quant_pair_tc_kernel<FMT_INT8, false>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int pairs = resident_cta_pairs(kern, THREADS, SMEM_BYTES);
    // the last, partly filled wave is cut into half-width tiles when that makes it shorter
    const int tiles = p.m_tiles * p.n_tiles;
    const int rem = tiles % pairs;
    const bool split = rem > 0 && 2 * rem <= pairs;
    p.full_items = split ? tiles - rem : tiles;
    p.num_items = split ? tiles + rem : tiles;
    const unsigned grid = 2u * (unsigned)(p.num_items < pairs ? p.num_items : pairs);
    void* args[] = {(void*)&tm_x, (void*)&tm_a, (void*)&p};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelExC(&cfg, kern, args);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- offline fold on the tensor cores ------------------------------------------------------------------------
// fp32 -> three bf16 terms, stacked [3][K][K]:  a = hi + mid + lo up to 2^-24 |a| (each difference is exact in fp32).
__global__ void __launch_bounds__(256) split_f32_to_3bf16_kernel(const float* __restrict__ a, int64_t n, __nv_bfloat16* __restrict__ out) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const float v = a[i];
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        const float r1 = v - __bfloat162float(hi);
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        out[i] = hi; out[n + i] = mid; out[2 * n + i] = lo;
    }
}

size_t fold_tc_scratch_bytes(int64_t K) { return (size_t)3 * (size_t)K * (size_t)K * 2; }

bool fold_tc_supported(int64_t K, int64_t N, int w_is_bf16) {
    // tensor maps want row pitches that are multiples of 16 bytes: N (rows of W) and K (rows of the terms) multiples of 8
    return w_is_bf16 && K > 0 && N > 0 && K % 32 == 0 && N % 8 == 0 && K < (1ll << 30) && N < (1ll << 30) && 3 * K < (1ll << 31);
}

// The fold-mode product in its general form:
//   result[r][c] = sum_{j < red_len} P[j][r] * sum_t terms[t][c][j mod wrap],   r < R, c < C,
// written as fp32 to `dump` (row pitch C) and, unless `codes` is null, MX-quantised along c.
struct FoldProductArgs {
    const void* P; int64_t red_len, R;             // bf16 [red_len][R]
    const void* terms; int num_terms; int64_t C, wrap;   // bf16 [num_terms][C][wrap]
    int fmt, sf_layout;
    uint8_t* codes; uint8_t* scales; float* dump;
    uint32_t* status; uint32_t flags;
};

static cudaError_t launch_fold_product(const FoldProductArgs& a, cudaStream_t st) {
    using namespace tqp;
    CUtensorMap tm_p, tm_t;
    if (!make_tensor_map_2d(&tm_p, a.P, 1, (uint64_t)a.R, (uint64_t)a.red_len, (uint64_t)a.R * 2, 64, SLAB_K) ||
        !make_tensor_map_2d(&tm_t, a.terms, 1, (uint64_t)a.wrap, (uint64_t)(a.num_terms * a.C), (uint64_t)a.wrap * 2, SLAB_K, 128))
        return cudaErrorInvalidValue;
    TransformQuantPairParams p;
    p.term_rows = (int)a.C; p.num_terms = a.num_terms; p.wrap = (int)a.wrap;
    p.b = nullptr; p.codes = a.codes; p.scales = a.scales; p.Y_dump = a.dump;
    p.M = (int)a.R; p.K = (int)a.C;
    p.num_kb = (int)((a.red_len + SLAB_K - 1) / SLAB_K);
    p.m_tiles = (int)((a.R + 255) / 256);
    p.n_tiles = (int)((a.C + BLOCK_N - 1) / BLOCK_N);
    p.sf_layout = a.sf_layout; p.sf_kt_total = (int)(a.fmt == FMT_NVFP4 ? nvfp4_sf_k_tiles(a.C) : sf_k_tiles(a.C));
    p.status = a.status; p.flags = a.flags;
    const void* kern = a.fmt == FMT_FP4 ? (const void*)transform_quant_pair_tc_kernel<FMT_FP4, true>
                     : a.fmt == FMT_FP8 ? (const void*)transform_quant_pair_tc_kernel<FMT_FP8, true>
                     : a.fmt == FMT_INT4 ? (const void*)transform_quant_pair_tc_kernel<FMT_INT4, true>
                     : a.fmt == FMT_NVFP4 ? (const void*)transform_quant_pair_tc_kernel<FMT_NVFP4, true>
                                        : (const void*)transform_quant_pair_tc_kernel<FMT_INT8, true>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int pairs = resident_cta_pairs(kern, THREADS, SMEM_BYTES);
    const int tiles = p.m_tiles * p.n_tiles;
    const int rem = tiles % pairs;
    const bool split = rem > 0 && 2 * rem <= pairs;
    p.full_items = split ? tiles - rem : tiles;
    p.num_items = split ? tiles + rem : tiles;
    const unsigned grid = 2u * (unsigned)(p.num_items < pairs ? p.num_items : pairs);
    void* args[] = {(void*)&tm_p, (void*)&tm_t, (void*)&p};
    e = cudaLaunchKernel(kern, dim3(grid), dim3(THREADS), args, SMEM_BYTES, st);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

static cudaError_t launch_split3(const float* a, int64_t n, __nv_bfloat16* out, cudaStream_t st) {
    const int sms = sm_count();
    split_f32_to_3bf16_kernel<<<(unsigned)(sms * 8), 256, 0, st>>>(a, n, out);
    count_launch();
    return cudaGetLastError();
}

// W~^T = W^T A_inv^T quantised along k: codes N x K, scales for N rows; `scratch` holds fold_tc_scratch_bytes(K) bytes.
cudaError_t launch_fold_quant_pair_tc(const float* A_inv, const void* W, int64_t K, int64_t N, int fmt, int sf_layout,
                                      uint8_t* codes, uint8_t* scales, float* dump, uint32_t* status, uint32_t flags,
                                      void* scratch, cudaStream_t st) {
    __nv_bfloat16* terms = static_cast<__nv_bfloat16*>(scratch);
    cudaError_t e = launch_split3(A_inv, K * K, terms, st);
    if (e != cudaSuccess) return e;
    FoldProductArgs a{W, K, N, terms, 3, K, K, fmt, sf_layout, codes, scales, dump, status, flags};
    return launch_fold_product(a, st);
}

// fp32 weights: W enters as three bf16 terms stacked along the summation index (3K rows), against the three terms of A_inv
// with the reduction coordinate wrapping at K: all nine products, fp32-accurate.  `scratch` holds the terms of A_inv
// (6 K^2 bytes) followed by those of W (6 K N bytes).
size_t fold_tc_f32_scratch_bytes(int64_t K, int64_t N) { return (size_t)6 * (size_t)K * (size_t)K + (size_t)6 * (size_t)K * (size_t)N; }
bool fold_tc_f32_supported(int64_t K, int64_t N) {
    return K > 0 && N > 0 && K % 64 == 0 && N % 8 == 0 && 3 * K < (1ll << 30) && N < (1ll << 30);
}
cudaError_t launch_fold_quant_pair_tc_f32(const float* A_inv, const float* W, int64_t K, int64_t N, int fmt, int sf_layout,
                                          uint8_t* codes, uint8_t* scales, float* dump, uint32_t* status, uint32_t flags,
                                          void* scratch, cudaStream_t st) {
    __nv_bfloat16* ai = static_cast<__nv_bfloat16*>(scratch);
    __nv_bfloat16* wt = ai + (size_t)3 * (size_t)K * (size_t)K;
    cudaError_t e;
    if ((e = launch_split3(A_inv, K * K, ai, st)) != cudaSuccess) return e;
    if ((e = launch_split3(W, K * N, wt, st)) != cudaSuccess) return e;
    FoldProductArgs a{wt, 3 * K, N, ai, 3, K, K, fmt, sf_layout, codes, scales, dump, status, flags};
    return launch_fold_product(a, st);
}

// ---- two-sided fold on the tensor cores ----------------------------------------------------------------------
// Transposes (32 x 32 tiles through shared memory).  in: rows x cols, out: cols x rows.
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ in, int64_t rows, int64_t cols,
                                                             __nv_bfloat16* __restrict__ out) {
    __shared__ __nv_bfloat16 t[32][34];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t r0 = (int64_t)blockIdx.y * 32, c0 = (int64_t)blockIdx.x * 32;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < rows && c0 + tx < cols) t[i][tx] = in[(r0 + i) * cols + c0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8)
        if (c0 + i < cols && r0 + tx < rows) out[(c0 + i) * rows + r0 + tx] = t[tx][i];
}

// fp32 rows x cols -> the three bf16 terms of its transpose, stacked [3][cols][rows]
__global__ void __launch_bounds__(256) split_transposed_f32_to_3bf16_kernel(const float* __restrict__ in, int64_t rows, int64_t cols,
                                                                            __nv_bfloat16* __restrict__ out) {
    __shared__ float t[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t r0 = (int64_t)blockIdx.y * 32, c0 = (int64_t)blockIdx.x * 32;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < rows && c0 + tx < cols) t[i][tx] = in[(r0 + i) * cols + c0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        if (c0 + i >= cols || r0 + tx >= rows) continue;
        const float v = t[tx][i];
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        const float r1 = v - __bfloat162float(hi);
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        const int64_t o = (c0 + i) * rows + r0 + tx;
        out[o] = hi; out[rows * cols + o] = mid; out[2 * rows * cols + o] = lo;
    }
}

static cudaError_t launch_split3_transposed(const float* in, int64_t rows, int64_t cols, __nv_bfloat16* out, cudaStream_t st) {
    split_transposed_f32_to_3bf16_kernel<<<dim3((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32)), 256, 0, st>>>(in, rows, cols, out);
    count_launch();
    return cudaGetLastError();
}

bool fold_two_sided_tc_supported(int64_t K, int64_t N, int w_is_bf16) {
    // stacked terms must start on a slab boundary of the reduction: both sizes multiples of 64
    return w_is_bf16 && K > 0 && N > 0 && K % 64 == 0 && N % 64 == 0 && 3 * K < (1ll << 30) && 3 * N < (1ll << 30);
}

size_t fold_two_sided_tc_scratch_bytes(int64_t K, int64_t N, bool both) {
    const size_t kn = (size_t)K * (size_t)N, nn = (size_t)N * (size_t)N, kk = (size_t)K * (size_t)K;
    // output side only: the three terms of A_out.  Both: W^T, terms of A_out^T, T = W A_out in fp32 and as three terms,
    // terms of A_in_inv.
    return both ? 2 * kn + 6 * nn + 4 * kn + 6 * kn + 6 * kk : 6 * nn;
}

// W~~^T = A_out^T W^T A_in_inv^T quantised along k.  Output side first, so that the exact bf16 weights meet the first
// three-term operand:  T = W A_out (fp32, K x N), then the one-sided fold of T with both operands as three terms.
// A_in_inv null = output side only.  `T_out` (nullable unless both sides) receives T for the bias fold.
cudaError_t launch_fold_two_sided_tc(const float* A_in_inv, const void* W, const float* A_out, int64_t K, int64_t N, int fmt,
                                     int sf_layout, uint8_t* codes, uint8_t* scales, float* dump, float** T_out,
                                     uint32_t* status, uint32_t flags, void* scratch, cudaStream_t st) {
    uint8_t* sc = static_cast<uint8_t*>(scratch);
    const size_t kn = (size_t)K * (size_t)N, nn = (size_t)N * (size_t)N;
    cudaError_t e;
    if (A_in_inv == nullptr) {
        // result[n][k] = sum_i A_out[i][n] W[k][i]: left operand = the three terms of A_out stacked along the reduction,
        // right operand = W itself (one exact term), its reduction coordinate wrapping at N
        __nv_bfloat16* ao = reinterpret_cast<__nv_bfloat16*>(sc);
        if ((e = launch_split3(A_out, (int64_t)nn, ao, st)) != cudaSuccess) return e;
        FoldProductArgs a{ao, 3 * N, N, W, 1, K, N, fmt, sf_layout, codes, scales, dump, status, flags};
        return launch_fold_product(a, st);
    }
    __nv_bfloat16* wt = reinterpret_cast<__nv_bfloat16*>(sc);                     // W^T, N x K
    __nv_bfloat16* aot = reinterpret_cast<__nv_bfloat16*>(sc + 2 * kn);           // terms of A_out^T
    float* T = reinterpret_cast<float*>(sc + 2 * kn + 6 * nn);                    // W A_out, K x N
    __nv_bfloat16* tt = reinterpret_cast<__nv_bfloat16*>(sc + 6 * kn + 6 * nn);   // its three terms, stacked [3K][N]
    __nv_bfloat16* ai = reinterpret_cast<__nv_bfloat16*>(sc + 12 * kn + 6 * nn);  // terms of A_in_inv
    transpose_bf16_kernel<<<dim3((unsigned)((N + 31) / 32), (unsigned)((K + 31) / 32)), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(W), K, N, wt);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = launch_split3_transposed(A_out, N, N, aot, st)) != cudaSuccess) return e;
    // T[j][n] = sum_i W[j][i] A_out[i][n]: left operand W^T ([i][j]), right operand the terms of A_out^T ([n][i]); product only
    FoldProductArgs a1{wt, N, K, aot, 3, N, N, FMT_FP4, LATMIX_SF_LINEAR, nullptr, nullptr, T, status, flags};
    if ((e = launch_fold_product(a1, st)) != cudaSuccess) return e;
    if ((e = launch_split3(T, (int64_t)kn, tt, st)) != cudaSuccess) return e;
    if ((e = launch_split3(A_in_inv, K * K, ai, st)) != cudaSuccess) return e;
    // result[n][k] = sum_j T[j][n] A_in_inv[k][j] with T as three terms stacked along the reduction (all nine products)
    FoldProductArgs a2{tt, 3 * K, N, ai, 3, K, K, fmt, sf_layout, codes, scales, dump, status, flags};
    if (T_out != nullptr) *T_out = T;
    return launch_fold_product(a2, st);
}

// ---- the error of the transformed domain mapped back: E = D A_inv (M x K, fp32-accurate) -----------------------
bool backmap_tc_supported(int64_t M, int64_t K) {
    return M >= 64 && M % 8 == 0 && K > 0 && K % 64 == 0 && 3 * K < (1ll << 30) && M < (1ll << 30);
}
size_t backmap_tc_scratch_bytes(int64_t M, int64_t K) { return (size_t)6 * (size_t)M * (size_t)K + (size_t)6 * (size_t)K * (size_t)K; }

// E[m][k] = sum_j D[m][j] A_inv[j][k]: left operand the three terms of D^T stacked along the reduction, right operand the
// three terms of A_inv^T, reduction coordinate wrapping at K.  E may alias D (the product reads the copies in `scratch`).
cudaError_t launch_backmap_tc(const float* D, const float* A_inv, int64_t M, int64_t K, float* E, uint32_t* status,
                              void* scratch, cudaStream_t st) {
    __nv_bfloat16* dt = static_cast<__nv_bfloat16*>(scratch);                       // [3][K][M]
    __nv_bfloat16* ait = dt + (size_t)3 * (size_t)M * (size_t)K;                    // [3][K][K]
    cudaError_t e;
    if ((e = launch_split3_transposed(D, M, K, dt, st)) != cudaSuccess) return e;
    if ((e = launch_split3_transposed(A_inv, K, K, ait, st)) != cudaSuccess) return e;
    FoldProductArgs a{dt, 3 * K, M, ait, 3, K, K, FMT_FP4, LATMIX_SF_LINEAR, nullptr, nullptr, E, status, 0u};
    return launch_fold_product(a, st);
}

}  // namespace latmix
