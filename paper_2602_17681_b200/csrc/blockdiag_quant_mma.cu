// Block-diagonal online transform (the paper's T_3: 32 x 32 blocks = MX blocks) fused with the MX quantiser, bf16
// inputs, the 32 x 32 products on the tensor cores.
//
// The blocks are far too small for a tcgen05 tile (128 rows of one operand, accumulators in tensor memory), so the
// products use the warp-level mma.sync m16n8k16: a warp owns 32 rows x one block, keeps the whole block as B fragments in
// registers, and -- by permuting the block's columns while loading those fragments -- receives, in each group of four
// lanes, eight CONSECUTIVE outputs of a row per lane, which is exactly the ownership the four-lane quantiser wants.
//
// The kernel reads X once.  An item = (four adjacent block columns, 32 consecutive rows): warp w of the CTA owns block
// column 4 c + w, so that the CTA's four warps read 256 contiguous bytes of each row at about the same time (with one
// block column per CTA every 64-byte piece was a DRAM access of its own, 2 K bytes from the next: 2.2 TB/s).  A lane
// needs 16 bytes of each 64-byte row piece, the four loads of a warp's 32 rows are issued together, and the rows of the
// next item are fetched as soon as the MMAs have consumed this item's, i.e. before its values are quantised and stored.  (Feeding the row pieces through the copy engine instead -- one 128 x 64-byte tiled copy
// per item into a ring in shared memory -- was measured and is slower: 26 us against 23 us at 4096 x 4096.)
//
// Work is dealt out block column major; a CTA takes a contiguous range of items (so it changes its blocks, and reloads
// the B fragments, at most once or twice) and the grid is one resident wave.  Everything the epilogue stores to is
// addressed from one pointer per item plus constants.
#include "internal.h"
#include "mx_math.cuh"

namespace latmix {

// D = A B + C with D and C in registers of their own (C is kept across items: the shift of the lane's columns)
__device__ __forceinline__ void mma_m16n8k16_bf16_first(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2], const float (&c)[4]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %11, %12, %13};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
__device__ __forceinline__ void mma_m16n8k16_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

struct TrueTag { static constexpr bool value = true; };
struct FalseTag { static constexpr bool value = false; };

// EXTRAS: dump of the pre-quantisation values and the non-finite check (the plain variant carries none of their
// registers and branches).  An opcode histogram of an earlier version showed 474 instructions per warp and item, 120 of
// them address arithmetic and register moves and 90 predicates and branches, against 150 that do the work: hence one
// pointer each for X, codes and scale bytes that advances by a constant from item to item, rows reached through 32-bit
// offsets, the shift entering as the C operand of the first MMA, the next item's rows loaded into the registers the
// MMAs have just consumed, and a path without row guards for the items that lie wholly inside the matrix.
template <int FMT, bool EXTRAS>
__global__ void __launch_bounds__(128, EXTRAS ? 4 : 5) blockdiag_quant_mma_kernel(const __nv_bfloat16* __restrict__ X,
                                                                  const __nv_bfloat16* __restrict__ A_blocks,
                                                                  const float* __restrict__ b, int64_t M, int64_t K,
                                                                  uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                                  int sf_layout, float* __restrict__ Y_dump, uint32_t* status,
                                                                  uint32_t flags, int64_t chunks, int64_t items) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = lane & 3, g = lane >> 2;                 // fragment coordinates: q = pair of k / of columns, g = row / column
    constexpr int CODE_SHIFT = FMT == FMT_FP4 ? 1 : 0;     // two codes per byte
    const int64_t first = items * (int64_t)blockIdx.x / gridDim.x, last = items * ((int64_t)blockIdx.x + 1) / gridDim.x;
    if (first >= last) return;
    int64_t quad = first / chunks, chunk = first - quad * chunks;      // chunk = 32 rows
    int64_t kb = quad * 4 + warp;                                       // this warp's block column (K is a multiple of 128)
    // B fragments (k16 x n8, "col"): this lane supplies fragment rows 16 s + 2 q + {0, 1, 8, 9} of fragment column g.
    // Both fragment axes are relabelled.  Columns: fragment column g = 2 q' + e of tile t stands for the block's column
    // 8 q' + 2 t + e, so that lane q' ends up with columns 8 q' .. 8 q' + 7.  Rows (the summation index, relabelled the
    // same way in the A fragments): fragment row 16 s + 2 q + 8 h + e stands for k = 8 q + 4 s + 2 h + e, so that a lane's
    // eight A values of a row are the contiguous X[row][8 q .. 8 q + 7]: one 16-byte load.
    uint32_t bf[2][4][2];
    float bias[4][4];                                      // C operand of tile t: {b[2t], b[2t+1]} for both of the lane's rows
    auto load_block = [&](int64_t blk) {
        const uint16_t* Ab = reinterpret_cast<const uint16_t*>(A_blocks) + blk * 1024;
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int col = 8 * (g >> 1) + 2 * t + (g & 1);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int k = 8 * q + 4 * s + 2 * h;
                    bf[s][t][h] = (uint32_t)__ldg(Ab + k * 32 + col) | ((uint32_t)__ldg(Ab + (k + 1) * 32 + col) << 16);
                }
            }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            bias[t][0] = bias[t][2] = b != nullptr ? __ldg(b + blk * 32 + 8 * q + 2 * t) : 0.f;
            bias[t][1] = bias[t][3] = b != nullptr ? __ldg(b + blk * 32 + 8 * q + 2 * t + 1) : 0.f;
        }
    };
    const bool linear = sf_layout == LATMIX_SF_LINEAR;
    const int64_t kt = sf_k_tiles(K);
    // byte offsets of this lane's rows 8 j further down (32-bit: K < 2^26 is checked on the host) and from item to item
    const uint32_t x_row8 = (uint32_t)(16 * K), c_row8 = (uint32_t)((8 * K) >> CODE_SHIFT);
    const uint32_t s_row8 = linear ? (uint32_t)(8 * (K >> 5)) : 128u;     // tiled layout: (row & 31) * 16
    const int64_t x_item = 64 * K, c_item = (32 * K) >> CODE_SHIFT;
    const uint8_t* px;                                                    // this lane's 16 bytes of row j = 0 of the item
    uint8_t* pc;
    auto set_pointers = [&]() {
        const int64_t row0 = chunk * 32 + g;
        px = reinterpret_cast<const uint8_t*>(X + row0 * K + kb * 32 + 8 * q);
        pc = codes + ((row0 * K + kb * 32 + 8 * q) >> CODE_SHIFT);
    };
    auto scale_pointer = [&]() {                                          // of row j = 0 of the current item
        return scales + (linear ? (chunk * 32 + g) * (K >> 5) + kb
                                : ((chunk >> 2) * kt + (kb >> 2)) * 512 + g * 16 + (chunk & 3) * 4 + (kb & 3));
    };
    uint4 xw[4];
    auto load_rows = [&](int64_t ch) {                                    // rows 8 j + g of the warp's 32, issued together
        if ((ch + 1) * 32 <= M) {
#pragma unroll
            for (int j = 0; j < 4; ++j) xw[j] = __ldg(reinterpret_cast<const uint4*>(px + j * x_row8));
        } else {
            const int64_t r0 = ch * 32 + g;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                xw[j] = r0 + 8 * j < M ? __ldg(reinterpret_cast<const uint4*>(px + j * x_row8)) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    load_block(kb);
    set_pointers();
    load_rows(chunk);
    for (int64_t item = first; item < last; ++item) {
        // ---- both 16-row tiles of the warp: rows g, g + 8 of tile mt are j = 2 mt, 2 mt + 1
        float acc[2][4][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            // A fragments (m16 x k16, row-major): rows g and g + 8; fragment columns 16 s + 2 q + {0, 1} and + 8 are, after
            // the relabelling above, words 2 s and 2 s + 1 of the row's 16-byte piece
            const uint32_t wa[4] = {xw[2 * mt].x, xw[2 * mt].y, xw[2 * mt].z, xw[2 * mt].w};
            const uint32_t wb[4] = {xw[2 * mt + 1].x, xw[2 * mt + 1].y, xw[2 * mt + 1].z, xw[2 * mt + 1].w};
            uint32_t af[2][4];
#pragma unroll
            for (int s = 0; s < 2; ++s) { af[s][0] = wa[2 * s]; af[s][1] = wb[2 * s]; af[s][2] = wa[2 * s + 1]; af[s][3] = wb[2 * s + 1]; }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                mma_m16n8k16_bf16_first(acc[mt][t], af[0], bf[0][t], bias[t]);
                mma_m16n8k16_bf16(acc[mt][t], af[1], bf[1][t]);
            }
        }
        // ---- this item's addresses, then on to the next item: its rows are in flight during the epilogue
        const uint8_t* dump_base = nullptr;
        if (EXTRAS) dump_base = reinterpret_cast<const uint8_t*>(Y_dump + (chunk * 32 + g) * K + kb * 32 + 8 * q);
        uint8_t* const pc_cur = pc;
        uint8_t* const ps_cur = scale_pointer();
        const int64_t rows_left = M - (chunk * 32 + g);                   // this lane's row j exists iff 8 j < rows_left
        const bool full = (chunk + 1) * 32 <= M;
        if (item + 1 < last) {
            if (++chunk == chunks) {
                chunk = 0; kb += 4;
                load_block(kb);
                set_pointers();
            } else {
                px += x_item; pc += c_item;
            }
            load_rows(chunk);
        }
        // ---- quantise and store (items wholly inside the matrix take the path without row guards)
        auto epilogue = [&](auto guarded) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) {              // h = 0: row g, h = 1: row g + 8
                    const int j = 2 * mt + h;
                    const bool active = !decltype(guarded)::value || 8 * j < rows_left;
                    float v[8];
#pragma unroll
                    for (int t = 0; t < 4; ++t) { v[2 * t] = acc[mt][t][2 * h]; v[2 * t + 1] = acc[mt][t][2 * h + 1]; }
                    if (EXTRAS && active) {
                        if (Y_dump != nullptr) {
                            float4* d = reinterpret_cast<float4*>(const_cast<uint8_t*>(dump_base) + (int64_t)(8 * j) * K * 4);
                            d[0] = make_float4(v[0], v[1], v[2], v[3]);
                            d[1] = make_float4(v[4], v[5], v[6], v[7]);
                        }
                        if (flags & LATMIX_FLAG_CHECK_FINITE) {
                            bool bad = false;
#pragma unroll
                            for (int i = 0; i < 8; ++i) bad |= !isfinite(v[i]);
                            if (bad) atomicOr(status, 1u << LATMIX_ERR_NONFINITE);
                        }
                    }
                    // rows past M were loaded as zeros and hold only the shift: they take part in the shuffles, store nothing
                    const uint32_t sb = scale_block_of_4_lanes<FMT>(v);
                    if (active) {
                        if (FMT == FMT_FP4) *reinterpret_cast<uint32_t*>(pc_cur + j * c_row8) = pack8_fp4(v);
                        else *reinterpret_cast<uint2*>(pc_cur + j * c_row8) = pack8_bytes<FMT>(v);
                        if (q == 0) ps_cur[j * s_row8] = (uint8_t)sb;
                    }
                }
        };
        if (full) epilogue(FalseTag{}); else epilogue(TrueTag{});
    }
}

bool blockdiag_quant_mma_supported(const QuantArgs& a) {
    return a.x_is_bf16 && a.M > 0 && a.K > 0 && a.K % 128 == 0 && a.K < (1ll << 26);     // 32-bit row offsets in the kernel (up to 48 K bytes)
}

template <int FMT, bool EXTRAS>
static cudaError_t launch_bd_mma_variant2(const QuantArgs& a, const void* A_blocks, int sms, cudaStream_t st) {
    static int occ = 0;                                    // resident CTAs per SM: a property of the compiled kernel
    if (occ == 0) {
        int o = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, blockdiag_quant_mma_kernel<FMT, EXTRAS>, 128, 0) != cudaSuccess || o < 1) o = 4;
        occ = o;
    }
    const int64_t chunks = (a.M + 31) / 32, items = chunks * (a.K / 128);      // (four block columns, 32 rows)
    int64_t ctas = (int64_t)sms * occ;
    if (ctas > items) ctas = items;
    blockdiag_quant_mma_kernel<FMT, EXTRAS><<<dim3((unsigned)ctas), dim3(128), 0, st>>>(
        static_cast<const __nv_bfloat16*>(a.X), static_cast<const __nv_bfloat16*>(A_blocks), a.b, a.M, a.K, a.codes, a.scales,
        a.sf_layout, a.Y_dump, a.status, a.flags, chunks, items);
    return cudaGetLastError();
}

template <int FMT>
static cudaError_t launch_bd_mma_variant(const QuantArgs& a, const void* A_blocks, int sms, cudaStream_t st) {
    const bool extras = a.Y_dump != nullptr || (a.flags & LATMIX_FLAG_CHECK_FINITE);
    return extras ? launch_bd_mma_variant2<FMT, true>(a, A_blocks, sms, st) : launch_bd_mma_variant2<FMT, false>(a, A_blocks, sms, st);
}

cudaError_t launch_blockdiag_quant_mma(const QuantArgs& a, const void* A_blocks, cudaStream_t st) {
    const int sms = sm_count();
    cudaError_t e;
    if (a.fmt == FMT_FP4) e = launch_bd_mma_variant<FMT_FP4>(a, A_blocks, sms, st);
    else if (a.fmt == FMT_FP8) e = launch_bd_mma_variant<FMT_FP8>(a, A_blocks, sms, st);
    else if (a.fmt == FMT_INT4) e = launch_bd_mma_variant<FMT_INT4>(a, A_blocks, sms, st);
    else e = launch_bd_mma_variant<FMT_INT8>(a, A_blocks, sms, st);
    count_launch();
    return e;
}

}  // namespace latmix
