// MXINT8 product for small batches (M <= 64) on the integer tensor-core kind:  out[M x N] = dq(Qa) dq(Qw)^T + c.
//
// An MXINT8 element is k 2^(E-6) with an 8-bit integer k and one exponent E per block of 32.  No block-scaled tcgen05 kind
// takes integers, but tcgen05.mma kind::i8 multiplies int8 codes as they are (K = 32 per instruction: exactly one MX
// block) and accumulates in int32, exactly.  So the codes go from the copy engine's shared-memory tiles straight into the
// tensor core, one MMA per block into a column range of its own, and the block scales are applied AFTERWARDS to the
// integer sums of a weight row (one per activation row), in fp32: sum over blocks of  S_blk 2^(Ea + Ew - 12),  |S_blk| <= 32 x 127^2 < 2^24 exact as a
// float.  Against converting the weights to bf16 first (the other small-batch MXINT8 kernel, 26 us at 4096 x 14336) that
// removes the conversion of every weight byte (about 700 cycles of issue slots per 16 KB slab) and halves the MMAs.
//   warp 0    producer: per 128-deep K slab the int8 weight tile (128 rows x 128 bytes), the int8 activation tile (16 to 64
//             rows) and the two 512-byte scale tiles, into a ring of raw stages
//   warp 1    per slab four tcgen05.mma kind::i8 (M = 128 weight rows, N = 16 to 64 activation rows, K = 32), each with a
//             fresh accumulator of N columns in one of the tensor-memory buffers (eight at N = 16, two at N = 64); one commit
//             hands the buffer to the scalers
//   warps 2-9 scalers (a thread = one weight row and half of the activation rows; two warps per tensor-memory lane
//             quarter): tcgen05.ld of the slab's integer sums (all four blocks at once at 16 rows, two or one at a time
//             beyond), times the weight block's scale, times the activation row's (a table of floats per slab that each warp
//             builds for itself in shared memory), added to fp32 accumulators in registers in K order; after the last slab
//             + c[n] and the store.  With four warps and sixteen rows each, and an integer-to-float conversion per sum
//             (quarter rate), this arithmetic was what bound the kernel at 16 rows (21 us; 15 us without it)
// Scale bytes of 233 and above (2^100 and more) take a branch of their own that combines the two exponents as integers
// first, so that no intermediate leaves fp32's range when the product does not.  Every wait is bounded.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace i8i {
constexpr int BLOCK_W = 128;
constexpr int RAW_W = BLOCK_W * 128, SF = 512;
constexpr int TMEM_COLS = 512;
constexpr int SCALER_WARPS = 8;                                    // two per tensor-memory lane quarter: the lower and the upper half of the activation rows
constexpr int BAR_BYTES = 512;
constexpr int THREADS = (2 + SCALER_WARPS) * 32;
// ROWS activation rows (16, 32, 48 or 64: the N side of the MMA)
template <int ROWS>
struct Cfg {
    static constexpr int RAW_A = ROWS * 128;
    static constexpr int RAW_BYTES = RAW_W + RAW_A + 2 * SF;                       // 19 KiB at 16 rows
    static constexpr int P_COLS = 4 * ROWS;                                        // integer sums: 4 blocks x ROWS activation rows per slab
    static constexpr int P_BUFS = TMEM_COLS / P_COLS > 8 ? 8 : TMEM_COLS / P_COLS;
    static constexpr int HALF_ROWS = ROWS / 2;
    static constexpr int TABLE_BYTES = SCALER_WARPS * HALF_ROWS * 4 * 4;           // per scaler warp: HALF_ROWS x 4 blocks of activation scales as floats
    static constexpr int RAW_STAGES = (227 * 1024 - 1024 - TABLE_BYTES - BAR_BYTES) / RAW_BYTES > 11 ? 11 : (227 * 1024 - 1024 - TABLE_BYTES - BAR_BYTES) / RAW_BYTES;
    static constexpr int SMEM_BYTES = 1024 + RAW_STAGES * RAW_BYTES + TABLE_BYTES + BAR_BYTES;
    static_assert(ROWS % 16 == 0 && ROWS >= 16 && ROWS <= 64, "activation rows");
    static_assert(RAW_BYTES % 1024 == 0 && SMEM_BYTES <= 227 * 1024 && P_BUFS >= 2 && P_BUFS * P_COLS <= TMEM_COLS, "memory layout");
    static_assert(8 * (2 * RAW_STAGES + 2 * P_BUFS + 1) <= BAR_BYTES, "barrier area");
    // instruction descriptor of kind::i8: D = S32 (2 at bit 4), A and B signed 8-bit (1 at bits 7 and 10), both K-major
    static constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(ROWS >> 3) << 17) | ((uint32_t)(BLOCK_W >> 4) << 24);
};
}  // namespace i8i

struct Mxint8DecodeI8Params {
    const uint8_t* a_scales; const uint8_t* w_scales; const float* c;
    float* out; int64_t ldo;
    int M, N, num_kb /* 128-deep slabs */, sf_kt_total, n_tiles;
    uint32_t* status;
};

__device__ __forceinline__ void mma_i8_lean(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, 0, 0;\n\t"       // never accumulates: every block starts from zero
        "mov.b64 da, {%1, %4};\n\tmov.b64 db, {%2, %4};\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(kDescHiSw128) : "memory");
}

__device__ __forceinline__ uint32_t lds32_i8i(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
// 2^x for x in [-149, 127], exact
__device__ __forceinline__ float pow2_int(int x) {
    return x >= -126 ? __uint_as_float((uint32_t)(x + 127) << 23) : __uint_as_float(1u << (x + 149));
}

template <int ROWS>
__global__ void __launch_bounds__(i8i::THREADS, 1)
mxint8_gemm_decode_i8_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a,
                                const Mxint8DecodeI8Params p) {
    using namespace i8i;
    using C = Cfg<ROWS>;
    constexpr int RAW_A = C::RAW_A, RAW_BYTES = C::RAW_BYTES, RAW_STAGES = C::RAW_STAGES, P_BUFS = C::P_BUFS, P_COLS = C::P_COLS;
    constexpr int HALF_ROWS = C::HALF_ROWS, TABLE_BYTES = C::TABLE_BYTES;
    constexpr uint32_t kIdesc = C::kIdesc;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t table_base = smem_base + RAW_STAGES * RAW_BYTES;
    const uint32_t bar_base = table_base + TABLE_BYTES;
    auto raw_full = [&](int s) { return bar_base + 8u * s; };                       // the slab's four copies have landed
    auto raw_empty = [&](int s) { return bar_base + 8u * (RAW_STAGES + s); };       // its MMAs are done and the scalers have its scales
    auto p_full = [&](int b) { return bar_base + 8u * (2 * RAW_STAGES + b); };      // the slab's integer sums are complete
    auto p_empty = [&](int b) { return bar_base + 8u * (2 * RAW_STAGES + P_BUFS + b); };   // the scaler warps have read them
    const uint32_t tmem_slot = bar_base + 8u * (2 * RAW_STAGES + 2 * P_BUFS);
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_w); prefetch_tmap(&tm_a);
        for (int s = 0; s < RAW_STAGES; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), SCALER_WARPS); }   // the scaler warps, each after the slab's MMAs are done and it has the scales
        for (int b = 0; b < P_BUFS; ++b) { mbar_init(p_full(b), 1); mbar_init(p_empty(b), SCALER_WARPS); }
        fence_mbar_init();
    }
    if (warp_idx == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    grid_dependency_wait();            // set-up above overlapped the previous kernel; its results are needed from here on

    if (warp_idx == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % RAW_STAGES;
                    if (!(ok = mbar_wait(raw_empty(s), ((it / RAW_STAGES) & 1u) ^ 1u, p.status))) break;
                    const uint32_t st = smem_base + s * RAW_BYTES;
                    mbar_expect_tx(raw_full(s), RAW_BYTES);
                    tma_load_2d(st, &tm_w, kb * 128, tile * BLOCK_W, raw_full(s));       // rows past N read as zero
                    tma_load_2d(st + RAW_W, &tm_a, kb * 128, 0, raw_full(s));            // rows past M read as zero
                    bulk_load(st + RAW_W + RAW_A, p.w_scales + ((size_t)tile * p.sf_kt_total + kb) * 512, SF, raw_full(s));
                    bulk_load(st + RAW_W + RAW_A + SF, p.a_scales + (size_t)kb * 512, SF, raw_full(s));
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % RAW_STAGES, b = it % P_BUFS;
                    if (!(ok = mbar_wait(raw_full(s), (it / RAW_STAGES) & 1u, p.status) &&
                               mbar_wait(p_empty(b), ((it / P_BUFS) & 1u) ^ 1u, p.status))) break;
                    tc_fence_after();
                    const uint32_t w_lo = desc_lo(smem_base + s * RAW_BYTES), a_lo = desc_lo(smem_base + s * RAW_BYTES + RAW_W);
                    const uint32_t d = tmem_base + (uint32_t)b * P_COLS;
#pragma unroll
                    for (int blk = 0; blk < 4; ++blk)      // one MX block = 32 bytes of K per row = one MMA, a fresh accumulator each
                        mma_i8_lean(d + (uint32_t)(ROWS * blk), w_lo + 2 * blk, a_lo + 2 * blk, kIdesc);
                    tc_commit(p_full(b));      // the scalers free the raw stage: they arrive on its barrier after they have seen this one
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ scalers (warps 2..9): a thread = one weight row and
        // half of the activation rows
        const int q = warp_idx & 3;                    // tensor-memory lane quarter this warp may read
        const int hm = (warp_idx - 2) >> 2;            // activation rows HALF_ROWS hm .. HALF_ROWS hm + HALF_ROWS - 1
        const int t = q * 32 + lane;                   // weight row within the tile = tensor-memory lane
        const uint32_t table = table_base + (uint32_t)(warp_idx - 2) * (HALF_ROWS * 16u);   // this warp's activation scales, [block][row] floats
        // byte offset of activation row m's word (its four blocks of a slab) in the 128-row x 4-block scale tile
        auto a_word = [](int m) { return (uint32_t)((m & 31) * 16 + (m >> 5) * 4); };
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
            float acc[HALF_ROWS];
#pragma unroll
            for (int m = 0; m < HALF_ROWS; ++m) acc[m] = 0.f;
            const bool row_valid = (int64_t)tile * BLOCK_W + t < p.N;
            for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                const int s = it % RAW_STAGES, b = it % P_BUFS;
                // one lane polls; the copies' barrier first (it orders this warp's reads of the scale tiles after the copies)
                if (lane == 0)
                    ok = mbar_wait(raw_full(s), (it / RAW_STAGES) & 1u, p.status) && mbar_wait(p_full(b), (it / P_BUFS) & 1u, p.status);
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                // the integer sums leave tensor memory G blocks at a time (all four while they fit the registers); the first group's
                // loads are in flight while the scales are prepared
                constexpr int G = HALF_ROWS <= 8 ? 4 : HALF_ROWS <= 16 ? 2 : 1;
                const uint32_t ta = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)b * P_COLS + (uint32_t)(hm * HALF_ROWS);
                uint32_t r[G][HALF_ROWS];              // per block the integer sums of this warp's activation rows
                auto load_group = [&](int g0) {
#pragma unroll
                    for (int gb = 0; gb < G; ++gb)
#pragma unroll
                        for (int c8 = 0; c8 < HALF_ROWS / 8; ++c8) {
                            uint32_t r8[8];
                            tc_ld_32x32b_x8(ta + (uint32_t)(ROWS * (g0 + gb) + 8 * c8), r8);
#pragma unroll
                            for (int z = 0; z < 8; ++z) r[gb][8 * c8 + z] = r8[z];
                        }
                };
                load_group(0);
                // the scales: this row's four weight blocks (one word of the 128-row x 4-block tile) and, as floats in this warp's
                // table, its activation rows' (index HALF_ROWS blk + row): HALF_ROWS / 8 per lane
                const uint32_t raw = smem_base + s * RAW_BYTES;
                const uint32_t sw = lds32_i8i(raw + RAW_W + RAW_A + (uint32_t)((t & 31) * 16 + (t >> 5) * 4));
                // rows past N and past M carry whatever their padding holds: they must not send the warp down the slow path
                uint32_t big = row_valid && (((sw & 0xFFu) >= 233u) | (((sw >> 8) & 0xFFu) >= 233u) | (((sw >> 16) & 0xFFu) >= 233u) | ((sw >> 24) >= 233u)) ? 1u : 0u;
#pragma unroll
                for (int h = 0; h < HALF_ROWS / 8; ++h) {
                    const int idx = lane + 32 * h, blk = idx / HALF_ROWS, mr = idx % HALF_ROWS, m = HALF_ROWS * hm + mr;
                    const uint32_t byte = (lds32_i8i(raw + RAW_W + RAW_A + SF + a_word(m)) >> (8 * blk)) & 0xFFu;
                    big |= (m < p.M && byte >= 233u) ? 1u : 0u;
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(table + 4u * idx), "f"(int8_mult(byte)) : "memory");
                }
                const bool any_big = __any_sync(0xffffffffu, big != 0u);
                __syncwarp();                          // orders the table's writes before its reads
                if (!any_big && lane == 0) mbar_arrive(raw_empty(s));     // the scales are in a register and in the table: the stage may go
#pragma unroll
                for (int g0 = 0; g0 < 4; g0 += G) {
                    if (g0 != 0) load_group(g0);
                    tc_wait_ld();
                    if (g0 + G == 4) {                 // the last of the buffer has been read
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(p_empty(b));
                    }
                    if (!any_big) {
                        float fa[G][HALF_ROWS];            // the group's activation scales, all loads issued before the first use
#pragma unroll
                        for (int gb = 0; gb < G; ++gb)
#pragma unroll
                            for (int m4 = 0; m4 < HALF_ROWS / 4; ++m4)
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                             : "=f"(fa[gb][4 * m4]), "=f"(fa[gb][4 * m4 + 1]), "=f"(fa[gb][4 * m4 + 2]), "=f"(fa[gb][4 * m4 + 3])
                                             : "r"(table + 4u * (uint32_t)(HALF_ROWS * (g0 + gb) + 4 * m4)));
#pragma unroll
                        for (int gb = 0; gb < G; ++gb) {
                            // S 2^(Ew-6) without an integer-to-float conversion (a quarter-rate instruction): 2^23 + 2^22 + S is a float
                            // whose bits are 0x4B400000 + S, and one fma takes it to S fw exactly (|S| < 2^19, fw < 2^100)
                            const float fw = int8_mult((sw >> (8 * (g0 + gb))) & 0xFFu), off = -12582912.0f * fw;
#pragma unroll
                            for (int m = 0; m < HALF_ROWS; ++m) {
                                const float sf = fmaf(__uint_as_float(0x4B400000u + r[gb][m]), fw, off);
                                acc[m] = fmaf(sf, fa[gb][m], acc[m]);       // one rounding per block, in K order
                            }
                        }
                    } else {
                        // a scale of 2^100 or more somewhere: the two exponents are added as integers and applied in two halves, so
                        // that nothing leaves fp32's range on the way unless the product itself does
#pragma unroll
                        for (int gb = 0; gb < G; ++gb)
#pragma unroll
                            for (int m = 0; m < HALF_ROWS; ++m) {
                                const uint32_t sa = lds32_i8i(raw + RAW_W + RAW_A + SF + a_word(HALF_ROWS * hm + m));
                                const int e = (int)((sa >> (8 * (g0 + gb))) & 0xFFu) + (int)((sw >> (8 * (g0 + gb))) & 0xFFu) - 266;   // -127 - 6, twice
                                const int e_hi = e >> 1;
                                acc[m] = fmaf((float)(int)r[gb][m] * pow2_int(e_hi), pow2_int(e - e_hi), acc[m]);
                            }
                    }
                }
                __syncwarp();                          // the table may be written again
                if (any_big && lane == 0) mbar_arrive(raw_empty(s));      // the slow path read the stage's scale tile to the end
            }
            if (!ok) break;
            if (row_valid) {
                const int64_t n = (int64_t)tile * BLOCK_W + t;
                const float cn = p.c != nullptr ? p.c[n] : 0.f;
#pragma unroll
                for (int m = 0; m < HALF_ROWS; ++m)
                    if (HALF_ROWS * hm + m < p.M) p.out[(int64_t)(HALF_ROWS * hm + m) * p.ldo + n] = acc[m] + cn;
            }
        }
    }
    // teardown: if any wait gave up, let copies still in flight land before shared memory goes away
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) tmem_dealloc(tmem_base, i8i::TMEM_COLS);
}

bool mxint8_gemm_decode_i8_tc_supported(const MxGemmArgs& a) {
    return a.fmt == FMT_INT8 && a.M > 0 && a.M <= 64 && a.K > 0 && a.K % 128 == 0 && a.N > 0 && a.N < (1ll << 30) &&
           a.K < (1ll << 30);
}

template <int ROWS>
static cudaError_t launch_i8_rows(const MxGemmArgs& a, cudaStream_t st) {
    using namespace i8i;
    using C = Cfg<ROWS>;
    CUtensorMap tm_w, tm_a;
    if (!make_tensor_map_2d(&tm_w, a.w_codes, 0, (uint64_t)a.K, (uint64_t)a.N, (uint64_t)a.K, 128, BLOCK_W) ||
        !make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K, 128, ROWS))
        return cudaErrorInvalidValue;
    Mxint8DecodeI8Params p;
    p.a_scales = a.a_scales; p.w_scales = a.w_scales; p.c = a.c;
    p.out = a.out; p.ldo = a.ldo;
    p.M = (int)a.M; p.N = (int)a.N; p.num_kb = (int)(a.K / 128);
    p.sf_kt_total = (int)sf_k_tiles(a.K);
    p.n_tiles = (int)((a.N + BLOCK_W - 1) / BLOCK_W);
    p.status = a.status;
    auto kern = mxint8_gemm_decode_i8_tc_kernel<ROWS>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(p.n_tiles < sms ? p.n_tiles : sms);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = C::SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, tm_w, tm_a, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mxint8_gemm_decode_i8_tc(const MxGemmArgs& a, cudaStream_t st) {
    if (a.M <= 16) return launch_i8_rows<16>(a, st);
    if (a.M <= 32) return launch_i8_rows<32>(a, st);
    if (a.M <= 48) return launch_i8_rows<48>(a, st);
    return launch_i8_rows<64>(a, st);
}

}  // namespace latmix
