// MXINT8 product for small batches (M <= 16):  out[M x N] = dq(Qa) dq(Qw)^T + c, without scratch memory.
//
// No block-scaled tcgen05 kind takes 8-bit integers, but k 2^(E-6), |k| <= 127, is exact in bf16.  The general path expands
// both operands to bf16 in scratch memory first; with a handful of activation rows that triples the bytes moved (read the
// int8 weights, write them as bf16, read them again) for a product that is bound by reading the weights once.  Here the
// expansion happens on the way from shared memory to the tensor core:
//   warp 0    producer: per 128-deep K slab the int8 weight tile (128 rows x 128 bytes), the int8 activation tile (16 rows),
//             and the two 512-byte scale tiles, into a ring of ten raw stages
//   warps 2-17 converters, two groups of eight warps that take alternate slabs (a thread = two MX blocks of one weight
//             row): int8 -> k 2^(E-6) as bf16 (exactly).  The converted WEIGHTS go into tensor memory (tcgen05.st: a thread's
//             row is its lane, a 32-bit column holds two consecutive K elements), from where the MMA reads its 128-row
//             operand; only the 16 activation rows go back to shared memory (two 64-deep K-major bf16 slabs, 128-byte
//             swizzle), which leaves shared memory for a ring of ten raw stages.  The first four warps also run the
//             epilogue of the tile.  Measured at 4096 x 14336, M = 16 (26 us): loads alone 14.7 us, + the handshakes and
//             the MMAs 19.4, + the conversion arithmetic 26; with the weights written back to shared memory instead
//             (103 KB of shared-memory traffic per slab) the same 26, with six tensor-memory stages the same: per slab
//             the eight N = 16 MMAs cost their issuing thread about 600 cycles, the conversion about 700 of issue slots,
//             the copies 870, and the three do not overlap fully
//   warp 1    tcgen05.mma kind::f16, eight per slab: the 128 rows of the MMA are weight rows (read from tensor memory), its
//             N side the 16 activation rows (operands swapped as in the small-batch block-scaled kernel)
// Products are exact, accumulation is the tensor core's fp32, as on every other path.  Every wait is bounded.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace i8d {
constexpr int BLOCK_W = 128, ROWS = 16;
constexpr int RAW_W = BLOCK_W * 128, RAW_A = ROWS * 128, SF = 512;
constexpr int RAW_BYTES = RAW_W + RAW_A + 2 * SF;                  // 19 KiB
constexpr int RAW_STAGES = 10;
constexpr int CONV_A = 2 * ROWS * 128;                             // two 64-deep bf16 slabs of the activations
constexpr int CONV_BYTES = CONV_A;                                 // 4 KiB: the converted weights live in tensor memory
constexpr int CONV_STAGES = 3;
constexpr int BAR_BYTES = 256;
constexpr int SMEM_BYTES = 1024 + RAW_STAGES * RAW_BYTES + CONV_STAGES * CONV_BYTES + BAR_BYTES;
constexpr int ACC_COLS = 32, W_COLS = 64;                          // accumulator; one slab of converted weights (128 K as bf16 pairs)
constexpr int TMEM_COLS = 256;                                     // 32 + 3 x 64 = 224, rounded up to a power of two
constexpr int CONV_WARPS = 16, THREADS = (2 + CONV_WARPS) * 32;
static_assert(RAW_BYTES % 1024 == 0 && CONV_BYTES % 1024 == 0 && SMEM_BYTES <= 227 * 1024, "shared memory layout");
static_assert(ACC_COLS + CONV_STAGES * W_COLS <= TMEM_COLS && 8 * (2 * RAW_STAGES + 2 * CONV_STAGES + 3) <= BAR_BYTES, "tensor memory and barrier area");
}  // namespace i8d

struct Mxint8DecodeParams {
    const uint8_t* a_scales; const uint8_t* w_scales; const float* c;
    float* out; int64_t ldo;
    int M, N, num_kb /* 128-deep slabs */, sf_kt_total, n_tiles;
    uint32_t* status;
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__global__ void __launch_bounds__(i8d::THREADS, 1)
mxint8_gemm_decode_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a,
                             const Mxint8DecodeParams p) {
    using namespace i8d;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t conv_base = smem_base + RAW_STAGES * RAW_BYTES;
    const uint32_t bar_base = conv_base + CONV_STAGES * CONV_BYTES;
    auto raw_full = [&](int s) { return bar_base + 8u * s; };
    auto raw_empty = [&](int s) { return bar_base + 8u * (RAW_STAGES + s); };
    auto conv_full = [&](int s) { return bar_base + 8u * (2 * RAW_STAGES + s); };
    auto conv_empty = [&](int s) { return bar_base + 8u * (2 * RAW_STAGES + CONV_STAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * RAW_STAGES + 2 * CONV_STAGES);
    const uint32_t tmem_slot = tfull_bar + 8u;
    const uint32_t tempty_bar = tfull_bar + 16u;                     // the four epilogue warps have read the accumulator
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp_idx == 0 && lane == 0) {
        prefetch_tmap(&tm_w); prefetch_tmap(&tm_a);
        for (int s = 0; s < RAW_STAGES; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), CONV_WARPS / 2); }
        for (int s = 0; s < CONV_STAGES; ++s) { mbar_init(conv_full(s), CONV_WARPS / 2); mbar_init(conv_empty(s), 1); }
        mbar_init(tfull_bar, 1); mbar_init(tempty_bar, 4);
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
            constexpr uint32_t kIdesc = make_idesc_bf16(BLOCK_W, ROWS, 0, 0);            // both operands K-major
            uint32_t it = 0, tiles_done = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++tiles_done) {
                // the first MMA of a tile overwrites the accumulator: the epilogue warps must have read the tile before (the
                // converter group that prepares this tile's first slab need not be the one that holds them)
                if (tiles_done > 0) {
                    ok = mbar_wait(tempty_bar, (tiles_done - 1u) & 1u, p.status);
                    tc_fence_after();
                }
                for (int kb = 0; kb < p.num_kb && ok; ++kb, ++it) {
                    const int s = it % CONV_STAGES;
                    if (!(ok = mbar_wait(conv_full(s), (it / CONV_STAGES) & 1u, p.status))) break;
                    tc_fence_after();
                    const uint32_t st = conv_base + s * CONV_BYTES, w_t = tmem_base + ACC_COLS + s * W_COLS;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {      // eight K = 16 steps: eight columns of weight pairs each
                        const uint32_t b_lo = desc_lo(st + (j >> 2) * (ROWS * 128) + (j & 3) * 32);
                        mma_bf16_tmem_a_lean(tmem_base, w_t + 8 * j, b_lo, kIdesc, (uint32_t)((kb | j) != 0));
                    }
                    tc_commit(conv_empty(s));
                }
                tc_commit(tfull_bar);                  // also when a wait gave up: the epilogue must not wait in vain
            }
        }
    } else {
        // ------------------------------------------------------------------ converters (warps 2..17) + epilogue (warps 2..5)
        const int cw = warp_idx - 2;
        const int grp = cw >> 3;                       // group 0 converts the even slabs of the launch, group 1 the odd ones
        const int q = warp_idx & 3;                    // tensor-memory lane quarter this warp may touch
        const int t = q * 32 + lane;                   // weight row this thread converts = its tensor-memory lane ...
        const int bp = (cw >> 2) & 1;                  // ... and which two of its four MX blocks (chunks 4 bp .. 4 bp + 3)
        const int ta = (cw & 3) * 32 + lane;           // activations: thread index within the group's first four warps
        const int am = ta >> 3, ac = ta & 7;           // activation row and 16-byte chunk (those warps only)
        uint32_t it = 0, tile_count = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++tile_count) {
            for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                if ((int)(it & 1u) != grp) continue;   // the other group's slab
                const int rs = it % RAW_STAGES, cs = it % CONV_STAGES;
                // one lane polls (512 polling threads would crowd the barriers the copies and commits complete on)
                if (lane == 0)
                    ok = mbar_wait(raw_full(rs), (it / RAW_STAGES) & 1u, p.status) &&
                         mbar_wait(conv_empty(cs), ((it / CONV_STAGES) & 1u) ^ 1u, p.status);
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const uint32_t raw = smem_base + rs * RAW_BYTES, conv = conv_base + cs * CONV_BYTES;
                // weights: row t; scale bytes of its four blocks are one word of the 128-row x 4-block tile
                {
                    const uint32_t sw = lds32(raw + RAW_W + RAW_A + (uint32_t)((t & 31) * 16 + (t >> 5) * 4));
                    const uint32_t row_in = raw + (uint32_t)t * 128u, sz = (uint32_t)(t & 7);
                    const uint32_t sb0 = (sw >> (16 * bp)) & 0xFFu, sb1 = (sw >> (16 * bp + 8)) & 0xFFu;
                    const float mult0 = int8_mult(sb0), mult1 = int8_mult(sb1);
                    // scales of 2^100 and above take the converter's two-step form; one vote keeps the common path free of it
                    const bool any_big = __any_sync(0xffffffffu, sb0 >= 233u || sb1 >= 233u);
                    uint32_t r[32];                    // 64 elements = 32 columns of bf16 pairs, in K order
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {   // chunk c = elements 16c .. 16c + 15, block c / 2, read from c ^ (row & 7)
                        const int c = 4 * bp + cc;
                        const float mult = cc < 2 ? mult0 : mult1;
                        const uint4 v = lds128(row_in + (((uint32_t)c ^ sz) << 4));
                        uint4 lo, hi;
                        if (!any_big) int8x16_to_bf16_impl<false>(v, mult, lo, hi);
                        else int8x16_to_bf16(v, mult, lo, hi);
                        r[8 * cc] = lo.x; r[8 * cc + 1] = lo.y; r[8 * cc + 2] = lo.z; r[8 * cc + 3] = lo.w;
                        r[8 * cc + 4] = hi.x; r[8 * cc + 5] = hi.y; r[8 * cc + 6] = hi.z; r[8 * cc + 7] = hi.w;
                    }
                    // this thread's row is its tensor-memory lane; columns [32 bp, 32 bp + 32) of the slab's weight buffer
                    tc_st_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + ACC_COLS + (uint32_t)cs * W_COLS + (uint32_t)bp * 32u, r);
                }
                // activations: 16 rows x 8 chunks, one chunk per thread of the group's first four warps
                if (bp == 0) {
                    const uint32_t sa = lds32(raw + RAW_W + RAW_A + SF + (uint32_t)(am * 16));      // rows 0..15 of the first row group
                    const uint32_t sz = (uint32_t)(am & 7);
                    const uint4 v = lds128(raw + RAW_W + (uint32_t)am * 128u + (((uint32_t)ac ^ sz) << 4));
                    uint4 lo, hi;
                    int8x16_to_bf16(v, int8_mult((sa >> (8 * (ac >> 1))) & 0xFFu), lo, hi);
                    const uint32_t row_out = conv + (uint32_t)(ac >> 2) * (ROWS * 128) + (uint32_t)am * 128u;
                    const uint32_t oc = (uint32_t)(ac & 3) * 2u;
                    sts128(row_out + ((oc ^ sz) << 4), lo);
                    sts128(row_out + (((oc + 1u) ^ sz) << 4), hi);
                }
                tc_wait_st();                          // the weights are in tensor memory ...
                tc_fence_before();
                fence_proxy_async_smem();              // ... the activations in shared memory before the tensor core reads them; the raw reads before the next copy
                __syncwarp();
                if (lane == 0) { mbar_arrive(conv_full(cs)); mbar_arrive(raw_empty(rs)); }
            }
            if (!ok) break;
            if (cw >= 4) continue;                     // the other converter warps go on to the next tile
            // epilogue of the tile: a thread = output column n, the activation rows along its registers
            ok = mbar_wait(tfull_bar, tile_count & 1u, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t r[32];
            tc_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16), r);     // columns 16..31 are not part of the accumulator
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
            const int64_t n = (int64_t)tile * BLOCK_W + q * 32 + lane;
            if (n < p.N) {
                const float cn = p.c != nullptr ? p.c[n] : 0.f;
#pragma unroll
                for (int m = 0; m < ROWS; ++m)
                    if (m < p.M) p.out[(int64_t)m * p.ldo + n] = __uint_as_float(r[m]) + cn;
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
    if (warp_idx == 1) tmem_dealloc(tmem_base, i8d::TMEM_COLS);
}

bool mxint8_gemm_decode_tc_supported(const MxGemmArgs& a) {
    return a.fmt == FMT_INT8 && a.M > 0 && a.M <= i8d::ROWS && a.K > 0 && a.K % 128 == 0 && a.N > 0 && a.N < (1ll << 30) &&
           a.K < (1ll << 30);
}

cudaError_t launch_mxint8_gemm_decode_tc(const MxGemmArgs& a, cudaStream_t st) {
    using namespace i8d;
    CUtensorMap tm_w, tm_a;
    if (!make_tensor_map_2d(&tm_w, a.w_codes, 0, (uint64_t)a.K, (uint64_t)a.N, (uint64_t)a.K, 128, BLOCK_W) ||
        !make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)a.K, (uint64_t)a.M, (uint64_t)a.K, 128, ROWS))
        return cudaErrorInvalidValue;
    Mxint8DecodeParams p;
    p.a_scales = a.a_scales; p.w_scales = a.w_scales; p.c = a.c;
    p.out = a.out; p.ldo = a.ldo;
    p.M = (int)a.M; p.N = (int)a.N; p.num_kb = (int)(a.K / 128);
    p.sf_kt_total = (int)sf_k_tiles(a.K);
    p.n_tiles = (int)((a.N + BLOCK_W - 1) / BLOCK_W);
    p.status = a.status;
    cudaError_t e = set_max_dynamic_smem((const void*)mxint8_gemm_decode_tc_kernel, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(p.n_tiles < sms ? p.n_tiles : sms);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, mxint8_gemm_decode_tc_kernel, tm_w, tm_a, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace latmix
