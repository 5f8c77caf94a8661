// Block-scaled MX GEMM for small batches (M <= 64, the decode regime):  out[M x N] = dq(Qa) dq(Qw)^T + c.
//
// With a handful of activation rows the product is bound by streaming the weights once.  The roles of the operands are
// therefore swapped: the 128 rows of the MMA are WEIGHT rows, its N side (16, 32, 48 or 64 columns) the activation
// rows, so that a stage of the ring holds 16 KB of weights and only 2-8 KB of activations (the general kernel spends
// half of every stage on a 128-row activation tile that is mostly padding).  Two K slabs per stage (one wait and one commit
// per eight MMAs), five stages for M <= 16, four up to M = 64: 160 KB of weights in flight per SM.  A tile ALONE (14 CTAs
// instead of 112) takes 12.9 us whatever the ring (2 x 4, 4 x 2, 5 x 2 slabs), however many warps issue the copies, and
// with the scale copies moved off the MMA thread (12.1 us): about 5 us are launch, descriptor fetch, first-byte latency and
// the epilogue tail, the rest is 608 KB through one SM's 64 B/clk port from L2.  112 tiles side by side are then bound by
// DRAM: 15.4 us against 9.3 us + those 5.
//   warp 0    producer: TMA loads of the weight slab (128 rows x 128 bytes) and the activation slab, bulk copies of the
//             two scale tiles
//   warp 1    tcgen05.cp of the scales, four tcgen05.mma .block_scale per slab into a 128-lane x N accumulator
//   warps 2-5 epilogue: tcgen05.ld (a thread = one weight row n, the activation rows m along the columns), + c[n],
//             stores out[m][n]: for every m a warp writes 32 consecutive n, no transposition needed
// Every wait is bounded.  Products of element values and power-of-two scales are exact; accumulation is fp32.
#include "internal.h"
#include "mx_math.cuh"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

namespace dec {
constexpr int BLOCK_W = 128;                       // weight rows per tile
constexpr int W_BYTES = BLOCK_W * 128, SF_BYTES = 1024;           // SF_BYTES per scale operand: up to 2 k-tiles
constexpr int SLABS = 2;                           // K slabs per stage
constexpr int NUM_ACC = 2;
constexpr int BAR_BYTES = 1024;
constexpr int TMEM_COLS = 256;
constexpr int SF_COLS = SLABS * 16;                // per buffer and slab: 2 k-tiles x 4 columns for each operand
template <int MAX_ACT_>                            // activation rows (MMA N) at most: 16 or 64
struct Cfg {
    static constexpr int MAX_ACT = MAX_ACT_;
    static constexpr int ACT_BYTES = MAX_ACT * 128;
    static constexpr int SLAB_BYTES = W_BYTES + ACT_BYTES + 2 * SF_BYTES;   // 20 KiB / 26 KiB
    static constexpr int STAGE_BYTES = SLABS * SLAB_BYTES;
    static constexpr int STAGES = (227 * 1024 - 1024 - BAR_BYTES) / STAGE_BYTES;   // 5 / 4
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + BAR_BYTES;
    static constexpr int ACC_COLS = NUM_ACC * MAX_ACT;
    static_assert(ACC_COLS + 2 * SF_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert(STAGES >= 3 && SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(SLAB_BYTES % 1024 == 0, "operand tiles must stay 1024-byte aligned");
};
}  // namespace dec

struct MxGemmDecodeParams {
    const uint8_t* a_scales; const uint8_t* w_scales; const float* c;
    float* out; int64_t ldo;
    int M, N, n_mma, num_kb, stages_per_tile, sf_kt_total, n_tiles;     // stages_per_tile = ceil(num_kb / SLABS)
    uint32_t* status;
};

template <int FMT, int MAX_ACT>
__global__ void __launch_bounds__(192, 1)
mx_gemm_decode_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_a,
                         const MxGemmDecodeParams p) {
    using namespace dec;
    using C = Cfg<MAX_ACT>;
    constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, SLAB_BYTES = C::SLAB_BYTES, ACT_BYTES = C::ACT_BYTES;
    constexpr int ACC_COLS = C::ACC_COLS;
    constexpr int SF_KT = FMT == FMT_FP4 ? 2 : 1;                // scale k-tiles (4 blocks each) per 128-byte K slab
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
        prefetch_tmap(&tm_w); prefetch_tmap(&tm_a);
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
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
        // (Spreading the four copies of a slab over three issuing warps changed nothing: 13.0 us for a tile alone either way.)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t slab_tx = (uint32_t)(W_BYTES + p.n_mma * 128 + 2 * SF_KT * 512);
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
                for (int stg = 0; stg < p.stages_per_tile; ++stg, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(empty_bar(s), ph ^ 1u, p.status))) break;
                    const int slabs = min(SLABS, p.num_kb - stg * SLABS);                // an odd count leaves the last stage half full
                    mbar_expect_tx(full_bar(s), (uint32_t)slabs * slab_tx);
                    for (int h = 0; h < slabs; ++h) {
                        const int kb = stg * SLABS + h;
                        const uint32_t st = smem_base + s * STAGE_BYTES + h * SLAB_BYTES;
                        tma_load_2d(st, &tm_w, kb * 128, tile * BLOCK_W, full_bar(s));   // rows past N read as zero
                        tma_load_2d(st + W_BYTES, &tm_a, kb * 128, 0, full_bar(s));      // box = n_mma rows; rows past M read as zero
                        bulk_load(st + W_BYTES + ACT_BYTES,
                                  p.w_scales + ((size_t)tile * p.sf_kt_total + (size_t)kb * SF_KT) * 512, SF_KT * 512, full_bar(s));
                        bulk_load(st + W_BYTES + ACT_BYTES + SF_BYTES, p.a_scales + (size_t)kb * SF_KT * 512, SF_KT * 512, full_bar(s));
                    }
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            const uint32_t idesc0 = make_idesc_block_scaled(BLOCK_W, p.n_mma, FMT == FMT_FP4 ? 1u : 0u);
            uint32_t it = 0, tile_count = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++tile_count) {
                const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
                if (!(ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, p.status))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * MAX_ACT;
                for (int stg = 0; stg < p.stages_per_tile; ++stg, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!(ok = mbar_wait(full_bar(s), ph, p.status))) break;
                    tc_fence_after();
                    const int slabs = min(SLABS, p.num_kb - stg * SLABS);
                    // scale buffers alternate by stage: the copies of stage i+1 must not overwrite what the MMAs of stage i read
                    const uint32_t sf_t = tmem_base + ACC_COLS + (it & 1u) * SF_COLS;
                    for (int h = 0; h < slabs; ++h) {
                        const uint32_t lo = desc_lo(smem_base + s * STAGE_BYTES + h * SLAB_BYTES);
                        const uint32_t sfw_lo = lo + ((W_BYTES + ACT_BYTES) >> 4), sfa_lo = sfw_lo + (SF_BYTES >> 4);
                        const uint32_t sfw_t = sf_t + h * 16, sfa_t = sfw_t + 8;
#pragma unroll
                        for (int kt = 0; kt < SF_KT; ++kt) {
                            tc_cp_scale_lean(sfw_t + kt * 4, sfw_lo + kt * 32);
                            tc_cp_scale_lean(sfa_t + kt * 4, sfa_lo + kt * 32);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {     // four MMAs, each 32 bytes of K per row
                            const int kt = FMT == FMT_FP4 ? (j >> 1) : 0;
                            const uint32_t sf_id = FMT == FMT_FP4 ? (uint32_t)(j & 1) * 2u : (uint32_t)j;
                            const uint32_t idesc = idesc0 | (sf_id << 4) | (sf_id << 29);
                            const uint32_t accum = (uint32_t)((stg | h | j) != 0);
                            // the MMA's "A" operand (128 rows) is the weight slab, its "B" operand the activation slab
                            if (FMT == FMT_FP4) mma_mxf4_lean(d_tmem, lo + 2 * j, lo + (W_BYTES >> 4) + 2 * j, idesc, sfw_t + kt * 4, sfa_t + kt * 4, accum);
                            else mma_mxf8_lean(d_tmem, lo + 2 * j, lo + (W_BYTES >> 4) + 2 * j, idesc, sfw_t + kt * 4, sfa_t + kt * 4, accum);
                        }
                    }
                    tc_commit(empty_bar(s));
                }
                if (ok) tc_commit(tfull_bar(acc));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp_idx & 3;                     // tensor-memory lane quarter this warp may read
        uint32_t tile_count = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++tile_count) {
            const uint32_t acc = tile_count % NUM_ACC, acc_ph = (tile_count / NUM_ACC) & 1u;
            ok = mbar_wait(tfull_bar(acc), acc_ph, p.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int64_t n = (int64_t)tile * BLOCK_W + q * 32 + lane;     // this thread's output column
            const float cn = (p.c != nullptr && n < p.N) ? p.c[n] : 0.f;
#pragma unroll 1
            for (int chunk = 0; chunk * 32 < p.n_mma; ++chunk) {
                uint32_t r[32];
                tc_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * MAX_ACT + chunk * 32, r);
                tc_wait_ld();
                if (n < p.N) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int m = chunk * 32 + i;
                        if (m < p.M) p.out[(int64_t)m * p.ldo + n] = __uint_as_float(r[i]) + cn;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(acc));
        }
    }
    // teardown: if any wait gave up, let copies still in flight land before shared memory goes away
    if (*reinterpret_cast<volatile uint32_t*>(p.status) & (1u << LATMIX_ERR_TIMEOUT)) {
        const long long t0 = clock64();
        while (clock64() - t0 < (1ll << 22)) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) tmem_dealloc(tmem_base, dec::TMEM_COLS);
}

// ----------------------------------------------------------------------------------------------------
bool mx_gemm_decode_tc_supported(const MxGemmArgs& a) {
    if (a.fmt == FMT_FP4) { if (a.K % 256 != 0) return false; }
    else if (a.fmt == FMT_FP8) { if (a.K % 128 != 0) return false; }
    else return false;
    return a.M > 0 && a.M <= 64 && a.K > 0 && a.N > 0 && a.N < (1ll << 30) && a.K < (1ll << 30);
}

template <int FMT, int MAX_ACT>
static cudaError_t launch_decode_fmt(const MxGemmArgs& a, cudaStream_t st) {
    using namespace dec;
    constexpr int SMEM_BYTES = Cfg<MAX_ACT>::SMEM_BYTES;
    const int64_t k_bytes = a.fmt == FMT_FP4 ? a.K / 2 : a.K;
    const int n_mma = (int)((a.M + 15) / 16) * 16;
    CUtensorMap tm_w, tm_a;
    if (!make_tensor_map_2d(&tm_w, a.w_codes, 0, (uint64_t)k_bytes, (uint64_t)a.N, (uint64_t)k_bytes, 128, BLOCK_W) ||
        !make_tensor_map_2d(&tm_a, a.a_codes, 0, (uint64_t)k_bytes, (uint64_t)a.M, (uint64_t)k_bytes, 128, (uint32_t)n_mma))
        return cudaErrorInvalidValue;
    MxGemmDecodeParams p;
    p.a_scales = a.a_scales; p.w_scales = a.w_scales; p.c = a.c;
    p.out = a.out; p.ldo = a.ldo;
    p.M = (int)a.M; p.N = (int)a.N; p.n_mma = n_mma;
    p.num_kb = (int)(k_bytes / 128);
    p.stages_per_tile = (p.num_kb + SLABS - 1) / SLABS;
    p.sf_kt_total = (int)sf_k_tiles(a.K);
    p.n_tiles = (int)((a.N + BLOCK_W - 1) / BLOCK_W);
    p.status = a.status;
    auto kern = mx_gemm_decode_tc_kernel<FMT, MAX_ACT>;
    cudaError_t e = set_max_dynamic_smem((const void*)kern, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(p.n_tiles < sms ? p.n_tiles : sms);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;      // the kernel waits for its predecessor itself, after its set-up
    cfg.attrs = &attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, tm_w, tm_a, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_mx_gemm_decode_tc(const MxGemmArgs& a, cudaStream_t st) {
    if (a.M <= 16) return a.fmt == FMT_FP4 ? launch_decode_fmt<FMT_FP4, 16>(a, st) : launch_decode_fmt<FMT_FP8, 16>(a, st);
    return a.fmt == FMT_FP4 ? launch_decode_fmt<FMT_FP4, 64>(a, st) : launch_decode_fmt<FMT_FP8, 64>(a, st);
}

}  // namespace latmix
