// Issue-rate probe of the tensor pipes: every SM issues MMAs back to back on operands that already sit in shared
// memory, so neither HBM nor L2 nor an epilogue takes part.  What it measures is the ceiling the contractions of the
// layer are compared with: kind::f16 (the affine transform), kind::mxf8f6f4 and kind::mxf4 (the block-scaled product),
// kind::mxf4nvf4 (the same product with blocks of 16 and E4M3 scales).  The operands are a fixed byte pattern of
// moderate, finite values; the results are not read.
#include "internal.h"
#include "tc_common.cuh"

namespace latmix {

using namespace tc;

constexpr int kProbeThreads = 128;
constexpr int kProbeA = 128 * 128, kProbeB = 256 * 128, kProbeSf = 3 * 512;    // one 128-byte K slab of A (128 rows) and B (256 rows)
constexpr int kProbeSmem = 200 * 1024;      // far more than needed: one CTA per SM, whatever the scheduler would like

template <int KIND>
__global__ void __launch_bounds__(kProbeThreads, 1) tensor_pipe_probe_kernel(long long mma_per_cta, uint32_t* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sf_base = smem_base + kProbeA + kProbeB, bar = sf_base + kProbeSf, tmem_slot = bar + 8;
    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // codes: bytes 0x38 .. 0x3F (finite in every element format read here); scales: 1.0 in the kind's scale format
    for (int i = threadIdx.x; i < (kProbeA + kProbeB) / 4; i += kProbeThreads)
        reinterpret_cast<uint32_t*>(smem_gen)[i] = 0x38383838u | ((uint32_t)(i * 2654435761u) & 0x07070707u);
    for (int i = threadIdx.x; i < kProbeSf / 4; i += kProbeThreads)
        reinterpret_cast<uint32_t*>(smem_gen + kProbeA + kProbeB)[i] = KIND == 3 ? 0x38383838u : 0x7F7F7F7Fu;
    if (threadIdx.x == 0) { mbar_init(bar, 1); fence_mbar_init(); }
    fence_proxy_async_smem();                      // the tensor core reads what these threads wrote
    if (warp_idx == 0) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    if (warp_idx == 1 && lane == 0) {
        const uint32_t sfa_t = tmem_base + 256, sfb_t = tmem_base + 260;
        if (KIND != 0) {
            tc_cp_scale_lean(sfa_t, desc_lo(sf_base));
            tc_cp_scale_lean(sfb_t, desc_lo(sf_base + 512));
            tc_cp_scale_lean(sfb_t + 4, desc_lo(sf_base + 1024));
        }
        const uint32_t a_lo = desc_lo(smem_base), b_lo = desc_lo(smem_base + kProbeA);
        constexpr uint32_t kIdBf16 = make_idesc_bf16(128, 256, 0, 0);
        constexpr uint32_t kIdMx = make_idesc_block_scaled(128, 256, KIND == 1 ? 0u : 1u);
        constexpr uint32_t kIdNv = kIdMx & ~(1u << 23);           // scale format: E4M3
        for (long long i = 0; i < mma_per_cta; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {                          // four K steps of the 128-byte slab
                const uint32_t accum = (i | j) != 0;
                if (KIND == 0) mma_bf16_lean(tmem_base, a_lo + 2 * j, b_lo + 2 * j, kIdBf16, accum);
                else if (KIND == 1) mma_mxf8_lean(tmem_base, a_lo + 2 * j, b_lo + 2 * j, kIdMx | ((uint32_t)j << 4) | ((uint32_t)j << 29), sfa_t, sfb_t, accum);
                else if (KIND == 2) mma_mxf4_lean(tmem_base, a_lo + 2 * j, b_lo + 2 * j, (j & 1) ? (kIdMx | (2u << 4) | (2u << 29)) : kIdMx, sfa_t, sfb_t, accum);
                else mma_nvf4_lean(tmem_base, a_lo + 2 * j, b_lo + 2 * j, kIdNv, sfa_t, sfb_t, accum);
            }
        }
        tc_commit(bar);
        mbar_wait(bar, 0, status);
    }
    tc_fence_before();
    __syncthreads();
    if (warp_idx == 0) tmem_dealloc(tmem_base, 512);
}

// The same probe on a CTA pair: one 256 x 256 x 64 kind::mxf4 MMA per step (cta_group::2), each CTA holding its 128 rows of
// A and half of the rows of B; the leader issues, both tensor cores work.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kProbeThreads, 1) tensor_pipe_probe_pair_kernel(long long mma_per_pair, int commit_every, uint32_t* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    constexpr int kA = 128 * 128, kBhalf = 128 * 128;
    const uint32_t sf_base = smem_base + kA + kBhalf, bar = sf_base + kProbeSf, tmem_slot = bar + 8, bar2 = bar + 16;
    const int warp_idx = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool leader = cluster_ctarank() == 0;
    for (int i = threadIdx.x; i < (kA + kBhalf) / 4; i += kProbeThreads)
        reinterpret_cast<uint32_t*>(smem_gen)[i] = 0x38383838u | ((uint32_t)(i * 2654435761u) & 0x07070707u);
    for (int i = threadIdx.x; i < kProbeSf / 4; i += kProbeThreads)
        reinterpret_cast<uint32_t*>(smem_gen + kA + kBhalf)[i] = 0x7F7F7F7Fu;
    if (threadIdx.x == 0) { mbar_init(bar, 1); mbar_init(bar2, 1); fence_mbar_init(); }
    fence_proxy_async_smem();
    if (warp_idx == 0) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem_gen + (tmem_slot - smem_base));
    if (leader && warp_idx == 1 && lane == 0) {
        const uint32_t sfa_t = tmem_base + 256, sfb_t = tmem_base + 260;
        tc_cp_scale_pair_lean(sfa_t, desc_lo(sf_base));
        tc_cp_scale_pair_lean(sfb_t, desc_lo(sf_base + 512));
        tc_cp_scale_pair_lean(sfb_t + 4, desc_lo(sf_base + 1024));
        const uint32_t a_lo = desc_lo(smem_base), b_lo = desc_lo(smem_base + kA);
        constexpr uint32_t kIdMx = make_idesc_block_scaled(256, 256, 1u);
        for (long long i = 0; i < mma_per_pair; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                mma_mxf4_pair_lean(tmem_base, a_lo + 2 * j, b_lo + 2 * j, (j & 1) ? (kIdMx | (2u << 4) | (2u << 29)) : kIdMx, sfa_t, sfb_t, (i | j) != 0);
            // a commit every so many MMAs, as a pipelined kernel issues them to release its stages (nobody waits on this one)
            if (commit_every > 0 && (i + 4) % commit_every == 0) tc_commit_pair(bar2, 1);
        }
        tc_commit_pair(bar, 1);
        mbar_wait(bar, 0, status);
    }
    tc_fence_before();
    cluster_sync_all();                 // the peer's shared and tensor memory stay until the leader's MMAs are done
    if (warp_idx == 0) tmem_dealloc_pair(tmem_base, 512);
}

}  // namespace latmix

using namespace latmix;

extern "C" latmix_status_t latmix_tensor_pipe_probe(int kind_and_interval, int64_t mma_per_cta, double* flops, void* workspace,
                                                    size_t workspace_bytes, void* cuda_stream) {
    const int kind = kind_and_interval & 0xFF, commit_every = (kind_and_interval >> 8) & 0xFFFF;
    if (commit_every != 0 && (kind != 4 || commit_every % 4 != 0)) return LATMIX_ERR_INVALID_ARG;
    if (kind < 0 || kind > 4 || mma_per_cta < 4 || mma_per_cta > (1ll << 22) || flops == nullptr) return LATMIX_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return LATMIX_ERR_WORKSPACE;
    int dev = 0, major = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (major != 10) return LATMIX_ERR_UNSUPPORTED;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long n = mma_per_cta / 4 * 4;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint32_t* status = static_cast<uint32_t*>(workspace);
    cudaError_t e = cudaSuccess;
#define LATMIX_PROBE(KIND)                                                                                              \
    do {                                                                                                                \
        e = cudaFuncSetAttribute(tensor_pipe_probe_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem); \
        if (e == cudaSuccess) tensor_pipe_probe_kernel<KIND><<<sms, kProbeThreads, kProbeSmem, st>>>(n, status);        \
    } while (0)
    if (kind == 0) LATMIX_PROBE(0); else if (kind == 1) LATMIX_PROBE(1); else if (kind == 2) LATMIX_PROBE(2); else if (kind == 3) LATMIX_PROBE(3);
    else {
        e = cudaFuncSetAttribute(tensor_pipe_probe_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem);
        sms = 2 * resident_cta_pairs((const void*)tensor_pipe_probe_pair_kernel, kProbeThreads, kProbeSmem);
        if (e == cudaSuccess) tensor_pipe_probe_pair_kernel<<<sms, kProbeThreads, kProbeSmem, st>>>(n, commit_every, status);
    }
#undef LATMIX_PROBE
    if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return LATMIX_ERR_CUDA;
    count_launch();
    const double k_per_mma = kind == 0 ? 16.0 : kind == 1 ? 32.0 : 64.0;
    *flops = 2.0 * 128.0 * 256.0 * k_per_mma * (double)n * (double)sms;
    return LATMIX_OK;
}
