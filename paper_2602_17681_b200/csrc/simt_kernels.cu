// CUDA-core kernels of the transformed MX-quantized linear layer:
//   * quantize_rows_kernel     -- Eq. "q_mx" on rows of X (+ b): the memory-bound standalone quantiser
//   * gemm_quant_simt_kernel   -- Y = P Q + b in fp32 FMA with the quantiser as epilogue
//                                 (fp32 transform inputs; offline fold W~^T = W^T A^-T, Eq. "fold_kqv_1")
//   * fold_bias kernels        -- c = bias - b A^-1 W with fp64 accumulation (and its output-side step c A_out + v)
//   * mx_gemm_simt_kernel      -- out = dq(Qa) dq(Qw)^T + c for any shape (small-M / fallback path)
#include "internal.h"
#include "mx_math.cuh"

namespace latmix {

// ----------------------------------------------------------------------------------------------------
// shared epilogue: 4 consecutive lanes own one MX block (8 values each)
// ----------------------------------------------------------------------------------------------------
template <int FMT>
__device__ __forceinline__ void quantize_block_by_4_lanes(float (&v)[8], bool active, int64_t row, int64_t k0,
                                                          int64_t K, uint8_t* codes, uint8_t* scales, int sf_layout,
                                                          uint32_t* status, uint32_t flags, int64_t rows_total) {
    if (FMT == FMT_NVFP4) {
        // a block of 16 = two neighbouring lanes: the even lane fetches its neighbour's eight values and quantises the block
        float w[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) { w[i] = v[i]; w[8 + i] = __shfl_down_sync(0xffffffffu, v[i], 1); }
        if ((flags & LATMIX_FLAG_CHECK_FINITE) && active) {
            bool bad = false;
#pragma unroll
            for (int i = 0; i < 8; ++i) bad |= !isfinite(v[i]);
            if (bad) atomicOr(status, 1u << LATMIX_ERR_NONFINITE);
        }
        if (!active || (k0 & 15) != 0) return;
        const float g = *nvfp4_tensor_scale_ptr(scales, rows_total, K, sf_layout);
        uint2 packed;
        const uint32_t d_code = nvfp4_quantize_block(w, g, packed);
        *reinterpret_cast<uint2*>(codes + row * (K >> 1) + (k0 >> 1)) = packed;
        const int64_t kb = k0 >> 4;
        scales[sf_layout == LATMIX_SF_LINEAR ? (size_t)(row * (K >> 4) + kb) : sf_tcgen05_offset(row, kb, nvfp4_sf_k_tiles(K))] = (uint8_t)d_code;
        return;
    }
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    if ((flags & LATMIX_FLAG_CHECK_FINITE) && active) {
        bool bad = false;
#pragma unroll
        for (int i = 0; i < 8; ++i) bad |= !isfinite(v[i]);
        if (bad) atomicOr(status, 1u << LATMIX_ERR_NONFINITE);
    }
    const uint32_t sb = scale_byte_from_amax(amax, FormatTraits<FMT == FMT_NVFP4 ? FMT_FP4 : FMT>::kRMax);
    const float2 f = inv_scale_factors(sb);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = (v[i] * f.x) * f.y;
    if (!active) return;
    if (FMT == FMT_FP4 || FMT == FMT_NVFP4) {
        *reinterpret_cast<uint32_t*>(codes + row * (K >> 1) + (k0 >> 1)) = pack8_fp4(v);
    } else {
        *reinterpret_cast<uint2*>(codes + row * K + k0) = pack8_bytes<FMT>(v);
    }
    if ((k0 & 31) == 0) {
        const int64_t kb = k0 >> 5;
        const size_t off = sf_layout == LATMIX_SF_LINEAR ? (size_t)(row * (K >> 5) + kb)
                                                         : sf_tcgen05_offset(row, kb, sf_k_tiles(K));
        scales[off] = (uint8_t)sb;
    }
}

// ----------------------------------------------------------------------------------------------------
// standalone quantiser
// ----------------------------------------------------------------------------------------------------
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p)), c = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {          // bf16 -> fp32 is a 16-bit shift
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// eight consecutive inputs of one lane as they come from memory (converted only when they are used, so that the
// loads of the next step can be in flight in few registers)
template <typename TIn> struct Raw8;
template <> struct Raw8<float> { float4 lo, hi; };
template <> struct Raw8<__nv_bfloat16> { uint4 w; };
__device__ __forceinline__ void load_raw8(const float* p, Raw8<float>& r) {
    r.lo = __ldg(reinterpret_cast<const float4*>(p)); r.hi = __ldg(reinterpret_cast<const float4*>(p) + 1);
}
__device__ __forceinline__ void load_raw8(const __nv_bfloat16* p, Raw8<__nv_bfloat16>& r) { r.w = __ldg(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void zero_raw8(Raw8<float>& r) { r.lo = r.hi = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void zero_raw8(Raw8<__nv_bfloat16>& r) { r.w = make_uint4(0u, 0u, 0u, 0u); }
__device__ __forceinline__ void unpack_raw8(const Raw8<float>& r, float (&v)[8]) {
    v[0] = r.lo.x; v[1] = r.lo.y; v[2] = r.lo.z; v[3] = r.lo.w; v[4] = r.hi.x; v[5] = r.hi.y; v[6] = r.hi.z; v[7] = r.hi.w;
}
__device__ __forceinline__ void unpack_raw8(const Raw8<__nv_bfloat16>& r, float (&v)[8]) {
    const uint32_t w[4] = {r.w.x, r.w.y, r.w.z, r.w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {          // bf16 -> fp32 is a 16-bit shift
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

template <int FMT, typename TIn, bool EXTRAS, bool FULL, bool TILED>
__global__ void __launch_bounds__(256, 4) quantize_rows_kernel(const TIn* __restrict__ X, const float* __restrict__ b,
                                                               int64_t M, int64_t K, uint8_t* __restrict__ codes,
                                                               uint8_t* __restrict__ scales, int sf_layout,
                                                               float* __restrict__ Y_dump, uint32_t* status, uint32_t flags) {
    const int lane = threadIdx.x & 31;
    // A warp covers 256 consecutive elements of a row per step (a lane = 8 elements, 4 lanes = one MX block), UNROLL
    // steps per iteration (64 bytes per lane in flight), and walks along the row; rows are dealt out to the warps.
    // The kernel is bound by instruction issue before it is bound by memory (at 17 instructions per element it reached
    // 60 % of the copy bandwidth with bf16 inputs), so everything that depends on the row only is computed once per row
    // and the lane's three pointers advance by constants: no multiplication and no 64-bit division in the loop.
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    constexpr int UNROLL = sizeof(TIn) == 2 ? 4 : 2;
    constexpr int CODE_SHIFT = FMT == FMT_FP4 ? 1 : 0;                 // two codes per byte
    constexpr bool linear = !TILED;                                    // the launcher picks the instance for sf_layout
    // EXTRAS: shift b, dump of the pre-quantisation values, non-finite check (the plain variant carries none of their
    // registers).  FULL: K is a multiple of the elements a warp covers per iteration, so no lane is ever past the row's end.
    const int64_t kt = sf_k_tiles(K);
    // scale bytes of this lane's block within a row: linear = block index; tiled = 512-byte tile per four blocks
    const int sf_lane = linear ? (lane >> 2) : (lane >> 4) * 512 + ((lane >> 2) & 3);
    constexpr int sf_step = linear ? 8 : 1024;                         // per 256 elements
    // The loads of the next iteration -- the next row's first ones included -- are issued before this iteration's values
    // are touched, so that a warp always has 64 bytes per lane in flight.
    int64_t row = warp0, k = lane * 8;
    Raw8<TIn> nxt[UNROLL];
    auto fetch = [&](const TIn* p, int64_t kk) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (FULL || kk + u * 256 < K) load_raw8(p + u * 256, nxt[u]); else zero_raw8(nxt[u]);
        }
    };
    const TIn* px = X + row * K + lane * 8;
    if (row < M) fetch(px, k);
    while (row < M) {
        uint8_t* pc = codes + ((row * K + k) >> CODE_SHIFT);
        uint8_t* ps = scales + (linear ? row * (K >> 5) : ((row >> 7) * kt) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4) + sf_lane;
        const int64_t cur_row = row;
        for (bool same_row = true; same_row; pc += (UNROLL * 256) >> CODE_SHIFT, ps += UNROLL * sf_step) {
            Raw8<TIn> raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) raw[u] = nxt[u];
            const int64_t k_cur = k;
            k += UNROLL * 256; px += UNROLL * 256;
            if (k - lane * 8 >= K) {                           // warp-uniform: on to this warp's next row
                same_row = false;
                row += n_warps; k = lane * 8;
                px = X + row * K + lane * 8;
            }
            if (row < M) fetch(px, k);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const bool active = FULL || k_cur + u * 256 < K;
                float v[8];
                unpack_raw8(raw[u], v);
                if (EXTRAS && active) {
                    if (b != nullptr) {
                        float bb[8];
                        load8(b + k_cur + u * 256, bb);
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] += bb[i];
                    }
                    if (Y_dump != nullptr) {
                        float4* d = reinterpret_cast<float4*>(Y_dump + cur_row * K + k_cur + u * 256);
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
                const uint32_t sb = scale_block_of_4_lanes<FMT>(v);
                if (active) {
                    if (FMT == FMT_FP4) *reinterpret_cast<uint32_t*>(pc + u * 128) = pack8_fp4(v);
                    else *reinterpret_cast<uint2*>(pc + u * 256) = pack8_bytes<FMT>(v);
                    if ((lane & 3) == 0) ps[u * sf_step] = (uint8_t)sb;
                }
            }
        }
    }
}

// NVFP4 (blocks of 16, E4M3 block scale, tensor scale from the scale buffer's trailer): a thread = one block.
template <typename TIn>
__global__ void __launch_bounds__(256) quantize_rows_nvfp4_kernel(const TIn* __restrict__ X, const float* __restrict__ b, int64_t M,
                                                                  int64_t K, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                                  int sf_layout, float* __restrict__ Y_dump, uint32_t* status,
                                                                  uint32_t flags) {
    const float g = *nvfp4_tensor_scale_ptr(scales, M, K, sf_layout);
    const int64_t nb = K >> 4, total = M * nb, kt = nvfp4_sf_k_tiles(K);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / nb, kb = i - row * nb, k0 = kb << 4;
        float v[16];
        load8(X + row * K + k0, *reinterpret_cast<float(*)[8]>(v));
        load8(X + row * K + k0 + 8, *reinterpret_cast<float(*)[8]>(v + 8));
        if (b != nullptr) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += b[k0 + j];
        }
        if (Y_dump != nullptr) {
            float4* d = reinterpret_cast<float4*>(Y_dump + row * K + k0);
#pragma unroll
            for (int j = 0; j < 4; ++j) d[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
        if (flags & LATMIX_FLAG_CHECK_FINITE) {
            bool bad = false;
#pragma unroll
            for (int j = 0; j < 16; ++j) bad |= !isfinite(v[j]);
            if (bad) atomicOr(status, 1u << LATMIX_ERR_NONFINITE);
        }
        uint2 packed;
        const uint32_t d_code = nvfp4_quantize_block(v, g, packed);
        *reinterpret_cast<uint2*>(codes + row * (K >> 1) + (k0 >> 1)) = packed;
        scales[sf_layout == LATMIX_SF_LINEAR ? (size_t)(row * nb + kb) : sf_tcgen05_offset(row, kb, kt)] = (uint8_t)d_code;
    }
}

cudaError_t launch_quantize_rows(const QuantArgs& a, cudaStream_t st) {
    if (a.M == 0 || a.K == 0) return cudaSuccess;
    if (a.fmt == FMT_NVFP4) {
        const int64_t total = a.M * (a.K >> 4);
        int64_t blocks = (total + 255) / 256;
        if (blocks > 148 * 16) blocks = 148 * 16;
        if (a.x_is_bf16)
            quantize_rows_nvfp4_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(a.X), a.b, a.M, a.K, a.codes, a.scales,
                                                                        a.sf_layout, a.Y_dump, a.status, a.flags);
        else
            quantize_rows_nvfp4_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<const float*>(a.X), a.b, a.M, a.K, a.codes, a.scales,
                                                                        a.sf_layout, a.Y_dump, a.status, a.flags);
        count_launch();
        return cudaGetLastError();
    }
    const int sms = sm_count();
    int64_t blocks = (a.M + 7) / 8;                             // one warp per row at a time
    if (blocks > (int64_t)sms * 4) blocks = (int64_t)sms * 4;   // persistent: 4 CTAs of 256 threads per SM, one wave
    dim3 grid((unsigned)blocks), block(256);
    const bool extras = a.b != nullptr || a.Y_dump != nullptr || (a.flags & LATMIX_FLAG_CHECK_FINITE);
    const bool tiled = a.sf_layout != LATMIX_SF_LINEAR;
#define LATMIX_LAUNCH_Q3(FMT, T, E, F, L)                                                                                  \
    quantize_rows_kernel<FMT, T, E, F, L><<<grid, block, 0, st>>>(static_cast<const T*>(a.X), a.b, a.M, a.K, a.codes,      \
                                                                   a.scales, a.sf_layout, a.Y_dump, a.status, a.flags)
#define LATMIX_LAUNCH_Q(FMT, T)                                                                                            \
    do {                                                                                                                   \
        const bool full = a.K % ((sizeof(T) == 2 ? 4 : 2) * 256) == 0;        /* the kernel's UNROLL x 256 */                \
        if (extras) { if (tiled) LATMIX_LAUNCH_Q3(FMT, T, true, false, true); else LATMIX_LAUNCH_Q3(FMT, T, true, false, false); } \
        else if (full) { if (tiled) LATMIX_LAUNCH_Q3(FMT, T, false, true, true); else LATMIX_LAUNCH_Q3(FMT, T, false, true, false); } \
        else { if (tiled) LATMIX_LAUNCH_Q3(FMT, T, false, false, true); else LATMIX_LAUNCH_Q3(FMT, T, false, false, false); } \
    } while (0)
    if (a.x_is_bf16) {
        if (a.fmt == FMT_FP4) LATMIX_LAUNCH_Q(FMT_FP4, __nv_bfloat16);
        else if (a.fmt == FMT_FP8) LATMIX_LAUNCH_Q(FMT_FP8, __nv_bfloat16);
        else if (a.fmt == FMT_INT4) LATMIX_LAUNCH_Q(FMT_INT4, __nv_bfloat16);
        else LATMIX_LAUNCH_Q(FMT_INT8, __nv_bfloat16);
    } else {
        if (a.fmt == FMT_FP4) LATMIX_LAUNCH_Q(FMT_FP4, float);
        else if (a.fmt == FMT_FP8) LATMIX_LAUNCH_Q(FMT_FP8, float);
        else if (a.fmt == FMT_INT4) LATMIX_LAUNCH_Q(FMT_INT4, float);
        else LATMIX_LAUNCH_Q(FMT_INT8, float);
    }
#undef LATMIX_LAUNCH_Q
#undef LATMIX_LAUNCH_Q3
    count_launch();
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// Block-diagonal online transform (the paper's T_3: blocks = MX blocks) fused with the quantiser.
// One thread owns one row's 32-element block: 32 inputs and 32 outputs in registers, the 32 x 32 block in shared
// memory (every thread of the CTA works on the same block column, so its rows are read as broadcasts).
// 64 flops per element against 2 bytes read: FMA-bound at about twice the time of a plain read of X.
// ----------------------------------------------------------------------------------------------------
template <int FMT, typename TIn>
__global__ void __launch_bounds__(128) blockdiag_quant_kernel(const TIn* __restrict__ X, const TIn* __restrict__ A_blocks,
                                                              const float* __restrict__ b, int64_t M, int64_t K,
                                                              uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                              int sf_layout, float* __restrict__ Y_dump, uint32_t* status,
                                                              uint32_t flags) {
    __shared__ __align__(16) float As[32][32];
    const int64_t kb = blockIdx.x, k0 = kb * 32;
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) As[i >> 5][i & 31] = load_as_float(A_blocks + kb * 1024 + i);
    __syncthreads();
    const int64_t kt = sf_k_tiles(K);
    for (int64_t row = (int64_t)blockIdx.y * blockDim.x + threadIdx.x; row < M; row += (int64_t)gridDim.y * blockDim.x) {
        float x[32], y[32];
#pragma unroll
        for (int g = 0; g < 4; ++g) load8(X + row * K + k0 + 8 * g, *reinterpret_cast<float(*)[8]>(x + 8 * g));
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float4 a = *reinterpret_cast<const float4*>(&As[i][4 * g]);
                y[4 * g] = fmaf(x[i], a.x, y[4 * g]);
                y[4 * g + 1] = fmaf(x[i], a.y, y[4 * g + 1]);
                y[4 * g + 2] = fmaf(x[i], a.z, y[4 * g + 2]);
                y[4 * g + 3] = fmaf(x[i], a.w, y[4 * g + 3]);
            }
        }
        if (b != nullptr) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float4 bb = __ldg(reinterpret_cast<const float4*>(b + k0) + g);
                y[4 * g] += bb.x; y[4 * g + 1] += bb.y; y[4 * g + 2] += bb.z; y[4 * g + 3] += bb.w;
            }
        }
        float amax = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(y[j]));
        if (Y_dump != nullptr) {
            float4* d = reinterpret_cast<float4*>(Y_dump + row * K + k0);
#pragma unroll
            for (int g = 0; g < 8; ++g) d[g] = make_float4(y[4 * g], y[4 * g + 1], y[4 * g + 2], y[4 * g + 3]);
        }
        if ((flags & LATMIX_FLAG_CHECK_FINITE) && !isfinite(amax)) atomicOr(status, 1u << LATMIX_ERR_NONFINITE);
        const uint32_t sb = scale_byte_from_amax(amax, FormatTraits<FMT>::kRMax);
        const float2 f = inv_scale_factors(sb);
#pragma unroll
        for (int j = 0; j < 32; ++j) y[j] = (y[j] * f.x) * f.y;
        if (FMT == FMT_FP4) {
            *reinterpret_cast<uint4*>(codes + row * (K >> 1) + (k0 >> 1)) =
                make_uint4(pack8_fp4(y), pack8_fp4(y + 8), pack8_fp4(y + 16), pack8_fp4(y + 24));
        } else {
            uint2 w0, w1, w2, w3;
            w0 = pack8_bytes<FMT>(y); w1 = pack8_bytes<FMT>(y + 8); w2 = pack8_bytes<FMT>(y + 16); w3 = pack8_bytes<FMT>(y + 24);
            uint4* d = reinterpret_cast<uint4*>(codes + row * K + k0);
            d[0] = make_uint4(w0.x, w0.y, w1.x, w1.y);
            d[1] = make_uint4(w2.x, w2.y, w3.x, w3.y);
        }
        scales[sf_layout == LATMIX_SF_LINEAR ? (size_t)(row * (K >> 5) + kb) : sf_tcgen05_offset(row, kb, kt)] = (uint8_t)sb;
    }
}

cudaError_t launch_blockdiag_quant(const QuantArgs& a, const void* A_blocks, cudaStream_t st) {
    if (a.M == 0 || a.K == 0) return cudaSuccess;
    const int sms = sm_count();
    // about ten CTAs per SM in total; each CTA keeps its block column and walks down the rows
    int64_t gy = (a.M + 127) / 128, cap = ((int64_t)sms * 10 + a.K / 32 - 1) / (a.K / 32);
    if (gy > cap) gy = cap < 1 ? 1 : cap;
    dim3 grid((unsigned)(a.K / 32), (unsigned)gy), block(128);
#define LATMIX_LAUNCH_BD(FMT, T)                                                                                    \
    blockdiag_quant_kernel<FMT, T><<<grid, block, 0, st>>>(static_cast<const T*>(a.X), static_cast<const T*>(A_blocks), \
                                                            a.b, a.M, a.K, a.codes, a.scales, a.sf_layout, a.Y_dump, \
                                                            a.status, a.flags)
    if (a.x_is_bf16 && !(a.flags & LATMIX_FLAG_FORCE_SIMT) && blockdiag_quant_mma_supported(a)) {
        return launch_blockdiag_quant_mma(a, A_blocks, st);
    } else if (a.x_is_bf16) {
        if (a.fmt == FMT_FP4) LATMIX_LAUNCH_BD(FMT_FP4, __nv_bfloat16);
        else if (a.fmt == FMT_FP8) LATMIX_LAUNCH_BD(FMT_FP8, __nv_bfloat16);
        else if (a.fmt == FMT_INT4) LATMIX_LAUNCH_BD(FMT_INT4, __nv_bfloat16);
        else LATMIX_LAUNCH_BD(FMT_INT8, __nv_bfloat16);
    } else {
        if (a.fmt == FMT_FP4) LATMIX_LAUNCH_BD(FMT_FP4, float);
        else if (a.fmt == FMT_FP8) LATMIX_LAUNCH_BD(FMT_FP8, float);
        else if (a.fmt == FMT_INT4) LATMIX_LAUNCH_BD(FMT_INT4, float);
        else LATMIX_LAUNCH_BD(FMT_INT8, float);
    }
#undef LATMIX_LAUNCH_BD
    count_launch();
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// fp32 FMA product + quantiser epilogue.  Tile 64 x 64, reduction step 16, 256 threads, 4 x 4 per thread.
// ----------------------------------------------------------------------------------------------------
constexpr int GQ_BM = 64, GQ_BN = 64, GQ_BK = 16;

template <int FMT, typename TP, typename TQ, bool P_KCONTIG, bool Q_KCONTIG>
__global__ void __launch_bounds__(256) gemm_quant_simt_kernel(const TP* __restrict__ P, int64_t p_rs, int64_t p_ks,
                                                              const TQ* __restrict__ Q, int64_t q_ks, int64_t q_cs,
                                                              const float* __restrict__ b, int64_t R, int64_t C,
                                                              int64_t Kred, uint8_t* __restrict__ codes,
                                                              uint8_t* __restrict__ scales, int sf_layout,
                                                              float* __restrict__ Y_dump, uint32_t* status,
                                                              uint32_t flags) {
    __shared__ float Ps[GQ_BK][GQ_BM + 4];
    __shared__ float Qs[GQ_BK][GQ_BN + 4];
    __shared__ float Ys[GQ_BM][GQ_BN + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t r0 = (int64_t)blockIdx.y * GQ_BM, c0 = (int64_t)blockIdx.x * GQ_BN;
    float acc[4][4] = {};
    for (int64_t k0 = 0; k0 < Kred; k0 += GQ_BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int r, k;
            if (P_KCONTIG) { r = tid >> 2; k = (tid & 3) * 4 + i; } else { k = tid >> 4; r = (tid & 15) * 4 + i; }
            const int64_t gr = r0 + r, gk = k0 + k;
            Ps[k][r] = (gr < R && gk < Kred) ? load_as_float(P + gr * p_rs + gk * p_ks) : 0.f;
            int c;
            if (Q_KCONTIG) { c = tid >> 2; k = (tid & 3) * 4 + i; } else { k = tid >> 4; c = (tid & 15) * 4 + i; }
            const int64_t gc = c0 + c, gk2 = k0 + k;
            Qs[k][c] = (gc < C && gk2 < Kred) ? load_as_float(Q + gk2 * q_ks + gc * q_cs) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < GQ_BK; ++k) {
            float p[4], q[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { p[i] = Ps[k][ty * 4 + i]; q[i] = Qs[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(p[i], q[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t gc = c0 + tx * 4 + j;
            Ys[ty * 4 + i][tx * 4 + j] = acc[i][j] + ((b != nullptr && gc < C) ? b[gc] : 0.f);
        }
    __syncthreads();
    // 64 rows x 2 blocks = 128 block tasks, 4 lanes each -> 2 rounds of 256 threads
#pragma unroll
    for (int round = 0; round < 2; ++round) {
        const int task = round * 64 + (tid >> 2);       // 0..127
        const int r = task >> 1, blk = task & 1, part = tid & 3;
        const int64_t gr = r0 + r, gk = c0 + blk * 32 + part * 8;
        const bool active = gr < R && gk < C;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = Ys[r][blk * 32 + part * 8 + i];
        if (active && Y_dump != nullptr) {
#pragma unroll
            for (int i = 0; i < 8; ++i) Y_dump[gr * C + gk + i] = v[i];
        }
        if (!active) {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
        quantize_block_by_4_lanes<FMT>(v, active, gr, gk, C, codes, scales, sf_layout, status, flags, R);
    }
}

template <int FMT, typename TP, typename TQ>
static void launch_gq(const GemmQuantArgs& a, cudaStream_t st) {
    dim3 grid((unsigned)((a.C + GQ_BN - 1) / GQ_BN), (unsigned)((a.R + GQ_BM - 1) / GQ_BM)), block(256);
    const bool pk = a.p_k_stride == 1, qk = a.q_k_stride == 1;
#define LATMIX_GQ(PK, QK)                                                                                         \
    gemm_quant_simt_kernel<FMT, TP, TQ, PK, QK><<<grid, block, 0, st>>>(                                           \
        static_cast<const TP*>(a.P), a.p_row_stride, a.p_k_stride, static_cast<const TQ*>(a.Q), a.q_k_stride,      \
        a.q_col_stride, a.b, a.R, a.C, a.Kred, a.codes, a.scales, a.sf_layout, a.Y_dump, a.status, a.flags)
    if (pk && qk) LATMIX_GQ(true, true);
    else if (pk) LATMIX_GQ(true, false);
    else if (qk) LATMIX_GQ(false, true);
    else LATMIX_GQ(false, false);
#undef LATMIX_GQ
}

template <int FMT>
static void launch_gq_fmt(const GemmQuantArgs& a, cudaStream_t st) {
    if (a.p_is_bf16 && a.q_is_bf16) launch_gq<FMT, __nv_bfloat16, __nv_bfloat16>(a, st);
    else if (a.p_is_bf16) launch_gq<FMT, __nv_bfloat16, float>(a, st);
    else if (a.q_is_bf16) launch_gq<FMT, float, __nv_bfloat16>(a, st);
    else launch_gq<FMT, float, float>(a, st);
}

cudaError_t launch_gemm_quant_simt(const GemmQuantArgs& a, cudaStream_t st) {
    if (a.R == 0 || a.C == 0) return cudaSuccess;
    if (a.fmt == FMT_FP4) launch_gq_fmt<FMT_FP4>(a, st);
    else if (a.fmt == FMT_FP8) launch_gq_fmt<FMT_FP8>(a, st);
    else if (a.fmt == FMT_INT4) launch_gq_fmt<FMT_INT4>(a, st);
    else if (a.fmt == FMT_NVFP4) launch_gq_fmt<FMT_NVFP4>(a, st);
    else launch_gq_fmt<FMT_INT8>(a, st);
    count_launch();
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// c = bias - (b A_inv) W, fp64 accumulation
// ----------------------------------------------------------------------------------------------------
// One block = 8 consecutive columns x 32 slices of the rows: thread (slice, column) sums its rows in fp64, the 32 partial
// sums of a column are added in a fixed order.  A warp reads 4 rows x 32 bytes per load; the column sums of a 4096-row
// matrix take 32 dependent steps per thread instead of 4096.
__device__ __forceinline__ double as_double(float v) { return (double)v; }
__device__ __forceinline__ double as_double(double v) { return v; }
__device__ __forceinline__ double as_double(__nv_bfloat16 v) { return (double)__bfloat162float(v); }

template <typename TX, typename TM>
__device__ __forceinline__ double column_dot(const TX* __restrict__ x, const TM* __restrict__ mat, int64_t rows, int64_t cols,
                                             int64_t col, int slice, double (*part)[8]) {
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    if (x != nullptr && col < cols) {
        int64_t k = slice;
        for (; k + 96 < rows; k += 128) {
            s0 += as_double(x[k]) * as_double(mat[k * cols + col]);
            s1 += as_double(x[k + 32]) * as_double(mat[(k + 32) * cols + col]);
            s2 += as_double(x[k + 64]) * as_double(mat[(k + 64) * cols + col]);
            s3 += as_double(x[k + 96]) * as_double(mat[(k + 96) * cols + col]);
        }
        for (; k < rows; k += 32) s0 += as_double(x[k]) * as_double(mat[k * cols + col]);
    }
    part[slice][threadIdx.x & 7] = (s0 + s1) + (s2 + s3);
    __syncthreads();
    double s = 0.0;
    if (slice == 0)
        for (int i = 0; i < 32; ++i) s += part[i][threadIdx.x & 7];
    return s;                                  // meaningful in slice 0 only
}

// u[j] = sum_k b[k] A_inv[k][j]
__global__ void __launch_bounds__(256) fold_bias_u_kernel(const float* __restrict__ A_inv, const float* __restrict__ b, int64_t K,
                                                          double* __restrict__ u) {
    __shared__ double part[32][8];
    const int64_t j = (int64_t)blockIdx.x * 8 + (threadIdx.x & 7);
    const double s = column_dot(b, A_inv, K, K, j, threadIdx.x >> 3, part);
    if ((threadIdx.x >> 3) == 0 && j < K) u[j] = s;
}

// c[n] = bias[n] - sum_j u[j] W[j][n]
template <typename TW>
__global__ void __launch_bounds__(256) fold_bias_c_kernel(const double* __restrict__ u, const TW* __restrict__ W,
                                                          const float* __restrict__ bias, int64_t K, int64_t N, float* __restrict__ c) {
    __shared__ double part[32][8];
    const int64_t n = (int64_t)blockIdx.x * 8 + (threadIdx.x & 7);
    const double s = column_dot(u, W, K, N, n, threadIdx.x >> 3, part);
    if ((threadIdx.x >> 3) == 0 && n < N) c[n] = (float)((bias != nullptr ? (double)bias[n] : 0.0) - s);
}

cudaError_t launch_fold_bias(const float* A_inv, const float* b, const void* W, int w_is_bf16, const float* bias,
                             int64_t K, int64_t N, double* u_tmp, float* c_out, cudaStream_t st) {
    fold_bias_u_kernel<<<(unsigned)((K + 7) / 8), 256, 0, st>>>(A_inv, b, K, u_tmp);
    if (w_is_bf16)
        fold_bias_c_kernel<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(u_tmp, static_cast<const __nv_bfloat16*>(W), bias, K, N, c_out);
    else
        fold_bias_c_kernel<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(u_tmp, static_cast<const float*>(W), bias, K, N, c_out);
    count_launch(2);
    return cudaGetLastError();
}

// Output-side part of the two-sided fold's bias: c[n] = sum_j c1[j] A_out[j][n] + v_out[n], fp64 accumulation.
__global__ void __launch_bounds__(256) fold_bias_out_kernel(const float* __restrict__ c1, const float* __restrict__ A_out,
                                                            const float* __restrict__ v_out, int64_t N, float* __restrict__ c) {
    __shared__ double part[32][8];
    const int64_t n = (int64_t)blockIdx.x * 8 + (threadIdx.x & 7);
    const double s = column_dot(c1, A_out, N, N, n, threadIdx.x >> 3, part);
    if ((threadIdx.x >> 3) == 0 && n < N) c[n] = (float)((v_out != nullptr ? (double)v_out[n] : 0.0) + s);
}

cudaError_t launch_fold_bias_out(const float* c1, const float* A_out, const float* v_out, int64_t N, float* c_out,
                                 cudaStream_t st) {
    fold_bias_out_kernel<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(c1, A_out, v_out, N, c_out);
    count_launch();
    return cudaGetLastError();
}

// ----------------------------------------------------------------------------------------------------
// CUDA-core block-scaled product.  One warp per output column n, up to 16 rows of activations at a time:
// lane l owns MX block (kb0 + l) of the weight row (16 or 32 bytes of codes + one scale byte), so weight
// bytes are read once per 16 activation rows, coalesced.
// ----------------------------------------------------------------------------------------------------
template <int FMT>
__device__ __forceinline__ void decode32(const uint8_t* p, float scale, float (&w)[32]) {
    if (FMT == FMT_FP4) {
        const uint4 r = *reinterpret_cast<const uint4*>(p);
        const uint32_t q[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 32; ++i) w[i] = decode_element<FMT_FP4>((q[i >> 3] >> (4 * (i & 7))) & 0xFu) * scale;
    } else {
        const uint4 r0 = *reinterpret_cast<const uint4*>(p), r1 = *(reinterpret_cast<const uint4*>(p) + 1);
        const uint32_t q[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int i = 0; i < 32; ++i) w[i] = decode_element<FMT>((q[i >> 2] >> (8 * (i & 3))) & 0xFFu) * scale;
    }
}

constexpr int SG_ROWS = 8;   // activation rows per pass

template <int FMT>
__global__ void __launch_bounds__(256) mx_gemm_simt_kernel(const uint8_t* __restrict__ a_codes, const uint8_t* __restrict__ a_scales,
                                                           const uint8_t* __restrict__ w_codes, const uint8_t* __restrict__ w_scales,
                                                           const float* __restrict__ c, int64_t M, int64_t K, int64_t N,
                                                           float* __restrict__ out, int64_t ldo) {
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const int64_t nkb = K >> 5, kt = sf_k_tiles(K);
    const int64_t row_bytes = FMT == FMT_FP4 ? (K >> 1) : K;
    constexpr int kBlockBytes = FMT == FMT_FP4 ? 16 : 32;
    for (int64_t m0 = (int64_t)blockIdx.y * SG_ROWS; m0 < M; m0 += (int64_t)gridDim.y * SG_ROWS) {
        float acc[SG_ROWS];
#pragma unroll
        for (int i = 0; i < SG_ROWS; ++i) acc[i] = 0.f;
        for (int64_t kb = lane; kb < nkb; kb += 32) {
            float w[32];
            decode32<FMT>(w_codes + n * row_bytes + kb * kBlockBytes, scale_to_float(w_scales[sf_tcgen05_offset(n, kb, kt)]), w);
#pragma unroll
            for (int i = 0; i < SG_ROWS; ++i) {
                const int64_t m = m0 + i;
                if (m < M) {
                    float x[32];
                    decode32<FMT>(a_codes + m * row_bytes + kb * kBlockBytes, scale_to_float(a_scales[sf_tcgen05_offset(m, kb, kt)]), x);
                    float s = 0.f;
#pragma unroll
                    for (int t = 0; t < 32; ++t) s = fmaf(x[t], w[t], s);
                    acc[i] += s;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < SG_ROWS; ++i) {
            float s = acc[i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0 && m0 + i < M) out[(m0 + i) * ldo + n] = s + (c != nullptr ? c[n] : 0.f);
        }
    }
}

// NVFP4 on the CUDA cores: one warp per output column, a lane per block of 16; out = (ga gw) sum + c.
__global__ void __launch_bounds__(256) nvfp4_gemm_simt_kernel(const uint8_t* __restrict__ a_codes, const uint8_t* __restrict__ a_scales,
                                                              const uint8_t* __restrict__ w_codes, const uint8_t* __restrict__ w_scales,
                                                              const float* __restrict__ ga, const float* __restrict__ gw,
                                                              const float* __restrict__ c, int64_t M, int64_t K, int64_t N,
                                                              float* __restrict__ out, int64_t ldo) {
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const int64_t nkb = K >> 4, kt = nvfp4_sf_k_tiles(K), row_bytes = K >> 1;
    const float g = *ga * *gw;
    for (int64_t m = blockIdx.y; m < M; m += gridDim.y) {
        float acc = 0.f;
        for (int64_t kb = lane; kb < nkb; kb += 32) {
            const uint2 wq = *reinterpret_cast<const uint2*>(w_codes + n * row_bytes + kb * 8);
            const uint2 aq = *reinterpret_cast<const uint2*>(a_codes + m * row_bytes + kb * 8);
            const uint32_t ww[2] = {wq.x, wq.y}, aw[2] = {aq.x, aq.y};
            float s = 0.f;
#pragma unroll
            for (int t = 0; t < 16; ++t)
                s = fmaf(decode_element<FMT_FP4>((aw[t >> 3] >> (4 * (t & 7))) & 0xFu), decode_element<FMT_FP4>((ww[t >> 3] >> (4 * (t & 7))) & 0xFu), s);
            acc = fmaf(s, decode_element<FMT_FP8>(a_scales[sf_tcgen05_offset(m, kb, kt)]) * decode_element<FMT_FP8>(w_scales[sf_tcgen05_offset(n, kb, kt)]), acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) out[m * ldo + n] = fmaf(acc, g, c != nullptr ? c[n] : 0.f);
    }
}

cudaError_t launch_mx_gemm_simt(const MxGemmArgs& a, cudaStream_t st) {
    if (a.M == 0 || a.N == 0) return cudaSuccess;
    if (a.fmt == FMT_NVFP4) {
        dim3 grid((unsigned)((a.N + 7) / 8), (unsigned)(a.M < 1024 ? a.M : 1024));
        nvfp4_gemm_simt_kernel<<<grid, 256, 0, st>>>(a.a_codes, a.a_scales, a.w_codes, a.w_scales, a.a_tensor_scale, a.w_tensor_scale, a.c,
                                                     a.M, a.K, a.N, a.out, a.ldo);
        count_launch();
        return cudaGetLastError();
    }
    int64_t gy = (a.M + SG_ROWS - 1) / SG_ROWS;
    if (gy > 512) gy = 512;
    dim3 grid((unsigned)((a.N + 7) / 8), (unsigned)gy), block(256);
    if (a.fmt == FMT_FP4)
        mx_gemm_simt_kernel<FMT_FP4><<<grid, block, 0, st>>>(a.a_codes, a.a_scales, a.w_codes, a.w_scales, a.c, a.M, a.K, a.N, a.out, a.ldo);
    else if (a.fmt == FMT_FP8 || a.fmt == FMT_INT4)      // MXINT4 codes are E4M3 bytes
        mx_gemm_simt_kernel<FMT_FP8><<<grid, block, 0, st>>>(a.a_codes, a.a_scales, a.w_codes, a.w_scales, a.c, a.M, a.K, a.N, a.out, a.ldo);
    else
        mx_gemm_simt_kernel<FMT_INT8><<<grid, block, 0, st>>>(a.a_codes, a.a_scales, a.w_codes, a.w_scales, a.c, a.M, a.K, a.N, a.out, a.ldo);
    count_launch();
    return cudaGetLastError();
}

}  // namespace latmix
