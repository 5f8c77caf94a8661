// Kernels of the transformation-MSE diagnostic (Eq. "q_error" and the block-wise error E_B^i of Sec. 3.1):
//   e = x - T^-1(Q(T(x))) = (y - Q(y)) A^-1,   E = mean e^2,   E_B^i = mean over rows and over the B coordinates of block i.
//   * dequant_diff_kernel   d = y - dq(codes, scales): the quantisation error in the transformed domain
//   * quant_error_block_kernel  d = y - Q_B(y) for a block size other than the layer's 32 (the sweep over block sizes)
//   * block_sumsq_kernel    fp64 sums of squares per block of B coordinates, fixed summation order
// The product d A^-1 between the two is the fold-mode tensor-core product (transform_quant_pair_tc.cu) or the fp32 FMA one.
#include "internal.h"
#include "mx_math.cuh"

namespace latmix {

// One thread = 8 consecutive elements of a row; scales in the linear layout [rows][K/32].
template <int FMT>
__global__ void __launch_bounds__(256) dequant_diff_kernel(const float* __restrict__ Y, const uint8_t* __restrict__ codes,
                                                           const uint8_t* __restrict__ scales, int64_t M, int64_t K,
                                                           float* __restrict__ D) {
    const int64_t per_row = K >> 3;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < M * per_row; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / per_row, k0 = (t - row * per_row) << 3;
        const float s = scale_to_float(scales[row * (K >> 5) + (k0 >> 5)]);
        uint32_t c[8];
        if (FMT == FMT_FP4) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(codes + row * (K >> 1) + (k0 >> 1));
#pragma unroll
            for (int i = 0; i < 8; ++i) c[i] = (w >> (4 * i)) & 0xFu;
        } else {
            const uint2 w = *reinterpret_cast<const uint2*>(codes + row * K + k0);
#pragma unroll
            for (int i = 0; i < 4; ++i) { c[i] = (w.x >> (8 * i)) & 0xFFu; c[4 + i] = (w.y >> (8 * i)) & 0xFFu; }
        }
        const float4* y = reinterpret_cast<const float4*>(Y + row * K + k0);
        const float4 y0 = y[0], y1 = y[1];
        float4 d0, d1;
        d0.x = y0.x - decode_element<FMT>(c[0]) * s; d0.y = y0.y - decode_element<FMT>(c[1]) * s;
        d0.z = y0.z - decode_element<FMT>(c[2]) * s; d0.w = y0.w - decode_element<FMT>(c[3]) * s;
        d1.x = y1.x - decode_element<FMT>(c[4]) * s; d1.y = y1.y - decode_element<FMT>(c[5]) * s;
        d1.z = y1.z - decode_element<FMT>(c[6]) * s; d1.w = y1.w - decode_element<FMT>(c[7]) * s;
        float4* d = reinterpret_cast<float4*>(D + row * K + k0);
        d[0] = d0; d[1] = d1;
    }
}

cudaError_t launch_dequant_diff(const float* Y, const uint8_t* codes, const uint8_t* scales, int64_t M, int64_t K, int fmt,
                                float* D, cudaStream_t st) {
    const int64_t work = M * (K >> 3);
    const unsigned grid = (unsigned)((work + 255) / 256 < 148 * 16 ? (work + 255) / 256 : 148 * 16);
    if (fmt == FMT_FP4) dequant_diff_kernel<FMT_FP4><<<grid, 256, 0, st>>>(Y, codes, scales, M, K, D);
    else if (fmt == FMT_FP8 || fmt == FMT_INT4) dequant_diff_kernel<FMT_FP8><<<grid, 256, 0, st>>>(Y, codes, scales, M, K, D);
    else dequant_diff_kernel<FMT_INT8><<<grid, 256, 0, st>>>(Y, codes, scales, M, K, D);
    count_launch();
    return cudaGetLastError();
}

// d = y - Q_B(y) for an MX block size B of 8, 16, 32, 64 or 128 (the block-size sweep of the numerical analysis in Sec. 3.1):
// a thread = 8 consecutive elements, B / 8 neighbouring lanes = one block; Eq. "q_mx" with the element conversions of the
// quantiser, the codes decoded again at once.
template <int FMT>
__global__ void __launch_bounds__(256) quant_error_block_kernel(const float* __restrict__ Y, int64_t M, int64_t K, int block,
                                                                float* __restrict__ D) {
    const int64_t per_row = K >> 3, total = M * per_row;
    const int lanes = block >> 3;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x; base < total; base += stride) {      // whole warps take part in the shuffles
        const int64_t t = base + threadIdx.x;
        const bool active = t < total;
        const int64_t row = active ? t / per_row : 0, k0 = active ? (t - row * per_row) << 3 : 0;
        float v[8], y[8];
        if (active) {
            const float4* src = reinterpret_cast<const float4*>(Y + row * K + k0);
            const float4 a = src[0], c = src[1];
            y[0] = a.x; y[1] = a.y; y[2] = a.z; y[3] = a.w; y[4] = c.x; y[5] = c.y; y[6] = c.z; y[7] = c.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) y[i] = 0.f;
        }
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(y[i]));
        for (int o = 1; o < lanes; o <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const uint32_t sb = scale_byte_from_amax(amax, FormatTraits<FMT>::kRMax);
        const float2 f = inv_scale_factors(sb);
        const float s = scale_to_float(sb);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (y[i] * f.x) * f.y;
        uint32_t c[8];
        if (FMT == FMT_FP4) {
            const uint32_t w = pack8_fp4(v);
#pragma unroll
            for (int i = 0; i < 8; ++i) c[i] = (w >> (4 * i)) & 0xFu;
        } else {
            const uint2 w = pack8_bytes<FMT>(v);
#pragma unroll
            for (int i = 0; i < 4; ++i) { c[i] = (w.x >> (8 * i)) & 0xFFu; c[4 + i] = (w.y >> (8 * i)) & 0xFFu; }
        }
        if (active) {
            float4* d = reinterpret_cast<float4*>(D + row * K + k0);
            d[0] = make_float4(y[0] - decode_element<FMT>(c[0]) * s, y[1] - decode_element<FMT>(c[1]) * s,
                               y[2] - decode_element<FMT>(c[2]) * s, y[3] - decode_element<FMT>(c[3]) * s);
            d[1] = make_float4(y[4] - decode_element<FMT>(c[4]) * s, y[5] - decode_element<FMT>(c[5]) * s,
                               y[6] - decode_element<FMT>(c[6]) * s, y[7] - decode_element<FMT>(c[7]) * s);
        }
    }
}

cudaError_t launch_quant_error_block(const float* Y, int64_t M, int64_t K, int fmt, int block, float* D, cudaStream_t st) {
    const int64_t work = M * (K >> 3);
    const unsigned grid = (unsigned)((work + 255) / 256 < 148 * 16 ? (work + 255) / 256 : 148 * 16);
    if (fmt == FMT_FP4) quant_error_block_kernel<FMT_FP4><<<grid, 256, 0, st>>>(Y, M, K, block, D);
    else if (fmt == FMT_FP8) quant_error_block_kernel<FMT_FP8><<<grid, 256, 0, st>>>(Y, M, K, block, D);
    else if (fmt == FMT_INT4) quant_error_block_kernel<FMT_INT4><<<grid, 256, 0, st>>>(Y, M, K, block, D);
    else quant_error_block_kernel<FMT_INT8><<<grid, 256, 0, st>>>(Y, M, K, block, D);
    count_launch();
    return cudaGetLastError();
}

// Block i of `block` coordinates: thread t sums the squares of rows t, t + 256, ... in fp64; the 256 partial sums are added
// pairwise in a fixed order.  block_err[i] = sum / (block M).
__global__ void __launch_bounds__(256) block_sumsq_kernel(const float* __restrict__ E, int64_t M, int64_t K, int block,
                                                          double* __restrict__ block_err) {
    __shared__ double part[256];
    const int64_t k0 = (int64_t)blockIdx.x * block;
    double s = 0.0;
    for (int64_t m = threadIdx.x; m < M; m += 256) {
        const float4* e = reinterpret_cast<const float4*>(E + m * K + k0);
        double r = 0.0;
        for (int j = 0; j < (block >> 2); ++j) {
            const float4 v = e[j];
            r += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
        }
        s += r;
    }
    part[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_err[blockIdx.x] = part[0] / ((double)block * (double)M);
}

// mse = mean of the block errors (every block has the same number of elements), summed in index order
__global__ void mean_of_blocks_kernel(const double* __restrict__ block_err, int64_t nblocks, double* __restrict__ mse) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double s = 0.0;
    for (int64_t i = 0; i < nblocks; ++i) s += block_err[i];
    *mse = s / (double)nblocks;
}

cudaError_t launch_block_sumsq(const float* E, int64_t M, int64_t K, int block, double* block_err, double* mse, cudaStream_t st) {
    block_sumsq_kernel<<<(unsigned)(K / block), 256, 0, st>>>(E, M, K, block, block_err);
    mean_of_blocks_kernel<<<1, 32, 0, st>>>(block_err, K / block, mse);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace latmix
