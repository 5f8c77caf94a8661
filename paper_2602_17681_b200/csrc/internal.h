// Internal host-side interfaces between the translation units of liblatmix (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/latmix.h"

namespace latmix {

// The first 256 bytes of every workspace: word 0 is the device status (bitwise OR of 1 << latmix_status_t).
constexpr size_t kWorkspaceHeaderBytes = 256;
// Header layout: word 0 status, word 1 wait limit in cycles (0 = default), bytes 16-19 the NVFP4 tensor scale of the
// activations that latmix_linear quantises (latmix_workspace_set_tensor_scale).
constexpr size_t kHeaderTensorScaleOffset = 16;

void count_launch(int n = 1);

struct QuantArgs {
    const void* X; int x_is_bf16;
    const float* b;            // nullable
    int64_t M, K;
    int fmt, sf_layout;
    uint8_t* codes; uint8_t* scales;
    float* Y_dump;             // nullable
    uint32_t* status; uint32_t flags;
};

// Plain quantiser: codes, scales = Q(X + b).  SIMT, memory-bound.
cudaError_t launch_quantize_rows(const QuantArgs& a, cudaStream_t st);

struct GemmQuantArgs {
    // Y[r][c] = sum_k P(r,k) Q(k,c) + b[c];  rows r < R, columns c < C (C = contraction width of the next step)
    const void* P; int p_is_bf16; int64_t p_row_stride, p_k_stride;
    const void* Q; int q_is_bf16; int64_t q_k_stride, q_col_stride;
    const float* b;
    int64_t R, C, Kred;
    int fmt, sf_layout;
    uint8_t* codes; uint8_t* scales; float* Y_dump;
    uint32_t* status; uint32_t flags;
};
// Block-diagonal transform (32 x 32 blocks = MX blocks) fused with the quantiser; `A` in QuantArgs terms is passed apart.
cudaError_t launch_blockdiag_quant(const QuantArgs& a, const void* A_blocks, cudaStream_t st);
bool blockdiag_quant_mma_supported(const QuantArgs& a);                       // bf16 inputs, K a multiple of 128
cudaError_t launch_blockdiag_quant_mma(const QuantArgs& a, const void* A_blocks, cudaStream_t st);

// fp32 FMA product with the quantiser as epilogue (fp32 inputs of the transform; the offline fold).
cudaError_t launch_gemm_quant_simt(const GemmQuantArgs& a, cudaStream_t st);

// c[n] = bias[n] - sum_j (b A_inv)[j] W[j][n], fp64 accumulation; `u_tmp` holds K doubles.
cudaError_t launch_fold_bias(const float* A_inv, const float* b, const void* W, int w_is_bf16, const float* bias,
                             int64_t K, int64_t N, double* u_tmp, float* c_out, cudaStream_t st);

// c[n] = sum_j c1[j] A_out[j][n] + v_out[n] (c1, v_out nullable = 0), fp64 accumulation; c1 and c_out must not alias.
cudaError_t launch_fold_bias_out(const float* c1, const float* A_out, const float* v_out, int64_t N, float* c_out,
                                 cudaStream_t st);

struct MxGemmArgs {
    const uint8_t* a_codes; const uint8_t* a_scales;
    const uint8_t* w_codes; const uint8_t* w_scales;
    const float* c;
    int64_t M, K, N;
    int fmt;
    float* out; int64_t ldo;
    uint32_t* status; uint32_t flags;
    const float* a_tensor_scale = nullptr;      // NVFP4: the fp32 scale of each operand (device memory)
    const float* w_tensor_scale = nullptr;
};
// CUDA-core block-scaled product: any shape; also the small-M (decode) path.
cudaError_t launch_mx_gemm_simt(const MxGemmArgs& a, cudaStream_t st);

// Tensor-core kernels (tcgen05).  `supported` reports whether the shape/format can take the path.
bool mx_gemm_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mx_gemm_tc(const MxGemmArgs& a, cudaStream_t st);
// Small batches (M <= 64): operands swapped, weight rows on the 128-row side of the MMA, eight 16 KB weight slabs in flight per SM.
bool mx_gemm_decode_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mx_gemm_decode_tc(const MxGemmArgs& a, cudaStream_t st);
// The same product on CTA pairs (cta_group::2, 256-row tiles): half the weight bytes per SM.
bool mx_gemm_pair_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mx_gemm_pair_tc(const MxGemmArgs& a, cudaStream_t st);

// CTA pairs with 256 x 256 tiles and two accumulators that overlap in tensor memory; also the NVFP4 product.
bool mx_gemm_wide_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mx_gemm_wide_tc(const MxGemmArgs& a, cudaStream_t st);

struct TransformQuantArgs {
    const void* X; const void* A;   // bf16, row-major M x K and K x K
    const float* b;
    int64_t M, K;
    int fmt, sf_layout;
    uint8_t* codes; uint8_t* scales; float* Y_dump;
    uint32_t* status; uint32_t flags;
};
bool transform_quant_tc_supported(const TransformQuantArgs& a);
cudaError_t launch_transform_quant_tc(const TransformQuantArgs& a, cudaStream_t st);
// A handful of rows (M <= 16): columns of A on the 128-row side of the MMA, clusters of four CTAs per tile.
bool transform_quant_decode_tc_supported(const TransformQuantArgs& a);
cudaError_t launch_transform_quant_decode_tc(const TransformQuantArgs& a, cudaStream_t st);
// The same on CTA pairs (cta_group::2, 256 x 256 tiles, half-width tiles in the last wave).
bool transform_quant_pair_tc_supported(const TransformQuantArgs& a);
cudaError_t launch_transform_quant_pair_tc(const TransformQuantArgs& a, cudaStream_t st);

// MXINT8 on the tensor cores: both operands expanded exactly to bf16 in `scratch`, then a bf16 CTA-pair GEMM.
size_t mxint8_gemm_tc_scratch_bytes(int64_t M, int64_t K, int64_t N);
bool mxint8_gemm_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mxint8_gemm_tc(const MxGemmArgs& a, void* scratch, cudaStream_t st);

// MXINT8 for M <= 16 without scratch: the expansion to bf16 happens in shared memory, between the copy engine and the MMA.
bool mxint8_gemm_decode_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mxint8_gemm_decode_tc(const MxGemmArgs& a, cudaStream_t st);
// the same product on the integer tensor-core kind (codes as they are, block scales applied to the integer sums)
bool mxint8_gemm_decode_i8_tc_supported(const MxGemmArgs& a);
cudaError_t launch_mxint8_gemm_decode_i8_tc(const MxGemmArgs& a, cudaStream_t st);

// Offline fold + weight quantisation on the tensor cores (bf16 W; fp32 A_inv split into three bf16 terms in `scratch`).
size_t fold_tc_scratch_bytes(int64_t K);
bool fold_tc_supported(int64_t K, int64_t N, int w_is_bf16);
cudaError_t launch_fold_quant_pair_tc(const float* A_inv, const void* W, int64_t K, int64_t N, int fmt, int sf_layout,
                                      uint8_t* codes, uint8_t* scales, float* dump, uint32_t* status, uint32_t flags,
                                      void* scratch, cudaStream_t st);

// Two-sided fold on the tensor cores (bf16 W, K and N multiples of 64): W~~^T = A_out^T W^T A_in_inv^T, fp32-accurate,
// quantised along k.  A_in_inv null = output side only.  With both sides, *T_out receives the address (inside `scratch`)
// of T = W A_out as K x N fp32, which the bias fold needs.
bool fold_two_sided_tc_supported(int64_t K, int64_t N, int w_is_bf16);
size_t fold_two_sided_tc_scratch_bytes(int64_t K, int64_t N, bool both);
cudaError_t launch_fold_two_sided_tc(const float* A_in_inv, const void* W, const float* A_out, int64_t K, int64_t N, int fmt,
                                     int sf_layout, uint8_t* codes, uint8_t* scales, float* dump, float** T_out,
                                     uint32_t* status, uint32_t flags, void* scratch, cudaStream_t st);

// Transformation-MSE diagnostic: D = Y - dq(codes, scales) (scales in the linear layout); E = D A_inv on the tensor
// cores (M a multiple of 8, K of 64; E may alias D); block_err[i] = mean of E^2 over rows and block i, mse = their mean.
cudaError_t launch_dequant_diff(const float* Y, const uint8_t* codes, const uint8_t* scales, int64_t M, int64_t K, int fmt,
                                float* D, cudaStream_t st);
bool backmap_tc_supported(int64_t M, int64_t K);
size_t backmap_tc_scratch_bytes(int64_t M, int64_t K);
cudaError_t launch_backmap_tc(const float* D, const float* A_inv, int64_t M, int64_t K, float* E, uint32_t* status,
                              void* scratch, cudaStream_t st);
cudaError_t launch_block_sumsq(const float* E, int64_t M, int64_t K, int block, double* block_err, double* mse, cudaStream_t st);
// D = Y - Q_B(Y) for an MX block size B of 8, 16, 32, 64 or 128 (K a multiple of B); D may alias Y.
cudaError_t launch_quant_error_block(const float* Y, int64_t M, int64_t K, int fmt, int block, float* D, cudaStream_t st);

// The same for fp32 weights (both operands as three bf16 terms, nine products); K a multiple of 64.
size_t fold_tc_f32_scratch_bytes(int64_t K, int64_t N);
bool fold_tc_f32_supported(int64_t K, int64_t N);
cudaError_t launch_fold_quant_pair_tc_f32(const float* A_inv, const float* W, int64_t K, int64_t N, int fmt, int sf_layout,
                                          uint8_t* codes, uint8_t* scales, float* dump, uint32_t* status, uint32_t flags,
                                          void* scratch, cudaStream_t st);

// Clusters of two CTAs of `kernel` that fit on the current device at once (cached).
int resident_cta_pairs(const void* kernel, int threads, int smem_bytes);
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize), issued once per kernel and device
cudaError_t set_max_dynamic_smem(const void* kernel, int smem_bytes);
// SMs of the current device (asked once per device)
int sm_count();

}  // namespace latmix
