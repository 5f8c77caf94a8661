// C ABI entry points of liblatmix: argument checking, path selection, workspace carving.  No kernels here.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "internal.h"
#include "mx_math.cuh"

namespace latmix {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool valid_fmt(int f) {
    return f == LATMIX_MXFP4_E2M1 || f == LATMIX_MXFP8_E4M3 || f == LATMIX_MXINT8 || f == LATMIX_MXINT4 || f == LATMIX_NVFP4;
}
static inline bool packs_two_codes(int f) { return f == LATMIX_MXFP4_E2M1 || f == LATMIX_NVFP4; }
static inline bool valid_dtype(int d) { return d == LATMIX_F32 || d == LATMIX_BF16; }
static inline bool valid_sf(int s) { return s == LATMIX_SF_LINEAR || s == LATMIX_SF_TCGEN05; }

// sm_100 check for the current device, cached per device ordinal.
static latmix_status_t check_device() {
    static std::atomic<int> cache[64];   // 0 unknown, 1 ok, 2 unsupported
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (dev < 0 || dev >= 64) return LATMIX_ERR_UNSUPPORTED;
    int c = cache[dev].load(std::memory_order_relaxed);
    if (c == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return LATMIX_ERR_CUDA;
        c = major == 10 ? 1 : 2;
        cache[dev].store(c, std::memory_order_relaxed);
    }
    return c == 1 ? LATMIX_OK : LATMIX_ERR_UNSUPPORTED;
}

static latmix_status_t shape_check(int64_t rows, int64_t K, int fmt) {
    if (rows < 0 || K < 0) return LATMIX_ERR_INVALID_ARG;
    if (K % 32 != 0) return LATMIX_ERR_SHAPE;
    if (packs_two_codes(fmt) && K % 64 != 0) return LATMIX_ERR_SHAPE;
    return LATMIX_OK;
}

constexpr size_t kTensorScaleTrailerBytes = 16;     // NVFP4: the tensor's fp32 scale sits behind the block scales

static void mx_sizes(int64_t rows, int64_t K, int fmt, int sf, size_t* code_bytes, size_t* scale_bytes) {
    *code_bytes = (size_t)rows * (size_t)(packs_two_codes(fmt) ? K / 2 : K);
    if (fmt == LATMIX_NVFP4) *scale_bytes = nvfp4_block_scale_bytes(rows, K, sf) + kTensorScaleTrailerBytes;
    else if (sf == LATMIX_SF_LINEAR) *scale_bytes = (size_t)rows * (size_t)(K / 32);
    else *scale_bytes = (size_t)((rows + 127) / 128) * (size_t)sf_k_tiles(K) * 512;
}

// Padding BLOCKS of the tiled scale layout (K/32 not a multiple of 8) are zeroed before the quantiser runs.  Padding ROWS
// are not: whatever they hold scales accumulator rows (or columns) that lie outside the result and are never stored.
static bool scales_have_block_padding(int64_t K, int sf, int fmt) {
    return sf == LATMIX_SF_TCGEN05 && (fmt == LATMIX_NVFP4 ? (K / 16) % 16 != 0 : (K / 32) % 8 != 0);
}
// Zero the block-scale part of a scale buffer (never the NVFP4 trailer: the caller's tensor scale lives there).
static cudaError_t zero_block_scales(void* scales, int64_t rows, int64_t K, int fmt, int sf, cudaStream_t st) {
    size_t cb, sb;
    mx_sizes(rows, K, fmt, sf, &cb, &sb);
    if (fmt == LATMIX_NVFP4) sb -= kTensorScaleTrailerBytes;
    return cudaMemsetAsync(scales, 0, sb, st);
}

}  // namespace latmix

using namespace latmix;

extern "C" {

latmix_status_t latmix_mx_sizes(int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf,
                                size_t* code_bytes, size_t* scale_bytes) {
    if (!valid_fmt(fmt) || !valid_sf(sf) || code_bytes == nullptr || scale_bytes == nullptr) return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(rows, K, fmt);
    if (s != LATMIX_OK) return s;
    mx_sizes(rows, K, fmt, sf, code_bytes, scale_bytes);
    return LATMIX_OK;
}

size_t latmix_scale_offset(int64_t row, int64_t kblock, int64_t rows, int64_t K, latmix_sf_layout_t sf) {
    if (!valid_sf(sf) || row < 0 || row >= rows || K <= 0 || K % 32 != 0 || kblock < 0 || kblock >= K / 32) return (size_t)-1;
    if (sf == LATMIX_SF_LINEAR) return (size_t)(row * (K / 32) + kblock);
    return sf_tcgen05_offset(row, kblock, sf_k_tiles(K));
}

size_t latmix_scale_offset_fmt(int64_t row, int64_t kblock, int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf) {
    if (fmt != LATMIX_NVFP4) return valid_fmt(fmt) ? latmix_scale_offset(row, kblock, rows, K, sf) : (size_t)-1;
    if (!valid_sf(sf) || row < 0 || row >= rows || K <= 0 || K % 64 != 0 || kblock < 0 || kblock >= K / 16) return (size_t)-1;
    if (sf == LATMIX_SF_LINEAR) return (size_t)(row * (K / 16) + kblock);
    return sf_tcgen05_offset(row, kblock, nvfp4_sf_k_tiles(K));
}

size_t latmix_tensor_scale_offset(int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf) {
    if (fmt != LATMIX_NVFP4 || !valid_sf(sf) || rows < 0 || K < 0 || K % 64 != 0) return (size_t)-1;
    return nvfp4_block_scale_bytes(rows, K, sf);
}

latmix_status_t latmix_workspace_set_tensor_scale(void* workspace, size_t workspace_bytes, float tensor_scale, void* cuda_stream) {
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes) return LATMIX_ERR_WORKSPACE;
    if (!aligned16(workspace) || !(tensor_scale > 0.0f) || !(tensor_scale < 3.0e38f)) return LATMIX_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(static_cast<uint8_t*>(workspace) + kHeaderTensorScaleOffset, &tensor_scale, sizeof(float), cudaMemcpyHostToDevice,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

latmix_status_t latmix_workspace_bytes(latmix_op_t op, int64_t M, int64_t K, int64_t N, latmix_format_t fmt, size_t* bytes) {
    if (bytes == nullptr || !valid_fmt(fmt) || M < 0 || K < 0 || N < 0) return LATMIX_ERR_INVALID_ARG;
    if (K % 32 != 0) return LATMIX_ERR_SHAPE;
    size_t total = kWorkspaceHeaderBytes;
    switch (op) {
        case LATMIX_OP_FOLD_WEIGHTS:
            // K doubles for the bias fold, then three bf16 copies of A_inv for the tensor-core fold; a workspace with
            // only the first part (the size this call needed before) still works and takes the CUDA-core fold
            total += align_up((size_t)K * sizeof(double), 256) + align_up(fold_tc_scratch_bytes(K), 256);
            break;
        case LATMIX_OP_FOLD_TWO_SIDED:
            // K doubles, N floats, then the larger of the two paths' scratch (both sides given)
            total += align_up((size_t)K * sizeof(double), 256) + align_up((size_t)N * sizeof(float), 256);
            {
                const size_t simt = align_up((size_t)N * (size_t)K * sizeof(float), 256) + align_up(fold_tc_scratch_bytes(K), 256);
                const size_t tc = fold_two_sided_tc_scratch_bytes(K, N, true);
                total += simt > tc ? simt : tc;
            }
            break;
        case LATMIX_OP_TRANSFORMATION_MSE: {
            // activation codes and (linear) scales, two M x K fp32 matrices, the three-term copies for the tensor-core product
            size_t cb, sb;
            mx_sizes(M, K, fmt, LATMIX_SF_LINEAR, &cb, &sb);
            total += align_up(cb, 256) + align_up(sb, 256) + 2 * align_up((size_t)M * (size_t)K * sizeof(float), 256) +
                     align_up(backmap_tc_scratch_bytes(M, K), 256);
            break;
        }
        case LATMIX_OP_QUANTIZE_MX: break;
        case LATMIX_OP_MX_GEMM:
            if (fmt == LATMIX_MXINT8) total += mxint8_gemm_tc_scratch_bytes(M, K, N);    // bf16 copies of both operands
            break;
        case LATMIX_OP_LINEAR: {
            size_t cb, sb;
            mx_sizes(M, K, fmt, LATMIX_SF_TCGEN05, &cb, &sb);
            total += align_up(cb, 256) + align_up(sb, 256);
            if (fmt == LATMIX_MXINT8) total += mxint8_gemm_tc_scratch_bytes(M, K, N);
            break;
        }
        default: return LATMIX_ERR_INVALID_ARG;
    }
    *bytes = total;
    return LATMIX_OK;
}

const char* latmix_status_string(latmix_status_t s) {
    switch (s) {
        case LATMIX_OK: return "ok";
        case LATMIX_ERR_INVALID_ARG: return "invalid argument";
        case LATMIX_ERR_SHAPE: return "unsupported shape (K must be a multiple of 32, 64 for MXFP4; leading dimension)";
        case LATMIX_ERR_UNSUPPORTED: return "unsupported combination or device (needs sm_100)";
        case LATMIX_ERR_WORKSPACE: return "workspace missing or too small";
        case LATMIX_ERR_CUDA: return "CUDA call failed";
        case LATMIX_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case LATMIX_ERR_NONFINITE: return "non-finite input";
    }
    return "unknown status";
}

uint64_t latmix_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

latmix_status_t latmix_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes) return LATMIX_ERR_WORKSPACE;
    if (!aligned16(workspace)) return LATMIX_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

latmix_status_t latmix_workspace_set_wait_limit(void* workspace, size_t workspace_bytes, uint32_t cycles, void* cuda_stream) {
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes) return LATMIX_ERR_WORKSPACE;
    if (!aligned16(workspace)) return LATMIX_ERR_INVALID_ARG;
    // word 1 of the header; the source is pageable host memory, which the runtime has read by the time the call returns
    if (cudaMemcpyAsync(static_cast<uint32_t*>(workspace) + 1, &cycles, sizeof(cycles), cudaMemcpyHostToDevice,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

latmix_status_t latmix_device_status(void* workspace, void* cuda_stream) {
    if (workspace == nullptr) return LATMIX_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (word & (1u << LATMIX_ERR_TIMEOUT)) return LATMIX_ERR_TIMEOUT;
    if (word & (1u << LATMIX_ERR_NONFINITE)) return LATMIX_ERR_NONFINITE;
    return word == 0 ? LATMIX_OK : LATMIX_ERR_CUDA;
}

latmix_status_t latmix_quantize_mx(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b, int64_t M,
                                   int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf, void* codes, void* scales,
                                   float* Y_dump, void* workspace, size_t workspace_bytes, uint32_t flags,
                                   void* cuda_stream) {
    if (!valid_fmt(fmt) || !valid_dtype(x_dtype) || !valid_sf(sf)) return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(M, K, fmt);
    if (s != LATMIX_OK) return s;
    if (M == 0 || K == 0) return LATMIX_OK;             // empty input: nothing to do, pointers may be null
    if (X == nullptr || codes == nullptr || scales == nullptr) return LATMIX_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(A) || !aligned16(b) || !aligned16(codes) || !aligned16(scales) || !aligned16(Y_dump))
        return LATMIX_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    if ((s = check_device()) != LATMIX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint32_t* status = static_cast<uint32_t*>(workspace);
    if (scales_have_block_padding(K, sf, fmt) && zero_block_scales(scales, M, K, fmt, sf, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    cudaError_t e;
    if (fmt == LATMIX_NVFP4 && (flags & LATMIX_FLAG_BLOCK_DIAG)) return LATMIX_ERR_UNSUPPORTED;
    if (A == nullptr || (flags & LATMIX_FLAG_BLOCK_DIAG)) {
        QuantArgs q{X, x_dtype == LATMIX_BF16, b, M, K, (int)fmt, (int)sf, static_cast<uint8_t*>(codes),
                    static_cast<uint8_t*>(scales), Y_dump, status, flags};
        e = A == nullptr ? launch_quantize_rows(q, st) : launch_blockdiag_quant(q, A, st);
    } else {
        TransformQuantArgs t{X, A, b, M, K, (int)fmt, (int)sf, static_cast<uint8_t*>(codes), static_cast<uint8_t*>(scales),
                             Y_dump, status, flags};
        const bool tc = x_dtype == LATMIX_BF16 && !(flags & LATMIX_FLAG_FORCE_SIMT);
        const uint32_t variant = (flags >> 8) & 0xFu;       // tuning override: 1-3 = single-CTA kernel, 4 = small-batch kernel, 8 = CTA pairs
        if (tc && fmt == LATMIX_NVFP4 && transform_quant_pair_tc_supported(t)) {
            e = launch_transform_quant_pair_tc(t, st);      // the one tensor-core kernel whose epilogue knows blocks of 16
        } else if (fmt == LATMIX_NVFP4) {
            GemmQuantArgs g{X, x_dtype == LATMIX_BF16, K, 1, A, x_dtype == LATMIX_BF16, K, 1, b, M, K, K, (int)fmt, (int)sf,
                            static_cast<uint8_t*>(codes), static_cast<uint8_t*>(scales), Y_dump, status, flags};
            e = launch_gemm_quant_simt(g, st);
        } else if (tc && (variant == 0 || variant == 4) && transform_quant_decode_tc_supported(t)) {
            e = launch_transform_quant_decode_tc(t, st);    // M <= 16: bound by reading A once
        } else if (tc && (variant == 0 || variant == 8) && transform_quant_pair_tc_supported(t)) {
            e = launch_transform_quant_pair_tc(t, st);
        } else if (tc && transform_quant_tc_supported(t)) {
            e = launch_transform_quant_tc(t, st);
        } else {
            const int bf = x_dtype == LATMIX_BF16;
            GemmQuantArgs g{X, bf, K, 1, A, bf, K, 1, b, M, K, K, (int)fmt, (int)sf, static_cast<uint8_t*>(codes),
                            static_cast<uint8_t*>(scales), Y_dump, status, flags};
            e = launch_gemm_quant_simt(g, st);
        }
    }
    return e == cudaSuccess ? LATMIX_OK : LATMIX_ERR_CUDA;
}

// The one-sided fold with its scratch given explicitly: `u_tmp` holds K doubles, `tc_scratch` (nullable) the three bf16
// copies of A_inv that the tensor-core product needs.  Arguments are checked by the callers.
static latmix_status_t run_fold(const float* A_inv, const float* b, const void* W, latmix_dtype_t w_dtype, const float* bias,
                                int64_t K, int64_t N, latmix_format_t fmt, latmix_sf_layout_t sf, uint8_t* codes,
                                uint8_t* scales, float* c_out, float* dump, uint32_t* status, double* u_tmp,
                                void* tc_scratch, size_t tc_scratch_bytes, uint32_t flags, cudaStream_t st) {
    if (!(flags & LATMIX_FLAG_FORCE_SIMT) && w_dtype == LATMIX_F32 && tc_scratch != nullptr &&
        tc_scratch_bytes >= fold_tc_f32_scratch_bytes(K, N) && fold_tc_f32_supported(K, N)) {
        if (launch_fold_quant_pair_tc_f32(A_inv, static_cast<const float*>(W), K, N, (int)fmt, (int)sf, codes, scales, dump, status,
                                          flags, tc_scratch, st) != cudaSuccess)
            return LATMIX_ERR_CUDA;
        if (launch_fold_bias(A_inv, b, W, 0, bias, K, N, u_tmp, c_out, st) != cudaSuccess) return LATMIX_ERR_CUDA;
        return LATMIX_OK;
    }
    if (!(flags & LATMIX_FLAG_FORCE_SIMT) && tc_scratch != nullptr && tc_scratch_bytes >= fold_tc_scratch_bytes(K) &&
        fold_tc_supported(K, N, w_dtype == LATMIX_BF16)) {
        if (launch_fold_quant_pair_tc(A_inv, W, K, N, (int)fmt, (int)sf, codes, scales, dump, status, flags, tc_scratch, st) != cudaSuccess)
            return LATMIX_ERR_CUDA;
        if (launch_fold_bias(A_inv, b, W, 1, bias, K, N, u_tmp, c_out, st) != cudaSuccess) return LATMIX_ERR_CUDA;
        return LATMIX_OK;
    }
    // W~^T[n][k] = sum_j W[j][n] A_inv[k][j]: rows n of W^T times columns k of A_inv^T
    GemmQuantArgs g{W, w_dtype == LATMIX_BF16, 1, N, A_inv, 0, 1, K, nullptr, N, K, K, (int)fmt, (int)sf,
                    codes, scales, dump, status, flags};
    if (launch_gemm_quant_simt(g, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (launch_fold_bias(A_inv, b, W, w_dtype == LATMIX_BF16, bias, K, N, u_tmp, c_out, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

latmix_status_t latmix_fold_weights(const void* A_inv, const float* b, const void* W, latmix_dtype_t w_dtype,
                                    const float* bias, int64_t K, int64_t N, latmix_format_t fmt, latmix_sf_layout_t sf,
                                    void* Wq_codes, void* Wq_scales, float* c_out, float* Wfold_dump, void* workspace,
                                    size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    if (A_inv == nullptr || W == nullptr || Wq_codes == nullptr || Wq_scales == nullptr || c_out == nullptr ||
        !valid_fmt(fmt) || !valid_dtype(w_dtype) || !valid_sf(sf))
        return LATMIX_ERR_INVALID_ARG;
    if (!aligned16(A_inv) || !aligned16(b) || !aligned16(W) || !aligned16(bias) || !aligned16(Wq_codes) ||
        !aligned16(Wq_scales) || !aligned16(c_out) || !aligned16(Wfold_dump))
        return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(N, K, fmt);
    if (s != LATMIX_OK) return s;
    const size_t need = kWorkspaceHeaderBytes + align_up((size_t)K * sizeof(double), 256);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    if ((s = check_device()) != LATMIX_OK) return s;
    if (N == 0 || K == 0) return LATMIX_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    if (scales_have_block_padding(K, sf, fmt) && zero_block_scales(Wq_scales, N, K, fmt, sf, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    return run_fold(static_cast<const float*>(A_inv), b, W, w_dtype, bias, K, N, fmt, sf, static_cast<uint8_t*>(Wq_codes),
                    static_cast<uint8_t*>(Wq_scales), c_out, Wfold_dump, static_cast<uint32_t*>(workspace),
                    reinterpret_cast<double*>(base + kWorkspaceHeaderBytes), workspace_bytes > need ? base + need : nullptr,
                    workspace_bytes > need ? workspace_bytes - need : 0, flags, st);
}

latmix_status_t latmix_fold_weights_two_sided(const float* A_in_inv, const float* b_in, const void* W, latmix_dtype_t w_dtype,
                                              const float* bias, const float* A_out, const float* v_out, int64_t K, int64_t N,
                                              latmix_format_t fmt, latmix_sf_layout_t sf, void* Wq_codes, void* Wq_scales,
                                              float* c_out, float* Wfold_dump, void* workspace, size_t workspace_bytes,
                                              uint32_t flags, void* cuda_stream) {
    if (W == nullptr || Wq_codes == nullptr || Wq_scales == nullptr || c_out == nullptr || !valid_fmt(fmt) ||
        !valid_dtype(w_dtype) || !valid_sf(sf))
        return LATMIX_ERR_INVALID_ARG;
    if (A_in_inv == nullptr && A_out == nullptr) return LATMIX_ERR_INVALID_ARG;          // nothing to fold
    if (fmt == LATMIX_NVFP4 && A_out != nullptr) return LATMIX_ERR_UNSUPPORTED;
    if ((A_in_inv == nullptr && b_in != nullptr) || (A_out == nullptr && v_out != nullptr)) return LATMIX_ERR_INVALID_ARG;
    if (!aligned16(A_in_inv) || !aligned16(b_in) || !aligned16(W) || !aligned16(bias) || !aligned16(A_out) || !aligned16(v_out) ||
        !aligned16(Wq_codes) || !aligned16(Wq_scales) || !aligned16(c_out) || !aligned16(Wfold_dump))
        return LATMIX_ERR_INVALID_ARG;
    if (A_out == nullptr)            // input side only: the one-sided fold, same workspace rules
        return latmix_fold_weights(A_in_inv, b_in, W, w_dtype, bias, K, N, fmt, sf, Wq_codes, Wq_scales, c_out, Wfold_dump,
                                   workspace, workspace_bytes, flags, cuda_stream);
    latmix_status_t s = shape_check(N, K, fmt);
    if (s != LATMIX_OK) return s;
    const bool both = A_in_inv != nullptr;
    // header | K doubles | N floats | scratch.  CUDA-core path (input side first): N x K floats (weights after the input
    // side) and, optionally, the three bf16 copies of A_in_inv for a tensor-core input-side product.  Tensor-core path
    // (output side first): fold_two_sided_tc_scratch_bytes.
    const size_t off_u = kWorkspaceHeaderBytes, off_c1 = off_u + align_up((size_t)K * sizeof(double), 256);
    const size_t off_f1 = off_c1 + align_up((size_t)N * sizeof(float), 256);
    const size_t need = off_f1 + (both ? align_up((size_t)N * (size_t)K * sizeof(float), 256) : 0);
    const size_t need_tc = need + align_up(fold_tc_scratch_bytes(K), 256);
    const bool tc2_ok = !(flags & LATMIX_FLAG_FORCE_SIMT) && fold_two_sided_tc_supported(K, N, w_dtype == LATMIX_BF16);
    const size_t need_tc2 = off_f1 + fold_two_sided_tc_scratch_bytes(K, N, both);
    if (workspace == nullptr || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    const bool use_tc2 = tc2_ok && workspace_bytes >= need_tc2;
    if (!use_tc2 && workspace_bytes < need) return LATMIX_ERR_WORKSPACE;
    if ((s = check_device()) != LATMIX_OK) return s;
    if (N == 0 || K == 0) return LATMIX_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint32_t* status = static_cast<uint32_t*>(workspace);
    uint8_t* codes = static_cast<uint8_t*>(Wq_codes);
    uint8_t* scales = static_cast<uint8_t*>(Wq_scales);
    if (scales_have_block_padding(K, sf, fmt) && zero_block_scales(Wq_scales, N, K, fmt, sf, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (use_tc2) {
        float* T = nullptr;
        if (launch_fold_two_sided_tc(A_in_inv, W, A_out, K, N, (int)fmt, (int)sf, codes, scales, Wfold_dump, &T, status, flags,
                                     base + off_f1, st) != cudaSuccess)
            return LATMIX_ERR_CUDA;
        if (!both) return launch_fold_bias_out(bias, A_out, v_out, N, c_out, st) == cudaSuccess ? LATMIX_OK : LATMIX_ERR_CUDA;
        // c = (bias A_out + v_out) - b_in A_in_inv T
        float* c1w = reinterpret_cast<float*>(base + off_c1);
        if (launch_fold_bias_out(bias, A_out, v_out, N, c1w, st) != cudaSuccess) return LATMIX_ERR_CUDA;
        if (launch_fold_bias(A_in_inv, b_in, T, 0, c1w, K, N, reinterpret_cast<double*>(base + off_u), c_out, st) != cudaSuccess)
            return LATMIX_ERR_CUDA;
        return LATMIX_OK;
    }
    const float* c1 = bias;
    GemmQuantArgs g{};
    g.P = A_out; g.p_is_bf16 = 0; g.p_row_stride = 1; g.p_k_stride = N;        // P(n, j) = A_out[j][n]
    if (both) {
        // input side first: F1 = (A_in_inv W)^T as N x K fp32 and c1 = bias - b_in A_in_inv W; the codes this step
        // writes are replaced below
        float* f1 = reinterpret_cast<float*>(base + off_f1);
        float* c1w = reinterpret_cast<float*>(base + off_c1);
        s = run_fold(A_in_inv, b_in, W, w_dtype, bias, K, N, fmt, sf, codes, scales, c1w, f1, status,
                     reinterpret_cast<double*>(base + off_u), workspace_bytes >= need_tc ? base + need : nullptr,
                     workspace_bytes >= need_tc ? workspace_bytes - need : 0, flags, st);
        if (s != LATMIX_OK) return s;
        c1 = c1w;
        g.Q = f1; g.q_is_bf16 = 0; g.q_k_stride = K; g.q_col_stride = 1;      // Q(j, k) = F1[j][k]
    } else {
        g.Q = W; g.q_is_bf16 = w_dtype == LATMIX_BF16; g.q_k_stride = 1; g.q_col_stride = N;   // Q(j, k) = W[k][j]
    }
    // W~~^T[n][k] = sum_j A_out[j][n] (A_in_inv W)[k][j], quantised along k
    g.b = nullptr; g.R = N; g.C = K; g.Kred = N; g.fmt = (int)fmt; g.sf_layout = (int)sf;
    g.codes = codes; g.scales = scales; g.Y_dump = Wfold_dump; g.status = status; g.flags = flags;
    if (launch_gemm_quant_simt(g, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    if (launch_fold_bias_out(c1, A_out, v_out, N, c_out, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

latmix_status_t latmix_transformation_mse(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                          const float* A_inv, int64_t M, int64_t K, latmix_format_t fmt, double* block_err,
                                          double* mse, void* workspace, size_t workspace_bytes, uint32_t flags,
                                          void* cuda_stream) {
    return latmix_transformation_mse_block(X, x_dtype, A, b, A_inv, M, K, fmt, 32, block_err, mse, workspace, workspace_bytes, flags,
                                           cuda_stream);
}

latmix_status_t latmix_transformation_mse_block(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                                const float* A_inv, int64_t M, int64_t K, latmix_format_t fmt, int block,
                                                double* block_err, double* mse, void* workspace, size_t workspace_bytes,
                                                uint32_t flags, void* cuda_stream) {
    if (block != 8 && block != 16 && block != 32 && block != 64 && block != 128) return LATMIX_ERR_INVALID_ARG;
    if (X == nullptr || block_err == nullptr || mse == nullptr || !valid_fmt(fmt) || !valid_dtype(x_dtype)) return LATMIX_ERR_INVALID_ARG;
    if ((A == nullptr) != (A_inv == nullptr)) return LATMIX_ERR_INVALID_ARG;        // a transform comes with its inverse
    if (fmt == LATMIX_NVFP4) return LATMIX_ERR_UNSUPPORTED;
    if (!aligned16(A_inv) || !aligned16(block_err) || (reinterpret_cast<uintptr_t>(mse) & 7u)) return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(M, K, fmt);
    if (s != LATMIX_OK) return s;
    if (K % block != 0) return LATMIX_ERR_SHAPE;
    size_t cb, sb;
    mx_sizes(M, K, fmt, LATMIX_SF_LINEAR, &cb, &sb);
    const size_t mk = align_up((size_t)M * (size_t)K * sizeof(float), 256);
    const size_t off_codes = kWorkspaceHeaderBytes, off_scales = off_codes + align_up(cb, 256);
    const size_t off_d = off_scales + align_up(sb, 256), off_e = off_d + mk, need = off_e + mk;
    const size_t need_tc = need + align_up(backmap_tc_scratch_bytes(M, K), 256);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    if ((s = check_device()) != LATMIX_OK) return s;
    if (M == 0 || K == 0) return LATMIX_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint32_t* status = static_cast<uint32_t*>(workspace);
    uint8_t* codes = base + off_codes;
    uint8_t* scales = base + off_scales;
    float* D = reinterpret_cast<float*>(base + off_d);
    float* E = reinterpret_cast<float*>(base + off_e);
    // y = T(x) as it enters the quantiser, Q(y) as codes and scales: the online path itself
    s = latmix_quantize_mx(X, x_dtype, A, b, M, K, fmt, LATMIX_SF_LINEAR, codes, scales, D, workspace, kWorkspaceHeaderBytes, flags,
                           cuda_stream);
    if (s != LATMIX_OK) return s;
    // d = y - Q(y), in place: from the codes the path just produced (B = 32), or re-quantised with the asked block size
    if (block == 32) { if (launch_dequant_diff(D, codes, scales, M, K, (int)fmt, D, st) != cudaSuccess) return LATMIX_ERR_CUDA; }
    else if (launch_quant_error_block(D, M, K, (int)fmt, block, D, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    const float* err = D;                                // identity transform: the error needs no mapping back
    if (A_inv != nullptr) {
        if (!(flags & LATMIX_FLAG_FORCE_SIMT) && workspace_bytes >= need_tc && backmap_tc_supported(M, K)) {
            if (launch_backmap_tc(D, A_inv, M, K, E, status, base + need, st) != cudaSuccess) return LATMIX_ERR_CUDA;
        } else {
            // e[m][k] = sum_j d[m][j] A_inv[j][k] as an fp32 FMA product; the codes it writes (of e) land in the consumed buffers
            GemmQuantArgs g{D, 0, K, 1, A_inv, 0, K, 1, nullptr, M, K, K, (int)fmt, (int)LATMIX_SF_LINEAR, codes, scales, E, status, 0u};
            if (launch_gemm_quant_simt(g, st) != cudaSuccess) return LATMIX_ERR_CUDA;
        }
        err = E;
    }
    if (launch_block_sumsq(err, M, K, block, block_err, mse, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    return LATMIX_OK;
}

// The block-scaled product with its scratch region given explicitly (`scratch` may be null when scratch_bytes is 0):
// latmix_mx_gemm keeps scratch right behind the workspace header, latmix_linear behind the activation codes and scales.
static latmix_status_t run_mx_gemm(const void* a_codes, const void* a_scales, const void* w_codes, const void* w_scales,
                                   const float* c, int64_t M, int64_t K, int64_t N, latmix_format_t fmt, float* out,
                                   int64_t ldo, void* workspace, size_t workspace_bytes, void* scratch, size_t scratch_bytes,
                                   uint32_t flags, void* cuda_stream) {
    if (a_codes == nullptr || a_scales == nullptr || w_codes == nullptr || w_scales == nullptr || out == nullptr || !valid_fmt(fmt))
        return LATMIX_ERR_INVALID_ARG;
    if (!aligned16(a_codes) || !aligned16(a_scales) || !aligned16(w_codes) || !aligned16(w_scales) || !aligned16(c) || !aligned16(out))
        return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(M, K, fmt);
    if (s != LATMIX_OK) return s;
    if (N < 0) return LATMIX_ERR_INVALID_ARG;
    if (ldo < N || ldo % 4 != 0) return LATMIX_ERR_SHAPE;
    if (workspace == nullptr || workspace_bytes < kWorkspaceHeaderBytes || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    if ((s = check_device()) != LATMIX_OK) return s;
    if (M == 0 || N == 0) return LATMIX_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    MxGemmArgs g{static_cast<const uint8_t*>(a_codes), static_cast<const uint8_t*>(a_scales),
                 static_cast<const uint8_t*>(w_codes), static_cast<const uint8_t*>(w_scales), c, M, K, N,
                 // MXINT4 codes are the E4M3 bytes of the integers: the contraction is the MXFP8 one, products exact
                 fmt == LATMIX_MXINT4 ? (int)LATMIX_MXFP8_E4M3 : (int)fmt, out, ldo, static_cast<uint32_t*>(workspace), flags};
    if (fmt == LATMIX_NVFP4) {
        g.a_tensor_scale = nvfp4_tensor_scale_ptr(g.a_scales, M, K, LATMIX_SF_TCGEN05);
        g.w_tensor_scale = nvfp4_tensor_scale_ptr(g.w_scales, N, K, LATMIX_SF_TCGEN05);
        cudaError_t en = (!(flags & LATMIX_FLAG_FORCE_SIMT) && mx_gemm_wide_tc_supported(g)) ? launch_mx_gemm_wide_tc(g, st)
                                                                                              : launch_mx_gemm_simt(g, st);
        return en == cudaSuccess ? LATMIX_OK : LATMIX_ERR_CUDA;
    }
    cudaError_t e;
    // tuning override in flag bits 8-11: 0 = default choice (small-batch kernel for M <= 64, CTA pairs with 256 x 256 tiles for
    // M > 128, single CTA in between), 1-3 = single-CTA tile shapes, 4 = small-batch kernel, 8 = CTA pairs with 256 x 192
    // tiles, 9 = CTA pairs with 256 x 256 tiles
    const uint32_t variant = (flags >> 8) & 0xFu;
    const bool tc = !(flags & LATMIX_FLAG_FORCE_SIMT);
    if (tc && (variant == 0 || variant == 4) && mx_gemm_decode_tc_supported(g)) e = launch_mx_gemm_decode_tc(g, st);   // M <= 64
    else if (tc && (variant == 0 || variant == 4) && mxint8_gemm_decode_i8_tc_supported(g)) e = launch_mxint8_gemm_decode_i8_tc(g, st);   // MXINT8, M <= 64: integer MMAs, no scratch
    else if (tc && variant == 5 && mxint8_gemm_decode_tc_supported(g)) e = launch_mxint8_gemm_decode_tc(g, st);   // the same through bf16 in tensor memory
    else if (tc && (variant == 0 || variant == 9) && mx_gemm_wide_tc_supported(g)) e = launch_mx_gemm_wide_tc(g, st);   // M > 128
    else if (tc && (variant == 0 || variant == 8) && mx_gemm_pair_tc_supported(g)) e = launch_mx_gemm_pair_tc(g, st);
    else if (tc && mx_gemm_tc_supported(g)) e = launch_mx_gemm_tc(g, st);
    else if (tc && mxint8_gemm_tc_supported(g) && scratch != nullptr && scratch_bytes >= mxint8_gemm_tc_scratch_bytes(M, K, N))
        e = launch_mxint8_gemm_tc(g, scratch, st);       // a workspace sized before this path existed takes the CUDA-core kernel
    else e = launch_mx_gemm_simt(g, st);
    return e == cudaSuccess ? LATMIX_OK : LATMIX_ERR_CUDA;
}

latmix_status_t latmix_mx_gemm(const void* a_codes, const void* a_scales, const void* w_codes, const void* w_scales,
                               const float* c, int64_t M, int64_t K, int64_t N, latmix_format_t fmt, float* out,
                               int64_t ldo, void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    const bool has_scratch = workspace != nullptr && workspace_bytes > kWorkspaceHeaderBytes;
    return run_mx_gemm(a_codes, a_scales, w_codes, w_scales, c, M, K, N, fmt, out, ldo, workspace, workspace_bytes,
                       has_scratch ? static_cast<uint8_t*>(workspace) + kWorkspaceHeaderBytes : nullptr,
                       has_scratch ? workspace_bytes - kWorkspaceHeaderBytes : 0, flags, cuda_stream);
}

latmix_status_t latmix_linear(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b, const void* Wq_codes,
                              const void* Wq_scales, const float* c, int64_t M, int64_t K, int64_t N, latmix_format_t fmt,
                              float* out, int64_t ldo, void* workspace, size_t workspace_bytes, uint32_t flags,
                              void* cuda_stream) {
    if (!valid_fmt(fmt)) return LATMIX_ERR_INVALID_ARG;
    latmix_status_t s = shape_check(M, K, fmt);
    if (s != LATMIX_OK) return s;
    if (N < 0) return LATMIX_ERR_INVALID_ARG;
    size_t cb, sb;
    mx_sizes(M, K, fmt, LATMIX_SF_TCGEN05, &cb, &sb);
    // header + activation codes + scales are required; what latmix_workspace_bytes adds for MXINT8 (bf16 copies of both
    // operands) is used when it is there
    const size_t need = kWorkspaceHeaderBytes + align_up(cb, 256) + align_up(sb, 256);
    if (workspace == nullptr || workspace_bytes < need || !aligned16(workspace)) return LATMIX_ERR_WORKSPACE;
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t* a_codes = base + kWorkspaceHeaderBytes;
    uint8_t* a_scales = a_codes + align_up(cb, 256);
    // validate the second half's arguments before launching the first half
    if (Wq_codes == nullptr || Wq_scales == nullptr || out == nullptr || N < 0) return LATMIX_ERR_INVALID_ARG;
    if (!aligned16(Wq_codes) || !aligned16(Wq_scales) || !aligned16(c) || !aligned16(out)) return LATMIX_ERR_INVALID_ARG;
    if (ldo < N || ldo % 4 != 0) return LATMIX_ERR_SHAPE;
    if (fmt == LATMIX_NVFP4) {
        // the activations' tensor scale: from the workspace header (latmix_workspace_set_tensor_scale) to the trailer of
        // the activation scale buffer, where the quantiser and the product look for it
        if ((s = check_device()) != LATMIX_OK) return s;
        if (M > 0 && K > 0 &&
            cudaMemcpyAsync(a_scales + nvfp4_block_scale_bytes(M, K, LATMIX_SF_TCGEN05), base + kHeaderTensorScaleOffset, sizeof(float),
                            cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
            return LATMIX_ERR_CUDA;
    }
    s = latmix_quantize_mx(X, x_dtype, A, b, M, K, fmt, LATMIX_SF_TCGEN05, a_codes, a_scales, nullptr, workspace,
                           workspace_bytes, flags, cuda_stream);
    if (s != LATMIX_OK) return s;
    const size_t used = kWorkspaceHeaderBytes + align_up(cb, 256) + align_up(sb, 256);
    return run_mx_gemm(a_codes, a_scales, Wq_codes, Wq_scales, c, M, K, N, fmt, out, ldo, workspace, workspace_bytes,
                       base + used, workspace_bytes - used, flags, cuda_stream);
}

}  // extern "C"
