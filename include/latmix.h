/*
 * latmix.h -- C ABI of the transformed MX-quantized linear layer (LATMiX hot path) for NVIDIA B200 (sm_100a).
 *
 * The layer, in the row form of the paper's appendix on affine transforms inside attention
 * (T(X) = X A + V) and of its single-linear fold (Eq. "fold_kqv_1", transposed):
 *
 *     Y   = X A + 1 b^T                         affine transform (Definition "General Affine Transformation")
 *     Qa  = Q(Y)                                MX quantisation along each row, blocks of 32 (Eq. "q_mx")
 *     W~  = A^-1 W,  c = bias - b W~            offline fold (Eq. "fold_kqv_1"); weights are quantised AFTER folding
 *     Qw  = Q(W~) with blocks along K           round-to-nearest MX quantisation of the folded weights
 *     out = dq(Qa) dq(Qw)^T + c                 block-scaled contraction
 *
 * X is M x K (one token per row), A is K x K, b has K entries, W is K x N, bias has N entries.
 *
 * MX quantisation (Eq. "q_mx"): for each block i of 32 consecutive elements of a row,
 * s_i = 2^(floor(log2 max|y_j|) - r_max) and Q(y)_j = s_i Q_e(y_j / s_i).  The paper leaves Q_e to the
 * element format; this library fixes: round to nearest, ties to the even code; magnitudes beyond the
 * largest finite element saturate to it; an all-zero block (or an exponent below -127) gets scale byte 0;
 * exponents above 127 clamp to 127; a value that rounds to zero keeps its sign bit in the floating formats.
 * The scale is stored as an E8M0 byte (exponent + 127).  Inputs must be finite.
 *
 * General rules
 *  - Every data pointer is a DEVICE pointer owned by the caller, unless a parameter says "host".
 *    The library allocates no device memory: scratch comes from the caller's `workspace`.
 *  - All matrices are row-major and dense (leading dimension = number of columns) unless a leading
 *    dimension is passed.  Pointers must be 16-byte aligned.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream) and return
 *    without waiting.  Argument errors are returned synchronously and launch nothing.
 *  - Problems found on the device (a bounded wait that expired, a non-finite input when checking is on)
 *    are recorded in a status word at the start of `workspace`; read it with latmix_device_status().
 *  - There is no CPU fallback: on a device that is not sm_100 every compute call returns
 *    LATMIX_ERR_UNSUPPORTED.
 *  - Calls are re-entrant across streams as long as they use distinct workspaces.
 *  - The library remembers host-side set-up between calls: per host thread the copy-engine descriptors of the buffers it
 *    has seen (they depend on address and geometry only, never on contents), per device each kernel's attributes, the
 *    occupancy of CTA pairs and the SM count.  A process that destroys a device's context (cudaDeviceReset) must not call
 *    the library on that device afterwards.
 */
#ifndef LATMIX_H_
#define LATMIX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LATMIX_OK = 0,
    LATMIX_ERR_INVALID_ARG = 1,  /* null pointer, unknown enum value, negative size, misaligned pointer */
    LATMIX_ERR_SHAPE = 2,        /* K not a multiple of 32 (64 for MXFP4), leading dimension too small or unaligned */
    LATMIX_ERR_UNSUPPORTED = 3,  /* combination not implemented, or device is not sm_100 */
    LATMIX_ERR_WORKSPACE = 4,    /* workspace pointer null or smaller than latmix_workspace_bytes() */
    LATMIX_ERR_CUDA = 5,         /* a CUDA runtime / driver call failed */
    LATMIX_ERR_TIMEOUT = 6,      /* device status: a bounded wait inside a kernel expired */
    LATMIX_ERR_NONFINITE = 7     /* device status: non-finite value met while LATMIX_FLAG_CHECK_FINITE was set */
} latmix_status_t;

/* Element formats (OCP Microscaling v1.0, the MX definition the paper cites).  Block size 32, E8M0 scale. */
typedef enum {
    LATMIX_MXFP4_E2M1 = 0, /* r_max 2; magnitudes 0 .5 1 1.5 2 3 4 6; two codes per byte, element 2t in the LOW nibble */
    LATMIX_MXFP8_E4M3 = 1, /* r_max 8; max 448; one code per byte */
    LATMIX_MXINT8 = 2,     /* r_max 0; value = k / 64, k in [-127, 127], two's complement; one code per byte */
    /* MXINT4, which the paper evaluates but neither it nor the OCP text defines.  Taken here as integers k in [-7, 7]
     * (symmetric 4-bit range), value = k, r_max 2, round to nearest even, |k| = 8 saturates to 7.  Each element is STORED
     * as one byte holding the E4M3 encoding of k (zero always as +0): the 8-bit block-scaled tensor-core kind then consumes
     * the codes unchanged and every product stays exact; buffer sizes and the GEMM are those of LATMIX_MXFP8_E4M3. */
    LATMIX_MXINT4 = 3,
    /* NVFP4, which the paper evaluates in its appendix "NVFP Quantization Format Evaluation" without defining it; taken from
     * the vendor's public description: E2M1 elements packed like MXFP4, blocks of 16 (not 32) along K, one E4M3 scale byte
     * per block (positive, finite), and one fp32 scale g per tensor:  x ~ element * block scale * g.  The caller chooses g
     * (commonly max|x| / (448 * 6)) and stores it as an fp32 number in the 16-byte trailer at the end of the scale buffer
     * (latmix_tensor_scale_offset) BEFORE the quantising call; the calls that consume the buffer read it from there.
     * Quantisation, in fp32, one correctly rounded operation per step: t = (amax / 6) / g; d = E4M3(t) (nearest even,
     * saturating); s = d * g; r = 1 / s (0 if s = 0); code = E2M1(x * r) (nearest even, saturating, sign kept).
     * g must be a normal fp32 number in [2^-96, 2^96].  K must be a multiple of 64.  The choice of d is a reading of the
     * vendor's recipe.  Supported by latmix_quantize_mx (not with LATMIX_FLAG_BLOCK_DIAG), latmix_fold_weights,
     * latmix_mx_gemm and latmix_linear; the other calls return LATMIX_ERR_UNSUPPORTED. */
    LATMIX_NVFP4 = 4
} latmix_format_t;

typedef enum { LATMIX_F32 = 0, LATMIX_BF16 = 1 } latmix_dtype_t;

/* Where the E8M0 byte of (row r, block kb) lives inside a scale buffer. */
typedef enum {
    LATMIX_SF_LINEAR = 0,  /* [rows][K/32], byte (r, kb) at r * (K/32) + kb */
    LATMIX_SF_TCGEN05 = 1  /* tiles of 128 rows x 4 blocks = 512 bytes, ordered row-tile-major then k-tile;
                              inside a tile byte (r, kb) sits at (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4.
                              Rows are padded to a multiple of 128 and blocks to a multiple of 8.  When K/32 is not
                              a multiple of 8 the whole buffer is zeroed before the scales are written; otherwise
                              the bytes of padding rows keep what the buffer held (they scale rows or columns
                              outside the result, which are never stored).  This is the layout the block-scaled
                              tensor-core GEMM reads. */
} latmix_sf_layout_t;

/* Which call a workspace is sized for. */
typedef enum {
    LATMIX_OP_FOLD_WEIGHTS = 0, LATMIX_OP_QUANTIZE_MX = 1, LATMIX_OP_LINEAR = 2, LATMIX_OP_MX_GEMM = 3,
    LATMIX_OP_FOLD_TWO_SIDED = 4, LATMIX_OP_TRANSFORMATION_MSE = 5
} latmix_op_t;

/* Flags (bitwise or). */
enum {
    LATMIX_FLAG_NONE = 0,
    LATMIX_FLAG_CHECK_FINITE = 1,  /* quantiser records LATMIX_ERR_NONFINITE in the status word on NaN/Inf input */
    LATMIX_FLAG_FORCE_SIMT = 2,    /* use the plain CUDA-core kernels even where a tensor-core kernel applies */
    LATMIX_FLAG_BLOCK_DIAG = 4,    /* latmix_quantize_mx / latmix_linear: A is block-diagonal with 32 x 32 blocks that
                                      coincide with the MX blocks (the paper's online transform T_3, a block Hadamard
                                      there); A then points to K/32 blocks [K/32][32][32], block i acting on elements
                                      32 i .. 32 i + 31:  Y[:, block i] = X[:, block i] A_i + b[block i] */
    LATMIX_FLAG_TEST_DROP_LOAD = 1 << 16  /* for tests of the failure path only: the single-CTA block-scaled product (kernel
                                      selection 1-3 below) leaves out the loads of the second 128-byte K slab of output tile
                                      0, so that the waits for them expire and the call ends with LATMIX_ERR_TIMEOUT in the
                                      status word; tile 0's part of `out` is then not written */
};
/* Bits 8-11 of `flags` select a kernel where several apply (for tests and measurements; results agree bit for bit in the
 * block-scaled product, up to near-ties in the transform): 0 = the library's choice by shape, 1-3 = single-CTA tensor-core
 * kernels (tile 128 x 128, 128 x 192, 128 x 256), 4 = the small-batch kernels (product and transform: M <= 64,
 * transform K <= 16384), 5 = the small-batch MXINT8 product that converts the weights to bf16 on the way to the tensor
 * core instead of multiplying the integer codes (M <= 16 only; same results up to the order of fp32 roundings), 8 = the CTA-pair
 * kernels (product: 256 x 192 tiles), 9 = the product on CTA pairs with 256 x 256 tiles (the default for M > 128).  A value
 * whose kernel does not take the shape falls back to the next that does. */
#define LATMIX_FLAG_KERNEL(v) ((uint32_t)(v) << 8)

/* Host helpers (no device work). ------------------------------------------------------------------------- */

/* Bytes of the code buffer and of the scale buffer for `rows` rows of K elements. */
latmix_status_t latmix_mx_sizes(int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf,
                                size_t* code_bytes, size_t* scale_bytes);

/* Byte offset of the scale of (row, kblock) in a scale buffer with the given layout; (size_t)-1 on bad input. */
size_t latmix_scale_offset(int64_t row, int64_t kblock, int64_t rows, int64_t K, latmix_sf_layout_t sf);

/* The same for any format: for LATMIX_NVFP4 `kblock` counts blocks of 16 elements (K/16 per row, tiles of 128 rows x 4
 * blocks, blocks padded to a multiple of 16); for the MX formats it is latmix_scale_offset. */
size_t latmix_scale_offset_fmt(int64_t row, int64_t kblock, int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf);

/* LATMIX_NVFP4: byte offset, inside a scale buffer of latmix_mx_sizes(rows, K, LATMIX_NVFP4, sf) bytes, of the fp32 tensor
 * scale (the start of the 16-byte trailer behind the block scales); (size_t)-1 for the other formats. */
size_t latmix_tensor_scale_offset(int64_t rows, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf);

/* Bytes of device workspace the given call needs for these sizes (always >= 256: the status word lives there). */
latmix_status_t latmix_workspace_bytes(latmix_op_t op, int64_t M, int64_t K, int64_t N, latmix_format_t fmt,
                                       size_t* bytes);

const char* latmix_status_string(latmix_status_t s);

/* Number of kernel launches this library has enqueued from the calling process so far (host counter). */
uint64_t latmix_launch_count(void);

/* Device calls. ------------------------------------------------------------------------------------------ */

/*
 * Offline fold and weight quantisation (Eq. "fold_kqv_1" in row form, then Eq. "q_mx" per output column):
 *   W~ = A_inv W (fp32-accurate), c = bias - b W~ (from the unquantised W~, accumulated in fp64),
 *   Wq = Q(W~) with blocks of 32 along K for each of the N output columns.
 * A_inv : K x K fp32.  b : K fp32 or NULL (= 0).  W : K x N of `w_dtype`.  bias : N fp32 or NULL (= 0).
 * Wq_codes  : N x K codes, K-major (N x K/2 bytes for MXFP4, N x K bytes otherwise).
 * Wq_scales : N x K/32 E8M0 bytes in layout `sf` (sizes from latmix_mx_sizes(N, K, ...)).
 * c_out     : N fp32.   Wfold_dump : NULL, or N x K fp32 receiving W~^T (the values that were quantised).
 * With bf16 weights and a workspace of latmix_workspace_bytes(LATMIX_OP_FOLD_WEIGHTS, ...) bytes (which includes room for
 * three bf16 copies of A_inv) the product runs on the tensor cores, A_inv entering as the sum of three bf16 terms;
 * with fp32 weights it does so too if the workspace has 6 K N more bytes (W as three bf16 terms as well, nine products; K a
 * multiple of 64); otherwise, or with a workspace of only 256 + 8 K bytes (rounded up to 256), it is an fp32 FMA product.
 */
latmix_status_t latmix_fold_weights(const void* A_inv, const float* b, const void* W, latmix_dtype_t w_dtype,
                                    const float* bias, int64_t K, int64_t N, latmix_format_t fmt,
                                    latmix_sf_layout_t sf, void* Wq_codes, void* Wq_scales, float* c_out,
                                    float* Wfold_dump, void* workspace, size_t workspace_bytes, uint32_t flags,
                                    void* cuda_stream);

/*
 * Offline fold with a transform on each side of the linear map (Sec. "Folding of T_1" and "Folding of T_2" of the
 * appendix on folding, in row form): the layer f(x) = x W + bias is replaced by f~~(x') = T_out(f(T_in^-1(x'))) with
 * T_in(x) = x A_in + b_in and T_out(y) = y A_out + v_out, i.e.
 *   W~~ = A_in_inv W A_out (fp32-accurate),  c = (bias - b_in A_in_inv W) A_out + v_out (fp64 accumulation),
 *   Wq = Q(W~~) with blocks of 32 along K for each of the N output columns.
 * The paper's cases: K and Q projections (A_1^-1, v_1 | none), Eq. "fold_kqv_1"; FFN and MHA output (none | A_1, no
 * shift), Eq. "fold_out_ffn"; V projection (A_1^-1, v_1 | A_2, v_2); MHA output projection (A_2^-1, v_2 | A_1, no shift).
 * For the last one the bias is b_O A_1 - v_2 A_2^-1 W_O A_1, which is what expanding f~_O(T_2^-1(x)) gives (the printed
 * equation puts both terms under one minus sign).
 * A_in_inv : K x K fp32 or NULL (no input side; b_in must then be NULL).  A_out : N x N fp32 or NULL (no output side;
 * v_out must then be NULL).  At least one side must be given.  b_in : K, bias / v_out : N, fp32 or NULL (= 0).
 * W, Wq_codes, Wq_scales, c_out, Wfold_dump (N x K fp32, W~~^T) as for latmix_fold_weights.
 * With A_out == NULL this is latmix_fold_weights, workspace included.  Otherwise the workspace must hold at least
 * 256 + 8 K + 4 N (+ 4 N K if both sides are given) bytes, each part rounded up to 256: the output-side product
 * (2 K N^2 flops) is then an fp32 FMA product.  With bf16 weights, K and N multiples of 64 and a workspace of
 * latmix_workspace_bytes(LATMIX_OP_FOLD_TWO_SIDED, ...) bytes (12 K N + 6 N^2 + 6 K^2 beyond the above, for transposed and
 * three-term bf16 copies of the operands) both products run on the tensor cores: T = W A_out with A_out as three bf16
 * terms, then A_in_inv T with both operands as three terms.
 */
latmix_status_t latmix_fold_weights_two_sided(const float* A_in_inv, const float* b_in, const void* W,
                                              latmix_dtype_t w_dtype, const float* bias, const float* A_out,
                                              const float* v_out, int64_t K, int64_t N, latmix_format_t fmt,
                                              latmix_sf_layout_t sf, void* Wq_codes, void* Wq_scales, float* c_out,
                                              float* Wfold_dump, void* workspace, size_t workspace_bytes,
                                              uint32_t flags, void* cuda_stream);

/*
 * Online transform + MX quantisation: codes, scales = Q(X A + b) (Definition of T, then Eq. "q_mx").
 * X : M x K of `x_dtype`.  A : K x K of the same dtype, or NULL for the identity (plain MX quantisation of
 * X + b).  b : K fp32 or NULL.  codes / scales as for the weights, with M rows.
 * Y_dump : NULL, or M x K fp32 receiving the transformed values exactly as they entered the quantiser.
 * With bf16 inputs the product runs on the tensor cores (bf16 x bf16 -> fp32); with fp32 inputs it is an
 * fp32 FMA product.  The accumulated fp32 value is quantised directly (never rounded to bf16 first).
 * With LATMIX_FLAG_BLOCK_DIAG, A holds K/32 blocks of 32 x 32 (same dtype as X) and the transform costs 64 flops per
 * element instead of 2 K: with bf16 inputs and K a multiple of 128 a warp-level tensor-core product (mma.sync, the blocks
 * held in registers), otherwise an fp32 FMA product; either way fused with the quantiser and bound by reading X.
 */
latmix_status_t latmix_quantize_mx(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                   int64_t M, int64_t K, latmix_format_t fmt, latmix_sf_layout_t sf,
                                   void* codes, void* scales, float* Y_dump, void* workspace,
                                   size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * Transformation mean squared error (Eq. "q_error") and the block-wise quantisation error of Sec. 3.1:
 *   e = x - T^-1(Q(T(x))) = (y - Q(y)) A_inv  with y = X A + b quantised exactly as latmix_quantize_mx does,
 *   block_err[i] = mean over the M rows and the 32 coordinates of block i of e^2   (K/32 doubles, device memory),
 *   *mse = mean of e^2 over all M K elements = mean of block_err                   (one double, device memory).
 * X, A, b as for latmix_quantize_mx (LATMIX_FLAG_BLOCK_DIAG included); A_inv : K x K fp32, the full inverse matrix also
 * when A is given as blocks.  A == NULL and A_inv == NULL together mean the identity (plain MX quantisation error of X + b).
 * The product (y - Q(y)) A_inv is fp32-accurate: on the tensor cores with both operands as three bf16 terms when M >= 64 is
 * a multiple of 8, K a multiple of 64 and the workspace has latmix_workspace_bytes(LATMIX_OP_TRANSFORMATION_MSE, ...) bytes;
 * as an fp32 FMA product otherwise.  Minimum workspace: 256 + codes + K/32 scale bytes per row + 8 M K bytes, each part
 * rounded up to 256.  Sums of squares are accumulated in fp64 in a fixed order: results are reproducible bit for bit.
 */
latmix_status_t latmix_transformation_mse(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                          const float* A_inv, int64_t M, int64_t K, latmix_format_t fmt, double* block_err,
                                          double* mse, void* workspace, size_t workspace_bytes, uint32_t flags,
                                          void* cuda_stream);

/*
 * The same diagnostic for another MX block size B (8, 16, 32, 64 or 128; K a multiple of B): the sweep over block sizes of
 * the numerical analysis in Sec. 3.1 (MSE against block size, block-wise error against block index).  y is computed as
 * above; its quantisation Q_B follows Eq. "q_mx" with blocks of B elements; block_err has K/B entries, each the mean over
 * the rows and the B coordinates of that block.  B = 32 is latmix_transformation_mse.  The block-scaled product of the layer
 * always works with B = 32: other sizes exist for this diagnostic only.
 */
latmix_status_t latmix_transformation_mse_block(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                                const float* A_inv, int64_t M, int64_t K, latmix_format_t fmt, int block,
                                                double* block_err, double* mse, void* workspace, size_t workspace_bytes,
                                                uint32_t flags, void* cuda_stream);

/*
 * Block-scaled contraction alone: out[M x N] = dq(a) dq(w)^T + c, fp32 output with leading dimension ldo.
 * a_codes / a_scales : M rows, w_codes / w_scales : N rows, both K-major with LATMIX_SF_TCGEN05 scales.
 * c : N fp32 or NULL.  Products of element values and power-of-two scales are exact; accumulation is fp32.
 * MXINT8 has no block-scaled tensor-core form: with a workspace of latmix_workspace_bytes(LATMIX_OP_MX_GEMM, ...) bytes
 * both operands are first expanded (exactly) to bf16 inside the workspace and multiplied on the tensor cores; with a
 * smaller workspace (at least the 256-byte header) the product runs on the CUDA cores.  For M <= 64 (and K a multiple of
 * 128) no scratch is used: the int8 codes are multiplied as they are on the integer tensor-core kind, one MX block per
 * instruction, and the block scales are applied to the exact int32 sums, which are then added in fp32 in K order.
 */
latmix_status_t latmix_mx_gemm(const void* a_codes, const void* a_scales, const void* w_codes,
                               const void* w_scales, const float* c, int64_t M, int64_t K, int64_t N,
                               latmix_format_t fmt, float* out, int64_t ldo, void* workspace,
                               size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * The whole layer: out[M x N] = Q(X A + b) Wq + c, i.e. latmix_quantize_mx into the workspace followed by
 * latmix_mx_gemm, on one stream.  Wq_codes / Wq_scales / c are what latmix_fold_weights produced with
 * LATMIX_SF_TCGEN05.  The activation codes and scales live in `workspace` and are overwritten by each call.
 * The workspace must hold the 256-byte header and those codes and scales; latmix_workspace_bytes(LATMIX_OP_LINEAR, ...)
 * asks for more with MXINT8 (room for the bf16 copies the tensor-core product uses), without which the MXINT8 product
 * runs on the CUDA cores.
 */
latmix_status_t latmix_linear(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                              const void* Wq_codes, const void* Wq_scales, const float* c, int64_t M, int64_t K,
                              int64_t N, latmix_format_t fmt, float* out, int64_t ldo, void* workspace,
                              size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * The whole layer again, for callers that cannot give the library a workspace (the paper has no counterpart: this
 * is a packaging variant of latmix_linear, same arithmetic, same kernels).  Meant for code that must not allocate
 * device memory: a plug-in running under a host application's allocator, a latency-critical loop whose memory map
 * is frozen after start-up, or any place where reaching cudaMalloc -- which synchronises the device -- is not
 * acceptable.  The status word and the activation codes and scales that latmix_linear keeps in the caller's
 * workspace live instead in one device array built into the library, LATMIX_STATIC_SCRATCH_BYTES long; every GPU
 * that loads the library holds that array until the process exits.
 *  - Sizes whose activation codes and scales (latmix_mx_sizes with LATMIX_SF_TCGEN05, each rounded up to 256 bytes, plus
 *    the 256-byte header) exceed LATMIX_STATIC_SCRATCH_BYTES are refused with LATMIX_ERR_WORKSPACE and nothing is
 *    launched; use latmix_linear for those.
 *  - The call allocates nothing and frees nothing.  The first call on each device looks up the array's device
 *    address (with that device current); make that first call outside of any stream capture.
 *  - All calls on a device share the one array and it keeps the previous call's contents; the status word is
 *    cleared at the start of each call.  Two calls that overlap on the GPU (different streams, no ordering
 *    between them) race on it: order them, or give all but one a workspace through latmix_linear.
 *  - device_status (host pointer, may be NULL): when given, the call waits for the stream and stores what
 *    latmix_device_status would report; when NULL the call returns without waiting and device-side problems of
 *    this call go unreported.
 * Every other argument is as for latmix_linear.
 */
#define LATMIX_STATIC_SCRATCH_BYTES ((size_t)256 + ((size_t)16 << 20))
latmix_status_t latmix_linear_static(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                     const void* Wq_codes, const void* Wq_scales, const float* c, int64_t M,
                                     int64_t K, int64_t N, latmix_format_t fmt, float* out, int64_t ldo,
                                     uint32_t flags, latmix_status_t* device_status, void* cuda_stream);

/*
 * Measurement aid (the paper has no counterpart; its Sec. 5.3 reports throughput only end to end): the rate at which the
 * tensor pipes retire MMAs when nothing else limits them.  One CTA per SM issues `mma_per_cta` (rounded down to a
 * multiple of 4; 4 .. 2^22) tcgen05.mma of shape 128 x 256 x k back to back on operands that sit in shared memory; the
 * results are discarded.  kind: 0 = kind::f16 with bf16 operands (k = 16), 1 = kind::mxf8f6f4 with E4M3 elements and E8M0
 * block scales (k = 32), 2 = kind::mxf4 with E2M1 elements and E8M0 block scales (k = 64), 3 = kind::mxf4nvf4 with E2M1
 * elements and E4M3 scales per 16 elements (k = 64), 4 = kind::mxf4 again but issued by CTA pairs (cta_group::2, one 256 x 256 x
 * 64 MMA per step and pair, `mma_per_cta` steps per pair; bits 8-23 of `kind`, a multiple of 4 or 0, make the issuing thread add
 * a tcgen05.commit after every so many MMAs, as a pipelined kernel does to release its stages).  *flops (host pointer) receives the floating-point operations the
 * launch performs on the whole device, 2 x 128 x 256 x k per MMA; time the stream around the call to get a rate.
 * workspace: at least the 256-byte header (the status word records a wait that expired).
 */
latmix_status_t latmix_tensor_pipe_probe(int kind, int64_t mma_per_cta, double* flops, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream);

/* Zero the header of a workspace: the status word and the wait limit (enqueued on the stream).  Call once after allocating it. */
latmix_status_t latmix_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Every wait inside a kernel (on a copy, on the tensor core, on another CTA of a cluster) gives up after about one
 * second, records LATMIX_ERR_TIMEOUT in the status word and lets the kernel end.  This call replaces that limit, for
 * kernels launched with this workspace, by `cycles` SM clock cycles (0 = back to the default; values below 32768 act as
 * 32768).  Enqueued on the stream.  Meant for tests of the failure path and for callers with a tighter deadline.
 */
latmix_status_t latmix_workspace_set_wait_limit(void* workspace, size_t workspace_bytes, uint32_t cycles, void* cuda_stream);

/*
 * LATMIX_NVFP4 with latmix_linear: the activation codes and scales live in the workspace, so the activations' tensor scale
 * cannot be written into their trailer by the caller; this call stores it in the workspace header (enqueued on the stream),
 * and latmix_linear moves it to the trailer on every call.  It stays until the header is re-initialised.  Must be positive.
 */
latmix_status_t latmix_workspace_set_tensor_scale(void* workspace, size_t workspace_bytes, float tensor_scale, void* cuda_stream);

/* Synchronise the stream and return the status word of `workspace` (LATMIX_OK if no kernel recorded a problem). */
latmix_status_t latmix_device_status(void* workspace, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LATMIX_H_ */
