// Device-side arithmetic of the MX quantiser (Eq. "q_mx"): shared-scale exponent, exact power-of-two
// scaling, element conversion and packing.  Everything here works on fp32 values; the element conversions
// are the hardware round-to-nearest-even, saturate-to-finite conversions.
#pragma once
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace latmix {

// FMT_INT4: integers k in [-7, 7], each stored as the E4M3 byte of k, so that the 8-bit block-scaled tensor-core kind
// consumes the codes as they are (the products stay exact)
// FMT_NVFP4: E2M1 elements packed like FMT_FP4, blocks of 16 with an E4M3 scale each, one fp32 scale per tensor
enum : int { FMT_FP4 = 0, FMT_FP8 = 1, FMT_INT8 = 2, FMT_INT4 = 3, FMT_NVFP4 = 4 };

// r_max of Eq. "q_mx": exponent of the top binade of the element format.
template <int FMT> struct FormatTraits;
template <> struct FormatTraits<FMT_FP4>  { static constexpr int kRMax = 2; static constexpr int kBitsLog2 = 2; };
template <> struct FormatTraits<FMT_FP8>  { static constexpr int kRMax = 8; static constexpr int kBitsLog2 = 3; };
template <> struct FormatTraits<FMT_INT8> { static constexpr int kRMax = 0; static constexpr int kBitsLog2 = 3; };
template <> struct FormatTraits<FMT_INT4> { static constexpr int kRMax = 2; static constexpr int kBitsLog2 = 3; };

// E8M0 byte of s_i = 2^(floor(log2 amax) - r_max): the biased exponent field of amax minus r_max, clamped
// at 0.  amax == 0 and subnormal amax have field 0 and so clamp to byte 0 (scale 2^-127).
__device__ __forceinline__ uint32_t scale_byte_from_amax(float amax, int r_max) {
    int e = (int)((__float_as_uint(amax) >> 23) & 0xFFu) - r_max;
    return (uint32_t)(e < 0 ? 0 : e);
}

// The two factors whose product is 2^-E = 2^(127 - byte).  Both are normal fp32 numbers, so
// (y * f.x) * f.y is the exact quotient y / s_i whenever that quotient is a normal number, and a value
// far below every rounding boundary otherwise.
__device__ __forceinline__ float2 inv_scale_factors(uint32_t scale_byte) {
    int p = 127 - (int)scale_byte;       // in [-127, 127]
    int h1 = p / 2, h2 = p - h1;
    return make_float2(__uint_as_float((uint32_t)(h1 + 127) << 23), __uint_as_float((uint32_t)(h2 + 127) << 23));
}

// 2^-E = 2^(127 - byte) as ONE fp32 factor: a normal number except for byte 254, where it is the subnormal 2^-127
// (fp32 multiplication takes subnormal operands as they are; nothing here is compiled with flush-to-zero).
// y * factor is the exact quotient y / s_i whenever that quotient is a normal number.
__device__ __forceinline__ float inv_scale_factor(uint32_t scale_byte) {
    const uint32_t e = 254u - min(scale_byte, 254u);
    return __uint_as_float(e == 0u ? 0x00400000u : e << 23);
}

__device__ __forceinline__ float scale_to_float(uint32_t scale_byte) {   // 2^(byte-127); byte 0 is subnormal
    return scale_byte == 0 ? __uint_as_float(0x00400000u) : __uint_as_float(scale_byte << 23);
}

// 8 scaled values -> packed codes.  FP4: one 32-bit word, element 2t in the low nibble of byte t.
__device__ __forceinline__ uint32_t pack8_fp4(const float* v) {
    // cvt.rn.satfinite.e2m1x2.f32 d, a, b: a lands in the upper four bits of the byte, b in the lower four
    uint32_t w;
    asm("{\n\t.reg .b8 q0, q1, q2, q3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 q0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 q1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 q2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 q3, %8, %7;\n\t"
        "mov.b32 %0, {q0, q1, q2, q3};\n\t}"
        : "=r"(w)
        : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
    return w;
}

// 8 scaled values -> 8 bytes (two 32-bit words), FP8 E4M3.
__device__ __forceinline__ uint2 pack8_fp8(const float* v) {
    uint32_t w[2] = {0, 0};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        __nv_fp8x2_storage_t p = __nv_cvt_float2_to_fp8x2(make_float2(v[2 * t], v[2 * t + 1]), __NV_SATFINITE, __NV_E4M3);
        w[t >> 1] |= (uint32_t)p << (16 * (t & 1));
    }
    return make_uint2(w[0], w[1]);
}

// 8 scaled values -> 8 two's complement bytes, value k/64 with k clamped to +-127.
__device__ __forceinline__ uint2 pack8_int8(const float* v) {
    uint32_t w[2] = {0, 0};
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        int k = __float2int_rn(v[t] * 64.0f);
        k = max(-127, min(127, k));
        w[t >> 2] |= ((uint32_t)k & 0xFFu) << (8 * (t & 3));
    }
    return make_uint2(w[0], w[1]);
}

// 8 scaled values -> 8 bytes, each the E4M3 encoding of the integer k = round-to-nearest-even(v) clamped to +-7 (every such
// k is exact in E4M3; adding +0 turns a negative zero into the one zero an integer format has).
__device__ __forceinline__ uint2 pack8_int4(const float* v) {
    float k[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) k[t] = fminf(fmaxf(rintf(v[t]), -7.0f), 7.0f) + 0.0f;
    return pack8_fp8(k);
}

// The 8-bit formats by template argument.
template <int FMT> __device__ __forceinline__ uint2 pack8_bytes(const float* v) {
    if (FMT == FMT_FP8) return pack8_fp8(v);
    if (FMT == FMT_INT4) return pack8_int4(v);
    return pack8_int8(v);
}

// Value of one element code (no block scale).
template <int FMT> __device__ __forceinline__ float decode_element(uint32_t code);
template <> __device__ __forceinline__ float decode_element<FMT_FP4>(uint32_t c) {
    uint32_t m = c & 7u;
    // 0 .5 1 1.5 2 3 4 6: subnormal .5*m for m<2, else (1 + (m&1)/2) * 2^((m>>1)-1)
    float mag = m < 2 ? 0.5f * (float)m : __uint_as_float(((126u + (m >> 1)) << 23) | ((m & 1u) << 22));
    return (c & 8u) ? -mag : mag;
}
template <> __device__ __forceinline__ float decode_element<FMT_FP8>(uint32_t c) {
    uint32_t e = (c >> 3) & 15u, m = c & 7u;
    float mag = e == 0 ? (float)m * 0.001953125f : __uint_as_float(((e + 120u) << 23) | (m << 20));
    return (c & 0x80u) ? -mag : mag;
}
template <> __device__ __forceinline__ float decode_element<FMT_INT4>(uint32_t c) { return decode_element<FMT_FP8>(c); }
template <> __device__ __forceinline__ float decode_element<FMT_INT8>(uint32_t c) {
    return (float)(int)(int8_t)(c & 0xFFu) * 0.015625f;
}

// Byte offset of the scale of (row, kblock) in the tcgen05 layout: tiles of 128 rows x 4 blocks.
__host__ __device__ __forceinline__ size_t sf_tcgen05_offset(int64_t row, int64_t kb, int64_t k_tiles) {
    return (size_t)((row >> 7) * k_tiles + (kb >> 2)) * 512 + (size_t)((row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb & 3));
}
__host__ __device__ __forceinline__ int64_t sf_k_tiles(int64_t K) { return ((K / 32 + 7) / 8) * 2; }  // blocks padded to 8
// NVFP4: a tile holds 128 rows x 4 blocks of 16 elements; blocks padded to 16, i.e. k-tiles to a multiple of 4 (one 128-byte slab)
__host__ __device__ __forceinline__ int64_t nvfp4_sf_k_tiles(int64_t K) { return ((K / 16 + 15) / 16) * 4; }

// NVFP4 scale buffers end with a 16-byte trailer whose first four bytes hold the tensor's fp32 scale; this is the
// trailer's offset, i.e. the bytes the block scales take (linear: rows x K/16 bytes rounded up to 16; tiled: whole tiles).
__host__ __device__ __forceinline__ size_t nvfp4_block_scale_bytes(int64_t rows, int64_t K, int sf_layout) {
    return sf_layout == 0 ? (size_t)((rows * (K / 16) + 15) / 16 * 16) : (size_t)((rows + 127) / 128) * (size_t)nvfp4_sf_k_tiles(K) * 512;
}
__host__ __device__ __forceinline__ const float* nvfp4_tensor_scale_ptr(const uint8_t* scales, int64_t rows, int64_t K, int sf_layout) {
    return reinterpret_cast<const float*>(scales + nvfp4_block_scale_bytes(rows, K, sf_layout));
}

// One NVFP4 block: 16 fp32 values -> the block's E4M3 scale code and eight bytes of E2M1 codes, for tensor scale g.
// fp32 arithmetic, one IEEE operation per step, in this order (no fused multiply-add, no reciprocal approximation):
//   t = (amax / 6) / g;  d = E4M3(t), round to nearest even, saturating;  s = d * g;  r = 1 / s (0 if s == 0);
//   code_j = E2M1(v_j * r), round to nearest even, saturating, sign kept.
__device__ __forceinline__ uint32_t nvfp4_quantize_block(const float* v, float g, uint2& packed) {
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
    const float t = __fdiv_rn(__fdiv_rn(amax, 6.0f), g);
    const uint32_t d_code = (uint32_t)__nv_cvt_float_to_fp8(t, __NV_SATFINITE, __NV_E4M3) & 0xFFu;
    const uint32_t e = (d_code >> 3) & 15u, m = d_code & 7u;
    const float d = e == 0 ? (float)m * 0.001953125f : __uint_as_float(((e + 120u) << 23) | (m << 20));
    const float s = __fmul_rn(d, g);
    const float r = s > 0.f ? __fdiv_rn(1.0f, s) : 0.f;
    float w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = __fmul_rn(v[i], r);
    packed = make_uint2(pack8_fp4(w), pack8_fp4(w + 8));
    return d_code;
}

// 2^(E-6) for scale byte E + 127, exact (byte 0: 2^-133, a subnormal)
__device__ __forceinline__ float int8_mult(uint32_t scale_byte) { return scale_to_float(scale_byte) * 0.015625f; }

// 16 int8 codes (one 16-byte chunk) times the block's scale -> 16 bf16 (two 16-byte chunks).  A byte b ^ 0x80 placed in the
// mantissa of 2^23 is the float 2^23 + 128 + k; one fused multiply-add takes it to k * mult exactly (k * mult is
// representable, so the single rounding of the fma changes nothing).  For the largest scales (2^23 + 128) * mult would
// leave fp32's range although k * mult does not: those blocks are converted with mult * 2^-32 and scaled back, on a
// branch of its own so that the common path carries none of its instructions.
template <bool BIG>
__device__ __forceinline__ void int8x16_to_bf16_impl(const uint4& raw, float mult, uint4& lo, uint4& hi) {
    const float m = BIG ? mult * 2.3283064e-10f : mult;   // * 2^-32
    const float off = -8388736.0f * m;                    // -(2^23 + 128) * m, exact
    const uint32_t w[4] = {raw.x ^ 0x80808080u, raw.y ^ 0x80808080u, raw.z ^ 0x80808080u, raw.w ^ 0x80808080u};
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float f0 = fmaf(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7440)), m, off);
        float f1 = fmaf(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7441)), m, off);
        float f2 = fmaf(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7442)), m, off);
        float f3 = fmaf(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7443)), m, off);
        if (BIG) { f0 *= 4294967296.0f; f1 *= 4294967296.0f; f2 *= 4294967296.0f; f3 *= 4294967296.0f; }
        // k * mult has at most seven significant bits (and is a multiple of bf16's smallest subnormal), so its bf16 form is the
        // upper half of its fp32 form: a byte permutation instead of a rounding conversion (a quarter-rate instruction)
        o[2 * i] = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
        o[2 * i + 1] = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
    }
    lo = make_uint4(o[0], o[1], o[2], o[3]);
    hi = make_uint4(o[4], o[5], o[6], o[7]);
}
__device__ __forceinline__ void int8x16_to_bf16(const uint4& raw, float mult, uint4& lo, uint4& hi) {
    if (mult >= 1.2676506e30f) int8x16_to_bf16_impl<true>(raw, mult, lo, hi);      // 2^100 and above: rare
    else int8x16_to_bf16_impl<false>(raw, mult, lo, hi);
}

// Four consecutive lanes own one MX block, eight values each: block maximum over the four lanes, scale byte, and the
// eight values divided by the
// scale (one multiplication: 2^(127 - byte) is a single fp32 number).  All 32 lanes must call it.
template <int FMT>
__device__ __forceinline__ uint32_t scale_block_of_4_lanes(float (&v)[8]) {
    float amax = fmaxf(fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3]))),
                       fmaxf(fmaxf(fabsf(v[4]), fabsf(v[5])), fmaxf(fabsf(v[6]), fabsf(v[7]))));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    const uint32_t sb = scale_byte_from_amax(amax, FormatTraits<FMT>::kRMax);
    const float f = inv_scale_factor(sb);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] *= f;
    return sb;
}

__device__ __forceinline__ float load_as_float(const float* p) { return *p; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

}  // namespace latmix
