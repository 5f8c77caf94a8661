"""Helpers shared by the GPU parity tests: moving MX tensors between the oracle's unpacked numpy form and the
library's packed device buffers.  Layout arithmetic only; no quantiser arithmetic."""
import numpy as np
import torch

from oracle import latmix_oracle as orc

FMT_NAME = {0: "mxfp4", 1: "mxfp8", 2: "mxint8", 3: "mxint4", 4: "nvfp4"}


def sf_offsets(rows, K):
    r = np.arange(rows)[:, None]
    kb = np.arange(K // 32)[None, :]
    kt = ((K // 32 + 7) // 8) * 2
    return ((r >> 7) * kt + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3)


def scales_to_linear(B, scales, rows, K, sf):
    """Gather the scale bytes of a device scale buffer into a [rows, K/32] uint8 array."""
    buf = scales.cpu().numpy()
    if sf == B.SF_LINEAR:
        return buf[: rows * (K // 32)].reshape(rows, K // 32).copy()
    off = sf_offsets(rows, K)
    assert off[-1, -1] == B.scale_offset(rows - 1, K // 32 - 1, rows, K, sf)
    return buf[off]


def codes_to_numpy(codes_t, rows, K, fmt):
    buf = codes_t.cpu().numpy()
    if fmt == 0:
        return orc.unpack_fp4(buf[: rows * K // 2].reshape(rows, K // 2))
    return bytes_to_codes(buf[: rows * K].reshape(rows, K).copy(), fmt)


def bytes_to_codes(out, fmt):
    """One-byte-per-element buffers as the oracle's codes.  MXFP8 / MXINT8: the byte is the code.  MXINT4: the library
    stores element k as the E4M3 byte of k, the oracle's code is 4-bit two's complement: container -> integer -> code; a
    container that holds anything but an integer in [-7, 7], or a negative zero, maps to the impossible code 0xFF."""
    if fmt != 3:
        return out
    val = orc.decode_elements(out, "mxfp8")
    ok = (val == np.rint(val)) & (np.abs(val) <= 7) & (out != 0x80) & ((out & 0x7F) != 0x7F)
    return np.where(ok, val.astype(np.int64) & 0xF, 0xFF).astype(np.uint8)


def mx_to_device(B, codes, scale_bytes, fmt, dev="cuda"):
    rows, K = codes.shape
    cb, sb = B.mx_sizes(rows, K, fmt, B.SF_TCGEN05)
    packed = orc.pack_fp4(codes) if fmt == 0 else codes
    if fmt == 3:                                  # 4-bit two's complement -> integer -> its E4M3 byte
        packed = orc.quantize_elements_arith(orc.decode_elements(codes, "mxint4"), "mxfp8")
        packed[packed == 0x80] = 0
    buf = np.zeros(max(sb, 16), dtype=np.uint8)
    buf[sf_offsets(rows, K)] = scale_bytes
    flat = np.zeros(max(cb, 16), dtype=np.uint8)
    flat[:cb] = packed.reshape(-1)
    return torch.from_numpy(flat).to(dev), torch.from_numpy(buf).to(dev)


def random_mx(rows, K, fmt, seed, spread=6):
    rng = np.random.default_rng(seed)
    if fmt == 0:
        codes = rng.integers(0, 16, (rows, K), dtype=np.uint8)
    elif fmt == 1:
        codes = rng.integers(0, 256, (rows, K), dtype=np.uint8)
        codes[(codes & 0x7F) == 0x7F] = 0x31
    elif fmt == 3:
        codes = rng.integers(0, 16, (rows, K), dtype=np.uint8)
        codes[codes == 0x8] = 0x9                 # -8 is outside the symmetric range
    else:
        codes = rng.integers(0, 256, (rows, K), dtype=np.uint8)
        codes[codes == 0x80] = 0x7F
    scales = rng.integers(127 - spread, 128 + spread, (rows, K // 32), dtype=np.uint8)
    return codes, scales


def rel_fro(a, b):
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def tensor_core_unit(K):
    """Relative size of the accumulation error of the bf16 tensor-core product, per unit of sum |x||a|.

    Products of bf16 values are exact in fp32; the accumulator in tensor memory is rounded (or truncated)
    to fp32 once per instruction, i.e. K/16 times, each time by at most 2^-24 (2^-23 if truncated) of a
    partial sum that never exceeds sum |x||a|; 16 more roundings cover the sum inside one instruction.
    Measured on B200 the largest error is 4 to 12 times below this bound (2^-19.9, 2^-18.9, 2^-17.8 of
    sum |x||a| at K = 1024, 4096, 14336)."""
    return (K / 16.0 + 16.0) * 2.0 ** -24


def fma_unit(K):
    """Same for a sequential fp32 FMA chain of length K (the CUDA-core product): gamma_K ~ K 2^-24."""
    return (K + 2.0) * 2.0 ** -24


def accumulation_tau(X64, A64, unit):
    """Per-element bound on the difference between an fp32-accumulated and the exact product."""
    return unit * (np.abs(X64) @ np.abs(A64)) + 1e-30


K_PER_MMA = {"mxfp4": 64, "mxfp8": 32, "mxint4": 32, "mxint8": 16}      # MXINT8 runs as an exact bf16 product


def block_scaled_unit(K, fmt_name, simt=False):
    """Relative size of the accumulation error of the block-scaled product, per unit of sum |dq(a)||dq(w)|.

    Products of element values and power-of-two scales are exact.  On the tensor cores the products of one MMA
    instruction are aligned to the largest exponent among them and added to the fp32 accumulator with truncation, so an
    instruction can lose up to 2^-23 of a partial sum that never exceeds sum |a||w|; there are K / k_per_mma instructions,
    and four more units cover the sum inside one instruction.  The CUDA-core kernel adds one 32-term fp32 FMA chain per
    block and then K/32 block sums across 32 lanes and a five-step shuffle tree.
    This is a worst-case bound.  Measured on B200 with random codes and block scales spread over 2^+-6 the largest error is
    7 to 15 units of 2^-24 where the bound is 24 to 72 (K = 256 to 2048; a bound of one 2^-24 per instruction was exceeded
    by 7 of 15.7 million elements at K = 256, MXFP8); on layer data, whose products cancel, it stays below 1 unit."""
    if simt:
        return (32 + K / 1024.0 + 6.0) * 2.0 ** -24
    return (K / K_PER_MMA[fmt_name] + 4.0) * 2.0 ** -23


def gemm_error_ratio(out, ref, a_codes, a_scales, w_codes, w_scales, fmt_name, c=None):
    """Largest |out - ref| in units of 2^-24 of sum_k |dq(a)_k| |dq(w)_k| (+ |c|)."""
    Ad = np.abs(orc.mx_dequantize(a_codes, a_scales, fmt_name))
    Wd = np.abs(orc.mx_dequantize(w_codes, w_scales, fmt_name))
    mag = Ad @ Wd.T + (0.0 if c is None else np.abs(np.asarray(c, dtype=np.float64))[None, :])
    err = np.abs(np.asarray(out, dtype=np.float64) - ref)
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(mag > 0, err / (mag * 2.0 ** -24), np.where(err > 0, np.inf, 0.0))
    return float(ratio.max()), mag


def assert_gemm_parity(out, ref, a_codes, a_scales, w_codes, w_scales, fmt_name, K, c=None, simt=False, tol=1e-4, tag=""):
    """Block-scaled product against the fp64 contraction of the same codes: relative Frobenius norm within `tol` AND every
    element within the accumulation bound  |out - ref| <= u (sum_k |dq(a)_k||dq(w)_k| + |c|) + one fp32 rounding of the
    result (u: block_scaled_unit; simt=None takes the larger of the two kernels' units where the shape decides which one
    runs).  A single wrong element fails the second check at any matrix size."""
    out = np.asarray(out, dtype=np.float64)
    assert np.isfinite(out).all(), tag
    assert rel_fro(out, ref) < tol, (tag, rel_fro(out, ref))
    ratio, mag = gemm_error_ratio(out, ref, a_codes, a_scales, w_codes, w_scales, fmt_name, c)
    unit = (max(block_scaled_unit(K, fmt_name, False), block_scaled_unit(K, fmt_name, True)) if simt is None
            else block_scaled_unit(K, fmt_name, simt))
    bound = unit * mag + 2.0 ** -23 * np.abs(ref) + 1e-300
    bad = np.abs(out - ref) > bound
    print(f"GEMM_ERR {tag} fmt={fmt_name} K={K} max_err_over_2^-24_mag={ratio:.2f} bound={unit * 2 ** 24:.1f}")
    assert not bad.any(), (tag, int(bad.sum()), ratio)


# ---- NVFP4 (blocks of 16, E4M3 block scales, tensor scale in the scale buffer's trailer)
def nvfp4_sf_offsets(rows, K):
    r = np.arange(rows)[:, None]
    kb = np.arange(K // 16)[None, :]
    kt = ((K // 16 + 15) // 16) * 4
    return ((r >> 7) * kt + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3)


def nvfp4_scales_to_linear(B, scales, rows, K, sf):
    buf = scales.cpu().numpy()
    if sf == B.SF_LINEAR:
        return buf[: rows * (K // 16)].reshape(rows, K // 16).copy()
    off = nvfp4_sf_offsets(rows, K)
    assert off[-1, -1] == B.scale_offset_fmt(rows - 1, K // 16 - 1, rows, K, B.NVFP4, sf)
    return buf[off]


def nvfp4_to_device(B, codes, scale_codes, g, dev="cuda"):
    rows, K = codes.shape
    cb, sb = B.mx_sizes(rows, K, B.NVFP4, B.SF_TCGEN05)
    buf = np.zeros(sb, dtype=np.uint8)
    buf[nvfp4_sf_offsets(rows, K)] = scale_codes
    off = B.tensor_scale_offset(rows, K, B.NVFP4, B.SF_TCGEN05)
    buf[off:off + 4] = np.frombuffer(np.float32(g).tobytes(), dtype=np.uint8)
    flat = np.zeros(max(cb, 16), dtype=np.uint8)
    flat[:cb] = orc.pack_fp4(codes).reshape(-1)
    return torch.from_numpy(flat).to(dev), torch.from_numpy(buf).to(dev)
