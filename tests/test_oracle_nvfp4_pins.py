"""Pins for the oracle's NVFP4 quantiser (blocks of 16, E2M1 elements, E4M3 block scale, fp32 tensor scale).

The paper evaluates the format (appendix "NVFP Quantization Format Evaluation") but defines nothing, so what is pinned
here is what the format's public description and arithmetic fix: a worked example derived by hand, an exact-rational
brute force that does every rounding on integers, the reduction to plain E2M1 rounding when the block scale is a power of
two, NVIDIA's host E4M3 conversion for the block scale, and invariants any implementation of the format must have.  The
choice of the block scale (amax / 6 over the tensor scale, rounded to nearest) is a reading: parity unpinned."""
import os
import shutil
import subprocess

import numpy as np
import pytest

from oracle import latmix_oracle as orc
from tests.conftest import read_golden

HERE = os.path.dirname(os.path.abspath(__file__))
E2M1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])


def _blocks(rng, rows, nb, spread=3.0):
    Y = rng.standard_normal((rows, nb * 16)) * np.exp(rng.standard_normal((rows, nb)) * spread).repeat(16, axis=1)
    return Y.astype(np.float32).astype(np.float64)


def test_worked_example():
    g = read_golden("nvfp4_example.txt")
    Y = np.zeros((1, 32))
    b0, b1 = [float(t) for t in g["block0"]], [float(t) for t in g["block1"]]
    Y[0, :len(b0)] = b0
    Y[0, 16:16 + len(b1)] = b1
    codes, scales = orc.nvfp4_quantize(Y, float(g["g"][0]))
    assert codes[0, :len(b0)].tolist() == [int(t) for t in g["codes0"]]
    assert codes[0, 16:16 + len(b1)].tolist() == [int(t) for t in g["codes1"]]
    assert scales[0].tolist() == [int(g["scale0"][0]), int(g["scale1"][0])]
    assert not codes[0, len(b0):16].any() and not codes[0, 16 + len(b1):].any()
    dq = orc.nvfp4_dequantize(codes, scales, float(g["g"][0]))
    assert dq[0, 16:18].tolist() == [float(t) for t in g["dq1"]]


def test_against_exact_rational_brute_force():
    rng = np.random.default_rng(3)
    for trial in range(40):
        g = np.float32(np.exp(rng.uniform(-12, 6)))
        Y = _blocks(rng, 2, 2)
        if trial % 5 == 0:
            Y[0, :16] = 0.0                                    # an all-zero block
        if trial % 7 == 0:
            Y[1, 16:] = np.float32(6.0 * 448.0 * g) * np.sign(Y[1, 16:])   # the largest representable magnitudes
        if trial % 9 == 0:
            Y[0, 16:] *= 1e-6                                  # a scale that rounds to an E4M3 subnormal or to zero
        codes, scales = orc.nvfp4_quantize(Y, g)
        for r in range(2):
            for b in range(2):
                want_c, want_s = orc.nvfp4_quantize_block_exact(Y[r, 16 * b:16 * b + 16], g)
                assert codes[r, 16 * b:16 * b + 16].tolist() == want_c, (trial, r, b)
                assert scales[r, b] == want_s, (trial, r, b)


def test_power_of_two_scale_reduces_to_plain_e2m1_rounding():
    """g = 2^j and amax = 6 * 2^k make every step exact: the block scale is 2^(k-j) and the codes are Q_e(y / 2^k), which the
    search quantiser (an implementation of its own) gives directly."""
    rng = np.random.default_rng(4)
    for j, k in [(0, 0), (-3, 2), (5, -1), (-6, -9), (2, 9)]:
        Y = rng.uniform(-6, 6, (8, 64))
        Y[:, ::16] = 6.0                                        # pins amax of every block
        Y = np.ldexp(Y.astype(np.float32).astype(np.float64), k)
        codes, scales = orc.nvfp4_quantize(Y, 2.0 ** j)
        assert np.array_equal(orc.decode_elements(scales, "mxfp8"), np.full(scales.shape, 2.0 ** (k - j)))
        assert np.array_equal(codes, orc.quantize_elements_search(np.ldexp(Y, -k), "mxfp4"))


def test_invariants():
    rng = np.random.default_rng(5)
    Y = _blocks(rng, 64, 8)
    g = orc.nvfp4_tensor_scale(np.abs(Y).max())
    codes, scales = orc.nvfp4_quantize(Y, g)
    assert codes.max() <= 0xF and (scales < 0x7F).all()        # scale: positive, finite E4M3
    d = orc.decode_elements(scales, "mxfp8")
    s = (d.astype(np.float32) * g).astype(np.float64)
    dq = orc.nvfp4_dequantize(codes, scales, g)
    exact_s = d * float(g)                                      # dequantisation multiplies exactly; s is its fp32 rounding
    for e in np.unique(codes & 7):                              # every value is an E2M1 element times the block's d * g
        sel = ((codes & 7) == e).reshape(64, 8, 16)
        assert np.array_equal(np.abs(dq).reshape(64, 8, 16)[sel], (E2M1[e] * np.broadcast_to(exact_s[:, :, None], sel.shape))[sel])
    # Blocks whose scale is a normal E4M3 number (d >= 2^-6: the rounding of the scale is then within 2^-4 relative).
    # The largest gap of E2M1 is 2 (between 4 and 6): the error never exceeds one unit of the block's scale; and the
    # block's largest element always lands on the largest code, because amax / s lies within E4M3's rounding of 6.
    normal = d >= 2.0 ** -6
    assert normal.mean() > 0.5 and (~normal).any()              # the sample has both kinds
    err = np.abs(Y - dq).reshape(64, 8, 16)
    assert (err <= s[:, :, None] * (1 + 2.0 ** -20))[normal].all()
    amax_pos = np.abs(Y).reshape(64, 8, 16).argmax(axis=2)
    top = np.take_along_axis(codes.reshape(64, 8, 16), amax_pos[:, :, None], axis=2)[:, :, 0]
    assert ((top & 7) == 7)[normal].all()
    # a scale that underflows E4M3 altogether leaves a block of (signed) zeros
    assert not ((codes & 7).reshape(64, 8, 16)[d == 0]).any()
    # the tensor's largest block uses the largest scale code region: d <= 448
    assert d.max() <= 448.0 and d.max() >= 448.0 / 1.07
    # negation flips sign bits only; scaling values and tensor scale together changes nothing
    c2, s2 = orc.nvfp4_quantize(-Y, g)
    assert np.array_equal(c2, codes ^ 8) and np.array_equal(s2, scales)
    c3, s3 = orc.nvfp4_quantize(np.ldexp(Y, 7), np.ldexp(g, 7))
    assert np.array_equal(c3, codes) and np.array_equal(s3, scales)
    # zero block: zero scale, zero codes (sign bits kept)
    Z = np.zeros((1, 16)); Z[0, 3] = -0.0
    cz, sz = orc.nvfp4_quantize(Z, g)
    assert sz.tolist() == [[0]] and cz[0, 3] == 8 and not (cz & 7).any()
    # idempotent where the scale is a normal E4M3 number: quantising the dequantised values gives the same codes and scales
    c4, s4 = orc.nvfp4_quantize(dq, g)
    assert np.array_equal(s4[normal], scales[normal])
    assert np.array_equal((c4 & 7).reshape(64, 8, 16)[normal], (codes & 7).reshape(64, 8, 16)[normal])


def test_matmul_against_explicit_loops():
    rng = np.random.default_rng(6)
    A, W = _blocks(rng, 3, 2, 1.0), _blocks(rng, 4, 2, 1.0)
    ga, gw = orc.nvfp4_tensor_scale(np.abs(A).max()), orc.nvfp4_tensor_scale(np.abs(W).max())
    ac, asc = orc.nvfp4_quantize(A, ga)
    wc, wsc = orc.nvfp4_quantize(W, gw)
    c = rng.standard_normal(4)
    got = orc.nvfp4_matmul(ac, asc, ga, wc, wsc, gw, c)
    sign = lambda code: -1.0 if code & 8 else 1.0
    for m in range(3):
        for n in range(4):
            tot = 0.0
            for k in range(32):
                a = sign(ac[m, k]) * E2M1[ac[m, k] & 7] * orc.MXFP8.grid[asc[m, k // 16]] * float(ga)
                w = sign(wc[n, k]) * E2M1[wc[n, k] & 7] * orc.MXFP8.grid[wsc[n, k // 16]] * float(gw)
                tot += a * w
            assert np.isclose(got[m, n], tot + c[n], rtol=1e-13, atol=0)


def test_block_scale_matches_nvidia_host_e4m3_conversion(tmp_path):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not available")
    exe = str(tmp_path / "nv_host_cvt")
    subprocess.run([nvcc, "-O1", "-o", exe, os.path.join(HERE, "nv_host_cvt.cu")], check=True)
    rng = np.random.default_rng(7)
    Y = _blocks(rng, 200, 4)
    g = orc.nvfp4_tensor_scale(np.abs(Y).max())
    _, scales = orc.nvfp4_quantize(Y, g)
    amax = np.abs(Y.astype(np.float32)).reshape(200, 4, 16).max(axis=2)
    t = (amax / np.float32(6.0)) / g                            # the two fp32 divisions, then NVIDIA's conversion
    text = "\n".join(float(v).hex() for v in t.ravel()) + "\n"
    out = subprocess.run([exe], input=text, capture_output=True, text=True, check=True).stdout
    nv = np.array([int(line.split()[1]) for line in out.strip().splitlines()]).reshape(200, 4)
    assert np.array_equal(nv, scales)
