"""Pins for the CPU oracle: what the paper prints, what the mathematics fixes,
and brute force on tiny inputs.  None of these re-type the oracle's formulas;
each would fail for a plausible mistake (dropped term, wrong sign, floor vs
ceil, transposed operand, wrong tie rule, wrong nibble)."""
import itertools
import math

import numpy as np
import pytest

from oracle import latmix_oracle as orc
from tests.conftest import read_golden

FMTS = ["mxfp4", "mxfp8", "mxint8", "mxint4"]
OCP_FMTS = ["mxfp4", "mxfp8", "mxint8"]        # the formats the OCP specification tabulates


def hadamard4():
    h2 = np.array([[1.0, 1.0], [1.0, -1.0]])
    return np.kron(h2, h2) / 2.0  # orthonormal Walsh-Hadamard


# ---------------------------------------------------------------- paper example
def test_paper_hadamard_example_transform():
    g = read_golden("hadamard_example.txt")
    x = np.array([float(t) for t in g["x"]])
    want = np.array([float(t) for t in g["H4x"]])
    got = orc.affine_transform(x[None, :], hadamard4(), None)[0]
    assert np.array_equal(got, want)
    # column form A x of the main text agrees because H4 is symmetric
    assert np.array_equal(hadamard4() @ x, want)


def test_paper_hadamard_example_block_errors():
    """With MXFP4 elements and B=2 the example behaves as the paper says:
    block 0 gets better after the rotation, block 1 gets worse.  The exact
    codes follow from Eq. q_mx by hand:
      [10,1]   -> floor(log2 10)=3, E=1: 10/2=5 ties to 4 (even), 1/2=.5 -> dq [8,1],  err^2 4
      [.5,.5]  -> floor(log2 .5)=-1, E=-3: 4,4                        -> dq exact,   err^2 0
      [6,4.5]  -> E=0: 6, 4.5 ties to 4                               -> dq [6,4],   err^2 .25
      [5,4.5]  -> E=0: 5 ties to 4, 4.5 ties to 4                     -> dq [4,4],   err^2 1.25
    """
    g = read_golden("hadamard_example.txt")
    B = int(g["block"][0])
    x = np.array([[float(t) for t in g["x"]]])
    y = np.array([[float(t) for t in g["H4x"]]])
    cx, sx = orc.mx_quantize(x, "mxfp4", block=B)
    cy, sy = orc.mx_quantize(y, "mxfp4", block=B)
    assert cx.tolist() == [[0x6, 0x1, 0x6, 0x6]] and sx.tolist() == [[128, 124]]
    assert cy.tolist() == [[0x7, 0x6, 0x6, 0x6]] and sy.tolist() == [[127, 127]]
    ex = ((x - orc.mx_dequantize(cx, sx, "mxfp4", B)) ** 2).reshape(2, 2).sum(1)
    ey = ((y - orc.mx_dequantize(cy, sy, "mxfp4", B)) ** 2).reshape(2, 2).sum(1)
    assert ex.tolist() == [4.0, 0.0] and ey.tolist() == [0.25, 1.25]
    assert ey[0] < ex[0] and ey[1] > ex[1]            # the paper's qualitative claim
    # transformation MSE goes through T^-1 = H4^T; orthonormal => same total squared error.  Block-wise error in the
    # ORIGINAL domain (Sec. 3.1, numerical analysis), by hand: y - Q(y) = [0, .5, 1, .5]; times H4 (= its own inverse,
    # rows .5 [1 1 1 1], .5 [1 -1 1 -1], .5 [1 1 -1 -1], .5 [1 -1 -1 1]) gives x - x^ = [1, 0, -.5, -.5]; squares
    # [1, 0, .25, .25]; means over blocks of two: [.5, .25]
    mse, per_block = orc.transformation_mse(x, hadamard4(), hadamard4().T, None, "mxfp4", block=B)
    assert math.isclose(mse, (0.25 + 1.25) / 4.0, rel_tol=1e-12)
    assert np.allclose(per_block, [0.5, 0.25], rtol=0, atol=1e-15)
    # without a transform the same quantities are the plain quantisation error of x: [4, 0] / 2 per block
    mse0, per_block0 = orc.transformation_mse(x, None, None, None, "mxfp4", block=B)
    assert math.isclose(mse0, 1.0, rel_tol=1e-12) and np.allclose(per_block0, [2.0, 0.0])


# ---------------------------------------------------------------- format facts
def test_format_tables_match_ocp_fixture():
    g = read_golden("ocp_element_formats.txt")
    for name in OCP_FMTS:
        r_max, vmax, vmin, count = g[name]
        f = orc.FORMATS[name]
        assert f.r_max == int(r_max)
        assert f.max == float(vmax)
        assert f.grid[1] == float(vmin)
        assert len(f.grid) == int(count)
        assert np.all(np.diff(f.grid) > 0)
        # top binade of the grid is [2^r_max, 2^(r_max+1))
        assert 2.0 ** f.r_max <= f.max < 2.0 ** (f.r_max + 1)
    assert orc.MXFP4.grid.tolist() == [float(t) for t in g["e2m1_grid"]]


def test_e2m1_tie_table():
    g = read_golden("ocp_element_formats.txt")
    for tok in g["e2m1_ties"]:
        v, want = (float(t) for t in tok.split(":"))
        for q in (orc.quantize_elements_arith, orc.quantize_elements_search):
            assert orc.decode_elements(q(np.array([v]), "mxfp4"), "mxfp4")[0] == want
            assert orc.decode_elements(q(np.array([-v]), "mxfp4"), "mxfp4")[0] == -want


# ---------------------------------------------------------------- Q_e: two implementations + exact brute force
@pytest.mark.parametrize("fmt", FMTS)
def test_element_quantizers_agree_dense_sweep(fmt):
    f = orc.FORMATS[fmt]
    rng = np.random.default_rng(1)
    top = 2.0 ** (f.r_max + 1)
    mids = (f.grid[1:] + f.grid[:-1]) / 2
    special = np.concatenate([f.grid, mids, np.nextafter(mids, 0), np.nextafter(mids, np.inf),
                              [top, np.nextafter(top, 0), 0.0, 1e-30, 5e-324]])
    v = np.concatenate([special, -special, rng.uniform(-top, top, 200000),
                        rng.standard_normal(100000) * f.grid[1] * 4])
    a = orc.quantize_elements_arith(v, fmt)
    s = orc.quantize_elements_search(v, fmt)
    assert np.array_equal(a, s)
    dq = orc.decode_elements(a, fmt)
    assert np.all(np.abs(dq) <= f.max)
    # nearest-ness: no grid point is strictly closer than the chosen one
    signed_grid = np.concatenate([-f.grid[::-1], f.grid])
    clipped = np.clip(v, -f.max, f.max)
    best = np.abs(clipped[:, None] - signed_grid[None, :]).min(1) if v.size * signed_grid.size < 2e8 else None
    if best is not None:
        assert np.all(np.abs(clipped - dq) <= best)


@pytest.mark.parametrize("fmt", FMTS)
def test_block_quantizer_matches_exact_rational_brute_force(fmt):
    rng = np.random.default_rng(2)
    f = orc.FORMATS[fmt]
    for trial in range(200):
        B = [2, 4, 32][trial % 3]
        scale = 2.0 ** rng.integers(-20, 20)
        blk = rng.standard_normal(B) * scale
        if trial % 5 == 0:   # plant exact ties and saturating values relative to the block max
            blk[0] = scale * 4
            blk[1:] = rng.choice(np.concatenate([(f.grid[1:] + f.grid[:-1]) / 2, [f.max * 1.1]]), B - 1) \
                * 2.0 ** (2 - f.r_max) * scale * rng.choice([-1, 1], B - 1)
        codes, sb = orc.mx_quantize(blk[None, :], fmt, block=B)
        ref_codes, ref_sb = orc.mx_quantize_block_exact(blk, fmt)
        assert codes[0].tolist() == ref_codes, (trial, blk)
        assert int(sb[0, 0]) == ref_sb


def test_fp4_all_code_pairs_roundtrip():
    """Every pair of 4-bit codes: dequantise, re-quantise, pack, unpack."""
    pairs = np.array(list(itertools.product(range(16), repeat=2)), dtype=np.uint8)
    vals = orc.decode_elements(pairs, "mxfp4")
    again = orc.quantize_elements_arith(vals, "mxfp4")
    assert np.array_equal(again, pairs)                 # includes -0 -> 0x8
    packed = orc.pack_fp4(pairs)
    assert np.array_equal(packed[:, 0], pairs[:, 0] | (pairs[:, 1] << 4))   # element 0 in the low nibble
    assert np.array_equal(orc.unpack_fp4(packed), pairs)


@pytest.mark.parametrize("fmt", ["mxfp8", "mxint8"])
def test_8bit_all_codes_roundtrip(fmt):
    codes = np.arange(256, dtype=np.uint8)
    if fmt == "mxfp8":
        codes = codes[(codes & 0x7F) != 0x7F]           # NaN encodings are never produced
    else:
        codes = codes[codes != 0x80]                    # -128 is outside the symmetric range
    vals = orc.decode_elements(codes, fmt)
    assert np.array_equal(orc.quantize_elements_arith(vals, fmt), codes)
    assert np.array_equal(orc.quantize_elements_search(vals, fmt), codes)


# ---------------------------------------------------------------- OCP / Eq. q_mx invariants
def _rand_rows(rng, rows=64, K=256, outliers=True):
    Y = rng.standard_normal((rows, K)) * np.exp(rng.uniform(-6, 6, (rows, 1)))
    if outliers:
        Y[:, rng.integers(0, K, 4)] *= 50
    return Y


@pytest.mark.parametrize("fmt", FMTS)
def test_mx_invariants(fmt):
    f = orc.FORMATS[fmt]
    rng = np.random.default_rng(3)
    Y = _rand_rows(rng)
    codes, sb = orc.mx_quantize(Y, fmt)
    dq = orc.mx_dequantize(codes, sb, fmt)
    E = sb.astype(np.int64) - 127
    s = np.ldexp(1.0, E)
    amax = np.abs(Y).reshape(64, -1, 32).max(2)
    # scale is a power of two with FLOOR: 2^E <= amax 2^-r_max < 2^(E+1)  (Appendix A, last step of the lemma)
    assert np.all(s <= amax * 2.0 ** -f.r_max) and np.all(amax * 2.0 ** -f.r_max < 2 * s)
    # every dequantised value is (grid value) * 2^E
    ratio = np.abs(dq).reshape(64, -1, 32) / s[:, :, None]
    assert np.all(np.isin(ratio, f.grid))
    # error bounds: half the largest gap when not saturated, (2^(r_max+1) - max) when saturated
    err = np.abs(Y - dq).reshape(64, -1, 32) / s[:, :, None]
    sat = np.abs(Y).reshape(64, -1, 32) / s[:, :, None] > f.max
    half_gap = np.diff(f.grid).max() / 2
    assert np.all(err[~sat] <= half_gap)
    assert np.all(err[sat] <= 2.0 ** (f.r_max + 1) - f.max)
    assert np.all(ratio[sat] == f.max)                  # saturation only at +-max*scale
    if fmt != "mxint8":
        assert np.any(sat)                              # the test really exercises saturation
    # sign is preserved
    nz = dq != 0
    assert np.all(np.sign(dq[nz]) == np.sign(Y[nz]))


@pytest.mark.parametrize("fmt", FMTS)
def test_mx_equivariances(fmt):
    rng = np.random.default_rng(4)
    Y = _rand_rows(rng, rows=16)
    codes, sb = orc.mx_quantize(Y, fmt)
    # power-of-two scaling: same codes, scale byte shifts
    for k in (-7, 3):
        c2, s2 = orc.mx_quantize(np.ldexp(Y, k), fmt)
        assert np.array_equal(c2, codes) and np.array_equal(s2.astype(int), sb.astype(int) + k)
    # negation flips signs only
    c3, s3 = orc.mx_quantize(-Y, fmt)
    assert np.array_equal(s3, sb)
    assert np.array_equal(orc.mx_dequantize(c3, s3, fmt), -orc.mx_dequantize(codes, sb, fmt))
    # permutation inside blocks permutes codes
    perm = rng.permutation(32)
    Yp = Y.reshape(16, -1, 32)[:, :, perm].reshape(16, -1)
    c4, s4 = orc.mx_quantize(Yp, fmt)
    assert np.array_equal(s4, sb)
    assert np.array_equal(c4, codes.reshape(16, -1, 32)[:, :, perm].reshape(16, -1))
    # idempotence
    dq = orc.mx_dequantize(codes, sb, fmt)
    c5, s5 = orc.mx_quantize(dq, fmt)
    assert np.array_equal(orc.mx_dequantize(c5, s5, fmt), dq)
    # blocks are contiguous index ranges: changing block i only changes block i
    Y2 = Y.copy()
    Y2[:, 32:64] *= 1000.0
    c6, s6 = orc.mx_quantize(Y2, fmt)
    keep = np.r_[0:32, 64:Y.shape[1]]
    assert np.array_equal(c6[:, keep], codes[:, keep])
    assert np.array_equal(np.delete(s6, 1, axis=1), np.delete(sb, 1, axis=1))


def test_zero_block_and_exponent_clamps():
    Y = np.zeros((1, 64))
    Y[0, 32] = -0.0
    Y[0, 40] = 2.0 ** -140            # below E8M0's smallest scale for fp4: E clamps to -127
    codes, sb = orc.mx_quantize(Y, "mxfp4")
    assert sb.tolist() == [[0, 0]]
    assert codes[0, :32].tolist() == [0] * 32
    assert codes[0, 32] == 0x8         # -0 keeps its sign bit
    assert codes[0, 40] == 0           # 2^-140 / 2^-127 = 2^-13 rounds to zero
    big = np.full((1, 32), 2.0 ** 200)
    codes, sb = orc.mx_quantize(big, "mxfp4")
    assert sb[0, 0] == 254 and np.all(codes == 0x7)    # upper clamp + saturation


def test_identity_transform_reduces_to_plain_mx():
    rng = np.random.default_rng(5)
    X = _rand_rows(rng, rows=8, K=64)
    c0, s0 = orc.mx_quantize(X, "mxfp4")
    c1, s1, Y = orc.transform_quantize(X, np.eye(64), np.zeros(64), "mxfp4")
    c2, s2, _ = orc.transform_quantize(X, None, None, "mxfp4")
    assert np.array_equal(Y, X)
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1)
    assert np.array_equal(c0, c2) and np.array_equal(s0, s2)


# ---------------------------------------------------------------- transform, fold, error structure
def _affine(rng, K):
    Q, R = np.linalg.qr(rng.standard_normal((K, K)))
    A = (Q * np.sign(np.diag(R))) * np.exp(rng.uniform(np.log(0.5), np.log(2.0), K))[None, :]
    return A, np.linalg.inv(A), rng.standard_normal(K) * 0.1


def test_affine_inverse_roundtrip():
    rng = np.random.default_rng(6)
    A, A_inv, b = _affine(rng, 48)
    X = rng.standard_normal((10, 48))
    assert np.allclose(orc.affine_inverse(orc.affine_transform(X, A, b), A_inv, b), X, atol=1e-12)


def test_affine_transform_is_row_form_not_transposed():
    """T(X) = X A + b: row i of the result is A^T x_i + b (column form of the main text)."""
    rng = np.random.default_rng(7)
    A = rng.standard_normal((5, 5))
    b = rng.standard_normal(5)
    X = rng.standard_normal((3, 5))
    Y = orc.affine_transform(X, A, b)
    for i in range(3):
        want = [sum(X[i, k] * A[k, j] for k in range(5)) + b[j] for j in range(5)]
        assert np.allclose(Y[i], want, atol=1e-13)


def test_fold_identity_fp64():
    """x W + bias == (x A + b)(A^-1 W) + (bias - b A^-1 W): Eq. fold_kqv_1 in row form."""
    rng = np.random.default_rng(8)
    K, N = 64, 96
    A, A_inv, b = _affine(rng, K)
    W = rng.standard_normal((K, N)) * 0.02
    bias = rng.standard_normal(N) * 0.01
    X = rng.standard_normal((7, K))
    _, _, c, Wf = orc.fold_weights(A_inv, b, W, bias, "mxfp4")
    lhs = X @ W + bias
    rhs = orc.affine_transform(X, A, b) @ Wf + (bias - b @ Wf)
    assert np.abs(lhs - rhs).max() < 1e-12
    assert np.allclose(c, bias - b @ Wf, rtol=1e-6, atol=1e-9)     # c is that vector in fp32
    # dropping the correction is detectably wrong
    assert np.abs(lhs - (orc.affine_transform(X, A, b) @ Wf + bias)).max() > 1e-3


def test_fold_weight_blocks_run_along_K():
    rng = np.random.default_rng(9)
    K, N = 64, 8
    W = rng.standard_normal((K, N))
    W[40, 3] = 1000.0                      # one huge input-channel entry in output column 3
    codes, sb, _, _ = orc.fold_weights(np.eye(K), None, W, None, "mxfp4")
    assert codes.shape == (N, K) and sb.shape == (N, K // 32)
    base_codes, base_sb = orc.mx_quantize(W.T.copy(), "mxfp4")
    assert np.array_equal(codes, base_codes) and np.array_equal(sb, base_sb)
    assert sb[3, 1] > sb[3, 0] + 5         # only column 3's second K-block sees the outlier
    assert abs(int(sb[2, 1]) - int(sb[2, 0])) <= 2


def test_error_identity_and_spectral_bound():
    """x - T^-1(Q(T(x))) = (T(x) - Q(T(x))) A^-1 exactly, hence
    E(T) <= ||A^-1||_sigma^2 / d * E||T(x) - Q(T(x))||^2  (Eq. matrix_projection)."""
    rng = np.random.default_rng(10)
    K = 64
    A, A_inv, b = _affine(rng, K)
    X = rng.standard_normal((32, K))
    X[:, 5] *= 50
    for fmt in FMTS:
        codes, sb, Y = orc.transform_quantize(X, A, b, fmt)
        Yq = orc.mx_dequantize(codes, sb, fmt)
        lhs = X - orc.affine_inverse(Yq, A_inv, b)
        assert np.allclose(lhs, (Y - Yq) @ A_inv, atol=1e-10)
        mse, _ = orc.transformation_mse(X, A, A_inv, b, fmt)
        bound = np.linalg.norm(A_inv, 2) ** 2 * np.mean((Y - Yq) ** 2)
        assert mse <= bound * (1 + 1e-12)
        assert mse > 0


def test_latmix_linear_approximates_plain_linear():
    """The quantised folded layer approximates x W + bias, and exactly equals the
    dequantised contraction it is defined as."""
    rng = np.random.default_rng(11)
    K, N, M = 128, 64, 16
    A, A_inv, b = _affine(rng, K)
    W = rng.standard_normal((K, N)) * 0.02
    bias = rng.standard_normal(N) * 0.01
    X = rng.standard_normal((M, K))
    for fmt, tol in (("mxfp4", 0.25), ("mxfp8", 0.06), ("mxint8", 0.02)):
        wc, ws, c, _ = orc.fold_weights(A_inv, b, W, bias, fmt)
        out = orc.latmix_linear(X, A, b, wc, ws, c, fmt)
        ref = X @ W + bias
        rel = np.linalg.norm(out - ref) / np.linalg.norm(ref)
        assert rel < tol, (fmt, rel)
        ac, asb, _ = orc.transform_quantize(X, A, b, fmt)
        manual = np.zeros((M, N))
        Ad, Wd = orc.mx_dequantize(ac, asb, fmt), orc.mx_dequantize(wc, ws, fmt)
        for i in range(M):
            for j in range(N):
                manual[i, j] = float(np.dot(Ad[i], Wd[j])) + float(c[j])
        assert np.allclose(out, manual, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- near-tie accounting
def test_check_codes_classification():
    rng = np.random.default_rng(12)
    Y = _rand_rows(rng, rows=8, K=64)
    codes, sb = orc.mx_quantize(Y, "mxfp4")
    r = orc.check_codes(Y, codes, sb, 0.0, "mxfp4")
    assert r["equal"] == r["total"] and r["illegal"] == 0
    bad = codes.copy()
    bad[0, 0] ^= 0x3                                    # a code two grid steps away
    r = orc.check_codes(Y, bad, sb, 1e-9 * np.abs(Y).max(), "mxfp4")
    assert r["illegal"] == 1
    # a value sitting on a rounding boundary may legally land on either side
    Yt = np.zeros((1, 32)); Yt[0, 0] = 4.0; Yt[0, 1] = 2.5      # E=0; 2.5 ties -> 2 (code 4)
    ct, st = orc.mx_quantize(Yt, "mxfp4")
    alt = ct.copy(); alt[0, 1] = 0x5                             # 3.0
    assert orc.check_codes(Yt, alt, st, 0.0, "mxfp4")["illegal"] == 1
    r = orc.check_codes(Yt, alt, st, 1e-6, "mxfp4")
    assert r["alternate"] == 1 and r["illegal"] == 0
    # block maximum on a power of two: exponent may legally differ by one
    Yp = np.zeros((1, 32)); Yp[0, 0] = 8.0 - 1e-9; Yp[0, 1] = 1.0
    cp, sp = orc.mx_quantize(Yp, "mxfp4")                       # E = 0
    up_c, up_s = orc.mx_quantize(np.where(Yp > 7, 8.0, Yp), "mxfp4")   # E = 1
    assert int(up_s[0, 0]) == int(sp[0, 0]) + 1
    assert orc.check_codes(Yp, up_c, up_s, 0.0, "mxfp4")["illegal"] > 0
    assert orc.check_codes(Yp, up_c, up_s, 1e-6, "mxfp4")["illegal"] == 0


# ------------------------------------------------------------------ block-wise online transform (T_3)
def test_hadamard_block_matches_the_papers_example_and_is_an_involution():
    g = read_golden("hadamard_example.txt")
    x = np.array([float(t) for t in g["x"]])
    want = np.array([float(t) for t in g["H4x"]])
    H4 = orc.hadamard_block(4)
    # one block of size four is the whole worked example of Sec. 3.1
    got = orc.block_diag_transform(x[None, :], H4[None, :, :], None, block=4)[0]
    assert np.allclose(got, want, atol=1e-12)
    H32 = orc.hadamard_block(32)
    assert np.allclose(H32 @ H32, np.eye(32), atol=1e-12)           # symmetric and orthonormal: its own inverse
    assert np.allclose(np.abs(H32), 1 / np.sqrt(32))


def test_block_diag_transform_acts_block_by_block():
    rng = np.random.default_rng(5)
    M, K = 7, 96
    X = rng.normal(size=(M, K))
    blocks = rng.normal(size=(K // 32, 32, 32))
    b = rng.normal(size=K)
    Y = orc.block_diag_transform(X, blocks, b)
    # same thing through a dense block-diagonal matrix built entry by entry
    A = np.zeros((K, K))
    for i in range(K // 32):
        for r in range(32):
            for c in range(32):
                A[32 * i + r, 32 * i + c] = blocks[i, r, c]
    assert np.allclose(Y, X @ A + b, atol=1e-12)
    # a change in block 1 of the input moves block 1 of the output only
    X2 = X.copy(); X2[:, 40] += 3.0
    D = orc.block_diag_transform(X2, blocks, b) - Y
    assert np.all(D[:, :32] == 0) and np.all(D[:, 64:] == 0) and np.any(D[:, 32:64] != 0)
    # row form, not transposed: element j of the output takes column j of the block
    e = np.zeros((1, K)); e[0, 33] = 1.0
    assert np.allclose(orc.block_diag_transform(e, blocks)[0, 32:64], blocks[1, 1, :])
    # orthonormal blocks keep the energy of every MX block (Parseval), and applying Hadamard blocks twice gives x back
    H = np.stack([orc.hadamard_block(32)] * (K // 32))
    Z = orc.block_diag_transform(X, H)
    for i in range(K // 32):
        assert np.allclose(np.sum(Z[:, 32 * i:32 * i + 32] ** 2, axis=1), np.sum(X[:, 32 * i:32 * i + 32] ** 2, axis=1))
    assert np.allclose(orc.block_diag_transform(Z, H), X, atol=1e-12)


# ---------------------------------------------------------------- two-sided fold (App. "Folding ...", T_1 and T_2)
def _well_conditioned(rng, n):
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    return q * np.exp(rng.uniform(np.log(0.5), np.log(2.0), n))[None, :]


def test_two_sided_fold_equals_the_unfolded_maps():
    """f~~(x') = T_out(f(T_in^-1(x'))) for every combination of sides, evaluated with the transform functions
    rather than with the fold's own algebra."""
    rng = np.random.default_rng(21)
    T, K, N = 9, 64, 96
    X = rng.standard_normal((T, K))
    W, bias = rng.standard_normal((K, N)) * 0.1, rng.standard_normal(N)
    A_in, b_in = _well_conditioned(rng, K), rng.standard_normal(K)
    A_out, v_out = _well_conditioned(rng, N), rng.standard_normal(N)
    A_in_inv = np.linalg.inv(A_in)
    for use_in in (False, True):
        for use_out in (False, True):
            for shifts in (False, True):
                bi = b_in if (use_in and shifts) else None
                vo = v_out if (use_out and shifts) else None
                _, _, c, Wf = orc.fold_weights_two_sided(A_in_inv if use_in else None, bi, W, bias,
                                                         A_out if use_out else None, vo, "mxfp4")
                Xp = orc.affine_transform(X, A_in, bi) if use_in else X          # what the folded layer is fed
                x_back = orc.affine_inverse(Xp, A_in_inv, bi) if use_in else Xp
                y = x_back @ W + bias
                want = orc.affine_transform(y, A_out, vo) if use_out else y
                got = Xp @ Wf + c.astype(np.float64)
                assert np.abs(got - want).max() <= 2e-6 * np.abs(want).max(), (use_in, use_out, shifts)


def test_two_sided_fold_reduces_to_the_one_sided_fold_and_to_plain_quantisation():
    rng = np.random.default_rng(22)
    K, N = 64, 32
    W, bias = rng.standard_normal((K, N)), rng.standard_normal(N)
    A_inv, b = np.linalg.inv(_well_conditioned(rng, K)), rng.standard_normal(K)
    one = orc.fold_weights(A_inv, b, W, bias, "mxfp8")
    two = orc.fold_weights_two_sided(A_inv, b, W, bias, None, None, "mxfp8")
    for u, v in zip(one, two):
        assert np.array_equal(u, v)
    codes, scales, c, Wf = orc.fold_weights_two_sided(None, None, W, None, np.eye(N), None, "mxfp8")
    want_codes, want_scales = orc.mx_quantize(np.ascontiguousarray(W.T), "mxfp8")
    assert np.array_equal(codes, want_codes) and np.array_equal(scales, want_scales)
    assert np.array_equal(Wf, W) and not c.any()


def test_value_and_output_projection_folds_cancel_through_attention_mixing():
    """V projection carries (T_1^-1 | T_2), the MHA output projection (T_2^-1 | A_1).  Attention mixes value rows
    with weights that sum to one, so T_2's shift survives the mixing and T_2^-1 removes it: the folded chain must
    equal the plain chain times A_1.  With the output-projection bias taken as -(b_O A_1 + v_2 A_2^-1 W_O A_1), the
    grouping the printed equation suggests, the same chain is off by 2 b_O A_1."""
    rng = np.random.default_rng(23)
    T, d, dv = 7, 64, 32
    X = rng.standard_normal((T, d))
    W_V, b_V = rng.standard_normal((d, dv)) * 0.2, rng.standard_normal(dv)
    W_O, b_O = rng.standard_normal((dv, d)) * 0.2, rng.standard_normal(d)
    A1, v1 = _well_conditioned(rng, d), rng.standard_normal(d)
    A2, v2 = _well_conditioned(rng, dv), rng.standard_normal(dv)
    P = rng.uniform(size=(T, T)); P /= P.sum(axis=1, keepdims=True)
    plain = (P @ (X @ W_V + b_V)) @ W_O + b_O
    _, _, cV, GV = orc.fold_weights_two_sided(np.linalg.inv(A1), v1, W_V, b_V, A2, v2, "mxfp4")
    _, _, cO, GO = orc.fold_weights_two_sided(np.linalg.inv(A2), v2, W_O, b_O, A1, None, "mxfp4")
    Xp = orc.affine_transform(X, A1, v1)
    folded = (P @ (Xp @ GV + cV.astype(np.float64))) @ GO + cO.astype(np.float64)
    want = plain @ A1
    assert np.abs(folded - want).max() <= 5e-6 * np.abs(want).max()
    wrong_c = -(b_O @ A1 + v2 @ np.linalg.inv(A2) @ W_O @ A1)
    wrong = (P @ (Xp @ GV + cV.astype(np.float64))) @ GO + wrong_c
    assert np.abs(wrong - want).max() > 0.1 * np.abs(want).max()


def test_two_sided_fold_quantises_the_folded_weight_along_K():
    rng = np.random.default_rng(24)
    K, N = 64, 32
    W = rng.standard_normal((K, N))
    A_in_inv, A_out = np.linalg.inv(_well_conditioned(rng, K)), _well_conditioned(rng, N)
    codes, scales, _, Wf = orc.fold_weights_two_sided(A_in_inv, None, W, None, A_out, None, "mxfp4")
    assert codes.shape == (N, K) and scales.shape == (N, K // 32)
    assert np.allclose(Wf, A_in_inv @ W @ A_out, rtol=0, atol=1e-12)
    col = 5
    want_codes, want_scale = orc.mx_quantize_block_exact(Wf[32:64, col], "mxfp4")
    assert list(codes[col, 32:64]) == want_codes and int(scales[col, 1]) == want_scale


# ---------------------------------------------------------------- MXINT4 (this repository's reading: parity unpinned)
def test_mxint4_reading_by_hand():
    """k in [-7, 7], value k, r_max = 2.  [10, 1, -3.5, 0.4]: floor(log2 10) = 3, E = 1: 5, .5 (tie -> 0, even),
    -1.75 -> -2, .2 -> 0.  [7.9, -7.6]: E = 0: both round to magnitude 8, which the symmetric range clamps to 7."""
    codes, scales = orc.mx_quantize(np.array([[10.0, 1.0, -3.5, 0.4]]), "mxint4", block=4)
    assert codes.tolist() == [[5, 0, 0xE, 0]] and scales.tolist() == [[128]]
    assert orc.mx_dequantize(codes, scales, "mxint4", 4).tolist() == [[10.0, 0.0, -4.0, 0.0]]
    codes, scales = orc.mx_quantize(np.array([[7.9, -7.6]]), "mxint4", block=2)
    assert codes.tolist() == [[7, 9]] and scales.tolist() == [[127]]


# ---------------------------------------------------------------- other block sizes (the block-size sweep of Sec. 3.1)
@pytest.mark.parametrize("block", [8, 16, 64, 128])
@pytest.mark.parametrize("fmt", OCP_FMTS)
def test_other_block_sizes_brute_force_and_invariants(fmt, block):
    """Eq. q_mx with a block size other than 32, as the sweep over block sizes uses it: whole blocks against the
    exact-rational brute force, the floor rule of the scale, values on grid x 2^E; and the transformation MSE with a
    block as long as the row equals a plain per-row quantisation error."""
    f = orc.FORMATS[fmt]
    rng = np.random.default_rng(40 + block)
    Y = rng.standard_normal((6, 2 * block)) * np.exp(rng.standard_normal((6, 1)) * 3)
    Y[:, 3] *= 40
    codes, sb = orc.mx_quantize(Y, fmt, block=block)
    for r in range(6):
        for i in range(2):
            want_codes, want_sb = orc.mx_quantize_block_exact(Y[r, i * block:(i + 1) * block], fmt)
            assert codes[r, i * block:(i + 1) * block].tolist() == want_codes and int(sb[r, i]) == want_sb
    dq = orc.mx_dequantize(codes, sb, fmt, block=block)
    s = np.ldexp(1.0, sb.astype(np.int64) - 127)
    amax = np.abs(Y).reshape(6, 2, block).max(2)
    assert np.all(s <= amax * 2.0 ** -f.r_max) and np.all(amax * 2.0 ** -f.r_max < 2 * s)
    assert np.all(np.isin(np.abs(dq).reshape(6, 2, block) / s[:, :, None], f.grid))
    # identity transform: E(T) is the mean squared quantisation error, block by block
    mse, per_block = orc.transformation_mse(Y, None, None, None, fmt, block=block)
    want = ((Y - dq) ** 2).reshape(6, 2, block).mean(axis=(0, 2))
    assert np.allclose(per_block, want, rtol=1e-13) and math.isclose(mse, want.mean(), rel_tol=1e-13)
    # a coarser block never has a smaller scale than the finer blocks it contains
    if block >= 16:
        _, sb_fine = orc.mx_quantize(Y, fmt, block=block // 2)
        assert np.all(sb == sb_fine.reshape(6, 2, 2).max(2))
