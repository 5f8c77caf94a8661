"""Parity of the CUDA path with the CPU oracle, through the C ABI, on seeded inputs that span several tiles
and ragged tails.  Integer work (codes, scale bytes) must match bit for bit; fp32 GEMM outputs must match
the oracle's fp64 result within 1e-4 relative Frobenius on identical codes (only accumulation rounds) and
within 1e-3 on the whole fp64 chain."""
import numpy as np
import pytest
import torch

from oracle import latmix_oracle as orc
from paper_2602_17681_b200 import synth
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

GEMM_TOL_SAME_CODES = 1e-4      # products are exact; only fp32 accumulation order differs
CHAIN_TOL = 1e-3                # tolerance stated for the layer output against the fp64 chain


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _acts(M, K, dtype, seed=1):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g, dtype=torch.float64) * torch.exp(torch.randn(M, 1, generator=g, dtype=torch.float64) * 3)
    X[:, 5] *= 50
    if M > 3:
        X[3, 64:96] = 0                      # an all-zero block
        X[2, 32:64] = 2.0 ** -135            # below the smallest scale: clamps to byte 0
        X[1, 0] = -0.0
    return X.to(dtype)


# ------------------------------------------------------------------ S2: plain quantiser, bit exact
@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("sf", [0, 1])
def test_plain_quantizer_bit_exact(B, fmt, dtype, sf):
    M, K = 301, 1088 if fmt else 1088 + 64        # ragged rows, K not a multiple of 256
    X = _acts(M, K, dtype).cuda()
    codes, scales, _ = B.quantize_mx(X, None, None, fmt, sf)
    rc, rs = orc.mx_quantize(X.double().cpu().numpy(), H.FMT_NAME[fmt])
    assert np.array_equal(H.codes_to_numpy(codes, M, K, fmt), rc)
    assert np.array_equal(H.scales_to_linear(B, scales, M, K, sf), rs)
    if sf == B.SF_TCGEN05:                         # K/32 is not a multiple of 8 here: the buffer is zeroed first, so every padding byte is zero
        used = np.zeros(scales.numel(), dtype=bool)
        used[H.sf_offsets(M, K)] = True
        assert not scales.cpu().numpy()[~used].any()


def test_stale_scale_padding_rows_do_not_reach_the_output(B):
    """M is not a multiple of 128 and K/32 is a multiple of 8: the quantiser then leaves the scale bytes of the padding
    rows as it finds them.  A workspace full of 0xFF bytes (a NaN scale) must give the bits a zeroed one gives."""
    cfg = synth.LayerConfig("stale", 200, 1024, 320, seed=77)
    L = {k: v.cuda() for k, v in synth.make_layer(cfg).items()}
    for fmt in (0, 1):
        wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], fmt)
        outs = []
        for fill in (0x00, 0xFF):
            ws = torch.full((B.workspace_bytes(B.OP_LINEAR, cfg.M, cfg.K, cfg.N, fmt),), fill, dtype=torch.uint8, device="cuda")
            B.workspace_init(ws)
            n0 = B.launch_count()
            outs.append(B.linear(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, fmt, ws=ws))
            assert B.launch_count() - n0 == 2 and B.device_status(ws) == B.OK
        assert torch.isfinite(outs[1]).all() and torch.equal(outs[0], outs[1])


def test_tensor_pipe_probe_runs(B):
    ws = B.new_workspace(B.OP_QUANTIZE_MX, 0, 64, 0, 0)
    for k in ("bf16", "mxf8", "mxf4", "nvf4"):            # first launches carry module loading
        B.tensor_pipe_probe(k, ws, mma_per_cta=64)
    rates = {k: max(B.tensor_pipe_probe(k, ws) for _ in range(3)) for k in ("bf16", "mxf8", "mxf4", "nvf4")}
    assert B.device_status(ws) == B.OK
    # the pipes' nominal ratios 1 : 2 : 4 : 4, loosely (clocks move between launches)
    assert 1.5 < rates["mxf8"] / rates["bf16"] < 2.5 and 3.0 < rates["mxf4"] / rates["bf16"] < 5.0, rates
    assert 0.8 < rates["nvf4"] / rates["mxf4"] < 1.25, rates
    assert 1000 < rates["bf16"] < 2600, rates              # TFLOP/s: between half and a little above the nominal 2250


def test_quantizer_edge_cases(B):
    ws = B.new_workspace(B.OP_QUANTIZE_MX, 0, 64, 0, 0)
    # empty input: accepted, nothing launched
    n0 = B.launch_count()
    empty = torch.empty(0, 64, dtype=torch.bfloat16, device="cuda")
    B.quantize_mx(empty, None, None, 0, ws=ws)
    assert B.launch_count() == n0
    # extremes of fp32: largest finite and smallest subnormal values
    X = torch.zeros(4, 64, dtype=torch.float32)
    X[0, :32] = torch.finfo(torch.float32).max
    X[0, 32:] = -torch.finfo(torch.float32).max
    X[1, 0] = 1e-45
    X[2, :] = torch.linspace(-8, 8, 64)
    X[3, 0::2] = 6.0; X[3, 1::2] = -5.0           # saturation boundary and a tie
    for fmt in (0, 1, 2):
        codes, scales, _ = B.quantize_mx(X.cuda(), None, None, fmt, B.SF_LINEAR, ws=ws)
        rc, rs = orc.mx_quantize(X.double().numpy(), H.FMT_NAME[fmt])
        assert np.array_equal(H.codes_to_numpy(codes, 4, 64, fmt), rc)
        assert np.array_equal(H.scales_to_linear(B, scales, 4, 64, B.SF_LINEAR), rs)
    assert B.device_status(ws) == B.OK


def test_quantizer_with_bias_matches_oracle_on_its_own_sum(B):
    M, K = 64, 512
    X = _acts(M, K, torch.bfloat16).cuda()
    b = (torch.randn(K) * 0.1).cuda()
    codes, scales, Y = B.quantize_mx(X, None, b, 0, dump=True)
    assert torch.equal(Y, X.float() + b[None, :])
    rc, rs = orc.mx_quantize(Y.double().cpu().numpy(), "mxfp4")
    assert np.array_equal(H.codes_to_numpy(codes, M, K, 0), rc)
    assert np.array_equal(H.scales_to_linear(B, scales, M, K, 1), rs)


def test_nonfinite_input_is_reported_not_faulted(B):
    X = torch.randn(8, 128, dtype=torch.float32)
    X[3, 7] = float("nan")
    ws = B.new_workspace(B.OP_QUANTIZE_MX, 8, 128, 0, 0)
    B.quantize_mx(X.cuda(), None, None, 0, ws=ws, flags=B.FLAG_CHECK_FINITE)
    assert B.device_status(ws) == B.ERR_NONFINITE
    ws2 = B.new_workspace(B.OP_QUANTIZE_MX, 8, 128, 0, 0)
    B.quantize_mx(torch.randn(8, 128).cuda(), None, None, 0, ws=ws2, flags=B.FLAG_CHECK_FINITE)
    assert B.device_status(ws2) == B.OK


# ------------------------------------------------------------------ S1+S2: transform + quantise
def _check_transform(B, X, A, b, fmt, sf, flags, y_tol, unit):
    M, K = X.shape
    name = H.FMT_NAME[fmt]
    ws = B.new_workspace(B.OP_QUANTIZE_MX, M, K, 0, fmt)
    codes, scales, Y = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), fmt, sf, dump=True, ws=ws, flags=flags)
    codes2, scales2, _ = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), fmt, sf, dump=False, ws=ws, flags=flags)
    assert B.device_status(ws) == B.OK
    gc, gs = H.codes_to_numpy(codes, M, K, fmt), H.scales_to_linear(B, scales, M, K, sf)
    # the production variant (no dump) produces the same bits as the dumping variant
    assert np.array_equal(H.codes_to_numpy(codes2, M, K, fmt), gc)
    assert np.array_equal(H.scales_to_linear(B, scales2, M, K, sf), gs)
    # bit-exact against the oracle's quantiser applied to the kernel's own pre-quantisation values
    Yg = Y.double().cpu().numpy()
    rc, rs = orc.mx_quantize(Yg, name)
    assert np.array_equal(gc, rc) and np.array_equal(gs, rs)
    # the pre-quantisation values against the fp64 transform
    X64, A64, b64 = X.double().numpy(), A.double().numpy(), b.double().numpy()
    Y64 = orc.affine_transform(X64, A64, b64)
    assert H.rel_fro(Yg, Y64) < y_tol
    tau = H.accumulation_tau(X64, A64, unit)
    assert np.all(np.abs(Yg - Y64) <= tau)
    # accounting against the all-fp64 chain: differences only where a value sits on a rounding boundary
    acc = orc.check_codes(Y64, gc, gs, tau, name)
    assert acc["illegal"] == 0, acc
    assert acc["alternate"] <= 2e-3 * acc["total"], acc
    return acc


@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("sf", [0, 1])
@pytest.mark.parametrize("variant", [0, 1])       # 0: CTA pairs (all tiles cut into half-width tiles here), 1: single-CTA kernel
def test_transform_quantize_tensor_core(B, fmt, sf, variant):
    M, K = 300, 1088 if fmt else 1088 + 64        # 3 row tiles (ragged), 5 column tiles (ragged), 18 k-slabs
    X = synth.make_activations(M, K, 5, dtype="bf16")
    A, b, _ = synth.make_transform(K, 5, "bf16")
    _check_transform(B, X, A, b, fmt, sf, variant << 8, 1e-5, H.tensor_core_unit(K))


@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("M,K", [(1, 4096), (5, 1088 + 64), (16, 2048), (16, 64), (3, 5120 + 64), (17, 2048), (40, 4096), (64, 1088 + 64)])
def test_transform_quantize_small_batch_kernel(B, fmt, M, K):
    """M <= 64 takes the kernel with the columns of A on the 128-row side of the MMA (16 or 64 rows of X on its N side) and a
    cluster of four CTAs per tile, each
    with a quarter of the summation index: slices that end or start past K, idle CTAs (K = 64), tiles that reach past K,
    an odd number of slabs, a K beyond one wave's worth of tiles, both scale layouts."""
    X = synth.make_activations(M, K, 71, dtype="bf16")
    A, b, _ = synth.make_transform(K, 71, "bf16")
    for sf in (0, 1):
        n0 = B.launch_count()
        _check_transform(B, X, A, b, fmt, sf, 0, 1e-5, H.tensor_core_unit(K))
        assert B.launch_count() - n0 == 2
    # the tiled tensor-core kernel quantises its own values just as exactly; the two may differ on near-ties only
    c0, s0, y0 = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), fmt, dump=True)
    c8, s8, y8 = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), fmt, dump=True, flags=8 << 8)
    assert H.rel_fro(y0.double().cpu().numpy(), y8.double().cpu().numpy()) < 1e-5
    assert np.mean(H.codes_to_numpy(c0, M, K, fmt) != H.codes_to_numpy(c8, M, K, fmt)) < 5e-3


def test_transform_quantize_pairs_whole_and_half_tiles(B):
    """81 tiles of 256 x 256 on at most 74 resident CTA pairs: whole tiles first, the remainder as half-width tiles."""
    M = K = 2304
    X = synth.make_activations(M, K, 15, dtype="bf16")
    A, b, _ = synth.make_transform(K, 15, "bf16")
    _check_transform(B, X, A, b, 0, 1, 0, 1e-5, H.tensor_core_unit(K))


def test_transform_quantize_fp32_inputs_cfg0(B):
    cfg = synth.CONFIGS["cfg0"]
    L = synth.make_layer(cfg)
    assert L["X"].dtype == torch.float32
    _check_transform(B, L["X"], L["A"], L["b"], 0, 1, 0, 1e-5, H.fma_unit(cfg.K))


def test_transform_quantize_cuda_core_path_bf16(B):
    X = synth.make_activations(100, 320, 6, dtype="bf16")
    A, b, _ = synth.make_transform(320, 6, "bf16")
    _check_transform(B, X, A, b, 0, 1, B.FLAG_FORCE_SIMT, 1e-5, H.fma_unit(320))


def test_identity_transform_reduces_to_plain_quantizer(B):
    M, K = 128, 256
    X = synth.make_activations(M, K, 8, dtype="bf16")      # no signed zeros: (-0) * 1 + 0 + ... is +0 in any arithmetic
    eye = torch.eye(K, dtype=torch.bfloat16)
    zero = torch.zeros(K)
    c0, s0, _ = B.quantize_mx(X.cuda(), None, None, 0)
    c1, s1, _ = B.quantize_mx(X.cuda(), eye.cuda(), zero.cuda(), 0)
    assert torch.equal(c0, c1) and torch.equal(s0, s1)


# ------------------------------------------------------------------ block-wise online transform (T_3) + quantise
@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype,kind", [("bf16", "haar"), ("f32", "haar"), ("bf16", "hadamard")])
@pytest.mark.parametrize("sf", [0, 1])
def test_block_diag_transform_quantize(B, fmt, dtype, kind, sf):
    M, K = 333, 448 if fmt else 448 + 64        # ragged row tail, 14 or 16 blocks
    name = H.FMT_NAME[fmt]
    X = synth.make_activations(M, K, 31, dtype=dtype)
    blocks, b, _ = synth.make_block_transform(K, 31, kind, a_dtype=dtype, b_std=0.0 if kind == "hadamard" else 0.1)
    ws = B.new_workspace(B.OP_QUANTIZE_MX, M, K, 0, fmt)
    dev_b = None if b is None else b.cuda()
    codes, scales, Y = B.quantize_mx(X.cuda(), blocks.cuda(), dev_b, fmt, sf, dump=True, ws=ws, flags=B.FLAG_BLOCK_DIAG)
    codes2, scales2, _ = B.quantize_mx(X.cuda(), blocks.cuda(), dev_b, fmt, sf, ws=ws, flags=B.FLAG_BLOCK_DIAG)
    assert B.device_status(ws) == B.OK
    gc, gs = H.codes_to_numpy(codes, M, K, fmt), H.scales_to_linear(B, scales, M, K, sf)
    assert np.array_equal(H.codes_to_numpy(codes2, M, K, fmt), gc) and np.array_equal(H.scales_to_linear(B, scales2, M, K, sf), gs)
    Yg = Y.double().cpu().numpy()
    rc, rs = orc.mx_quantize(Yg, name)
    assert np.array_equal(gc, rc) and np.array_equal(gs, rs)            # bit-exact on its own transformed values
    X64, A64 = X.double().numpy(), blocks.double().numpy()
    b64 = None if b is None else b.double().numpy()
    Y64 = orc.block_diag_transform(X64, A64, b64)
    # 32-term fp32 FMA chain per output (+ one add for the bias)
    absprod = np.concatenate([np.abs(X64[:, 32 * i:32 * i + 32]) @ np.abs(A64[i]) for i in range(K // 32)], axis=1)
    tau = H.fma_unit(32) * (absprod + (0 if b64 is None else np.abs(b64)[None, :])) + 1e-30
    assert np.all(np.abs(Yg - Y64) <= tau)
    acc = orc.check_codes(Y64, gc, gs, tau, name)
    assert acc["illegal"] == 0, acc


def test_block_diag_cuda_core_and_tensor_core_paths_agree_on_codes(B):
    """bf16 inputs take the mma.sync kernel, LATMIX_FLAG_FORCE_SIMT the FMA kernel: both must quantise their own values
    exactly, and may differ from each other only on near-ties."""
    M, K = 200, 512
    X = synth.make_activations(M, K, 33, dtype="bf16")
    blocks, b, _ = synth.make_block_transform(K, 33, "haar", b_std=0.1)
    outs = []
    for flags in (B.FLAG_BLOCK_DIAG, B.FLAG_BLOCK_DIAG | B.FLAG_FORCE_SIMT):
        codes, scales, Y = B.quantize_mx(X.cuda(), blocks.cuda(), b.cuda(), B.MXFP4, dump=True, flags=flags)
        gc, gs = H.codes_to_numpy(codes, M, K, 0), H.scales_to_linear(B, scales, M, K, 1)
        rc, rs = orc.mx_quantize(Y.double().cpu().numpy(), "mxfp4")
        assert np.array_equal(gc, rc) and np.array_equal(gs, rs)
        outs.append((gc, Y.double().cpu().numpy()))
    assert H.rel_fro(outs[0][1], outs[1][1]) < 1e-6
    assert np.mean(outs[0][0] != outs[1][0]) < 2e-3


def test_block_diag_layer_against_fp64_chain(B):
    """latmix_linear with the block-wise transform: fold with the dense inverse, run, compare with the oracle chain."""
    M, K, N = 320, 512, 448
    X = synth.make_activations(M, K, 41, dtype="bf16")
    blocks, b, A_inv = synth.make_block_transform(K, 41, "haar", b_std=0.1)
    W, bias = synth.make_weights(K, N, 41)
    wq, wsc, c, _ = B.fold_weights(A_inv.cuda(), b.cuda(), W.cuda(), bias.cuda(), B.MXFP4)
    ws = B.new_workspace(B.OP_LINEAR, M, K, N, B.MXFP4)
    out = B.linear(X.cuda(), blocks.cuda(), b.cuda(), wq, wsc, c, N, B.MXFP4, ws=ws, flags=B.FLAG_BLOCK_DIAG)
    codes, scales, _ = B.quantize_mx(X.cuda(), blocks.cuda(), b.cuda(), B.MXFP4, ws=ws, flags=B.FLAG_BLOCK_DIAG)
    assert B.device_status(ws) == B.OK
    a_codes, a_scales = H.codes_to_numpy(codes, M, K, 0), H.scales_to_linear(B, scales, M, K, 1)
    w_codes, w_scales = H.codes_to_numpy(wq, N, K, 0), H.scales_to_linear(B, wsc, N, K, 1)
    ref_own = orc.mx_matmul(a_codes, a_scales, w_codes, w_scales, c.cpu().numpy(), "mxfp4")
    H.assert_gemm_parity(out.cpu().numpy(), ref_own, a_codes, a_scales, w_codes, w_scales, "mxfp4", K, c.cpu().numpy(), tag="block-diag layer")
    # the whole chain in fp64: block transform, quantise, folded weights
    wc64, ws64, c64, _ = orc.fold_weights(A_inv.double().numpy(), b.double().numpy(), W.double().numpy(), bias.double().numpy(), "mxfp4")
    qc, qs = orc.mx_quantize(orc.block_diag_transform(X.double().numpy(), blocks.double().numpy(), b.double().numpy()), "mxfp4")
    ref = orc.mx_matmul(qc, qs, wc64, ws64, c64, "mxfp4")
    assert H.rel_fro(out.cpu().numpy(), ref) < 1e-2                     # tie flips only (see the layer test below)
    # and the layer still approximates the plain linear layer it replaces
    plain = X.double().numpy() @ W.double().numpy() + bias.double().numpy()
    # (W4A4 on outlier-heavy inputs is lossy by itself: the distance to the plain layer is the oracle chain's, not small)
    assert abs(H.rel_fro(out.cpu().numpy(), plain) - H.rel_fro(ref, plain)) < 5e-3


# ------------------------------------------------------------------ S0: fold + weight quantisation
@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("w_dtype", ["bf16", "f32"])
def test_fold_weights(B, fmt, w_dtype):
    K, N = 320 if fmt else 320 + 64, 200
    name = H.FMT_NAME[fmt]
    A, b, A_inv = synth.make_transform(K, 7, "bf16")
    W, bias = synth.make_weights(K, N, 7, dtype=w_dtype)
    wc, wsc, c, dump = B.fold_weights(A_inv.cuda(), b.cuda(), W.cuda(), bias.cuda(), fmt, dump=True)
    rcodes, rscales, rc, Wf = orc.fold_weights(A_inv.double().numpy(), b.double().numpy(), W.double().numpy(),
                                               bias.double().numpy(), name)
    D = dump.double().cpu().numpy()
    gc, gs = H.codes_to_numpy(wc, N, K, fmt), H.scales_to_linear(B, wsc, N, K, 1)
    qc, qs = orc.mx_quantize(D, name)
    assert np.array_equal(gc, qc) and np.array_equal(gs, qs)            # bit-exact on its own folded values
    # fp32-accurate fold.  fp32 weights take the FMA kernel (round-to-nearest chain, ~1e-7); bf16 weights take the tensor
    # cores with A_inv as three bf16 terms: products exact, 3K/16 accumulator updates that may truncate (~1e-6)
    assert H.rel_fro(D, Wf.T) < (5e-6 if w_dtype == "bf16" else 1e-6)
    tau = H.accumulation_tau(W.double().numpy().T, A_inv.double().numpy().T, H.fma_unit(K))
    acc = orc.check_codes(Wf.T, gc, gs, tau, name)
    assert acc["illegal"] == 0, acc
    assert np.allclose(c.cpu().numpy(), rc, rtol=2e-7, atol=1e-9)       # fp64 accumulation, rounded once
    # no transform bias / no layer bias -> c == 0
    _, _, c0, _ = B.fold_weights(A_inv.cuda(), None, W.cuda(), None, fmt)
    assert not c0.cpu().numpy().any()
    if w_dtype == "f32" and K % 64 == 0:
        # with 6 K N more bytes of workspace fp32 weights take the tensor cores too (both operands as three bf16 terms)
        big = torch.zeros(B.workspace_bytes(B.OP_FOLD_WEIGHTS, 0, K, N, fmt) + 6 * K * N, dtype=torch.uint8, device="cuda")
        n0 = B.launch_count()
        wc2, wsc2, c2, dump2 = B.fold_weights(A_inv.cuda(), b.cuda(), W.cuda(), bias.cuda(), fmt, dump=True, ws=big)
        assert B.launch_count() - n0 == 5 and B.device_status(big) == B.OK       # two splits, product, two bias kernels
        D2 = dump2.double().cpu().numpy()
        gc2, gs2 = H.codes_to_numpy(wc2, N, K, fmt), H.scales_to_linear(B, wsc2, N, K, 1)
        qc2, qs2 = orc.mx_quantize(D2, name)
        assert np.array_equal(gc2, qc2) and np.array_equal(gs2, qs2)
        assert H.rel_fro(D2, Wf.T) < 5e-6
        tau2 = H.accumulation_tau(W.double().numpy().T, A_inv.double().numpy().T, H.tensor_core_unit(9 * K) + 2.0 ** -22)
        assert orc.check_codes(Wf.T, gc2, gs2, tau2, name)["illegal"] == 0
        assert torch.equal(c2, c)


@pytest.mark.parametrize("fmt", [0, 1, 2])
@pytest.mark.parametrize("w_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("sides", ["out", "both"])
@pytest.mark.parametrize("N", [200, 320])
def test_fold_weights_two_sided(B, fmt, w_dtype, sides, N):
    """W~~ = A_in_inv W A_out, c = (bias - b_in A_in_inv W) A_out + v_out: the V projection (both sides) and the FFN / MHA
    output (output side only) of the appendix on folding.  N = 320 with bf16 weights takes the tensor-core products
    (several tiles in both directions, a half-filled last one), everything else the fp32 FMA products."""
    K = 320 if fmt else 320 + 64
    name = H.FMT_NAME[fmt]
    _, b_in, A_in_inv = synth.make_transform(K, 7, "bf16")
    A_out, v_out, _ = synth.make_transform(N, 9, "f32")
    W, bias = synth.make_weights(K, N, 7, dtype=w_dtype)
    both = sides == "both"
    wc, wsc, c, dump = B.fold_weights_two_sided(A_in_inv.cuda() if both else None, b_in.cuda() if both else None, W.cuda(),
                                                bias.cuda(), A_out.cuda(), v_out.cuda(), fmt, dump=True)
    rcodes, rscales, rc, Wf = orc.fold_weights_two_sided(A_in_inv.double().numpy() if both else None,
                                                         b_in.double().numpy() if both else None, W.double().numpy(),
                                                         bias.double().numpy(), A_out.double().numpy(), v_out.double().numpy(), name)
    D = dump.double().cpu().numpy()
    gc, gs = H.codes_to_numpy(wc, N, K, fmt), H.scales_to_linear(B, wsc, N, K, 1)
    qc, qs = orc.mx_quantize(D, name)
    assert np.array_equal(gc, qc) and np.array_equal(gs, qs)            # bit-exact on its own folded values
    # two fp32-accurate products in a row: the first as in the one-sided fold, the second an fp32 FMA chain of length N
    # tensor-core products (bf16 weights; fp32 weights on the input side, as three terms) accumulate with up to 9K / 16
    # roundings that may truncate; the fp32 FMA chain of the output side alone is tighter
    assert H.rel_fro(D, Wf.T) < (6e-6 if (w_dtype == "bf16" or both) else 2e-6)
    inner = (A_in_inv.double().numpy() @ W.double().numpy()) if both else W.double().numpy()     # K x N
    At = A_out.double().numpy().T
    tau = H.accumulation_tau(At, inner.T, H.fma_unit(N) + H.tensor_core_unit(9 * max(K, N)))
    if both:     # the other product's own error, carried through |A_out|
        tau1 = H.accumulation_tau(W.double().numpy().T, A_in_inv.double().numpy().T, H.fma_unit(K) + H.tensor_core_unit(9 * K))
        tau = tau + np.abs(At) @ tau1
    acc = orc.check_codes(Wf.T, gc, gs, tau, name)
    assert acc["illegal"] == 0, acc
    # c is accumulated in fp64 but from fp32 intermediates (the bias after one side, the weights after one side): the bound
    # is relative to the sum of the magnitudes that enter it, not to c itself
    mag = np.abs(bias.double().numpy()) @ np.abs(At.T) + np.abs(v_out.double().numpy())
    if both:
        mag = mag + np.abs(b_in.double().numpy()) @ np.abs(A_in_inv.double().numpy()) @ np.abs(W.double().numpy()) @ np.abs(At.T)
    assert (np.abs(c.cpu().numpy() - rc) <= 4e-7 * mag + 1e-9).all()
    # every codes / scales byte equals the oracle's except at legal near-ties
    assert (gc != rcodes).mean() < 2e-3


def test_fold_weights_two_sided_argument_rules(B):
    K, N, fmt = 128, 64, 0
    _, b_in, A_in_inv = synth.make_transform(K, 3, "bf16")
    A_out, v_out, _ = synth.make_transform(N, 4, "f32")
    W, bias = synth.make_weights(K, N, 3, dtype="bf16")
    d = lambda t: t.cuda()
    # input side only == the one-sided fold, byte for byte
    a = B.fold_weights_two_sided(d(A_in_inv), d(b_in), d(W), d(bias), None, None, fmt, dump=True)
    b = B.fold_weights(d(A_in_inv), d(b_in), d(W), d(bias), fmt, dump=True)
    for u, v in zip(a, b):
        assert torch.equal(u, v)
    for args in [(None, None, None, None),                 # nothing to fold
                 (None, d(b_in), d(A_out), None),          # shift without its matrix
                 (d(A_in_inv), None, None, d(v_out))]:
        with pytest.raises(B.LatmixError) as e:
            B.fold_weights_two_sided(args[0], args[1], d(W), d(bias), args[2], args[3], fmt)
        assert e.value.code == B.ERR_INVALID_ARG
    small = torch.zeros(256 + 8 * K + 4 * N, dtype=torch.uint8, device="cuda")     # lacks the N x K intermediate
    with pytest.raises(B.LatmixError) as e:
        B.fold_weights_two_sided(d(A_in_inv), None, d(W), None, d(A_out), None, fmt, ws=small)
    assert e.value.code == B.ERR_WORKSPACE


# ------------------------------------------------------------------ S3: block-scaled GEMM
@pytest.mark.parametrize("fmt,variant", [(0, 0), (0, 1), (0, 2), (0, 3), (1, 0), (1, 1), (1, 3), (0, 8), (1, 8), (3, 0), (3, 1),
                                         (0, 9), (1, 9), (3, 9)])
def test_mx_gemm_tensor_core(B, fmt, variant):
    M, K, N = 300, 2048, 712                   # ragged M and N tails for every tile width, 8 or 16 k-slabs
    ac, asc = H.random_mx(M, K, fmt, 11)
    wc, wsc = H.random_mx(N, K, fmt, 12)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, fmt)
    out = torch.full((M, N), float("nan"), device="cuda")
    n0 = B.launch_count()
    B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, out=out, ws=ws, flags=variant << 8)
    assert B.launch_count() == n0 + 1
    assert B.device_status(ws) == B.OK
    ref = orc.mx_matmul(ac, asc, wc, wsc, c.numpy(), H.FMT_NAME[fmt])
    H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), tag=f"tc variant {variant}")


@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("kernel", [8, 9])
@pytest.mark.parametrize("M,K,N", [(520, 1536, 392), (129, 256, 64), (1024, 512, 1024), (4096, 256, 3840), (2304, 768, 1000),
                                   (2560, 2048, 8192)])
def test_mx_gemm_cta_pairs(B, fmt, kernel, M, K, N):
    """The CTA-pair kernels (8: 256 x 192 tiles, 9: 256 x 256 tiles as two halves in three rotating accumulators, the second
    half catching up on the first at tile boundaries): odd slab counts, a second CTA with a single valid row, fewer weight rows than one tile, whole
    tiles, and several tiles per CTA pair (up to 320 tiles on at most 74 pairs) so that both tile streams, both
    accumulators and every wrap of the rings are in use at once."""
    ac, asc = H.random_mx(M, K, fmt, 31)
    wc, wsc = H.random_mx(N, K, fmt, 32)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, fmt)
    out = torch.full((M, N), float("nan"), device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, out=out, ws=ws, flags=kernel << 8)
    assert B.device_status(ws) == B.OK
    ref = orc.mx_matmul(ac, asc, wc, wsc, c.numpy(), H.FMT_NAME[fmt])
    H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), tag=f"pairs kernel {kernel}")
    # same sums in the same order per output element as the single-CTA kernel: identical bits
    out1 = B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, ws=ws, flags=1 << 8)
    assert torch.equal(out, out1)


def test_mx_gemm_same_addresses_other_shapes(B):
    """The launchers keep the TMA tensor maps they have built (per host thread, keyed by address and geometry).  Three
    products of different shapes whose operands, scales and results start at the SAME device addresses, then the first one
    again: every result must match its own oracle, which a map reused for another geometry would not."""
    fmt = 0
    shapes = [(256, 512, 256), (200, 1024, 320), (384, 256, 132), (256, 512, 256)]
    pool = {name: torch.zeros(1 << 20, dtype=torch.uint8, device="cuda") for name in ("a", "sa", "w", "sw")}
    out_pool = torch.zeros(1 << 18, dtype=torch.float32, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    B.workspace_init(ws)
    for i, (M, K, N) in enumerate(shapes):
        ac, asc = H.random_mx(M, K, fmt, 51 + (i % 3))
        wc, wsc = H.random_mx(N, K, fmt, 61 + (i % 3))
        da, dsa = H.mx_to_device(B, ac, asc, fmt)
        dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
        views = {}
        for name, t in (("a", da), ("sa", dsa), ("w", dw), ("sw", dsw)):
            views[name] = pool[name][:t.numel()]
            views[name].copy_(t)
        out = out_pool[:M * N].view(M, N)
        out.fill_(float("nan"))
        for kernel in (9, 8, 1):
            B.mx_gemm(views["a"], views["sa"], views["w"], views["sw"], None, M, K, N, fmt, out=out, ws=ws, flags=kernel << 8)
            assert B.device_status(ws) == B.OK
            ref = orc.mx_matmul(ac, asc, wc, wsc, None, "mxfp4")
            H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, "mxfp4", K, tag=f"shape {i} kernel {kernel}")


def test_mx_gemm_padded_leading_dimension_and_no_bias(B):
    M, K, N, ldo = 130, 512, 200, 256
    ac, asc = H.random_mx(M, K, 0, 3)
    wc, wsc = H.random_mx(N, K, 0, 4)
    da, dsa = H.mx_to_device(B, ac, asc, 0)
    dw, dsw = H.mx_to_device(B, wc, wsc, 0)
    big = torch.full((M, ldo), -7.0, device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 0, out=big[:, :N])
    ref = orc.mx_matmul(ac, asc, wc, wsc, None, "mxfp4")
    H.assert_gemm_parity(big[:, :N].cpu().numpy(), ref, ac, asc, wc, wsc, "mxfp4", K, tag="ldo")
    assert torch.all(big[:, N:] == -7.0)           # nothing written past column N


@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("M", [1, 16, 37])
def test_mx_gemm_cuda_core_small_m(B, fmt, M):
    K, N = 1024, 300
    ac, asc = H.random_mx(M, K, fmt, 21)
    wc, wsc = H.random_mx(N, K, fmt, 22)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    out = B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, flags=B.FLAG_FORCE_SIMT)
    ref = orc.mx_matmul(ac, asc, wc, wsc, c.numpy(), H.FMT_NAME[fmt])
    H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), simt=True, tag="cuda cores")


@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("M", [1, 7, 16, 17, 48, 64])
def test_mx_gemm_small_batch_kernel(B, fmt, M):
    """M <= 64 takes the kernel with swapped operands (weight rows on the 128-row side of the MMA): ragged last weight
    tile, every MMA width (16 to 64 activation rows), several tiles per CTA are not reached at this N (covered at full size);
    a padded leading dimension and no bias in the second call."""
    K, N = 2048, 712
    ac, asc = H.random_mx(M, K, fmt, 61)
    wc, wsc = H.random_mx(N, K, fmt, 62)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, fmt)
    out = torch.full((M, N), float("nan"), device="cuda")
    n0 = B.launch_count()
    B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, out=out, ws=ws)
    # one launch for every format: MXINT8 multiplies the integer codes as they are up to M = 64
    assert B.launch_count() == n0 + 1 and B.device_status(ws) == B.OK
    ref = orc.mx_matmul(ac, asc, wc, wsc, c.numpy(), H.FMT_NAME[fmt])
    H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), tag=f"small batch M={M}")
    if fmt == 2 and M <= 16:
        # kernel selection 5: the same product with the weights converted to bf16 on their way to the tensor core (exact
        # products, fp32 sums in another order than the integer kernel's)
        out5 = B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, ws=ws, flags=5 << 8)
        assert B.device_status(ws) == B.OK
        H.assert_gemm_parity(out5.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), tag=f"small batch, bf16 path M={M}")
        assert H.rel_fro(out5.cpu().numpy(), out.cpu().numpy()) < 1e-5      # both within the bound of the oracle; fp32 sums in different orders
    if fmt != 2:
        # the general single-CTA kernel (variant 1) computes the same sums in the same order per output: identical bits
        out1 = B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, ws=ws, flags=1 << 8)
        assert torch.equal(out, out1)
    wide = torch.full((M, N + 12), float("nan"), device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt, out=wide[:, :N], ws=ws)
    ref0 = orc.mx_matmul(ac, asc, wc, wsc, None, H.FMT_NAME[fmt])
    H.assert_gemm_parity(wide[:, :N].cpu().numpy(), ref0, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, tag=f"small batch, no bias M={M}")
    assert torch.isnan(wide[:, N:]).all()


@pytest.mark.parametrize("fmt,kernel", [(1, 0), (2, 0), (2, 5)])
def test_mx_gemm_small_batch_more_tiles_than_sms(B, fmt, kernel):
    """150 weight tiles of 128 rows on at most 148 SMs: some CTAs of the small-batch kernels take a second tile (the rings, the
    accumulator hand-back and the per-tile epilogue wrap around), the last tile is ragged."""
    M, K, N = 5, 384, 19132
    ac, asc = H.random_mx(M, K, fmt, 71)
    wc, wsc = H.random_mx(N, K, fmt, 72)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, fmt)
    out = torch.full((M, N), float("nan"), device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, fmt, out=out, ws=ws, flags=kernel << 8)
    assert B.device_status(ws) == B.OK
    ref = orc.mx_matmul(ac, asc, wc, wsc, c.numpy(), H.FMT_NAME[fmt])
    H.assert_gemm_parity(out.cpu().numpy(), ref, ac, asc, wc, wsc, H.FMT_NAME[fmt], K, c.numpy(), tag=f"small batch, 150 tiles, kernel {kernel}")


def test_saturated_and_extreme_scales_in_gemm(B):
    """Largest codes with large and tiny block scales: products stay exact, nothing overflows to inf."""
    M, K, N = 128, 256, 128
    ac = np.full((M, K), 0x7, dtype=np.uint8); wc = np.full((N, K), 0xF, dtype=np.uint8)      # +6 and -6
    asc = np.full((M, K // 32), 127 + 40, dtype=np.uint8); wsc = np.full((N, K // 32), 127 - 60, dtype=np.uint8)
    da, dsa = H.mx_to_device(B, ac, asc, 0)
    dw, dsw = H.mx_to_device(B, wc, wsc, 0)
    out = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 0)
    assert torch.all(out == -36.0 * K * 2.0 ** -20)


@pytest.mark.parametrize("M", [4, 16, 40])
def test_mxint8_extreme_scales_in_gemm(B, M):
    """MXINT8 with the largest codes and scale bytes at both ends of E8M0, mixed per block: the in-kernel expansion (M <= 16)
    and the expansion through the workspace (M = 40) must both reproduce the exact products, subnormal ones included."""
    K, N = 256, 136
    rng = np.random.default_rng(5)
    ac = rng.choice(np.array([0x7F, 0x81, 0x01, 0xFF, 0x00], dtype=np.uint8), size=(M, K))       # 127, -127, 1, -1, 0
    wc = rng.choice(np.array([0x7F, 0x81, 0x01, 0xFF, 0x00], dtype=np.uint8), size=(N, K))
    asc = rng.choice(np.array([0, 1, 120, 127, 160], dtype=np.uint8), size=(M, K // 32))
    wsc = rng.choice(np.array([0, 2, 100, 127, 150], dtype=np.uint8), size=(N, K // 32))
    da, dsa = H.mx_to_device(B, ac, asc, 2)
    dw, dsw = H.mx_to_device(B, wc, wsc, 2)
    out = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 2).double().cpu().numpy()
    ref = orc.mx_matmul(ac, asc, wc, wsc, None, "mxint8")
    assert np.isfinite(out).all()
    # every product is exact; eight-block sums of values of very different magnitude round in fp32
    assert np.abs(out - ref).max() <= 2.0 ** -20 * np.abs(ref).max()
    if M <= 16:                                        # the bf16 form of the small-batch kernel (kernel selection 5)
        out5 = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 2, flags=5 << 8).double().cpu().numpy()
        assert np.isfinite(out5).all() and np.abs(out5 - ref).max() <= 2.0 ** -20 * np.abs(ref).max()
    # a block whose scale product underflows fp32 contributes nothing on either side; a single huge block must come out exactly
    ac1 = np.zeros((M, K), dtype=np.uint8); ac1[:, :32] = 0x7F
    asc1 = np.full((M, K // 32), 127, dtype=np.uint8); asc1[:, 0] = 160
    da, dsa = H.mx_to_device(B, ac1, asc1, 2)
    out1 = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 2).double().cpu().numpy()
    assert np.array_equal(out1, orc.mx_matmul(ac1, asc1, wc, wsc, None, "mxint8").astype(np.float32).astype(np.float64))
    # scales near the top of E8M0 on one side against tiny ones on the other: every element and product is representable
    asc2 = np.full((M, K // 32), 127 + 118, dtype=np.uint8); wsc2 = np.full((N, K // 32), 127 - 117, dtype=np.uint8)
    da, dsa = H.mx_to_device(B, ac, asc2, 2)
    dw, dsw = H.mx_to_device(B, wc, wsc2, 2)
    out2 = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, 2).double().cpu().numpy()
    ref2 = orc.mx_matmul(ac, asc2, wc, wsc2, None, "mxint8")
    assert np.isfinite(out2).all() and np.abs(out2 - ref2).max() <= 2.0 ** -20 * np.abs(ref2).max()


# ------------------------------------------------------------------ whole layer
@pytest.mark.parametrize("cfg_name", ["cfg0", "mid_fp4", "mid_fp8", "mid_int8"])
def test_linear_layer_against_fp64_chain(B, cfg_name):
    cfg = {"cfg0": synth.CONFIGS["cfg0"],
           "mid_fp4": synth.LayerConfig("mid_fp4", 384, 1024, 832, seed=21),
           "mid_fp8": synth.LayerConfig("mid_fp8", 200, 512, 320, fmt="mxfp8", seed=22),
           "mid_int8": synth.LayerConfig("mid_int8", 200, 512, 320, fmt="mxint8", seed=23)}[cfg_name]
    fmt = B.FORMATS[cfg.fmt]
    L = synth.make_layer(cfg)
    d = {k: v.cuda() for k, v in L.items()}
    wq, wsc, c, _ = B.fold_weights(d["A_inv"], d["b"], d["W"], d["bias"], fmt)
    ws = B.new_workspace(B.OP_LINEAR, cfg.M, cfg.K, cfg.N, fmt)
    out = B.linear(d["X"], d["A"], d["b"], wq, wsc, c, cfg.N, fmt, ws=ws).cpu().numpy()
    assert B.device_status(ws) == B.OK
    n64 = {k: v.double().numpy() for k, v in L.items()}
    # (a) exact contraction of the codes the GPU produced
    a_codes, a_scales, _ = B.quantize_mx(d["X"], d["A"], d["b"], fmt, ws=ws)
    gac, gas = H.codes_to_numpy(a_codes, cfg.M, cfg.K, fmt), H.scales_to_linear(B, a_scales, cfg.M, cfg.K, 1)
    gwc, gws = H.codes_to_numpy(wq, cfg.N, cfg.K, fmt), H.scales_to_linear(B, wsc, cfg.N, cfg.K, 1)
    ref_own = orc.mx_matmul(gac, gas, gwc, gws, c.cpu().numpy(), cfg.fmt)
    # cfg0 (fp32 inputs, M = 128) and the MXINT8 case without the larger workspace run the product on the CUDA cores
    H.assert_gemm_parity(out, ref_own, gac, gas, gwc, gws, cfg.fmt, cfg.K, c.cpu().numpy(), simt=None, tag=cfg_name)
    # (b) the whole chain in fp64.  Every code the GPU produced is either the chain's code or a legal
    # near-tie alternate (checked here), so the chain with the GPU's choice substituted on those elements is
    # ref_own and (a) already meets CHAIN_TOL; the unsubstituted difference is bounded loosely because one
    # tie flip moves an element by a whole grid step.
    wc64, ws64, c64, Wf = orc.fold_weights(n64["A_inv"], n64["b"], n64["W"], n64["bias"], cfg.fmt)
    Y64 = orc.affine_transform(n64["X"], n64["A"], n64["b"])
    unit_a = H.fma_unit(cfg.K) if cfg.x_dtype == "f32" else H.tensor_core_unit(cfg.K)
    acc_a = orc.check_codes(Y64, gac, gas, H.accumulation_tau(n64["X"], n64["A"], unit_a), cfg.fmt)
    acc_w = orc.check_codes(Wf.T, gwc, gws, H.accumulation_tau(n64["W"].T, n64["A_inv"].T, H.fma_unit(cfg.K)), cfg.fmt)
    assert acc_a["illegal"] == 0 and acc_w["illegal"] == 0, (acc_a, acc_w)
    assert H.rel_fro(out, ref_own) < CHAIN_TOL
    ref = orc.latmix_linear(n64["X"], n64["A"], n64["b"], wc64, ws64, c64, cfg.fmt)
    chain = H.rel_fro(out, ref)
    print(f"PARITY {cfg_name} activations {acc_a} weights {acc_w} rel_fro_vs_fp64_chain_unsubstituted={chain:.3e}")
    assert chain < 1e-2
    # and the layer does what it is for: it approximates x W + bias
    plain = n64["X"] @ n64["W"] + n64["bias"]
    assert H.rel_fro(out, plain) < {"mxfp4": 0.3, "mxfp8": 0.08, "mxint8": 0.03}[cfg.fmt]


@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
def test_small_and_ragged_shapes_whole_path(B, fmt):
    """Fold, transform + quantise and GEMM at sizes far below one tile and off every tile boundary (one row, K of a single
    slab or less, a handful of output columns): every default kernel choice must still agree with the oracle."""
    name = H.FMT_NAME[fmt]
    ks = [64, 128, 192, 320] if fmt == 0 else [32, 96, 128, 320]          # MXINT4 (3) is stored and sized like the 8-bit formats
    for M, K, N in [(1, ks[0], 8), (5, ks[1], 40), (129, ks[2], 200), (300, ks[3], 8), (1, ks[3], 200)]:
        X = synth.make_activations(M, K, 3, dtype="bf16")
        A, b, A_inv = synth.make_transform(K, 3, "bf16")
        W, bias = synth.make_weights(K, N, 3)
        wq, wsc, c, wd = B.fold_weights(A_inv.cuda(), b.cuda(), W.cuda(), bias.cuda(), fmt, dump=True)
        ws = B.new_workspace(B.OP_LINEAR, M, K, N, fmt)
        out = B.linear(X.cuda(), A.cuda(), b.cuda(), wq, wsc, c, N, fmt, ws=ws)
        codes, scales, Y = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), fmt, dump=True, ws=ws)
        assert B.device_status(ws) == B.OK
        gc, gs = H.codes_to_numpy(codes, M, K, fmt), H.scales_to_linear(B, scales, M, K, 1)
        rc, rs = orc.mx_quantize(Y.double().cpu().numpy(), name)
        assert np.array_equal(gc, rc) and np.array_equal(gs, rs), (M, K, N)
        wc, wss = H.codes_to_numpy(wq, N, K, fmt), H.scales_to_linear(B, wsc, N, K, 1)
        rwc, rws = orc.mx_quantize(wd.double().cpu().numpy(), name)
        assert np.array_equal(wc, rwc) and np.array_equal(wss, rws), (M, K, N)
        Y64 = orc.affine_transform(X.double().numpy(), A.double().numpy(), b.double().numpy())
        assert H.rel_fro(Y.double().cpu().numpy(), Y64) < 1e-5, (M, K, N)
        ref = orc.mx_matmul(gc, gs, wc, wss, c.cpu().numpy(), name)
        H.assert_gemm_parity(out.cpu().numpy(), ref, gc, gs, wc, wss, name, K, c.cpu().numpy(), simt=None, tag=f"ragged {(M, K, N)}")


def test_results_are_deterministic(B):
    cfg = synth.LayerConfig("det", 256, 512, 384, seed=31)
    L = {k: v.cuda() for k, v in synth.make_layer(cfg).items()}
    wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], 0)
    o1 = B.linear(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, 0)
    o2 = B.linear(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, 0)
    assert torch.equal(o1, o2)


@pytest.mark.parametrize("M", [16, 300])
def test_layer_can_be_captured_in_a_cuda_graph(B, M):
    """The calls allocate nothing and only enqueue work on the caller's stream, so a whole layer can be recorded once and
    replayed: same bits as the eager call, also after the input buffer's contents change."""
    cfg = synth.LayerConfig("graph", M, 512, 448, seed=32)
    L = {k: v.cuda() for k, v in synth.make_layer(cfg).items()}
    wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], 0)
    ws = B.new_workspace(B.OP_LINEAR, cfg.M, cfg.K, cfg.N, 0)
    X = L["X"].clone()
    out = torch.empty(cfg.M, cfg.N, device="cuda")
    eager = B.linear(X, L["A"], L["b"], wq, wsc, c, cfg.N, 0, ws=ws).clone()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        B.linear(X, L["A"], L["b"], wq, wsc, c, cfg.N, 0, out=out, ws=ws)          # warm-up on the capture stream
        with torch.cuda.graph(g, stream=side):
            B.linear(X, L["A"], L["b"], wq, wsc, c, cfg.N, 0, out=out, ws=ws)
    torch.cuda.current_stream().wait_stream(side)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    X2 = synth.make_activations(cfg.M, cfg.K, 99, dtype="bf16").cuda()
    eager2 = B.linear(X2, L["A"], L["b"], wq, wsc, c, cfg.N, 0).clone()
    X.copy_(X2)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager2) and not torch.equal(eager2, eager)
    assert B.device_status(ws) == B.OK


# ------------------------------------------------------------------ transformation MSE (Eq. q_error, block-wise error)
@pytest.mark.parametrize("fmt", [0, 1, 2, 3])
@pytest.mark.parametrize("case", ["tensor_core", "cuda_core", "f32", "identity", "blocks"])
def test_transformation_mse(B, fmt, case):
    """E(T) and E_B^i(T): (a) against the oracle evaluated on the kernel's own transformed values (tight: only the
    fp32-accurate back-mapping product and fp64 sums differ), (b) against the all-fp64 chain (loose: near-tie flips)."""
    name = H.FMT_NAME[fmt]
    M, K = (192, 384) if case in ("tensor_core", "blocks", "identity") else (50, 192)
    dtype = "f32" if case == "f32" else "bf16"
    X = synth.make_activations(M, K, 51, dtype=dtype)
    flags = 0
    if case == "identity":
        A = A_inv = None
        b = (torch.randn(K) * 0.1).float()
    elif case == "blocks":
        A, b, A_inv = synth.make_block_transform(K, 51, "haar", a_dtype=dtype, b_std=0.1)
        flags = B.FLAG_BLOCK_DIAG
    else:
        A, b, A_inv = synth.make_transform(K, 51, dtype)
    dA = None if A is None else A.cuda()
    dAi = None if A_inv is None else A_inv.cuda()
    ws = B.new_workspace(B.OP_TRANSFORMATION_MSE, M, K, 0, fmt)
    if case == "cuda_core":
        flags |= B.FLAG_FORCE_SIMT
    n0 = B.launch_count()
    mse, blk = B.transformation_mse(X.cuda(), dA, b.cuda(), dAi, fmt, ws=ws, flags=flags)
    n1 = B.launch_count()
    assert B.device_status(ws) == B.OK
    if case in ("tensor_core", "blocks"):
        assert n1 - n0 == 1 + 1 + 3 + 2          # quantiser, difference, two splits + product, sums
    # (a) the same transform + quantiser call, dumped
    _, _, Y = B.quantize_mx(X.cuda(), dA, b.cuda(), fmt, B.SF_LINEAR, dump=True, flags=flags)
    Yg = Y.double().cpu().numpy()
    qc, qs = orc.mx_quantize(Yg, name)
    d = Yg - orc.mx_dequantize(qc, qs, name)
    e = d if A_inv is None else d @ A_inv.double().numpy()
    want_blk = (e ** 2).reshape(M, K // 32, 32).mean(axis=(0, 2))
    assert np.allclose(blk.cpu().numpy(), want_blk, rtol=2e-5, atol=0)
    assert np.isclose(float(mse), (e ** 2).mean(), rtol=2e-5, atol=0)
    assert np.isclose(float(mse), blk.cpu().numpy().mean(), rtol=1e-14, atol=0)
    # (b) the oracle's own chain
    X64, b64 = X.double().numpy(), b.double().numpy()
    if case == "identity":
        ref_mse, ref_blk = orc.transformation_mse(X64, None, None, b64, name)
    elif case == "blocks":
        dense = np.zeros((K, K))
        for i in range(K // 32):
            dense[32 * i:32 * i + 32, 32 * i:32 * i + 32] = A[i].double().numpy()
        ref_mse, ref_blk = orc.transformation_mse(X64, dense, A_inv.double().numpy(), b64, name)
    else:
        ref_mse, ref_blk = orc.transformation_mse(X64, A.double().numpy(), A_inv.double().numpy(), b64, name)
    assert np.isclose(float(mse), ref_mse, rtol=5e-3)
    assert np.allclose(blk.cpu().numpy(), ref_blk, rtol=5e-2)


@pytest.mark.parametrize("block", [8, 16, 64, 128])
@pytest.mark.parametrize("fmt", [0, 1, 2])
@pytest.mark.parametrize("case", ["full", "identity", "hadamard"])
def test_transformation_mse_block_size_sweep(B, block, fmt, case):
    """E(T) and E_B^i for MX block sizes other than the layer's 32 (the block-size sweep of the numerical analysis in
    Sec. 3.1): against the oracle's quantiser with that block size, on the kernel's own transformed values (tight) and on
    the all-fp64 chain (loose: near-ties)."""
    name = H.FMT_NAME[fmt]
    M, K = 200, 384
    X = synth.make_activations(M, K, 53, dtype="bf16")
    flags = 0
    if case == "identity":
        A = A_inv = None
        b = (torch.randn(K) * 0.1).float()
    elif case == "hadamard":
        A, b, A_inv = synth.make_block_transform(K, 53, "hadamard")
        flags = B.FLAG_BLOCK_DIAG
    else:
        A, b, A_inv = synth.make_transform(K, 53, "bf16")
    d = lambda t: None if t is None else t.cuda()
    mse, blk = B.transformation_mse(X.cuda(), d(A), d(b), d(A_inv), fmt, flags=flags, block=block)
    assert blk.numel() == K // block
    _, _, Y = B.quantize_mx(X.cuda(), d(A), d(b), fmt, B.SF_LINEAR, dump=True, flags=flags)
    Yg = Y.double().cpu().numpy()
    qc, qs = orc.mx_quantize(Yg, name, block=block)
    e = Yg - orc.mx_dequantize(qc, qs, name, block=block)
    if A_inv is not None:
        e = e @ A_inv.double().numpy()
    want = (e ** 2).reshape(M, K // block, block).mean(axis=(0, 2))
    assert np.allclose(blk.cpu().numpy(), want, rtol=2e-5, atol=0)
    assert np.isclose(float(mse), (e ** 2).mean(), rtol=2e-5, atol=0)
    X64 = X.double().numpy()
    b64 = None if b is None else b.double().numpy()
    if case == "identity":
        ref_mse, _ = orc.transformation_mse(X64, None, None, b64, name, block=block)
    elif case == "hadamard":
        dense = np.kron(np.eye(K // 32), orc.hadamard_block(32))
        ref_mse, _ = orc.transformation_mse(X64, dense, A_inv.double().numpy(), b64, name, block=block)
    else:
        ref_mse, _ = orc.transformation_mse(X64, A.double().numpy(), A_inv.double().numpy(), b64, name, block=block)
    # Hadamard blocks of bf16 inputs put many values exactly on rounding boundaries, where fp32 and fp64 sums part ways
    assert np.isclose(float(mse), ref_mse, rtol=3e-2)
    with pytest.raises(B.LatmixError) as err:
        B.transformation_mse(X.cuda(), d(A), d(b), d(A_inv), fmt, flags=flags, block=24)
    assert err.value.code == B.ERR_INVALID_ARG


def test_transformation_mse_is_reproducible_and_checks_arguments(B):
    M, K, fmt = 128, 256, 0
    X = synth.make_activations(M, K, 52, dtype="bf16")
    A, b, A_inv = synth.make_transform(K, 52, "bf16")
    r1 = B.transformation_mse(X.cuda(), A.cuda(), b.cuda(), A_inv.cuda(), fmt)
    r2 = B.transformation_mse(X.cuda(), A.cuda(), b.cuda(), A_inv.cuda(), fmt)
    assert torch.equal(r1[0], r2[0]) and torch.equal(r1[1], r2[1])
    with pytest.raises(B.LatmixError) as e:
        B.transformation_mse(X.cuda(), A.cuda(), b.cuda(), None, fmt)          # a transform without its inverse
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.LatmixError) as e:
        B.transformation_mse(X.cuda(), A.cuda(), b.cuda(), A_inv.cuda(), fmt, ws=torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.code == B.ERR_WORKSPACE
