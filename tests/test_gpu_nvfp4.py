"""NVFP4 (blocks of 16 E2M1 elements, E4M3 block scale, fp32 tensor scale): parity of the CUDA path with the oracle.

Codes and scale bytes must match the oracle bit for bit -- for the plain quantiser on any input, for the fused
transform and the offline fold on the kernel's own fp32 pre-quantisation values -- and the product must match the fp64
contraction of the same codes within the accumulation bound."""
import numpy as np
import pytest
import torch

from oracle import latmix_oracle as orc
from paper_2602_17681_b200 import synth
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import binding
    return binding


def _codes(codes_t, rows, K):
    return orc.unpack_fp4(codes_t.cpu().numpy()[: rows * K // 2].reshape(rows, K // 2))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("sf", [0, 1])
def test_plain_quantizer_bit_exact(B, dtype, sf):
    M, K = 301, 1088 + 64                                   # ragged rows, K/16 not a multiple of 16
    g0 = torch.Generator().manual_seed(3)
    X = torch.randn(M, K, generator=g0, dtype=torch.float64) * torch.exp(torch.randn(M, 1, generator=g0, dtype=torch.float64) * 2)
    X[:, 5] *= 50
    X[3, 64:96] = 0
    X[1, 0] = -0.0
    X = X.to(dtype)
    g = orc.nvfp4_tensor_scale(float(X.abs().max()))
    codes, scales, _ = B.quantize_mx(X.cuda(), None, None, B.NVFP4, sf, tensor_scale=g)
    rc, rs = orc.nvfp4_quantize(X.double().numpy(), g)
    assert np.array_equal(_codes(codes, M, K), rc)
    assert np.array_equal(H.nvfp4_scales_to_linear(B, scales, M, K, sf), rs)
    # the trailer still holds the tensor scale
    off = B.tensor_scale_offset(M, K, B.NVFP4, sf)
    assert scales[off:off + 4].view(torch.float32).item() == float(g)
    # with a shift and a dump: quantises exactly the values it reports
    b = (torch.randn(K) * 0.1).cuda()
    codes, scales, Y = B.quantize_mx(X.cuda(), None, b, B.NVFP4, sf, dump=True, tensor_scale=g)
    assert torch.equal(Y, X.cuda().float() + b[None, :])
    rc, rs = orc.nvfp4_quantize(Y.double().cpu().numpy(), g)
    assert np.array_equal(_codes(codes, M, K), rc) and np.array_equal(H.nvfp4_scales_to_linear(B, scales, M, K, sf), rs)


@pytest.mark.parametrize("sf", [0, 1])
@pytest.mark.parametrize("path", ["tensor_core", "cuda_core", "f32"])
def test_transform_quantize(B, sf, path):
    M, K = (300, 1088 + 64) if path == "tensor_core" else (100, 320)
    dtype = "f32" if path == "f32" else "bf16"
    X = synth.make_activations(M, K, 5, dtype=dtype)
    A, b, _ = synth.make_transform(K, 5, dtype)
    flags = B.FLAG_FORCE_SIMT if path == "cuda_core" else 0
    Y64 = orc.affine_transform(X.double().numpy(), A.double().numpy(), b.double().numpy())
    g = orc.nvfp4_tensor_scale(np.abs(Y64).max())
    ws = B.new_workspace(B.OP_QUANTIZE_MX, M, K, 0, B.NVFP4)
    codes, scales, Y = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), B.NVFP4, sf, dump=True, ws=ws, flags=flags, tensor_scale=g)
    codes2, scales2, _ = B.quantize_mx(X.cuda(), A.cuda(), b.cuda(), B.NVFP4, sf, ws=ws, flags=flags, tensor_scale=g)
    assert B.device_status(ws) == B.OK
    gc, gs = _codes(codes, M, K), H.nvfp4_scales_to_linear(B, scales, M, K, sf)
    assert np.array_equal(_codes(codes2, M, K), gc) and np.array_equal(H.nvfp4_scales_to_linear(B, scales2, M, K, sf), gs)
    Yg = Y.double().cpu().numpy()
    rc, rs = orc.nvfp4_quantize(Yg, g)
    assert np.array_equal(gc, rc) and np.array_equal(gs, rs)            # bit-exact on the kernel's own values
    unit = H.tensor_core_unit(K) if path == "tensor_core" else H.fma_unit(K)
    assert np.all(np.abs(Yg - Y64) <= H.accumulation_tau(X.double().numpy(), A.double().numpy(), unit))
    # against the all-fp64 chain only near-ties may differ
    c64, s64 = orc.nvfp4_quantize(Y64, g)
    assert (c64 != gc).mean() < 5e-3 and (s64 != gs).mean() < 5e-3


@pytest.mark.parametrize("w_dtype", ["bf16", "f32"])
def test_fold_weights(B, w_dtype):
    K, N = 384, 200
    A, b, A_inv = synth.make_transform(K, 7, "bf16")
    W, bias = synth.make_weights(K, N, 7, dtype=w_dtype)
    _, _, rc64, Wf = orc.fold_weights(A_inv.double().numpy(), b.double().numpy(), W.double().numpy(), bias.double().numpy(), "mxfp4")
    g = orc.nvfp4_tensor_scale(np.abs(Wf).max())
    wc, wsc, c, dump = B.fold_weights(A_inv.cuda(), b.cuda(), W.cuda(), bias.cuda(), B.NVFP4, dump=True, tensor_scale=g)
    D = dump.double().cpu().numpy()
    assert H.rel_fro(D, Wf.T) < 5e-6
    qc, qs = orc.nvfp4_quantize(D, g)
    assert np.array_equal(_codes(wc, N, K), qc) and np.array_equal(H.nvfp4_scales_to_linear(B, wsc, N, K, 1), qs)
    assert np.allclose(c.cpu().numpy(), rc64, rtol=2e-7, atol=1e-9)


def _random_nvfp4(rows, K, seed):
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, 16, (rows, K), dtype=np.uint8)
    scales = rng.integers(0x28, 0x48, (rows, K // 16), dtype=np.uint8)      # E4M3 values 2^-2 .. 2^2
    return codes, scales


@pytest.mark.parametrize("M,K,N,flags", [(300, 2048, 712, 0), (2560, 1024, 4096, 0), (129, 256, 64, 0), (37, 1024, 300, 0),
                                         (300, 320, 200, 0), (130, 512, 136, 2)])
def test_gemm(B, M, K, N, flags):
    """Tensor cores (kind::mxf4nvf4, M > 128 and K a multiple of 256: ragged tiles, many tiles per CTA pair) and the CUDA-core
    kernel (small M, other K, LATMIX_FLAG_FORCE_SIMT)."""
    ac, asc = _random_nvfp4(M, K, 11)
    wc, wsc = _random_nvfp4(N, K, 12)
    ga, gw = np.float32(0.37), np.float32(2.0 ** -5 * 1.3)
    c = (torch.randn(N) * 0.1).float()
    da, dsa = H.nvfp4_to_device(B, ac, asc, ga)
    dw, dsw = H.nvfp4_to_device(B, wc, wsc, gw)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, B.NVFP4)
    out = torch.full((M, N), float("nan"), device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, c.cuda(), M, K, N, B.NVFP4, out=out, ws=ws, flags=flags)
    assert B.device_status(ws) == B.OK
    ref = orc.nvfp4_matmul(ac, asc, ga, wc, wsc, gw, c.numpy())
    got = out.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert H.rel_fro(got, ref) < 1e-4
    mag = np.abs(orc.nvfp4_dequantize(ac, asc, ga)) @ np.abs(orc.nvfp4_dequantize(wc, wsc, gw)).T + np.abs(c.numpy())[None, :]
    # per element: one fp32 rounding per MMA (K / 64 of them) or per block on the CUDA cores, the product of the two tensor
    # scales and the fused multiply-add of the epilogue
    unit = (K / 16 + 8) * 2.0 ** -23
    assert np.all(np.abs(got - ref) <= unit * mag + 2.0 ** -22 * np.abs(ref))
    print(f"GEMM_ERR nvfp4 {(M, K, N, flags)} max_err_over_2^-24_mag={np.max(np.abs(got - ref) / (mag * 2.0 ** -24)):.2f}")


def test_layer_against_fp64_chain(B):
    cfg = synth.LayerConfig("nv_mid", 384, 1024, 832, seed=21)
    L = synth.make_layer(cfg)
    d = {k: v.cuda() for k, v in L.items()}
    n64 = {k: v.double().numpy() for k, v in L.items()}
    Y64 = orc.affine_transform(n64["X"], n64["A"], n64["b"])
    Wf64 = n64["A_inv"] @ n64["W"]
    ga, gw = orc.nvfp4_tensor_scale(np.abs(Y64).max()), orc.nvfp4_tensor_scale(np.abs(Wf64).max())
    wq, wsc, c, _ = B.fold_weights(d["A_inv"], d["b"], d["W"], d["bias"], B.NVFP4, tensor_scale=gw)
    ws = B.new_workspace(B.OP_LINEAR, cfg.M, cfg.K, cfg.N, B.NVFP4)
    B.workspace_set_tensor_scale(ws, ga)
    n0 = B.launch_count()
    out = B.linear(d["X"], d["A"], d["b"], wq, wsc, c, cfg.N, B.NVFP4, ws=ws).double().cpu().numpy()
    assert B.launch_count() - n0 == 2 and B.device_status(ws) == B.OK
    a_codes, a_scales, _ = B.quantize_mx(d["X"], d["A"], d["b"], B.NVFP4, ws=ws, tensor_scale=ga)
    gac, gas = _codes(a_codes, cfg.M, cfg.K), H.nvfp4_scales_to_linear(B, a_scales, cfg.M, cfg.K, 1)
    gwc, gws = _codes(wq, cfg.N, cfg.K), H.nvfp4_scales_to_linear(B, wsc, cfg.N, cfg.K, 1)
    ref_own = orc.nvfp4_matmul(gac, gas, ga, gwc, gws, gw, c.cpu().numpy())
    assert H.rel_fro(out, ref_own) < 1e-4
    # the oracle's own chain: fp64 transform and fold, NVFP4 quantisation of both, fp64 contraction
    qc, qs = orc.nvfp4_quantize(Y64, ga)
    wc64, ws64 = orc.nvfp4_quantize(np.ascontiguousarray(Wf64.T), gw)
    c64 = n64["bias"] - n64["b"] @ Wf64
    ref = orc.nvfp4_matmul(qc, qs, ga, wc64, ws64, gw, c64)
    assert H.rel_fro(out, ref) < 1e-2                                   # near-tie flips only
    plain = n64["X"] @ n64["W"] + n64["bias"]
    assert H.rel_fro(out, plain) < 0.3


def test_full_size_cfg2_gate_up_sampled(B):
    """cfg2 gate/up with NVFP4 in the default launch configuration: sampled rows and columns against the oracle."""
    cfg = synth.CONFIGS["cfg2_gate_up"]
    M, K, N = cfg.M, cfg.K, cfg.N
    dev = torch.device("cuda")
    L = synth.make_layer(cfg, device=dev)
    ga = np.float32(float((L["X"].float().abs().max() * 4)) / (448 * 6))      # a calibration-style guess, not the exact maximum
    gw = np.float32(0.5 / (448 * 6))
    wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], B.NVFP4, tensor_scale=gw)
    ws = B.new_workspace(B.OP_LINEAR, M, K, N, B.NVFP4, dev)
    B.workspace_set_tensor_scale(ws, ga)
    out = B.linear(L["X"], L["A"], L["b"], wq, wsc, c, N, B.NVFP4, ws=ws)
    a_codes, a_scales, Y = B.quantize_mx(L["X"], L["A"], L["b"], B.NVFP4, dump=True, ws=ws, tensor_scale=ga)
    assert B.device_status(ws) == B.OK and torch.isfinite(out).all()
    rng = np.random.default_rng(2)
    rows = np.array(sorted(set(rng.choice(M, 24, replace=False).tolist()) | {0, 127, 128, 255, 256, M - 1}))
    cols = np.array(sorted(set(rng.choice(N, 48, replace=False).tolist()) | {0, 127, 128, 255, 256, N - 1}))
    ri, ci = torch.as_tensor(rows, device=dev), torch.as_tensor(cols, device=dev)
    # activations: bit-exact on the kernel's own values of the sampled rows
    Yg = Y[ri].double().cpu().numpy()
    rc, rs = orc.nvfp4_quantize(Yg, ga)
    gac = orc.unpack_fp4(a_codes[: M * K // 2].view(M, K // 2)[ri].cpu().numpy())
    gas = a_scales.cpu().numpy()[H.nvfp4_sf_offsets(M, K)[rows]]
    assert np.array_equal(gac, rc) and np.array_equal(gas, rs)
    gwc = orc.unpack_fp4(wq[: N * K // 2].view(N, K // 2)[ci].cpu().numpy())
    gws = wsc.cpu().numpy()[H.nvfp4_sf_offsets(N, K)[cols]]
    # weights of the sampled columns against the fp64 fold: near-ties aside
    Wf = L["A_inv"].double().cpu().numpy() @ L["W"][:, ci].double().cpu().numpy()
    wc64, ws64 = orc.nvfp4_quantize(np.ascontiguousarray(Wf.T), gw)
    assert (wc64 != gwc).mean() < 5e-3 and (ws64 != gws).mean() < 5e-3
    ref = orc.nvfp4_matmul(gac, gas, ga, gwc, gws, gw, c[ci].cpu().numpy())
    got = out[ri][:, ci].double().cpu().numpy()
    assert H.rel_fro(got, ref) < 1e-4
    mag = np.abs(orc.nvfp4_dequantize(gac, gas, ga)) @ np.abs(orc.nvfp4_dequantize(gwc, gws, gw)).T + np.abs(c[ci].cpu().numpy())[None, :]
    assert np.all(np.abs(got - ref) <= (K / 64 + 8) * 2.0 ** -23 * mag + 2.0 ** -22 * np.abs(ref))


def test_unsupported_combinations_are_refused(B):
    X = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros(8, 32, 32, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.LatmixError) as e:
        B.quantize_mx(X, A, None, B.NVFP4, flags=B.FLAG_BLOCK_DIAG, tensor_scale=1.0)
    assert e.value.code == B.ERR_UNSUPPORTED
    with pytest.raises(B.LatmixError) as e:
        B.transformation_mse(X, None, None, None, B.NVFP4)
    assert e.value.code == B.ERR_UNSUPPORTED
