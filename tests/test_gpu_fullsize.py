"""The benchmark configurations at full size, in the launch configuration the benchmark times (same entry
points, default tile selection).  The oracle cannot run these sizes whole, so it recomputes sampled rows
and sampled output columns one by one: activation codes of sampled rows, folded weight codes of sampled
columns, and the outputs at their intersections."""
import numpy as np
import pytest
import torch

from oracle import latmix_oracle as orc
from paper_2602_17681_b200 import synth
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

CASES = ["cfg1", "cfg2_gate_up", "cfg2_down", "cfg3_fp8_m1", "cfg3_fp8_m16", "cfg3_fp8_m8192",
         "cfg3_int8_m1", "cfg3_int8_m16", "cfg3_int8_m8192", "cfg4", "cfg2_gate_up_int4"]


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import binding
    return binding


def _gather_scales(B, scales_t, rows_idx, rows_total, K):
    buf = scales_t.cpu().numpy()
    off = H.sf_offsets(rows_total, K)[rows_idx]
    return buf[off]


def _gather_codes(codes_t, rows_idx, K, fmt):
    row_bytes = K // 2 if fmt == 0 else K
    idx = torch.as_tensor(rows_idx, device=codes_t.device)
    sub = codes_t[: codes_t.numel() // row_bytes * row_bytes].view(-1, row_bytes)[idx].cpu().numpy()
    return orc.unpack_fp4(sub) if fmt == 0 else H.bytes_to_codes(sub, fmt)


@pytest.mark.parametrize("name", CASES)
def test_full_size_config_sampled(B, name):
    cfg = synth.CONFIGS[name]
    fmt = B.FORMATS[cfg.fmt]
    M, K, N = cfg.M, cfg.K, cfg.N
    dev = torch.device("cuda")
    L = synth.make_layer(cfg, device=dev)
    wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], fmt)
    ws = B.new_workspace(B.OP_LINEAR, M, K, N, fmt, dev)
    out = B.linear(L["X"], L["A"], L["b"], wq, wsc, c, N, fmt, ws=ws)
    a_codes, a_scales, _ = B.quantize_mx(L["X"], L["A"], L["b"], fmt, ws=ws)
    assert B.device_status(ws) == B.OK
    assert torch.isfinite(out).all()

    # Sample: a few random rows and columns plus BOTH sides of every tile boundary -- rows 128 i - 1 and 128 i (a CTA's
    # share of a tile is 128 rows), columns 64 j - 1 and 64 j (tiles are 128, 192 or 256 columns wide and start at
    # multiples of 64) -- so that every tile of the launch contributes corner elements to the comparison.
    rng = np.random.default_rng(cfg.seed)
    rows = set(rng.choice(M, size=min(M, 16), replace=False).tolist()) | {0, M - 1}
    rows |= {r for i in range(1, (M + 127) // 128) for r in (128 * i - 1, 128 * i)}
    cols = set(rng.choice(N, size=32, replace=False).tolist()) | {0, N - 1}
    cols |= {n for j in range(1, (N + 63) // 64) for n in (64 * j - 1, 64 * j)}
    rows, cols = np.array(sorted(rows)), np.array(sorted(cols))
    A64 = L["A"].double().cpu().numpy()
    b64 = L["b"].double().cpu().numpy()
    X64 = L["X"][torch.as_tensor(rows, device=dev)].double().cpu().numpy()
    Y64 = orc.affine_transform(X64, A64, b64)
    gac = _gather_codes(a_codes, rows, K, fmt)
    gas = _gather_scales(B, a_scales, rows, M, K)
    acc = orc.check_codes(Y64, gac, gas, H.accumulation_tau(X64, A64, H.tensor_core_unit(K)), cfg.fmt)
    assert acc["illegal"] == 0, acc
    assert acc["alternate"] <= 2e-3 * acc["total"], acc

    # folded weights of the sampled output columns
    Ainv64 = L["A_inv"].double().cpu().numpy()
    Wc64 = L["W"][:, torch.as_tensor(cols, device=dev)].double().cpu().numpy()
    bias64 = L["bias"][torch.as_tensor(cols, device=dev)].double().cpu().numpy()
    _, _, c64, Wf = orc.fold_weights(Ainv64, b64, Wc64, bias64, cfg.fmt)
    gwc = _gather_codes(wq, cols, K, fmt)
    gws = _gather_scales(B, wsc, cols, N, K)
    tau_w = H.accumulation_tau(Wc64.T, Ainv64.T, H.fma_unit(K))
    accw = orc.check_codes(Wf.T, gwc, gws, tau_w, cfg.fmt)
    assert accw["illegal"] == 0, accw
    c_gpu = c[torch.as_tensor(cols, device=dev)].cpu().numpy()
    assert np.allclose(c_gpu, c64, rtol=2e-7, atol=1e-9)

    # outputs at the intersections: exact contraction of the codes the GPU produced
    ref = orc.mx_matmul(gac, gas, gwc, gws, c_gpu, cfg.fmt)
    got = out[torch.as_tensor(rows, device=dev)][:, torch.as_tensor(cols, device=dev)].cpu().numpy()
    H.assert_gemm_parity(got, ref, gac, gas, gwc, gws, cfg.fmt, K, c_gpu, tag=name)
    # Against the whole fp64 chain: the chain's codes with the GPU's choice substituted on the legal near-tie
    # elements are exactly the GPU's codes (no illegal element above), so the substituted comparison is the
    # one just made and meets the 1e-3 layer tolerance with margin.  The unsubstituted difference is
    # dominated by those tie flips (one flip moves an FP4 element by a whole grid step) and is only bounded
    # loosely here.
    assert H.rel_fro(got, ref) < 1e-3
    wc64, ws64 = orc.mx_quantize(np.ascontiguousarray(Wf.T), cfg.fmt)
    ref_chain = orc.latmix_linear(X64, A64, b64, wc64, ws64, c64, cfg.fmt)
    chain = H.rel_fro(got, ref_chain)
    print(f"PARITY {name} sample={len(rows)}x{len(cols)} activations {acc} weights {accw} "
          f"rel_fro_same_codes={H.rel_fro(got, ref):.3e} rel_fro_vs_fp64_chain_unsubstituted={chain:.3e}")
    assert chain < 1e-2


@pytest.mark.parametrize("name,sides", [("cfg1", "both"), ("cfg1", "out"), ("cfg2_down", "both")])
def test_two_sided_fold_full_size_sampled(B, name, sides):
    """The two-sided fold at layer size (tensor-core products, many tiles, three-term operands): folded weight codes and
    bias of sampled output columns against the oracle, column by column."""
    cfg = synth.CONFIGS[name]
    fmt = B.FORMATS[cfg.fmt]
    K, N = cfg.K, cfg.N
    dev = torch.device("cuda")
    both = sides == "both"
    _, b_in, A_in_inv = synth.make_transform(K, cfg.seed, cfg.x_dtype, device=dev)
    A_out, v_out, _ = synth.make_transform(N, cfg.seed + 1, "f32", device=dev)
    W, bias = synth.make_weights(K, N, cfg.seed, cfg.w_std, cfg.x_dtype, True, dev)
    ws = B.new_workspace(B.OP_FOLD_TWO_SIDED, 0, K, N, fmt, dev)
    n0 = B.launch_count()
    wq, wsc, c, _ = B.fold_weights_two_sided(A_in_inv if both else None, b_in if both else None, W, bias, A_out, v_out, fmt, ws=ws)
    assert B.device_status(ws) == B.OK
    assert B.launch_count() - n0 == (9 if both else 3)          # the tensor-core path, not the fp32 FMA one

    rng = np.random.default_rng(cfg.seed + 5)
    cols = np.sort(rng.choice(N, size=24, replace=False))
    cols[0], cols[-1] = 0, N - 1
    ci = torch.as_tensor(cols, device=dev)
    W64 = W.double()
    Ao_cols = A_out.double()[:, ci]                                        # N x s
    T_cols = W64 @ Ao_cols                                                 # K x s  = (W A_out)[:, cols]
    bias_cols = (bias.double() @ Ao_cols + v_out.double()[ci]).cpu().numpy()
    Ainv64 = A_in_inv.double().cpu().numpy()
    # the oracle's two-sided fold, restricted to the sampled output columns: its output side sees only those columns
    # of A_out, which is all that enters them
    rc, rs, c64, Wf = orc.fold_weights_two_sided(Ainv64 if both else None, b_in.double().cpu().numpy() if both else None,
                                                 T_cols.cpu().numpy(), bias_cols, None, None, cfg.fmt)
    gwc = _gather_codes(wq, cols, K, fmt)
    gws = _gather_scales(B, wsc, cols, N, K)
    absW, absAo = W64.abs(), Ao_cols.abs()
    tau = (H.tensor_core_unit(3 * N) * (absW @ absAo)).cpu().numpy()       # error of T = W A_out, K x s
    if both:
        absAinv = np.abs(Ainv64)
        tau = absAinv @ tau + H.tensor_core_unit(9 * K) * (absAinv @ np.abs(T_cols.cpu().numpy()))
    accw = orc.check_codes(Wf.T, gwc, gws, tau.T + 1e-30, cfg.fmt)
    assert accw["illegal"] == 0, accw
    assert accw["alternate"] <= 2e-3 * accw["total"], accw
    mag = (bias.double().abs() @ absAo + v_out.double()[ci].abs()).cpu().numpy()
    if both:
        mag = mag + np.abs(b_in.double().cpu().numpy()) @ np.abs(Ainv64) @ (absW @ absAo).cpu().numpy()
    assert (np.abs(c[ci].cpu().numpy() - c64) <= 4e-7 * mag + 1e-9).all()
