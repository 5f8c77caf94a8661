"""Seeded synthetic inputs for the transformed MX-quantized linear layer.

This module only draws random tensors with the shapes and outlier structure of
the workloads (Llama-shaped layers with a few very large activation channels);
it contains none of the method's arithmetic and imports neither the CUDA
binding nor the CPU oracle.  Tests and the benchmark hand the same tensors to
both sides.

Stand-in note: the paper calibrates and evaluates on real LLM activations;
those models and datasets are not available here, so activations are i.i.d.
Gaussian (or Student-t) with a seeded subset of channels multiplied by a large
factor, which is the feature of real activations that MX block scales react to.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    M: int
    K: int
    N: int
    fmt: str = "mxfp4"            # mxfp4 | mxfp8 | mxint8 | mxint4 | nvfp4
    x_dtype: str = "bf16"         # bf16 | f32
    act: str = "normal"           # normal | student_t3
    outlier_frac: float = 0.01    # fraction of channels scaled up (or an absolute count if >= 1)
    outlier_scale: float = 50.0
    w_std: float = 0.02
    b_std: float = 0.1
    seed: int = 0


# The five benchmark configurations (index = seed).
CONFIGS = {
    "cfg0": LayerConfig("cfg0", 128, 256, 256, x_dtype="f32", outlier_frac=4, seed=0),
    "cfg1": LayerConfig("cfg1", 2048, 4096, 4096, seed=1),
    "cfg2_gate_up": LayerConfig("cfg2_gate_up", 4096, 4096, 14336, seed=2),
    # gate and up projections share the input transform: concatenated along N they are one layer call
    "cfg2_gate_up_fused": LayerConfig("cfg2_gate_up_fused", 4096, 4096, 28672, seed=2),
    "cfg2_down": LayerConfig("cfg2_down", 4096, 14336, 4096, seed=2),
    "cfg2_gate_up_int4": LayerConfig("cfg2_gate_up_int4", 4096, 4096, 14336, fmt="mxint4", seed=2),
    "cfg2_gate_up_nvfp4": LayerConfig("cfg2_gate_up_nvfp4", 4096, 4096, 14336, fmt="nvfp4", seed=2),
    "cfg3_fp8_m1": LayerConfig("cfg3_fp8_m1", 1, 4096, 14336, fmt="mxfp8", seed=3),
    "cfg3_fp8_m16": LayerConfig("cfg3_fp8_m16", 16, 4096, 14336, fmt="mxfp8", seed=3),
    "cfg3_fp8_m8192": LayerConfig("cfg3_fp8_m8192", 8192, 4096, 14336, fmt="mxfp8", seed=3),
    "cfg3_int8_m1": LayerConfig("cfg3_int8_m1", 1, 4096, 14336, fmt="mxint8", seed=3),
    "cfg3_int8_m16": LayerConfig("cfg3_int8_m16", 16, 4096, 14336, fmt="mxint8", seed=3),
    "cfg3_int8_m8192": LayerConfig("cfg3_int8_m8192", 8192, 4096, 14336, fmt="mxint8", seed=3),
    "cfg4": LayerConfig("cfg4", 8192, 8192, 28672, act="student_t3", outlier_frac=0.005,
                        outlier_scale=100.0, w_std=0.01, seed=4),
}


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _storage(t, dtype):
    return t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()


def make_activations(M, K, seed, act="normal", outlier_frac=0.01, outlier_scale=50.0,
                     dtype="bf16", device="cpu"):
    """M x K activations with seeded outlier channels."""
    g = _gen(seed * 7919 + 1, device)
    x = torch.randn(M, K, generator=g, device=device, dtype=torch.float64)
    if act == "student_t3":
        z = torch.randn(M, K, 3, generator=g, device=device, dtype=torch.float64)
        x = x / torch.sqrt((z * z).sum(-1) / 3.0)
    n_out = int(outlier_frac) if outlier_frac >= 1 else int(round(outlier_frac * K))
    if n_out > 0:
        idx = torch.randperm(K, generator=g, device=device)[:n_out]
        x[:, idx] *= outlier_scale
    return _storage(x, dtype)


def make_transform(K, seed, a_dtype="bf16", b_std=0.1, device="cpu"):
    """A = Q diag(s) with Q Haar-orthogonal and s log-uniform in [0.5, 2]; b ~ N(0, b_std^2).

    Returns (A in its storage dtype, b fp32, A_inv fp32) where A_inv inverts the
    STORED (rounded) A, so that the fold identity is not polluted by the
    rounding of A.
    """
    g = _gen(seed * 7919 + 2, device)
    G = torch.randn(K, K, generator=g, device=device, dtype=torch.float64)
    Q, R = torch.linalg.qr(G)
    Q = Q * torch.sign(torch.diagonal(R))[None, :]
    s = torch.exp(torch.empty(K, device=device, dtype=torch.float64).uniform_(
        math.log(0.5), math.log(2.0), generator=g))
    A = _storage(Q * s[None, :], a_dtype)
    b = (torch.randn(K, generator=g, device=device, dtype=torch.float64) * b_std).float()
    A_inv = torch.linalg.inv(A.double()).float().contiguous()
    return A, b, A_inv


def make_block_transform(K, seed, kind="haar", block=32, a_dtype="bf16", b_std=0.0, device="cpu"):
    """Block-wise online transform as [K/block, block, block] blocks (block i acts on elements i*block ...).

    kind "hadamard": every block is the orthonormal Walsh-Hadamard matrix (the paper's online transform, no bias);
    kind "haar": independent Haar blocks times a log-uniform column scale.  Returns (blocks in the storage dtype,
    b fp32 or None, dense fp32 inverse of the STORED block-diagonal matrix, for the offline fold)."""
    g = _gen(seed * 7919 + 6, device)
    nb = K // block
    if kind == "hadamard":
        H = torch.ones(1, 1, dtype=torch.float64, device=device)
        while H.shape[0] < block:
            H = torch.cat([torch.cat([H, H], 1), torch.cat([H, -H], 1)], 0)
        blocks = (H / math.sqrt(block)).expand(nb, block, block).clone()
    else:
        G = torch.randn(nb, block, block, generator=g, device=device, dtype=torch.float64)
        Q, R = torch.linalg.qr(G)
        Q = Q * torch.sign(torch.diagonal(R, dim1=1, dim2=2))[:, None, :]
        s = torch.exp(torch.empty(nb, 1, block, device=device, dtype=torch.float64).uniform_(
            math.log(0.5), math.log(2.0), generator=g))
        blocks = Q * s
    blocks = _storage(blocks, a_dtype)
    b = (torch.randn(K, generator=g, device=device, dtype=torch.float64) * b_std).float() if b_std > 0 else None
    A_inv = torch.block_diag(*torch.linalg.inv(blocks.double())).float().contiguous()
    return blocks, b, A_inv


def make_weights(K, N, seed, std=0.02, dtype="bf16", with_bias=True, device="cpu"):
    g = _gen(seed * 7919 + 3, device)
    W = _storage(torch.randn(K, N, generator=g, device=device, dtype=torch.float64) * std, dtype)
    bias = (torch.randn(N, generator=g, device=device, dtype=torch.float64) * 0.01).float() if with_bias else None
    return W, bias


def make_layer(cfg: LayerConfig, device="cpu", M=None):
    """All tensors of one configuration: dict(X, A, b, A_inv, W, bias)."""
    M = cfg.M if M is None else M
    X = make_activations(M, cfg.K, cfg.seed, cfg.act, cfg.outlier_frac, cfg.outlier_scale,
                         cfg.x_dtype, device)
    A, b, A_inv = make_transform(cfg.K, cfg.seed, cfg.x_dtype, cfg.b_std, device)
    W, bias = make_weights(cfg.K, cfg.N, cfg.seed, cfg.w_std, cfg.x_dtype, True, device)
    return dict(X=X, A=A, b=b, A_inv=A_inv, W=W, bias=bias)
