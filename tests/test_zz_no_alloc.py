"""latmix_linear_static: the layer call for users who cannot allocate device memory (its scratch is an array
built into the library).  It must give what latmix_linear gives with a caller workspace, call after call, although
every call reuses the same scratch and finds the previous call's bytes in it.

Collected last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from paper_2602_17681_b200 import synth
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import binding
    return binding


def _layer(B, cfg, dev):
    L = synth.make_layer(cfg, device=dev)
    fmt = B.FORMATS[cfg.fmt]
    wq, wsc, c, _ = B.fold_weights(L["A_inv"], L["b"], L["W"], L["bias"], fmt)
    return L, fmt, wq, wsc, c


def test_static_scratch_matches_workspace_call_twice_in_a_row(B):
    dev = torch.device("cuda")
    # first a shape that fills whole scale tiles, then a ragged one in another format: the second call meets
    # stale codes, stale scales (where it needs zero padding) and a used status word in the shared scratch
    cases = [synth.LayerConfig("static_a", 384, 1024, 640, fmt="mxfp4", seed=21),
             synth.LayerConfig("static_b", 200, 768, 416, fmt="mxfp8", seed=22)]
    for cfg in cases:
        L, fmt, wq, wsc, c = _layer(B, cfg, dev)
        ws = B.new_workspace(B.OP_LINEAR, cfg.M, cfg.K, cfg.N, fmt, dev)
        want = B.linear(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, fmt, ws=ws)
        assert B.device_status(ws) == B.OK
        got = torch.full((cfg.M, cfg.N), float("nan"), dtype=torch.float32, device=dev)
        B.linear_static(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, fmt, out=got)
        # once more, now that the driver has loaded every kernel the call uses (it loads them lazily, on first launch):
        # the call itself takes no device memory (cudaMemGetInfo before and after)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        got.fill_(float("nan"))
        B.linear_static(L["X"], L["A"], L["b"], wq, wsc, c, cfg.N, fmt, out=got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.isfinite(got).all()
        # same kernels, same inputs: the tolerance of the layer tests (relative Frobenius 1e-4) is met with zero
        assert H.rel_fro(got.cpu().numpy(), want.double().cpu().numpy()) <= 1e-4
        assert torch.equal(got, want)


def test_static_scratch_refuses_sizes_beyond_its_limit(B):
    dev = torch.device("cuda")
    M, K, N = 8192, 8192, 64                      # 8192 x 8192 MXFP4 codes alone are 32 MiB
    assert B.workspace_bytes(B.OP_LINEAR, M, K, N, B.MXFP4) > B.STATIC_SCRATCH_BYTES
    X = torch.zeros(M, K, dtype=torch.bfloat16, device=dev)
    A = torch.zeros(16, dtype=torch.bfloat16, device=dev)      # never read: the call is refused before any launch
    wq, wsc = B.alloc_mx(N, K, B.MXFP4, B.SF_TCGEN05, dev)
    out = torch.zeros(M, N, dtype=torch.float32, device=dev)
    before = B.launch_count()
    with pytest.raises(B.LatmixError) as e:
        B.linear_static(X, A, None, wq, wsc, None, N, B.MXFP4, out=out)
    assert e.value.code == B.ERR_WORKSPACE
    assert B.launch_count() == before
