"""The failure path of the bounded device-side waits, taken without harming the GPU.

Every wait inside a kernel gives up after a limit, records LATMIX_ERR_TIMEOUT in the workspace's status word and lets
the kernel run to its end.  Here the limit is set to a fraction of a millisecond and one CTA of the single-CTA
block-scaled product is told (LATMIX_FLAG_TEST_DROP_LOAD) to leave out the loads of one K slab: it neither arms the
stage's barrier nor issues the copies, so the waits that depend on that slab expire while nothing of it is in flight.
No trap, no bad address, no unbounded loop: the kernel returns normally, the host reads the status, and the same
workspace serves an ordinary call afterwards."""
import numpy as np
import pytest
import torch

from oracle import latmix_oracle as orc
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_17681_b200 import binding
    return binding


def test_expired_wait_is_reported_and_the_workspace_stays_usable(B):
    M, K, N, fmt = 128, 1024, 512, B.MXFP4                 # 4 tiles of 128 x 128, four K slabs each
    ac, asc = H.random_mx(M, K, fmt, 91)
    wc, wsc = H.random_mx(N, K, fmt, 92)
    da, dsa = H.mx_to_device(B, ac, asc, fmt)
    dw, dsw = H.mx_to_device(B, wc, wsc, fmt)
    ws = B.new_workspace(B.OP_MX_GEMM, M, K, N, fmt)
    single_cta = 1 << 8
    good = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt, ws=ws, flags=single_cta).clone()
    assert B.device_status(ws) == B.OK

    # a short limit alone changes nothing: no wait of a healthy launch lasts that long
    B.workspace_set_wait_limit(ws, 200_000)
    again = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt, ws=ws, flags=single_cta)
    assert B.device_status(ws) == B.OK and torch.equal(again, good)

    # one slab of tile 0 never arrives: the call returns, the status word says which kind of problem it was
    out = torch.full((M, N), float("nan"), device="cuda")
    B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt, out=out, ws=ws, flags=single_cta | B.FLAG_TEST_DROP_LOAD)
    torch.cuda.synchronize()                                # the launch ends by itself
    assert B.device_status(ws) == B.ERR_TIMEOUT
    assert B.status_string(B.ERR_TIMEOUT) == "a bounded device-side wait expired"
    # the other tiles were computed by CTAs that met no problem; tile 0 was given up and never stored
    assert torch.isnan(out[:, :128]).all()
    assert torch.equal(out[:, 128:], good[:, 128:])
    # the status is sticky until the header is cleared
    assert B.device_status(ws) == B.ERR_TIMEOUT

    # after re-initialising the header the same workspace, buffers and context give the same bits as before
    B.workspace_init(ws)
    after = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt, ws=ws, flags=single_cta)
    assert B.device_status(ws) == B.OK
    assert torch.equal(after, good)
    ref = orc.mx_matmul(ac, asc, wc, wsc, None, "mxfp4")
    H.assert_gemm_parity(after.cpu().numpy(), ref, ac, asc, wc, wsc, "mxfp4", K, tag="after an expired wait")
    # and so does the default kernel choice on a fresh workspace
    other = B.mx_gemm(da, dsa, dw, dsw, None, M, K, N, fmt)
    assert torch.equal(other, good)
