"""ctypes binding of liblatmix.so: the same calls as include/latmix.h, taking torch CUDA tensors.

Argument marshalling only -- every step of the path runs inside the library's kernels.  PyTorch is used
for device memory and the current stream.  There is no fallback: if the library is missing, importing
this module raises; if the device is not sm_100 the library returns an error that is raised here.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblatmix.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2602_17681_b200.build` "
                      "(there is no CPU or PyTorch fallback)")
_lib = ctypes.CDLL(LIB_PATH)

# enums of include/latmix.h
OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = range(8)
MXFP4, MXFP8, MXINT8, MXINT4, NVFP4 = 0, 1, 2, 3, 4
F32, BF16 = 0, 1
SF_LINEAR, SF_TCGEN05 = 0, 1
OP_FOLD_WEIGHTS, OP_QUANTIZE_MX, OP_LINEAR, OP_MX_GEMM, OP_FOLD_TWO_SIDED, OP_TRANSFORMATION_MSE = 0, 1, 2, 3, 4, 5
FLAG_NONE, FLAG_CHECK_FINITE, FLAG_FORCE_SIMT, FLAG_BLOCK_DIAG = 0, 1, 2, 4
FLAG_TEST_DROP_LOAD = 1 << 16
FORMATS = {"mxfp4": MXFP4, "mxfp8": MXFP8, "mxint8": MXINT8, "mxint4": MXINT4, "nvfp4": NVFP4}

_vp, _i64, _sz, _u32, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_uint32, ctypes.c_int
_szp = ctypes.POINTER(ctypes.c_size_t)

EXPORTS = {
    "latmix_mx_sizes": (_int, [_i64, _i64, _int, _int, _szp, _szp]),
    "latmix_scale_offset": (_sz, [_i64, _i64, _i64, _i64, _int]),
    "latmix_scale_offset_fmt": (_sz, [_i64, _i64, _i64, _i64, _int, _int]),
    "latmix_tensor_scale_offset": (_sz, [_i64, _i64, _int, _int]),
    "latmix_workspace_set_tensor_scale": (_int, [_vp, _sz, ctypes.c_float, _vp]),
    "latmix_workspace_bytes": (_int, [_int, _i64, _i64, _i64, _int, _szp]),
    "latmix_status_string": (ctypes.c_char_p, [_int]),
    "latmix_launch_count": (ctypes.c_uint64, []),
    "latmix_fold_weights": (_int, [_vp, _vp, _vp, _int, _vp, _i64, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp, _sz, _u32, _vp]),
    "latmix_fold_weights_two_sided": (_int, [_vp, _vp, _vp, _int, _vp, _vp, _vp, _i64, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp,
                                             _sz, _u32, _vp]),
    "latmix_quantize_mx": (_int, [_vp, _int, _vp, _vp, _i64, _i64, _int, _int, _vp, _vp, _vp, _vp, _sz, _u32, _vp]),
    "latmix_transformation_mse": (_int, [_vp, _int, _vp, _vp, _vp, _i64, _i64, _int, _vp, _vp, _vp, _sz, _u32, _vp]),
    "latmix_transformation_mse_block": (_int, [_vp, _int, _vp, _vp, _vp, _i64, _i64, _int, _int, _vp, _vp, _vp, _sz, _u32, _vp]),
    "latmix_mx_gemm": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _i64, _vp, _sz, _u32, _vp]),
    "latmix_linear": (_int, [_vp, _int, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _i64, _vp, _sz, _u32, _vp]),
    "latmix_linear_static": (_int, [_vp, _int, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _i64, _u32,
                                    ctypes.POINTER(ctypes.c_int), _vp]),
    "latmix_tensor_pipe_probe": (_int, [_int, _i64, ctypes.POINTER(ctypes.c_double), _vp, _sz, _vp]),
    "latmix_workspace_init": (_int, [_vp, _sz, _vp]),
    "latmix_workspace_set_wait_limit": (_int, [_vp, _sz, _u32, _vp]),
    "latmix_device_status": (_int, [_vp, _vp]),
}
for _name, (_res, _args) in EXPORTS.items():
    _f = getattr(_lib, _name)
    _f.restype, _f.argtypes = _res, _args


class LatmixError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def status_string(code):
    return _lib.latmix_status_string(int(code)).decode()


def _check(code, where):
    if code != OK:
        raise LatmixError(code, where)


def _ptr(t, rows_strided=False):
    if t is None:
        return None
    assert t.is_cuda, "device tensors must be CUDA tensors"
    if rows_strided:
        assert t.dim() == 2 and t.stride(1) == 1, "output must be row-major with unit column stride"
    else:
        assert t.is_contiguous(), "device tensors must be contiguous"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _dtype(t):
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def mx_sizes(rows, K, fmt, sf=SF_TCGEN05):
    cb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    _check(_lib.latmix_mx_sizes(rows, K, fmt, sf, ctypes.byref(cb), ctypes.byref(sb)), "latmix_mx_sizes")
    return cb.value, sb.value


def scale_offset(row, kblock, rows, K, sf=SF_TCGEN05):
    return _lib.latmix_scale_offset(row, kblock, rows, K, sf)


def scale_offset_fmt(row, kblock, rows, K, fmt, sf=SF_TCGEN05):
    return _lib.latmix_scale_offset_fmt(row, kblock, rows, K, fmt, sf)


def tensor_scale_offset(rows, K, fmt, sf=SF_TCGEN05):
    return _lib.latmix_tensor_scale_offset(rows, K, fmt, sf)


def set_tensor_scale(scales, rows, K, fmt, sf, value):
    """NVFP4: write the tensor's fp32 scale into the trailer of a scale buffer (a device-side copy on the current stream)."""
    off = tensor_scale_offset(rows, K, fmt, sf)
    assert off != ctypes.c_size_t(-1).value
    scales[off:off + 4].view(torch.float32).fill_(float(value))


def workspace_set_tensor_scale(ws, value):
    _check(_lib.latmix_workspace_set_tensor_scale(_ptr(ws), ws.numel(), float(value), _stream()), "latmix_workspace_set_tensor_scale")


def workspace_bytes(op, M, K, N, fmt):
    n = ctypes.c_size_t()
    _check(_lib.latmix_workspace_bytes(op, M, K, N, fmt, ctypes.byref(n)), "latmix_workspace_bytes")
    return n.value


def launch_count():
    return int(_lib.latmix_launch_count())


def new_workspace(op, M, K, N, fmt, device="cuda"):
    """Allocate and initialise a workspace tensor (uint8) for the given call."""
    ws = torch.empty(workspace_bytes(op, M, K, N, fmt), dtype=torch.uint8, device=device)
    _check(_lib.latmix_workspace_init(_ptr(ws), ws.numel(), _stream()), "latmix_workspace_init")
    return ws


def workspace_init(ws):
    _check(_lib.latmix_workspace_init(_ptr(ws), ws.numel(), _stream()), "latmix_workspace_init")


def workspace_set_wait_limit(ws, cycles):
    _check(_lib.latmix_workspace_set_wait_limit(_ptr(ws), ws.numel(), cycles, _stream()), "latmix_workspace_set_wait_limit")


def device_status(ws):
    return _lib.latmix_device_status(_ptr(ws), _stream())


def alloc_mx(rows, K, fmt, sf=SF_TCGEN05, device="cuda"):
    cb, sb = mx_sizes(rows, K, fmt, sf)
    return (torch.empty(max(cb, 16), dtype=torch.uint8, device=device),
            torch.empty(max(sb, 16), dtype=torch.uint8, device=device))


def fold_weights(A_inv, b, W, bias, fmt, sf=SF_TCGEN05, dump=False, ws=None, flags=0, tensor_scale=None):
    """-> (Wq_codes, Wq_scales, c, W~^T dump or None).  W is K x N; codes are N x K (K-major).  NVFP4: tensor_scale is
    written into the new scale buffer's trailer before the call."""
    K, N = W.shape
    codes, scales = alloc_mx(N, K, fmt, sf, W.device)
    if tensor_scale is not None:
        set_tensor_scale(scales, N, K, fmt, sf, tensor_scale)
    c = torch.empty(N, dtype=torch.float32, device=W.device)
    dumped = torch.empty(N, K, dtype=torch.float32, device=W.device) if dump else None
    ws = new_workspace(OP_FOLD_WEIGHTS, 0, K, N, fmt, W.device) if ws is None else ws
    _check(_lib.latmix_fold_weights(_ptr(A_inv), _ptr(b), _ptr(W), _dtype(W), _ptr(bias), K, N, fmt, sf, _ptr(codes),
                                    _ptr(scales), _ptr(c), _ptr(dumped), _ptr(ws), ws.numel(), flags, _stream()),
           "latmix_fold_weights")
    return codes, scales, c, dumped


def fold_weights_two_sided(A_in_inv, b_in, W, bias, A_out, v_out, fmt, sf=SF_TCGEN05, dump=False, ws=None, flags=0):
    """-> (Wq_codes, Wq_scales, c, W~~^T dump or None) for W~~ = A_in_inv W A_out; either side may be None."""
    K, N = W.shape
    codes, scales = alloc_mx(N, K, fmt, sf, W.device)
    c = torch.empty(N, dtype=torch.float32, device=W.device)
    dumped = torch.empty(N, K, dtype=torch.float32, device=W.device) if dump else None
    ws = new_workspace(OP_FOLD_TWO_SIDED, 0, K, N, fmt, W.device) if ws is None else ws
    _check(_lib.latmix_fold_weights_two_sided(_ptr(A_in_inv), _ptr(b_in), _ptr(W), _dtype(W), _ptr(bias), _ptr(A_out),
                                              _ptr(v_out), K, N, fmt, sf, _ptr(codes), _ptr(scales), _ptr(c), _ptr(dumped),
                                              _ptr(ws), ws.numel(), flags, _stream()), "latmix_fold_weights_two_sided")
    return codes, scales, c, dumped


def quantize_mx(X, A, b, fmt, sf=SF_TCGEN05, dump=False, ws=None, flags=0, out=None, tensor_scale=None):
    """-> (codes, scales, Y dump or None) = Q(X A + b); A None = identity.  NVFP4: tensor_scale is written into the scale
    buffer's trailer before the call (leave it None if the buffer passed in `out` already carries it)."""
    M, K = X.shape
    codes, scales = alloc_mx(M, K, fmt, sf, X.device) if out is None else out
    if tensor_scale is not None:
        set_tensor_scale(scales, M, K, fmt, sf, tensor_scale)
    dumped = torch.empty(M, K, dtype=torch.float32, device=X.device) if dump else None
    ws = new_workspace(OP_QUANTIZE_MX, M, K, 0, fmt, X.device) if ws is None else ws
    _check(_lib.latmix_quantize_mx(_ptr(X), _dtype(X), _ptr(A), _ptr(b), M, K, fmt, sf, _ptr(codes), _ptr(scales),
                                   _ptr(dumped), _ptr(ws), ws.numel(), flags, _stream()), "latmix_quantize_mx")
    return codes, scales, dumped


def transformation_mse(X, A, b, A_inv, fmt, ws=None, flags=0, block=32):
    """-> (E(T) as a 0-d float64 tensor, block-wise error as K/block float64) for T(x) = x A + b; A None = identity."""
    M, K = X.shape
    block_err = torch.empty(K // block, dtype=torch.float64, device=X.device)
    mse = torch.empty((), dtype=torch.float64, device=X.device)
    ws = new_workspace(OP_TRANSFORMATION_MSE, M, K, 0, fmt, X.device) if ws is None else ws
    if block == 32:
        _check(_lib.latmix_transformation_mse(_ptr(X), _dtype(X), _ptr(A), _ptr(b), _ptr(A_inv), M, K, fmt, _ptr(block_err), _ptr(mse),
                                              _ptr(ws), ws.numel(), flags, _stream()), "latmix_transformation_mse")
    else:
        _check(_lib.latmix_transformation_mse_block(_ptr(X), _dtype(X), _ptr(A), _ptr(b), _ptr(A_inv), M, K, fmt, block,
                                                    _ptr(block_err), _ptr(mse), _ptr(ws), ws.numel(), flags, _stream()),
               "latmix_transformation_mse_block")
    return mse, block_err


def mx_gemm(a_codes, a_scales, w_codes, w_scales, c, M, K, N, fmt, out=None, ws=None, flags=0):
    out = torch.empty(M, N, dtype=torch.float32, device=a_codes.device) if out is None else out
    ws = new_workspace(OP_MX_GEMM, M, K, N, fmt, a_codes.device) if ws is None else ws
    _check(_lib.latmix_mx_gemm(_ptr(a_codes), _ptr(a_scales), _ptr(w_codes), _ptr(w_scales), _ptr(c), M, K, N, fmt,
                               _ptr(out, True), out.stride(0), _ptr(ws), ws.numel(), flags, _stream()),
           "latmix_mx_gemm")
    return out


def linear(X, A, b, Wq_codes, Wq_scales, c, N, fmt, out=None, ws=None, flags=0):
    """out[M x N] = Q(X A + b) Wq + c -- the whole forward path."""
    M, K = X.shape
    out = torch.empty(M, N, dtype=torch.float32, device=X.device) if out is None else out
    ws = new_workspace(OP_LINEAR, M, K, N, fmt, X.device) if ws is None else ws
    _check(_lib.latmix_linear(_ptr(X), _dtype(X), _ptr(A), _ptr(b), _ptr(Wq_codes), _ptr(Wq_scales), _ptr(c), M, K, N, fmt,
                              _ptr(out, True), out.stride(0), _ptr(ws), ws.numel(), flags, _stream()), "latmix_linear")
    return out


PIPE_KINDS = {"bf16": 0, "mxf8": 1, "mxf4": 2, "nvf4": 3, "mxf4_pair": 4}


def tensor_pipe_probe(kind, ws, mma_per_cta=28672, commit_every=0):
    """TFLOP/s of back-to-back MMAs of the given kind on every SM (latmix_tensor_pipe_probe timed with two events)."""
    flops = ctypes.c_double()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    _check(_lib.latmix_tensor_pipe_probe(PIPE_KINDS[kind] | (commit_every << 8), mma_per_cta, ctypes.byref(flops), _ptr(ws), ws.numel(), _stream()),
           "latmix_tensor_pipe_probe")
    ev1.record()
    ev1.synchronize()
    _check(device_status(ws), "latmix_tensor_pipe_probe (device status)")
    return flops.value / (ev0.elapsed_time(ev1) * 1e-3) / 1e12


STATIC_SCRATCH_BYTES = 256 + (16 << 20)     # LATMIX_STATIC_SCRATCH_BYTES of include/latmix.h


def linear_static(X, A, b, Wq_codes, Wq_scales, c, N, fmt, out, flags=0, wait=True):
    """latmix_linear_static: the whole layer with the library's built-in scratch instead of a workspace.

    For callers that must not allocate: `out` is required (this wrapper allocates nothing either).  With
    wait=True the call waits for the stream and raises if the device reported a problem; returns `out`.
    Sizes beyond STATIC_SCRATCH_BYTES of scratch raise LatmixError(ERR_WORKSPACE).  Calls on one device share
    the scratch: do not let two of them overlap on the GPU."""
    M, K = X.shape
    dev_status = ctypes.c_int(OK)
    _check(_lib.latmix_linear_static(_ptr(X), _dtype(X), _ptr(A), _ptr(b), _ptr(Wq_codes), _ptr(Wq_scales), _ptr(c), M, K, N,
                                     fmt, _ptr(out, True), out.stride(0), flags,
                                     ctypes.byref(dev_status) if wait else None, _stream()), "latmix_linear_static")
    _check(dev_status.value, "latmix_linear_static (device status)")
    return out
