"""Thin ctypes binding of libmxq (argument marshalling only; every step runs in the CUDA kernels).

The functions carry the names of the C-ABI declared in ``include/mxq.h`` and take torch CUDA
tensors (torch supplies device memory and streams, nothing else).  There is no CPU fallback: if
``libmxq.so`` is missing or a call is made without a CUDA device, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MXQ_LIB: path of another build of the library; the default is the in-tree build
LIB_PATH = os.environ.get("MXQ_LIB") or os.path.join(_HERE, "libmxq.so")

MXQ_F32, MXQ_BF16 = 0, 1
MXQ_SF_UE8M0, MXQ_SF_UE4M3, MXQ_SF_UE5M3 = 0, 1, 2
MXQ_ABSMAX, MXQ_ABSMAX_PZ, MXQ_4O6, MXQ_4O6_PZ, MXQ_BRUTE, MXQ_BRUTE_PZ, MXQ_ABSMAX_OCP, MXQ_ABSMAX_CLIP7 = range(8)
MXQ_OPT_BRUTE_PRUNE = 1

EXPORTS = (
    "mxq_quantize", "mxq_quantize_ex", "mxq_quantize_mse", "mxq_quantize_batch", "mxq_fake_quantize", "mxq_tensor_amax", "mxq_global_scale_from_amax",
    "mxq_tensor_mse_workspace_bytes", "mxq_tensor_mse", "mxq_tensor_mse_static", "mxq_dequantize", "mxq_dequantize_ex",
    "mxq_block_clip_sse", "mxq_histograms", "mxq_segment_mse", "mxq_mask_interval", "mxq_set_option", "mxq_get_option", "mxq_launch_count",
    "mxq_status_string", "mxq_last_cuda_error", "mxq_version",
)


class MxqError(RuntimeError):
    pass


class TensorDesc(ctypes.Structure):
    """mxq_tensor_desc of include/mxq.h (one tensor of a multi-tensor launch)."""
    _fields_ = [("x", ctypes.c_void_p), ("out_codes", ctypes.c_void_p), ("out_scales", ctypes.c_void_p),
                ("out_block_sse", ctypes.c_void_p), ("n", ctypes.c_size_t)]


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libmxq.so (built by ``paper_2605_08565_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise MxqError(f"{LIB_PATH} not found: build it with `python -m paper_2605_08565_b200.build` "
                       "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    c = ctypes
    vp, sz, i32, f32 = c.c_void_p, c.c_size_t, c.c_int, c.c_float
    L.mxq_quantize.restype = i32
    L.mxq_quantize.argtypes = [vp, sz, i32, i32, i32, f32, vp, vp, vp]
    L.mxq_quantize_ex.restype = i32
    L.mxq_quantize_ex.argtypes = [vp, i32, sz, i32, i32, i32, f32, vp, vp, vp, vp, vp]
    L.mxq_quantize_mse.restype = i32
    L.mxq_quantize_mse.argtypes = [vp, i32, sz, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.mxq_quantize_batch.restype = i32
    L.mxq_quantize_batch.argtypes = [vp, vp, sz, i32, i32, i32, i32, f32, vp, vp]
    L.mxq_fake_quantize.restype = i32
    L.mxq_fake_quantize.argtypes = [vp, i32, sz, i32, i32, i32, f32, vp, vp, i32, vp]
    L.mxq_tensor_amax.restype = i32
    L.mxq_tensor_amax.argtypes = [vp, i32, sz, vp, vp, vp]
    L.mxq_global_scale_from_amax.restype = f32
    L.mxq_global_scale_from_amax.argtypes = [f32]
    L.mxq_tensor_mse_workspace_bytes.restype = sz
    L.mxq_tensor_mse_workspace_bytes.argtypes = [sz]
    L.mxq_tensor_mse.restype = i32
    L.mxq_tensor_mse.argtypes = [vp, sz, sz, vp, vp, sz, vp]
    L.mxq_tensor_mse_static.restype = i32
    L.mxq_tensor_mse_static.argtypes = [vp, sz, sz, vp, vp]
    L.mxq_dequantize.restype = i32
    L.mxq_dequantize.argtypes = [vp, vp, sz, i32, i32, f32, vp, i32, vp]
    L.mxq_dequantize_ex.restype = i32
    L.mxq_dequantize_ex.argtypes = [vp, vp, sz, i32, i32, f32, vp, vp, i32, vp]
    L.mxq_block_clip_sse.restype = i32
    L.mxq_block_clip_sse.argtypes = [vp, i32, sz, i32, i32, f32, vp, vp, vp, vp]
    L.mxq_histograms.restype = i32
    L.mxq_histograms.argtypes = [vp, vp, sz, i32, vp, vp, vp]
    L.mxq_segment_mse.restype = i32
    L.mxq_segment_mse.argtypes = [vp, sz, sz, sz, vp, vp]
    L.mxq_mask_interval.restype = i32
    L.mxq_mask_interval.argtypes = [vp, i32, sz, f32, f32, vp, vp]
    L.mxq_set_option.restype = i32
    L.mxq_set_option.argtypes = [i32, i32]
    L.mxq_get_option.restype = i32
    L.mxq_get_option.argtypes = [i32, c.POINTER(c.c_int)]
    L.mxq_launch_count.restype = c.c_ulonglong
    L.mxq_launch_count.argtypes = []
    L.mxq_status_string.restype = c.c_char_p
    L.mxq_status_string.argtypes = [i32]
    L.mxq_last_cuda_error.restype = i32
    L.mxq_last_cuda_error.argtypes = []
    L.mxq_version.restype = i32
    L.mxq_version.argtypes = []
    _lib = L
    return L


def _check(status: int) -> None:
    if status != 0:
        L = load_library()
        msg = L.mxq_status_string(status).decode()
        if status == 7:
            msg += f" [cudaError {L.mxq_last_cuda_error()}]"
        raise MxqError(f"libmxq status {status}: {msg}")


def _ptr(t) -> int:
    if t is None:
        return 0
    if not t.is_cuda:
        raise MxqError("libmxq takes CUDA tensors only (no CPU fallback)")
    if not t.is_contiguous():
        raise MxqError("tensor must be contiguous")
    return t.data_ptr()


def _dtype_id(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return MXQ_F32
    if t.dtype == torch.bfloat16:
        return MXQ_BF16
    raise MxqError(f"unsupported dtype {t.dtype}")


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream, like=None) -> int:
    """cudaStream_t of `stream`, or of torch's current stream on the device of tensor `like`."""
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None and like is not None and like.is_cuda:
        return _raw_stream(like.device.index if like.device.index is not None else torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


# ---- C-ABI names ---------------------------------------------------------------------------
def mxq_quantize(x, n, block_size, scale_fmt, recipe, global_scale, out_codes, out_scales, out_block_sse) -> None:
    """float32 input, default stream (synchronises with torch's current stream by stream order
    only if that is the default stream)."""
    _check(load_library().mxq_quantize(_ptr(x), n, block_size, scale_fmt, recipe, global_scale,
                                       _ptr(out_codes), _ptr(out_scales), _ptr(out_block_sse)))


def mxq_quantize_ex(x, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, out_codes, out_scales,
                    out_block_sse, stream=None) -> None:
    _check(load_library().mxq_quantize_ex(_ptr(x), _dtype_id(x), n, block_size, scale_fmt, recipe, global_scale,
                                          _ptr(d_global_scale), _ptr(out_codes), _ptr(out_scales),
                                          _ptr(out_block_sse), _stream(stream, x)))


def mxq_quantize_mse(x, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, out_codes, out_scales,
                     out_block_sse, d_out_mse, d_workspace, stream=None) -> None:
    """Quantize and score in one call: the tensor MSE comes from partial sums formed inside the quantization kernel."""
    ws_bytes = d_workspace.numel() * d_workspace.element_size() if d_workspace is not None else 0
    _check(load_library().mxq_quantize_mse(_ptr(x), _dtype_id(x), n, block_size, scale_fmt, recipe, global_scale,
                                           _ptr(d_global_scale), _ptr(out_codes), _ptr(out_scales), _ptr(out_block_sse),
                                           _ptr(d_out_mse), _ptr(d_workspace), ws_bytes, _stream(stream, x)))


def make_tensor_descs(items):
    """Descriptor arrays for ``mxq_quantize_batch``: items = [(x, out_codes, out_scales, out_block_sse or None), ...]
    (flat CUDA tensors of one dtype on one device).  Returns (host ctypes array, device uint8 tensor holding
    the same bytes); both must be kept alive until the launch that uses them has run."""
    if not items:
        raise MxqError("empty tensor list")
    arr = (TensorDesc * len(items))()
    for d, (x, codes, scales, sse) in zip(arr, items):
        d.x, d.out_codes, d.out_scales, d.out_block_sse, d.n = _ptr(x), _ptr(codes), _ptr(scales), _ptr(sse), x.numel()
    host = torch.frombuffer(bytearray(bytes(arr)), dtype=torch.uint8)
    return arr, host.to(items[0][0].device)


def mxq_quantize_batch(h_descs, d_descs, n_tensors, dtype_id, block_size, scale_fmt, recipe, global_scale=1.0,
                       d_global_scale=None, stream=None) -> None:
    """One launch over a list of tensors; h_descs / d_descs from ``make_tensor_descs``."""
    _check(load_library().mxq_quantize_batch(ctypes.addressof(h_descs), _ptr(d_descs), n_tensors, dtype_id, block_size,
                                             scale_fmt, recipe, global_scale, _ptr(d_global_scale),
                                             _stream(stream, d_descs)))


def mxq_fake_quantize(x, n, block_size, scale_fmt, recipe, global_scale, d_global_scale, d_out, stream=None) -> None:
    _check(load_library().mxq_fake_quantize(_ptr(x), _dtype_id(x), n, block_size, scale_fmt, recipe, global_scale,
                                            _ptr(d_global_scale), _ptr(d_out), _dtype_id(d_out), _stream(stream, x)))


def mxq_tensor_amax(x, n, d_out_amax, d_out_global_scale=None, stream=None) -> None:
    _check(load_library().mxq_tensor_amax(_ptr(x), _dtype_id(x), n, _ptr(d_out_amax), _ptr(d_out_global_scale),
                                          _stream(stream, x)))


def mxq_global_scale_from_amax(amax: float) -> float:
    return float(load_library().mxq_global_scale_from_amax(amax))


def mxq_tensor_mse_workspace_bytes(n_blocks: int) -> int:
    return int(load_library().mxq_tensor_mse_workspace_bytes(n_blocks))


def mxq_tensor_mse(d_block_sse, n_blocks, n, d_out_mse, d_workspace, stream=None) -> None:
    ws_bytes = d_workspace.numel() * d_workspace.element_size() if d_workspace is not None else 0
    _check(load_library().mxq_tensor_mse(_ptr(d_block_sse), n_blocks, n, _ptr(d_out_mse), _ptr(d_workspace),
                                         ws_bytes, _stream(stream, d_block_sse)))


def mxq_tensor_mse_static(d_block_sse, n_blocks, n, d_out_mse, stream=None) -> None:
    """Tensor MSE with the library's built-in scratch array: no workspace argument, nothing allocated."""
    _check(load_library().mxq_tensor_mse_static(_ptr(d_block_sse), n_blocks, n, _ptr(d_out_mse), _stream(stream, d_block_sse)))


def mxq_dequantize(d_codes, d_scales, n, block_size, scale_fmt, global_scale, d_out, stream=None) -> None:
    _check(load_library().mxq_dequantize(_ptr(d_codes), _ptr(d_scales), n, block_size, scale_fmt, global_scale,
                                         _ptr(d_out), _dtype_id(d_out), _stream(stream, d_out)))


def mxq_dequantize_ex(d_codes, d_scales, n, block_size, scale_fmt, global_scale, d_global_scale, d_out, stream=None) -> None:
    _check(load_library().mxq_dequantize_ex(_ptr(d_codes), _ptr(d_scales), n, block_size, scale_fmt, global_scale,
                                            _ptr(d_global_scale), _ptr(d_out), _dtype_id(d_out), _stream(stream, d_out)))


def mxq_block_clip_sse(x, n, block_size, scale_fmt, global_scale, d_global_scale, d_scales, out_clip_sse,
                       stream=None) -> None:
    _check(load_library().mxq_block_clip_sse(_ptr(x), _dtype_id(x), n, block_size, scale_fmt, global_scale,
                                             _ptr(d_global_scale), _ptr(d_scales), _ptr(out_clip_sse), _stream(stream, x)))


def mxq_histograms(d_codes, d_scales, n, block_size, d_code_hist, d_scale_hist, stream=None) -> None:
    """d_code_hist: 16 and d_scale_hist: 256 int64/uint64 CUDA counters; counts are added to them."""
    _check(load_library().mxq_histograms(_ptr(d_codes), _ptr(d_scales), n, block_size, _ptr(d_code_hist),
                                         _ptr(d_scale_hist), _stream(stream, d_codes)))


def mxq_segment_mse(d_block_sse, n_blocks, blocks_per_segment, elems_per_segment, d_out_mse, stream=None) -> None:
    _check(load_library().mxq_segment_mse(_ptr(d_block_sse), n_blocks, blocks_per_segment, elems_per_segment,
                                          _ptr(d_out_mse), _stream(stream, d_block_sse)))


def mxq_mask_interval(x, n, lo, hi, d_out, stream=None) -> None:
    _check(load_library().mxq_mask_interval(_ptr(x), _dtype_id(x), n, lo, hi, _ptr(d_out), _stream(stream, x)))


def mxq_set_option(option: int, value: int) -> None:
    _check(load_library().mxq_set_option(int(option), int(value)))


def mxq_get_option(option: int) -> int:
    out = ctypes.c_int(0)
    _check(load_library().mxq_get_option(int(option), ctypes.byref(out)))
    return int(out.value)


def mxq_launch_count() -> int:
    return int(load_library().mxq_launch_count())


def mxq_version() -> int:
    return int(load_library().mxq_version())


# ---- convenience: allocate outputs with torch, then call the C-ABI -----------------------------
def alloc_outputs(n: int, block_size: int, device, with_sse: bool = True):
    codes = torch.empty(n // 2, dtype=torch.uint8, device=device)
    scales = torch.empty(n // block_size, dtype=torch.uint8, device=device)
    sse = torch.empty(n // block_size, dtype=torch.float32, device=device) if with_sse else None
    return codes, scales, sse


def quantize(x: torch.Tensor, block_size: int, scale_fmt: int, recipe: int, global_scale: float = 1.0,
             d_global_scale=None, with_sse: bool = True, stream=None):
    """Allocates (codes, scales, block_sse) and runs mxq_quantize_ex on the flat tensor."""
    x = x.reshape(-1)
    codes, scales, sse = alloc_outputs(x.numel(), block_size, x.device, with_sse)
    mxq_quantize_ex(x, x.numel(), block_size, scale_fmt, recipe, global_scale, d_global_scale, codes, scales, sse,
                    stream)
    return codes, scales, sse


def tensor_mse(block_sse: torch.Tensor, n: int, stream=None) -> torch.Tensor:
    ws = torch.empty(mxq_tensor_mse_workspace_bytes(block_sse.numel()) // 8, dtype=torch.float64,
                     device=block_sse.device)
    out = torch.empty(1, dtype=torch.float64, device=block_sse.device)
    mxq_tensor_mse(block_sse, block_sse.numel(), n, out, ws, stream)
    return out
