"""ctypes loader for the CPU oracle (``mxq_oracle.c``) -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only the tests, the smoke check and the benchmark's cpu-baseline leg may import this module.
It compiles ``mxq_oracle.c`` with gcc on first use (no CUDA, no torch) and exposes the C
functions on numpy arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxq_oracle.c")
_LIB = os.path.join(_HERE, "libmxq_oracle.so")

F32, BF16 = 0, 1
UE8M0, UE4M3, UE5M3 = 0, 1, 2
ABSMAX, ABSMAX_PZ, R4O6, R4O6_PZ, BRUTE, BRUTE_PZ, ABSMAX_OCP, ABSMAX_CLIP7 = range(8)

_CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-pthread"]


def build(force: bool = False) -> str:
    """Compile the oracle into ``libmxq_oracle.so`` next to its source; returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        # MXQ_ORACLE_LIB: load another build of the oracle (the tests plant mistakes in copies of the
        # C source to show that the pins notice them)
        L = ctypes.CDLL(os.environ.get("MXQ_ORACLE_LIB") or build())
        c = ctypes
        L.mxq_oracle_num_codes.restype = c.c_int
        L.mxq_oracle_num_codes.argtypes = [c.c_int]
        L.mxq_oracle_scale_value.restype = c.c_float
        L.mxq_oracle_scale_value.argtypes = [c.c_int, c.c_int]
        L.mxq_oracle_round_scale.restype = c.c_int
        L.mxq_oracle_round_scale.argtypes = [c.c_int, c.c_float]
        L.mxq_oracle_e2m1_index.restype = c.c_int
        L.mxq_oracle_e2m1_index.argtypes = [c.c_float]
        L.mxq_oracle_e2m1_value.restype = c.c_float
        L.mxq_oracle_e2m1_value.argtypes = [c.c_int]
        L.mxq_oracle_block_sse.restype = c.c_float
        L.mxq_oracle_block_sse.argtypes = [c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_float, c.c_void_p]
        L.mxq_oracle_quantize.restype = c.c_int
        L.mxq_oracle_quantize.argtypes = [c.c_void_p, c.c_int, c.c_size_t, c.c_int, c.c_int, c.c_int, c.c_float,
                                          c.c_void_p, c.c_void_p, c.c_void_p]
        L.mxq_oracle_quantize_mt.restype = c.c_int
        L.mxq_oracle_quantize_mt.argtypes = L.mxq_oracle_quantize.argtypes + [c.c_int]
        L.mxq_oracle_tensor_amax.restype = c.c_float
        L.mxq_oracle_tensor_amax.argtypes = [c.c_void_p, c.c_int, c.c_size_t]
        L.mxq_oracle_tensor_mse.restype = c.c_double
        L.mxq_oracle_tensor_mse.argtypes = [c.c_void_p, c.c_size_t, c.c_size_t]
        L.mxq_oracle_dequantize.restype = c.c_int
        L.mxq_oracle_dequantize.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_int, c.c_int, c.c_float,
                                            c.c_void_p, c.c_int]
        L.mxq_oracle_ocp_code.restype = c.c_int
        L.mxq_oracle_ocp_code.argtypes = [c.c_float, c.c_float]
        L.mxq_oracle_clip7_code.restype = c.c_int
        L.mxq_oracle_clip7_code.argtypes = [c.c_float, c.c_float]
        L.mxq_oracle_block_clip_sse.restype = c.c_int
        L.mxq_oracle_block_clip_sse.argtypes = [c.c_void_p, c.c_int, c.c_size_t, c.c_int, c.c_int, c.c_void_p, c.c_float,
                                                c.c_void_p]
        L.mxq_oracle_histograms.restype = c.c_int
        L.mxq_oracle_histograms.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_int, c.c_void_p, c.c_void_p]
        L.mxq_oracle_segment_mse.restype = c.c_int
        L.mxq_oracle_segment_mse.argtypes = [c.c_void_p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_void_p]
        _lib = L
    return _lib


def _as_input(x):
    """float32 array -> (array, F32); uint16 array of bf16 bit patterns -> (array, BF16)."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    raise TypeError("oracle input must be float32 or uint16 (bf16 bit patterns)")


def num_codes(fmt: int) -> int:
    return lib().mxq_oracle_num_codes(fmt)


def scale_value(fmt: int, code: int) -> float:
    return float(lib().mxq_oracle_scale_value(fmt, code))


def round_scale(fmt: int, w) -> int:
    return lib().mxq_oracle_round_scale(fmt, float(np.float32(w)))


def e2m1_index(t) -> int:
    return lib().mxq_oracle_e2m1_index(float(np.float32(t)))


def e2m1_value(code4: int) -> float:
    return float(lib().mxq_oracle_e2m1_value(code4))


def block_sse(v, fmt: int, code: int, g: float = 1.0):
    """SSE (float32) and the unpacked 4-bit codes of one block under one given scale code."""
    v = np.ascontiguousarray(v, dtype=np.float32)
    c4 = np.empty(v.size, dtype=np.uint8)
    s = lib().mxq_oracle_block_sse(v.ctypes.data, v.size, fmt, code, float(np.float32(g)), c4.ctypes.data)
    return np.float32(s), c4


def quantize(x, block_size: int, fmt: int, recipe: int, g: float = 1.0, threads: int = 1):
    """Returns (codes uint8[n/2], scales uint8[n/B], block_sse float32[n/B])."""
    x, dt = _as_input(x)
    n = x.size
    codes = np.empty(n // 2, dtype=np.uint8)
    scales = np.empty(n // block_size, dtype=np.uint8)
    sse = np.empty(n // block_size, dtype=np.float32)
    rc = lib().mxq_oracle_quantize_mt(x.ctypes.data, dt, n, block_size, fmt, recipe, float(np.float32(g)),
                                      codes.ctypes.data, scales.ctypes.data, sse.ctypes.data, int(threads))
    if rc != 0:
        raise ValueError("mxq_oracle_quantize: bad argument")
    return codes, scales, sse


def tensor_amax(x) -> np.float32:
    x, dt = _as_input(x)
    return np.float32(lib().mxq_oracle_tensor_amax(x.ctypes.data, dt, x.size))


def tensor_mse(block_sse_arr, n: int) -> float:
    s = np.ascontiguousarray(block_sse_arr, dtype=np.float32)
    return float(lib().mxq_oracle_tensor_mse(s.ctypes.data, s.size, n))


def dequantize(codes, scales, n: int, block_size: int, fmt: int, g: float = 1.0, out_dtype: int = F32):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    out = np.empty(n, dtype=np.float32 if out_dtype == F32 else np.uint16)
    rc = lib().mxq_oracle_dequantize(codes.ctypes.data, scales.ctypes.data, n, block_size, fmt,
                                     float(np.float32(g)), out.ctypes.data, out_dtype)
    if rc != 0:
        raise ValueError("mxq_oracle_dequantize: bad argument")
    return out


def global_scale_from_amax(amax) -> np.float32:
    """Hierarchical tensor scale g = amax / (6 * 448) in float32 (1 when the tensor is all zero)."""
    a = np.float32(amax)
    return np.float32(a / np.float32(2688.0)) if a > 0 else np.float32(1.0)


def block_clip_sse(x, scales, block_size: int, fmt: int, g: float = 1.0):
    """Per-block SSE of the elements clipped to +-6 (float32[n/B])."""
    x, dt = _as_input(x)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    out = np.empty(x.size // block_size, dtype=np.float32)
    rc = lib().mxq_oracle_block_clip_sse(x.ctypes.data, dt, x.size, block_size, fmt, scales.ctypes.data,
                                         float(np.float32(g)), out.ctypes.data)
    if rc != 0:
        raise ValueError("mxq_oracle_block_clip_sse: bad argument")
    return out


def histograms(codes, scales, n: int, block_size: int):
    """(code histogram uint64[16], scale-code histogram uint64[256])."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    ch = np.zeros(16, dtype=np.uint64)
    sh = np.zeros(256, dtype=np.uint64)
    rc = lib().mxq_oracle_histograms(codes.ctypes.data, scales.ctypes.data, n, block_size, ch.ctypes.data, sh.ctypes.data)
    if rc != 0:
        raise ValueError("mxq_oracle_histograms: bad argument")
    return ch, sh


def segment_mse(block_sse_arr, blocks_per_segment: int, elems_per_segment: int):
    s = np.ascontiguousarray(block_sse_arr, dtype=np.float32)
    out = np.empty(s.size // blocks_per_segment, dtype=np.float64)
    rc = lib().mxq_oracle_segment_mse(s.ctypes.data, s.size, blocks_per_segment, elems_per_segment, out.ctypes.data)
    if rc != 0:
        raise ValueError("mxq_oracle_segment_mse: bad argument")
    return out


def ocp_code(amax, g: float = 1.0) -> int:
    return lib().mxq_oracle_ocp_code(float(np.float32(amax)), float(np.float32(g)))


def clip7_code(amax, g: float = 1.0) -> int:
    return lib().mxq_oracle_clip7_code(float(np.float32(amax)), float(np.float32(g)))


def fake_quantize(x, block_size: int, fmt: int, recipe: int, g: float = 1.0, out_dtype: int = F32, threads: int = 1):
    """dequantize(quantize(x)): what a model sees when its weights or activations are quantized."""
    codes, scales, _ = quantize(x, block_size, fmt, recipe, g, threads)
    return dequantize(codes, scales, np.ascontiguousarray(x).size, block_size, fmt, g, out_dtype)


def mask_interval(x, lo: float, hi: float):
    """Magnitude-interval masking of the appendix ablation: entries with lo <= |x| < hi become zero
    (+0), all others pass unchanged.  x: float32 array or uint16 bf16 bit patterns; same type out."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        mag = (x.astype(np.uint32) << 16).view(np.float32)
        keep = ~((np.abs(mag) >= np.float32(lo)) & (np.abs(mag) < np.float32(hi)))
        return np.where(keep, x, np.uint16(0)).astype(np.uint16)
    keep = ~((np.abs(x) >= np.float32(lo)) & (np.abs(x) < np.float32(hi)))
    return np.where(keep, x, np.float32(0.0)).astype(np.float32)
