"""CPU oracle for the block-rotated MXFP4 linear layer — TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``bro_ref.c`` (plain C, fp32 rotation in a fixed operation order, fp64
GEMM).  Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package; the CUDA library never does, and the two share no code.

All arrays are numpy: bf16 tensors are passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libbro_ref.so")
_SRC = [os.path.join(_HERE, "bro_ref.c")]
_HDR = [os.path.join(_HERE, "bro_ref.h")]
_lib = None

MX_GROUP = 32


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    newest = max(os.path.getmtime(p) for p in _SRC + _HDR)
    if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= newest:
        return _SO
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-shared", "-fPIC", "-Wall", "-Wextra", "-o", _SO] + _SRC + ["-lm"]
    subprocess.run(cmd, check=True)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_SO)
        i64, p, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.bro_ref_num_threads.restype = ci
        L.bro_ref_set_num_threads.argtypes = [ci]
        L.bro_ref_hadamard_norm.restype = ctypes.c_float
        L.bro_ref_hadamard_norm.argtypes = [i64]
        L.bro_ref_rotate.argtypes = [p, i64, i64, i64, ci, p]
        L.bro_ref_rotate_rs.argtypes = [p, i64, i64, i64, ci, p, p]
        L.bro_ref_rotate_quantize_mxfp4_rs.argtypes = [p, i64, i64, i64, ci, p, p, p]
        L.bro_ref_quantize.argtypes = [p, i64, i64, p, p]
        L.bro_ref_decode.argtypes = [p, p, i64, i64, p]
        L.bro_ref_rotate_quantize_mxfp4.argtypes = [p, i64, i64, i64, ci, p, p]
        L.bro_ref_pack_weights.argtypes = [p, i64, i64, i64, ci, p, p]
        L.bro_ref_gemm_mxfp4.argtypes = [p, p, p, p, i64, i64, i64, p, p]
        L.bro_ref_gemm_mxfp4_points.argtypes = [p, p, p, p, i64, i64, i64, p, p, i64, p, p]
        L.bro_ref_linear.argtypes = [p, i64, i64, i64, ci, p, p, i64, p, p]
        L.bro_ref_group_mse.argtypes = [p, p, p, i64, i64, p]
        L.bro_ref_fake_quantize.argtypes = [p, i64, i64, ci, p]
        L.bro_ref_fake_quantize.restype = ci
        L.bro_ref_swiglu_f32.argtypes = [p, p, i64, p]
        L.bro_ref_swiglu_f32.restype = ci
        L.bro_ref_swiglu.argtypes = [p, p, i64, i64, i64, i64, p]
        L.bro_ref_swiglu.restype = ci
        L.bro_ref_swiglu_rotate_quantize_mxfp4.argtypes = [p, p, i64, i64, i64, i64, ci, p, p, p]
        L.bro_ref_swiglu_rotate_quantize_mxfp4.restype = ci
        L.bro_ref_outlier_groups.argtypes = [p, i64, i64, i64, i64, p, p]
        L.bro_ref_outlier_groups.restype = ci
        L.bro_ref_scale_histogram.argtypes = [p, p, i64, p]
        L.bro_ref_scale_histogram.restype = ci
        L.bro_ref_scale_inflation.argtypes = [p, p, p, i64, p]
        L.bro_ref_scale_inflation.restype = ci
        for name in ("rotate_rs", "rotate_quantize_mxfp4_rs", "rotate", "quantize", "decode", "rotate_quantize_mxfp4", "pack_weights",
                     "gemm_mxfp4", "gemm_mxfp4_points", "linear", "group_mse"):
            getattr(L, "bro_ref_" + name).restype = ci
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"bro_ref_{what} failed with code {rc}")


def _as_bf16_bits(x) -> np.ndarray:
    a = np.ascontiguousarray(x)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed to the oracle as uint16 bit patterns")
    if a.ndim != 2:
        raise ValueError("expected a 2-D array")
    return a


def num_threads() -> int:
    return int(lib().bro_ref_num_threads())


def set_num_threads(n: int) -> None:
    lib().bro_ref_set_num_threads(int(n))


def hadamard_norm(block: int) -> np.float32:
    return np.float32(lib().bro_ref_hadamard_norm(int(block)))


def _signs(signs_bits, K: int):
    if signs_bits is None:
        return None
    s = np.ascontiguousarray(signs_bits)
    if s.dtype != np.uint16 or s.shape != (K,):
        raise TypeError("signs are passed as a uint16 [K] array of bf16 bit patterns (+1 / -1)")
    return s


def rotate(x_bits, block: int, signs_bits=None) -> np.ndarray:
    """Rotation only.  ``signs_bits`` ([K] bf16 bit patterns of +-1) selects the randomised form
    R_i = diag(s) H / sqrt(block); None is the plain normalised Hadamard."""
    x = _as_bf16_bits(x_bits)
    M, K = x.shape
    y = np.empty((M, K), dtype=np.float32)
    s = _signs(signs_bits, K)
    _check(lib().bro_ref_rotate_rs(_ptr(x), M, K, K, int(block), None if s is None else _ptr(s),
                                   _ptr(y)), "rotate_rs")
    return y


def quantize(y) -> tuple[np.ndarray, np.ndarray]:
    y = np.ascontiguousarray(y, dtype=np.float32)
    rows, K = y.shape
    codes = np.empty((rows, K // 2), dtype=np.uint8)
    scales = np.empty((rows, K // MX_GROUP), dtype=np.uint8)
    _check(lib().bro_ref_quantize(_ptr(y), rows, K, _ptr(codes), _ptr(scales)), "quantize")
    return codes, scales


def decode(codes, scales) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, K), dtype=np.float64)
    _check(lib().bro_ref_decode(_ptr(codes), _ptr(scales), rows, K, _ptr(out)), "decode")
    return out


def rotate_quantize_mxfp4(x_bits, block: int, signs_bits=None) -> tuple[np.ndarray, np.ndarray]:
    x = _as_bf16_bits(x_bits)
    M, K = x.shape
    codes = np.empty((M, K // 2), dtype=np.uint8)
    scales = np.empty((M, K // MX_GROUP), dtype=np.uint8)
    s = _signs(signs_bits, K)
    _check(lib().bro_ref_rotate_quantize_mxfp4_rs(_ptr(x), M, K, K, int(block),
                                                  None if s is None else _ptr(s), _ptr(codes),
                                                  _ptr(scales)), "rotate_quantize_mxfp4_rs")
    return codes, scales


def pack_weights(w_bits, block: int, signs_bits=None) -> tuple[np.ndarray, np.ndarray]:
    if signs_bits is not None:           # the same arithmetic on the rows of W, same sign vector
        return rotate_quantize_mxfp4(w_bits, block, signs_bits)
    w = _as_bf16_bits(w_bits)
    N, K = w.shape
    codes = np.empty((N, K // 2), dtype=np.uint8)
    scales = np.empty((N, K // MX_GROUP), dtype=np.uint8)
    _check(lib().bro_ref_pack_weights(_ptr(w), N, K, K, int(block), _ptr(codes), _ptr(scales)),
           "pack_weights")
    return codes, scales


def gemm_mxfp4(acodes, ascales, wcodes, wscales) -> tuple[np.ndarray, np.ndarray]:
    acodes = np.ascontiguousarray(acodes, dtype=np.uint8)
    ascales = np.ascontiguousarray(ascales, dtype=np.uint8)
    wcodes = np.ascontiguousarray(wcodes, dtype=np.uint8)
    wscales = np.ascontiguousarray(wscales, dtype=np.uint8)
    M, K = acodes.shape[0], acodes.shape[1] * 2
    N = wcodes.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    _check(lib().bro_ref_gemm_mxfp4(_ptr(acodes), _ptr(ascales), _ptr(wcodes), _ptr(wscales),
                                    M, N, K, _ptr(y), _ptr(S)), "gemm_mxfp4")
    return y, S


def gemm_mxfp4_points(acodes, ascales, wcodes, wscales, pm, pn) -> tuple[np.ndarray, np.ndarray]:
    acodes = np.ascontiguousarray(acodes, dtype=np.uint8)
    ascales = np.ascontiguousarray(ascales, dtype=np.uint8)
    wcodes = np.ascontiguousarray(wcodes, dtype=np.uint8)
    wscales = np.ascontiguousarray(wscales, dtype=np.uint8)
    pm = np.ascontiguousarray(pm, dtype=np.int64)
    pn = np.ascontiguousarray(pn, dtype=np.int64)
    M, K = acodes.shape[0], acodes.shape[1] * 2
    N = wcodes.shape[0]
    y = np.empty(pm.shape[0], dtype=np.float64)
    S = np.empty(pm.shape[0], dtype=np.float64)
    _check(lib().bro_ref_gemm_mxfp4_points(_ptr(acodes), _ptr(ascales), _ptr(wcodes),
                                           _ptr(wscales), M, N, K, _ptr(pm), _ptr(pn),
                                           pm.shape[0], _ptr(y), _ptr(S)), "gemm_mxfp4_points")
    return y, S


def linear(x_bits, block: int, wcodes, wscales, signs_bits=None) -> tuple[np.ndarray, np.ndarray]:
    if signs_bits is not None:
        ac, asc = rotate_quantize_mxfp4(x_bits, block, signs_bits)
        return gemm_mxfp4(ac, asc, wcodes, wscales)
    x = _as_bf16_bits(x_bits)
    wcodes = np.ascontiguousarray(wcodes, dtype=np.uint8)
    wscales = np.ascontiguousarray(wscales, dtype=np.uint8)
    M, K = x.shape
    N = wcodes.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    _check(lib().bro_ref_linear(_ptr(x), M, K, K, int(block), _ptr(wcodes), _ptr(wscales), N,
                                _ptr(y), _ptr(S)), "linear")
    return y, S


def group_mse(y, codes, scales) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, K = y.shape
    mse = np.empty((rows, K // MX_GROUP), dtype=np.float64)
    _check(lib().bro_ref_group_mse(_ptr(y), _ptr(codes), _ptr(scales), rows, K, _ptr(mse)),
           "group_mse")
    return mse


FORMATS = {"mxfp4": 0, "bfp4": 1, "mxint4": 2, "bint4": 3, "int4_row_sym": 4, "int4_row_asym": 5}


def fake_quantize(y, fmt) -> np.ndarray:
    """Dequantised values (fp64) of fp32 rows under one of the compared 4-bit formats."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    rows, K = y.shape
    out = np.empty((rows, K), dtype=np.float64)
    f = FORMATS[fmt] if isinstance(fmt, str) else int(fmt)
    _check(lib().bro_ref_fake_quantize(_ptr(y), rows, K, f, _ptr(out)), "fake_quantize")
    return out


def group_error(y, fmt) -> np.ndarray:
    """mean_i (y_i - deq_i)^2 per group of 32, fp64, for any of the compared formats."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    d = y.astype(np.float64) - fake_quantize(y, fmt)
    return (d * d).reshape(y.shape[0], y.shape[1] // MX_GROUP, MX_GROUP).mean(-1)


def group_scale_bytes(x_bits, block: int, signs_bits=None) -> np.ndarray:
    """E8M0 scale byte of every MX group of x R_block ([M, K/32]); block = 1 is the identity rotation,
    i.e. the scales of the activations as they are."""
    _, scales = quantize(rotate(x_bits, block, signs_bits))
    return scales


def outlier_groups(x_bits, top_ppm: int = 1000) -> tuple[np.ndarray, int]:
    """(mask [M, K/32] uint8, threshold bf16 bits): groups holding one of the top ``top_ppm`` millionths
    of the entries by absolute value (Sec. 4.2, Fig. 6: the top 0.1 % -> 1000 ppm)."""
    x = _as_bf16_bits(x_bits)
    M, K = x.shape
    mask = np.empty((M, K // MX_GROUP), dtype=np.uint8)
    t = np.zeros(1, dtype=np.uint16)
    _check(lib().bro_ref_outlier_groups(_ptr(x), M, K, K, int(top_ppm), _ptr(mask), _ptr(t)), "outlier_groups")
    return mask, int(t[0])


def scale_histogram(scales, mask) -> np.ndarray:
    """[2, 256] uint64: scale-byte histogram of the regular (row 0) and outlier (row 1) groups."""
    s = np.ascontiguousarray(scales, dtype=np.uint8).ravel()
    m = np.ascontiguousarray(mask, dtype=np.uint8).ravel()
    assert s.shape == m.shape
    hist = np.empty((2, 256), dtype=np.uint64)
    _check(lib().bro_ref_scale_histogram(_ptr(s), _ptr(m), s.size, _ptr(hist)), "scale_histogram")
    return hist


def scale_inflation(scales_before, scales_after, mask) -> np.ndarray:
    """[2, 3] uint64: per class (regular, outlier) the number of groups whose scale byte went down,
    stayed, went up under the rotation."""
    b = np.ascontiguousarray(scales_before, dtype=np.uint8).ravel()
    a = np.ascontiguousarray(scales_after, dtype=np.uint8).ravel()
    m = np.ascontiguousarray(mask, dtype=np.uint8).ravel()
    assert a.shape == b.shape == m.shape
    counts = np.empty((2, 3), dtype=np.uint64)
    _check(lib().bro_ref_scale_inflation(_ptr(b), _ptr(a), _ptr(m), b.size, _ptr(counts)), "scale_inflation")
    return counts


def swiglu_f32(gate_bits, up_bits) -> np.ndarray:
    """fp32 value of silu(gate) * up before the bf16 rounding (the fixed fp32 operation sequence)."""
    g = np.ascontiguousarray(gate_bits, dtype=np.uint16).ravel()
    u = np.ascontiguousarray(up_bits, dtype=np.uint16).ravel()
    assert g.shape == u.shape
    out = np.empty(g.shape, dtype=np.float32)
    _check(lib().bro_ref_swiglu_f32(_ptr(g), _ptr(u), g.size, _ptr(out)), "swiglu_f32")
    return out


def swiglu(gate_bits, up_bits) -> np.ndarray:
    """h = bf16(silu(gate) * up) as uint16 bit patterns [M, K]: the input of down_proj, which the online
    rotation acts on (Sec. 4.3)."""
    g = _as_bf16_bits(gate_bits)
    u = _as_bf16_bits(up_bits)
    assert g.shape == u.shape
    M, K = g.shape
    h = np.empty((M, K), dtype=np.uint16)
    _check(lib().bro_ref_swiglu(_ptr(g), _ptr(u), M, K, K, K, _ptr(h)), "swiglu")
    return h


def swiglu_rotate_quantize_mxfp4(gate_bits, up_bits, block: int, signs_bits=None) -> tuple[np.ndarray, np.ndarray]:
    g = _as_bf16_bits(gate_bits)
    u = _as_bf16_bits(up_bits)
    assert g.shape == u.shape
    M, K = g.shape
    codes = np.empty((M, K // 2), dtype=np.uint8)
    scales = np.empty((M, K // MX_GROUP), dtype=np.uint8)
    s = _signs(signs_bits, K)
    _check(lib().bro_ref_swiglu_rotate_quantize_mxfp4(_ptr(g), _ptr(u), M, K, K, K, int(block),
                                                      None if s is None else _ptr(s), _ptr(codes), _ptr(scales)),
           "swiglu_rotate_quantize_mxfp4")
    return codes, scales
