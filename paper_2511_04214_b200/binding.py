"""ctypes binding for libbro — argument marshalling only.

Every function takes torch CUDA tensors (device memory owned by the caller), passes raw pointers
and sizes to the C ABI declared in ``include/bro.h`` and raises :class:`BroError` on a non-zero
status.  No step of the method runs in Python or in PyTorch ops, and there is no CPU fallback:
if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libbro.so")

LAYOUT_CANONICAL = 0
LAYOUT_GEMM = 1
OUT_BF16 = 0
OUT_F32 = 1

EXPORTS = [
    "bro_status_string", "bro_last_cuda_error", "bro_codes_bytes", "bro_scales_bytes", "bro_scale_offset",
    "bro_gemm_workspace_bytes", "bro_linear_workspace_bytes", "bro_last_device_status",
    "bro_rotate_quantize_mxfp4", "bro_pack_weights", "bro_gemm_mxfp4", "bro_linear",
    "bro_linear_host", "bro_linear_static",
    "bro_rotate_quantize_mxfp4_rs", "bro_pack_weights_rs", "bro_linear_rs", "bro_group_quant_error", "bro_group_quant_error_fmt", "bro_rotate_fake_quantize", "bro_rotate_fake_quantize_ws", "bro_fake_quantize_workspace_bytes",
    "bro_last_device_status_ex", "bro_selftest_expire_wait",
    "bro_rotate_quantize_mxfp4_ex", "bro_gemm_mxfp4_ex", "bro_linear_ex",
    "bro_group_scale_bytes", "bro_outlier_workspace_bytes", "bro_outlier_groups", "bro_scale_histogram",
    "bro_scale_inflation", "bro_pack_weights_desc", "bro_linear_packed",
    "bro_swiglu_rotate_quantize_mxfp4", "bro_swiglu_bf16", "bro_swiglu_linear",
]


class PackedWeights(ctypes.Structure):
    """Host-side descriptor of packed weights (bro_packed_weights of include/bro.h)."""
    _fields_ = [("magic", ctypes.c_uint32), ("version", ctypes.c_uint32), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("block", ctypes.c_int32), ("randomised", ctypes.c_int32), ("codes", ctypes.c_void_p),
                ("scales", ctypes.c_void_p)]

# kernel-selection flags of the *_ex entry points (testing and tuning)
FLAG_RQ_TMA_RING = 0x1
FLAG_RQ_DIRECT = 0x2
FLAG_GEMM_PAIR = 0x10
FLAG_GEMM_TILE_N128 = 0x20
FLAG_GEMM_TILE_N256 = 0x40
FLAG_GEMM_NO_SPLIT = 0x80
FLAG_GEMM_SINGLE = 0x100


class BroError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        detail = lib.bro_last_cuda_error().decode() if int(code) == 6 else ""
        super().__init__(f"{where}: {status_string(code)} ({code}) {detail}".rstrip())


def _load() -> ctypes.CDLL:
    if not os.path.exists(_SO):
        raise ImportError(
            f"{_SO} is missing: build it with `python -m paper_2511_04214_b200.build` "
            "(there is no fallback path)")
    L = ctypes.CDLL(_SO)
    i64, p, ci, sz, u32, u64 = (ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_uint32,
                                ctypes.c_uint64)
    L.bro_status_string.restype = ctypes.c_char_p
    L.bro_status_string.argtypes = [ci]
    L.bro_last_cuda_error.restype = ctypes.c_char_p
    L.bro_last_cuda_error.argtypes = []
    L.bro_codes_bytes.restype = sz
    L.bro_codes_bytes.argtypes = [i64, i64]
    L.bro_scales_bytes.restype = sz
    L.bro_scales_bytes.argtypes = [i64, i64, ci]
    L.bro_scale_offset.restype = sz
    L.bro_scale_offset.argtypes = [i64, i64, i64, i64, ci]
    L.bro_gemm_workspace_bytes.restype = sz
    L.bro_gemm_workspace_bytes.argtypes = [i64, i64, i64]
    L.bro_linear_workspace_bytes.restype = sz
    L.bro_linear_workspace_bytes.argtypes = [i64, i64, i64]
    L.bro_last_device_status.restype = ci
    L.bro_last_device_status.argtypes = [p]
    L.bro_rotate_quantize_mxfp4.restype = ci
    L.bro_rotate_quantize_mxfp4.argtypes = [p, i64, i64, i64, ci, p, p, ci, p]
    L.bro_pack_weights.restype = ci
    L.bro_pack_weights.argtypes = [p, i64, i64, i64, ci, p, p, p]
    L.bro_gemm_mxfp4.restype = ci
    L.bro_gemm_mxfp4.argtypes = [p, p, p, p, i64, i64, i64, p, i64, ci, p, sz, p]
    L.bro_linear.restype = ci
    L.bro_linear.argtypes = [p, i64, i64, i64, ci, p, p, i64, p, i64, p, sz, p]
    L.bro_linear_host.restype = ci
    L.bro_linear_host.argtypes = [p, i64, i64, ci, p, p, i64, p, p, p, p, sz, p]
    L.bro_rotate_quantize_mxfp4_rs.restype = ci
    L.bro_rotate_quantize_mxfp4_rs.argtypes = [p, i64, i64, i64, ci, p, p, p, ci, p]
    L.bro_pack_weights_rs.restype = ci
    L.bro_pack_weights_rs.argtypes = [p, i64, i64, i64, ci, p, p, p, p]
    L.bro_linear_rs.restype = ci
    L.bro_linear_rs.argtypes = [p, i64, i64, i64, ci, p, p, p, i64, p, i64, p, sz, p]
    L.bro_group_quant_error.restype = ci
    L.bro_group_quant_error.argtypes = [p, i64, i64, i64, ci, p, p, p]
    L.bro_group_quant_error_fmt.restype = ci
    L.bro_group_quant_error_fmt.argtypes = [p, i64, i64, i64, ci, p, ci, p, p]
    L.bro_rotate_fake_quantize.restype = ci
    L.bro_rotate_fake_quantize.argtypes = [p, i64, i64, i64, ci, p, ci, p, i64, p]
    L.bro_rotate_fake_quantize_ws.restype = ci
    L.bro_rotate_fake_quantize_ws.argtypes = [p, i64, i64, i64, ci, p, ci, p, i64, p, sz, p]
    L.bro_fake_quantize_workspace_bytes.restype = sz
    L.bro_fake_quantize_workspace_bytes.argtypes = [i64, ci]
    L.bro_linear_static.restype = ci
    L.bro_linear_static.argtypes = [p, i64, i64, i64, ci, p, p, i64, p, i64, p]
    L.bro_group_scale_bytes.restype = ci
    L.bro_group_scale_bytes.argtypes = [p, i64, i64, i64, ci, p, p, p]
    L.bro_outlier_workspace_bytes.restype = sz
    L.bro_outlier_workspace_bytes.argtypes = []
    L.bro_outlier_groups.restype = ci
    L.bro_outlier_groups.argtypes = [p, i64, i64, i64, i64, p, p, p, sz, p]
    L.bro_scale_histogram.restype = ci
    L.bro_scale_histogram.argtypes = [p, p, i64, p, p]
    L.bro_scale_inflation.restype = ci
    L.bro_scale_inflation.argtypes = [p, p, p, i64, p, p]
    L.bro_swiglu_rotate_quantize_mxfp4.restype = ci
    L.bro_swiglu_rotate_quantize_mxfp4.argtypes = [p, p, i64, i64, i64, i64, ci, p, p, p, ci, p]
    L.bro_swiglu_bf16.restype = ci
    L.bro_swiglu_bf16.argtypes = [p, p, i64, i64, i64, i64, p, i64, p]
    L.bro_swiglu_linear.restype = ci
    L.bro_swiglu_linear.argtypes = [p, p, i64, i64, i64, i64, ci, p, p, p, i64, p, i64, p, sz, p]
    L.bro_pack_weights_desc.restype = ci
    L.bro_pack_weights_desc.argtypes = [p, i64, i64, i64, ci, p, p, p, ctypes.POINTER(PackedWeights), p]
    L.bro_linear_packed.restype = ci
    L.bro_linear_packed.argtypes = [p, i64, i64, i64, ci, p, ctypes.POINTER(PackedWeights), p, i64, p, sz, p]
    L.bro_last_device_status_ex.restype = ci
    L.bro_last_device_status_ex.argtypes = [p, ctypes.POINTER(ci)]
    L.bro_selftest_expire_wait.restype = ci
    L.bro_selftest_expire_wait.argtypes = [u64, p]
    L.bro_rotate_quantize_mxfp4_ex.restype = ci
    L.bro_rotate_quantize_mxfp4_ex.argtypes = [p, i64, i64, i64, ci, p, p, p, ci, u32, p]
    L.bro_gemm_mxfp4_ex.restype = ci
    L.bro_gemm_mxfp4_ex.argtypes = [p, p, p, p, i64, i64, i64, p, i64, ci, p, sz, u32, p]
    L.bro_linear_ex.restype = ci
    L.bro_linear_ex.argtypes = [p, i64, i64, i64, ci, p, p, p, i64, p, i64, p, sz, u32, p]
    return L


lib = _load()


def status_string(code: int) -> str:
    return lib.bro_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise BroError(code, where)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def codes_bytes(rows: int, K: int) -> int:
    return int(lib.bro_codes_bytes(rows, K))


def scales_bytes(rows: int, K: int, layout: int) -> int:
    return int(lib.bro_scales_bytes(rows, K, layout))


def scale_offset(row: int, group: int, rows: int, K: int, layout: int) -> int:
    return int(lib.bro_scale_offset(row, group, rows, K, layout))


def gemm_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib.bro_gemm_workspace_bytes(M, N, K))


def linear_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib.bro_linear_workspace_bytes(M, N, K))


def last_device_status(stream=None) -> int:
    return int(lib.bro_last_device_status(_stream(stream)))


def last_device_status_ex(stream=None):
    """(status, site): the device status word of the current device, read and cleared."""
    site = ctypes.c_int(0)
    code = int(lib.bro_last_device_status_ex(_stream(stream), ctypes.byref(site)))
    return code, int(site.value)


def selftest_expire_wait(budget_ns: int = 1_000_000, stream=None) -> None:
    """Launch the one-warp self-test whose bounded wait runs out (see include/bro.h)."""
    _check(lib.bro_selftest_expire_wait(int(budget_ns), _stream(stream)), "bro_selftest_expire_wait")


def alloc_codes(rows: int, K: int, device="cuda") -> torch.Tensor:
    return torch.empty((rows, K // 2), dtype=torch.uint8, device=device)


def alloc_scales(rows: int, K: int, layout: int, device="cuda") -> torch.Tensor:
    return torch.empty(scales_bytes(rows, K, layout), dtype=torch.uint8, device=device)


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """uint8 buffer of at least ``nbytes`` whose start is 1024-byte aligned."""
    raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 1024
    return raw[off:off + max(nbytes, 1)]


def rotate_quantize_mxfp4(x: torch.Tensor, block: int, codes: torch.Tensor, scales: torch.Tensor,
                          layout: int = LAYOUT_GEMM, stream=None, flags: int = 0, signs=None) -> None:
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    if flags or signs is not None:
        _check(lib.bro_rotate_quantize_mxfp4_ex(_ptr(x), M, K, x.stride(0) if M > 1 else max(x.stride(0), K), block,
                                                _ptr(signs), _ptr(codes), _ptr(scales), layout, flags,
                                                _stream(stream)), "bro_rotate_quantize_mxfp4_ex")
        return
    _check(lib.bro_rotate_quantize_mxfp4(_ptr(x), M, K, x.stride(0) if M > 1 else max(x.stride(0), K),
                                         block, _ptr(codes), _ptr(scales), layout, _stream(stream)),
           "bro_rotate_quantize_mxfp4")


def pack_weights(w: torch.Tensor, block: int, wcodes: torch.Tensor, wscales: torch.Tensor,
                 stream=None) -> None:
    assert w.dtype == torch.bfloat16 and w.dim() == 2 and w.stride(1) == 1
    N, K = w.shape
    _check(lib.bro_pack_weights(_ptr(w), N, K, w.stride(0) if N > 1 else max(w.stride(0), K), block,
                                _ptr(wcodes), _ptr(wscales), _stream(stream)), "bro_pack_weights")


def gemm_mxfp4(acodes, ascales, wcodes, wscales, M: int, N: int, K: int, y: torch.Tensor,
               workspace=None, stream=None, flags: int = 0) -> None:
    out = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_F32
    assert y.dtype in (torch.bfloat16, torch.float32) and y.stride(1) == 1
    wsb = 0 if workspace is None else workspace.numel()
    if flags:
        _check(lib.bro_gemm_mxfp4_ex(_ptr(acodes), _ptr(ascales), _ptr(wcodes), _ptr(wscales), M, N, K,
                                     _ptr(y), y.stride(0) if M > 1 else max(y.stride(0), N), out,
                                     _ptr(workspace), wsb, flags, _stream(stream)), "bro_gemm_mxfp4_ex")
        return
    _check(lib.bro_gemm_mxfp4(_ptr(acodes), _ptr(ascales), _ptr(wcodes), _ptr(wscales), M, N, K,
                              _ptr(y), y.stride(0) if M > 1 else max(y.stride(0), N), out,
                              _ptr(workspace), wsb, _stream(stream)), "bro_gemm_mxfp4")


def linear(x: torch.Tensor, block: int, wcodes, wscales, N: int, y: torch.Tensor,
           workspace: torch.Tensor, stream=None, flags: int = 0, signs=None) -> None:
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
    M, K = x.shape
    if flags:
        _check(lib.bro_linear_ex(_ptr(x), M, K, x.stride(0) if M > 1 else max(x.stride(0), K), block, _ptr(signs),
                                 _ptr(wcodes), _ptr(wscales), N, _ptr(y),
                                 y.stride(0) if M > 1 else max(y.stride(0), N), _ptr(workspace),
                                 workspace.numel(), flags, _stream(stream)), "bro_linear_ex")
        return
    assert signs is None, "use linear_rs (or pass flags) for the randomised rotation"
    _check(lib.bro_linear(_ptr(x), M, K, x.stride(0) if M > 1 else max(x.stride(0), K), block,
                          _ptr(wcodes), _ptr(wscales), N, _ptr(y),
                          y.stride(0) if M > 1 else max(y.stride(0), N), _ptr(workspace),
                          workspace.numel(), _stream(stream)), "bro_linear")


def linear_host(x_host: torch.Tensor, block: int, wcodes, wscales, N: int, y_host: torch.Tensor,
                x_stage: torch.Tensor, y_stage: torch.Tensor, workspace: torch.Tensor,
                stream=None) -> None:
    """Host-buffer variant: x_host / y_host are (ideally pinned) CPU bf16 tensors."""
    assert x_host.device.type == "cpu" and y_host.device.type == "cpu"
    assert x_host.is_contiguous() and y_host.is_contiguous()
    M, K = x_host.shape
    _check(lib.bro_linear_host(_ptr(x_host), M, K, block, _ptr(wcodes), _ptr(wscales), N,
                               _ptr(y_host), _ptr(x_stage), _ptr(y_stage), _ptr(workspace),
                               workspace.numel(), _stream(stream)), "bro_linear_host")


STATIC_SCRATCH_BYTES = 16 << 20


def linear_static(x: torch.Tensor, block: int, wcodes, wscales, N: int, y: torch.Tensor,
                  stream=None) -> None:
    """``linear`` for callers that may not allocate device memory (a plugin that only receives its
    input and output tensors, code running while someone else captures a CUDA graph, a server that
    forbids allocation after start-up): the quantised activations go to a ``STATIC_SCRATCH_BYTES``
    array built into the library, so the problem must fit it (roughly M*K <= 31 million).  Calls
    on one GPU share that array — keep them on one stream.  Make the first call per device outside
    stream capture."""
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
    M, K = x.shape
    code = lib.bro_linear_static(_ptr(x), M, K, x.stride(0) if M > 1 else max(x.stride(0), K), block,
                                 _ptr(wcodes), _ptr(wscales), N, _ptr(y),
                                 y.stride(0) if M > 1 else max(y.stride(0), N), _stream(stream))
    if code == 5:
        raise BroError(code, "bro_linear_static: " + lib.bro_last_cuda_error().decode())
    _check(code, "bro_linear_static")


def _ld(t, n):
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), n)


def rotate_quantize_mxfp4_rs(x: torch.Tensor, block: int, signs: torch.Tensor, codes, scales,
                             layout: int = LAYOUT_GEMM, stream=None) -> None:
    """Randomised rotation: ``signs`` is a bf16 [K] device vector of +1 / -1."""
    assert x.dtype == torch.bfloat16 and signs.dtype == torch.bfloat16 and signs.numel() == x.shape[1]
    M, K = x.shape
    _check(lib.bro_rotate_quantize_mxfp4_rs(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), _ptr(codes),
                                            _ptr(scales), layout, _stream(stream)),
           "bro_rotate_quantize_mxfp4_rs")


def pack_weights_rs(w: torch.Tensor, block: int, signs: torch.Tensor, wcodes, wscales, stream=None) -> None:
    assert w.dtype == torch.bfloat16 and signs.dtype == torch.bfloat16 and signs.numel() == w.shape[1]
    N, K = w.shape
    _check(lib.bro_pack_weights_rs(_ptr(w), N, K, _ld(w, K), block, _ptr(signs), _ptr(wcodes),
                                   _ptr(wscales), _stream(stream)), "bro_pack_weights_rs")


def linear_rs(x: torch.Tensor, block: int, signs: torch.Tensor, wcodes, wscales, N: int, y: torch.Tensor,
              workspace: torch.Tensor, stream=None) -> None:
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16 and signs.dtype == torch.bfloat16
    M, K = x.shape
    _check(lib.bro_linear_rs(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), _ptr(wcodes), _ptr(wscales), N,
                             _ptr(y), _ld(y, N), _ptr(workspace), workspace.numel(), _stream(stream)),
           "bro_linear_rs")


FORMATS = {"mxfp4": 0, "bfp4": 1, "mxint4": 2, "bint4": 3, "int4_row_sym": 4, "int4_row_asym": 5, "none": 6}


def group_quant_error(x: torch.Tensor, block: int, mse: torch.Tensor, signs: torch.Tensor = None,
                      stream=None, fmt: str = "mxfp4") -> None:
    """Per-group quantisation error of the rotated activations: ``mse`` is fp32 [M, K/32]."""
    assert x.dtype == torch.bfloat16 and mse.dtype == torch.float32 and mse.is_contiguous()
    M, K = x.shape
    assert mse.shape == (M, K // 32)
    _check(lib.bro_group_quant_error_fmt(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), FORMATS[fmt], _ptr(mse),
                                         _stream(stream)), "bro_group_quant_error_fmt")


def fake_quantize_workspace_bytes(M: int, fmt: str) -> int:
    return int(lib.bro_fake_quantize_workspace_bytes(M, FORMATS[fmt]))


def rotate_fake_quantize(x: torch.Tensor, block: int, deq: torch.Tensor, fmt: str = "mxfp4", signs: torch.Tensor = None,
                         workspace: torch.Tensor = None, stream=None) -> None:
    """Simulated quantisation: ``deq`` (fp32 [M, K], rows may be strided) receives the dequantised values of
    x R_block quantised to ``fmt``; block = 1: no rotation, 0: the full dimension.  The per-row formats
    ("int4_row_sym", "int4_row_asym") need ``workspace`` (fake_quantize_workspace_bytes); "none" returns the
    rotated values themselves."""
    assert x.dtype == torch.bfloat16 and deq.dtype == torch.float32
    M, K = x.shape
    assert deq.shape == (M, K)
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.bro_rotate_fake_quantize_ws(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), FORMATS[fmt], _ptr(deq), _ld(deq, K),
                                           _ptr(workspace), wbytes, _stream(stream)), "bro_rotate_fake_quantize_ws")


def group_scale_bytes(x: torch.Tensor, block: int, scales: torch.Tensor, signs: torch.Tensor = None, stream=None) -> None:
    """E8M0 byte of every MX group of x R_block into ``scales`` (uint8 [M, K/32]); block = 1: no rotation."""
    assert x.dtype == torch.bfloat16 and scales.dtype == torch.uint8 and scales.is_contiguous()
    M, K = x.shape
    assert scales.shape == (M, K // 32)
    _check(lib.bro_group_scale_bytes(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), _ptr(scales), _stream(stream)),
           "bro_group_scale_bytes")


def outlier_groups(x: torch.Tensor, mask: torch.Tensor, info: torch.Tensor, workspace: torch.Tensor,
                   top_ppm: int = 1000, stream=None) -> None:
    """Groups holding one of the top ``top_ppm`` millionths of |x| -> ``mask`` (uint8 [M, K/32]);
    ``info`` (int32/uint32 [4] on the device) receives the threshold's bf16 pattern and k."""
    assert x.dtype == torch.bfloat16 and mask.dtype == torch.uint8 and mask.is_contiguous()
    M, K = x.shape
    assert mask.shape == (M, K // 32) and info.numel() >= 4 and info.element_size() == 4
    _check(lib.bro_outlier_groups(_ptr(x), M, K, _ld(x, K), int(top_ppm), _ptr(mask), _ptr(info), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)), "bro_outlier_groups")


def outlier_workspace_bytes() -> int:
    return int(lib.bro_outlier_workspace_bytes())


def scale_histogram(scales: torch.Tensor, mask: torch.Tensor, hist: torch.Tensor, stream=None) -> None:
    """``hist`` (int64 [2, 256] on the device) <- scale-byte histograms of the regular / outlier groups."""
    assert scales.dtype == torch.uint8 and mask.dtype == torch.uint8 and hist.dtype == torch.int64
    assert scales.is_contiguous() and mask.is_contiguous() and hist.is_contiguous() and hist.numel() == 512
    assert scales.numel() == mask.numel()
    _check(lib.bro_scale_histogram(_ptr(scales), _ptr(mask), scales.numel(), _ptr(hist), _stream(stream)),
           "bro_scale_histogram")


def scale_inflation(before: torch.Tensor, after: torch.Tensor, mask: torch.Tensor, counts: torch.Tensor,
                    stream=None) -> None:
    """``counts`` (int64 [2, 3] on the device) <- per class, groups whose byte went down / stayed / went up."""
    assert before.dtype == after.dtype == mask.dtype == torch.uint8 and counts.dtype == torch.int64
    assert before.is_contiguous() and after.is_contiguous() and mask.is_contiguous() and counts.numel() == 6
    assert before.numel() == after.numel() == mask.numel()
    _check(lib.bro_scale_inflation(_ptr(before), _ptr(after), _ptr(mask), before.numel(), _ptr(counts),
                                   _stream(stream)), "bro_scale_inflation")


def pack_weights_desc(w: torch.Tensor, block: int, wcodes, wscales, signs: torch.Tensor = None, stream=None) -> PackedWeights:
    """pack_weights that also returns the host-side descriptor (N, K, block, randomised, buffers)."""
    assert w.dtype == torch.bfloat16 and w.dim() == 2 and w.stride(1) == 1
    N, K = w.shape
    desc = PackedWeights()
    _check(lib.bro_pack_weights_desc(_ptr(w), N, K, _ld(w, K), block, _ptr(signs), _ptr(wcodes), _ptr(wscales),
                                     ctypes.byref(desc), _stream(stream)), "bro_pack_weights_desc")
    return desc


def linear_packed(x: torch.Tensor, block: int, weights: PackedWeights, y: torch.Tensor, workspace: torch.Tensor,
                  signs: torch.Tensor = None, stream=None) -> None:
    """linear that first checks the descriptor against K, block and the use of a sign vector."""
    assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16
    M, K = x.shape
    _check(lib.bro_linear_packed(_ptr(x), M, K, _ld(x, K), block, _ptr(signs), ctypes.byref(weights), _ptr(y),
                                 _ld(y, weights.N), _ptr(workspace), workspace.numel(), _stream(stream)),
           "bro_linear_packed")


def swiglu_rotate_quantize_mxfp4(gate: torch.Tensor, up: torch.Tensor, block: int, codes, scales,
                                 layout: int = LAYOUT_GEMM, signs: torch.Tensor = None, stream=None) -> None:
    """rotate_quantize_mxfp4 of h = silu(gate) * up, with h computed inside the kernel."""
    assert gate.dtype == up.dtype == torch.bfloat16 and gate.shape == up.shape
    assert gate.stride(1) == 1 and up.stride(1) == 1
    M, K = gate.shape
    _check(lib.bro_swiglu_rotate_quantize_mxfp4(_ptr(gate), _ptr(up), M, K, _ld(gate, K), _ld(up, K), block, _ptr(signs),
                                                _ptr(codes), _ptr(scales), layout, _stream(stream)),
           "bro_swiglu_rotate_quantize_mxfp4")


def swiglu_bf16(gate: torch.Tensor, up: torch.Tensor, h: torch.Tensor, stream=None) -> None:
    """h = bf16(silu(gate) * up): the producer alone."""
    assert gate.dtype == up.dtype == h.dtype == torch.bfloat16 and gate.shape == up.shape == h.shape
    M, K = gate.shape
    _check(lib.bro_swiglu_bf16(_ptr(gate), _ptr(up), M, K, _ld(gate, K), _ld(up, K), _ptr(h), _ld(h, K), _stream(stream)),
           "bro_swiglu_bf16")


def swiglu_linear(gate: torch.Tensor, up: torch.Tensor, block: int, wcodes, wscales, N: int, y: torch.Tensor,
                  workspace: torch.Tensor, signs: torch.Tensor = None, stream=None) -> None:
    """linear(_rs) on h = silu(gate) * up with the producer fused into rotate+quantize."""
    assert gate.dtype == up.dtype == y.dtype == torch.bfloat16 and gate.shape == up.shape
    M, K = gate.shape
    _check(lib.bro_swiglu_linear(_ptr(gate), _ptr(up), M, K, _ld(gate, K), _ld(up, K), block, _ptr(signs), _ptr(wcodes),
                                 _ptr(wscales), N, _ptr(y), _ld(y, N), _ptr(workspace), workspace.numel(),
                                 _stream(stream)), "bro_swiglu_linear")
