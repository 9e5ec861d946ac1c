"""The C-ABI library loads without a GPU and exports every symbol include/bro.h declares; the
pure host-side helpers (sizes, offsets, status strings, argument validation that happens before
any CUDA call) behave as documented.  No compute call is made here."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_04214_b200 import build
    build.build()
    from paper_2511_04214_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bro.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bro_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib.lib, n), n
    assert sorted(lib.EXPORTS) == names


def test_status_strings(lib):
    assert lib.status_string(0) == "BRO_OK"
    assert lib.status_string(7) == "BRO_ERR_TIMEOUT"
    assert lib.status_string(99) == "BRO_ERR_UNKNOWN"


def test_sizes(lib):
    assert lib.codes_bytes(64, 2048) == 64 * 1024
    assert lib.codes_bytes(3, 48) == 0            # K not a multiple of 32
    assert lib.scales_bytes(64, 2048, lib.LAYOUT_CANONICAL) == 64 * 64
    # GEMM layout: rows padded to 128, K padded to 256 -> 8 blocks of 512 B
    assert lib.scales_bytes(64, 2048, lib.LAYOUT_GEMM) == 1 * 16 * 512
    assert lib.scales_bytes(129, 160, lib.LAYOUT_GEMM) == 2 * 2 * 512
    assert lib.linear_workspace_bytes(64, 2048, 2048) >= 64 * 1024 + 8192


def test_gemm_scale_layout_is_a_bijection(lib):
    rows, K = 300, 416            # 13 groups: ragged in both directions
    nbytes = lib.scales_bytes(rows, K, lib.LAYOUT_GEMM)
    seen = set()
    for r in range(rows):
        for g in range(K // 32):
            off = lib.scale_offset(r, g, rows, K, lib.LAYOUT_GEMM)
            assert 0 <= off < nbytes
            assert off not in seen
            seen.add(off)
    # spot values of the documented formula
    assert lib.scale_offset(0, 0, rows, K, lib.LAYOUT_GEMM) == 0
    assert lib.scale_offset(1, 0, rows, K, lib.LAYOUT_GEMM) == 16
    assert lib.scale_offset(32, 0, rows, K, lib.LAYOUT_GEMM) == 4
    assert lib.scale_offset(0, 3, rows, K, lib.LAYOUT_GEMM) == 3
    assert lib.scale_offset(0, 4, rows, K, lib.LAYOUT_GEMM) == 512
    kb = 2 * ((K + 255) // 256)
    assert lib.scale_offset(128, 0, rows, K, lib.LAYOUT_GEMM) == kb * 512
    assert lib.scale_offset(5, 7, rows, K, lib.LAYOUT_CANONICAL) == 5 * 13 + 7


def test_argument_validation_needs_no_device(lib):
    """Checks that run before any CUDA call return their codes on a GPU-less machine too."""
    L = lib.lib
    buf = (ctypes.c_uint8 * 4096)()
    a = ctypes.addressof(buf)
    a16 = (a + 15) // 16 * 16
    p = ctypes.c_void_p
    assert L.bro_rotate_quantize_mxfp4(None, 1, 32, 32, 32, p(a16), p(a16), 0, None) == 1
    assert L.bro_rotate_quantize_mxfp4(p(a16), 1, 48, 48, 32, p(a16), p(a16), 0, None) == 2
    assert L.bro_rotate_quantize_mxfp4(p(a16), 1, 64, 64, 48, p(a16), p(a16), 0, None) == 2
    assert L.bro_rotate_quantize_mxfp4(p(a16), 1, 96, 96, 64, p(a16), p(a16), 0, None) == 2
    assert L.bro_rotate_quantize_mxfp4(p(a16), 1, 96, 96, 0, p(a16), p(a16), 0, None) == 4
    assert L.bro_rotate_quantize_mxfp4(p(a16 + 2), 1, 64, 64, 32, p(a16), p(a16), 0, None) == 3
    assert L.bro_rotate_quantize_mxfp4(p(a16), 1, 64, 68, 32, p(a16), p(a16), 0, None) == 3
    assert L.bro_rotate_quantize_mxfp4(p(a16), 0, 64, 64, 32, p(a16), p(a16), 0, None) == 0
    a128 = (a + 127) // 128 * 128
    assert L.bro_gemm_mxfp4(p(a128), p(a128), p(a128), None, 1, 8, 32, p(a128), 8, 0, None, 0, None) == 1
    assert L.bro_gemm_mxfp4(None, None, None, None, 0, 8, 32, None, 8, 0, None, 0, None) == 0
    assert L.bro_gemm_mxfp4(p(a128), p(a128), p(a128), p(a128), 1, 8, 40, p(a128), 8, 0, None, 0, None) == 2
    assert L.bro_gemm_mxfp4(p(a128), p(a128), p(a128), p(a128), 1, 8, 32, p(a128), 4, 0, None, 0, None) == 2
    assert L.bro_gemm_mxfp4(p(a128 + 16), p(a128), p(a128), p(a128), 1, 8, 32, p(a128), 8, 0, None, 0, None) == 3
    assert L.bro_gemm_mxfp4(p(a128), p(a128), p(a128), p(a128), 0, 8, 32, p(a128), 8, 0, None, 0, None) == 0
    assert L.bro_linear(p(a128), 4, 32, 32, 32, p(a128), p(a128), 8, p(a128), 8, None, 0, None) == 1


def test_fake_quantize_argument_validation_needs_no_device(lib):
    L = lib.lib
    buf = (ctypes.c_uint8 * 4096)()
    a16 = (ctypes.addressof(buf) + 15) // 16 * 16
    p = ctypes.c_void_p
    fq = L.bro_rotate_fake_quantize
    assert fq(None, 1, 64, 64, 32, None, 0, p(a16), 64, None) == 1
    assert fq(p(a16), 1, 64, 64, 32, None, 0, None, 64, None) == 1
    assert fq(p(a16), 1, 64, 64, 32, None, 7, p(a16), 64, None) == 2         # no such format
    assert fq(p(a16), 1, 64, 64, 32, None, 4, p(a16), 64, None) == 5         # the per-row formats need a workspace
    ws = L.bro_rotate_fake_quantize_ws
    assert L.bro_fake_quantize_workspace_bytes(100, 4) == 800 and L.bro_fake_quantize_workspace_bytes(100, 5) == 800
    assert L.bro_fake_quantize_workspace_bytes(100, 0) == 0 and L.bro_fake_quantize_workspace_bytes(100, 6) == 0
    assert ws(p(a16), 2, 64, 64, 32, None, 5, p(a16), 64, p(a16), 15, None) == 5       # too small
    assert ws(p(a16), 2, 64, 64, 32, None, 5, p(a16), 64, p(a16 + 4), 16, None) == 3   # not 8-byte aligned
    assert ws(p(a16), 0, 64, 64, 32, None, 5, p(a16), 64, None, 0, None) == 0          # no rows: nothing to do
    assert fq(p(a16), 1, 48, 48, 32, None, 0, p(a16), 48, None) == 2         # K not a multiple of 32
    assert fq(p(a16), 1, 96, 96, 24, None, 0, p(a16), 96, None) == 2         # no such block
    assert fq(p(a16), 1, 256, 256, 256, None, 0, p(a16), 256, None) == 2
    assert fq(p(a16), 1, 96, 96, 64, None, 0, p(a16), 96, None) == 2         # K not a multiple of the block
    assert fq(p(a16), 1, 64, 64, 32, None, 0, p(a16), 60, None) == 2         # ldd < K
    assert fq(p(a16), 1, 96, 96, 0, None, 0, p(a16), 96, None) == 4          # full-dimension rotation needs a power of two
    assert fq(p(a16), 1, 64, 64, 32, None, 0, p(a16), 66, None) == 3         # ldd not a multiple of 4
    assert fq(p(a16), 1, 64, 64, 32, None, 0, p(a16 + 4), 64, None) == 3
    assert fq(p(a16), 1, 64, 64, 32, p(a16 + 2), 0, p(a16), 64, None) == 3
    assert fq(p(a16), 0, 64, 64, 1, None, 3, p(a16), 64, None) == 0          # no rows: nothing to do


def test_packed_weight_descriptor_is_checked_before_any_device_work(lib):
    """bro_linear_packed refuses weights packed with another block size, another K, with / without a sign
    vector, or a descriptor that is not one — all on the host, before any CUDA call."""
    L = lib.lib
    buf = (ctypes.c_uint8 * 4096)()
    a = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    p = ctypes.c_void_p
    d = lib.PackedWeights(magic=0x344F5242, version=1, N=8, K=64, block=32, randomised=0, codes=a, scales=a)
    ref = ctypes.byref(d)
    assert L.bro_linear_packed(p(a), 4, 64, 64, 64, None, ref, p(a), 8, p(a), 1 << 20, None) == 2      # block differs
    assert L.bro_linear_packed(p(a), 4, 128, 128, 32, None, ref, p(a), 8, p(a), 1 << 20, None) == 2    # K differs
    assert L.bro_linear_packed(p(a), 4, 64, 64, 32, p(a), ref, p(a), 8, p(a), 1 << 20, None) == 2      # signs on one side only
    d.randomised = 1
    assert L.bro_linear_packed(p(a), 4, 64, 64, 32, None, ref, p(a), 8, p(a), 1 << 20, None) == 2
    d.randomised = 0
    d.version = 7
    assert L.bro_linear_packed(p(a), 4, 64, 64, 32, None, ref, p(a), 8, p(a), 1 << 20, None) == 4      # unknown layout version
    d.version, d.magic = 1, 0
    assert L.bro_linear_packed(p(a), 4, 64, 64, 32, None, ref, p(a), 8, p(a), 1 << 20, None) == 4      # not a descriptor
    assert L.bro_linear_packed(p(a), 4, 64, 64, 32, None, None, p(a), 8, p(a), 1 << 20, None) == 1
    d.magic = 0x344F5242
    assert L.bro_linear_packed(p(a), 0, 64, 64, 32, None, ref, p(a), 8, p(a), 1 << 20, None) == 0      # M == 0: nothing to do
    # a failed packing leaves the descriptor invalid
    out = lib.PackedWeights(magic=0x344F5242)
    assert L.bro_pack_weights_desc(p(a), 8, 48, 48, 32, None, p(a), p(a), ctypes.byref(out), None) == 2
    assert out.magic == 0


def test_fused_producer_argument_validation_needs_no_device(lib):
    L = lib.lib
    buf = (ctypes.c_uint8 * 4096)()
    a = (ctypes.addressof(buf) + 15) // 16 * 16
    p = ctypes.c_void_p
    f = L.bro_swiglu_rotate_quantize_mxfp4
    assert f(p(a), None, 1, 64, 64, 64, 32, None, p(a), p(a), 0, None) == 1          # up missing
    assert f(p(a), p(a), 1, 64, 64, 64, 0, None, p(a), p(a), 0, None) == 4           # no full-dimension form
    assert f(p(a), p(a), 1, 64, 64, 32, 32, None, p(a), p(a), 0, None) == 2          # ldu < K
    assert f(p(a), p(a), 1, 64, 64, 68, 32, None, p(a), p(a), 0, None) == 3          # ldu not a multiple of 8
    assert f(p(a), p(a + 2), 1, 64, 64, 64, 32, None, p(a), p(a), 0, None) == 3      # up misaligned
    assert f(p(a), p(a), 1, 48, 48, 48, 32, None, p(a), p(a), 0, None) == 2          # K not a multiple of 32
    assert f(p(a), p(a), 0, 64, 64, 64, 32, None, p(a), p(a), 0, None) == 0          # nothing to do
    g = L.bro_swiglu_bf16
    assert g(p(a), p(a), 1, 60, 64, 64, p(a), 64, None) == 2                          # K not a multiple of 8
    assert g(p(a), None, 1, 64, 64, 64, p(a), 64, None) == 1
    assert g(p(a), p(a), 1, 64, 64, 64, p(a), 32, None) == 2                          # ldh < K
    assert g(p(a), p(a), 0, 64, 64, 64, p(a), 64, None) == 0
    a1k = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    h = L.bro_swiglu_linear
    assert h(p(a), p(a), 4, 64, 64, 64, 0, None, p(a), p(a), 8, p(a), 8, p(a1k), 1 << 20, None) == 4
    assert h(p(a), p(a), 4, 64, 64, 64, 32, None, p(a), p(a), 8, p(a), 8, None, 0, None) == 1
    assert h(p(a), p(a), 4, 64, 64, 64, 32, None, p(a), p(a), 8, p(a), 8, p(a1k), 16, None) == 5
