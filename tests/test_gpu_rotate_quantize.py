"""GPU parity, kernel 1: fused block-Hadamard rotation + MXFP4 quantisation against the CPU
oracle, bit-exact on every code byte and every scale byte (Sec. 4.1, Sec. 4.3 Eq. 1)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth
from gpu_util import Guarded, to_canonical, gemm_scale_index

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


@pytest.fixture(params=["default", "direct", "tma_ring"])
def form(request, bro):
    """The two kernels behind block 32 / 64 / 128 — the register-streaming one and the shared-memory
    ring fed by TMA — each forced through the `flags` word of bro_rotate_quantize_mxfp4_ex, next to the
    library's own choice.  (The full-dimension rotation has one kernel; it ignores the flags.)"""
    return {"default": 0, "direct": bro.FLAG_RQ_DIRECT, "tma_ring": bro.FLAG_RQ_TMA_RING}[request.param]


def run_gpu(bro, x_dev, block, layout, flags=0):
    M, K = x_dev.shape
    codes = Guarded(bro.codes_bytes(M, K))
    scales = Guarded(bro.scales_bytes(M, K, layout))
    bro.rotate_quantize_mxfp4(x_dev, block, codes.view, scales.view, layout, flags=flags)
    assert bro.last_device_status() == 0
    codes.check()
    scales.check()
    c = codes.numpy().reshape(M, K // 2)
    s = scales.numpy()
    if layout == bro.LAYOUT_GEMM:
        full = s
        s = to_canonical(full, M, K)
        # every padding byte of the tiled layout must be zero
        mask = np.ones(full.shape, dtype=bool)
        mask[gemm_scale_index(M, K).ravel()] = False
        assert (full[mask] == 0).all()
    else:
        s = s.reshape(M, K // 32)
    return c, s


def compare(bro, x_cpu, block, layout, flags=0):
    bits = synth.bf16_bits(x_cpu)
    rc, rs = oracle.rotate_quantize_mxfp4(bits, block)
    gc, gs = run_gpu(bro, x_cpu.cuda(), block, layout, flags)
    assert np.array_equal(gs, rs), f"scale mismatch: {(gs != rs).sum()} of {rs.size}"
    bad = gc != rc
    assert not bad.any(), f"code mismatch: {bad.sum()} bytes of {rc.size}, first at {np.argwhere(bad)[0]}"


@pytest.mark.parametrize("block", [32, 64, 128, 0])
@pytest.mark.parametrize("layout", [0, 1])
def test_config1_activations(bro, form, block, layout):
    x = synth.activations(64, 2048, seed=0, recipe=synth.CFG1_RECIPE)
    compare(bro, x, block, layout, form)


@pytest.mark.parametrize("block", [2, 4, 8, 16])
@pytest.mark.parametrize("M,K", [(1, 32), (7, 160), (129, 416), (300, 1024), (64, 4096)])
def test_rotations_inside_the_mx_group(bro, M, K, block):
    """Rotation dimensions below the MX group (Sec. 5.2 sweeps the dimension both ways): the butterfly of a
    group stops early; codes and scales bit-exact in both layouts."""
    x = synth.activations(M, K, seed=900 + M + block)
    compare(bro, x, block, 1)
    compare(bro, x, block, 0)
    compare(bro, x, block, 1, bro.FLAG_RQ_TMA_RING)        # (the flag has no say at these sizes)


RAGGED = [(M, K, b) for (M, K) in [(1, 32), (1, 128), (7, 160), (129, 416), (300, 1024), (513, 2176), (1024, 4096)]
          for b in (32, 64, 128) if K % b == 0]


@pytest.mark.parametrize("M,K,block", RAGGED)
def test_ragged_shapes(bro, form, M, K, block):
    """Ragged in both directions (rows beyond M inside the last 128-row tile, K that ends inside a
    128-column tile or a 256-column scale block) and several row tiles, through both kernels."""
    x = synth.activations(M, K, seed=100 + M + K)
    compare(bro, x, block, 1, form)
    compare(bro, x, block, 0, form)


@pytest.mark.parametrize("K", [32, 64, 256, 1024, 2048, 4096, 8192, 16384, 32768])
def test_global_rotation_sizes(bro, K):
    x = synth.activations(37, K, seed=K)
    compare(bro, x, 0, 0)
    compare(bro, x, 0, 1)


def test_weights_path_and_heavy_tails(bro):
    w = synth.weights(384, 1024, seed=3)
    bits = synth.bf16_bits(w)
    rc, rs = oracle.pack_weights(bits, 32)
    codes = Guarded(bro.codes_bytes(384, 1024))
    scales = Guarded(bro.scales_bytes(384, 1024, 1))
    bro.pack_weights(w.cuda(), 32, codes.view, scales.view)
    assert bro.last_device_status() == 0
    codes.check(); scales.check()
    assert np.array_equal(codes.numpy().reshape(384, 512), rc)
    assert np.array_equal(to_canonical(scales.numpy(), 384, 1024), rs)
    x = synth.activations(2048, 2048, seed=2000)        # spikes x20 and 1% outlier channels
    for block in (32, 128):
        compare(bro, x, block, 1)


def test_row_stride_larger_than_K(bro, form):
    base = synth.activations(200, 512, seed=77)
    x_dev = base.cuda()[:, 64:64 + 256]                  # ldx = 512, K = 256, offset 128 bytes
    assert x_dev.stride(0) == 512
    sub = base[:, 64:64 + 256].contiguous()
    rc, rs = oracle.rotate_quantize_mxfp4(synth.bf16_bits(sub), 64)
    gc, gs = run_gpu(bro, x_dev, 64, 0, form)
    assert np.array_equal(gc, rc) and np.array_equal(gs, rs)


@pytest.mark.parametrize("block", [32, 64, 128, 0])
def test_degenerate_values(bro, form, block):
    """All-zero rows, negative zeros, groups far below / above the fast-path exponent window,
    exact cancellations (equal neighbours) and bf16 subnormals."""
    K = 256
    rows = []
    rows.append(np.zeros(K, dtype=np.float32))
    z = np.zeros(K, dtype=np.float32); z[::3] = -0.0; rows.append(z)
    rows.append(np.full(K, 3.0, dtype=np.float32))                      # exact zeros after rotation
    rows.append(np.tile(np.array([1, -1], dtype=np.float32), K // 2))
    rng = np.random.default_rng(0)
    g = rng.standard_normal(K).astype(np.float32)
    for e in (-130, -120, -110, -100, -95, -60, 60, 100, 110, 118):
        rows.append((g * np.float32(2.0) ** e if e > -126 else g * np.float32(2.0 ** -100) * np.float32(2.0 ** (e + 100))).astype(np.float32))
    rows.append(np.where(rng.random(K) < 0.5, np.float32(1e-40), np.float32(-1e-40)).astype(np.float32))
    big = rng.standard_normal(K).astype(np.float32) * np.float32(1e30); rows.append(big)
    x32 = torch.from_numpy(np.stack(rows))
    x = x32.to(torch.bfloat16)
    assert torch.isfinite(x.float()).all()
    compare(bro, x, block, 0, form)
    compare(bro, x, block, 1, form)


def test_config4_slice_all_blocks(bro):
    """A 1024-row slice of the block-size sweep tensor: several row tiles, all four rotations."""
    x = synth.activations(1024, 4096, seed=4000, recipe=synth.CFG4_RECIPE)
    for block in (32, 64, 128, 0):
        compare(bro, x, block, 1)


def test_empty_input_is_a_no_op(bro):
    x = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    codes = Guarded(16); scales = Guarded(16)
    bro.rotate_quantize_mxfp4(x, 32, codes.view, scales.view, 0)
    codes.check(); scales.check()
    assert (codes.numpy() == 0xA5).all()
