"""Seeded random shapes through the whole C ABI (rotate+quantize, weight packing, GEMM with both
output types, whole layer) against the CPU oracle: codes and scales bit for bit, outputs within the
GEMM tolerance (Sec. 4.1 quantiser, Sec. 4.3 Eq. 1 rotation, W4A4 product).  The shapes are small
and ragged on purpose: rows that do not fill a tile, K that does not fill a K step, N that is not a
multiple of 8 (no TMA store for the last columns), every rotation size that divides K."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth
from gpu_util import Guarded, to_canonical

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def draw_case(seed):
    rng = np.random.default_rng(9000 + seed)
    M = int(rng.choice([1, 2, 7, 31, 64, 127, 128, 129, 200, 333]))
    K = 32 * int(rng.integers(1, 41))
    N = int(rng.choice([1, 8, 24, 100, 128, 129, 255, 256, 257, 391, 520, 777]))
    blocks = [b for b in (32, 64, 128) if K % b == 0]
    if K & (K - 1) == 0:
        blocks.append(0)
    block = int(rng.choice(blocks))
    if seed >= 24:                       # the later seeds draw a rotation dimension below the MX group
        block = int(rng.choice([2, 4, 8, 16]))
    return M, K, N, block


@pytest.mark.parametrize("seed", range(32))
def test_random_case(bro, seed):
    M, K, N, block = draw_case(seed)
    x = synth.activations(M, K, seed=seed)
    w = synth.weights(N, K, seed=1000 + seed)
    xb, wb = synth.bf16_bits(x), synth.bf16_bits(w)
    ac_ref, as_ref = oracle.rotate_quantize_mxfp4(xb, block)
    wc_ref, ws_ref = oracle.pack_weights(wb, block)
    y_ref, S = oracle.linear(xb, block, wc_ref, ws_ref)

    # rotate + quantize, both scale layouts, with guard bands around the outputs
    for layout in (bro.LAYOUT_CANONICAL, bro.LAYOUT_GEMM):
        codes = Guarded(bro.codes_bytes(M, K))
        scales = Guarded(bro.scales_bytes(M, K, layout))
        bro.rotate_quantize_mxfp4(x.cuda(), block, codes.view, scales.view, layout)
        assert bro.last_device_status() == 0
        codes.check(); scales.check()
        got_s = scales.numpy()
        got_s = to_canonical(got_s, M, K) if layout == bro.LAYOUT_GEMM else got_s.reshape(M, K // 32)
        assert np.array_equal(codes.numpy().reshape(M, K // 2), ac_ref)
        assert np.array_equal(got_s, as_ref)

    # weights
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w.cuda(), block, wcodes, wscales)
    assert np.array_equal(wcodes.cpu().numpy(), wc_ref)
    assert np.array_equal(to_canonical(wscales.cpu().numpy(), N, K), ws_ref)

    # GEMM on the quantised operands: fp32 output against the strict bound
    acodes = bro.alloc_codes(M, K)
    ascales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
    bro.rotate_quantize_mxfp4(x.cuda(), block, acodes, ascales, bro.LAYOUT_GEMM)
    ld32 = (N + 3) // 4 * 4          # rows of the output start on 16-byte boundaries
    y32buf = torch.full((M, ld32), float("nan"), dtype=torch.float32, device="cuda")
    y32 = y32buf[:, :N]
    for flags in (0, bro.FLAG_GEMM_PAIR, bro.FLAG_GEMM_TILE_N128):      # the library's choice, then the other kernels
        y32buf.fill_(float("nan"))
        bro.gemm_mxfp4(acodes, ascales, wcodes, wscales, M, N, K, y32, flags=flags)
        assert bro.last_device_status() == 0
        got32 = y32.cpu().numpy().astype(np.float64)
        assert not np.isnan(got32).any()
        assert np.all(np.abs(got32 - y_ref) <= 1e-5 * S + 1e-6), hex(flags)
        if ld32 > N:
            assert torch.isnan(y32buf[:, N:]).all()

    # whole layer, bf16 output (a row pitch that keeps rows 16-byte aligned)
    ldy = (N + 7) // 8 * 8
    ybuf = torch.full((M, ldy), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = ybuf[:, :N]
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    bro.linear(x.cuda(), block, wcodes, wscales, N, y, ws)
    assert bro.last_device_status() == 0
    got = y.float().cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - y_ref) <= 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8)
    if ldy > N:      # the pitch padding is not written
        assert torch.isnan(ybuf[:, N:].float()).all()
