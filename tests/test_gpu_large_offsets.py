"""Tensors beyond 2^32 bytes: a 5.4 GB activation tensor through both rotate+quantize kernels and a 9.4 GB
output through both GEMM kernels.  No measured workload reaches these sizes (the largest output of the
configs is 1.9 GB), so address arithmetic that silently wrapped at 32 bits would otherwise go unseen.

The inputs repeat a small seeded tile with a period of 4099 rows (a prime: the repeats do not line up
with any tile of the kernels), so the expected result of every row is known from the oracle's result for
the tile, and the whole output is compared on the device, block of rows by block of rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth
from gpu_util import to_canonical

pytestmark = pytest.mark.gpu

PERIOD = 4099


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def free_bytes():
    return torch.cuda.mem_get_info()[0]


@pytest.mark.parametrize("form", ["direct", "tma_ring"])
def test_rotate_quantize_input_beyond_4_gib(bro, form):
    K, reps = 8192, 80
    M = PERIOD * reps                                   # 327 920 rows: 5.37 GB of bf16
    if free_bytes() < 12 << 30:
        pytest.skip("needs 12 GB of free device memory")
    tile = synth.activations(PERIOD, K, seed=31)
    rc, rs = oracle.rotate_quantize_mxfp4(synth.bf16_bits(tile), 32)
    x = tile.cuda().repeat(reps, 1)
    assert x.numel() * 2 > 1 << 32
    codes = bro.alloc_codes(M, K)
    scales = bro.alloc_scales(M, K, bro.LAYOUT_CANONICAL)
    flags = bro.FLAG_RQ_DIRECT if form == "direct" else bro.FLAG_RQ_TMA_RING
    bro.rotate_quantize_mxfp4(x, 32, codes, scales, bro.LAYOUT_CANONICAL, flags=flags)
    assert bro.last_device_status() == 0
    exp_c = torch.from_numpy(rc).cuda()
    exp_s = torch.from_numpy(rs).cuda()
    c = codes[: M * (K // 2)].view(reps, PERIOD, K // 2)
    s = scales[: M * (K // 32)].view(reps, PERIOD, K // 32)
    for r in range(reps):
        assert torch.equal(c[r], exp_c), f"codes of repeat {r} differ"
        assert torch.equal(s[r], exp_s), f"scales of repeat {r} differ"


@pytest.mark.parametrize("kernel", ["single", "pair"])
def test_gemm_output_beyond_8_gib(bro, kernel):
    K, N, reps = 256, 28672, 40
    M = PERIOD * reps                                   # 163 960 rows: 9.4 GB of bf16 output
    if free_bytes() < 14 << 30:
        pytest.skip("needs 14 GB of free device memory")
    tile = synth.activations(PERIOD, K, seed=32)
    w = synth.weights(N, K, seed=33)
    ac_ref, as_ref = oracle.rotate_quantize_mxfp4(synth.bf16_bits(tile), 32)
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), 32)
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w.cuda(), 32, wcodes, wscales)
    x = tile.cuda().repeat(reps, 1)
    acodes = bro.alloc_codes(M, K)
    ascales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
    bro.rotate_quantize_mxfp4(x, 32, acodes, ascales, bro.LAYOUT_GEMM)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    assert y.numel() * 2 > 1 << 33
    flags = bro.FLAG_GEMM_SINGLE if kernel == "single" else bro.FLAG_GEMM_PAIR
    bro.gemm_mxfp4(acodes, ascales, wcodes, wscales, M, N, K, y, flags=flags)
    assert bro.last_device_status() == 0
    # the first period against the oracle on sampled outputs ...
    rng = np.random.default_rng(5)
    pm = np.concatenate([rng.integers(0, PERIOD, 4000), np.full(512, PERIOD - 1), np.zeros(512, dtype=np.int64)]).astype(np.int64)
    pn = np.concatenate([rng.integers(0, N, 4000), rng.integers(0, N, 512), rng.integers(0, N, 512)]).astype(np.int64)
    y_ref, S = oracle.gemm_mxfp4_points(ac_ref, as_ref, wc_ref, ws_ref, pm, pn)
    got = y[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - y_ref) <= 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8)
    # ... and every later period against the first, bit for bit (same operands, same accumulation order)
    yv = y.view(reps, PERIOD, N)
    for r in range(1, reps):
        assert torch.equal(yv[r], yv[0]), f"rows of repeat {r} differ from the first period"
