"""GPU parity at the full sizes of the measured workloads, in the launch configuration the benchmark
times (bro_linear: rotate+quantize into the workspace, then the GEMM with the default tile).

The activation codes and scales are compared with the CPU oracle bit for bit over the whole
tensor.  The GEMM output is too large for the oracle's fp64 triple loop, so it is checked on
sampled outputs that the oracle computes one by one: whole 128x128 tiles (corners + one interior),
full rows and full columns, and random points.  bf16 output: |y - y_ref| <= 1e-5 * sum|a w| + 1e-6
plus half a bf16 ulp of y_ref."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth
from gpu_util import to_canonical

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def sample_points(M, N, rng, n_random):
    pm, pn = [], []
    tiles_m, tiles_n = (M + 127) // 128, (N + 127) // 128
    tiles = {(0, 0), (0, tiles_n - 1), (tiles_m - 1, 0), (tiles_m - 1, tiles_n - 1),
             (tiles_m // 2, tiles_n // 3)}
    for (tm, tn) in sorted(tiles):
        r = np.arange(tm * 128, min(tm * 128 + 128, M))
        c = np.arange(tn * 128, min(tn * 128 + 128, N))
        mm, nn = np.meshgrid(r, c, indexing="ij")
        pm.append(mm.ravel()); pn.append(nn.ravel())
    for n in rng.integers(0, N, 2):
        rows = np.arange(M) if M <= 4096 else rng.integers(0, M, 4096)
        pm.append(rows); pn.append(np.full(rows.shape[0], n))
    for m in rng.integers(0, M, 2):
        cols = np.arange(N) if N <= 4096 else rng.integers(0, N, 4096)
        pm.append(np.full(cols.shape[0], m)); pn.append(cols)
    pm.append(rng.integers(0, M, n_random)); pn.append(rng.integers(0, N, n_random))
    return np.concatenate(pm).astype(np.int64), np.concatenate(pn).astype(np.int64)


def check_layer(bro, x, wc_ref, ws_ref, wcodes, wscales, N, block, n_random, seed, flags=0):
    M, K = x.shape
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    bro.linear(x.cuda(), block, wcodes, wscales, N, y, ws, flags=flags)
    assert bro.last_device_status() == 0
    ac_ref, as_ref = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), block)
    nc = bro.codes_bytes(M, K)
    acodes = ws[:nc].cpu().numpy().reshape(M, K // 2)
    assert np.array_equal(acodes, ac_ref), "activation codes differ from the oracle"
    off = (nc + 1023) // 1024 * 1024
    ascales = ws[off:off + bro.scales_bytes(M, K, bro.LAYOUT_GEMM)].cpu().numpy()
    assert np.array_equal(to_canonical(ascales, M, K), as_ref), "activation scales differ from the oracle"
    pm, pn = sample_points(M, N, np.random.default_rng(seed), n_random)
    y_ref, S = oracle.gemm_mxfp4_points(ac_ref, as_ref, wc_ref, ws_ref, pm, pn)
    got = y[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()].float().cpu().numpy().astype(np.float64)
    tol = 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8
    bad = np.abs(got - y_ref) > tol
    assert not bad.any(), f"{bad.sum()} of {bad.size} sampled outputs outside tolerance"


def pack_both(bro, w, block):
    N, K = w.shape
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), block)
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w.cuda(), block, wcodes, wscales)
    assert bro.last_device_status() == 0
    assert np.array_equal(wcodes.cpu().numpy(), wc_ref), "weight codes differ from the oracle"
    assert np.array_equal(to_canonical(wscales.cpu().numpy(), N, K), ws_ref), "weight scales differ"
    return wc_ref, ws_ref, wcodes, wscales


SHAPES = [("cfg2", i) for i in range(3)] + [("cfg3", i) for i in range(4)]


@pytest.mark.parametrize("name,index", SHAPES)
def test_llm_shaped_layers_full_size(bro, name, index):
    """The 1B- and 8B-shaped layers (M = 2048 / 4096 tokens), block 32."""
    cfg = synth.CONFIGS[name]
    M, K, N = cfg["shapes"][index]
    seed = synth.config_seed(name, index)
    x = synth.activations(M, K, seed=seed, recipe=cfg["recipe"])
    w = synth.weights(N, K, seed=seed)
    wc_ref, ws_ref, wcodes, wscales = pack_both(bro, w, 32)
    check_layer(bro, x, wc_ref, ws_ref, wcodes, wscales, N, 32, 100000, seed)


@pytest.mark.parametrize("variant", ["pair", "single", "tile_n128", "no_split"])
def test_other_gemm_kernels_on_a_many_tile_shape(bro, variant):
    """M = 4096, K = 4096, N = 14336 (1792 tiles of 128 x 256: twelve per CTA, across raster bands)
    through every GEMM variant by flag — the two-CTA kernel (the library's own choice at this size), the
    single-CTA kernel, 128-column tiles, and the schedule without half-width units — so that each
    variant's accumulator ping-pong over many tiles per CTA is compared with the oracle."""
    cfg = synth.CONFIGS["cfg3"]
    M, K, N = cfg["shapes"][1]
    seed = synth.config_seed("cfg3", 1)
    x = synth.activations(M, K, seed=seed, recipe=cfg["recipe"])
    w = synth.weights(N, K, seed=seed)
    wc_ref, ws_ref, wcodes, wscales = pack_both(bro, w, 32)
    flags = {"pair": bro.FLAG_GEMM_PAIR, "single": bro.FLAG_GEMM_SINGLE, "tile_n128": bro.FLAG_GEMM_TILE_N128,
             "no_split": bro.FLAG_GEMM_NO_SPLIT}[variant]
    check_layer(bro, x, wc_ref, ws_ref, wcodes, wscales, N, 32, 100000, seed, flags=flags)


@pytest.fixture(scope="module")
def packed_70b(bro):
    cfg = synth.CONFIGS["cfg5"]
    _, K, N = cfg["shapes"][0]
    w = synth.weights(N, K, seed=cfg["seed"])
    return pack_both(bro, w, 32)


@pytest.mark.parametrize("M", [1, 16, 128, 1024, 8192, 32768])
def test_70b_shaped_layer_m_sweep(bro, packed_70b, M):
    """Decode-to-prefill sweep against one weight matrix packed offline (K = 8192, N = 28672)."""
    cfg = synth.CONFIGS["cfg5"]
    _, K, N = cfg["shapes"][0]
    wc_ref, ws_ref, wcodes, wscales = packed_70b
    x = synth.activations(M, K, seed=cfg["seed"] + M, recipe=cfg["recipe"])
    check_layer(bro, x, wc_ref, ws_ref, wcodes, wscales, N, 32, 50000, M)


def test_block_sweep_tensor_full_size(bro):
    """The rotate+quantize-only tensor [16384, 4096] for every rotation size, whole tensor."""
    cfg = synth.CONFIGS["cfg4"]
    M, K, _ = cfg["shapes"][0]
    x = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"])
    xd = x.cuda()
    bits = synth.bf16_bits(x)
    for block in cfg["blocks"]:
        codes = bro.alloc_codes(M, K)
        scales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
        bro.rotate_quantize_mxfp4(xd, block, codes, scales, bro.LAYOUT_GEMM)
        assert bro.last_device_status() == 0
        rc, rs = oracle.rotate_quantize_mxfp4(bits, block)
        assert np.array_equal(codes.cpu().numpy(), rc), f"codes differ, block {block}"
        assert np.array_equal(to_canonical(scales.cpu().numpy(), M, K), rs), f"scales differ, block {block}"


@pytest.mark.parametrize("block", [32, 64, 128])
@pytest.mark.parametrize("form", ["default", "direct", "tma_ring"])
def test_block_sweep_tensor_randomised_rotation_both_kernels(bro, block, form):
    """The same [16384, 4096] tensor with the randomised rotation diag(s) H / sqrt(block) (Sec. 5.1),
    whole tensor, through the library's own choice at this size and through each block kernel forced."""
    cfg = synth.CONFIGS["cfg4"]
    M, K, _ = cfg["shapes"][0]
    x = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"])
    signs = synth.rotation_signs(K, seed=cfg["seed"])
    flags = {"default": 0, "direct": bro.FLAG_RQ_DIRECT, "tma_ring": bro.FLAG_RQ_TMA_RING}[form]
    codes = bro.alloc_codes(M, K)
    scales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
    bro.rotate_quantize_mxfp4(x.cuda(), block, codes, scales, bro.LAYOUT_GEMM, flags=flags, signs=signs.cuda())
    assert bro.last_device_status() == 0
    rc, rs = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), block, synth.bf16_bits(signs))
    assert np.array_equal(codes.cpu().numpy(), rc), f"codes differ, block {block}"
    assert np.array_equal(to_canonical(scales.cpu().numpy(), M, K), rs), f"scales differ, block {block}"
