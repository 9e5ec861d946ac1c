"""GPU parity, kernel 2 and the whole layer: block-scaled MXFP4 x MXFP4 GEMM (tcgen05) against the
CPU oracle's fp64 sums.  Tolerance (fp32 result): |y - y_ref| <= 1e-5 * sum_k |a_k w_k| + 1e-6.
bf16 output: within that tolerance plus half a bf16 ulp of y_ref, and bit-identical to the
round-to-nearest-even bf16 of the same kernel's fp32 result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth
from gpu_util import Guarded, to_gemm_layout

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def upload_operand(codes: np.ndarray, scales_canon: np.ndarray):
    rows, K = codes.shape[0], codes.shape[1] * 2
    c = torch.from_numpy(np.ascontiguousarray(codes)).cuda()
    s = torch.from_numpy(to_gemm_layout(scales_canon, rows, K)).cuda()
    return c, s


def gpu_gemm(bro, ac, asc, wc, wsc, dtype, ldy=None, flags=0):
    M, K = ac.shape[0], ac.shape[1] * 2
    N = wc.shape[0]
    a_c, a_s = upload_operand(ac, asc)
    w_c, w_s = upload_operand(wc, wsc)
    ldy = ldy or (N + 7) // 8 * 8          # row pitch must be a multiple of 16 bytes
    esz = 2 if dtype == torch.bfloat16 else 4
    buf = Guarded(M * ldy * esz, fill=0x7F)
    y = buf.view.view(dtype).view(M, ldy)[:, :N]
    ws = bro.alloc_workspace(bro.gemm_workspace_bytes(M, N, K))
    bro.gemm_mxfp4(a_c, a_s, w_c, w_s, M, N, K, y, workspace=ws, flags=flags)
    assert bro.last_device_status() == 0
    buf.check()
    if ldy > N:   # the gap between rows must be untouched
        gap = buf.view.view(dtype).view(M, ldy)[:, N:].contiguous().view(torch.uint8).cpu().numpy()
        assert (gap == 0x7F).all()
    return y.float().cpu().numpy().astype(np.float64), y


def check_f32(y, y_ref, S):
    tol = 1e-5 * S + 1e-6
    err = np.abs(y - y_ref)
    worst = np.max(err / tol)
    assert worst <= 1.0, f"max err/tol = {worst:.3f} at {np.unravel_index(np.argmax(err / tol), err.shape)}"


def check_bf16(y16, y32_dev, y_ref, S):
    tol = 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8
    assert np.all(np.abs(y16 - y_ref) <= tol)
    expect = y32_dev.to(torch.bfloat16)          # round-to-nearest-even
    return expect


def run_case(bro, ac, asc, wc, wsc, ldy=None, flags=0):
    y_ref, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    y32, y32_dev = gpu_gemm(bro, ac, asc, wc, wsc, torch.float32, ldy, flags)
    check_f32(y32, y_ref, S)
    y16, y16_dev = gpu_gemm(bro, ac, asc, wc, wsc, torch.bfloat16, ldy, flags)
    expect = check_bf16(y16, y32_dev, y_ref, S)
    assert torch.equal(y16_dev.contiguous().view(torch.int16), expect.contiguous().view(torch.int16))


def quantized_pair(M, N, K, seed, block=32, recipe=synth.HEAVY_RECIPE):
    x = synth.activations(M, K, seed=seed, recipe=recipe)
    w = synth.weights(N, K, seed=seed + 1)
    ac, asc = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), block)
    wc, wsc = oracle.pack_weights(synth.bf16_bits(w), block)
    return x, w, ac, asc, wc, wsc


@pytest.fixture(params=["default", "cta1_n128", "cta1_n256", "pair", "single"])
def tile_n(request, bro):
    """Each GEMM kernel variant in turn, as the `flags` word of bro_gemm_mxfp4_ex: the library's own
    choice, the single-CTA kernel forced to 128- or 256-column tiles, and the two-CTA (cta_group::2)
    kernel with 256 x 256 tiles."""
    return {"default": 0, "cta1_n128": bro.FLAG_GEMM_TILE_N128, "cta1_n256": bro.FLAG_GEMM_TILE_N256,
            "pair": bro.FLAG_GEMM_PAIR, "single": bro.FLAG_GEMM_SINGLE}[request.param]


def test_unit_scales_small_integers_exact(bro, tile_n):
    """All scales 2^0 and half-integer codes: every partial sum is exactly representable, so the
    tensor-core result must equal the integer matmul bit for bit."""
    rng = np.random.default_rng(0)
    M, N, K = 128, 256, 256
    ac = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    wc = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    asc = np.full((M, K // 32), 127, dtype=np.uint8)
    wsc = np.full((N, K // 32), 127, dtype=np.uint8)
    y_ref, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    y32, _ = gpu_gemm(bro, ac, asc, wc, wsc, torch.float32, flags=tile_n)
    assert np.array_equal(y32, y_ref)


def test_scale_bytes_reach_the_right_rows_and_groups(bro, tile_n):
    """One-hot structure: a single non-zero code per row of A at k = 37*m mod K, distinct scales per
    (row, group) on both sides; each output is one product, so a misplaced scale byte or a swapped
    operand shows up exactly."""
    rng = np.random.default_rng(1)
    M, N, K = 256, 384, 512
    ac = np.zeros((M, K // 2), dtype=np.uint8)
    for m in range(M):
        k = (37 * m + 5) % K
        ac[m, k // 2] = (2 + (m % 5)) << (4 * (k & 1))
    wc = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    asc = rng.integers(110, 140, size=(M, K // 32), dtype=np.uint8)
    wsc = rng.integers(110, 140, size=(N, K // 32), dtype=np.uint8)
    y_ref, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    y32, _ = gpu_gemm(bro, ac, asc, wc, wsc, torch.float32, flags=tile_n)
    assert np.array_equal(y32, y_ref)


def test_config1_full_output(bro, tile_n):
    _, _, ac, asc, wc, wsc = quantized_pair(64, 2048, 2048, seed=0, recipe=synth.CFG1_RECIPE)
    run_case(bro, ac, asc, wc, wsc, flags=tile_n)


@pytest.mark.parametrize("M,N,K", [(1, 8, 32), (129, 136, 160), (300, 520, 416), (128, 256, 288),
                                   (257, 129, 1024), (64, 384, 3072), (700, 1300, 512), (2304, 1000, 768)])
def test_ragged_shapes(bro, tile_n, M, N, K):
    _, _, ac, asc, wc, wsc = quantized_pair(M, N, K, seed=M + N + K)
    run_case(bro, ac, asc, wc, wsc, flags=tile_n)


@pytest.mark.parametrize("M,N,K", [(128 * 19, 2048, 256), (128 * 5, 300, 512), (128 * 3, 4 * 256 + 40, 288),
                                   (256 * 19, 1024, 512), (256 * 3, 7 * 256 + 40, 288)])
@pytest.mark.parametrize("kernel", ["single", "pair"])
def test_half_width_units_of_the_last_round(bro, kernel, M, N, K):
    """Tile counts that leave the last round of the persistent grid less than half full (e.g. 152 = 148 + 4
    tiles of 128 x 256, or 76 = 74 + 2 tiles of 256 x 256 for the two-CTA kernel; 10, 15 and 24 tiles, fewer
    than half the SMs): the remaining tiles are computed as two half-width units each.  Includes ragged N
    whose last half-width unit lies beyond N.  With and without the split, in both kernels."""
    flag = bro.FLAG_GEMM_SINGLE if kernel == "single" else bro.FLAG_GEMM_PAIR
    _, _, ac, asc, wc, wsc = quantized_pair(M, N, K, seed=M + N)
    run_case(bro, ac, asc, wc, wsc, flags=flag)
    run_case(bro, ac, asc, wc, wsc, flags=flag | bro.FLAG_GEMM_NO_SPLIT)


def test_row_stride_of_y(bro, tile_n):
    _, _, ac, asc, wc, wsc = quantized_pair(130, 136, 256, seed=9)
    run_case(bro, ac, asc, wc, wsc, ldy=136 + 24, flags=tile_n)


def test_wide_scale_range_and_all_positive_stress(bro, tile_n):
    """Scales spread over 2^-40..2^40, and an all-positive operand pair with K = 14336 (the longest
    accumulation chain in the configs) where there is no cancellation to hide accumulation error."""
    rng = np.random.default_rng(3)
    M, N, K = 128, 128, 1024
    ac = rng.integers(0, 256, size=(M, K // 2), dtype=np.uint8)
    wc = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    asc = rng.integers(87, 167, size=(M, K // 32), dtype=np.uint8)
    wsc = rng.integers(87, 167, size=(N, K // 32), dtype=np.uint8)
    y_ref, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    y32, _ = gpu_gemm(bro, ac, asc, wc, wsc, torch.float32, flags=tile_n)
    # with an 80-binade spread the absolute floor 1e-6 is meaningless: relative criterion only
    assert np.all(np.abs(y32 - y_ref) <= 1e-5 * S)
    K = 14336
    ac = (rng.integers(0, 256, size=(64, K // 2), dtype=np.uint8) & 0x77)
    wc = (rng.integers(0, 256, size=(128, K // 2), dtype=np.uint8) & 0x77)
    asc = rng.integers(125, 130, size=(64, K // 32), dtype=np.uint8)
    wsc = rng.integers(125, 130, size=(128, K // 32), dtype=np.uint8)
    run_case(bro, ac, asc, wc, wsc, flags=tile_n)


def test_linear_end_to_end_config1(bro):
    """bro_linear = kernel 1 + kernel 2 on device, against the oracle's whole-layer result."""
    x = synth.activations(64, 2048, seed=0, recipe=synth.CFG1_RECIPE)
    w = synth.weights(2048, 2048, seed=0)
    for block in (32, 64, 128, 0, 8, 16):          # (8, 16: rotation dimensions below the MX group)
        wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), block)
        y_ref, S = oracle.linear(synth.bf16_bits(x), block, wc_ref, ws_ref)
        wcodes = bro.alloc_codes(2048, 2048)
        wscales = bro.alloc_scales(2048, 2048, bro.LAYOUT_GEMM)
        bro.pack_weights(w.cuda(), block, wcodes, wscales)
        ws = bro.alloc_workspace(bro.linear_workspace_bytes(64, 2048, 2048))
        y = torch.empty((64, 2048), dtype=torch.bfloat16, device="cuda")
        bro.linear(x.cuda(), block, wcodes, wscales, 2048, y, ws)
        assert bro.last_device_status() == 0
        got = y.float().cpu().numpy().astype(np.float64)
        tol = 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8
        assert np.all(np.abs(got - y_ref) <= tol)


def test_linear_host_buffers(bro):
    x = synth.activations(200, 512, seed=5)
    w = synth.weights(264, 512, seed=6)
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), 32)
    y_ref, S = oracle.linear(synth.bf16_bits(x), 32, wc_ref, ws_ref)
    wcodes = bro.alloc_codes(264, 512); wscales = bro.alloc_scales(264, 512, bro.LAYOUT_GEMM)
    bro.pack_weights(w.cuda(), 32, wcodes, wscales)
    xh = x.pin_memory()
    yh = torch.empty((200, 264), dtype=torch.bfloat16).pin_memory()
    xs = torch.empty((200, 512), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((200, 264), dtype=torch.bfloat16, device="cuda")
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(200, 264, 512))
    bro.linear_host(xh, 32, wcodes, wscales, 264, yh, xs, ys, ws)
    assert bro.last_device_status() == 0
    got = yh.float().numpy().astype(np.float64)
    tol = 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8
    assert np.all(np.abs(got - y_ref) <= tol)


def test_config2_shape_sampled(bro):
    """M=2048, K=2048, N=8192 (one of the 1B-shaped layers): whole tiles, full rows/columns and
    random points against the oracle."""
    M, K, N = 2048, 2048, 8192
    x = synth.activations(M, K, seed=2001)
    w = synth.weights(N, K, seed=2001)
    xd, wd = x.cuda(), w.cuda()
    acodes = bro.alloc_codes(M, K); ascales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
    wcodes = bro.alloc_codes(N, K); wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.rotate_quantize_mxfp4(xd, 32, acodes, ascales, bro.LAYOUT_GEMM)
    bro.pack_weights(wd, 32, wcodes, wscales)
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    bro.gemm_mxfp4(acodes, ascales, wcodes, wscales, M, N, K, y)
    assert bro.last_device_status() == 0
    ac, asc = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), 32)
    wc, wsc = oracle.pack_weights(synth.bf16_bits(w), 32)
    assert np.array_equal(acodes.cpu().numpy(), ac) and np.array_equal(wcodes.cpu().numpy(), wc)
    rng = np.random.default_rng(0)
    pts_m, pts_n = [], []
    for (tm, tn) in [(0, 0), (0, N // 128 - 1), (M // 128 - 1, 0), (M // 128 - 1, N // 128 - 1), (7, 33)]:
        mm, nn = np.meshgrid(np.arange(tm * 128, tm * 128 + 128), np.arange(tn * 128, tn * 128 + 128), indexing="ij")
        pts_m.append(mm.ravel()); pts_n.append(nn.ravel())
    for n in rng.integers(0, N, 4):
        pts_m.append(np.arange(M)); pts_n.append(np.full(M, n))
    for m in rng.integers(0, M, 4):
        pts_m.append(np.full(N, m)); pts_n.append(np.arange(N))
    pts_m.append(rng.integers(0, M, 200000)); pts_n.append(rng.integers(0, N, 200000))
    pm = np.concatenate(pts_m).astype(np.int64); pn = np.concatenate(pts_n).astype(np.int64)
    y_ref, S = oracle.gemm_mxfp4_points(ac, asc, wc, wsc, pm, pn)
    got = y[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - y_ref) <= 1e-5 * S + 1e-6)


def test_whole_layer_is_deterministic_and_graph_safe(bro):
    """Same inputs -> same bits, call after call and when replayed from a CUDA graph (no atomics, a
    fixed order of tensor-core operations, no allocation or synchronisation inside the calls)."""
    M, K, N = 300, 1024, 776
    x = synth.activations(M, K, seed=77).cuda()
    w = synth.weights(N, K, seed=78).cuda()
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w, 32, wcodes, wscales)
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    y1 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    bro.linear(x, 32, wcodes, wscales, N, y1, ws)
    bro.linear(x, 32, wcodes, wscales, N, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    y3 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        bro.linear(x, 32, wcodes, wscales, N, y3, ws, stream=s)        # warm-up outside capture
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            bro.linear(x, 32, wcodes, wscales, N, y3, ws, stream=s)
        y3.fill_(float("nan"))
        g.replay()
        g.replay()
    torch.cuda.synchronize()
    assert bro.last_device_status() == 0
    assert torch.equal(y1.view(torch.int16), y3.view(torch.int16))
