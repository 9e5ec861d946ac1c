"""GPU parity for the randomised block rotation R_i = diag(s) H / sqrt(block) (Sec. 5.1): codes and
scales bit-exact against the CPU oracle for every block size, the weight path, and the whole layer
within the GEMM tolerance (fp32 criterion plus half a bf16 ulp)."""
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


@pytest.fixture(params=["default", "direct", "tma_ring"])
def form(request, bro):
    """The library's own kernel choice, then each of the two block kernels forced (flags of the _ex entry point)."""
    return {"default": 0, "direct": bro.FLAG_RQ_DIRECT, "tma_ring": bro.FLAG_RQ_TMA_RING}[request.param]


def compare(bro, x, signs, block, layout, flags=0):
    M, K = x.shape
    rc, rs = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), block, synth.bf16_bits(signs))
    codes = Guarded(bro.codes_bytes(M, K))
    scales = Guarded(bro.scales_bytes(M, K, layout))
    if flags:
        bro.rotate_quantize_mxfp4(x.cuda(), block, codes.view, scales.view, layout, flags=flags, signs=signs.cuda())
    else:
        bro.rotate_quantize_mxfp4_rs(x.cuda(), block, signs.cuda(), codes.view, scales.view, layout)
    assert bro.last_device_status() == 0
    codes.check(); scales.check()
    gs = scales.numpy()
    gs = to_canonical(gs, M, K) if layout == bro.LAYOUT_GEMM else gs.reshape(M, K // 32)
    assert np.array_equal(gs, rs)
    assert np.array_equal(codes.numpy().reshape(M, K // 2), rc)


@pytest.mark.parametrize("block", [32, 64, 128, 0])
@pytest.mark.parametrize("M,K", [(64, 2048), (300, 1024), (7, 256), (513, 2176), (1024, 4096)])
def test_codes_and_scales_bit_exact(bro, form, block, M, K):
    if block and K % block:
        pytest.skip("K not a multiple of the block")
    if block == 0 and K & (K - 1):
        pytest.skip("the full-dimension rotation needs a power-of-two K")
    x = synth.activations(M, K, seed=40 + M)
    signs = synth.rotation_signs(K, seed=K)
    compare(bro, x, signs, block, 1, form)
    compare(bro, x, signs, block, 0, form)


@pytest.mark.parametrize("block", [2, 4, 8, 16])
def test_rotations_inside_the_mx_group(bro, block):
    x = synth.activations(129, 416, seed=60 + block)
    signs = synth.rotation_signs(416, seed=61)
    compare(bro, x, signs, block, 1)
    compare(bro, x, signs, block, 0)


def test_ragged_k_and_all_plus_signs(bro):
    x = synth.activations(129, 416, seed=2)
    compare(bro, x, synth.rotation_signs(416, seed=3), 32, 1)
    plus = torch.ones(416, dtype=torch.bfloat16)
    compare(bro, x, plus, 32, 0)
    # all +1 must equal the plain entry point
    c1 = bro.alloc_codes(129, 416); s1 = bro.alloc_scales(129, 416, 0)
    c2 = bro.alloc_codes(129, 416); s2 = bro.alloc_scales(129, 416, 0)
    bro.rotate_quantize_mxfp4_rs(x.cuda(), 32, plus.cuda(), c1, s1, 0)
    bro.rotate_quantize_mxfp4(x.cuda(), 32, c2, s2, 0)
    assert torch.equal(c1, c2) and torch.equal(s1, s2)


@pytest.mark.parametrize("block", [32, 0])
def test_whole_layer_with_randomised_rotation(bro, block):
    M, K, N = 200, 1024, 520
    x = synth.activations(M, K, seed=21)
    w = synth.weights(N, K, seed=22)
    signs = synth.rotation_signs(K, seed=23)
    sb = synth.bf16_bits(signs)
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), block, sb)
    y_ref, S = oracle.linear(synth.bf16_bits(x), block, wc_ref, ws_ref, sb)
    wcodes = bro.alloc_codes(N, K); wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights_rs(w.cuda(), block, signs.cuda(), wcodes, wscales)
    assert np.array_equal(wcodes.cpu().numpy(), wc_ref)
    assert np.array_equal(to_canonical(wscales.cpu().numpy(), N, K), ws_ref)
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    bro.linear_rs(x.cuda(), block, signs.cuda(), wcodes, wscales, N, y, ws)
    assert bro.last_device_status() == 0
    got = y.float().cpu().numpy().astype(np.float64)
    tol = 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8
    assert np.all(np.abs(got - y_ref) <= tol)
    # the rotation cancels in exact arithmetic: the quantised layer tracks x W^T
    exact = x.double().numpy() @ w.double().numpy().T
    rel = np.linalg.norm(got - exact) / np.linalg.norm(exact)
    assert rel < 0.25


def test_packed_weight_descriptor_round_trip_and_mismatch(bro):
    """bro_pack_weights_desc / bro_linear_packed: the same bits as bro_linear(_rs) when the descriptor
    matches, BRO_ERR_SHAPE when the activations ask for another rotation than the weights carry."""
    M, K, N = 130, 512, 264
    x = synth.activations(M, K, seed=31).cuda()
    w = synth.weights(N, K, seed=32).cuda()
    signs = synth.rotation_signs(K, seed=33).cuda()
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    for s in (None, signs):
        wcodes = bro.alloc_codes(N, K); wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
        desc = bro.pack_weights_desc(w, 64, wcodes, wscales, signs=s)
        assert (desc.N, desc.K, desc.block, desc.randomised) == (N, K, 64, 0 if s is None else 1)
        y1 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        if s is None:
            bro.linear(x, 64, wcodes, wscales, N, y1, ws)
        else:
            bro.linear_rs(x, 64, s, wcodes, wscales, N, y1, ws)
        bro.linear_packed(x, 64, desc, y2, ws, signs=s)
        assert bro.last_device_status() == 0
        assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
        with pytest.raises(bro.BroError) as e:
            bro.linear_packed(x, 32, desc, y2, ws, signs=s)              # another block size
        assert e.value.code == 2
        with pytest.raises(bro.BroError) as e:
            bro.linear_packed(x, 64, desc, y2, ws, signs=(signs if s is None else None))
        assert e.value.code == 2
