"""GPU parity of the rotation fused into its producer: h = bf16(silu(gate) * up) computed inside the
rotate+quantize kernel (Sec. 4.3: the online rotation sits before down_proj).  Codes and scales bit-exact
against the oracle, the stand-alone producer bit-exact, the fused call equal to the two-step path, and the
whole layer within the GEMM tolerance."""
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


def gate_up(M, K, seed):
    """Gate pre-activations with the heavy tails of the recipe, a Gaussian up projection."""
    g = synth.activations(M, K, seed=seed) * 0.5
    u = synth.weights(M, K, seed=seed + 1, std=1.5)
    return g.to(torch.bfloat16), u


@pytest.mark.parametrize("block", [32, 64, 128])
@pytest.mark.parametrize("M,K", [(1, 128), (7, 256), (64, 2048), (300, 1024), (513, 2176)])
def test_fused_codes_and_scales_bit_exact(bro, block, M, K):
    if K % block:
        pytest.skip("K not a multiple of the block")
    g, u = gate_up(M, K, 60 + M)
    gb, ub = synth.bf16_bits(g), synth.bf16_bits(u)
    for layout in (bro.LAYOUT_GEMM, bro.LAYOUT_CANONICAL):
        for signs in (None, synth.rotation_signs(K, seed=K)):
            rc, rs = oracle.swiglu_rotate_quantize_mxfp4(gb, ub, block, None if signs is None else synth.bf16_bits(signs))
            codes = Guarded(bro.codes_bytes(M, K)); scales = Guarded(bro.scales_bytes(M, K, layout))
            bro.swiglu_rotate_quantize_mxfp4(g.cuda(), u.cuda(), block, codes.view, scales.view, layout,
                                             signs=None if signs is None else signs.cuda())
            assert bro.last_device_status() == 0
            codes.check(); scales.check()
            gs = scales.numpy()
            gs = to_canonical(gs, M, K) if layout == bro.LAYOUT_GEMM else gs.reshape(M, K // 32)
            assert np.array_equal(gs, rs)
            assert np.array_equal(codes.numpy().reshape(M, K // 2), rc)


def test_producer_alone_is_bit_exact_over_the_whole_bf16_range(bro):
    pats = np.arange(0, 0x7F80, dtype=np.uint16)
    gb = np.concatenate([pats, pats | 0x8000]).astype(np.uint16).reshape(-1, 64)     # every finite bf16 gate
    rng = np.random.default_rng(5)
    ub = synth.bf16_bits(torch.from_numpy((rng.standard_normal(gb.shape) * 3).astype(np.float32)).to(torch.bfloat16))
    ref = oracle.swiglu(gb, ub)
    g, u = synth.bits_to_bf16(gb).cuda(), synth.bits_to_bf16(ub).cuda()
    h = torch.full(g.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    bro.swiglu_bf16(g, u, h)
    assert bro.last_device_status() == 0
    got = synth.bf16_bits(h.cpu())
    bad = got != ref
    assert not bad.any(), (int(bad.sum()), gb[bad][:4], got[bad][:4], ref[bad][:4])


def test_fused_equals_the_two_step_path_with_row_strides(bro):
    base_g, base_u = gate_up(200, 1024, 9)
    g = base_g.cuda()[:, 128:128 + 512]                      # ldg = 1024, K = 512
    u = base_u.cuda()[:, 256:256 + 512]
    h = torch.empty((200, 512), dtype=torch.bfloat16, device="cuda")
    bro.swiglu_bf16(g, u, h)
    c1 = bro.alloc_codes(200, 512); s1 = bro.alloc_scales(200, 512, bro.LAYOUT_GEMM)
    c2 = bro.alloc_codes(200, 512); s2 = bro.alloc_scales(200, 512, bro.LAYOUT_GEMM)
    bro.rotate_quantize_mxfp4(h, 64, c1, s1, bro.LAYOUT_GEMM)
    bro.swiglu_rotate_quantize_mxfp4(g, u, 64, c2, s2, bro.LAYOUT_GEMM)
    assert torch.equal(c1, c2) and torch.equal(s1, s2)
    rc, rs = oracle.swiglu_rotate_quantize_mxfp4(synth.bf16_bits(base_g[:, 128:640].contiguous()),
                                                 synth.bf16_bits(base_u[:, 256:768].contiguous()), 64)
    assert np.array_equal(c2.cpu().numpy(), rc)


def test_whole_layer_with_the_fused_producer(bro):
    M, K, N = 300, 1024, 520
    g, u = gate_up(M, K, 21)
    w = synth.weights(N, K, seed=22)
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(w), 32)
    hb = oracle.swiglu(synth.bf16_bits(g), synth.bf16_bits(u))
    y_ref, S = oracle.linear(hb, 32, wc_ref, ws_ref)
    wcodes = bro.alloc_codes(N, K); wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w.cuda(), 32, wcodes, wscales)
    ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    bro.swiglu_linear(g.cuda(), u.cuda(), 32, wcodes, wscales, N, y, ws)
    assert bro.last_device_status() == 0
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - y_ref) <= 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8)
    # and it tracks the unquantised layer h W^T
    exact = synth.bits_to_bf16(hb).double().numpy() @ w.double().numpy().T
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.25


def test_full_size_tensor_and_argument_checks(bro):
    M, K = 4096, 4096
    g, u = gate_up(M, K, 4000)
    rc, rs = oracle.swiglu_rotate_quantize_mxfp4(synth.bf16_bits(g), synth.bf16_bits(u), 32)
    codes = bro.alloc_codes(M, K); scales = bro.alloc_scales(M, K, bro.LAYOUT_GEMM)
    bro.swiglu_rotate_quantize_mxfp4(g.cuda(), u.cuda(), 32, codes, scales, bro.LAYOUT_GEMM)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(to_canonical(scales.cpu().numpy(), M, K), rs)
    with pytest.raises(bro.BroError) as e:
        bro.swiglu_rotate_quantize_mxfp4(g.cuda(), u.cuda(), 0, codes, scales, bro.LAYOUT_GEMM)
    assert e.value.code == 4
