"""bro_linear_static: the whole layer for a caller that cannot allocate device memory.

Some users of this library only ever hold their input and output tensors: a plugin inside a
framework that owns the allocator, code that runs while an outer layer is capturing a CUDA graph,
a server that bans cudaMalloc once it is up.  For them the library keeps the intermediate
(quantised activations) in a 16 MiB array compiled into it.  The test drives that entry point
through the C ABI twice in a row — the second problem is smaller and has a different K, so it
runs on top of what the first call left in the array — and compares each result with what the
ordinary workspace-based bro_linear writes for the same inputs.  Both routes launch the same two
kernels, so the outputs must agree bit for bit (well inside the GEMM tolerance used elsewhere).

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2511_04214_b200 import synth


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import build
    build.build()
    from paper_2511_04214_b200 import binding
    return binding


def layer_inputs(bro, M, K, N, seed, block):
    x = synth.activations(M, K, seed=seed).cuda()
    w = synth.weights(N, K, seed=seed).cuda()
    wcodes = bro.alloc_codes(N, K)
    wscales = bro.alloc_scales(N, K, bro.LAYOUT_GEMM)
    bro.pack_weights(w, block, wcodes, wscales)
    return x, wcodes, wscales


@pytest.mark.gpu
def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row(bro):
    cases = [(1500, 2048, 1032, 11, 32), (77, 384, 264, 12, 128)]
    prepared = []
    for (M, K, N, seed, block) in cases:
        x, wcodes, wscales = layer_inputs(bro, M, K, N, seed, block)
        ws = bro.alloc_workspace(bro.linear_workspace_bytes(M, N, K))
        expect = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        bro.linear(x, block, wcodes, wscales, N, expect, ws)
        prepared.append((x, wcodes, wscales, N, block, expect))
    assert bro.last_device_status() == 0
    outs = []
    for (x, wcodes, wscales, N, block, expect) in prepared:          # two calls, back to back
        y = torch.full(expect.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        bro.linear_static(x, block, wcodes, wscales, N, y)
        outs.append(y)
    assert bro.last_device_status() == 0
    for y, (_, _, _, _, _, expect) in zip(outs, prepared):
        assert torch.equal(y.view(torch.int16), expect.view(torch.int16))
    # ... and the second problem directly against the CPU oracle, within the GEMM tolerance of the
    # other tests (fp32 criterion plus half a bf16 ulp)
    import oracle
    (M, K, N, seed, block) = cases[1]
    xb = synth.bf16_bits(synth.activations(M, K, seed=seed))
    wc_ref, ws_ref = oracle.pack_weights(synth.bf16_bits(synth.weights(N, K, seed=seed)), block)
    y_ref, S = oracle.linear(xb, block, wc_ref, ws_ref)
    got = outs[1].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - y_ref) <= 1e-5 * S + 1e-6 + np.abs(y_ref) * 2.0 ** -8)


def test_static_scratch_rejects_a_problem_that_does_not_fit(bro):
    """The size check comes before any CUDA call, so it can be exercised without a GPU."""
    buf = (ctypes.c_uint8 * 512)()
    a = (ctypes.addressof(buf) + 127) // 128 * 128
    p = ctypes.c_void_p
    M, K, N = 8192, 8192, 64                       # 32 MiB of codes alone
    rc = bro.lib.bro_linear_static(p(a), M, K, K, 32, p(a), p(a), N, p(a), N, None)
    assert rc == 5
    assert "bro_linear_static" in bro.lib.bro_last_cuda_error().decode()
    assert bro.STATIC_SCRATCH_BYTES == 16 << 20
    assert bro.lib.bro_linear_static(None, 4, 32, 32, 32, p(a), p(a), 8, p(a), 8, None) == 1
    assert bro.lib.bro_linear_static(p(a), 0, 32, 32, 32, p(a), p(a), 8, p(a), 8, None) == 0
