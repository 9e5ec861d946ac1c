"""Pins for the oracle's block-scaled GEMM and the whole-layer path — CPU only.

y[m,n] = sum_k deq_a[m,k] * deq_w[n,k]  (the W4A4 product of Sec. 1 / 4.2 on decoded MXFP4
operands).  Checked against numpy integer matmuls (exact special cases), one-hot selection,
an independent numpy decode + matmul, and the layer identity (x R)(W R)^T ~ x W^T.
"""
import numpy as np

import oracle
from paper_2511_04214_b200 import synth

GRID = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)


def np_decode(codes, scales):
    """Decode written out independently in numpy (from the E2M1 / E8M0 definitions)."""
    u = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    u[:, 0::2] = codes & 0xF
    u[:, 1::2] = codes >> 4
    val = GRID[u & 7] * np.where(u >> 3, -1.0, 1.0)
    return val * np.repeat(2.0 ** (scales.astype(np.float64) - 127), 32, axis=1)


def random_codes(rng, rows, K):
    return rng.integers(0, 256, size=(rows, K // 2), dtype=np.uint8)


def test_unit_scales_equal_integer_matmul():
    """All scale bytes 127 (2^0): values are half-integers, so 2a and 2w are integers and
    y = (2a)(2w)^T / 4 exactly, computed here with int64."""
    rng = np.random.default_rng(0)
    M, N, K = 9, 13, 96
    ac, wc = random_codes(rng, M, K), random_codes(rng, N, K)
    one = lambda r: np.full((r, K // 32), 127, dtype=np.uint8)
    y, S = oracle.gemm_mxfp4(ac, one(M), wc, one(N))
    a2 = (2 * np_decode(ac, one(M))).astype(np.int64)
    w2 = (2 * np_decode(wc, one(N))).astype(np.int64)
    assert np.array_equal(y, (a2 @ w2.T) / 4.0)
    assert np.array_equal(S, (np.abs(a2) @ np.abs(w2).T) / 4.0)
    assert np.all(S >= np.abs(y))


def test_scales_multiply_per_group():
    """Changing one group's scale byte of A by +3 multiplies only that group's contribution by 8."""
    rng = np.random.default_rng(1)
    M, N, K = 4, 5, 128
    ac, wc = random_codes(rng, M, K), random_codes(rng, N, K)
    asc = rng.integers(120, 134, size=(M, K // 32), dtype=np.uint8)
    wsc = rng.integers(120, 134, size=(N, K // 32), dtype=np.uint8)
    y0, _ = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    A, W = np_decode(ac, asc), np_decode(wc, wsc)
    assert np.array_equal(y0, A @ W.T) or np.allclose(y0, A @ W.T, rtol=1e-14, atol=0)
    asc2 = asc.copy()
    asc2[:, 2] += 3
    y1, _ = oracle.gemm_mxfp4(ac, asc2, wc, wsc)
    part = A[:, 64:96] @ W[:, 64:96].T
    assert np.allclose(y1 - y0, 7.0 * part, rtol=1e-12, atol=1e-12)


def test_one_hot_rows_select_single_weights():
    """A row of A with a single non-zero code picks out one decoded weight (times that code)."""
    rng = np.random.default_rng(2)
    N, K = 7, 64
    wc = random_codes(rng, N, K)
    wsc = rng.integers(100, 140, size=(N, K // 32), dtype=np.uint8)
    W = np_decode(wc, wsc)
    ac = np.zeros((K, K // 2), dtype=np.uint8)
    for k in range(K):
        ac[k, k // 2] = 0x2 << (4 * (k & 1))      # code 2 = +1.0 at position k
    asc = np.full((K, K // 32), 127, dtype=np.uint8)
    y, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    assert np.array_equal(y, W.T)
    assert np.array_equal(S, np.abs(W.T))
    # transposed operands: the product is symmetric in its roles
    y2, _ = oracle.gemm_mxfp4(wc, wsc, ac, asc)
    assert np.array_equal(y2, W)


def test_points_agree_with_full_and_with_numpy():
    x = synth.activations(40, 256, seed=31)
    w = synth.weights(24, 256, seed=32)
    ac, asc = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), 32)
    wc, wsc = oracle.pack_weights(synth.bf16_bits(w), 32)
    y, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    ref = np_decode(ac, asc) @ np_decode(wc, wsc).T
    assert np.allclose(y, ref, rtol=0, atol=1e-12 * np.abs(ref).max())
    rng = np.random.default_rng(3)
    pm = rng.integers(0, 40, size=200)
    pn = rng.integers(0, 24, size=200)
    yp, Sp = oracle.gemm_mxfp4_points(ac, asc, wc, wsc, pm, pn)
    assert np.array_equal(yp, y[pm, pn]) and np.array_equal(Sp, S[pm, pn])


def test_linear_is_rotate_quantize_then_gemm_and_tracks_the_fp_product():
    """bro_ref_linear == the two steps; and, since R R^T = I (Eq. 1), the quantised layer output
    tracks x W^T with the error expected of 4-bit operands (a loose sanity bound)."""
    x = synth.activations(32, 512, seed=41)
    w = synth.weights(48, 512, seed=42)
    for B in (32, 64, 128, 0):
        wc, wsc = oracle.pack_weights(synth.bf16_bits(w), B)
        y, S = oracle.linear(synth.bf16_bits(x), B, wc, wsc)
        ac, asc = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), B)
        y2, S2 = oracle.gemm_mxfp4(ac, asc, wc, wsc)
        assert np.array_equal(y, y2) and np.array_equal(S, S2)
        ref = x.double().numpy() @ w.double().numpy().T
        rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
        assert rel < 0.25, (B, rel)


def test_empty_problem_is_ok():
    ac = np.zeros((0, 16), dtype=np.uint8)
    asc = np.zeros((0, 1), dtype=np.uint8)
    wc = np.zeros((3, 16), dtype=np.uint8)
    wsc = np.zeros((3, 1), dtype=np.uint8)
    y, S = oracle.gemm_mxfp4(ac, asc, wc, wsc)
    assert y.shape == (0, 3)
