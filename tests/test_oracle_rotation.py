"""Pins for the oracle's rotation (Eq. 1 with Hadamard blocks) — CPU only.

Each test checks the oracle against something fixed by the paper or by mathematics, never
against the oracle's own formula: orthogonality and norm preservation (Eq. 1, Sec. 4.2), exact
inversion, closed forms, an independent O(B^2) definition of the Sylvester matrix, block
independence (Sec. 4.3) and the reduction of block = K to the global rotation.
"""
import numpy as np
import pytest

import oracle
from paper_2511_04214_b200 import synth


def to_bits(a: np.ndarray) -> np.ndarray:
    """fp32 array of bf16-representable values -> uint16 bf16 bit patterns (exactness asserted)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "test input must be exactly representable in bf16"
    return (u >> 16).astype(np.uint16)


def sylvester(B: int) -> np.ndarray:
    """H[i][j] = (-1)^popcount(i & j): the textbook definition, no recursion, no fast transform."""
    i = np.arange(B, dtype=np.uint32)[:, None]
    j = np.arange(B, dtype=np.uint32)[None, :]
    v = i & j
    parity = np.zeros_like(v)
    for bit in range(32):
        parity ^= (v >> np.uint32(bit)) & np.uint32(1)
    return np.where(parity == 0, 1.0, -1.0)


def small_int_rows(rng, M, K, lo=-8, hi=8):
    return rng.integers(lo, hi + 1, size=(M, K)).astype(np.float32)


@pytest.mark.parametrize("B,bits", [(32, 0x3E3504F3), (64, 0x3E000000), (128, 0x3DB504F3),
                                    (4096, 0x3C800000), (2, 0x3F3504F3), (4, 0x3F000000)])
def test_norm_constant_is_nearest_fp32(B, bits):
    c = oracle.hadamard_norm(B)
    assert np.float32(c).view(np.uint32) == bits
    # nearest: |c - 1/sqrt(B)| is no larger than for either fp32 neighbour
    exact = 1.0 / np.sqrt(np.float64(B))
    lo = np.nextafter(np.float32(c), np.float32(0))
    hi = np.nextafter(np.float32(c), np.float32(1))
    assert abs(float(c) - exact) <= abs(float(lo) - exact)
    assert abs(float(c) - exact) <= abs(float(hi) - exact)


@pytest.mark.parametrize("B", [32, 64, 128])
def test_orthogonality(B):
    """Rows of the rotation matrix, obtained by rotating unit vectors, satisfy R R^T = I (Eq. 1)."""
    eye = np.eye(B, dtype=np.float32)
    R = oracle.rotate(to_bits(eye), B).astype(np.float64)
    tol = 0.0 if B == 64 else 1e-6
    assert np.max(np.abs(R @ R.T - np.eye(B))) <= tol
    # symmetric Hadamard: applying the rotation to e_j gives column j = row j
    assert np.array_equal(R, R.T)


@pytest.mark.parametrize("B", [32, 64, 128, 0])
def test_norm_preserved(B):
    """Rotation does not change the L2 norm of a token (Sec. 4.2)."""
    x = synth.activations(16, 1024, seed=11)
    y = oracle.rotate(synth.bf16_bits(x), B).astype(np.float64)
    n0 = np.linalg.norm(x.double().numpy(), axis=1)
    n1 = np.linalg.norm(y, axis=1)
    assert np.max(np.abs(n1 - n0) / n0) < 1e-5


def test_exact_inversion_B64():
    """H/sqrt(B) is an involution.  With B = 64 (c = 1/8 exactly) and inputs in {-1, 0, 1} every
    intermediate is a small multiple of 1/8, so no operation rounds and rotating twice returns
    the input bit for bit."""
    rng = np.random.default_rng(5)
    x = small_int_rows(rng, 8, 256, -1, 1)
    y = oracle.rotate(to_bits(x), 64)          # multiples of 1/8, |y| <= 8: exact in bf16
    back = oracle.rotate(to_bits(y), 64)
    assert np.array_equal(back, x)


@pytest.mark.parametrize("B", [32, 64, 128])
def test_closed_forms(B):
    """x = c e_j  ->  |y_i| = |c|/sqrt(B) with the signs of column j of the Sylvester matrix;
    x = c 1  ->  y_0 = c sqrt(B), all other outputs exactly zero."""
    H = sylvester(B)
    cB = np.float64(oracle.hadamard_norm(B))
    for j in (0, 1, 5, B - 1):
        x = np.zeros((1, B), dtype=np.float32)
        x[0, j] = 3.0
        y = oracle.rotate(to_bits(x), B)[0].astype(np.float64)
        assert np.array_equal(y, np.float32(3.0 * cB).astype(np.float64) * H[:, j])
    ones = np.full((1, B), 2.0, dtype=np.float32)
    y = oracle.rotate(to_bits(ones), B)[0].astype(np.float64)
    assert y[0] == np.float64(np.float32(np.float32(2.0 * B) * np.float32(cB)))
    assert np.all(y[1:] == 0.0)
    assert abs(y[0] - 2.0 * np.sqrt(B)) < 1e-5


@pytest.mark.parametrize("B", [32, 64, 128, 256])
def test_matches_quadratic_definition_exactly_on_integers(B):
    """Fast transform == the O(B^2) sum with (-1)^popcount(i&j).  On small integers no fp32
    operation rounds before the final multiply, so equality is exact."""
    rng = np.random.default_rng(B)
    x = small_int_rows(rng, 6, 2 * B, -4, 4)
    y = oracle.rotate(to_bits(x), B)
    H = sylvester(B)
    c = oracle.hadamard_norm(B)
    for blk in range(2):
        ref = x[:, blk * B:(blk + 1) * B].astype(np.float64) @ H.T   # exact integers
        expect = (ref.astype(np.float32) * np.float32(c)).astype(np.float32)
        assert np.array_equal(y[:, blk * B:(blk + 1) * B], expect)


@pytest.mark.parametrize("B", [32, 128])
def test_matches_quadratic_definition_on_random_data(B):
    x = synth.activations(4, 4 * B, seed=3)
    y = oracle.rotate(synth.bf16_bits(x), B).astype(np.float64)
    H = sylvester(B) / np.sqrt(B)
    xd = x.double().numpy()
    for blk in range(4):
        ref = xd[:, blk * B:(blk + 1) * B] @ H.T
        err = np.abs(y[:, blk * B:(blk + 1) * B] - ref)
        scale = np.abs(xd[:, blk * B:(blk + 1) * B]).sum(axis=1, keepdims=True) / np.sqrt(B)
        assert np.all(err <= 1e-6 * scale + 1e-30)


def test_block_independence():
    """Each block is rotated on its own (Sec. 4.3): perturbing one block of x changes only that
    block of the output."""
    x = synth.activations(3, 512, seed=9)
    bits = synth.bf16_bits(x).copy()
    y0 = oracle.rotate(bits, 64)
    bits2 = bits.copy()
    bits2[:, 128:192] ^= 0x0040      # flip a mantissa bit in block 2 only
    y1 = oracle.rotate(bits2, 64)
    changed = np.any(y0 != y1, axis=0)
    assert changed[128:192].any()
    assert not changed[:128].any() and not changed[192:].any()


def test_block_equal_K_is_global_rotation():
    """block = 0 (B = K) is one K-point transform: it equals the O(K^2) definition, and B = 32
    on the same data equals K/32 independent 32-point transforms."""
    K = 4096
    rng = np.random.default_rng(1)
    x = small_int_rows(rng, 2, K, -2, 2)
    yg = oracle.rotate(to_bits(x), 0)
    assert np.array_equal(yg, oracle.rotate(to_bits(x), K))
    H = sylvester(K)
    ref = (x.astype(np.float64) @ H.T).astype(np.float32) * np.float32(2.0 ** -6)
    assert np.array_equal(yg, ref)
    y32 = oracle.rotate(to_bits(x), 32)
    for blk in range(0, K, 32 * 17):       # a few blocks
        sub = oracle.rotate(to_bits(x[:, blk:blk + 32]), 32)
        assert np.array_equal(y32[:, blk:blk + 32], sub)


def test_rotation_invariance_of_the_product():
    """(x R)(W R)^T = x W^T before quantisation (R R^T = I, Eq. 1): both operands must be rotated
    on the K axis by the same matrix."""
    x = synth.activations(8, 512, seed=21)
    w = synth.weights(16, 512, seed=22)
    for B in (32, 64, 128, 0):
        xr = oracle.rotate(synth.bf16_bits(x), B).astype(np.float64)
        wr = oracle.rotate(synth.bf16_bits(w), B).astype(np.float64)
        ref = x.double().numpy() @ w.double().numpy().T
        got = xr @ wr.T
        denom = np.abs(x.double().numpy()) @ np.abs(w.double().numpy()).T
        assert np.max(np.abs(got - ref) / denom) < 1e-6


def test_bad_arguments_rejected():
    x = np.zeros((2, 96), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.rotate(x, 64)          # 96 % 64 != 0
    with pytest.raises(ValueError):
        oracle.rotate(x, 0)           # global needs a power-of-two K
    with pytest.raises(ValueError):
        oracle.rotate(x, 48)          # not a power of two


# ---- randomised block rotation: R_i = diag(s) H / sqrt(B)  (Sec. 5.1) ---------------------------
def sign_bits(rng, K):
    s = np.where(rng.random(K) < 0.5, 1.0, -1.0).astype(np.float32)
    return s, to_bits(s)


@pytest.mark.parametrize("B", [32, 64, 128])
def test_randomised_rotation_is_orthogonal_and_is_diag_s_times_hadamard(B):
    rng = np.random.default_rng(B)
    s, sb = sign_bits(rng, B)
    R = oracle.rotate(to_bits(np.eye(B, dtype=np.float32)), B, sb).astype(np.float64)   # rows e_j R
    tol = 0.0 if B == 64 else 1e-6
    assert np.max(np.abs(R @ R.T - np.eye(B))) <= tol                                 # Eq. 1
    expect = np.diag(s.astype(np.float64)) @ sylvester(B) / np.sqrt(B)
    assert np.max(np.abs(R - expect)) <= 1e-7


def test_randomised_rotation_equals_plain_rotation_of_sign_flipped_input():
    """x diag(s) is exact in bf16, so rotating with signs must equal, bit for bit, the plain rotation
    of an input that was negated channel by channel beforehand (done here in numpy)."""
    rng = np.random.default_rng(5)
    K = 256
    x = synth.activations(9, K, seed=3).float().numpy()
    s, sb = sign_bits(rng, K)
    for B in (32, 128, 0):
        a = oracle.rotate(to_bits(x), B, sb)
        b = oracle.rotate(to_bits(x * s[None, :]), B)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    allplus = to_bits(np.ones(K, dtype=np.float32))
    assert np.array_equal(oracle.rotate(to_bits(x), 32, allplus), oracle.rotate(to_bits(x), 32))
    # only the sign bit of the sign vector counts
    assert np.array_equal(oracle.rotate(to_bits(x), 32, to_bits(s * 3.0)), oracle.rotate(to_bits(x), 32, sb))


def test_randomised_rotation_leaves_the_unquantised_product_unchanged():
    """(x R)(W R)^T = x W^T for the same sign vector on both operands; with different sign vectors
    it is not (a plausible mistake: signs applied to one side only)."""
    rng = np.random.default_rng(8)
    M, N, K = 5, 7, 128
    x = small_int_rows(rng, M, K)
    w = small_int_rows(rng, N, K)
    s, sb = sign_bits(rng, K)
    xr = oracle.rotate(to_bits(x), 32, sb).astype(np.float64)
    wr = oracle.rotate(to_bits(w), 32, sb).astype(np.float64)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.max(np.abs(xr @ wr.T - ref)) <= 1e-4 * np.max(np.abs(ref))
    w_plain = oracle.rotate(to_bits(w), 32).astype(np.float64)
    assert np.max(np.abs(xr @ w_plain.T - ref)) > 1e-2 * np.max(np.abs(ref))


def test_randomised_quantisation_uses_the_rotated_values():
    x = synth.activations(6, 128, seed=12)
    sb = synth.bf16_bits(synth.rotation_signs(128, seed=1))
    y = oracle.rotate(synth.bf16_bits(x), 64, sb)
    c1, s1 = oracle.quantize(y)
    c2, s2 = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), 64, sb)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
    c3, _ = oracle.rotate_quantize_mxfp4(synth.bf16_bits(x), 64)
    assert not np.array_equal(c1, c3)
    c4, s4 = oracle.pack_weights(synth.bf16_bits(x), 64, sb)
    assert np.array_equal(c4, c2) and np.array_equal(s4, s2)
