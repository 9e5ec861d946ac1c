"""Pins for the oracle's MXFP4 quantiser (Sec. 4.1: E2M1 elements, groups of 32, one E8M0
power-of-two scale; scale/rounding rule = the OCP Microscaling rule cited in Sec. 1) — CPU only.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2511_04214_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def load_grid():
    grid = {}
    with open(os.path.join(GOLDEN, "e2m1_grid.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            c, v = line.split()
            grid[int(c)] = float(v)
    return grid


def load_worked():
    rows = []
    with open(os.path.join(GOLDEN, "mx_worked_examples.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            amax, el, E, code = line.split()
            rows.append((float(amax), float(el), int(E), int(code)))
    return rows


def unpack(codes: np.ndarray) -> np.ndarray:
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = codes & 0xF
    out[..., 1::2] = codes >> 4
    return out


def test_grid_follows_from_the_format_definition():
    """The golden grid is E2M1 as the paper describes it (1 sign, 2 exponent, 1 mantissa bit):
    re-derive every value from the bit fields, then check the oracle's decoder against it."""
    grid = load_grid()
    for code in range(16):
        s, e, m = code >> 3, (code >> 1) & 3, code & 1
        val = (m * 0.5) if e == 0 else (1 + m / 2) * 2.0 ** (e - 1)
        assert grid[code] == (-val if s else val)
    codes = np.array([[c | (c << 4) for c in range(16)] * 1], dtype=np.uint8)  # [1,16] -> K=32
    for sbyte in (0, 1, 100, 127, 130, 252, 254):
        dec = oracle.decode(codes, np.array([[sbyte]], dtype=np.uint8))[0]
        for c in range(16):
            expect = grid[c] * 2.0 ** (sbyte - 127)
            assert dec[2 * c] == expect and dec[2 * c + 1] == expect
            assert np.signbit(dec[2 * c]) == bool(c >> 3)


@pytest.mark.parametrize("amax,el,E,code", load_worked())
def test_worked_examples(amax, el, E, code):
    y = np.zeros((1, 32), dtype=np.float32)
    y[0, 0] = amax
    y[0, 1] = el
    codes, scales = oracle.quantize(y)
    assert int(scales[0, 0]) - 127 == E
    assert int(unpack(codes)[0, 1]) == code
    # position must not matter: put the pair elsewhere in the group
    y2 = np.zeros((1, 32), dtype=np.float32)
    y2[0, 31] = amax
    y2[0, 18] = el
    codes2, scales2 = oracle.quantize(y2)
    assert int(scales2[0, 0]) - 127 == E
    assert int(unpack(codes2)[0, 18]) == code


def test_brute_force_nearest_grid_value():
    """For random r in [0, 8) under a scale of 1 (amax pinned to 6 -> E = 0), the chosen magnitude
    minimises |r - grid| over all eight magnitudes; ties go to the even code."""
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    rng = np.random.default_rng(0)
    r = rng.uniform(0, 6.0, size=(4096, 31)).astype(np.float32)
    # add exact ties and near-ties
    ties = np.array([.25, .75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32)
    near = np.concatenate([np.nextafter(ties, np.float32(0)), ties, np.nextafter(ties, np.float32(9))])
    r[:len(near), 0] = near
    sign = rng.integers(0, 2, size=r.shape).astype(bool)
    y = np.empty((4096, 32), dtype=np.float32)
    y[:, 0] = 6.0
    y[:, 1:] = np.where(sign, -r, r)
    codes, scales = oracle.quantize(y)
    assert np.all(scales == 127)
    got = unpack(codes)[:, 1:]
    dist = np.abs(r.astype(np.float64)[..., None] - grid)           # [rows, 31, 8]
    best = dist.min(axis=-1)
    mag = got & 7
    assert np.all(np.take_along_axis(dist, mag[..., None].astype(np.int64), -1)[..., 0] == best)
    # ties: two magnitudes at the same distance -> the even code wins
    is_tie = (dist == best[..., None]).sum(-1) == 2
    assert is_tie.sum() >= 7
    assert np.all(mag[is_tie] % 2 == 0)
    assert np.array_equal((got >> 3).astype(bool), sign)


def test_saturation_region():
    """floor (not ceil) in the shared exponent: values in (6, 8)*2^E clip to 6*2^E."""
    for E in (-20, 0, 9):
        y = np.zeros((1, 32), dtype=np.float32)
        y[0, :4] = np.array([7.99, 6.5, -7.0, 6.0], dtype=np.float32) * np.float32(2.0 ** E)
        codes, scales = oracle.quantize(y)
        assert int(scales[0, 0]) - 127 == E
        assert list(unpack(codes)[0, :4]) == [7, 7, 15, 7]
        dec = oracle.decode(codes, scales)[0, :4]
        assert list(dec) == [6 * 2.0 ** E, 6 * 2.0 ** E, -6 * 2.0 ** E, 6 * 2.0 ** E]


def test_zero_and_tiny_groups():
    """An all-zero group and a group below the E8M0 range both take the smallest scale byte (0,
    i.e. 2^-127) with no special case; the sign of a zero is kept in the code."""
    y = np.zeros((1, 64), dtype=np.float32)
    y[0, 32] = np.float32(2.0 ** -126)      # smallest normal: exponent field 1 -> clamped to 0
    y[0, 33] = -0.0
    codes, scales = oracle.quantize(y)
    assert scales[0, 0] == 0 and np.all(codes[0, :16] == 0)
    assert scales[0, 1] == 0
    u = unpack(codes)[0]
    assert u[32] == 4          # 2^-126 / 2^-127 = 2.0 -> code 4
    assert u[33] == 8          # -0.0 keeps its sign bit
    assert np.all(u[34:] == 0)


def test_roundtrip_all_grid_values_all_scales():
    """Every representable value survives quantise(decode(.)): 15 non-zero codes x scales."""
    grid = load_grid()
    for sbyte in list(range(0, 253, 7)) + [1, 2, 126, 127, 128, 251, 252]:
        E = sbyte - 127
        vals = np.zeros((1, 32), dtype=np.float64)
        vals[0, 0] = 6.0 * 2.0 ** E        # fixes the group's shared exponent at E
        for c in range(1, 16):
            vals[0, c] = grid[c] * 2.0 ** E
        if sbyte == 0:
            continue   # amax = 6*2^-127 is an fp32 subnormal whose exponent field is 0: clamp case
        y = vals.astype(np.float32)
        assert np.array_equal(y.astype(np.float64), vals)
        codes, scales = oracle.quantize(y)
        assert scales[0, 0] == sbyte
        u = unpack(codes)[0]
        assert u[0] == 7
        assert list(u[1:16]) == list(range(1, 16))


def test_idempotent_on_representable_values():
    """Q(deq(Q(y))) == Q(y): codes and scales, for every group whose largest code is 6 or 7... which
    is every non-degenerate group, because amax/2^E lies in [4, 8)."""
    x = synth.activations(64, 1024, seed=4)
    y = oracle.rotate(synth.bf16_bits(x), 32)
    codes, scales = oracle.quantize(y)
    u = unpack(codes).reshape(64, 32, 32)
    assert np.all((u & 7).max(axis=-1) >= 6)
    deq = oracle.decode(codes, scales).astype(np.float32)
    codes2, scales2 = oracle.quantize(deq)
    assert np.array_equal(codes, codes2) and np.array_equal(scales, scales2)


def test_error_bound_per_element():
    """|y - deq| <= 2^E (half the top grid step) when |y|/2^E <= 6, and <= 2*2^E in (6, 8)."""
    x = synth.activations(64, 2048, seed=6)
    for B in (32, 0):
        y = oracle.rotate(synth.bf16_bits(x), B)
        codes, scales = oracle.quantize(y)
        deq = oracle.decode(codes, scales)
        step = np.repeat(2.0 ** (scales.astype(np.float64) - 127), 32, axis=1)
        r = np.abs(y.astype(np.float64)) / step
        err = np.abs(y.astype(np.float64) - deq)
        assert np.all(r < 8.0)
        assert np.all(err[r <= 6] <= step[r <= 6])
        assert np.all(err[r > 6] <= 2 * step[r > 6])
        # and finer: inside [0,2) the grid step is 0.5 -> error <= 0.25*2^E
        fine = r <= 2
        assert np.all(err[fine] <= 0.25 * step[fine])


def test_group_and_block_independence_of_codes():
    """Perturbing one rotation block changes only that block's B/2 code bytes and B/32 scales."""
    x = synth.activations(4, 1024, seed=8)
    bits = synth.bf16_bits(x).copy()
    for B in (32, 64, 128):
        c0, s0 = oracle.rotate_quantize_mxfp4(bits, B)
        b2 = bits.copy()
        b2[:, 3 * B:4 * B] ^= 0x4000        # big exponent change in block 3
        c1, s1 = oracle.rotate_quantize_mxfp4(b2, B)
        cc = np.any(c0 != c1, axis=0)
        sc = np.any(s0 != s1, axis=0)
        assert cc[3 * B // 2:4 * B // 2].any()
        assert not cc[:3 * B // 2].any() and not cc[4 * B // 2:].any()
        assert not sc[:3 * B // 32].any() and not sc[4 * B // 32:].any()


def test_pack_weights_is_the_same_arithmetic():
    w = synth.weights(48, 512, seed=2)
    a = oracle.rotate_quantize_mxfp4(synth.bf16_bits(w), 32)
    b = oracle.pack_weights(synth.bf16_bits(w), 32)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    # and equals the two-step path rotate -> quantize
    c = oracle.quantize(oracle.rotate(synth.bf16_bits(w), 32))
    assert np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])


def test_group_mse_matches_a_numpy_restatement_and_orders_sanely():
    """The MSE arithmetic is pinned against numpy.  The ordering (block-32 rotation beats the global
    rotation on outlier-channel data, Sec. 4.2-4.3 / Fig. 6-7) is reported by the paper only as
    figures; it is checked softly here (parity unpinned by printed numbers)."""
    x = synth.activations(256, 4096, seed=4000, recipe=synth.CFG4_RECIPE)
    bits = synth.bf16_bits(x)
    mse = {}
    for B in (32, 0):
        y = oracle.rotate(bits, B)
        codes, scales = oracle.quantize(y)
        got = oracle.group_mse(y, codes, scales)
        deq = oracle.decode(codes, scales)
        ref = ((y.astype(np.float64) - deq) ** 2).reshape(256, 128, 32).mean(-1)
        assert np.allclose(got, ref, rtol=1e-12, atol=0)
        mse[B] = np.median(got)          # the typical ("regular") group
    # Global rotation spreads outlier energy into every group and inflates regular-group error;
    # block-32 rotation leaves regular groups alone.
    assert mse[32] < 0.2 * mse[0]
