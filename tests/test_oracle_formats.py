"""Pins for the oracle's comparison formats (BFP4, MXINT4, BINT4 beside MXFP4; Sec. 3.1, Fig. 2-3).
The paper names the formats without formulas, so the pins are mathematical: every dequantised
value is the nearest point of the format's own grid for the group's scale (brute force over all
codes), error bounds that follow from the grid spacing, scales that are what their format can
store, zero error on representable inputs, and agreement of format 0 with the MXFP4 quantiser."""
import numpy as np
import pytest

import oracle

E2M1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
GRIDS = {"mxfp4": E2M1, "bfp4": E2M1, "mxint4": np.arange(8) / 4.0, "bint4": np.arange(8.0)}


def rows(seed, n=64, K=128, spread=6):
    rng = np.random.default_rng(seed)
    y = rng.standard_normal((n, K)) * np.exp2(rng.integers(-spread, spread, size=(n, 1)))
    y[:, ::17] *= 9.0                                   # a few large entries per group
    return y.astype(np.float32)


def group_scale(y, fmt):
    """The scale the format must have used, recomputed here from its definition with numpy."""
    amax = np.abs(y).reshape(y.shape[0], -1, 32).max(-1)
    if fmt in ("mxfp4", "mxint4"):
        e = np.floor(np.log2(amax.astype(np.float64))) - (2 if fmt == "mxfp4" else 0)
        return np.exp2(e)
    q = np.float32(6.0 if fmt == "bfp4" else 7.0)
    return (amax / q).astype(np.float16).astype(np.float64)      # numpy: IEEE round-to-nearest-even fp16


@pytest.mark.parametrize("fmt", ["mxfp4", "bfp4", "mxint4", "bint4"])
def test_every_value_is_the_nearest_grid_point_for_the_groups_scale(fmt):
    y = rows(1)
    deq = oracle.fake_quantize(y, fmt)
    s = np.repeat(group_scale(y, fmt), 32, axis=1)
    grid = GRIDS[fmt]
    # what was stored, in units of the scale, must be a grid point with the sign of y
    q = np.abs(deq) / s
    assert np.all(np.min(np.abs(q[..., None] - grid), axis=-1) < 1e-12)
    assert np.all((deq == 0) | (np.sign(deq) == np.sign(y)))
    # and no other grid point is closer to |y| / scale (ties allowed), saturating at the top;
    # the scaled value is formed in fp32 by the oracle, hence the small slack
    r = np.abs(y).astype(np.float64) / s
    best = np.min(np.abs(r[..., None] - grid), axis=-1)
    assert np.all(np.abs(r - q) <= best + 1e-6 * (1 + r))


@pytest.mark.parametrize("fmt", ["mxfp4", "bfp4", "mxint4", "bint4"])
def test_error_bounds_from_the_grid_spacing(fmt):
    y = rows(2)
    s = np.repeat(group_scale(y, fmt), 32, axis=1)
    err = np.abs(y.astype(np.float64) - oracle.fake_quantize(y, fmt)) / s
    r = np.abs(y).astype(np.float64) / s
    if fmt in ("mxfp4", "bfp4"):
        assert np.all(err[r <= 6] <= 1.0 + 1e-6)                   # half the widest step (4 -> 6)
        assert np.all(err[r <= 2] <= 0.25 + 1e-6)
    elif fmt == "mxint4":
        assert np.all(err[r <= 1.75] <= 0.125 + 1e-6)
        assert np.all(err <= 0.25 + 1e-6)                          # r < 2 always; clipped at 1.75
    else:
        assert np.all(err <= 0.5 + 4e-3)                           # fp16 scale: amax/s is 7 within 2^-11
    if fmt == "mxfp4":
        assert r.max() < 8.0
    if fmt == "mxint4":
        assert r.max() < 2.0 and np.all(r.reshape(len(y), -1, 32).max(-1) >= 1.0)


def test_fp16_scales_map_the_group_maximum_onto_the_top_code():
    y = rows(3)
    for fmt, top in (("bfp4", 6.0), ("bint4", 7.0)):
        deq = oracle.fake_quantize(y, fmt)
        amax = np.abs(y).reshape(len(y), -1, 32).max(-1).astype(np.float64)
        dmax = np.abs(deq).reshape(len(y), -1, 32).max(-1)
        s = group_scale(y, fmt)
        assert np.allclose(dmax, top * s, rtol=0, atol=0)          # the maximum takes the top code
        assert np.all(np.abs(dmax - amax) <= amax * 2.0 ** -10)      # and is off by the fp16 rounding only


@pytest.mark.parametrize("fmt", ["mxfp4", "bfp4", "mxint4", "bint4"])
def test_representable_groups_have_no_error_and_zero_groups_stay_zero(fmt):
    rng = np.random.default_rng(4)
    grid = GRIDS[fmt]
    codes = rng.integers(0, 8, size=(16, 64))
    codes[:, 0] = 7; codes[:, 32] = 7                               # the group maximum is the top code
    signs = np.where(rng.random((16, 64)) < 0.5, -1.0, 1.0)
    scale = 0.375 if fmt in ("bfp4", "bint4") else 0.25             # exactly representable scales
    y = (signs * grid[codes] * scale).astype(np.float32)
    y[3] = 0.0
    deq = oracle.fake_quantize(y, fmt)
    assert np.array_equal(deq, y.astype(np.float64))


def test_format_0_is_the_mxfp4_quantiser_and_finer_scales_do_not_hurt():
    y = rows(5, n=128)
    c, s = oracle.quantize(y)
    assert np.array_equal(oracle.fake_quantize(y, "mxfp4"), oracle.decode(c, s))
    assert np.allclose(oracle.group_error(y, "mxfp4"), oracle.group_mse(y, c, s), rtol=1e-12, atol=0)
    # Fig. 3: with the same elements, the power-of-two scale can only be coarser than the FP16 one
    assert oracle.group_error(y, "bfp4").mean() < oracle.group_error(y, "mxfp4").mean()
    assert oracle.group_error(y, "bint4").mean() < oracle.group_error(y, "mxint4").mean()


# ---- INT4 with one scale per row (Sec. 3.2 / Fig. 2: per-channel symmetric weights, per-token asymmetric
# activations).  Pins: the symmetric form on a single group IS the pinned BINT4; both forms against a
# brute-force search over all 16 codes with the scale recomputed by numpy's float16; the error bound of a
# uniform grid; exact zeros; the asymmetric range ends on the outermost codes.
def test_row_symmetric_int4_on_one_group_is_bint4():
    y = rows(11, n=200, K=32)
    assert np.array_equal(oracle.fake_quantize(y, "int4_row_sym"), oracle.fake_quantize(y, "bint4"))


def test_row_symmetric_int4_is_the_nearest_code_for_the_rows_scale():
    y = rows(12, n=48, K=256)
    deq = oracle.fake_quantize(y, "int4_row_sym")
    s = (np.abs(y).max(1) / np.float32(7.0)).astype(np.float16).astype(np.float64)[:, None]
    k = deq / s
    assert np.all(np.abs(k - np.rint(k)) < 1e-12) and np.all(np.abs(k) <= 7)
    r = y.astype(np.float64) / s
    best = np.min(np.abs(np.clip(r, -7, 7)[..., None] - np.arange(-7, 8.0)), axis=-1)
    assert np.all(np.abs(np.clip(r, -7, 7) - k) <= best + 1e-6 * (1 + np.abs(r)))
    assert np.all(np.abs(y - deq) <= 0.5 * s * (1 + 2.0 ** -6))
    assert np.all(np.abs(deq).max(1) == 7 * s[:, 0])               # the row maximum takes the top code


def asym_params(y):
    lo = np.minimum(y.min(1), 0).astype(np.float32)
    hi = np.maximum(y.max(1), 0).astype(np.float32)
    s = ((hi - lo) / np.float32(15.0)).astype(np.float16).astype(np.float64)
    z = np.minimum(np.rint((-lo / s.astype(np.float32)).astype(np.float32).astype(np.float64)), 15)
    return lo.astype(np.float64), hi.astype(np.float64), s[:, None], z[:, None]


def test_row_asymmetric_int4_codes_and_error_bound():
    rng = np.random.default_rng(13)
    y = rows(13, n=64, K=256)
    y[8:16] = np.abs(y[8:16])                  # non-negative rows: zero point 0
    y[16:24] = -np.abs(y[16:24])               # non-positive rows: zero point 15
    y[24:32] += (rng.standard_normal((8, 1)) * 3).astype(np.float32)      # shifted rows
    deq = oracle.fake_quantize(y, "int4_row_asym")
    lo, hi, s, z = asym_params(y)
    q = deq / s + z
    assert np.all(np.abs(q - np.rint(q)) < 1e-9) and q.min() >= 0 and q.max() <= 15
    assert np.all(z[8:16] == 0) and np.all(z[16:24] == 15)
    # nearest code (brute force over the 16 codes; ties allowed), saturating at the ends
    r = y.astype(np.float64) / s + z
    best = np.min(np.abs(np.clip(r, 0, 15)[..., None] - np.arange(16.0)), axis=-1)
    assert np.all(np.abs(np.clip(r, 0, 15) - q) <= best + 1e-5 * (1 + np.abs(r)))
    # a uniform grid that covers [lo, hi] up to the rounding of scale and zero point
    assert np.all(np.abs(y - deq) <= s * (0.5 + 0.5 + 15 * 2.0 ** -11))
    inside = (r >= 0) & (r <= 15)
    assert inside.mean() > 0.97 and np.all(np.abs(y - deq)[inside] <= 0.5 * s.repeat(256, 1)[inside] * (1 + 1e-5))
    # zero is a code: exact zeros stay exact zeros, and the ends of the range land on the outermost codes
    y0 = y.copy()
    y0[:, ::5] = 0.0
    d0 = oracle.fake_quantize(y0, "int4_row_asym")
    assert np.all(d0[:, ::5] == 0.0)
    neg, pos = y.min(1) < 0, y.max(1) > 0       # (an end that is the added zero need not be attained)
    assert np.all(q.min(1)[neg] <= 1) and np.all(q.max(1)[pos] >= 14)


def test_row_formats_degenerate_rows():
    y = np.zeros((3, 64), dtype=np.float32)
    y[1] = 1e-12                                # fp16 scale underflows to zero: all zeros
    y[2, 7] = 5.0
    for fmt in ("int4_row_sym", "int4_row_asym"):
        d = oracle.fake_quantize(y, fmt)
        assert np.all(d[0] == 0) and np.all(d[1] == 0)
        assert d[2, 7] == pytest.approx(5.0, rel=2e-3) and np.count_nonzero(d[2]) == 1
