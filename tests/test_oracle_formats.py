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
