"""Pins for the oracle's producer of the online-rotated activations, h = bf16(silu(gate) * up) (the
input of down_proj, where the paper's one online rotation sits: Sec. 4.3 "Reduced online computing").
The fp32 operation sequence is this build's reading; what pins it is the function it approximates
(error bound against float64), its special values, an independent bf16 rounding, and the composition
with the already-pinned rotate+quantize."""
import numpy as np
import torch

import oracle
from paper_2511_04214_b200 import synth


def bits(x32):
    return synth.bf16_bits(torch.from_numpy(np.asarray(x32, dtype=np.float32)).to(torch.bfloat16))


def as_f64(b):
    return synth.bits_to_bf16(b).double().numpy()


def test_matches_the_exact_function_within_a_few_fp32_ulps():
    rng = np.random.default_rng(0)
    g = np.concatenate([rng.standard_normal(200000) * 4, np.linspace(-100, 100, 20001), rng.standard_normal(5000) * 40])
    u = rng.standard_normal(g.size) * 3
    gb, ub = bits(g), bits(u)
    got = oracle.swiglu_f32(gb, ub).astype(np.float64)
    gg, uu = as_f64(gb), as_f64(ub)
    with np.errstate(over="ignore"):
        exact = gg / (1.0 + np.exp(-gg)) * uu
    err = np.abs(got - exact)
    # (gates below -86 are flushed: exp(-86) = 4.5e-38, so what is dropped is below 4e-36 |u|)
    assert np.all(err <= 4e-7 * np.abs(exact) + 4e-36 * np.abs(uu) + 1e-38), float(np.max(err / (np.abs(exact) + 1e-300)))


def test_every_bf16_gate_value_in_range_is_accurate_and_ordered():
    """All 2 x 32640 finite bf16 gates against float64, and monotone behaviour where silu is monotone."""
    pats = np.arange(0, 0x7F80, dtype=np.uint16)                    # +0 .. largest finite
    gb = np.concatenate([pats, pats | 0x8000]).astype(np.uint16)
    one = np.full(gb.shape, 0x3F80, dtype=np.uint16)                # up = 1
    got = oracle.swiglu_f32(gb, one).astype(np.float64)
    g = as_f64(gb)
    with np.errstate(over="ignore", under="ignore"):
        exact = g / (1.0 + np.exp(-g))
    ok = np.abs(got - exact) <= 4e-7 * np.abs(exact) + 4e-36
    assert ok.all(), (g[~ok][:5], got[~ok][:5], exact[~ok][:5])
    pos = got[: pats.size]
    assert np.all(np.diff(pos[pos > 0]) >= 0)                        # silu is increasing for g >= 0


def test_special_values():
    def one(g, u=1.0):
        return float(oracle.swiglu_f32(bits([g]), bits([u]))[0])
    assert one(0.0) == 0.0
    assert one(128.0) == 128.0 and one(1e30) == float(np.float32(bits_to_f32(bits([1e30]))))
    assert one(-128.0) == 0.0 and np.signbit(np.float32(one(-128.0)))          # g * 0 keeps the sign
    assert one(0.0, 5.0) == 0.0
    x = float(np.float32(bits_to_f32(bits([1.0]))))
    assert abs(one(1.0) - x / (1 + np.exp(-x))) < 1e-7
    assert one(2.0, -3.0) == -one(2.0, 3.0)


def bits_to_f32(b):
    return synth.bits_to_bf16(np.asarray(b, dtype=np.uint16)).float().numpy()[0]


def test_bf16_rounding_is_round_to_nearest_even():
    rng = np.random.default_rng(1)
    g, u = bits(rng.standard_normal((64, 256)) * 3), bits(rng.standard_normal((64, 256)))
    h32 = oracle.swiglu_f32(g, u).reshape(64, 256)
    h = oracle.swiglu(g, u)
    expect = synth.bf16_bits(torch.from_numpy(h32).to(torch.bfloat16))     # torch rounds to nearest even
    assert np.array_equal(h, expect)


def test_fused_entry_is_the_composition_with_rotate_quantize():
    rng = np.random.default_rng(2)
    g, u = bits(rng.standard_normal((33, 512)) * 3), bits(rng.standard_normal((33, 512)) * 2)
    signs = synth.bf16_bits(synth.rotation_signs(512, seed=3))
    for block, s in ((32, None), (64, signs), (128, None), (0, signs)):
        c, sc = oracle.swiglu_rotate_quantize_mxfp4(g, u, block, s)
        c2, sc2 = oracle.rotate_quantize_mxfp4(oracle.swiglu(g, u), block, s)
        assert np.array_equal(c, c2) and np.array_equal(sc, sc2)
