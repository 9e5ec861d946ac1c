"""Pins for the oracle's scale statistics (Sec. 4.1 regular / outlier blocks; Sec. 4.2 Fig. 6: outliers
are the top 0.1 % by absolute value; App. A.3: scale growth of regular blocks under global vs block
rotation).  Everything here is integer work, pinned by brute force in numpy, by conservation, and by a
hand-built row whose answer follows from the Hadamard transform of a single spike."""
import numpy as np
import pytest

import oracle
from paper_2511_04214_b200 import synth


def bits_of(x32: np.ndarray) -> np.ndarray:
    import torch
    return synth.bf16_bits(torch.from_numpy(np.asarray(x32, dtype=np.float32)).to(torch.bfloat16))


def test_identity_rotation_gives_the_inputs_own_scale_bytes():
    """block = 1 is the identity: the byte must be floor(log2 amax) - 2 + 127 of the raw group."""
    x = synth.activations(16, 512, seed=3)
    s = oracle.group_scale_bytes(synth.bf16_bits(x), 1)
    amax = np.abs(x.float().numpy()).reshape(16, 16, 32).max(-1)
    _, e = np.frexp(amax)                       # amax = f * 2^e, f in [0.5, 1) -> floor(log2) = e - 1
    expect = np.where(amax > 0, np.maximum((e - 1) - 2 + 127, 0), 0)
    assert np.array_equal(s, expect.astype(np.uint8))
    # and the identity rotation really is the identity
    assert np.array_equal(oracle.rotate(synth.bf16_bits(x), 1), x.float().numpy())


@pytest.mark.parametrize("ppm", [1000, 1, 50000, 1000000])
def test_outlier_threshold_is_the_kth_largest_magnitude(ppm):
    x = synth.activations(40, 256, seed=9)
    bits = synth.bf16_bits(x)
    mask, t = oracle.outlier_groups(bits, ppm)
    a = np.abs(x.float().numpy())
    n = a.size
    k = max(1, -(-n * ppm // 1000000))
    kth = np.sort(a.ravel())[::-1][k - 1]
    t_val = synth.bits_to_bf16(np.array([t], dtype=np.uint16)).float().numpy()[0]
    assert t_val == kth
    assert (a >= kth).sum() >= k                       # ties at the threshold all count
    expect = (a.reshape(40, 8, 32) >= kth).any(-1)
    assert np.array_equal(mask.astype(bool), expect)
    if ppm == 1000000:
        assert mask.all()


def test_outlier_mask_ignores_the_sign_and_respects_ties():
    x = np.ones((2, 64), dtype=np.float32)
    x[0, 5] = -8.0
    x[1, 40] = 8.0                                         # a tie at the top
    mask, t = oracle.outlier_groups(bits_of(x), 1)         # k = 1
    assert t == 0x4100                                     # bf16(8.0)
    assert mask.tolist() == [[1, 0], [0, 1]]


def test_histograms_count_every_group_once_and_split_by_class():
    x = synth.activations(64, 1024, seed=5)
    bits = synth.bf16_bits(x)
    mask, _ = oracle.outlier_groups(bits, 1000)
    for block in (1, 32, 0):
        s = oracle.group_scale_bytes(bits, block)
        h = oracle.scale_histogram(s, mask)
        assert h.sum() == s.size
        assert h[1].sum() == int(mask.sum())
        for c in (0, 1):
            assert np.array_equal(h[c], np.bincount(s[mask == c].ravel(), minlength=256).astype(np.uint64))


def test_inflation_counts_match_a_numpy_restatement_and_conserve():
    x = synth.activations(64, 1024, seed=6)
    bits = synth.bf16_bits(x)
    mask, _ = oracle.outlier_groups(bits, 1000)
    before = oracle.group_scale_bytes(bits, 1)
    for block in (32, 128, 0):
        after = oracle.group_scale_bytes(bits, block)
        c = oracle.scale_inflation(before, after, mask)
        assert c.sum() == before.size
        for cls in (0, 1):
            sel = mask == cls
            b, a = before[sel].astype(int), after[sel].astype(int)
            assert c[cls].tolist() == [(a < b).sum(), (a == b).sum(), (a > b).sum()]
    same = oracle.scale_inflation(before, before, mask)
    assert same[:, 0].sum() == 0 and same[:, 2].sum() == 0


def test_one_outlier_channel_inflates_every_group_globally_but_only_its_own_block_locally():
    """A row of small values with one large spike.  The Hadamard transform spreads the spike evenly
    over the block it sits in (|H_ij| = 1): under the full-dimension rotation every group of the row
    receives spike/sqrt(K), far above the background, so every regular group's scale byte rises;
    under the block-32 rotation only the spike's own group changes.  This is the mechanism of
    Sec. 4.2 / App. A.3 in its simplest form."""
    K = 1024
    rng = np.random.default_rng(0)
    x = (rng.standard_normal((1, K)) * 0.01).astype(np.float32)
    x[0, 70] = 1024.0                                       # group 2
    bits = bits_of(x)
    mask, _ = oracle.outlier_groups(bits, 1000)             # k = ceil(1024 * 0.001) = 2 -> the spike + one more
    assert mask[0, 2] == 1
    before = oracle.group_scale_bytes(bits, 1)
    glob = oracle.group_scale_bytes(bits, 0)
    blk = oracle.group_scale_bytes(bits, 32)
    others = np.arange(K // 32) != 2
    assert (glob[0, others] > before[0, others]).all()      # 1024 / 32 = 32 >> 0.01 everywhere
    assert np.all(np.abs(blk[0, others].astype(int) - before[0, others].astype(int)) <= 3)   # sqrt(32)-scale mixing of noise only
    assert blk[0, 2] < before[0, 2]                          # the spike's own group: 1024 -> 1024 / sqrt(32)
    # the spread value is spike / sqrt(K) = 32 -> floor(log2 32) - 2 + 127 = 130 in every group
    assert (glob[0] == 130).all()
    c_glob = oracle.scale_inflation(before, glob, mask)
    regular = int((mask == 0).sum())
    assert c_glob[0].tolist() == [0, 0, regular]


def test_qualitative_ordering_on_synthetic_activations_is_soft():
    """Not a pin (the paper gives figures, not numbers): with 1 % outlier channels the fraction of
    regular groups whose scale rises is larger for the full-dimension rotation than for block 32."""
    x = synth.activations(256, 4096, seed=4000, recipe=synth.CFG4_RECIPE)
    bits = synth.bf16_bits(x)
    mask, _ = oracle.outlier_groups(bits, 1000)
    before = oracle.group_scale_bytes(bits, 1)
    up = {}
    for block in (32, 0):
        c = oracle.scale_inflation(before, oracle.group_scale_bytes(bits, block), mask)
        up[block] = c[0, 2] / c[0].sum()
    assert up[0] > up[32]
