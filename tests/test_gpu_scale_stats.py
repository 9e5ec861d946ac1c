"""GPU parity of the scale statistics (Sec. 4.1 regular / outlier blocks; Sec. 4.2 Fig. 6; App. A.3)
against the CPU oracle.  Integer work throughout: every byte, mask entry, histogram bin and count must
be equal."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def gpu_scale_bytes(bro, xd, block, signs=None):
    M, K = xd.shape
    out = torch.full((M, K // 32), 0xEE, dtype=torch.uint8, device="cuda")
    bro.group_scale_bytes(xd, block, out, signs=signs)
    return out


def gpu_outliers(bro, xd, ppm):
    M, K = xd.shape
    mask = torch.full((M, K // 32), 0xEE, dtype=torch.uint8, device="cuda")
    info = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(bro.outlier_workspace_bytes(), dtype=torch.uint8, device="cuda")
    bro.outlier_groups(xd, mask, info, ws, top_ppm=ppm)
    return mask, info.cpu().numpy()


@pytest.mark.parametrize("M,K", [(1, 32), (7, 160), (64, 2048), (300, 1024), (513, 2176)])
def test_scale_bytes_all_rotations(bro, M, K):
    x = synth.activations(M, K, seed=M + K)
    bits = synth.bf16_bits(x)
    xd = x.cuda()
    blocks = [1, 2, 4, 8, 16] + [b for b in (32, 64, 128) if K % b == 0] + ([0] if K & (K - 1) == 0 else [])
    for block in blocks:
        got = gpu_scale_bytes(bro, xd, block).cpu().numpy()
        assert np.array_equal(got, oracle.group_scale_bytes(bits, block)), f"block {block}"
    signs = synth.rotation_signs(K, seed=1)
    got = gpu_scale_bytes(bro, xd, 32, signs=signs.cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.group_scale_bytes(bits, 32, synth.bf16_bits(signs)))
    assert bro.last_device_status() == 0


@pytest.mark.parametrize("block", [1, 2, 8, 16, 32, 64, 128, 0])
def test_scale_bytes_with_a_sign_vector(bro, block):
    """A sign vector changes the rotated values (not their magnitudes under the identity): every rotation
    size against the oracle's randomised rotation."""
    M, K = 130, 1024
    x = synth.activations(M, K, seed=77)
    signs = synth.rotation_signs(K, seed=78)
    got = gpu_scale_bytes(bro, x.cuda(), block, signs=signs.cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.group_scale_bytes(synth.bf16_bits(x), block, synth.bf16_bits(signs)))


def test_scale_bytes_equal_the_quantisers_own(bro):
    """The analysis call and bro_rotate_quantize_mxfp4 must agree on every byte."""
    x = synth.activations(300, 1024, seed=8).cuda()
    for block in (32, 64, 128, 0):
        codes = bro.alloc_codes(300, 1024)
        scales = bro.alloc_scales(300, 1024, bro.LAYOUT_CANONICAL)
        bro.rotate_quantize_mxfp4(x, block, codes, scales, bro.LAYOUT_CANONICAL)
        assert torch.equal(gpu_scale_bytes(bro, x, block).flatten(), scales)


@pytest.mark.parametrize("ppm", [1, 1000, 50000, 1000000])
@pytest.mark.parametrize("M,K", [(40, 256), (300, 1024), (1, 32)])
def test_outlier_groups(bro, M, K, ppm):
    x = synth.activations(M, K, seed=9 + M)
    mask_ref, t_ref = oracle.outlier_groups(synth.bf16_bits(x), ppm)
    mask, info = gpu_outliers(bro, x.cuda(), ppm)
    assert int(info[0]) == t_ref
    n = M * K
    assert int(info[2]) == max(1, -(-n * ppm // 1000000))
    assert np.array_equal(mask.cpu().numpy(), mask_ref)


def test_outlier_groups_with_a_row_stride_and_ties(bro):
    base = synth.activations(50, 512, seed=4)
    base[3, 100] = 4096.0
    base[17, 300] = -4096.0                                   # a tie at the top, opposite signs
    xd = base.cuda()[:, 64:64 + 384]
    sub = base[:, 64:64 + 384].contiguous()
    mask_ref, t_ref = oracle.outlier_groups(synth.bf16_bits(sub), 1)
    mask, info = gpu_outliers(bro, xd, 1)
    assert int(info[0]) == t_ref == 0x4580
    assert np.array_equal(mask.cpu().numpy(), mask_ref) and mask.sum().item() == 2


def test_histograms_and_inflation_counts(bro):
    M, K = 512, 4096
    x = synth.activations(M, K, seed=4000, recipe=synth.CFG4_RECIPE)
    bits = synth.bf16_bits(x)
    xd = x.cuda()
    mask_ref, _ = oracle.outlier_groups(bits, 1000)
    mask, _ = gpu_outliers(bro, xd, 1000)
    assert np.array_equal(mask.cpu().numpy(), mask_ref)
    before = gpu_scale_bytes(bro, xd, 1)
    before_ref = oracle.group_scale_bytes(bits, 1)
    hist = torch.full((2, 256), -1, dtype=torch.int64, device="cuda")
    counts = torch.full((2, 3), -1, dtype=torch.int64, device="cuda")
    for block in (32, 64, 128, 0):
        after = gpu_scale_bytes(bro, xd, block)
        after_ref = oracle.group_scale_bytes(bits, block)
        bro.scale_histogram(after, mask, hist)
        bro.scale_inflation(before, after, mask, counts)
        assert np.array_equal(hist.cpu().numpy().astype(np.uint64), oracle.scale_histogram(after_ref, mask_ref))
        assert np.array_equal(counts.cpu().numpy().astype(np.uint64), oracle.scale_inflation(before_ref, after_ref, mask_ref))
    assert bro.last_device_status() == 0


def test_block_sweep_tensor_full_size_statistics(bro):
    """The whole [16384, 4096] tensor: mask and threshold against the oracle, scale bytes of every
    rotation against the oracle's, histograms and inflation counts equal."""
    cfg = synth.CONFIGS["cfg4"]
    M, K, _ = cfg["shapes"][0]
    x = synth.activations(M, K, seed=cfg["seed"], recipe=cfg["recipe"])
    bits = synth.bf16_bits(x)
    xd = x.cuda()
    mask_ref, t_ref = oracle.outlier_groups(bits, 1000)
    mask, info = gpu_outliers(bro, xd, 1000)
    assert int(info[0]) == t_ref
    assert np.array_equal(mask.cpu().numpy(), mask_ref)
    before = gpu_scale_bytes(bro, xd, 1)
    before_ref = oracle.group_scale_bytes(bits, 1)
    assert np.array_equal(before.cpu().numpy(), before_ref)
    hist = torch.empty((2, 256), dtype=torch.int64, device="cuda")
    counts = torch.empty((2, 3), dtype=torch.int64, device="cuda")
    for block in (32, 0):
        after = gpu_scale_bytes(bro, xd, block)
        after_ref = oracle.group_scale_bytes(bits, block)
        assert np.array_equal(after.cpu().numpy(), after_ref)
        bro.scale_histogram(after, mask, hist)
        bro.scale_inflation(before, after, mask, counts)
        assert np.array_equal(hist.cpu().numpy().astype(np.uint64), oracle.scale_histogram(after_ref, mask_ref))
        assert np.array_equal(counts.cpu().numpy().astype(np.uint64), oracle.scale_inflation(before_ref, after_ref, mask_ref))


def test_empty_inputs_and_argument_checks(bro):
    hist = torch.full((2, 256), 5, dtype=torch.int64, device="cuda")
    e = torch.empty(0, dtype=torch.uint8, device="cuda")
    bro.scale_histogram(e, e, hist)
    assert int(hist.abs().sum()) == 0
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((4, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(bro.BroError):
        bro.group_scale_bytes(x, 24, out)          # not a power of two
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(bro.BroError):
        bro.outlier_groups(x, out, torch.zeros(4, dtype=torch.int32, device="cuda"), ws)
