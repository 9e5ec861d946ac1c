"""GPU parity for bro_rotate_fake_quantize — simulated quantisation, the way the paper evaluates the
formats (Sec. 3.1 set-up; Sec. 3.2 / Fig. 2 and Sec. 4.1 / Fig. 3 format study): the dequantised values
of the rotated activations under MXFP4, BFP4, MXINT4 and BINT4 against the CPU oracle.  Every value is
exactly representable in fp32 and both sides take their rounding decisions in fp32, so the comparison
is exact, signs of zeros included."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_04214_b200 import synth

pytestmark = pytest.mark.gpu

FORMATS = ["mxfp4", "bfp4", "mxint4", "bint4", "int4_row_sym", "int4_row_asym"]


@pytest.fixture(scope="module")
def bro():
    from paper_2511_04214_b200 import binding
    return binding


def rotated(x, block, signs=None):
    """fp32 rows of x diag(s) R_block from the oracle; block 1 is the identity (exact in fp32)."""
    if block == 1:
        y = x.float().numpy()
        return y if signs is None else y * signs.float().numpy()[None, :]
    return oracle.rotate(synth.bf16_bits(x), block, None if signs is None else synth.bf16_bits(signs))


def gpu(bro, x, block, fmt, signs=None, ldd=None):
    M, K = x.shape
    ldd = K if ldd is None else ldd
    buf = torch.full((M, ldd), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.full((bro.fake_quantize_workspace_bytes(M, fmt) + 8,), 0xAB, dtype=torch.uint8, device="cuda")   # (dirty on purpose)
    bro.rotate_fake_quantize(x.cuda(), block, buf[:, :K], fmt, None if signs is None else signs.cuda(), workspace=ws)
    assert bro.last_device_status() == 0
    out = buf.cpu().numpy()
    assert np.isnan(out[:, K:]).all()              # nothing beyond column K is written
    return out[:, :K]


def check(got, ref):
    ref32 = ref.astype(np.float32)
    assert np.array_equal(ref32.astype(np.float64), ref)          # the oracle's values are fp32 numbers
    assert np.array_equal(got.view(np.uint32), ref32.view(np.uint32))


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("block,M,K", [(1, 37, 416), (32, 37, 416), (64, 37, 448), (128, 37, 640), (32, 300, 4096),
                                       (0, 37, 512), (0, 21, 2048), (128, 130, 1024),
                                       (2, 37, 416), (4, 37, 416), (8, 37, 416), (16, 37, 416)])
def test_matches_the_oracle_exactly(bro, fmt, block, M, K):
    x = synth.activations(M, K, seed=300 + M + block)
    check(gpu(bro, x, block, fmt), oracle.fake_quantize(rotated(x, block), fmt))


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("block,K", [(1, 416), (4, 416), (16, 416), (32, 416), (128, 640), (0, 1024)])
def test_randomised_rotation(bro, fmt, block, K):
    x = synth.activations(45, K, seed=9)
    signs = synth.rotation_signs(K, seed=10)
    check(gpu(bro, x, block, fmt, signs), oracle.fake_quantize(rotated(x, block, signs), fmt))


@pytest.mark.parametrize("fmt", FORMATS)
def test_row_strides_and_untouched_padding(bro, fmt):
    M, K = 19, 384
    big = synth.activations(M, K + 64, seed=12)
    x = big[:, :K]                                  # ldx = K + 64
    xs = big.cuda()[:, :K]
    buf = torch.full((M, K + 12), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(bro.fake_quantize_workspace_bytes(M, fmt) + 8, dtype=torch.uint8, device="cuda")
    bro.rotate_fake_quantize(xs, 64, buf[:, :K], fmt, workspace=ws)
    out = buf.cpu().numpy()
    assert np.isnan(out[:, K:]).all()
    check(np.ascontiguousarray(out[:, :K]), oracle.fake_quantize(rotated(x.contiguous(), 64), fmt))


@pytest.mark.parametrize("fmt", FORMATS)
def test_degenerate_groups(bro, fmt):
    """All-zero groups, negative zeros, values below every format's smallest step, a saturating outlier."""
    K = 128
    x = torch.zeros((6, K), dtype=torch.bfloat16)
    x[1] = -0.0
    x[2, :32] = 1e-38
    x[2, 32:64] = -3e-39
    x[3, 5] = 3e38
    x[3, 40] = -2.5e38
    x[4] = torch.linspace(-6, 6, K).to(torch.bfloat16)
    x[5, ::3] = 7.0
    x[5, 1::3] = -0.26
    check(gpu(bro, x, 1, fmt), oracle.fake_quantize(rotated(x, 1), fmt))
    check(gpu(bro, x[:, :K], 32, fmt), oracle.fake_quantize(rotated(x, 32), fmt))


def test_mxfp4_agrees_with_the_codes_the_gemm_reads(bro):
    """The MXFP4 mode is the dequantisation of exactly the codes and scales bro_rotate_quantize_mxfp4 emits."""
    M, K = 64, 1024
    x = synth.activations(M, K, seed=77)
    codes = bro.alloc_codes(M, K, "cuda")
    scales = bro.alloc_scales(M, K, bro.LAYOUT_CANONICAL, "cuda")
    bro.rotate_quantize_mxfp4(x.cuda(), 32, codes, scales, bro.LAYOUT_CANONICAL)
    deq = oracle.decode(codes.cpu().numpy().reshape(M, K // 2), scales.cpu().numpy()[: M * (K // 32)].reshape(M, K // 32))
    got = gpu(bro, x, 32, "mxfp4")
    assert np.array_equal(got.astype(np.float64), np.asarray(deq, dtype=np.float64))


@pytest.mark.parametrize("block,M,K", [(1, 37, 416), (8, 37, 416), (32, 300, 1024), (128, 37, 640), (0, 37, 512), (0, 9, 4096)])
def test_no_quantisation_returns_the_rotation_itself(bro, block, M, K):
    """BRO_FMT_NONE: the fp32 rotated values, bit for bit the oracle's rotation."""
    x = synth.activations(M, K, seed=800 + block)
    signs = synth.rotation_signs(K, seed=801)
    for sg in (None, signs):
        got = gpu(bro, x, block, "none", sg)
        ref = rotated(x, block, sg)
        assert np.array_equal(got.view(np.uint32), np.ascontiguousarray(ref, dtype=np.float32).view(np.uint32))


def test_row_formats_need_their_workspace(bro):
    x = synth.activations(4, 64, seed=1).cuda()
    out = torch.empty((4, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(bro.BroError):
        bro.rotate_fake_quantize(x, 32, out, "int4_row_asym")
    with pytest.raises(bro.BroError):
        bro.rotate_fake_quantize(x, 32, out, "int4_row_sym", workspace=torch.empty(31, dtype=torch.uint8, device="cuda"))


def test_full_size_sample(bro):
    """The block-sweep tensor [16384, 4096]: every format at block 32 on sampled rows."""
    M, K = 16384, 4096
    x = synth.activations(M, K, seed=4000, recipe=synth.CFG4_RECIPE)
    rows = np.unique(np.concatenate([np.arange(0, 8), np.arange(M - 8, M), np.random.default_rng(1).integers(0, M, 48)]))
    xd = x.cuda()
    out = torch.empty((M, K), dtype=torch.float32, device="cuda")
    ws = torch.empty(8 * M, dtype=torch.uint8, device="cuda")
    for fmt in FORMATS:
        bro.rotate_fake_quantize(xd, 32, out, fmt, workspace=ws)
        got = out[torch.as_tensor(rows, device="cuda")].cpu().numpy()
        check(got, oracle.fake_quantize(rotated(x[torch.as_tensor(rows)].contiguous(), 32), fmt))
    assert bro.last_device_status() == 0
