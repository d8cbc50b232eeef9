"""Bit-exact parity of lqlora_encode / lqlora_unpack / lqlora_dequant with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2311_12023_b200 import binding, inputs
from gpu_util import assert_codec_parity, encode_both

pytestmark = pytest.mark.gpu

C = inputs.QuantConfig


@pytest.mark.parametrize("b0", [2, 3, 4, 8])
@pytest.mark.parametrize("B0,B1", [(16, 64), (32, 16), (64, 256), (128, 64), (256, 256)])
def test_codec_small_all_configs(b0, B0, B1):
    # 200 rows: not a multiple of 32 or 128; K = 768 spans 3 CTA column tiles of 256
    A = inputs.student_t(10 * b0 + B0, (200, 768), 5.0, 0.02)
    A[7, 64:128] = 0.0                      # an all-zero block (for B0 <= 64)
    q, ref = encode_both(A, C(b0, B0, 8, B1, 32), check=False)
    assert_codec_parity(q, ref)


def test_codec_groups_straddle_rows_and_ragged_tail():
    # K / B0 = 3 blocks per row, B1 = 16: groups straddle rows; 131 rows * 3 = 393 blocks -> last group has 9
    A = inputs.gaussian(21, (131, 192), 0.02)
    q, ref = encode_both(A, C(3, 64, 8, 16, 32), check=False)
    assert ref["v"].shape[0] == 25
    assert_codec_parity(q, ref)


@pytest.mark.parametrize("B1", [16, 32, 128, 256, 512, 4096])
def test_codec_second_level_group_sizes(B1):
    """Every group size class of the scale quantization: runs of lanes (16, 32), two and four loads per lane (128, 256),
    one warp per group beyond that; 131 x 3 = 393 and 77 x 25 = 1925 blocks (odd counts, short last group), 3200 blocks, and
    a matrix with zero groups and huge / tiny magnitudes."""
    for shape, B0 in (((131, 192), 64), ((77, 1600), 64), ((50, 1024), 16)):
        A = inputs.gaussian_outliers(60 + B1, shape, 0.02, 0.01, 8.0)
        q, ref = encode_both(A, C(3, B0, 8, B1, 32), check=False)
        assert_codec_parity(q, ref)
    g = inputs.rng(61 + B1)
    A = (g.standard_normal((64, 1024)) * 10.0 ** g.integers(-40, 30, size=(64, 1))).astype(np.float32)
    A[7:23] = 0.0
    q, ref = encode_both(A, C(2, 16, 8, B1, 32), check=False)
    assert_codec_parity(q, ref)


def test_codec_degenerate_inputs():
    cfg = C(4, 64, 8, 256, 32)
    zero = np.zeros((64, 128), dtype=np.float32)
    q, ref = encode_both(zero, cfg, check=False)
    assert_codec_parity(q, ref)
    assert np.all(ref["codes"] == 7) and np.all(ref["sc"] == 0)
    one = np.zeros((1, 64), dtype=np.float32)       # smallest legal matrix
    one[0, 5] = -1.5
    q, ref = encode_both(one, C(2, 64, 8, 16, 32), check=False)
    assert_codec_parity(q, ref)
    # exact midpoints between neighbouring code-book values must go to the lower code
    cb = binding.nf_codebook(3).astype(np.float64)
    rows = []
    for i in range(7):
        mid = 0.5 * (cb[i] + cb[i + 1])
        blk = np.zeros(64, dtype=np.float32)
        blk[0] = 1.0
        blk[1] = np.float32(mid)
        rows.append(blk)
    q, ref = encode_both(np.stack(rows), C(3, 64, 8, 16, 32), check=False)
    assert_codec_parity(q, ref)
    # huge and tiny magnitudes, subnormal block maxima
    g = inputs.rng(5)
    A = (g.standard_normal((32, 256)) * 10.0 ** g.integers(-42, 30, size=(32, 1))).astype(np.float32)
    q, ref = encode_both(A, C(4, 32, 8, 64, 32), check=False)
    assert_codec_parity(q, ref)


@pytest.mark.parametrize("b0,B0", [(2, 16), (2, 64), (3, 16), (3, 128), (4, 64), (8, 32)])
def test_codec_values_next_to_thresholds(b0, B0):
    """The fast searches (saturating arithmetic for 2- and 3-bit codes, a bin table for 4 and 8 bits) decide from
    u * fl(1/s) and fall back to the exact quotient when that comes within a micro-unit of a midpoint: elements u = fl((mid + d) s) for every midpoint, offsets d from 0 to 3e-6 on both
    sides and random block maxima s (so that the rounding of u / s matters), plus block maxima whose reciprocal is not
    a normal number.  Codes must equal the oracle's bit for bit."""
    g = inputs.rng(40 + b0 + B0)
    cb = binding.nf_codebook(b0).astype(np.float64)
    mids = 0.5 * (cb[:-1] + cb[1:])
    offs = np.array([0.0, 1e-9, 3e-8, 6e-8, 1.2e-7, 2.4e-7, 5e-7, 8.5e-7, 9.6e-7, 1.5e-6, 3e-6])
    offs = np.concatenate([offs, -offs[1:]])
    vals = (mids[:, None] + offs[None, :]).ravel()
    rows = []
    for rep in range(96):
        s = np.float32(10.0 ** g.uniform(-3.0, 1.0))
        row = np.zeros(1024, dtype=np.float32)
        pick = g.choice(vals, size=1024)
        row[:] = (pick * np.float64(s)).astype(np.float32)
        row[::B0] = s * np.float32(1.0 if rep % 2 else -1.0)       # the block maximum itself
        rows.append(row)
    A = np.stack(rows)
    A[5, :B0] *= np.float32(1e-38)        # subnormal block maximum: no usable reciprocal
    A[6, :B0] = 0.0
    q, ref = encode_both(A, C(b0, B0, 8, 64, 32), check=False)
    assert_codec_parity(q, ref)


def test_codec_config1_roberta_proj():
    spec = inputs.workload(1)["matrices"][0]
    A, _, _ = inputs.make_matrix(spec)
    q, ref = encode_both(A, spec.cfg, check=False)
    assert_codec_parity(q, ref)


def test_codec_config2_planted_residual_full_size():
    spec = inputs.workload(2)["matrices"][0]
    A, _, _ = inputs.make_matrix(spec)
    q, ref = encode_both(A, spec.cfg, check=False)
    assert_codec_parity(q, ref)


def test_codec_config3_heavy_tailed_rectangular():
    spec = inputs.workload(3)["matrices"][0]        # 11008 x 4096, Student-t, NF4
    A, _, _ = inputs.make_matrix(spec)
    q, ref = encode_both(A, spec.cfg, check=False)
    assert_codec_parity(q, ref)


def test_codec_config4_outliers_mixed_configs():
    for spec in inputs.workload(4)["matrices"]:
        if spec.name not in ("k", "q"):             # 1024x8192 and 8192x8192 with their drawn configs
            continue
        A, _, _ = inputs.make_matrix(spec)
        q, ref = encode_both(A, spec.cfg, check=False)
        assert_codec_parity(q, ref)


@pytest.mark.parametrize("b0,B0", [(2, 16), (8, 256)])
def test_codec_config5_sweep_corners(b0, B0):
    A = inputs.gaussian(5000, (8192, 8192), 0.02)[:2048]     # a 2048-row band of the sweep matrix
    q, ref = encode_both(np.ascontiguousarray(A), C(b0, B0, 8, 256, 32), check=False)
    assert_codec_parity(q, ref)


def test_encode_is_deterministic_and_reloadable():
    A = inputs.gaussian(33, (256, 512), 0.02)
    cfg = C(3, 64, 8, 256, 32)
    q1 = binding.encode(torch.from_numpy(A).cuda(), cfg)
    q2 = binding.encode(torch.from_numpy(A).cuda(), cfg)
    assert torch.equal(q1.codes, q2.codes) and torch.equal(q1.scale_codes, q2.scale_codes)
    # a blob copied through the host dequantizes to the same bits
    q3 = binding.QMatrix(q1.codes.cpu().cuda(), q1.scale_codes.cpu().cuda(), q1.scale2.cpu().cuda(), q1.N, q1.K, cfg)
    a, b = binding.dequant(q1), binding.dequant(q3)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1].view(torch.int16), b[1].view(torch.int16))
