"""Codec variants of Table 1 (Sec. 3.2): b1 in {2, 3, 4} packed scale codes, b2 in {bf16, fp16} second-level scales, and the
layer with NF-8 quantized factors (Sec. 4.2).  Bit-exact against the oracle for the codec, tolerance parity for Y / dX."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_12023_b200 import binding, inputs
from gpu_util import check_close, to_np

pytestmark = pytest.mark.gpu

C = inputs.QuantConfig
FP16, BF16, FP32 = 16, -16, 32


def _encode_both(A, cfg):
    q = binding.encode(torch.from_numpy(A).cuda(), cfg)
    codes, _, sc, v = oracle.encode(A, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    vc = oracle.cast_scale2(v, cfg.b2)
    d32, d16 = oracle.dequant(codes, sc, vc, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    return q, dict(codes=codes, sc=sc, v=vc, d32=d32, d16=d16)


def _assert_parity(q, ref):
    assert np.array_equal(binding.unpack(q).cpu().numpy(), ref["codes"])
    sc, v = binding.unpack_scales(q)
    assert np.array_equal(sc.cpu().numpy(), ref["sc"])
    assert np.array_equal(v.cpu().numpy().view(np.uint32), ref["v"].view(np.uint32))
    g32, g16 = binding.dequant(q)
    assert np.array_equal(g32.cpu().numpy().view(np.uint32), ref["d32"].view(np.uint32))
    assert np.array_equal(binding.bits_from_bf16(g16), ref["d16"])


@pytest.mark.parametrize("b1", [2, 3, 4, 8])
@pytest.mark.parametrize("b2", [FP32, FP16, BF16])
@pytest.mark.parametrize("b0,B0,B1", [(3, 16, 16), (4, 64, 64), (2, 32, 256)])
def test_codec_variants_bit_exact(b1, b2, b0, B0, B1):
    A = inputs.student_t(40 + b1 + B0, (200, 768), 5.0, 0.02)
    A[3, :64] = 0.0
    cfg = C(b0, B0, b1, B1, b2)
    q, ref = _encode_both(A, cfg)
    _assert_parity(q, ref)
    # storage: codes + scale codes + second-level scales add up to Eq. (2) (rows padded to 128 for the codes)
    cb, sb, s2b, _ = binding.packed_sizes(256, 768, cfg)
    bits = (cb + sb + s2b) * 8 / (256 * 768)
    assert abs(bits - binding.storage_bits_per_param(cfg)) < 1e-3
    assert abs(binding.storage_bits_per_param(cfg) - oracle.storage_bits_per_param(b0, b1, abs(b2), B0, B1)) < 1e-12


def test_codec_variant_ragged_block_count():
    # 131 rows x 3 blocks per row = 393 blocks: not a multiple of eight codes; last group short
    A = inputs.gaussian(21, (131, 192), 0.02)
    q, ref = _encode_both(A, C(3, 64, 3, 16, FP16))
    _assert_parity(q, ref)


@pytest.mark.parametrize("cfg", [C(3, 64, 4, 256, BF16), C(4, 32, 3, 64, FP16), C(2, 16, 2, 16, FP32)])
@pytest.mark.parametrize("M", [3, 16, 100, 600])
def test_linear_with_variant_scales(cfg, M):
    """Every kernel family (weight-streaming, one-CTA and CTA-pair tcgen05) reads the expanded scales."""
    N, K = 1152, 1536
    A = inputs.gaussian(500 + cfg.b1, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(501, N, K, 64, 0.01)
    q, ref = _encode_both(A, cfg)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    xb, gb = inputs.activations(502 + M, M, K), inputs.activations(503 + M, M, N)
    Y = binding.linear_fwd(q, L1, L2, binding.bf16_from_bits(xb))
    dX = binding.linear_bwd_input(q, L1, L2, binding.bf16_from_bits(gb))
    check_close(to_np(Y), oracle.linear_fwd(ref["d32"], l1b, l2b, xb), f"Y M={M}")
    check_close(to_np(dX), oracle.linear_bwd_input(ref["d32"], l1b, l2b, gb), f"dX M={M}")


@pytest.mark.parametrize("M", [4, 300])
def test_layer_with_nf8_factors(M):
    """Sec. 4.2: L1 and L2 stored in NF-8 (first level 8 bits, the rest as in NF-4); the layer dequantizes them too."""
    N, K, r = 512, 1024, 64
    cfg = C(3, 64, 8, 256, 32)
    nf8 = C(8, 64, 8, 256, 32)
    A = inputs.gaussian(600, (N, K), 0.02)
    g = inputs.rng(601)
    F1 = (0.01 * g.standard_normal((N, r))).astype(np.float32)
    F2 = (0.01 * g.standard_normal((r, K))).astype(np.float32)
    q, ref = _encode_both(A, cfg)
    q1, r1 = _encode_both(F1, nf8)
    q2, r2 = _encode_both(F2, nf8)
    _assert_parity(q1, r1)
    _assert_parity(q2, r2)
    xb, gb = inputs.activations(602 + M, M, K), inputs.activations(603 + M, M, N)
    Y = binding.linear_qfactors(q, q1, q2, binding.bf16_from_bits(xb))
    dX = binding.linear_qfactors(q, q1, q2, binding.bf16_from_bits(gb), backward=True)
    # the oracle's layer with the bf16 dequantized factors
    check_close(to_np(Y), oracle.linear_fwd(ref["d32"], r1["d16"], r2["d16"], xb), f"Y M={M}")
    check_close(to_np(dX), oracle.linear_bwd_input(ref["d32"], r1["d16"], r2["d16"], gb), f"dX M={M}")
    # effective bits of the factors: 8.127 per entry (the figure behind the paper's 2.95 / 2.85 effective bits)
    assert abs(binding.storage_bits_per_param(nf8) - 8.127) < 5e-4
