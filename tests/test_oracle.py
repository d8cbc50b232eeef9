"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each pins one part of the oracle to
something other than itself: a library routine (scipy's normal quantile, numpy's fp64
matmul), values the paper prints (tests/golden), closed forms, constructed inputs whose
answer is known in advance, brute force on tiny inputs, and error bounds.
"""
import itertools
import os

import numpy as np
import pytest
from scipy.special import ndtri

import oracle
from paper_2311_12023_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- codebook
@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_codebook_matches_quantile_construction(b):
    """Sec. 2.2: two linspaces of probabilities, Gaussian quantiles, divide by the last."""
    cb = oracle.nf_codebook(b)
    half = 1 << (b - 1)
    delta = 0.5 * (1 / 30 + 1 / 32)
    p = np.concatenate([np.linspace(delta, 0.5, half), np.linspace(0.5, 1 - delta, half + 1)[1:]])
    assert len(p) == 1 << b                       # the shared 1/2 counted once leaves 2^b probabilities (Sec. 2.2)
    assert p[0] == delta and p[half - 1] == 0.5   # p_1 = delta, p_{2^(b-1)} = 1/2
    q = ndtri(p)
    ref = (q / q[-1]).astype(np.float32)
    ref[half - 1] = 0.0
    # independent quantile routine (scipy's rational approximation vs the oracle's bisection)
    assert np.array_equal(cb, ref)


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_codebook_invariants(b):
    cb = oracle.nf_codebook(b)
    half = 1 << (b - 1)
    assert cb[0] == np.float32(-1.0) and cb[-1] == np.float32(1.0)
    assert cb[half - 1] == 0.0
    assert np.all(np.diff(cb.astype(np.float64)) > 0)
    assert (cb < 0).sum() == half - 1 and (cb > 0).sum() == half
    # not mirror symmetric inside: one more positive value than negative
    if b < 8:
        nxt = oracle.nf_codebook(b + 1)
        # the positive half is a nested linspace: every positive value of NF_b is in NF_{b+1}
        pos, pos_n = cb[cb > 0], nxt[nxt > 0]
        for x in pos:
            assert np.min(np.abs(pos_n.astype(np.float64) - float(x))) < 1e-7


def test_codebook_known_values():
    """Spot values of the construction (delta = 0.0322916..., quantile of 1-delta = 1.8481...)."""
    cb3 = oracle.nf_codebook(3).astype(np.float64)
    # p = 1/2 + (1/2 - delta) * 1/4 -> quantile / quantile(1 - delta)
    delta = 0.5 * (1 / 30 + 1 / 32)
    assert abs(cb3[4] - ndtri(0.5 + (0.5 - delta) / 4) / ndtri(1 - delta)) < 1e-7
    assert abs(cb3[1] - ndtri(delta + (0.5 - delta) / 3) / ndtri(1 - delta)) < 1e-7
    cb8 = oracle.nf_codebook(8)
    assert cb8[127] == 0.0 and cb8[126] < 0 < cb8[128]


# --------------------------------------------------------------------------- storage
def test_storage_formula_printed_values():
    for line in open(os.path.join(GOLDEN, "storage_bits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, b0, b1, b2, B0, B1, printed = line.split()
        got = oracle.storage_bits_per_param(int(b0), int(b1), int(b2), int(B0), int(B1))
        assert round(got, 3) == float(printed), (name, got)


def test_effective_bits_printed_values():
    """2.75-bit budget + rank-64 factors stored at NF-8 = the paper's 2.95 / 2.85 bits."""
    shapes = {
        "llama2_7b": [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)],
        "llama2_70b": [(8192, 8192)] * 2 + [(1024, 8192)] * 2 + [(28672, 8192)] * 2 + [(8192, 28672)],
    }
    nf8 = oracle.storage_bits_per_param(8, 8, 32, 64, 256)
    for line in open(os.path.join(GOLDEN, "effective_bits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        model, budget, rank, printed = line.split()
        pw = sum(n * k for n, k in shapes[model])
        pl = sum(int(rank) * (n + k) for n, k in shapes[model])
        eff = (float(budget) * pw + nf8 * pl) / pw
        assert round(eff, 2) == float(printed), (model, eff)


# --------------------------------------------------------------------------- encode
def brute_force_codes(A, cb, B0):
    """argmin_i |q_i - u/s| by exhaustive search, pure Python, smallest index on ties."""
    N, K = A.shape
    out = np.zeros((N, K), dtype=np.uint8)
    zero = int(np.where(cb == 0)[0][0])
    for n in range(N):
        for k0 in range(0, K, B0):
            blk = A[n, k0:k0 + B0]
            s = np.float32(np.max(np.abs(blk)))
            for j, u in enumerate(blk):
                if s == 0:
                    out[n, k0 + j] = zero
                    continue
                x = float(np.float32(u) / s)          # fp32 quotient, then exact comparisons
                best, bestd = 0, None
                for i, q in enumerate(cb):
                    d = abs(float(q) - x)
                    if bestd is None or d < bestd:
                        best, bestd = i, d
                out[n, k0 + j] = best
    return out


@pytest.mark.parametrize("b0,B0", [(2, 16), (3, 16), (4, 32), (8, 16)])
def test_encode_brute_force_tiny(b0, B0):
    A = inputs.gaussian(7 + b0, (6, 4 * B0), 0.02)
    A[1, :B0] = 0.0                                   # an all-zero block
    A[2, 3] = 0.5                                     # an outlier
    codes, absmax, sc, v = oracle.encode(A, b0, B0, 8, 4)
    cb = oracle.nf_codebook(b0)
    assert np.array_equal(codes, brute_force_codes(A, cb, B0))
    assert np.array_equal(absmax, np.abs(A).reshape(-1, B0).max(axis=1))
    zero = (1 << (b0 - 1)) - 1
    assert np.all(codes[1, :B0] == zero)


@pytest.mark.parametrize("b0", [2, 3, 4, 8])
def test_encode_recovers_constructed_codes(b0):
    """A block built as s * q[c] (with one entry of |q| = 1) must encode back to c."""
    B0, nblk = 32, 24
    g = inputs.rng(100 + b0)
    cb = oracle.nf_codebook(b0)
    codes = g.integers(0, 1 << b0, size=(nblk, B0)).astype(np.uint8)
    codes[:, 0] = np.where(g.random(nblk) < 0.5, 0, (1 << b0) - 1)   # a -1 or +1 in each block
    s = (2.0 ** g.integers(-8, -2, size=nblk)).astype(np.float32)    # powers of two: products exact
    A = (cb[codes] * s[:, None]).astype(np.float32).reshape(4, -1)
    got, absmax, sc, v = oracle.encode(A, b0, B0, 8, 8)
    assert np.array_equal(got.reshape(nblk, B0), codes)
    assert np.array_equal(absmax, s)


@pytest.mark.parametrize("b0", [2, 3, 4, 8])
def test_encode_midpoint_ties_go_to_lower_index(b0):
    cb = oracle.nf_codebook(b0).astype(np.float64)
    B0 = 16
    rows, expect = [], []
    for i in range(len(cb) - 1):
        mid = 0.5 * (cb[i] + cb[i + 1])
        if float(np.float32(mid)) != mid:
            continue                                   # midpoint not representable in fp32
        blk = np.zeros(B0, dtype=np.float32)
        blk[0] = 1.0                                   # s = 1 so that u / s = u exactly
        blk[1] = np.float32(mid)
        blk[2] = np.nextafter(np.float32(mid), np.float32(2))    # just above -> upper code
        blk[3] = np.nextafter(np.float32(mid), np.float32(-2))   # just below -> lower code
        rows.append(blk)
        expect.append((i, i + 1, i))
    assert rows, "the midpoint next to zero is always representable"
    A = np.stack(rows)
    codes, *_ = oracle.encode(A, b0, B0, 8, 4)
    for r, (tie, up, dn) in enumerate(expect):
        assert (codes[r, 1], codes[r, 2], codes[r, 3]) == (tie, up, dn)
    assert np.all(codes[:, 0] == len(cb) - 1)


def test_encode_extreme_codes():
    A = np.zeros((1, 16), dtype=np.float32)
    A[0, 0], A[0, 1] = -3.0, 3.0
    codes, absmax, sc, v = oracle.encode(A, 4, 16, 8, 4)
    assert codes[0, 0] == 0 and codes[0, 1] == 15 and np.all(codes[0, 2:] == 7)
    assert absmax[0] == 3.0 and v[0] == 3.0 and sc[0] == 127


def test_scale_quantization_rtn_special_case():
    """Sec. 2.2 RTN: absmax values that are integer multiples of v/127 are stored exactly."""
    B0, B1 = 16, 8
    mult = np.array([127, 1, 64, 0, 100, 3, 126, 55,      # group 0, step 2^-10
                     127, 127, 2, 90, 17, 0, 5, 33,       # group 1, step 2^-6
                     9, 127, 4], dtype=np.float32)        # ragged group 2 (3 blocks), step 2^-3
    step = np.array([2.0 ** -10] * 8 + [2.0 ** -6] * 8 + [2.0 ** -3] * 3, dtype=np.float32)
    s = mult * step
    A = np.zeros((len(s), B0), dtype=np.float32)
    A[:, 5] = -s                                          # block absmax = s
    A = A.reshape(1, -1)
    codes, absmax, sc, v = oracle.encode(A, 3, B0, 8, B1)
    assert np.array_equal(absmax, s)
    assert np.array_equal(sc, mult.astype(np.uint8))
    assert np.array_equal(v, np.array([127 * 2.0 ** -10, 127 * 2.0 ** -6, 127 * 2.0 ** -3], np.float32))
    d32, d16 = oracle.dequant(codes, sc, v, 3, B0, 8, B1)
    assert np.array_equal(d32, A)                         # -1 * s recovered exactly
    assert np.array_equal(inputs.bf16_bits_to_f32(d16), A)   # these s have <= 8 significant bits


def test_scale_rounding_is_half_even_and_clamped():
    B0, B1 = 16, 4
    # sigma = 2^-7 exactly (v = 127 * 2^-7); s / sigma = 2.5, 3.5, 0.5 -> 2, 4, 0 under ties-to-even
    s = np.array([127.0, 2.5, 3.5, 0.5], dtype=np.float32) * np.float32(2.0 ** -7)
    A = np.zeros((4, B0), dtype=np.float32)
    A[:, 0] = s
    _, _, sc, _ = oracle.encode(A.reshape(1, -1), 2, B0, 8, B1)
    assert list(sc) == [127, 2, 4, 0]


def test_groups_follow_flattened_block_order_and_straddle_rows():
    """K/B0 = 3 blocks per row, B1 = 4: groups straddle rows; last group is short."""
    B0, B1, N, K = 16, 4, 3, 48
    A = np.zeros((N, K), dtype=np.float32)
    peaks = np.array([1, 2, 3, 4, 50, 6, 7, 8, 9], dtype=np.float32)   # block index 0..8
    for i, pk in enumerate(peaks):
        A.reshape(-1, B0)[i, 0] = pk
    _, absmax, sc, v = oracle.encode(A, 4, B0, 8, B1)
    assert np.array_equal(absmax, peaks)
    assert np.array_equal(v, np.array([4, 50, 9], dtype=np.float32))   # blocks 0-3, 4-7, 8
    assert sc[3] == 127 and sc[4] == 127 and sc[8] == 127
    assert sc[5] == round(6 / (50 / 127))


@pytest.mark.parametrize("b0,B0,B1", [(2, 16, 64), (3, 64, 256), (4, 64, 256), (8, 32, 64), (4, 128, 64)])
def test_encode_of_dequant_is_idempotent(b0, B0, B1):
    """Dequantization reverses quantization (Sec. 3.2): re-encoding changes nothing."""
    A = inputs.student_t(31 + b0, (24, 1024), 5.0, 0.02)
    codes, absmax, sc, v = oracle.encode(A, b0, B0, 8, B1)
    d32, _ = oracle.dequant(codes, sc, v, b0, B0, 8, B1)
    codes2, absmax2, sc2, v2 = oracle.encode(d32, b0, B0, 8, B1)
    live = np.repeat(sc > 0, B0).reshape(codes.shape)     # blocks whose scale code is 0 decode to zeros
    assert np.array_equal(codes2[live], codes[live])
    assert np.array_equal(sc2, sc)
    assert np.allclose(v2, v, rtol=3e-7, atol=0)
    d32b, _ = oracle.dequant(codes2, sc2, v2, b0, B0, 8, B1)
    assert np.allclose(d32b, d32, rtol=1e-6, atol=0)


@pytest.mark.parametrize("b0,B0,B1", [(3, 64, 256), (4, 64, 256), (2, 32, 64), (8, 16, 64)])
def test_quantization_error_bound(b0, B0, B1):
    """|w - w~| <= s * (largest half gap of the codebook) + |s - s~|, with |s - s~| <= v / 254."""
    A = inputs.gaussian(55 + b0, (16, 2048), 0.02)
    codes, absmax, sc, v = oracle.encode(A, b0, B0, 8, B1)
    d32, d16 = oracle.dequant(codes, sc, v, b0, B0, 8, B1)
    cb = oracle.nf_codebook(b0).astype(np.float64)
    halfgap = np.max(np.diff(cb)) / 2
    s = np.repeat(absmax.astype(np.float64), B0).reshape(A.shape)
    vv = np.repeat(np.repeat(v.astype(np.float64), B1)[:len(absmax)], B0).reshape(A.shape)
    bound = s * halfgap + vv / 254 + 1e-9
    assert np.all(np.abs(A.astype(np.float64) - d32) <= bound)
    # bf16 copy is the fp32 value rounded to nearest: 8 significant bits, so the relative error is at most 2^-8
    f16 = inputs.bf16_bits_to_f32(d16).astype(np.float64)
    assert np.all(np.abs(f16 - d32) <= np.abs(d32) * 2.0 ** -8 + 1e-45)
    # rounding an already-bf16 value changes nothing
    assert np.array_equal(inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(d16)), d16)


def test_dequant_elementwise_definition():
    """w~ = q[c] * (s^ * (v / 127)) written out with numpy fp32 scalars."""
    b0, B0, B1 = 3, 16, 4
    A = inputs.gaussian(77, (5, 96), 0.02)
    codes, _, sc, v = oracle.encode(A, b0, B0, 8, B1)
    d32, d16 = oracle.dequant(codes, sc, v, b0, B0, 8, B1)
    cb = oracle.nf_codebook(b0)
    flat = codes.reshape(-1)
    for idx in range(0, flat.size, 7):
        blk = idx // B0
        sigma = np.float32(v[blk // B1]) / np.float32(127)
        st = np.float32(sc[blk]) * sigma
        w = np.float32(cb[flat[idx]]) * st
        assert d32.reshape(-1)[idx] == w
        assert d16.reshape(-1)[idx] == inputs.f32_to_bf16_bits(np.array([w]))[0]


def test_dequant_bf16_rounding_ties_go_to_even():
    """The cast to bf16 (App. A) is round-to-nearest-even.  Constructed ties, with hand-written expected bit patterns:
    scale code 1 and v = 127 t make s~ = fl32(v / 127) = t exactly; the top code (q = +1) and the bottom code
    (q = -1) then dequantize to +-t.  t = 1 + 2^-8 lies half way between the bf16 values 1 (0x3F80, even mantissa)
    and 1 + 2^-7 (0x3F81); t = 1 + 3 * 2^-8 half way between 0x3F81 and 0x3F82 (even).  One ulp of fp32 above or
    below a tie must leave the tie (nearest wins)."""
    b0, B0, B1 = 3, 16, 16
    top, bottom = 7, 0
    cases = [
        (1.0 + 2.0 ** -8, 0x3F80), (1.0 + 3 * 2.0 ** -8, 0x3F82),
        (0.5 + 2.0 ** -9, 0x3F00), (0.5 + 3 * 2.0 ** -9, 0x3F02),
    ]
    for t, want in cases:
        v = np.array([127.0 * t], dtype=np.float32)
        assert float(v[0]) == 127.0 * t                  # exactly representable
        codes = np.full((1, B0), top, dtype=np.uint8)
        codes[0, 1] = bottom
        sc = np.array([1], dtype=np.uint8)
        d32, d16 = oracle.dequant(codes, sc, v, b0, B0, 8, B1)
        assert float(d32[0, 0]) == t and float(d32[0, 1]) == -t
        assert d16[0, 0] == want and d16[0, 1] == (want | 0x8000)
    # just off the tie: the nearer neighbour
    t = np.float32(1.0 + 2.0 ** -8)
    for tt, want in ((np.nextafter(t, np.float32(2)), 0x3F81), (np.nextafter(t, np.float32(0)), 0x3F80)):
        # s~ = fl32(1 * fl32(v / 127)): pick v by search so that the quotient is tt
        v = np.array([np.float32(127) * tt], dtype=np.float32)
        if np.float32(v[0] / np.float32(127)) != tt:
            continue
        codes = np.full((1, B0), top, dtype=np.uint8)
        d32, d16 = oracle.dequant(codes, np.array([1], dtype=np.uint8), v, b0, B0, 8, B1)
        assert d32[0, 0] == tt and d16[0, 0] == want


def test_cast_of_second_level_scales():
    """cast(v, b2) (Sec. 3.2, Table 1: bf16 / fp16 / fp32) against numpy's own half-precision conversion, on random
    values, exact ties, subnormals and the overflow edge; bf16 against hand-written ties; fp32 is the identity."""
    g = inputs.rng(31)
    v = np.concatenate([
        np.abs(g.standard_normal(4000)).astype(np.float32) * np.float32(0.05),
        (10.0 ** g.uniform(-9, 4.8, 4000)).astype(np.float32),
        np.array([0.0, 1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25, 65504.0, 65519.9, 65520.0,
                  6.1e-5, 5.9e-8], dtype=np.float32)])
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).astype(np.float32)
    assert np.array_equal(oracle.cast_scale2(v, 16), want)
    assert np.array_equal(oracle.cast_scale2(v, 32), v)
    b = oracle.cast_scale2(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 0.3], dtype=np.float32), -16)
    assert b[0] == 1.0 and b[1] == 1.0 + 2.0 ** -6 and b[2] == inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(np.array([0.3])))[0]
    with pytest.raises(ValueError):
        oracle.cast_scale2(v, 8)


@pytest.mark.parametrize("b1", [2, 3, 4])
def test_scale_quantization_with_fewer_bits(b1):
    """Quantize-INT with b1 bits (Table 1): levels 2^(b1-1) - 1; multiples of v / levels are stored exactly, the block
    that holds the group maximum gets the top level, everything else rounds to the nearest level."""
    levels = 2 ** (b1 - 1) - 1
    B0, B1 = 16, 16
    v = np.float32(0.75)
    step = np.float32(v / np.float32(levels))
    A = np.zeros((1, B0 * B1), dtype=np.float32)
    want = [(i % (levels + 1)) for i in range(B1)]
    want[0] = levels
    for i, lv in enumerate(want):
        A[0, i * B0] = np.float32(lv) * step
    _, absmax, sc, v2 = oracle.encode(A, 3, B0, b1, B1)
    assert v2[0] == absmax.max() and list(sc) == want
    codes = np.full((1, B0 * B1), 7, dtype=np.uint8)                 # q = +1 everywhere: w~ = s~
    d32, _ = oracle.dequant(codes, sc, v2, 3, B0, b1, B1)
    assert np.array_equal(d32[0, ::B0], np.array(want, dtype=np.float32) * np.float32(v2[0] / np.float32(levels)))


# --------------------------------------------------------------------------- layer
def _layer_case(seed, N, K, M, r):
    W = inputs.gaussian(seed, (N, K), 0.02)
    l1, l2 = inputs.lowrank_factors(seed + 1, N, K, r, 0.05)
    X = inputs.activations(seed + 2, M, K)
    dY = inputs.activations(seed + 3, M, N)
    return W, l1, l2, X, dY


def test_forward_matches_numpy_matmul():
    W, l1, l2, X, _ = _layer_case(11, 40, 96, 9, 16)
    Y = oracle.linear_fwd(W, l1, l2, X)
    Xd = inputs.bf16_bits_to_f32(X).astype(np.float64)
    L1 = inputs.bf16_bits_to_f32(l1).astype(np.float64)
    L2 = inputs.bf16_bits_to_f32(l2).astype(np.float64)
    ref = Xd @ (W.astype(np.float64) + L1 @ L2).T            # X (W + L1 L2), Sec. 2.1
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12)
    # row sampling returns those rows
    rows = np.array([8, 0, 3], dtype=np.int64)
    assert np.array_equal(oracle.linear_fwd(W, l1, l2, X, rows), Y[rows])


def test_backward_matches_numpy_matmul():
    W, l1, l2, _, dY = _layer_case(12, 40, 96, 9, 16)
    dX = oracle.linear_bwd_input(W, l1, l2, dY)
    G = inputs.bf16_bits_to_f32(dY).astype(np.float64)
    L1 = inputs.bf16_bits_to_f32(l1).astype(np.float64)
    L2 = inputs.bf16_bits_to_f32(l2).astype(np.float64)
    ref = G @ (W.astype(np.float64) + L1 @ L2)
    assert np.allclose(dX, ref, rtol=1e-12, atol=1e-12)


def test_forward_identity_rows_return_weight_columns():
    N, K, r = 24, 32, 16
    W, l1, l2, _, _ = _layer_case(13, N, K, K, r)
    X = inputs.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    Y = oracle.linear_fwd(W, l1, l2, X)
    L1 = inputs.bf16_bits_to_f32(l1).astype(np.float64)
    L2 = inputs.bf16_bits_to_f32(l2).astype(np.float64)
    assert np.allclose(Y.T, W.astype(np.float64) + L1 @ L2, rtol=0, atol=1e-15)
    # zero low-rank factors: exactly the weights; zero weights: exactly the low-rank product
    z1, z2 = np.zeros_like(l1), np.zeros_like(l2)
    assert np.array_equal(oracle.linear_fwd(W, z1, z2, X).T, W.astype(np.float64))
    assert np.allclose(oracle.linear_fwd(np.zeros_like(W), l1, l2, X).T, L1 @ L2, rtol=0, atol=1e-15)


def test_adjoint_identity():
    """<dY, fwd(X)> = <bwd_input(dY), X>: forward and input gradient are transposes."""
    W, l1, l2, X, dY = _layer_case(14, 48, 64, 7, 16)
    Y = oracle.linear_fwd(W, l1, l2, X)
    dX = oracle.linear_bwd_input(W, l1, l2, dY)
    lhs = np.sum(inputs.bf16_bits_to_f32(dY).astype(np.float64) * Y)
    rhs = np.sum(dX * inputs.bf16_bits_to_f32(X).astype(np.float64))
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))


def test_lora_grads_are_the_derivatives_of_the_forward_pass():
    """Y is linear in L1 and in L2, so for any two factor matrices
    <dY, Y(L1a, L2) - Y(L1b, L2)> = <dL1, L1a - L1b>  and  <dY, Y(L1, L2a) - Y(L1, L2b)> = <dL2, L2a - L2b>
    hold exactly; the left sides come from the forward oracle, which is pinned on its own."""
    N, K, M, r = 40, 96, 9, 16
    W, l1a, l2a, X, dY = _layer_case(21, N, K, M, r)
    l1b, l2b = inputs.lowrank_factors(2100, N, K, r, 0.05)
    G = inputs.bf16_bits_to_f32(dY).astype(np.float64)
    f = lambda b: inputs.bf16_bits_to_f32(b).astype(np.float64)
    dL1, _ = oracle.lora_grads(l1a, l2a, X, dY)           # dL1 depends on L2 only
    lhs = np.sum(G * (oracle.linear_fwd(W, l1a, l2a, X) - oracle.linear_fwd(W, l1b, l2a, X)))
    rhs = np.sum(dL1 * (f(l1a) - f(l1b)))
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
    _, dL2 = oracle.lora_grads(l1a, l2a, X, dY)           # dL2 depends on L1 only
    lhs = np.sum(G * (oracle.linear_fwd(W, l1a, l2a, X) - oracle.linear_fwd(W, l1a, l2b, X)))
    rhs = np.sum(dL2 * (f(l2a) - f(l2b)))
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
    # a dropped term, a transposed operand or a swapped factor breaks the identities: dL1 must not depend on L1
    dL1_other, dL2_other = oracle.lora_grads(l1b, l2a, X, dY)
    assert np.array_equal(dL1_other, dL1) and not np.array_equal(dL2_other, dL2)


def test_lora_grads_one_hot_closed_form():
    """X = e_a (one token, one-hot), dY = e_b:  dL1[n, j] = [n == b] L2[j, a],  dL2[j, k] = L1[b, j] [k == a]."""
    N, K, r = 24, 32, 16
    l1, l2 = inputs.lowrank_factors(2200, N, K, r, 0.05)
    a, b = 5, 17
    X = np.zeros((1, K), np.float32); X[0, a] = 1.0
    dY = np.zeros((1, N), np.float32); dY[0, b] = 1.0
    dL1, dL2 = oracle.lora_grads(l1, l2, inputs.f32_to_bf16_bits(X), inputs.f32_to_bf16_bits(dY))
    L1 = inputs.bf16_bits_to_f32(l1).astype(np.float64)
    L2 = inputs.bf16_bits_to_f32(l2).astype(np.float64)
    e1 = np.zeros((N, r)); e1[b, :] = L2[:, a]
    e2 = np.zeros((r, K)); e2[:, a] = L1[b, :]
    assert np.array_equal(dL1, e1) and np.array_equal(dL2, e2)


# --------------------------------------------------------------------------- inputs
def test_input_generators_are_seeded():
    a = inputs.gaussian(5, (8, 8), 0.02)
    assert np.array_equal(a, inputs.gaussian(5, (8, 8), 0.02))
    assert not np.array_equal(a, inputs.gaussian(6, (8, 8), 0.02))
    t = inputs.student_t(9, (256, 256), 5.0, 0.02)
    assert 0.015 < t.std() < 0.025
    specs = inputs.config_c4_draw()
    tot = sum(s.N * s.K for s in specs)
    avg = sum(oracle.storage_bits_per_param(s.cfg.b0, 8, 32, s.cfg.B0, s.cfg.B1) * s.N * s.K for s in specs) / tot
    assert 2.70 <= avg <= 2.80
    # the stored table is what the committed script (which calls only the oracle) writes
    import json
    from oracle import make_c4_draw
    with open(make_c4_draw.OUT) as f:
        assert json.load(f) == make_c4_draw.table()
    rows = inputs.sample_rows(1, 2048)
    assert len(rows) <= 64 and rows[0] == 0 and rows[-1] == 2047 and 127 in rows and 128 in rows
