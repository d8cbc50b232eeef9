"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host-side logic (code book, storage formula, sizes, argument validation) is right.  No kernel
is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2311_12023_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2311_12023_b200 import build
    build.build()
    from paper_2311_12023_b200 import binding as b
    return b


def test_every_declared_symbol_is_exported(binding):
    header = open(os.path.join(ROOT, "include", "lqlora.h")).read()
    declared = set(re.findall(r"\b(lqlora_[a-z0-9_]+)\s*\(", header))
    declared -= {"lqlora_status", "lqlora_config", "lqlora_qmatrix"}
    assert declared, "no declarations found"
    L = binding.lib()
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert declared == set(binding.EXPORTS) | (declared - set(binding.EXPORTS))
    for name in binding.EXPORTS:
        assert name in declared, f"{name} is bound but not declared in the header"


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_library_codebook_is_bit_identical_to_oracle(binding, b):
    # built by different quantile routines (Newton vs bisection), must agree to the last bit
    assert np.array_equal(binding.nf_codebook(b), oracle.nf_codebook(b))


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_encoder_bin_table_keeps_thresholds_away_from_bin_edges(binding, b):
    # the fast nearest-code search is exact only if no threshold sits within its 1e-6 guard band of a bin edge
    assert binding.lib().lqlora_encode_search_clearance(b) >= 1e-5


def test_storage_formula_and_packed_sizes(binding):
    for b0 in (2, 3, 4, 8):
        for B0 in (16, 32, 64, 128, 256):
            for B1 in (64, 256):
                cfg = inputs.QuantConfig(b0, B0, 8, B1, 32)
                bits = binding.storage_bits_per_param(cfg)
                assert bits == oracle.storage_bits_per_param(b0, 8, 32, B0, B1)
                N, K = 1024, 2048
                cb, sb, s2b, _ = binding.packed_sizes(N, K, cfg)
                assert (cb + sb + s2b) * 8 == bits * N * K      # Eq. (2) to the bit
    assert round(binding.storage_bits_per_param(inputs.QuantConfig(4, 64, 8, 256, 32)), 3) == 4.127
    assert round(binding.storage_bits_per_param(inputs.QuantConfig(3, 64, 8, 256, 32)), 3) == 3.127
    # rows are padded to a multiple of 128 in the packed codes only
    cb, sb, s2b, _ = binding.packed_sizes(100, 64, inputs.QuantConfig(4, 16, 8, 16, 32))
    assert cb == 128 * 64 * 4 // 8 and sb == 100 * 4 and s2b == 4 * ((400 + 15) // 16)


def test_invalid_arguments_are_rejected_before_any_launch(binding):
    L = binding.lib()
    good = inputs.QuantConfig(3, 64, 8, 256, 32)
    sz = ctypes.c_size_t(0)

    def sizes(N, K, cfg):
        c = binding._cfg(cfg)
        return L.lqlora_packed_sizes(N, K, ctypes.byref(c), ctypes.byref(sz), None, None, None)

    assert sizes(128, 128, good) == 0
    assert sizes(128, 128, inputs.QuantConfig(5, 64, 8, 256, 32)) == -1      # b0
    assert sizes(128, 128, inputs.QuantConfig(3, 48, 8, 256, 32)) == -1      # B0 not a power of two
    assert sizes(128, 128, inputs.QuantConfig(3, 64, 5, 256, 32)) == -1      # b1 not in {2, 3, 4, 8}
    assert sizes(128, 128, inputs.QuantConfig(3, 64, 8, 256, 8)) == -1       # b2 not fp32 / fp16 / bf16
    for b1 in (2, 3, 4, 8):
        for b2 in (32, 16, -16):
            assert sizes(128, 128, inputs.QuantConfig(3, 64, b1, 256, b2)) == 0
    assert sizes(128, 100, good) == -2                                       # K % 64
    assert sizes(128, 128, inputs.QuantConfig(3, 256, 8, 256, 32)) == -2     # K % B0
    assert sizes(0, 128, good) == -2

    fake = 0x10000   # never dereferenced: validation fails first
    q = binding.CQMatrix(fake, fake, fake, 128, 128, binding._cfg(good))
    ws = 1 << 30
    fwd = L.lqlora_linear_fwd
    assert fwd(None, fake, fake, 64, fake, 4, fake, fake, ws, None) == -3
    assert fwd(ctypes.byref(q), fake, fake, 64, None, 4, fake, fake, ws, None) == -3
    assert fwd(ctypes.byref(q), None, fake, 64, fake, 4, fake, fake, ws, None) == -3
    assert fwd(ctypes.byref(q), fake, fake, 24, fake, 4, fake, fake, ws, None) == -2      # r % 16
    assert fwd(ctypes.byref(q), fake, fake, 64, fake, 0, fake, fake, ws, None) == -2      # M
    assert fwd(ctypes.byref(q), fake, fake, 64, fake + 2, 4, fake, fake, ws, None) == -4  # alignment
    assert fwd(ctypes.byref(q), fake, fake, 64, fake, 4, fake, fake, 16, None) == -5      # workspace
    qbad = binding.CQMatrix(fake, fake + 1, fake, 128, 128, binding._cfg(good))
    assert L.lqlora_linear_bwd_input(ctypes.byref(qbad), fake, fake, 64, fake, 4, fake, fake, ws, None) == -4
    assert L.lqlora_encode(None, ctypes.byref(q), fake, ws, None) == -3
    assert L.lqlora_encode(fake, ctypes.byref(q), fake, 8, None) == -5
    assert binding.status_string(-7) == "device-side wait timed out"


def test_no_fallback_without_a_device(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    L = binding.lib()
    fake = 0x10000
    q = binding.CQMatrix(fake, fake, fake, 128, 128, binding._cfg(inputs.QuantConfig()))
    assert L.lqlora_unpack(ctypes.byref(q), fake, None) == -6      # LQLORA_ERR_CUDA, nothing computed


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2311_12023_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in txt and "from oracle" not in txt and "lqlora_oracle" not in txt, f
    src = open(os.path.join(ROOT, "oracle", "__init__.py")).read() + open(os.path.join(ROOT, "oracle", "lqlora_oracle.cpp")).read()
    assert "paper_2311_12023_b200" not in src and "liblqlora.so" not in src


def test_dispatch_between_the_weight_streaming_and_the_tensor_core_kernels(binding):
    """lqlora_linear_path (host only) names the kernel: up to 16 rows stream the packed weights; from 17 rows the
    one-CTA tcgen05 kernel takes over (the input gradient of 9..16 rows too when the matrix has at least 2048 rows);
    CTA pairs run once their [512, 256] tiles fill more than half of the SMs; shapes without 16-byte rows fall back
    to the plain kernels."""
    S, ONE, PAIR, PLAIN = binding.PATH_STREAM, binding.PATH_TC_ONE, binding.PATH_TC_PAIR, binding.PATH_PLAIN
    cfg = inputs.QuantConfig(3, 64, 8, 256, 32)
    for M, want in ((1, S), (16, S), (17, ONE), (256, ONE), (512, ONE), (2048, PAIR)):
        assert binding.linear_path(4096, 4096, cfg, 64, M, False) == want
    for M, want in ((1, S), (8, S), (9, ONE), (16, ONE), (17, ONE), (8192, PAIR)):
        assert binding.linear_path(4096, 4096, cfg, 64, M, True) == want
    for M, want in ((8, S), (9, S), (16, S), (17, ONE)):
        assert binding.linear_path(1024, 8192, cfg, 64, M, True) == want
    odd = inputs.QuantConfig(4, 64, 8, 16, 32)          # 201 rows: the rows of dY do not start on 16-byte boundaries
    assert binding.linear_path(201, 192, odd, 16, 1, False) == S and binding.linear_path(201, 192, odd, 16, 1, True) == PLAIN
    # the contraction of an output tile is shared by a cluster where few tiles would leave SMs idle
    kernel, splits = binding.linear_route(8192, 8192, cfg, 64, 128, False)
    assert kernel == ONE and 2 <= splits <= 8
    kernel, splits = binding.linear_route(8192, 8192, cfg, 64, 2048, False)
    assert kernel == PAIR and splits == 1
    kernel, splits = binding.linear_route(4096, 4096, cfg, 64, 1, False)
    assert kernel == S and 1 <= splits <= 8


def test_budgeted_assignment_matches_exhaustive_search(binding):
    """lqlora_assign_configs (Sec. 3.2, Algorithm 3) against the oracle's enumeration on random small instances."""
    from oracle import lq
    g = inputs.rng(123)
    for trial in range(30):
        n, m = int(g.integers(1, 6)), int(g.integers(1, 5))
        S = np.sort(g.uniform(1.0, 10.0, (n, m)), axis=1)
        E = -np.sort(-g.uniform(0.0, 5.0, (n, m)), axis=1)          # more storage, less error
        budget = float(g.uniform(S[:, 0].sum() * 0.9, S[:, -1].sum() * 1.1))
        want = lq.ilp_solve(S, E, budget)
        got = binding.assign_configs(E, S, budget)
        if want is None:
            assert got is None
            continue
        assert got is not None and got[2] <= budget + 1e-12
        assert abs(got[1] - want[1]) < 1e-12                          # same optimal error (the argmin may tie)
        assert abs(sum(E[i, a] for i, a in enumerate(got[0])) - got[1]) < 1e-12
    # non-monotone tables are handled too (a configuration that is worse in both respects is never chosen)
    S = np.array([[1.0, 2.0, 3.0]])
    E = np.array([[5.0, 7.0, 1.0]])
    assert binding.assign_configs(E, S, 2.5)[0] == [0]
    assert binding.assign_configs(E, S, 3.0)[0] == [2]
