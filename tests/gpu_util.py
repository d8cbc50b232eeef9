"""Helpers shared by the GPU parity tests (oracle on the host, library through the C ABI)."""
import numpy as np
import torch

import oracle
from paper_2311_12023_b200 import binding, inputs

REL_TOL = 5e-3      # ||dY||_F / ||Y||_F
MAX_TOL = 2e-2      # max |dY| / ||Y||_inf


def encode_both(A: np.ndarray, cfg, check: bool = True):
    """Runs the oracle and the library on the same host buffer and asserts bit-exact codec parity (codes, scale
    codes, second-level scales, fp32 and bf16 dequantized weights) unless ``check`` is False."""
    q = binding.encode(torch.from_numpy(A).cuda(), cfg)
    codes, absmax, sc, v = oracle.encode(A, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    d32, d16 = oracle.dequant(codes, sc, v, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    ref = dict(codes=codes, sc=sc, v=v, d32=d32, d16=d16)
    if check:
        assert_codec_parity(q, ref)
    return q, ref


def _same_bits(got: torch.Tensor, ref: np.ndarray, what: str):
    """Compares on the device (the reference is uploaded): large matrices would take long to compare on the host."""
    want = torch.from_numpy(ref).to(got.device)
    if got.dtype != want.dtype:
        got = got.view(want.dtype)
    if not torch.equal(got.reshape(-1), want.reshape(-1)):
        n = int((got.reshape(-1) != want.reshape(-1)).sum().item())
        raise AssertionError(f"{what}: {n} of {want.numel()} elements differ")


def assert_codec_parity(q, ref):
    _same_bits(binding.unpack(q), ref["codes"], "codes")
    _same_bits(q.scale_codes, ref["sc"], "scale codes")
    _same_bits(q.scale2.view(torch.int32), ref["v"].view(np.int32), "second-level scales")
    g32, g16 = binding.dequant(q)
    _same_bits(g32.view(torch.int32), ref["d32"].view(np.int32), "deq32")
    del g32
    _same_bits(g16.view(torch.int16), ref["d16"].view(np.int16), "deq16")


def check_close(got: np.ndarray, ref: np.ndarray, what=""):
    got = got.astype(np.float64)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    mx = np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-300)
    assert rel <= REL_TOL and mx <= MAX_TOL, f"{what}: rel {rel:.3e} max {mx:.3e}"
    return rel, mx


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()
