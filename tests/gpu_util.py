"""Helpers shared by the GPU parity tests (oracle on the host, library through the C ABI)."""
import numpy as np
import torch

import oracle
from paper_2311_12023_b200 import binding, inputs

REL_TOL = 5e-3      # ||dY||_F / ||Y||_F
MAX_TOL = 2e-2      # max |dY| / ||Y||_inf


def encode_both(A: np.ndarray, cfg):
    """Runs the oracle and the library on the same host buffer; asserts bit-exact codec parity."""
    q = binding.encode(torch.from_numpy(A).cuda(), cfg)
    codes, absmax, sc, v = oracle.encode(A, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    d32, d16 = oracle.dequant(codes, sc, v, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    return q, dict(codes=codes, sc=sc, v=v, d32=d32, d16=d16)


def assert_codec_parity(q, ref):
    got = binding.unpack(q).cpu().numpy()
    assert np.array_equal(got, ref["codes"]), f"{(got != ref['codes']).sum()} codes differ"
    assert np.array_equal(q.scale_codes.cpu().numpy(), ref["sc"])
    assert np.array_equal(q.scale2.cpu().numpy().view(np.uint32), ref["v"].view(np.uint32))
    g32, g16 = binding.dequant(q)
    assert np.array_equal(g32.cpu().numpy().view(np.uint32), ref["d32"].view(np.uint32))
    assert np.array_equal(binding.bits_from_bf16(g16), ref["d16"])


def check_close(got: np.ndarray, ref: np.ndarray, what=""):
    got = got.astype(np.float64)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    mx = np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-300)
    assert rel <= REL_TOL and mx <= MAX_TOL, f"{what}: rel {rel:.3e} max {mx:.3e}"
    return rel, mx


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()
