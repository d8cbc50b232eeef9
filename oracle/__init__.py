"""ctypes front end of the CPU oracle (``lqlora_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never imports this package, and this
package never imports the CUDA path.  The wrapper only marshals numpy arrays; all
arithmetic is in the C++ file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lqlora_oracle.cpp")
_LIB = os.path.join(_HERE, "liblqlora_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (IEEE arithmetic: no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_i64, c_int, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
        lib.oracle_nf_codebook.argtypes = [c_int, vp]
        lib.oracle_storage_bits_per_param.argtypes = [c_int] * 5
        lib.oracle_storage_bits_per_param.restype = ctypes.c_double
        lib.oracle_encode.argtypes = [vp, c_i64, c_i64, c_int, c_int, c_int, c_int, vp, vp, vp, vp]
        lib.oracle_cast_scale2.argtypes = [vp, c_i64, c_int, vp]
        lib.oracle_dequant.argtypes = [vp, vp, vp, c_i64, c_i64, c_int, c_int, c_int, c_int, vp, vp]
        lib.oracle_linear_fwd.argtypes = [vp, vp, vp, c_int, vp, c_i64, c_i64, c_i64, vp, c_i64, vp]
        lib.oracle_linear_bwd_input.argtypes = [vp, vp, vp, c_int, vp, c_i64, c_i64, c_i64, vp, c_i64, vp]
        lib.oracle_lora_grads.argtypes = [vp, vp, c_int, vp, vp, c_i64, c_i64, c_i64, vp, vp]
        lib.oracle_num_threads.restype = c_int
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(a: np.ndarray, dtype, shape=None) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def nf_codebook(b: int) -> np.ndarray:
    out = np.zeros(1 << b, dtype=np.float32)
    rc = _load().oracle_nf_codebook(b, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_nf_codebook({b}) failed")
    return out


def storage_bits_per_param(b0: int, b1: int, b2: int, B0: int, B1: int) -> float:
    return float(_load().oracle_storage_bits_per_param(b0, b1, b2, B0, B1))


def encode(A: np.ndarray, b0: int, B0: int, b1: int = 8, B1: int = 256):
    """Returns (codes [N,K] u8, absmax [nblk] f32, scale_codes [nblk] u8, scale2 [ngrp] f32)."""
    A = _chk(A, np.float32)
    N, K = A.shape
    nblk = N * K // B0
    ngrp = (nblk + B1 - 1) // B1
    codes = np.empty((N, K), dtype=np.uint8)
    absmax = np.empty(nblk, dtype=np.float32)
    sc = np.empty(nblk, dtype=np.uint8)
    v = np.empty(ngrp, dtype=np.float32)
    rc = _load().oracle_encode(_p(A), N, K, b0, B0, b1, B1, _p(codes), _p(absmax), _p(sc), _p(v))
    if rc != 0:
        raise ValueError("oracle_encode: invalid arguments")
    return codes, absmax, sc, v


def cast_scale2(v: np.ndarray, b2: int) -> np.ndarray:
    """cast(v, b2): 32 = fp32, 16 = fp16, -16 = bf16; returns the fp32 values the stored numbers decode to."""
    v = _chk(v, np.float32)
    out = np.empty_like(v)
    if _load().oracle_cast_scale2(_p(v), v.size, b2, _p(out)) != 0:
        raise ValueError("oracle_cast_scale2: invalid kind")
    return out


def dequant(codes: np.ndarray, scale_codes: np.ndarray, scale2: np.ndarray, b0: int, B0: int,
            b1: int = 8, B1: int = 256) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (deq32 [N,K] f32, deq16 [N,K] bf16 bit patterns)."""
    codes = _chk(codes, np.uint8)
    N, K = codes.shape
    sc = _chk(scale_codes, np.uint8, (N * K // B0,))
    v = _chk(scale2, np.float32)
    d32 = np.empty((N, K), dtype=np.float32)
    d16 = np.empty((N, K), dtype=np.uint16)
    rc = _load().oracle_dequant(_p(codes), _p(sc), _p(v), N, K, b0, B0, b1, B1, _p(d32), _p(d16))
    if rc != 0:
        raise ValueError("oracle_dequant: invalid arguments")
    return d32, d16


def linear_fwd(W32: np.ndarray, L1: np.ndarray, L2: np.ndarray, X: np.ndarray,
               rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Y[rows] in fp64.  W32 [N,K] f32; L1 [N,r], L2 [r,K], X [M,K] are bf16 bit patterns."""
    W32 = _chk(W32, np.float32)
    N, K = W32.shape
    X = _chk(X, np.uint16)
    M = X.shape[0]
    assert X.shape[1] == K
    r = 0 if L1 is None else L1.shape[1]
    if r:
        L1 = _chk(L1, np.uint16, (N, r))
        L2 = _chk(L2, np.uint16, (r, K))
    rows = np.arange(M, dtype=np.int64) if rows is None else _chk(rows, np.int64)
    Y = np.empty((len(rows), N), dtype=np.float64)
    rc = _load().oracle_linear_fwd(_p(W32), _p(L1) if r else None, _p(L2) if r else None, r, _p(X),
                                   M, N, K, _p(rows), len(rows), _p(Y))
    if rc != 0:
        raise ValueError("oracle_linear_fwd: invalid arguments")
    return Y


def linear_bwd_input(W32: np.ndarray, L1: np.ndarray, L2: np.ndarray, dY: np.ndarray,
                     rows: Optional[np.ndarray] = None) -> np.ndarray:
    """dX[rows] in fp64.  dY [M,N] bf16 bit patterns."""
    W32 = _chk(W32, np.float32)
    N, K = W32.shape
    dY = _chk(dY, np.uint16)
    M = dY.shape[0]
    assert dY.shape[1] == N
    r = 0 if L1 is None else L1.shape[1]
    if r:
        L1 = _chk(L1, np.uint16, (N, r))
        L2 = _chk(L2, np.uint16, (r, K))
    rows = np.arange(M, dtype=np.int64) if rows is None else _chk(rows, np.int64)
    dX = np.empty((len(rows), K), dtype=np.float64)
    rc = _load().oracle_linear_bwd_input(_p(W32), _p(L1) if r else None, _p(L2) if r else None, r,
                                         _p(dY), M, N, K, _p(rows), len(rows), _p(dX))
    if rc != 0:
        raise ValueError("oracle_linear_bwd_input: invalid arguments")
    return dX


def lora_grads(L1: np.ndarray, L2: np.ndarray, X: np.ndarray, dY: np.ndarray):
    """(dL1 [N,r], dL2 [r,K]) in fp64 for Y = X W^T + (X L2^T) L1^T: dL1 = dY^T (X L2^T), dL2 = (dY L1)^T X.
    All four inputs are bf16 bit patterns."""
    L1 = _chk(L1, np.uint16)
    L2 = _chk(L2, np.uint16)
    N, r = L1.shape
    K = L2.shape[1]
    assert L2.shape[0] == r
    X = _chk(X, np.uint16)
    dY = _chk(dY, np.uint16)
    M = X.shape[0]
    assert X.shape[1] == K and dY.shape == (M, N)
    dL1 = np.empty((N, r), dtype=np.float64)
    dL2 = np.empty((r, K), dtype=np.float64)
    rc = _load().oracle_lora_grads(_p(L1), _p(L2), r, _p(X), _p(dY), M, N, K, _p(dL1), _p(dL2))
    if rc != 0:
        raise ValueError("oracle_lora_grads: invalid arguments")
    return dL1, dL2
