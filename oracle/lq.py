"""CPU oracle of the matrix decomposition and of the configuration search (test infrastructure only).

Plain numpy fp64 restatement of Algorithms 2-4 and of the integer program of Sec. 3.2 of arXiv 2311.12023, in the
paper's orientation (W is d x k, L1 is d x r, L2 is r x k).  ``Quantize`` is the oracle's own Quantize / dequantize
(``oracle.encode`` / ``oracle.dequant``); the SVD is numpy's.  Nothing here is tuned and nothing is shared with the
CUDA path.  Only tests, ``__graft_entry__.smoke()`` and ``bench.py``'s baseline leg may import this module.

Readings (the paper is silent or ambiguous):
  * Algorithm 2 breaks when the error rises and prints the current iterate as its output; Sec. 3.1 says the algorithm
    terminates "if the error increases".  Taken here: the iterate with the smaller error (the one before the rise) is
    returned, with the whole error history beside it.
  * Quantize takes the fp32 rounding of W - L1 L2 (the quantizer's input type); Q is its fp32 dequantized value.
  * T (the iteration cap) is a parameter; the paper gives no value.
"""
from __future__ import annotations

import itertools
from typing import List, Optional, Sequence, Tuple

import numpy as np

import oracle


def factorize(A: np.ndarray, r: int, F: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 4 (Sec. 3.3, Eq. (4)).  Without F: L1 = U sqrt(S), L2 = sqrt(S) V^T of the rank-r truncated SVD.
    With F: D_row / D_col = row / column means of sqrt(F); SVD of D_row A D_col; L1 = D_row^-1 U sqrt(S),
    L2 = sqrt(S) V^T D_col^-1."""
    A = np.asarray(A, dtype=np.float64)
    if F is None:
        U, S, Vt = np.linalg.svd(A, full_matrices=False)
        sq = np.sqrt(S[:r])
        return U[:, :r] * sq[None, :], sq[:, None] * Vt[:r, :]
    rootF = np.sqrt(np.asarray(F, dtype=np.float64))
    d_row = rootF.mean(axis=1)
    d_col = rootF.mean(axis=0)
    U, S, Vt = np.linalg.svd(d_row[:, None] * A * d_col[None, :], full_matrices=False)
    sq = np.sqrt(S[:r])
    L1 = (U[:, :r] * sq[None, :]) / d_row[:, None]
    L2 = (sq[:, None] * Vt[:r, :]) / d_col[None, :]
    return L1, L2


def quantize(A: np.ndarray, cfg) -> np.ndarray:
    """Quantize(A, c) followed by dequantization: the member of the quantizable set that A is mapped to (fp32 values)."""
    b0, B0, b1, B1 = cfg.b0, cfg.B0, cfg.b1, cfg.B1
    A32 = np.ascontiguousarray(A, dtype=np.float32)
    codes, _, sc, v = oracle.encode(A32, b0, B0, b1, B1)
    d32, _ = oracle.dequant(codes, sc, v, b0, B0, b1, B1)
    return d32


def weighted_norm(E: np.ndarray, F: Optional[np.ndarray]) -> float:
    """|| E ||_F, or || sqrt(F) o E ||_F (Eq. (3))."""
    E = np.asarray(E, dtype=np.float64)
    if F is None:
        return float(np.sqrt(np.sum(E * E)))
    return float(np.sqrt(np.sum(np.asarray(F, dtype=np.float64) * E * E)))


def lq_decompose(W: np.ndarray, cfg, r: int, F: Optional[np.ndarray] = None, T: int = 20):
    """Algorithm 2: Q <- 0; repeat (L1, L2 <- Factorize(W - Q, F, r); Q <- Quantize(W - L1 L2, c); error) until the
    error rises or T steps are done.  Returns (Q fp32, L1, L2, error, history, steps_taken)."""
    W = np.asarray(W, dtype=np.float64)
    Q = np.zeros_like(W)
    best = None
    history: List[float] = []
    prev = np.inf
    for _ in range(T):
        L1, L2 = factorize(W - Q, r, F)
        Qn = quantize(W - L1 @ L2, cfg).astype(np.float64)
        err = weighted_norm(W - (Qn + L1 @ L2), F)
        history.append(err)
        if err > prev:
            break
        best = (Qn.astype(np.float32), L1, L2, err)
        Q, prev = Qn, err
    assert best is not None
    return best + (history, len(history))


def storage_bits(shape: Sequence[int], cfg) -> float:
    """storage(A, c) = sizeof(A) * (b0 + b1 / B0 + b2 / (B0 B1))   (Eq. (2))."""
    return float(shape[0]) * float(shape[1]) * oracle.storage_bits_per_param(cfg.b0, cfg.b1, cfg.b2, cfg.B0, cfg.B1)


def error_storage_tables(Ws, configs, r: int, Fs=None, T: int = 20):
    """Algorithm 3, first part: E[i, c] = error^2 of LQ(W_i, F_i, c, r), S[i, c] = storage(W_i, c)."""
    E = np.zeros((len(Ws), len(configs)))
    S = np.zeros((len(Ws), len(configs)))
    for i, W in enumerate(Ws):
        for j, c in enumerate(configs):
            F = None if Fs is None else Fs[i]
            err = lq_decompose(W, c, r, F, T)[3]
            E[i, j] = err * err
            S[i, j] = storage_bits(W.shape, c)
    return E, S


def ilp_solve(S: np.ndarray, E: np.ndarray, budget: float):
    """The integer program of Sec. 3.2 by exhaustive enumeration (small instances only): one configuration per matrix,
    total storage <= budget, minimal total error.  Ties go to the lexicographically first assignment.  Returns
    (assignment, total error, total storage) or None when nothing fits."""
    n, m = S.shape
    best = None
    for assign in itertools.product(range(m), repeat=n):
        st = sum(S[i, a] for i, a in enumerate(assign))
        if st > budget:
            continue
        er = sum(E[i, a] for i, a in enumerate(assign))
        if best is None or er < best[1]:
            best = (list(assign), er, st)
    return best
