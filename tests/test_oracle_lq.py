"""Pins of the decomposition / configuration-search oracle (oracle/lq.py) against what the mathematics fixes:
Eckart-Young closed forms for Factorize, the exact weighted optimum when F has rank one, the invariants of the
alternation (Algorithm 2), hand-solvable instances of the integer program (Sec. 3.2) and Eq. (2) for the storage."""
import numpy as np
import pytest

import oracle
from oracle import lq
from paper_2311_12023_b200 import inputs

C = inputs.QuantConfig


def _orthonormal(g, n, r):
    q, _ = np.linalg.qr(g.standard_normal((n, r)))
    return q


def test_factorize_recovers_planted_singular_triplets():
    """A = U diag(s) V^T with known orthonormal U, V: the rank-r Factorize must return U_r diag(s_r) V_r^T, split as
    L1 = U sqrt(S), L2 = sqrt(S) V^T (so L1^T L1 = L2 L2^T = diag(s_r)), and leave exactly the tail energy (Eckart-Young)."""
    g = inputs.rng(1)
    d, k, r = 48, 80, 5
    U, V = _orthonormal(g, d, 12), _orthonormal(g, k, 12)
    s = np.array([9.0, 7.5, 6.0, 4.0, 3.0, 2.0, 1.5, 1.0, 0.7, 0.5, 0.2, 0.1])
    A = (U * s) @ V.T
    L1, L2 = lq.factorize(A, r)
    assert L1.shape == (d, r) and L2.shape == (r, k)
    np.testing.assert_allclose(L1 @ L2, (U[:, :r] * s[:r]) @ V[:, :r].T, atol=1e-10)
    np.testing.assert_allclose(L1.T @ L1, np.diag(s[:r]), atol=1e-10)
    np.testing.assert_allclose(L2 @ L2.T, np.diag(s[:r]), atol=1e-10)
    assert abs(np.sum((A - L1 @ L2) ** 2) - np.sum(s[r:] ** 2)) < 1e-9


def test_weighted_factorize_is_exact_when_fisher_has_rank_one():
    """sqrt(F) = a b^T (identical rows / columns up to scale, the assumption of Sec. 3.3): D_row E D_col is a multiple of
    sqrt(F) o E, so the weighted problem is an ordinary SVD and its optimum is the tail energy of sqrt(F) o E."""
    g = inputs.rng(2)
    d, k, r = 40, 56, 4
    a, b = g.uniform(0.5, 2.0, d), g.uniform(0.2, 3.0, k)
    F = np.outer(a, b) ** 2
    E = g.standard_normal((d, k))
    L1, L2 = lq.factorize(E, r, F)
    tail = np.linalg.svd(np.outer(a, b) * E, compute_uv=False)[r:]
    got = lq.weighted_norm(E - L1 @ L2, F) ** 2
    assert abs(got - np.sum(tail ** 2)) < 1e-9 * np.sum(tail ** 2) + 1e-12
    # and no rank-r perturbation of it does better
    for _ in range(5):
        P1, P2 = L1 + 1e-3 * g.standard_normal(L1.shape), L2 + 1e-3 * g.standard_normal(L2.shape)
        assert lq.weighted_norm(E - P1 @ P2, F) ** 2 >= got - 1e-12
    # F = const reduces to the unweighted case
    U1, U2 = lq.factorize(E, r, np.full((d, k), 3.0))
    V1, V2 = lq.factorize(E, r)
    np.testing.assert_allclose(U1 @ U2, V1 @ V2, atol=1e-10)


@pytest.mark.parametrize("cfg", [C(3, 16, 8, 16, 32), C(2, 32, 8, 16, 32), C(4, 64, 8, 64, 32)])
def test_alternation_invariants(cfg):
    """Algorithm 2 on a planted rank-r matrix plus noise: the recorded errors fall until the stop, the result is the
    iterate before the rise, Q is a fixed point of Quantize (it lies in the quantizable set), the first step is
    'SVD, then quantize the residual', and the decomposition beats plain quantization of W."""
    g = inputs.rng(3)
    d, k, r = 64, 128, 4
    W = 0.05 * g.standard_normal((d, r)) @ g.standard_normal((r, k)) + 0.02 * g.standard_normal((d, k))
    Q, L1, L2, err, hist, steps = lq.lq_decompose(W, cfg, r, T=12)
    assert steps == len(hist) and 1 <= steps <= 12
    body = hist[:-1] if (steps < 12 and hist[-1] > hist[-2]) else hist
    assert all(body[i + 1] <= body[i] for i in range(len(body) - 1))
    assert err == min(hist)
    assert abs(err - np.linalg.norm(W - (Q.astype(np.float64) + L1 @ L2))) < 1e-12
    assert np.array_equal(lq.quantize(Q, cfg), Q)
    # first step by hand
    U, S, Vt = np.linalg.svd(W, full_matrices=False)
    L = (U[:, :r] * S[:r]) @ Vt[:r]
    e1 = np.linalg.norm(W - (lq.quantize(W - L, cfg).astype(np.float64) + L))
    assert abs(hist[0] - e1) < 1e-9
    # rank 0 is plain quantization, and the low-rank term helps
    q0 = lq.lq_decompose(W, cfg, 0, T=3)
    assert abs(q0[3] - np.linalg.norm(W - lq.quantize(W, cfg))) < 1e-12 and len(set(q0[4])) == 1
    assert err < q0[3]


def test_alternation_with_fisher_weights_uses_the_weighted_error():
    g = inputs.rng(4)
    d, k, r = 32, 64, 3
    W = 0.02 * g.standard_normal((d, k))
    F = g.uniform(0.1, 4.0, (d, k))
    cfg = C(3, 16, 8, 16, 32)
    Q, L1, L2, err, hist, _ = lq.lq_decompose(W, cfg, r, F, T=6)
    assert abs(err - np.sqrt(np.sum(F * (W - (Q + L1 @ L2)) ** 2))) < 1e-12
    assert err == min(hist)


def test_storage_and_integer_program_on_hand_solvable_instances():
    nf4 = C(4, 64, 8, 256, 32)
    assert abs(lq.storage_bits((10, 20), nf4) - 200 * 4.127) < 200 * 5e-4          # 4.127 bits per parameter (Sec. 3.2)
    # two matrices, three configurations: storage 2 / 3 / 4, errors fall with storage
    S = np.array([[2.0, 3.0, 4.0], [20.0, 30.0, 40.0]])
    E = np.array([[9.0, 4.0, 1.0], [90.0, 20.0, 10.0]])
    assert lq.ilp_solve(S, E, 21.9) is None                         # even the cheapest pair (22) does not fit
    assert lq.ilp_solve(S, E, 22.0)[0] == [0, 0]
    assert lq.ilp_solve(S, E, 32.0)[0] == [0, 1]                    # 2 + 30: upgrading the large matrix pays most
    assert lq.ilp_solve(S, E, 34.0)[0] == [2, 1]                    # 4 + 30
    assert lq.ilp_solve(S, E, 44.0)[0] == [2, 2]
    prev = np.inf
    for budget in np.arange(22.0, 45.0, 1.0):
        a, er, st = lq.ilp_solve(S, E, budget)
        assert st <= budget and er <= prev
        prev = er


def test_error_and_storage_tables_feed_the_integer_program():
    """Algorithm 3 end to end on a toy model: tables from the alternation, then the budgeted assignment."""
    g = inputs.rng(5)
    Ws = [0.02 * g.standard_normal((32, 64)), 0.02 * g.standard_normal((64, 64))]
    configs = [C(2, 16, 8, 16, 32), C(3, 16, 8, 16, 32), C(4, 16, 8, 16, 32)]
    E, S = lq.error_storage_tables(Ws, configs, r=2, T=4)
    assert np.all(E[:, 0] > E[:, 1]) and np.all(E[:, 1] > E[:, 2])          # more bits, less error
    assert np.all(S[:, 0] < S[:, 1]) and np.all(S[:, 1] < S[:, 2])
    params = sum(w.size for w in Ws)
    lo = lq.ilp_solve(S, E, params * oracle.storage_bits_per_param(2, 8, 32, 16, 16))
    hi = lq.ilp_solve(S, E, params * oracle.storage_bits_per_param(4, 8, 32, 16, 16))
    assert lo[0] == [0, 0] and hi[0] == [2, 2]
    mid = lq.ilp_solve(S, E, params * 3.6)
    assert lo[1] > mid[1] > hi[1] and mid[2] <= params * 3.6
