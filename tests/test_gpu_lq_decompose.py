"""lqlora_lq_decompose (Algorithm 2 with a randomized Factorize) against the exact-SVD oracle.  The SVD is not unique and
the range finder is randomized, so parity is a validity check: error history close to the oracle's, the reported error
reproduced on the host in fp64 from the returned Q, L1, L2, Q inside the quantizable set, balanced factors
(L1^T L1 = L2 L2^T = diag), and the stopping rule honoured."""
import numpy as np
import pytest
import torch

import oracle
from oracle import lq
from paper_2311_12023_b200 import binding, inputs

pytestmark = pytest.mark.gpu

C = inputs.QuantConfig


def _planted(seed, N, K, r, factor_std, noise_std):
    g = inputs.rng(seed)
    return (factor_std * g.standard_normal((N, r)) @ g.standard_normal((r, K)) + noise_std * g.standard_normal((N, K))).astype(np.float32)


def _omega(seed, K, l):
    return torch.from_numpy(inputs.rng(seed).standard_normal((K, l)).astype(np.float32)).cuda()


def _host_error(W, q, L1, L2, F=None):
    d32, _ = binding.dequant(q, want16=False)
    E = W.astype(np.float64) - (d32.cpu().numpy().astype(np.float64) + L1.cpu().numpy().astype(np.float64) @ L2.cpu().numpy().astype(np.float64))
    return lq.weighted_norm(E, F)


@pytest.mark.parametrize("N,K,r,cfg", [(256, 512, 8, C(3, 64, 8, 16, 32)), (384, 320, 16, C(2, 16, 8, 64, 32)),
                                       (1024, 1024, 64, C(4, 64, 8, 256, 32))])
def test_decomposition_tracks_the_exact_svd_oracle(N, K, r, cfg):
    W = _planted(70 + N, N, K, r, 0.05, 0.02)
    T = 6
    q, L1, L2, errs = binding.lq_decompose(torch.from_numpy(W).cuda(), cfg, r, _omega(71, K, r + 8), max_steps=T, power_iters=4)
    Qo, L1o, L2o, erro, histo, stepso = lq.lq_decompose(W, cfg, r, T=T)
    assert 1 <= len(errs) <= T
    # stopping rule: errors fall until (at most) a final rise; the returned iterate is the best one
    body = errs[:-1] if (len(errs) >= 2 and errs[-1] > errs[-2]) else errs
    assert all(body[i + 1] <= body[i] for i in range(len(body) - 1))
    best = body[-1]
    assert abs(_host_error(W, q, L1, L2) - best) <= 1e-5 * best
    # close to the exact-SVD alternation, step by step and at the end
    n = min(len(body), len(histo))
    assert np.allclose(errs[:n], histo[:n], rtol=3e-3)
    assert abs(best - erro) <= 3e-3 * erro
    # the low-rank term helps: better than plain quantization
    assert best < np.linalg.norm(W.astype(np.float64) - lq.quantize(W, cfg))
    # Q lies in the quantizable set: encoding its dequantized value returns the same codes and scale codes
    d32, _ = binding.dequant(q, want16=False)
    q2 = binding.encode(d32, cfg)
    assert torch.equal(binding.unpack(q2), binding.unpack(q)) and torch.equal(q2.scale_codes, q.scale_codes)
    # balanced factors: L1 = U sqrt(S), L2 = sqrt(S) V^T
    g1 = (L1.double().T @ L1.double()).cpu().numpy()
    g2 = (L2.double() @ L2.double().T).cpu().numpy()
    assert np.allclose(g1, g2, atol=2e-3 * np.abs(g1).max())
    assert np.abs(g1 - np.diag(np.diag(g1))).max() <= 2e-3 * np.abs(g1).max()


def test_decomposition_with_fisher_weights():
    """F with identical rows / columns up to scale (sqrt(F) = a b^T): the weighted Factorize is exact there, so the
    weighted errors must track the oracle's."""
    N, K, r = 256, 384, 8
    cfg = C(3, 32, 8, 16, 32)
    g = inputs.rng(80)
    W = _planted(81, N, K, r, 0.05, 0.02)
    a, b = g.uniform(0.5, 2.0, N), g.uniform(0.3, 3.0, K)
    F = (np.outer(a, b) ** 2).astype(np.float32)
    T = 5
    q, L1, L2, errs = binding.lq_decompose(torch.from_numpy(W).cuda(), cfg, r, _omega(82, K, r + 8), F=torch.from_numpy(F).cuda(),
                                           max_steps=T, power_iters=4)
    _, _, _, erro, histo, _ = lq.lq_decompose(W, cfg, r, F.astype(np.float64), T=T)
    body = errs[:-1] if (len(errs) >= 2 and errs[-1] > errs[-2]) else errs
    best = body[-1]
    assert abs(_host_error(W, q, L1, L2, F.astype(np.float64)) - best) <= 1e-5 * best
    n = min(len(body), len(histo))
    assert np.allclose(errs[:n], histo[:n], rtol=3e-3)
    assert abs(best - erro) <= 3e-3 * erro


def test_layer_from_the_decomposition_reproduces_the_matrix():
    """End of the preparation path: the forward pass with (Q, bf16 L1, bf16 L2) applies W up to the decomposition error."""
    N, K, r = 512, 1024, 32
    cfg = C(3, 64, 8, 256, 32)
    W = _planted(90, N, K, r, 0.05, 0.01)
    q, L1, L2, errs = binding.lq_decompose(torch.from_numpy(W).cuda(), cfg, r, _omega(91, K, r + 8), max_steps=4)
    X = binding.bf16_from_bits(inputs.activations(92, 64, K))
    Y = binding.linear_fwd(q, binding.to_bf16(L1), binding.to_bf16(L2), X).double().cpu().numpy()
    ref = X.double().cpu().numpy() @ W.astype(np.float64).T
    rel = np.linalg.norm(Y - ref) / np.linalg.norm(ref)
    assert rel < 1.5 * min(errs) / np.linalg.norm(W) + 1e-2


def test_argument_checks():
    W = torch.zeros((128, 128), dtype=torch.float32, device="cuda")
    cfg = C(3, 64, 8, 16, 32)
    with pytest.raises(binding.LqloraError):
        binding.lq_decompose(W, cfg, 200, torch.zeros((128, 208), dtype=torch.float32, device="cuda"))       # r > 128
