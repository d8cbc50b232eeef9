"""Parity of lqlora_lora_grads (gradients of the low-rank factors) with the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_12023_b200 import binding, inputs
from gpu_util import check_close, to_np

pytestmark = pytest.mark.gpu


def run_case(N, K, M, r, seed):
    l1b, l2b = inputs.lowrank_factors(seed, N, K, r, 0.05)
    xb = inputs.activations(seed + 1, M, K)
    gb = inputs.activations(seed + 2, M, N)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    X, dY = binding.bf16_from_bits(xb), binding.bf16_from_bits(gb)
    ws = torch.empty(binding.lora_grads_workspace_bytes(N, K, r, M), dtype=torch.uint8, device="cuda")
    dL1, dL2 = binding.lora_grads(L1, L2, X, dY, workspace=ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    o1, o2 = oracle.lora_grads(l1b, l2b, xb, gb)
    assert tuple(dL1.shape) == (N, r) and tuple(dL2.shape) == (r, K)
    check_close(to_np(dL1), o1, f"dL1 N={N} K={K} M={M} r={r}")
    check_close(to_np(dL2), o2, f"dL2 N={N} K={K} M={M} r={r}")
    return dL1, dL2, ws, (L1, L2, X, dY)


@pytest.mark.parametrize("N,K,M,r", [(256, 512, 300, 64), (320, 192, 64, 16), (200, 1032, 1000, 32), (512, 256, 7, 64),
                                     (136, 136, 2049, 128), (1024, 768, 512, 48)])
def test_lora_grads_shapes(N, K, M, r):
    """Several row tiles and token slices, ragged last tiles (N, K, M not multiples of 128 / 64), all rank paddings."""
    run_case(N, K, M, r, seed=5000 + N + M)


def test_lora_grads_training_shape_and_repeatability():
    """LLaMA-2-7B attention projection at 2048 tokens; a second call into the same buffers gives the same bits."""
    N = K = 4096
    dL1, dL2, ws, (L1, L2, X, dY) = run_case(N, K, 2048, 64, seed=6000)
    a1, a2 = dL1.clone(), dL2.clone()
    binding.lora_grads(L1, L2, X, dY, out=(dL1, dL2), workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(a1, dL1) and torch.equal(a2, dL2)


@pytest.mark.parametrize("N,K,M,r,b0,B0", [(2304, 2560, 2100, 64, 3, 64), (512, 1024, 200, 64, 2, 16), (320, 768, 8, 32, 4, 32),
                                           (384, 640, 1000, 128, 3, 32)])
def test_lora_grads_from_the_intermediates_of_the_other_passes(N, K, M, r, b0, B0):
    """The layer's three passes on the same X and dY: forward, input gradient, then lqlora_lora_grads_from with the
    intermediates T, T' the first two left in their workspaces (CTA-pair kernel, one-CTA kernel, weight-streaming
    kernel, rank padded to 128).  Same tolerance against the fp64 oracle as lqlora_lora_grads."""
    from gpu_util import encode_both
    cfg = inputs.QuantConfig(b0, B0, 8, 64, 32)
    q, _ = encode_both(inputs.gaussian(5100 + N, (N, K), 0.02), cfg)
    l1b, l2b = inputs.lowrank_factors(5101 + N, N, K, r, 0.05)
    xb = inputs.activations(5102 + N, M, K)
    gb = inputs.activations(5103 + N, M, N)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    X, dY = binding.bf16_from_bits(xb), binding.bf16_from_bits(gb)
    ws_f, ws_b = binding.alloc_workspace(q, r, M), binding.alloc_workspace(q, r, M)
    binding.linear_fwd(q, L1, L2, X, workspace=ws_f)
    binding.linear_bwd_input(q, L1, L2, dY, workspace=ws_b)
    T = binding.linear_intermediate(ws_f, N, K, cfg, r, M, False)
    Tp = binding.linear_intermediate(ws_b, N, K, cfg, r, M, True)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    dL1, dL2 = binding.lora_grads_from(T, Tp, N, K, X, dY, workspace=ws)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    o1, o2 = oracle.lora_grads(l1b, l2b, xb, gb)
    check_close(to_np(dL1), o1, f"dL1 from T N={N} K={K} M={M} r={r}")
    check_close(to_np(dL2), o2, f"dL2 from T' N={N} K={K} M={M} r={r}")


def test_lora_grads_one_hot_tokens():
    """One-hot X and dY rows pick single entries of the factors: exact in any arithmetic."""
    N, K, r, M = 256, 384, 64, 3
    l1b, l2b = inputs.lowrank_factors(7000, N, K, r, 0.05)
    Xh = np.zeros((M, K), np.float32); dYh = np.zeros((M, N), np.float32)
    pos = [(5, 17), (200, 255), (383, 0)]
    for m, (a, b) in enumerate(pos):
        Xh[m, a] = 1.0; dYh[m, b] = 1.0
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    dL1, dL2 = binding.lora_grads(L1, L2, binding.bf16_from_bits(inputs.f32_to_bf16_bits(Xh)),
                                  binding.bf16_from_bits(inputs.f32_to_bf16_bits(dYh)))
    torch.cuda.synchronize()
    F1 = inputs.bf16_bits_to_f32(l1b).astype(np.float64); F2 = inputs.bf16_bits_to_f32(l2b).astype(np.float64)
    e1 = np.zeros((N, r)); e2 = np.zeros((r, K))
    for a, b in pos:
        e1[b, :] += F2[:, a]; e2[:, a] += F1[b, :]
    assert np.array_equal(to_np(dL1).astype(np.float64), e1) and np.array_equal(to_np(dL2).astype(np.float64), e2)


def test_lora_grads_rejects_bad_arguments():
    L1 = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda"); L2 = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    X = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda"); dY = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.LqloraError):
        binding.lora_grads(L1, L2, X, dY, workspace=small)          # workspace too small
    with pytest.raises(binding.LqloraError):
        binding.lora_grads_workspace_bytes(128, 128, 24, 4)          # rank not a multiple of 16
    with pytest.raises(binding.LqloraError):
        binding.lora_grads_workspace_bytes(100, 128, 64, 4)          # N not a multiple of 8
