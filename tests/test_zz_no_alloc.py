"""lqlora_linear_fwd_static: the forward pass for callers that cannot allocate device memory.

Such callers (a serving runtime that owns the whole device arena, a plugin running inside someone
else's stream) pass only inputs and outputs; the scratch comes from a fixed array inside the library.
The result must match the ordinary entry point, also when the call is repeated: the array keeps the
previous call's contents, so a second call checks that everything that must start at zero is cleared.
This file is collected last on purpose, so that a failure here cannot hide any other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2311_12023_b200 import binding, inputs
from gpu_util import check_close, to_np

pytestmark = pytest.mark.gpu


def _case(N, K, M, cfg, r, seed):
    A = inputs.gaussian(seed, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(seed + 1, N, K, r, 0.01)
    q = binding.encode(torch.from_numpy(A).cuda(), cfg)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    X = binding.bf16_from_bits(inputs.activations(seed + 2, M, K))
    return q, L1, L2, X


@pytest.mark.parametrize("M", [4, 16, 256])      # decode-sized (weight-streaming) and tensor-core paths
def test_static_scratch_forward_matches_ordinary_forward_twice_in_a_row(M):
    q, L1, L2, X = _case(512, 1024, M, inputs.QuantConfig(3, 64, 8, 256, 32), 64, 90 + M)
    ordinary = binding.linear_fwd(q, L1, L2, X)
    ref = to_np(ordinary).astype(np.float64)
    first = binding.linear_fwd_static(q, L1, L2, X)
    second = binding.linear_fwd_static(q, L1, L2, X)       # reuses the scratch the first call dirtied
    torch.cuda.synchronize()
    assert binding.static_scratch_status() == 0            # no bounded wait gave up
    check_close(to_np(first), ref, f"first static call, M={M}")
    check_close(to_np(second), ref, f"second static call, M={M}")
    # the same kernels ran on the same inputs: the bits are the same, not merely close
    assert torch.equal(first.view(torch.int16), ordinary.view(torch.int16))
    assert torch.equal(second.view(torch.int16), ordinary.view(torch.int16))
    # a different problem in between must not disturb the next call either
    q2, A1, A2, X2 = _case(256, 512, 8, inputs.QuantConfig(4, 32, 8, 64, 32), 32, 70)
    binding.linear_fwd_static(q2, A1, A2, X2)
    third = binding.linear_fwd_static(q, L1, L2, X)
    torch.cuda.synchronize()
    check_close(to_np(third), ref, f"third static call, M={M}")
    assert torch.equal(third.view(torch.int16), ordinary.view(torch.int16))


def test_static_scratch_rejects_oversized_problems_without_launching():
    cfg = inputs.QuantConfig(3, 64, 8, 256, 32)
    N = K = 4096
    M = 1 << 18                                # needs far more than 8 MiB of scratch
    assert int(binding.lib().lqlora_static_scratch_bytes()) == binding.STATIC_SCRATCH_BYTES
    assert binding.linear_workspace_bytes(N, K, cfg, 64, M) > binding.STATIC_SCRATCH_BYTES
    fake = 0x10000                             # never dereferenced: the size check comes first
    q = binding.CQMatrix(fake, fake, fake, N, K, binding._cfg(cfg))
    rc = binding.lib().lqlora_linear_fwd_static(ctypes.byref(q), fake, fake, 64, fake, M, fake, None)
    assert rc == -5 and "workspace" in binding.status_string(rc)
