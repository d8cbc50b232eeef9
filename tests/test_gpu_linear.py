"""Parity of lqlora_linear_fwd / lqlora_linear_bwd_input with the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2311_12023_b200 import binding, inputs
from gpu_util import check_close, encode_both, to_np

pytestmark = pytest.mark.gpu

C = inputs.QuantConfig


def run_case(A, l1b, l2b, cfg, M, seed, rows=None, passes=("fwd", "bwd"), route=None):
    """Encodes A on both sides (bit-exact codec parity is asserted inside encode_both for every matrix that comes
    through here), then compares Y and dX with the fp64 oracle.  route: expected kernel id of the forward dispatch."""
    N, K = A.shape
    q, ref = encode_both(A, cfg)
    if route is not None:
        r = 0 if l1b is None else l1b.shape[1]
        assert binding.linear_path(N, K, cfg, r, M, False) == route
    L1 = binding.bf16_from_bits(l1b) if l1b is not None else None
    L2 = binding.bf16_from_bits(l2b) if l2b is not None else None
    out = {}
    if "fwd" in passes:
        xb = inputs.activations(seed, M, K)
        Y = binding.linear_fwd(q, L1, L2, binding.bf16_from_bits(xb))
        torch.cuda.synchronize()
        Yo = oracle.linear_fwd(ref["d32"], l1b, l2b, xb, rows)
        got = to_np(Y) if rows is None else to_np(Y[torch.from_numpy(rows).cuda()])
        out["fwd"] = check_close(got, Yo, f"Y M={M}")
    if "bwd" in passes:
        gb = inputs.activations(seed + 1, M, N)
        dX = binding.linear_bwd_input(q, L1, L2, binding.bf16_from_bits(gb))
        torch.cuda.synchronize()
        dXo = oracle.linear_bwd_input(ref["d32"], l1b, l2b, gb, rows)
        got = to_np(dX) if rows is None else to_np(dX[torch.from_numpy(rows).cuda()])
        out["bwd"] = check_close(got, dXo, f"dX M={M}")
    return out


@pytest.mark.parametrize("b0,B0,B1", [(2, 16, 64), (3, 64, 256), (4, 32, 64), (4, 64, 256), (8, 128, 64), (3, 256, 256)])
@pytest.mark.parametrize("M", [1, 5, 16, 17, 24, 33])
def test_linear_small_shapes(b0, B0, B1, M):
    N, K = 320, 768            # N not a multiple of 128; several column windows
    A = inputs.gaussian(100 + b0, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(101, N, K, 64, 0.01)
    run_case(A, l1b, l2b, C(b0, B0, 8, B1, 32), M, seed=200 + M)


@pytest.mark.parametrize("M", [128, 200, 384])
@pytest.mark.parametrize("b0,B0", [(3, 64), (4, 64), (2, 16), (8, 32)])
def test_linear_training_shapes(b0, B0, M):
    N, K = 512, 1024
    A = inputs.student_t(300 + b0, (N, K), 5.0, 0.02)
    l1b, l2b = inputs.lowrank_factors(301, N, K, 64, 0.01)
    run_case(A, l1b, l2b, C(b0, B0, 8, 256, 32), M, seed=400 + M)


@pytest.mark.parametrize("N,K,M", [(200, 704, 3), (200, 704, 11), (1160, 64, 16), (72, 1984, 8)])
@pytest.mark.parametrize("b0,B0", [(3, 64), (2, 16), (8, 32)])
def test_linear_decode_kernels_ragged_shapes(N, K, M, b0, B0):
    """Decode kernels with a partial last tile row (N % 128 != 0), an odd number of 64-column tiles and fewer
    tiles than cluster ranks."""
    A = inputs.gaussian(800 + N, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(801 + K, N, K, 32, 0.01)
    run_case(A, l1b, l2b, C(b0, B0, 8, 16, 32), M, seed=900 + M)


@pytest.mark.parametrize("M", [2, 13])
@pytest.mark.parametrize("b0,B0,B1", [(3, 64, 256), (4, 32, 64), (2, 16, 64), (8, 128, 256), (3, 16, 16)])
def test_linear_decode_kernels_long_rows(b0, B0, B1, M):
    """Decode kernels on long rows: slices with 16-aligned runs of blocks (the compact scale table of the forward and
    of the input-gradient kernel, and the fp32 table where the runs are shorter)."""
    N, K = 256, 8192
    A = inputs.gaussian_outliers(1200 + b0, (N, K), 0.02, 0.001, 10.0)
    l1b, l2b = inputs.lowrank_factors(1201, N, K, 64, 0.01)
    run_case(A, l1b, l2b, C(b0, B0, 8, B1, 32), M, seed=1300 + M)


def test_linear_single_row_with_odd_feature_count_uses_the_fallback():
    # N % 8 != 0 is only legal for M = 1 (no vector loads on the rows of Y): the plain kernels take it
    N, K = 201, 192
    A = inputs.gaussian(850, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(851, N, K, 16, 0.01)
    run_case(A, l1b, l2b, C(4, 64, 8, 16, 32), 1, seed=950)


@pytest.mark.parametrize("N,K,M", [(640, 1088, 1000), (328, 704, 513), (896, 320, 700)])
@pytest.mark.parametrize("b0,B0", [(3, 64), (4, 32)])
def test_linear_many_rows_few_tiles(N, K, M, b0, B0):
    """More than 256 rows on matrices whose CTA-pair tiles would fill few SMs: the one-CTA kernel with several row
    tiles (grid.x > 1), split contraction, M, N, K not multiples of the tile."""
    A = inputs.gaussian(600 + N, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(601 + K, N, K, 64, 0.01)
    kernel, splits = binding.linear_route(N, K, C(b0, B0, 8, 64, 32), 64, M, False)
    assert kernel == binding.PATH_TC_ONE and (splits > 1 or K < 1024)      # 1088 columns: 17 steps, split over a cluster
    run_case(A, l1b, l2b, C(b0, B0, 8, 64, 32), M, seed=700 + M)


@pytest.mark.parametrize("N,K,M", [(2504, 2368, 2100), (2184, 2496, 2561)])
@pytest.mark.parametrize("b0,B0", [(3, 64), (4, 32)])
def test_linear_pair_kernel_ragged_tiles(N, K, M, b0, B0):
    """CTA-pair kernel (enough [512, 256] tiles to fill the SMs) with M, N, K that are not multiples of the pair tile:
    the second CTA of a pair may have few weight rows / columns, the TMA stores clip, and the contraction ends inside
    a 128-row tile.  Sampled rows (first, last, both sides of tile edges)."""
    assert binding.linear_route(N, K, C(b0, B0, 8, 64, 32), 64, M, False) == (binding.PATH_TC_PAIR, 1)
    assert binding.linear_path(N, K, C(b0, B0, 8, 64, 32), 64, M, True) == binding.PATH_TC_PAIR
    A = inputs.gaussian(650 + N, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(651 + K, N, K, 64, 0.01)
    rows = inputs.sample_rows(660 + M, M, count=24, tile=128)
    run_case(A, l1b, l2b, C(b0, B0, 8, 64, 32), M, seed=750 + M, rows=rows)


@pytest.mark.parametrize("b0,B0,r", [(3, 64, 64), (8, 32, 0)])
def test_linear_pair_kernel_with_peeled_last_wave(b0, B0, r):
    """80 pair tiles on 74 CTA pairs: the six tiles of the second wave are peeled off as two output column tiles and run
    on the one-CTA kernel (forward: N = 4096 at 2560 rows; the input gradient of the transposed shape likewise)."""
    M = 2560
    for N, K in ((4096, 512), (512, 4096)):
        A = inputs.gaussian(670 + N, (N, K), 0.02)
        l1b, l2b = inputs.lowrank_factors(671 + K, N, K, r, 0.01) if r else (None, None)
        rows = inputs.sample_rows(672, M, count=16, tile=256)
        run_case(A, l1b, l2b, C(b0, B0, 8, 64, 32), M, seed=760 + N, rows=rows, route=binding.PATH_TC_PAIR if N == 4096 else None)


@pytest.mark.parametrize("M", [4, 256])
def test_linear_without_lowrank_and_with_zero_weights(M):
    N, K = 256, 512
    cfg = C(4, 64, 8, 256, 32)
    A = inputs.gaussian(7, (N, K), 0.02)
    run_case(A, None, None, cfg, M, seed=8)                      # r = 0: quantized part alone
    l1b, l2b = inputs.lowrank_factors(9, N, K, 32, 0.05)
    run_case(np.zeros_like(A), l1b, l2b, cfg, M, seed=10)        # Q = 0: pure rank-32 product


@pytest.mark.parametrize("M", [16, 256])
def test_identity_rows_return_dequantized_columns(M):
    """X = rows of the identity and L = 0: Y[m, :] must equal column m of deq16 exactly."""
    N, K = 256, 256
    cfg = C(3, 64, 8, 256, 32)
    A = inputs.gaussian(11, (N, K), 0.02)
    q, ref = encode_both(A, cfg)
    X = torch.eye(K, dtype=torch.bfloat16, device="cuda")[:M].contiguous()
    Y = binding.linear_fwd(q, None, None, X)
    w16 = inputs.bf16_bits_to_f32(ref["d16"])
    assert np.array_equal(to_np(Y), w16[:, :M].T)
    G = torch.eye(N, dtype=torch.bfloat16, device="cuda")[:M].contiguous()
    dX = binding.linear_bwd_input(q, None, None, G)
    assert np.array_equal(to_np(dX), w16[:M, :])


@pytest.mark.parametrize("M", [8, 192])
def test_adjoint_identity_on_gpu(M):
    """<dY, fwd(X)> = <bwd_input(dY), X> up to the bf16 rounding of the outputs."""
    N, K = 384, 512
    cfg = C(4, 64, 8, 256, 32)
    A = inputs.gaussian(12, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(13, N, K, 64, 0.02)
    q, _ = encode_both(A, cfg)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    X = binding.bf16_from_bits(inputs.activations(14, M, K))
    G = binding.bf16_from_bits(inputs.activations(15, M, N))
    Y = binding.linear_fwd(q, L1, L2, X).double()
    dX = binding.linear_bwd_input(q, L1, L2, G).double()
    lhs = (G.double() * Y).sum().item()
    rhs = (dX * X.double()).sum().item()
    scale = (G.double().norm() * Y.norm()).item()
    assert abs(lhs - rhs) <= 2e-3 * scale


def test_config1_forward():
    w = inputs.workload(1)
    spec = w["matrices"][0]
    A, l1b, l2b = inputs.make_matrix(spec)
    run_case(A, l1b, l2b, spec.cfg, 512, seed=1100, passes=("fwd",), route=binding.PATH_TC_ONE)


@pytest.mark.parametrize("M", [1, 16, 2048])
def test_config2_forward_and_backward(M):
    spec = inputs.workload(2)["matrices"][0]
    A, l1b, l2b = inputs.make_matrix(spec)
    rows = inputs.sample_rows(2100 + M, M) if M > 512 else None
    run_case(A, l1b, l2b, spec.cfg, M, seed=2200 + M, rows=rows, route=binding.PATH_TC_PAIR if M > 16 else binding.PATH_STREAM)


def test_config3_down_projection_sampled_rows():
    spec = inputs.workload(3)["matrices"][2]          # 4096 x 11008
    A, l1b, l2b = inputs.make_matrix(spec)
    rows = inputs.sample_rows(3100, 4096, count=16)
    run_case(A, l1b, l2b, spec.cfg, 4096, seed=3200, rows=rows, route=binding.PATH_TC_PAIR)


def test_config4_kv_projection_mixed_config():
    spec = [s for s in inputs.workload(4)["matrices"] if s.name == "k"][0]    # 1024 x 8192
    A, l1b, l2b = inputs.make_matrix(spec)
    run_case(A, l1b, l2b, spec.cfg, 1, seed=4200)
    rows = inputs.sample_rows(4100, 2048, count=16)
    run_case(A, l1b, l2b, spec.cfg, 2048, seed=4300, rows=rows)


def test_config3_gate_projection_sampled_rows():
    spec = inputs.workload(3)["matrices"][0]          # 11008 x 4096, Student-t, NF4
    A, l1b, l2b = inputs.make_matrix(spec)
    rows = inputs.sample_rows(3300, 4096, count=16)
    run_case(A, l1b, l2b, spec.cfg, 4096, seed=3400, rows=rows, route=binding.PATH_TC_PAIR)


def test_config3_up_projection_sampled_rows():
    spec = inputs.workload(3)["matrices"][1]          # 11008 x 4096, its own seed
    A, l1b, l2b = inputs.make_matrix(spec)
    rows = inputs.sample_rows(3500, 4096, count=8)
    run_case(A, l1b, l2b, spec.cfg, 4096, seed=3600, rows=rows, route=binding.PATH_TC_PAIR)


def test_config4_query_projection_mixed_config():
    spec = [s for s in inputs.workload(4)["matrices"] if s.name == "q"][0]    # 8192 x 8192, drawn config
    A, l1b, l2b = inputs.make_matrix(spec)
    run_case(A, l1b, l2b, spec.cfg, 1, seed=4400)
    rows = inputs.sample_rows(4500, 2048, count=16)
    run_case(A, l1b, l2b, spec.cfg, 2048, seed=4600, rows=rows)


@pytest.mark.parametrize("name,M", [("gate", 1), ("down", 2048), ("gate", 2048)])
def test_config4_mlp_projections_largest_shapes(name, M):
    spec = [s for s in inputs.workload(4)["matrices"] if s.name == name][0]   # 28672 x 8192 / 8192 x 28672
    A, l1b, l2b = inputs.make_matrix(spec)
    rows = inputs.sample_rows(4700, M, count=8) if M > 16 else None
    run_case(A, l1b, l2b, spec.cfg, M, seed=4800 + M, rows=rows)


@pytest.mark.parametrize("name", ["v", "o", "up"])
def test_config4_remaining_matrices(name):
    """The other matrices of the 70B layer with their drawn configurations: bit-exact codec parity at full size (inside
    run_case) and the decode-sized forward and input gradient."""
    spec = [s for s in inputs.workload(4)["matrices"] if s.name == name][0]
    A, l1b, l2b = inputs.make_matrix(spec)
    run_case(A, l1b, l2b, spec.cfg, 1, seed=4900, route=binding.PATH_STREAM)


@pytest.mark.parametrize("b0,B0", [(2, 16), (3, 64), (4, 128), (8, 16), (8, 256)])
def test_config5_sweep_points(b0, B0):
    """Points of the 8192 x 8192 sweep at every M of the sweep (decode kernels, one-CTA and CTA-pair tensor-core
    kernels; 8192 rows = 16 x 32 pair tiles), whole-height bit-exact codec parity included (encode_both)."""
    A = inputs.gaussian(5000, (8192, 8192), 0.02)
    l1b, l2b = inputs.lowrank_factors(5700, 8192, 8192, 64, 0.01)
    cfg = C(b0, B0, 8, 256, 32)
    N, K = A.shape
    q, ref = encode_both(A, cfg)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    for M in (1, 16, 128, 2048, 8192):
        rows = inputs.sample_rows(5100 + M, M, count=8) if M > 16 else None
        want = binding.PATH_STREAM if M <= 16 else binding.PATH_TC_ONE if M == 128 else binding.PATH_TC_PAIR
        assert binding.linear_path(N, K, cfg, 64, M, False) == want
        xb = inputs.activations(5200 + M, M, K)
        gb = inputs.activations(5300 + M, M, N)
        Y = binding.linear_fwd(q, L1, L2, binding.bf16_from_bits(xb))
        dX = binding.linear_bwd_input(q, L1, L2, binding.bf16_from_bits(gb))
        torch.cuda.synchronize()
        sel = slice(None) if rows is None else torch.from_numpy(rows).cuda()
        check_close(to_np(Y[sel]), oracle.linear_fwd(ref["d32"], l1b, l2b, xb, rows), f"Y b0={b0} B0={B0} M={M}")
        check_close(to_np(dX[sel]), oracle.linear_bwd_input(ref["d32"], l1b, l2b, gb, rows), f"dX b0={b0} B0={B0} M={M}")


def test_workspace_status_is_clean_after_a_call():
    N, K, M = 256, 512, 8
    cfg = C(3, 64, 8, 256, 32)
    q, _ = encode_both(inputs.gaussian(1, (N, K), 0.02), cfg)
    ws = binding.alloc_workspace(q, 0, M)
    X = binding.bf16_from_bits(inputs.activations(2, M, K))
    binding.linear_fwd(q, None, None, X, workspace=ws)
    assert binding.workspace_status(ws) == 0


@pytest.mark.parametrize("N,K,M", [(256, 512, 8), (512, 1024, 200), (4096, 4096, 2048), (2304, 2048, 1100), (4096, 4096, 12)])
def test_workspace_may_hold_anything_before_a_call(N, K, M):
    """The workspace is scratch: whatever it holds (here all ones, i.e. a non-zero status word and non-zero arrival
    counters) a call gives the right result and leaves a clean status word -- whether the words that must start at
    zero are cleared by a memset or by the first kernel of the call."""
    cfg = C(3, 64, 8, 256, 32)
    A = inputs.gaussian(1400 + N, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(1401, N, K, 64, 0.01)
    q, ref = encode_both(A, cfg)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    rows = inputs.sample_rows(1402, M, count=16) if M > 512 else None
    ws = binding.alloc_workspace(q, 64, M)
    xb = inputs.activations(1403, M, K)
    gb = inputs.activations(1404, M, N)
    for _ in range(2):
        ws.fill_(0xFF)
        Y = binding.linear_fwd(q, L1, L2, binding.bf16_from_bits(xb), workspace=ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        ws.fill_(0xFF)
        dX = binding.linear_bwd_input(q, L1, L2, binding.bf16_from_bits(gb), workspace=ws)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
    got = to_np(Y) if rows is None else to_np(Y[torch.from_numpy(rows).cuda()])
    check_close(got, oracle.linear_fwd(ref["d32"], l1b, l2b, xb, rows), "Y")
    got = to_np(dX) if rows is None else to_np(dX[torch.from_numpy(rows).cuda()])
    check_close(got, oracle.linear_bwd_input(ref["d32"], l1b, l2b, gb, rows), "dX")


def test_a_bounded_wait_that_runs_out_sets_the_status_and_leaves_the_device_usable():
    """A wait on bytes that never arrive is abandoned after its budget (about a millisecond here): the status word says
    LQLORA_ERR_TIMEOUT, tensor memory was freed (the tcgen05 kernels that follow allocate all of it on every SM) and
    the same workspace serves correct calls afterwards.  Also the host-side reading of a non-zero status word."""
    N, K, M = 2560, 2304, 2100
    cfg = C(3, 64, 8, 256, 32)
    A = inputs.gaussian(1500, (N, K), 0.02)
    l1b, l2b = inputs.lowrank_factors(1501, N, K, 64, 0.01)
    q, ref = encode_both(A, cfg, check=False)
    L1, L2 = binding.bf16_from_bits(l1b), binding.bf16_from_bits(l2b)
    ws = binding.alloc_workspace(q, 64, M)
    for _ in range(3):
        binding.selftest_bounded_wait(ws, 2_000_000)
        assert binding.workspace_status(ws) == -7
        assert binding.status_string(-7) == "device-side wait timed out"
    # a status word written by anyone reads as a time-out until the next call clears it
    ws[:4] = torch.tensor([5, 0, 0, 0], dtype=torch.uint8, device="cuda")
    assert binding.workspace_status(ws) == -7
    rows = inputs.sample_rows(1502, M, count=8)
    xb = inputs.activations(1503, M, K)
    Y = binding.linear_fwd(q, L1, L2, binding.bf16_from_bits(xb), workspace=ws)
    assert binding.workspace_status(ws) == 0
    check_close(to_np(Y[torch.from_numpy(rows).cuda()]), oracle.linear_fwd(ref["d32"], l1b, l2b, xb, rows), "Y after the time-outs")
