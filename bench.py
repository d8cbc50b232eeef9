#!/usr/bin/env python
"""Benchmark of the LQ-LoRA linear hot path on B200.

One step = one pass of the whole hot path on the LLaMA-2-7B attention-projection workload
(4096x4096, NF3, B0 = 64, B1 = 256, rank 64; seeded synthetic data):

    encode(R)  ->  forward + input gradient at M = 2048 (training, tensor-core kernels)
               ->  forward + input gradient at M = 16 and M = 1 (decode, weight-streaming kernels)

`value` is the algorithmic TFLOP/s of the whole step: 2 M (N K + r K + N r) flop per linear
call, summed over the six calls, divided by the device time of the step (CUDA events).  The
JSON line also carries the per-phase figures (tensor TFLOP/s at M = 2048, packed-weight GB/s
at M = 1 / 16, encode GB/s), the roofline of the dominant kernel, the end-to-end number
through the host-buffer C ABI, and the CPU oracle timed on the host as a baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (torchrun) every rank runs the same per-GPU workload on its own tokens (data
parallel over tokens, no collective on the data path); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2311_12023_b200 import inputs  # noqa: E402

METRIC = "LQ-LoRA linear fwd/bwd TFLOP/s & packed-weight GB/s, % of B200 roofline"
WORKLOAD = "llama2-7b attn-proj 4096x4096 NF3 B0=64 B1=256 r=64; encode + fwd/dX at M=2048,16,1"
MS = (2048, 16, 1)
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per forward launch of tc_pair_linear_kernel<3, 0> at M = 2048 on this
# workload (profiles/kernels_c2_4096_nf3_ncu_full.txt): the operands are read once (X 16.8 MB + packed 6.6 MB +
# factors), the output stays in L2 during the capture
TC_TRAFFIC_BYTES = 24289024


def linear_flops(M: int, N: int, K: int, r: int) -> float:
    return 2.0 * M * (N * K + r * K + N * r)


def packed_bytes(N: int, K: int, cfg) -> float:
    return N * K * (cfg.b0 + cfg.b1 / cfg.B0 + cfg.b2 / (cfg.B0 * cfg.B1)) / 8.0


def encode_bytes(N: int, K: int, cfg) -> float:
    return 4.0 * N * K + packed_bytes(N, K, cfg)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK), "fallback"


# ------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------- reference arm
def oracle_sample(spec, A, l1b, l2b, rows_large: int = 24):
    """Times the CPU oracle on a bounded sample of the step; returns (flops_done, seconds, description)."""
    import oracle
    cfg = spec.cfg
    N, K, r = spec.N, spec.K, inputs.RANK
    t0 = time.perf_counter()
    codes, _, sc, v = oracle.encode(A, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    d32, _ = oracle.dequant(codes, sc, v, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
    flops = 0.0
    for M in MS:
        rows = inputs.sample_rows(900 + M, M, count=rows_large) if M > rows_large else None
        nrows = M if rows is None else len(rows)
        xb = inputs.activations(910 + M, M, K)
        gb = inputs.activations(920 + M, M, N)
        oracle.linear_fwd(d32, l1b, l2b, xb, rows)
        oracle.linear_bwd_input(d32, l1b, l2b, gb, rows)
        flops += 2 * linear_flops(nrows, N, K, r)
    dt = time.perf_counter() - t0
    desc = (f"encode+dequant of the full {N}x{K} matrix, then fwd and dX in fp64 on {rows_large} sampled rows "
            f"of M=2048 and all rows of M=16 and M=1")
    return flops, dt, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    spec = inputs.workload(2)["matrices"][0]
    A, l1b, l2b = inputs.make_matrix(spec)
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(spec, A, l1b, l2b, rows_large=4)
    times, flops = [], 0.0
    for _ in range(args.steps):
        flops, dt, desc = oracle_sample(spec, A, l1b, l2b, rows_large=64)
        times.append(dt)
    mean = sum(times) / len(times)
    val = flops / mean / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "each step is a bounded sample of the workload: " + desc},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------- device arm
def shard_info():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def reduce_max(value: float, world: int, device=None) -> float:
    """Max over ranks of a host scalar (identity when world == 1)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_device(args):
    import torch
    from paper_2311_12023_b200 import binding

    rank, world, local = shard_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    spec = inputs.workload(2)["matrices"][0]
    cfg, N, K, r = spec.cfg, spec.N, spec.K, inputs.RANK
    # every rank draws its own tokens (seed offset by rank); the weights are replicated
    A, l1b, l2b = inputs.make_matrix(spec)
    W_host = torch.from_numpy(A).pin_memory()
    W = W_host.to(dev)
    L1, L2 = binding.bf16_from_bits(l1b, dev), binding.bf16_from_bits(l2b, dev)
    q = binding.alloc_qmatrix(N, K, cfg, dev)
    enc_ws = torch.empty(binding.packed_sizes(N, K, cfg)[3], dtype=torch.uint8, device=dev)
    binding.encode(W, cfg, out=q, workspace=enc_ws)
    torch.cuda.synchronize()

    # cold copies of the packed matrix for the decode-sized calls: more than twice the L2 in total
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    ncopies = max(4, int(2.2 * l2_bytes / q.packed_bytes) + 1)
    copies = [binding.QMatrix(q.codes.clone(), q.scale_codes.clone(), q.scale2.clone(), N, K, cfg) for _ in range(ncopies)]

    X, G, Y, DX, WS, XH, GH, YH, DXH = {}, {}, {}, {}, {}, {}, {}, {}, {}
    for M in MS:
        XH[M] = torch.from_numpy(inputs.activations(7000 + 10 * rank + M, M, K).view(np.int16)).view(torch.bfloat16).pin_memory()
        GH[M] = torch.from_numpy(inputs.activations(7500 + 10 * rank + M, M, N).view(np.int16)).view(torch.bfloat16).pin_memory()
        X[M], G[M] = XH[M].to(dev), GH[M].to(dev)
        Y[M] = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        DX[M] = torch.empty((M, K), dtype=torch.bfloat16, device=dev)
        YH[M] = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        DXH[M] = torch.empty((M, K), dtype=torch.bfloat16).pin_memory()
        WS[M] = binding.alloc_workspace(q, r, M)
    flush = torch.empty(max(256 << 20, 2 * l2_bytes), dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(max(256 << 20, 2 * l2_bytes) // 4, dtype=torch.int32, device=dev)

    def flush_l2(v):
        """Evicts L2: writes a buffer larger than L2, then reads another one so that the lines left behind are clean
        (otherwise the first timed kernel also pays for writing the flush buffer back to HBM)."""
        flush.fill_(v)
        return flush_rd.max()


    seg_names = ["encode"] + [f"{p}{M}" for M in MS for p in ("fwd", "bwd")]
    nseg = len(seg_names)
    copy_idx = [0]

    def next_copy():
        c = copies[copy_idx[0] % ncopies]
        copy_idx[0] += 1
        return c

    def one_step(events=None, inner=True):
        """The whole hot path once, device-resident inputs.  events: list of nseg+1 CUDA events; with inner=False only
        the first and the last are recorded (the timed steps: no event records between the calls)."""
        def mark(i):
            if events and (inner or i == 0 or i == nseg):
                events[i].record()
        mark(0)
        binding.encode(W, cfg, out=q, workspace=enc_ws)
        i = 1
        mark(i)
        for M in MS:
            qq = q if M > 64 else next_copy()
            binding.linear_fwd(qq, L1, L2, X[M], out=Y[M], workspace=WS[M])
            i += 1
            mark(i)
            qq = q if M > 64 else next_copy()
            binding.linear_bwd_input(qq, L1, L2, G[M], out=DX[M], workspace=WS[M])
            i += 1
            mark(i)

    def one_step_host():
        """Same step through the host-buffer C ABI: H2D of W, X, dY and D2H of Y, dX inside."""
        binding.encode_host(W_host, W, q, enc_ws)
        for M in MS:
            qq = q if M > 64 else next_copy()
            binding.linear_fwd_host(qq, L1, L2, XH[M], YH[M], X[M], Y[M], WS[M])
            qq = q if M > 64 else next_copy()
            binding.linear_bwd_input_host(qq, L1, L2, GH[M], DXH[M], G[M], DX[M], WS[M])

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush_l2(1)
        one_step()
    torch.cuda.synchronize()
    for M in MS:
        st = binding.workspace_status(WS[M])
        if st != 0:
            raise SystemExit(f"kernel reported {binding.status_string(st)}")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nseg + 1)] for _ in range(args.steps)]
    launches0 = binding.launch_count()
    barrier()
    t_wall0 = time.perf_counter()
    for s in range(args.steps):
        flush_l2(s & 0xFF)             # evict L2 between steps (untimed: outside the step's events)
        one_step(evs[s], inner=False)
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = binding.launch_count() - launches0
    step_ms = [evs[s][0].elapsed_time(evs[s][nseg]) for s in range(args.steps)]
    # per-call breakdown: the same steps once more with an event after every call (these records perturb the step a
    # little, so they are kept out of the timed steps above)
    for s in range(args.steps):
        flush_l2(s & 0xFF)
        one_step(evs[s], inner=True)
    torch.cuda.synchronize()
    seg_ms = np.zeros(nseg)
    for s in range(args.steps):
        for i in range(nseg):
            seg_ms[i] += evs[s][i].elapsed_time(evs[s][i + 1])
    seg_ms /= args.steps
    ms_step = reduce_max(sum(step_ms) / len(step_ms), world, dev)

    # ---- back-to-back loops (no host gaps between launches): the tensor-core call over rotating activation
    # buffers (together larger than L2), the decode-sized calls over the cold copies as one CUDA graph
    loops = {}
    nrot = max(2, int(1.1 * l2_bytes / (2048 * (N + K) * 2)) + 1)
    Xr = [X[2048].clone() for _ in range(nrot)]
    Gr = [G[2048].clone() for _ in range(nrot)]
    Yr = [torch.empty_like(Y[2048]) for _ in range(nrot)]
    DXr = [torch.empty_like(DX[2048]) for _ in range(nrot)]
    reps = 4 * nrot

    def timed(fn, count):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / count

    def tc_fwd_loop():
        for i in range(reps):
            binding.linear_fwd(q, L1, L2, Xr[i % nrot], out=Yr[i % nrot], workspace=WS[2048])

    def tc_bwd_loop():
        for i in range(reps):
            binding.linear_bwd_input(q, L1, L2, Gr[i % nrot], out=DXr[i % nrot], workspace=WS[2048])

    loops["fwd2048"] = timed(tc_fwd_loop, reps)
    loops["bwd2048"] = timed(tc_bwd_loop, reps)

    def graph_loop(call, M):
        """ms per call of `ncopies` calls replayed as one CUDA graph (falls back to a plain loop)."""
        def body():
            for c in copies:
                call(c, M)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                body()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                body()
            return timed(g.replay, ncopies), "cuda graph"
        except Exception:
            torch.cuda.synchronize()
            return timed(body, ncopies), "stream loop"

    loop_kind = {}
    for M in (16, 1):
        loops[f"fwd{M}"], loop_kind[f"fwd{M}"] = graph_loop(lambda c, m: binding.linear_fwd(c, L1, L2, X[m], out=Y[m], workspace=WS[m]), M)
        loops[f"bwd{M}"], loop_kind[f"bwd{M}"] = graph_loop(lambda c, m: binding.linear_bwd_input(c, L1, L2, G[m], out=DX[m], workspace=WS[m]), M)
    # gradients of the low-rank factors at M = 2048 (the next piece of a training step; not part of the timed step):
    # rotating activation buffers, replayed as one CUDA graph
    dL = (torch.empty(N, r, dtype=torch.float32, device=dev), torch.empty(r, K, dtype=torch.float32, device=dev))
    gws = torch.empty(binding.lora_grads_workspace_bytes(N, K, r, 2048), dtype=torch.uint8, device=dev)

    def grads_body():
        for i in range(reps):
            binding.lora_grads(L1, L2, Xr[i % nrot], Gr[i % nrot], out=dL, workspace=gws)
    try:
        grads_body()
        torch.cuda.synchronize()
        gg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gg):
            grads_body()
        loops["grads2048"], loop_kind["grads2048"] = timed(gg.replay, reps), "cuda graph"
    except Exception:
        torch.cuda.synchronize()
        loops["grads2048"], loop_kind["grads2048"] = timed(grads_body, reps), "stream loop"
    if binding.workspace_status(gws) != 0:
        raise SystemExit("lora_grads reported a device-side error")
    for k in list(loops):
        loops[k] = reduce_max(loops[k], world, dev)

    # end to end through the host-buffer entry points
    for _ in range(max(1, min(args.warmup, 3))):
        one_step_host()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(3, min(args.steps, 10))
    e0.record()
    for _ in range(e2e_steps):
        one_step_host()
    e1.record()
    barrier()
    e2e_ms = reduce_max(e0.elapsed_time(e1) / e2e_steps, world, dev)
    clocks = sampler.stop() if rank == 0 else None

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    step_flops = sum(2 * linear_flops(M, N, K, r) for M in MS)
    value = world * step_flops / (ms_step * 1e-3) / 1e12
    pk, pk_kind = peaks()
    seg = dict(zip(seg_names, seg_ms.tolist()))
    pbytes = packed_bytes(N, K, cfg)
    small_bytes = pbytes + 2 * r * (N + K)
    breakdown = {
        "encode": {"ms": seg["encode"], "GB/s": encode_bytes(N, K, cfg) / seg["encode"] / 1e6,
                   "frac_of_hbm_" + pk_kind: encode_bytes(N, K, cfg) / seg["encode"] / 1e6 / pk["hbm_gbs"]},
    }
    for M in MS:
        for ps in ("fwd", "bwd"):
            ms = seg[f"{ps}{M}"]
            ent = {"ms": ms, "TFLOP/s": linear_flops(M, N, K, r) / ms / 1e9}
            if M > 64:
                ent["frac_of_bf16_" + pk_kind] = ent["TFLOP/s"] / pk["bf16_tflops"]
                ent["frac_of_bf16_nominal"] = ent["TFLOP/s"] / NOMINAL["bf16_tflops"]
            else:
                ent["packed_GB/s"] = pbytes / ms / 1e6
                ent["frac_of_hbm_" + pk_kind] = ent["packed_GB/s"] / pk["hbm_gbs"]
                ent["frac_of_hbm_nominal"] = ent["packed_GB/s"] / NOMINAL["hbm_gbs"]
                ent["all_bytes_GB/s"] = (small_bytes + 2 * M * (N + K)) / ms / 1e6
            lms = loops[f"{ps}{M}"]
            if M > 64:
                ent["back_to_back"] = {"ms": lms, "TFLOP/s": linear_flops(M, N, K, r) / lms / 1e9,
                                       "frac_of_bf16_" + pk_kind: linear_flops(M, N, K, r) / lms / 1e9 / pk["bf16_tflops"]}
            else:
                ent["back_to_back"] = {"ms": lms, "packed_GB/s": pbytes / lms / 1e6,
                                       "frac_of_hbm_" + pk_kind: pbytes / lms / 1e6 / pk["hbm_gbs"],
                                       "how": loop_kind[f"{ps}{M}"]}
            breakdown[f"{ps}_M{M}"] = ent

    gms = loops["grads2048"]
    gbytes = 2.0 * 2048 * (N + K)          # X and dY read once (bf16)
    breakdown["extra_lora_grads_M2048"] = {
        "ms": gms, "how": loop_kind["grads2048"], "in_timed_step": False,
        "GB/s": gbytes / gms / 1e6, "frac_of_hbm_" + pk_kind: gbytes / gms / 1e6 / pk["hbm_gbs"],
        "TFLOP/s": 8.0 * 2048 * r * (N + K) / gms / 1e9,
        "what": "lqlora_lora_grads: dL1 = dY^T (X L2^T), dL2 = (dY L1)^T X; bytes = X and dY read once"}

    # dominant kernel: the tensor-core linear (forward and input gradient at M = 2048)
    tc_ms = 0.5 * (loops["fwd2048"] + loops["bwd2048"])
    achieved = linear_flops(2048, N, K, r) / tc_ms / 1e9
    roofline = {"bound": "tensor", "achieved": achieved, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / pk["bf16_tflops"], "traffic": TC_TRAFFIC_BYTES,
                "kernel": "tc_pair_linear_kernel (mean of lqlora_linear_fwd and lqlora_linear_bwd_input at M=2048, launched back to "
                          f"back over {nrot} rotating activation buffers larger than L2; the rank-r pre-product kernel runs "
                          "beside it on the SMs its last wave leaves idle)",
                "ms_per_launch": tc_ms,
                "peak_kind": pk_kind + " cuBLAS bf16 burst", "frac_of_nominal_2250": achieved / NOMINAL["bf16_tflops"]}

    oflops, osec, odesc = oracle_sample(spec, A, l1b, l2b, rows_large=256)
    import oracle
    cpu = {"value": oflops / osec / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
           "sample": odesc, "seconds": osec}

    h2d = W_host.numel() * 4 + sum(XH[M].numel() * 2 + GH[M].numel() * 2 for M in MS)
    d2h = sum(YH[M].numel() * 2 + DXH[M].numel() * 2 for M in MS)
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "N": N, "K": K, "rank": r, "M": list(MS), "quant": list(cfg.as_tuple()),
                   "parallelism": f"dp{world} over tokens, weights replicated, no collective",
                   "l2": "flushed between steps by a 256 MiB device write followed by a 256 MiB device read (clean lines), both outside the timed events; decode-sized "
                         f"calls rotate over {ncopies} cold copies of the packed matrix",
                   "wall_ms_per_step_incl_flush": t_wall / args.steps * 1e3},
        "clocks": clocks,
        "e2e": {"value": world * step_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "breakdown": breakdown,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_sweep(args):
    """Sweep of one 8192 x 8192 matrix (b0 x B0 x M): encode GB/s, forward / input-gradient throughput and the
    fraction of the binding roofline per point, as a text table on stdout (not the one-line contract)."""
    import torch
    from paper_2311_12023_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk, pk_kind = peaks()
    N = K = 8192
    r = inputs.RANK
    W = torch.from_numpy(inputs.gaussian(5000, (N, K), 0.02)).to(dev)
    l1b, l2b = inputs.lowrank_factors(5700, N, K, r, 0.01)
    L1, L2 = binding.bf16_from_bits(l1b, dev), binding.bf16_from_bits(l2b, dev)
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    Ms = [int(m) for m in args.sweep_ms.split(",")]
    print(f"# sweep on one {N}x{K} matrix, rank {r}; peaks ({pk_kind}): HBM {pk['hbm_gbs']:.0f} GB/s, bf16 {pk['bf16_tflops']:.0f} TFLOP/s")
    print("# M <= 16: packed-weight GB/s and fraction of HBM peak (calls replayed as a CUDA graph over cold copies);")
    print("# M >= 128: algorithmic TFLOP/s and fraction of the bf16 peak (back to back over rotating activation buffers)")
    print(f"{'b0':>3} {'B0':>4} {'bits':>6} {'enc GB/s':>9} {'enc frac':>8} " + " ".join(f"{'fwd M=' + str(m):>12} {'frac':>6} {'bwd M=' + str(m):>12} {'frac':>6}" for m in Ms))

    def timed(fn, count):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / count

    for b0 in (2, 3, 4, 8):
        for B0 in (16, 32, 64, 128, 256):
            cfg = inputs.QuantConfig(b0, B0, 8, 256, 32)
            q = binding.alloc_qmatrix(N, K, cfg, dev)
            enc_ws = torch.empty(binding.packed_sizes(N, K, cfg)[3], dtype=torch.uint8, device=dev)
            enc_ms = timed(lambda: [binding.encode(W, cfg, out=q, workspace=enc_ws) for _ in range(3)], 3)
            enc_gbs = encode_bytes(N, K, cfg) / enc_ms / 1e6
            pbytes = packed_bytes(N, K, cfg)
            ncopies = max(2, int(2.2 * l2_bytes / q.packed_bytes) + 1)
            copies = [binding.QMatrix(q.codes.clone(), q.scale_codes.clone(), q.scale2.clone(), N, K, cfg) for _ in range(ncopies)]
            cells = []
            for M in Ms:
                X = binding.bf16_from_bits(inputs.activations(5200 + M, M, K), dev)
                G = binding.bf16_from_bits(inputs.activations(5300 + M, M, N), dev)
                ws = binding.alloc_workspace(q, r, M)
                for bwd in (False, True):
                    fn = binding.linear_bwd_input if bwd else binding.linear_fwd
                    A = G if bwd else X
                    if M <= 16:
                        out = torch.empty((M, K if bwd else N), dtype=torch.bfloat16, device=dev)

                        def body():
                            for c in copies:
                                fn(c, L1, L2, A, out=out, workspace=ws)
                        body()
                        torch.cuda.synchronize()
                        g = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(g):
                            body()
                        ms = timed(g.replay, ncopies)
                        val = pbytes / ms / 1e6
                        cells.append(f"{val:9.0f}GB/s {val / pk['hbm_gbs']:6.3f}")
                    else:
                        nrot = max(2, int(1.1 * l2_bytes / (M * (N + K) * 2)) + 1) if M < 8192 else 2
                        As = [A.clone() for _ in range(nrot)]
                        outs = [torch.empty((M, K if bwd else N), dtype=torch.bfloat16, device=dev) for _ in range(nrot)]
                        reps = max(2, min(4 * nrot, 16))
                        ms = timed(lambda: [fn(q, L1, L2, As[i % nrot], out=outs[i % nrot], workspace=ws) for i in range(reps)], reps)
                        val = linear_flops(M, N, K, r) / ms / 1e9
                        cells.append(f"{val:8.0f}TF/s {val / pk['bf16_tflops']:6.3f}")
                        del As, outs
            bits = cfg.b0 + cfg.b1 / cfg.B0 + cfg.b2 / (cfg.B0 * cfg.B1)
            print(f"{b0:>3} {B0:>4} {bits:6.3f} {enc_gbs:9.0f} {enc_gbs / pk['hbm_gbs']:8.3f} " + " ".join(cells), flush=True)
            del copies, q


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="print the b0 x B0 x M table of the 8192 x 8192 sweep instead")
    ap.add_argument("--sweep-ms", default="1,16,128,2048,8192")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_device(args)


if __name__ == "__main__":
    main()
