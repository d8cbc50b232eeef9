#!/usr/bin/env python
"""Benchmark of the LQ-LoRA linear hot path on B200.

One step = one pass of the whole hot path over the LLaMA-2-70B decoder-layer workload (seeded synthetic
data: q, o 8192x8192; k, v 1024x8192; gate, up 28672x8192; down 8192x28672; per-matrix mixed
configurations averaging about 2.73 bits per parameter; rank 64):

    encode of all seven matrices
    -> forward of all seven at M = 2048, input gradient of all seven at M = 2048   (tensor-core kernels)
    -> forward of all seven at M = 1,    input gradient of all seven at M = 1      (weight-streaming kernels)

`value` is the algorithmic TFLOP/s of the whole step: 2 M (N K + r K + N r) flop per linear call, summed
over the 28 calls, divided by the device time of the step (CUDA events).  The JSON line also carries the
roofline of the dominant kernel (the CTA-pair tcgen05 kernel on the 28672x8192 gate projection), per-call
figures of the step, the other seeded workloads (RoBERTa projection, LLaMA-2-7B attention projection and MLP
block, points of the 8192x8192 sweep) measured beside it, the end-to-end number through the host-buffer
C ABI, and the CPU oracle timed on the host as a baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
    python bench.py --sweep                      # the whole b0 x B0 x M table of the 8192x8192 sweep
    python bench.py --case gate --case-m 2048    # one matrix of the layer alone (small footprint, for profilers)

With N > 1 every rank runs the same per-GPU workload on its own tokens (data parallel over tokens, weights
replicated, no collective on the data path); time is the max over ranks.  Launched by torchrun the ranks
read RANK / LOCAL_RANK / WORLD_SIZE; without them `--gpus N` starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
WORKLOAD = ("llama2-70b decoder layer (GQA): q,o 8192x8192; k,v 1024x8192; gate,up 28672x8192; down 8192x28672; "
            "per-matrix mixed configs (about 2.73 bits/param), r=64; encode of all seven + fwd/dX of all seven at M=2048 and M=1")
MS = (2048, 1)
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (tc_pair_linear_kernel<3, forward> on
# the gate projection at M = 2048: 231.5 MB read + 101.4 MB written), from an ncu capture of
# `python bench.py --case gate --case-m 2048 --case-reps 2` (profiles/tc_pair_linear_gate_28672x8192_m2048_ncu_full.txt);
# algorithmic bytes: X 33.6 MB + packed codes and scales 107 MB + Y 117 MB.  Set to None when that kernel changes.
DOMINANT_TRAFFIC_BYTES = 332832512


def linear_flops(M: int, N: int, K: int, r: int) -> float:
    return 2.0 * M * (N * K + r * K + N * r)


def packed_bytes(N: int, K: int, cfg) -> float:
    return N * K * (cfg.b0 + cfg.b1 / cfg.B0 + abs(cfg.b2) / (cfg.B0 * cfg.B1)) / 8.0


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
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                pw.append(float(f[3]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------- reference arm
def oracle_sample(names, rows_large: int):
    """Times the CPU oracle on a bounded sample of the layer workload: the named matrices are encoded and dequantized
    in full, then forward and input gradient run in fp64 on `rows_large` sampled rows of M = 2048 and on the M = 1 row.
    Returns (flops_done, seconds, description)."""
    import oracle
    specs = [s for s in inputs.workload(4)["matrices"] if s.name in names]
    mats = [(s,) + tuple(inputs.make_matrix(s)) for s in specs]          # generation is not timed
    r = inputs.RANK
    flops = 0.0
    t0 = time.perf_counter()
    for spec, A, l1b, l2b in mats:
        cfg = spec.cfg
        codes, _, sc, v = oracle.encode(A, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
        d32, _ = oracle.dequant(codes, sc, v, cfg.b0, cfg.B0, cfg.b1, cfg.B1)
        for M in MS:
            rows = inputs.sample_rows(900 + M, M, count=rows_large) if M > rows_large else None
            nrows = M if rows is None else len(rows)
            xb = inputs.activations(910 + M, M, spec.K)
            gb = inputs.activations(920 + M, M, spec.N)
            oracle.linear_fwd(d32, l1b, l2b, xb, rows)
            oracle.linear_bwd_input(d32, l1b, l2b, gb, rows)
            flops += 2 * linear_flops(nrows, spec.N, spec.K, r)
    dt = time.perf_counter() - t0
    desc = (f"matrices {'+'.join(names)} of the layer: encode+dequant in full, then fwd and dX in fp64 on {rows_large} sampled "
            f"rows of M=2048 and on the M=1 row (input generation untimed)")
    return flops, dt, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(("k",), rows_large=4)
    times, flops, desc = [], 0.0, ""
    for _ in range(args.steps):
        flops, dt, desc = oracle_sample(("k",), rows_large=64)
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


# ------------------------------------------------------------------------------------- ranks
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


def spawn_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: starts N copies of this script, one per GPU, with RANK / LOCAL_RANK /
    WORLD_SIZE / MASTER_ADDR / MASTER_PORT set, and waits for them.  Rank 0's output is this process's output."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=None if rank == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def run_dry(args):
    """Host logic of the multi-rank path without a device (used by the CPU tests): rendezvous over gloo, barrier,
    max over ranks of a per-rank step time, and the one JSON line from rank 0.  No kernel runs and no throughput is
    claimed: `value` is null."""
    import torch.distributed as dist
    rank, world, local = shard_info()
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
        dist.barrier()
    ms = reduce_max(10.0 + 5.0 * rank, world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": None, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms, "dry_run": True, "scaling": "weak",
                          "config": {"workload": WORKLOAD}}), flush=True)


# ------------------------------------------------------------------------------------- device helpers
class Timer:
    def __init__(self, torch):
        self.torch = torch

    def __call__(self, fn, count):
        """ms per call of `fn()` (which issues `count` calls), after one untimed run."""
        torch = self.torch
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / count


def time_linear(binding, torch, q, L1, L2, A, M, bwd, l2_bytes, timer):
    """ms per call of one direction of the linear at M rows.  M <= 16: the calls run over cold copies of the packed
    matrix (together more than twice the L2) replayed as one CUDA graph; larger M: back to back over rotating
    activation and output buffers (together larger than L2)."""
    dev = A.device
    N, K, r = q.N, q.K, (0 if L1 is None else L1.shape[1])
    fn = binding.linear_bwd_input if bwd else binding.linear_fwd
    ws = binding.alloc_workspace(q, r, M)
    out_cols = K if bwd else N
    if M <= 16:
        ncopies = max(2, int(2.2 * l2_bytes / q.packed_bytes) + 1)
        copies = [q] + [binding.QMatrix(q.codes.clone(), q.scale_codes.clone(), q.scale2.clone(), N, K, q.cfg) for _ in range(ncopies - 1)]
        out = torch.empty((M, out_cols), dtype=torch.bfloat16, device=dev)

        def body():
            for c in copies:
                fn(c, L1, L2, A, out=out, workspace=ws)
        body()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            body()
        ms = timer(g.replay, ncopies)
        how = f"cuda graph over {ncopies} cold copies"
    else:
        per = M * (N + K) * 2
        nrot = min(8, max(2, int(1.1 * l2_bytes / per) + 1))
        As = [A] + [A.clone() for _ in range(nrot - 1)]
        outs = [torch.empty((M, out_cols), dtype=torch.bfloat16, device=dev) for _ in range(nrot)]
        reps = max(2, min(4 * nrot, 16))
        ms = timer(lambda: [fn(q, L1, L2, As[i % nrot], out=outs[i % nrot], workspace=ws) for i in range(reps)], reps)
        how = f"back to back over {nrot} rotating activation buffers"
    if binding.workspace_status(ws) != 0:
        raise SystemExit("a linear kernel reported a device-side error")
    return ms, how


def linear_entry(ms, M, N, K, r, cfg, pk, pk_kind, how=None):
    """Figures of one linear call: tensor roofline for M > 16, HBM roofline on packed-weight bytes for M <= 16."""
    ent = {"ms": ms, "TFLOP/s": linear_flops(M, N, K, r) / ms / 1e9}
    if M > 16:
        ent["frac_of_bf16_" + pk_kind] = ent["TFLOP/s"] / pk["bf16_tflops"]
        ent["frac_of_bf16_nominal"] = ent["TFLOP/s"] / NOMINAL["bf16_tflops"]
    else:
        pb = packed_bytes(N, K, cfg)
        ent["packed_GB/s"] = pb / ms / 1e6
        ent["frac_of_hbm_" + pk_kind] = ent["packed_GB/s"] / pk["hbm_gbs"]
        ent["frac_of_hbm_nominal"] = ent["packed_GB/s"] / NOMINAL["hbm_gbs"]
    if how:
        ent["how"] = how
    return ent


def measure_matrix(binding, torch, dev, A, l1b, l2b, cfg, Ms, passes, pk, pk_kind, l2_bytes, timer, seed=0):
    """Encode GB/s and per-M forward / input-gradient figures of one matrix (outside the timed step)."""
    N, K = A.shape
    r = l1b.shape[1]
    W = torch.from_numpy(A).to(dev)
    L1, L2 = binding.bf16_from_bits(l1b, dev), binding.bf16_from_bits(l2b, dev)
    q = binding.alloc_qmatrix(N, K, cfg, dev)
    enc_ws = torch.empty(binding.packed_sizes(N, K, cfg)[3], dtype=torch.uint8, device=dev)
    out = {"shape": [N, K], "quant": list(cfg.as_tuple())}
    enc_ms = timer(lambda: [binding.encode(W, cfg, out=q, workspace=enc_ws) for _ in range(3)], 3)
    gbs = encode_bytes(N, K, cfg) / enc_ms / 1e6
    out["encode"] = {"ms": enc_ms, "GB/s": gbs, "frac_of_hbm_" + pk_kind: gbs / pk["hbm_gbs"]}
    del W
    for M in Ms:
        X = binding.bf16_from_bits(inputs.activations(8000 + seed + M, M, K), dev)
        G = binding.bf16_from_bits(inputs.activations(8500 + seed + M, M, N), dev)
        for ps in passes:
            if ps not in ("fwd", "bwd"):
                continue
            ms, how = time_linear(binding, torch, q, L1, L2, G if ps == "bwd" else X, M, ps == "bwd", l2_bytes, timer)
            out[f"{ps}_M{M}"] = linear_entry(ms, M, N, K, r, cfg, pk, pk_kind, how)
        del X, G
    return out


# ------------------------------------------------------------------------------------- device arm
class Mat:
    pass


def build_layer(binding, torch, dev, rank, host_copy):
    """Device-resident state of the seven matrices of the layer (weights replicated on every rank; every rank draws
    its own tokens)."""
    mats = []
    r = inputs.RANK
    for spec in inputs.workload(4)["matrices"]:
        m = Mat()
        m.spec, m.cfg, m.N, m.K = spec, spec.cfg, spec.N, spec.K
        A, l1b, l2b = inputs.make_matrix(spec)
        m.W_host = torch.from_numpy(A).pin_memory() if host_copy else None
        m.W = torch.from_numpy(A).to(dev)
        del A
        m.L1, m.L2 = binding.bf16_from_bits(l1b, dev), binding.bf16_from_bits(l2b, dev)
        m.q = binding.alloc_qmatrix(m.N, m.K, m.cfg, dev)
        m.enc_ws = torch.empty(binding.packed_sizes(m.N, m.K, m.cfg)[3], dtype=torch.uint8, device=dev)
        m.ws = {M: binding.alloc_workspace(m.q, r, M) for M in MS}
        mats.append(m)
    # activations: q, k, v read the same input, gate and up read the same input (as in the layer); every matrix has its
    # own output gradient
    groups = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "gate": "mlp_in", "up": "mlp_in", "down": "down_in"}
    XH, X = {}, {}
    for m in mats:
        m.X, m.XH, m.G, m.GH, m.Y, m.DX, m.YH, m.DXH = {}, {}, {}, {}, {}, {}, {}, {}
        for M in MS:
            key = (groups[m.spec.name], M)
            if key not in X:
                h = torch.from_numpy(inputs.activations(7000 + 10 * rank + M + 100 * len(X), M, m.K).view(np.int16)).view(torch.bfloat16)
                XH[key] = h.pin_memory() if host_copy else h
                X[key] = XH[key].to(dev)
            m.X[M], m.XH[M] = X[key], XH[key]
            g = torch.from_numpy(inputs.activations(7500 + 10 * rank + M + 100 * mats.index(m), M, m.N).view(np.int16)).view(torch.bfloat16)
            m.GH[M] = g.pin_memory() if host_copy else g
            m.G[M] = m.GH[M].to(dev)
            m.Y[M] = torch.empty((M, m.N), dtype=torch.bfloat16, device=dev)
            m.DX[M] = torch.empty((M, m.K), dtype=torch.bfloat16, device=dev)
            if host_copy:
                m.YH[M] = torch.empty((M, m.N), dtype=torch.bfloat16).pin_memory()
                m.DXH[M] = torch.empty((M, m.K), dtype=torch.bfloat16).pin_memory()
    return mats


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
    timer = Timer(torch)
    pk, pk_kind = peaks()
    r = inputs.RANK
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size

    mats = build_layer(binding, torch, dev, rank, host_copy=True)
    for m in mats:
        binding.encode(m.W, m.cfg, out=m.q, workspace=m.enc_ws)
    torch.cuda.synchronize()

    # the calls of one step, in layer order: (label, kind, matrix, M, callable)
    calls = []
    for m in mats:
        calls.append((f"encode_{m.spec.name}", "encode", m, 0, lambda m=m: binding.encode(m.W, m.cfg, out=m.q, workspace=m.enc_ws)))
    for M in MS:
        for m in mats:
            calls.append((f"fwd{M}_{m.spec.name}", "fwd", m, M,
                          lambda m=m, M=M: binding.linear_fwd(m.q, m.L1, m.L2, m.X[M], out=m.Y[M], workspace=m.ws[M])))
        for m in reversed(mats):
            calls.append((f"bwd{M}_{m.spec.name}", "bwd", m, M,
                          lambda m=m, M=M: binding.linear_bwd_input(m.q, m.L1, m.L2, m.G[M], out=m.DX[M], workspace=m.ws[M])))
    ncalls = len(calls)

    def one_step(events=None):
        """The whole hot path once, device-resident inputs; one CUDA event after every call."""
        if events:
            events[0].record()
        for i, c in enumerate(calls):
            c[4]()
            if events:
                events[i + 1].record()

    def one_step_host():
        """Same step through the host-buffer C ABI: H2D of W, X, dY and D2H of Y, dX inside."""
        for m in mats:
            binding.encode_host(m.W_host, m.W, m.q, m.enc_ws)
        for M in MS:
            for m in mats:
                binding.linear_fwd_host(m.q, m.L1, m.L2, m.XH[M], m.YH[M], m.X[M], m.Y[M], m.ws[M])
            for m in reversed(mats):
                binding.linear_bwd_input_host(m.q, m.L1, m.L2, m.GH[M], m.DXH[M], m.G[M], m.DX[M], m.ws[M])

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    for m in mats:
        for M in MS:
            st = binding.workspace_status(m.ws[M])
            if st != 0:
                raise SystemExit(f"kernel reported {binding.status_string(st)}")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(ncalls + 1)] for _ in range(args.steps)]
    launches0 = binding.launch_count()
    barrier()
    t_wall0 = time.perf_counter()
    for s in range(args.steps):
        one_step(evs[s])
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = binding.launch_count() - launches0
    step_ms = [evs[s][0].elapsed_time(evs[s][ncalls]) for s in range(args.steps)]
    call_ms = np.zeros((args.steps, ncalls))
    for s in range(args.steps):
        for i in range(ncalls):
            call_ms[s, i] = evs[s][i].elapsed_time(evs[s][i + 1])
    ms_step = reduce_max(sum(step_ms) / len(step_ms), world, dev)

    # end to end through the host-buffer entry points
    for _ in range(2):
        one_step_host()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(3, min(args.steps, 5))
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

    # ---- the step, call by call (mean over the timed steps of the event intervals)
    mean_ms = call_ms.mean(axis=0)
    step_flops = sum(linear_flops(M, m.N, m.K, r) for (_, kind, m, M, _) in calls if kind != "encode")
    value = world * step_flops / (ms_step * 1e-3) / 1e12
    layer = {}
    for i, (label, kind, m, M, _) in enumerate(calls):
        if kind == "encode":
            gbs = encode_bytes(m.N, m.K, m.cfg) / mean_ms[i] / 1e6
            layer[label] = {"ms": float(mean_ms[i]), "GB/s": gbs, "frac_of_hbm_" + pk_kind: gbs / pk["hbm_gbs"],
                            "shape": [m.N, m.K], "quant": list(m.cfg.as_tuple())}
        else:
            layer[label] = linear_entry(float(mean_ms[i]), M, m.N, m.K, r, m.cfg, pk, pk_kind)
    phases = {}
    for ph in ("encode",) + tuple(f"{k}{M}" for M in MS for k in ("fwd", "bwd")):
        idx = [i for i, c in enumerate(calls) if c[0].startswith(ph + "_")]
        ms = float(mean_ms[idx].sum())
        ent = {"ms": ms}
        if ph == "encode":
            b = sum(encode_bytes(m.N, m.K, m.cfg) for m in mats)
            ent["GB/s"] = b / ms / 1e6
            ent["frac_of_hbm_" + pk_kind] = ent["GB/s"] / pk["hbm_gbs"]
        else:
            M = int(ph[3:])
            fl = sum(linear_flops(M, m.N, m.K, r) for m in mats)
            ent["TFLOP/s"] = fl / ms / 1e9
            if M > 16:
                ent["frac_of_bf16_" + pk_kind] = ent["TFLOP/s"] / pk["bf16_tflops"]
                ent["frac_of_bf16_sustained_" + pk_kind] = ent["TFLOP/s"] / pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
                ent["frac_of_bf16_nominal"] = ent["TFLOP/s"] / NOMINAL["bf16_tflops"]
            else:
                b = sum(packed_bytes(m.N, m.K, m.cfg) for m in mats)
                ent["packed_GB/s"] = b / ms / 1e6
                ent["frac_of_hbm_" + pk_kind] = ent["packed_GB/s"] / pk["hbm_gbs"]
                ent["frac_of_hbm_nominal"] = ent["packed_GB/s"] / NOMINAL["hbm_gbs"]
        phases[ph] = ent

    # ---- roofline of the dominant kernel: the CTA-pair tcgen05 kernel on the gate projection (forward, M = 2048),
    # timed by the events around that call inside the timed steps
    gi = [i for i, c in enumerate(calls) if c[0] == "fwd2048_gate"][0]
    gate = calls[gi][2]
    g_ms = float(mean_ms[gi])
    achieved = linear_flops(2048, gate.N, gate.K, r) / g_ms / 1e9
    sustained = pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
    roofline = {"bound": "tensor", "achieved": achieved, "peak": sustained, "unit": "TFLOP/s", "frac": achieved / sustained,
                "traffic": DOMINANT_TRAFFIC_BYTES,
                "kernel": f"tc_pair_linear_kernel<{gate.cfg.b0}, forward> on gate {gate.N}x{gate.K} at M=2048 (with the rank-r pre-product kernel "
                          "that runs beside it); duration = mean over the timed steps of the CUDA-event interval around the call",
                "ms_per_launch": g_ms, "ms_per_launch_median": float(np.median(call_ms[:, gi])),
                "ms_per_launch_min_max": [float(call_ms[:, gi].min()), float(call_ms[:, gi].max())],
                "flop_per_launch": linear_flops(2048, gate.N, gate.K, r),
                "peak_kind": pk_kind + " cuBLAS bf16, sustained figure (the kernel is timed inside a long step)",
                "frac_of_burst_" + pk_kind: achieved / pk["bf16_tflops"], "frac_of_nominal_2250": achieved / NOMINAL["bf16_tflops"]}

    # ---- the decode-sized calls of the layer once more, each matrix alone over cold copies as one CUDA graph
    decode = {}
    for m in mats:
        for ps in ("fwd", "bwd"):
            ms, how = time_linear(binding, torch, m.q, m.L1, m.L2, m.G[1] if ps == "bwd" else m.X[1], 1, ps == "bwd", l2_bytes, timer)
            decode[f"{ps}1_{m.spec.name}"] = linear_entry(ms, 1, m.N, m.K, r, m.cfg, pk, pk_kind, how)
    # gradients of the low-rank factors on the gate projection at M = 2048 (the next piece of a training step; not
    # part of the timed step)
    gm = gate
    dL = (torch.empty(gm.N, r, dtype=torch.float32, device=dev), torch.empty(r, gm.K, dtype=torch.float32, device=dev))
    gws = torch.empty(binding.lora_grads_workspace_bytes(gm.N, gm.K, r, 2048), dtype=torch.uint8, device=dev)
    g_ms2 = timer(lambda: [binding.lora_grads(gm.L1, gm.L2, gm.X[2048], gm.G[2048], out=dL, workspace=gws) for _ in range(4)], 4)
    if binding.workspace_status(gws) != 0:
        raise SystemExit("lora_grads reported a device-side error")
    gbytes = 2.0 * 2048 * (gm.N + gm.K)
    extra = {"lora_grads_gate_M2048": {"ms": g_ms2, "GB/s": gbytes / g_ms2 / 1e6, "frac_of_hbm_" + pk_kind: gbytes / g_ms2 / 1e6 / pk["hbm_gbs"],
                                       "in_timed_step": False, "what": "lqlora_lora_grads; bytes = X and dY read once"}}
    # the same gradients from the intermediates that the forward and the input-gradient call left in their workspaces
    ws_f, ws_b = binding.alloc_workspace(gm.q, r, 2048), binding.alloc_workspace(gm.q, r, 2048)
    binding.linear_fwd(gm.q, gm.L1, gm.L2, gm.X[2048], workspace=ws_f)
    binding.linear_bwd_input(gm.q, gm.L1, gm.L2, gm.G[2048], workspace=ws_b)
    T = binding.linear_intermediate(ws_f, gm.N, gm.K, gm.cfg, r, 2048, False)
    Tp = binding.linear_intermediate(ws_b, gm.N, gm.K, gm.cfg, r, 2048, True)
    sws = torch.empty(256, dtype=torch.uint8, device=dev)
    g_ms3 = timer(lambda: [binding.lora_grads_from(T, Tp, gm.N, gm.K, gm.X[2048], gm.G[2048], out=dL, workspace=sws) for _ in range(4)], 4)
    if binding.workspace_status(sws) != 0:
        raise SystemExit("lora_grads_from reported a device-side error")
    extra["lora_grads_from_gate_M2048"] = {"ms": g_ms3, "GB/s": gbytes / g_ms3 / 1e6, "frac_of_hbm_" + pk_kind: gbytes / g_ms3 / 1e6 / pk["hbm_gbs"],
                                           "in_timed_step": False, "what": "lqlora_lora_grads_from (T, T' reused); bytes = X and dY read once"}
    del ws_f, ws_b

    h2d = sum(m.W_host.numel() * 4 + sum(m.XH[M].numel() * 2 + m.GH[M].numel() * 2 for M in MS) for m in mats)
    d2h = sum(sum(m.YH[M].numel() * 2 + m.DXH[M].numel() * 2 for M in MS) for m in mats)
    del mats, calls, gate, gm
    torch.cuda.empty_cache()

    # ---- the other seeded workloads, measured beside the step (not part of `value`)
    other = {}
    if not args.no_configs:
        w1 = inputs.workload(1)
        A, l1b, l2b = inputs.make_matrix(w1["matrices"][0])
        other["config1_roberta_proj"] = measure_matrix(binding, torch, dev, A, l1b, l2b, w1["matrices"][0].cfg, [512], ("fwd",), pk, pk_kind, l2_bytes, timer)
        w2 = inputs.workload(2)
        A, l1b, l2b = inputs.make_matrix(w2["matrices"][0])
        other["config2_llama7b_attn_proj"] = measure_matrix(binding, torch, dev, A, l1b, l2b, w2["matrices"][0].cfg, [1, 16, 2048], ("fwd", "bwd"), pk, pk_kind, l2_bytes, timer)
        c3 = {}
        for spec in inputs.workload(3)["matrices"]:
            A, l1b, l2b = inputs.make_matrix(spec)
            c3[spec.name] = measure_matrix(binding, torch, dev, A, l1b, l2b, spec.cfg, [4096], ("fwd", "bwd"), pk, pk_kind, l2_bytes, timer)
        other["config3_llama7b_mlp"] = c3
        A = inputs.gaussian(5000, (8192, 8192), 0.02)
        l1b, l2b = inputs.lowrank_factors(5700, 8192, 8192, r, 0.01)
        c5 = {}
        for b0, B0 in ((3, 64), (2, 16), (2, 256), (8, 16), (8, 256)):
            cfg = inputs.QuantConfig(b0, B0, 8, 256, 32)
            c5[f"b{b0}_B{B0}"] = measure_matrix(binding, torch, dev, A, l1b, l2b, cfg, [1, 16, 128, 2048, 8192], ("fwd", "bwd"), pk, pk_kind, l2_bytes, timer)
        other["config5_sweep_points_8192x8192"] = c5
        del A

    oflops, osec, odesc = oracle_sample(("q", "k"), rows_large=256)
    import oracle
    cpu = {"value": oflops / osec / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
           "sample": odesc, "seconds": osec}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "rank": r, "M": list(MS), "calls_per_step": ncalls,
                   "parallelism": f"dp{world} over tokens, weights replicated, no collective",
                   "l2": "inputs larger than L2: a step reads 3.4 GB of fp32 weights, 0.29 GB of packed codes per pass and 0.5 GB of "
                         "activations, and no buffer is touched twice within 126 MB of traffic except the shared inputs of q/k/v and gate/up",
                   "ms_per_step_median": float(statistics.median(step_ms)), "ms_per_step_min_max": [min(step_ms), max(step_ms)],
                   "wall_ms_per_step": t_wall / args.steps * 1e3},
        "clocks": clocks,
        "e2e": {"value": world * step_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "breakdown": {"phases": phases, "calls": layer, "decode_calls_alone": decode, "extra": extra, "other_configs": other},
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_case(args):
    """One matrix of the layer alone, with random packed codes (no fp32 weights on the device): a few forward and
    input-gradient calls at one M.  Holds well under 1 GB, so that a profiler can capture the kernels of the largest
    shapes on their own."""
    import torch
    from paper_2311_12023_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    spec = [s for s in inputs.workload(4)["matrices"] if s.name == args.case][0]
    if args.case_cfg:
        import dataclasses
        spec = dataclasses.replace(spec, cfg=inputs.QuantConfig(*[int(x) for x in args.case_cfg.split(",")]))
    M, r = args.case_m, (inputs.RANK if args.case_r is None else args.case_r)
    q = binding.alloc_qmatrix(spec.N, spec.K, spec.cfg, dev)
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    if args.case_encode:
        # the encoder alone: seeded Gaussian weights made on the device (no host copy of the largest matrices)
        W = torch.empty((spec.N, spec.K), dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=g)
        enc_ws = torch.empty(binding.packed_sizes(spec.N, spec.K, spec.cfg)[3], dtype=torch.uint8, device=dev)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.case_reps + 1)]
        evs[0].record()
        for i in range(args.case_reps):
            binding.encode(W, spec.cfg, out=q, workspace=enc_ws)
            evs[i + 1].record()
        torch.cuda.synchronize()
        ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.case_reps)]
        gbs = [encode_bytes(spec.N, spec.K, spec.cfg) / t / 1e6 for t in ms]
        print(json.dumps({"case": args.case, "shape": [spec.N, spec.K], "quant": list(spec.cfg.as_tuple()),
                          "encode_ms": ms, "encode_GB/s": gbs}), flush=True)
        return
    q.codes.random_(0, 256, generator=g)
    q.scale_codes.random_(1, 128, generator=g)
    q.scale2.fill_(0.05)
    L1 = L2 = None
    if r > 0:
        l1b, l2b = inputs.lowrank_factors(spec.seed + 700, spec.N, spec.K, r, 0.01)
        L1, L2 = binding.bf16_from_bits(l1b, dev), binding.bf16_from_bits(l2b, dev)
    X = binding.bf16_from_bits(inputs.activations(1, M, spec.K), dev)
    G = binding.bf16_from_bits(inputs.activations(2, M, spec.N), dev)
    ws = binding.alloc_workspace(q, r, M)
    Y = torch.empty((M, spec.N), dtype=torch.bfloat16, device=dev)
    DX = torch.empty((M, spec.K), dtype=torch.bfloat16, device=dev)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.case_reps + 1)]
    evs[0].record()
    for i in range(args.case_reps):
        binding.linear_fwd(q, L1, L2, X, out=Y, workspace=ws)
        evs[2 * i + 1].record()
        binding.linear_bwd_input(q, L1, L2, G, out=DX, workspace=ws)
        evs[2 * i + 2].record()
    torch.cuda.synchronize()
    if binding.workspace_status(ws) != 0:
        raise SystemExit("a linear kernel reported a device-side error")
    f = [evs[2 * i].elapsed_time(evs[2 * i + 1]) for i in range(args.case_reps)]
    b = [evs[2 * i + 1].elapsed_time(evs[2 * i + 2]) for i in range(args.case_reps)]
    print(json.dumps({"case": args.case, "shape": [spec.N, spec.K], "quant": list(spec.cfg.as_tuple()), "M": M,
                      "fwd_ms": f, "bwd_ms": b}), flush=True)


def run_sweep(args):
    """Sweep of one 8192 x 8192 matrix (b0 x B0 x M): encode GB/s, forward / input-gradient throughput and the
    fraction of the binding roofline per point, as a text table on stdout (not the one-line contract)."""
    import torch
    from paper_2311_12023_b200 import binding

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk, pk_kind = peaks()
    timer = Timer(torch)
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
    for b0 in (2, 3, 4, 8):
        for B0 in (16, 32, 64, 128, 256):
            cfg = inputs.QuantConfig(b0, B0, 8, 256, 32)
            q = binding.alloc_qmatrix(N, K, cfg, dev)
            enc_ws = torch.empty(binding.packed_sizes(N, K, cfg)[3], dtype=torch.uint8, device=dev)
            enc_ms = timer(lambda: [binding.encode(W, cfg, out=q, workspace=enc_ws) for _ in range(3)], 3)
            enc_gbs = encode_bytes(N, K, cfg) / enc_ms / 1e6
            pbytes = packed_bytes(N, K, cfg)
            cells = []
            for M in Ms:
                X = binding.bf16_from_bits(inputs.activations(5200 + M, M, K), dev)
                G = binding.bf16_from_bits(inputs.activations(5300 + M, M, N), dev)
                for bwd in (False, True):
                    ms, _ = time_linear(binding, torch, q, L1, L2, G if bwd else X, M, bwd, l2_bytes, timer)
                    if M <= 16:
                        val = pbytes / ms / 1e6
                        cells.append(f"{val:9.0f}GB/s {val / pk['hbm_gbs']:6.3f}")
                    else:
                        val = linear_flops(M, N, K, r) / ms / 1e9
                        cells.append(f"{val:8.0f}TF/s {val / pk['bf16_tflops']:6.3f}")
            bits = cfg.b0 + cfg.b1 / cfg.B0 + cfg.b2 / (cfg.B0 * cfg.B1)
            print(f"{b0:>3} {B0:>4} {bits:6.3f} {enc_gbs:9.0f} {enc_gbs / pk['hbm_gbs']:8.3f} " + " ".join(cells), flush=True)
            del q


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-configs", action="store_true", help="skip the per-config figures measured beside the step")
    ap.add_argument("--dry-run", action="store_true", help="host logic of the multi-rank path only (gloo, no device work)")
    ap.add_argument("--sweep", action="store_true", help="print the b0 x B0 x M table of the 8192 x 8192 sweep instead")
    ap.add_argument("--sweep-ms", default="1,16,128,2048,8192")
    ap.add_argument("--case", default=None, help="run one matrix of the layer alone (q, k, v, o, gate, up, down)")
    ap.add_argument("--case-m", type=int, default=2048)
    ap.add_argument("--case-reps", type=int, default=3)
    ap.add_argument("--case-cfg", default=None, help="with --case: another configuration b0,B0,b1,B1,b2 for that matrix's shape")
    ap.add_argument("--case-r", type=int, default=None, help="with --case: rank of the low-rank term (0 = none; default 64)")
    ap.add_argument("--case-encode", action="store_true", help="with --case: time lqlora_encode of that matrix instead of the linear calls")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.case:
        run_case(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.dry_run:
        run_dry(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_device(args)


if __name__ == "__main__":
    main()
