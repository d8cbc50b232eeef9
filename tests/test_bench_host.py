"""Host-side logic of bench.py: flop / byte accounting, the JSON line of the reference arm, and the
multi-process path (replicas over tokens, max-over-ranks timing) on two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2311_12023_b200 import inputs  # noqa: E402


def test_flop_and_byte_accounting():
    cfg = inputs.QuantConfig(3, 64, 8, 256, 32)
    # 2 M (N K + r K + N r): the quantized product plus both rank-r products
    assert bench.linear_flops(2048, 4096, 4096, 64) == 2.0 * 2048 * (4096 * 4096 + 64 * 4096 + 4096 * 64)
    # Eq. (2): 3 + 8/64 + 32/(64*256) bits per weight
    assert bench.packed_bytes(4096, 4096, cfg) == 4096 * 4096 * (3 + 8 / 64 + 32 / (64 * 256)) / 8
    assert bench.encode_bytes(4096, 4096, cfg) == 4.0 * 4096 * 4096 + bench.packed_bytes(4096, 4096, cfg)
    pk, kind = bench.peaks()
    assert kind in ("measured", "fallback") and pk["hbm_gbs"] > 1000 and pk["bf16_tflops"] > 100


def test_shard_info_reads_the_launcher_environment(monkeypatch):
    monkeypatch.setenv("RANK", "3")
    monkeypatch.setenv("WORLD_SIZE", "8")
    monkeypatch.setenv("LOCAL_RANK", "3")
    assert bench.shard_info() == (3, 8, 3)
    monkeypatch.delenv("RANK")
    monkeypatch.delenv("WORLD_SIZE")
    monkeypatch.delenv("LOCAL_RANK")
    assert bench.shard_info() == (0, 1, 0)
    assert bench.reduce_max(1.5, 1) == 1.5          # single process: identity, no process group needed


_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank, world, local = bench.shard_info()
dist.init_process_group("gloo", rank=rank, world_size=world)
# every rank reports a different step time; the job's time is the slowest rank's
mine = 10.0 + 5.0 * rank
got = bench.reduce_max(mine, world)
assert got == 10.0 + 5.0 * (world - 1), got
# replicas over tokens: each rank draws its own activations (seed offset by rank), same weights
from paper_2311_12023_b200 import inputs
x = inputs.activations(7000 + 10 * rank + 16, 16, 64)
import numpy as np, torch
t = torch.from_numpy(x.astype(np.int64).sum(keepdims=True).reshape(1))
parts = [torch.zeros_like(t) for _ in range(world)]
dist.all_gather(parts, t)
assert len({int(p.item()) for p in parts}) == world, "ranks must not share tokens"
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_gloo_ranks_take_the_max_over_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29591")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
    assert all("ok" in o for o in outs)


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
    env["RANK"] = "1"
    env["WORLD_SIZE"] = "2"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_gpus_flag_starts_the_ranks_itself_and_reports_their_number():
    """`bench.py --gpus 2` without a launcher's environment starts two ranks (RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_* set per rank); they meet over gloo (--dry-run: the host logic of the multi-rank path, no device work), take
    the max over ranks of their step times (10 ms on rank 0, 15 ms on rank 1) and rank 0 alone prints the JSON line."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "2", "--warmup", "3"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["dry_run"] is True and line["ms_per_step"] == 15.0 and line["scaling"] == "weak"
    # one process when one GPU is asked for
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--dry-run"], env=env, capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0 and json.loads(out.stdout.strip().splitlines()[-1])["n_gpus"] == 1
