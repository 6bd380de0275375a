"""Host-side logic of bench.py: FLOP models, and the multi-rank reduction on two gloo ranks (CPU)."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_flop_models():
    import bench
    f, b = bench.flops_m1(4, 16, 4096, 128)
    assert abs(f / 1e12 - 0.2749) < 1e-3 and b == 2.5 * f
    f2, b2 = bench.flops_m2(4, 16, 4096, 128)
    assert f < f2 < 2 * f and b < b2 < 2 * b
    # version-chain step counts against a brute-force enumeration of (chunk, level) pairs
    N = 13
    nq, nk, nlev = bench._version_steps(N)
    bq = sum(bin(c).count("1") - 1 for c in range(1, N))
    bk = 0
    for J in range(N - 1):
        levels = [l for l in range(nlev) if not (J >> l) & 1 and (((J >> l) + 1) << l) <= N - 1]
        bk += max(len(levels) - 1, 0)
    assert (nq, nk) == (bq, bk)


WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world, local = bench.shard_info()
assert world == 2 and rank == int(os.environ["RANK"])
m = bench.max_over_ranks(10.0 + rank, world)
assert m == 11.0, m
open(os.path.join({out!r}, "rank%d.txt" % rank), "w").write("max %.1f" % m)
dist.destroy_process_group()
"""


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, out=str(tmp_path)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    assert [(tmp_path / f"rank{r}.txt").read_text() for r in (0, 1)] == ["max 11.0", "max 11.0"]


def test_reference_arm_under_torchrun_prints_one_line(tmp_path):
    """--impl reference: rank 0 alone prints the JSON line, the other rank exits 0 without work."""
    import json
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="4")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29518", os.path.join(ROOT, "bench.py"),
                          "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "C2"],
                         capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["cpu_baseline"]["kind"] == "oracle" and rec["value"] > 0
    assert rec["e2e"]["h2d_bytes_per_step"] == 0
