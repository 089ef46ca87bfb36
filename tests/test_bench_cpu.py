"""Host logic of bench.py that runs without a GPU: the max-over-ranks aggregation of the replica runs on two gloo
ranks, and the reference arm (the CPU oracle) under a two-process launch, where rank 0 alone works and prints."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], torch.device("cpu"))
assert got == [11.0, 5.0], got
open(os.path.join({out!r}, "rank%d.txt" % rank), "w").write(repr(got))
dist.destroy_process_group()
"""


def _torchrun(args, timeout):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="4")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", "29617"] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_on_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT, out=str(tmp_path)))
    r = _torchrun([str(script)], timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    for rank in (0, 1):
        assert (tmp_path / f"rank{rank}.txt").read_text() == "[11.0, 5.0]"


def test_reference_arm_prints_one_line_from_rank_zero_under_a_two_process_launch():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"], timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in (r.stdout + "\n" + r.stderr).splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert line["unit"] == "tokens/s" and line["higher_is_better"] is True
