"""Host logic of the multi-rank bench (no GPU): the path shards over the batch with no data-path
collective, so all that the ranks exchange is the slowest rank's time.  Two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")       # rank 1 is the slow one
dist.barrier()
print(json.dumps({{"rank": rank, "ms": ms, "value": bench.whole_job_value(world, 1000, ms)}}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29577")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads([l for l in out.splitlines() if l.startswith("{")][-1]))
    for o in outs:
        assert o["ms"] == pytest.approx(15.0)                      # max over ranks, on every rank
        assert o["value"] == pytest.approx(2 * 1000 / 15e-3)       # both ranks' units over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_value(1, 200704, 0.05) == pytest.approx(200704 / 0.05e-3)


def test_reference_arm_runs_on_rank_zero_only():
    """Under a multi-rank launch the other ranks of `--impl reference` exit 0 without work or output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stderr[-2000:]
    assert not [l for l in r.stdout.splitlines() if l.startswith("{")]
