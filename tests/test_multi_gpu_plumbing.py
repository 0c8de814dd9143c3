"""The N>1 path of bench.py on CPU: two gloo ranks exercise the max-over-ranks timing and the
whole-job aggregation for replicas, and the reference arm prints from rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
dist.barrier()
print(json.dumps({"rank": rank, "ms": ms, "tops": bench.whole_job_tops(1e12, dist.get_world_size(), ms)}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(code_or_args, world=2, as_code=True):
    port = str(_free_port())
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=port, OMP_NUM_THREADS="2")
        cmd = [sys.executable, "-c", code_or_args] if as_code else [sys.executable] + code_or_args
        procs.append(subprocess.Popen(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_replica_aggregation_with_two_gloo_ranks():
    outs = _launch(WORKER % ROOT)
    recs = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    for r in recs:
        assert r["ms"] == 15.0                          # the slower rank's time, on every rank
        assert r["tops"] == pytest.approx(2 * 2.0 * 1e12 / 15e-3 / 1e12)


def test_reference_arm_runs_on_rank_zero_only():
    outs = _launch([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                    "--warmup", "0", "--batch", "1"], as_code=False)
    assert outs[1].strip() == ""
    rec = json.loads(outs[0].strip().splitlines()[-1])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
    assert rec["unit"] == "TOPS" and rec["higher_is_better"] is True
