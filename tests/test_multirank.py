"""The N > 1 plumbing of bench.py on CPU: two gloo ranks.  The path shards by replicas / batch rows
with no exchange step, so the only multi-rank logic is the barrier, the MAX of the per-rank device
time, and the whole-job aggregate; the reference arm runs on rank 0 alone."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
assert bench.max_over_ranks(3.5) == 3.5            # no group yet: identity
dist.init_process_group("gloo")
bench.barrier()
slow = bench.max_over_ranks(10.0 + 5.0 * rank)      # rank 1 is the slow one
steps, batch = 4, 16
value = world * batch * steps / (slow / 1e3)
print(json.dumps({{"rank": rank, "max_ms": slow, "value": value}}), flush=True)
bench.barrier()
dist.destroy_process_group()
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def run_ranks(code, world=2, extra_env=None, args=()):
    port = free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, "-c", code, *args], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            out, err = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_two_gloo_ranks_agree_on_max_time_and_aggregate():
    outs = run_ranks(WORKER.format(root=ROOT))
    lines = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["max_ms"] == 15.0                                  # the slower rank decides
        assert l["value"] == pytest.approx(2 * 16 * 4 / 15e-3)      # units of all ranks / that time


def test_reference_arm_runs_on_rank_zero_only():
    code = ("import sys; sys.path.insert(0, %r); import bench; "
            "bench.main(['--impl', 'reference', '--gpus', '2', '--steps', '1', '--warmup', '0', "
            "'--workload', 'tiny'])" % ROOT)
    outs = run_ranks(code)
    assert outs[1].strip() == ""                                    # rank 1 exits 0 without work
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
