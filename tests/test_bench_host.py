"""Host-side logic of bench.py that needs no GPU: the replica aggregation over
two gloo ranks, and the reference arm (the CPU oracle) under one and two ranks."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
assert ms == 15.0, ms
gbs = bench.aggregate_gbs(1e9, world, ms)
assert abs(gbs - 2 * 1e9 / 15e-3 / 1e9) < 1e-9
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _env(**kw):
    env = dict(os.environ)
    env.update({k: str(v) for k, v in kw.items()})
    return env


def test_replica_aggregation_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    port = 29500 + os.getpid() % 2000
    procs = [subprocess.Popen([sys.executable, str(script)], stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True,
                              env=_env(RANK=r, WORLD_SIZE=2, LOCAL_RANK=r, MASTER_ADDR="127.0.0.1", MASTER_PORT=port))
             for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, o
        assert f"rank {r} ok" in o


@pytest.mark.parametrize("world", [1, 2])
def test_reference_arm_runs_the_oracle_on_rank_zero_only(world):
    outs = []
    for r in range(world):
        p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", str(world),
                            "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300,
                           env=_env(RANK=r, WORLD_SIZE=world, LOCAL_RANK=r))
        assert p.returncode == 0, p.stderr
        outs.append(p.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "qwen2304"
    assert all(o == "" for o in outs[1:])
