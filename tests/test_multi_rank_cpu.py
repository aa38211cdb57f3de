"""The N > 1 path of bench.py on CPU: two gloo ranks rendezvous on 127.0.0.1, agree on the slowest rank's time,
and only rank 0 reports. (The data path shards by sequence with no collective, so this is all the distributed
logic there is; the kernels themselves are covered by the single-GPU parity tests.)"""
import json
import os
import subprocess
import sys

REPO = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import json, os, sys
sys.path.insert(0, os.environ["IQ_REPO"])
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
bench.init_distributed(world, 0, backend="gloo")
import torch.distributed as dist
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)            # rank 1 is the slow one
dist.barrier()
val = bench.aggregate_gbs(1e9, ms, world)
dist.destroy_process_group()
print(json.dumps({"rank": rank, "ms": ms, "value": val}), flush=True)
"""


def _spawn(world, script, extra_env=None, args=()):
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29547", IQ_REPO=REPO)
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, *script, *args], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True, cwd=REPO))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_two_gloo_ranks_agree_on_the_slowest_time():
    outs = _spawn(2, ["-c", RANK_SCRIPT])
    res = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert {r["rank"] for r in res} == {0, 1}
    for r in res:
        assert r["ms"] == 15.0                                   # max over ranks, on every rank
        assert abs(r["value"] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9    # whole-job aggregate: both replicas against that time


def test_reference_arm_under_two_ranks_reports_once():
    # rank 0 alone runs and prints the oracle's line; the other rank exits 0 without work
    outs = _spawn(2, ["bench.py"], args=("--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                                         "--workload", "config5_B1_ctx4096"))
    assert outs[1].strip() == ""
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
