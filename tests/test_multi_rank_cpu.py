"""The N > 1 paths on CPU, two gloo ranks on 127.0.0.1: bench.py's replicas (the data path shards by sequence with no
collective: the ranks agree on the slowest rank's time and only rank 0 reports) and the one exchange step the method
has when the context itself is sharded (an all-gather of the split partials, merged on every rank). The kernels
themselves are covered by the single-GPU parity tests."""
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


SHARD_SCRIPT = r"""
import json, os, sys
import numpy as np, torch
sys.path.insert(0, os.environ["IQ_REPO"]); sys.path.insert(0, os.path.join(os.environ["IQ_REPO"], "tests"))
import torch.distributed as dist
import importlib.util
spec = importlib.util.spec_from_file_location("sharded", os.path.join(os.environ["IQ_REPO"], "paper_2608_08081_b200", "sharded.py"))
sharded = importlib.util.module_from_spec(spec); spec.loader.exec_module(sharded)      # (the package itself needs the CUDA library)
import oracle, workloads
from oracle import lloyd_max
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
d, B, H_q, H_kv, T = 128, 2, 4, 2, 300
lens = np.array([300, 41], np.int32)                       # the second sequence lives on rank 0 alone
w = workloads.tiny(33, B, H_q, H_kv, d, T, lens)
lv, th = lloyd_max.fp16_codebook(d)
cut = 128                                                  # rank 0: rows [0, 128), rank 1: rows [128, T)
lo = 0 if rank == 0 else cut
my_lens = np.clip(lens - lo, 0, cut if rank == 0 else T - cut).astype(np.int32)
cache = oracle.new_cache(B, H_kv, d, workloads.cap128(T))
oracle.quantize_append(w.quats, th, w.k[:, lo:], w.v[:, lo:], np.zeros(B, np.int32), my_lens, cache)
r = oracle.decode_attention(w.quats, lv, w.q, cache, my_lens, H_kv, want_rot=True)
# this rank's slice as one split partial per head: m = max score, l = sum exp(z - m), acc = l * (normalised rotated
# output); an empty slice: (-inf, 0, 0)
S = 1
m = np.full((B, H_q), -np.inf); l = np.zeros((B, H_q))
for b in range(B):
    for h in range(H_q):
        if my_lens[b] > 0:
            z = oracle.scores(w.quats, lv, w.q, cache, b, h, int(my_lens[b]), H_kv)
            m[b, h] = z.max(); l[b, h] = np.exp(z - z.max()).sum()
acc = torch.from_numpy((r["o_rot"] * l[:, :, None]).astype(np.float32)).reshape(B, H_q, S, d)
ml = torch.from_numpy(np.stack([m, l], -1).astype(np.float32)).reshape(B, H_q, S, 2)
am = torch.from_numpy(r["argmax"].astype(np.int32)).reshape(B, H_q, S)
bufs = sharded.ShardedBuffers(B, H_q, S, d, world, True, "cpu")             # allocated once; the step below allocates nothing
bufs.set_row_offsets(torch.full((B,), lo, dtype=torch.int32))
bufs.gather(acc, ml, am)
g_acc, g_ml, g_am = bufs.slot_major()
dist.barrier(); dist.destroy_process_group()
merged = oracle.combine_splits(w.quats, g_acc.numpy(), g_ml.numpy(), g_am.numpy(), H_kv)
full = oracle.new_cache(B, H_kv, d, workloads.cap128(T))
oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, full)
ref = oracle.decode_attention(w.quats, lv, w.q, full, lens, H_kv)
print(json.dumps({"rank": rank, "splits": int(g_acc.shape[2]), "err": float(np.abs(merged["out"] - ref["out"]).max()),
                  "lse_err": float(np.abs(merged["lse"] - ref["lse"]).max()), "argmax_equal": bool(np.array_equal(merged["argmax"], ref["argmax"]))}), flush=True)
"""


def test_context_sharded_partials_merge_to_the_unsharded_result():
    """Two ranks hold rows [0, 128) and [128, 300) of every sequence (one sequence ends inside the first slice, so the
    second rank contributes an empty partial for it): the gathered partials, merged, must be the unsharded attention
    output -- on both ranks, with global argmax rows."""
    outs = _spawn(2, ["-c", SHARD_SCRIPT], extra_env={"MASTER_PORT": "29551"})
    res = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert {r["rank"] for r in res} == {0, 1}
    for r in res:
        assert r["splits"] == 2 and r["err"] < 2e-6 and r["lse_err"] < 2e-6 and r["argmax_equal"]   # partials travel as fp32
