"""Host-side logic of multi-rank runs on CPU (gloo, world size 2): ranks take disjoint synthetic clients,
the step time is the maximum over ranks, and the reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench, co3_inputs as ci
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
cfg, sizes, fmts, clients = bench.workload(2, clients_override=2)
seeds = [ci.client_round_seed(cfg["seed"] + bench.RANK_SEED_STRIDE * rank, u, 0) for u in range(clients)]
g = bench.make_grads(cfg, sizes[:3], clients, sum(sizes[:3]) + 4, 0, "cpu", rank)
out = [None] * world
dist.all_gather_object(out, dict(rank=rank, ms=ms, seeds=seeds, head=g[:4].tolist(),
                                 elems=bench.elements_per_step(sum(sizes), clients, world)))
if rank == 0:
    print(json.dumps(out))
dist.destroy_process_group()
"""


def _torchrun(args, timeout=600):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29617"] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_ranks_shard_clients_and_take_the_max_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("[{")][-1]
    out = json.loads(line)
    assert [o["rank"] for o in out] == [0, 1]
    assert out[0]["ms"] == out[1]["ms"] == 15.0                       # the slower rank's time, on every rank
    assert not set(out[0]["seeds"]) & set(out[1]["seeds"])            # different synthetic clients per rank
    assert out[0]["head"] != out[1]["head"]
    assert out[0]["elems"] == 2 * 2 * 11_181_642                      # whole-job elements: clients x ranks


def test_reference_arm_prints_once_under_two_ranks():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup",
                   "0", "--config", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "gradient elements/s"
