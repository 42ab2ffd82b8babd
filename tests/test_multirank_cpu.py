"""The N > 1 path of bench.py on CPU: two gloo ranks.  Rows shard across ranks with replicated
weights and no data-path collective; the only exchange is the max-over-ranks of the timed interval,
and only rank 0 prints.  Also checks the reference arm under a multi-rank launch."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
slow = bench.max_over_ranks(10.0 + 5.0 * rank)            # rank 1 is the slow one
seeds = [bench.rank_batch_seed(rank, world, r) for r in range(bench.N_SETS)]
all_seeds = [None] * world
dist.all_gather_object(all_seeds, seeds)
val = bench.whole_job_value(10**12, world, 4, slow)
dist.barrier()
if rank == 0:
    print(json.dumps({"slow": slow, "seeds": all_seeds, "value": val}))
dist.destroy_process_group()
""" % ROOT


def _launch(code_or_args, world=2, port=29577):
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        cmd = [sys.executable, "-c", code_or_args] if isinstance(code_or_args, str) else [sys.executable] + code_or_args
        procs.append(subprocess.Popen(cmd, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    return [o for o, _ in outs]


def test_two_gloo_ranks_share_only_the_timing():
    outs = _launch(WORKER)
    assert outs[1].strip() == ""                       # only rank 0 prints
    res = json.loads(outs[0])
    assert res["slow"] == 15.0                         # max over ranks, seen by every rank
    flat = [s for per_rank in res["seeds"] for s in per_rank]
    assert len(set(flat)) == len(flat)                 # every rank and working set draws its own rows
    assert abs(res["value"] - 2 * 1.0 * 4 / 15e-3) < 1e-6   # work of both ranks / slowest rank's time, TFLOP/s


def test_reference_arm_runs_on_rank_zero_only():
    outs = _launch([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                   port=29578)
    assert outs[1].strip() == ""
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["gpu_launches"] == 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
