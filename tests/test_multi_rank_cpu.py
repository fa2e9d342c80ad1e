"""The N > 1 host logic of the benchmark on CPU: two gloo ranks.  The decode path shards by batch
(sequences are independent, there is no exchange step), so what ranks share is only the reduction
of their figures: device times by MAX, token counts by SUM; every rank decodes its own sequences
with the same weights; the reference arm runs on rank 0 alone."""
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["PD_ROOT"])
import numpy as np
import torch
import torch.distributed as dist
import bench
from paper_2506_23431_b200 import workload as W
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
wl = W.CONFIGS["tiny"].scaled(batch=3)
mine = bench.rank_workload(wl, rank)
times, counts = bench.reduce_over_ranks([10.0 + rank, 5.0 - rank], [100 + rank], dist, "cpu")
fl = W.make_forced_len(mine)
w0 = W.make_weights(wl)["embed"][:2, :4]
w1 = W.make_weights(bench.rank_workload(wl, 0))["embed"][:2, :4]
gathered = [None] * world
dist.all_gather_object(gathered, (fl.tolist(), float(W.make_encoder_memory(mine)[0, 0, 0])))
dist.barrier()
if rank == 0:
    print(json.dumps({"times": times, "counts": counts, "gathered": gathered, "same_weights": bool((w0 == w1).all())}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_reduce_times_by_max_and_tokens_by_sum(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, PD_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29731", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["times"] == [11.0, 5.0]            # max over ranks of (10, 11) and (5, 4)
    assert res["counts"] == [201]                  # 100 + 101
    (fl0, m0), (fl1, m1) = res["gathered"]
    assert fl0 != fl1 and m0 != m1                 # every rank decodes its own sequences ...
    assert res["same_weights"]                     # ... with the same (replicated) weights
    assert outs[1][0].strip() == ""                # only rank 0 reports


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_rank_workloads_are_a_partition_by_independent_seeds():
    import bench
    from paper_2506_23431_b200 import workload as W
    wl = W.CONFIGS["keyphrase"]
    a, b = bench.rank_workload(wl, 0), bench.rank_workload(wl, 3)
    assert a == wl and b.seed != wl.seed and b.batch == wl.batch
    assert not np.array_equal(W.make_forced_len(a), W.make_forced_len(b))


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment starts two ranks by itself (gloo here,
    NCCL on the GPU machine); rank 0 alone reports, and it saw both."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo", "--spawn-check"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    res = json.loads(lines[0])
    assert res["n_ranks"] == 2 and res["world_size"] == 2 and res["max_rank"] == 1.0
