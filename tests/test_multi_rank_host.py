"""Host logic of the multi-GPU benchmark path on CPU: two `gloo` ranks. The verify pass does not
exchange data between GPUs (sequences are independent; replicas only), so what N > 1 adds is the
per-rank batch (seed offset), the maximum of the timings over the ranks, the whole-job throughput,
and the rule that only rank 0 of `--impl reference` works and prints."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
from paper_2601_23180_b200 import inputs as gen
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3)
rcfg = bench.rank_config(cfg, rank)
tree = gen.make_tree(rcfg, 0).tolist()
times = bench.max_over_ranks([10.0 + 5.0 * rank, 7.0 - rank], world)     # rank-dependent timings
dist.barrier()
print(json.dumps({{"rank": rank, "seed": rcfg.seed, "tree": tree, "times": times,
                  "value": bench.aggregate_throughput(cfg, world, times[0])}}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_take_the_max_time_and_their_own_batches(tmp_path):
    port = 29000 + os.getpid() % 2000
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT, port=port))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    # every rank sees the maximum over ranks of each timing
    assert outs[0]["times"] == outs[1]["times"] == [15.0, 7.0]
    # different seeds, hence different draft trees, same shape
    assert outs[0]["seed"] + 1 == outs[1]["seed"] and outs[0]["tree"] != outs[1]["tree"]
    assert len(outs[0]["tree"]) == len(outs[1]["tree"])
    # whole-job throughput = 2 ranks x 3 sequences x 60 draft tokens per 15 ms
    assert abs(outs[0]["value"] - 2 * 3 * 60 / 15e-3) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny_chain", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"], env["LOCAL_RANK"] = "0", "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny_chain", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"].startswith("oracle") and line["extrapolated"] is True
    assert line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0
