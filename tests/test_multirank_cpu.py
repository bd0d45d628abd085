"""The N > 1 host logic of bench.py on CPU: two gloo ranks on 127.0.0.1.  Replicas exchange no
data; what is multi-rank is the choice of each rank's token batch, the max-over-ranks of the
timings, the whole-job throughput, and who prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import json, os, sys
sys.path.insert(0, %(root)r)
import torch
import torch.distributed as dist
import bench
from paper_2605_18643_b200 import inputs
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group(backend="gloo")
wl = inputs.tiny()
x = bench.rank_tokens(wl, rank)
ms, e2e = bench.max_over_ranks([1.0 + rank, 0.5 - 0.1 * rank], dist, torch.device("cpu"))
sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
dist.all_gather(sums, x.double().sum().reshape(1))
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "e2e": e2e, "value": bench.job_tokens_per_s(world, wl.T, ms),
                      "sums": [float(s) for s in sums], "shape": list(x.shape)}))
dist.destroy_process_group()
'''


def _env(rank, world, port):
    e = dict(os.environ)
    e.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
             MASTER_PORT=str(port))
    return e


def test_two_gloo_ranks_reduce_timings_and_use_their_own_batches():
    port = 29500 + os.getpid() % 2000
    procs = [subprocess.Popen([sys.executable, "-c", WORKER % {"root": ROOT}], env=_env(r, 2, port),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert outs[1][0].strip() == ""                      # only rank 0 prints
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ms"] == 2.0 and line["e2e"] == 0.5      # maximum over the ranks of each timing
    assert abs(line["value"] - 2 * 64 / 2.0e-3) < 1e-6   # whole-job tokens/s: both replicas' tokens over the slower time
    assert line["shape"] == [64, 256] and line["sums"][0] != line["sums"][1]   # a different batch per replica


def test_reference_arm_runs_on_rank_zero_only():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
           "--steps", "1", "--warmup", "0", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=_env(1, 2, port), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=_env(0, 2, port), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
