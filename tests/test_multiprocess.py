"""The N > 1 path of the benchmark on CPU: two gloo ranks.  Ranks are independent replicas (no data-path
collective); the only exchange is the max-over-ranks of the timed region, and only rank 0 reports."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    from paper_2410_16029_b200 import workload as wl

    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), world)
    w = bench.rank_workload(wl.tiny_workload([(16, 24)], r=4, s=2, T=3), rank)
    bits = wl.gradient_bits(w, 0, 0)
    gathered = [None] * world
    dist.all_gather_object(gathered, (ms, w.shapes, int(bits.astype(np.int64).sum())))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_only_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29741, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (ms0, shapes0, sum0), (ms1, shapes1, sum1) = got
    assert ms0 == ms1 == 15.0                 # every rank sees the slowest rank's time
    assert shapes0 == shapes1                 # same matrix set per replica
    assert sum0 != sum1                       # but its own gradient stream
    sys.path.insert(0, ROOT)
    import bench
    assert bench.job_throughput(2, 10, 20.0) == 1000.0   # 2 ranks x 10 steps in 20 ms


def test_reference_arm_under_two_ranks_prints_one_line():
    """`bench.py --impl reference` launched as two ranks: rank 0 times the oracle, rank 1 exits quietly."""
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29743", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "0", "--steps", "1", "--warmup", "0"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
