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


# ----------------------------------------------------------------------------- sharding one model over ranks

def test_partition_covers_every_matrix_once_and_balances():
    sys.path.insert(0, ROOT)
    from paper_2410_16029_b200 import sharding
    from paper_2410_16029_b200 import workload as wl

    w = wl.WORKLOADS[4]
    shapes = [(M, N) for _, M, N in w.shapes]
    for world in (1, 2, 3, 8):
        parts = sharding.partition(shapes, w.r, w.s, world)
        flat = sorted(i for p in parts for i in p)
        assert flat == list(range(len(shapes)))
        loads = [sum(sharding.matrix_cost(*shapes[i], w.r, w.s) for i in p) for p in parts]
        assert max(loads) <= 1.05 * sum(loads) / world          # longest-processing-time keeps ranks within 5 %
        assert sharding.owners(parts, len(shapes)) == [next(k for k, p in enumerate(parts) if i in p)
                                                       for i in range(len(shapes))]
    # the byte model is the benchmark's
    import bench
    assert sum(sharding.matrix_cost(M, N, w.r, w.s) for M, N in shapes) == bench.byte_model(w)[0]
    assert sum(sharding.matrix_cost(M, N, w.r, w.s, "short_side") for M, N in shapes) == bench.byte_model(w, "short_side")[0]


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2410_16029_b200 import sharding

    dist.init_process_group("gloo", rank=rank, world_size=world)
    shapes = [(8, 16), (24, 8), (16, 16), (8, 8), (32, 8)]
    parts = sharding.partition(shapes, 4, 2, world)
    # every rank starts from the same weights; each "steps" only its own matrices (a stand-in for the CUDA
    # optimizer: add rank + 1), then the owners' results are exchanged
    W = [torch.full(s, float(i)) for i, s in enumerate(shapes)]
    for i in parts[rank]:
        W[i] += rank + 1
    sharding.exchange_updated(W, parts)
    own = sharding.owners(parts, len(shapes))
    ok = all(torch.equal(W[i], torch.full(shapes[i], float(i + own[i] + 1))) for i in range(len(shapes)))
    gathered = [None] * world
    dist.all_gather_object(gathered, (ok, parts))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_exchange_their_shards():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, 29747, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (ok0, parts0), (ok1, parts1) = got
    assert ok0 and ok1
    assert parts0 == parts1 and sorted(parts0[0] + parts0[1]) == [0, 1, 2, 3, 4]


def _overlap_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2410_16029_b200 import sharding

    dist.init_process_group("gloo", rank=rank, world_size=world)
    shapes = [(8, 16), (24, 8), (16, 16), (8, 8), (32, 8), (8, 24)]
    parts = sharding.partition(shapes, 4, 2, world)
    # each rank's matrices in two update groups, as the library would report them (contiguous in its own order)
    groups = [[p[: (len(p) + 1) // 2], p[(len(p) + 1) // 2:]] for p in parts]
    results = {}
    for wire in ("fp32", "bf16"):
        W = [torch.full(s, float(i)) + 0.001 * torch.arange(s[0] * s[1], dtype=torch.float32).reshape(s)
             for i, s in enumerate(shapes)]
        for i in parts[rank]:
            W[i] += rank + 1                                   # the stand-in for this rank's optimizer step
        expect = []
        own = sharding.owners(parts, len(shapes))
        for i, s in enumerate(shapes):
            e = torch.full(s, float(i)) + 0.001 * torch.arange(s[0] * s[1], dtype=torch.float32).reshape(s) + own[i] + 1
            if wire == "bf16" and own[i] != rank:
                e = e.to(torch.bfloat16).to(torch.float32)     # the other ranks see the owner's weights rounded
            expect.append(e)
        log, waited = [], []
        sharding.exchange_overlapped(W, groups, wait_update=lambda g: waited.append(g), wire=wire, log=log)
        ok = all(torch.equal(a, b) for a, b in zip(W, expect))
        results[wire] = (ok, log, waited)
    gathered = [None] * world
    dist.all_gather_object(gathered, (results, groups))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_overlapped_exchange_order_and_wire_formats():
    """Two gloo ranks: the group-by-group exchange delivers every owner's weights (bit-exact in fp32, the owner's
    bf16 rounding on the bf16 wire), every rank issues the collectives in the same order, and an owner waits for the
    update event of a group before it packs that group, never for a later one."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_overlap_worker, args=(r, 2, 29751, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (res0, groups0), (res1, groups1) = got
    assert groups0 == groups1
    for wire in ("fp32", "bf16"):
        ok0, log0, waited0 = res0[wire]
        ok1, log1, waited1 = res1[wire]
        assert ok0 and ok1
        bcast0 = [e for e in log0 if e[0] == "bcast"]
        bcast1 = [e for e in log1 if e[0] == "bcast"]
        assert bcast0 == bcast1                                # same collectives, same order, on both ranks
        assert bcast0 == [("bcast", src, g) for src in range(2) for g in range(2) if groups0[src][g]]
        for rank, log, waited in ((0, log0, waited0), (1, log1, waited1)):
            mine = [g for g in range(2) if groups0[rank][g]]
            assert waited == mine                              # one wait per own group, in update order
            for g in mine:                                     # wait -> pack -> broadcast for every own group
                i = log.index(("wait", rank, g))
                assert log[i + 1] == ("pack", rank, g) and log[i + 2] == ("bcast", rank, g)
            assert all(e[1] != rank for e in log if e[0] == "unpack")
