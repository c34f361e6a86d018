#!/usr/bin/env python
"""Throughput of the Natural GaLore optimizer step on synthetic Llama-shaped gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl ours|reference]

One "step" is one optimizer step over every weight matrix of the workload (projection, history
Gram + solve, natural gradient + Adam moments, back-projection + W update).  Prints ONE JSON line.
With --gpus N > 1 (launched under torchrun) every rank steps its own replica of the matrix set
(weak scaling, no data-path collective); the time is the maximum over ranks.  --shard instead splits one
matrix set over the ranks and exchanges the updated weights after every step (strong scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes per launch of the step kernels from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# taken on the 1.1B shapes cut to 2 layers with a full history (profiles/step_kernels_llama-1.1b-2layers_ncu_full.md)
# and expressed per unit of work so that it scales to the full workload: the stream kernel's traffic grows with
# the low-rank elements sum(r' N), the GEMMs' with sum(M N).  Valid for r = 512, s = 16 only; set an entry to None
# when its kernel changes.
NCU_TRAFFIC_PER_UNIT = {"fused_stream_kernel": ("rn", 145.55), "tc_backproject_kernel": ("mn", 8.362),
                        "tc_project2_kernel": ("mn", 2.936)}

METRIC = "optimizer steps/sec over all matrices (device-timed)"
UNIT = "steps/s"


def pool_size(args, wl):
    """Gradient sets kept resident and cycled.  With fewer than s + 1 distinct sets a gradient would sit twice in
    the history ring and the Gram matrix would be singular up to lambda; the optimizer never sees that in training."""
    return args.pool if args.pool > 0 else wl.s + 1


def config_dict(args, wl, n_matrices, sharded):
    """The workload and protocol of a run; both arms (CUDA path and oracle) describe the same one."""
    grad_bytes = sum(M * N * 2 for _, M, N in wl.shapes)
    return {"workload": wl.name, "matrices": n_matrices, "r": wl.r, "s": wl.s, "T": wl.T,
            "projection": args.projection, "history": args.history, "moments": args.moments,
            "gram_fusion": args.gram_fusion, "small_rank_path": args.small_rank_path,
            "sharded": sharded, "history_filled": True, "refresh_in_timed_region": False,
            "l2": f"inputs larger than L2: {pool_size(args, wl)} gradient sets of {grad_bytes / 1e9:.2f} GB cycled"}


def measured_peaks():
    """(HBM copy GB/s, sustained bf16 TFLOP/s, "measured" | "fallback"): the machine's own measured peaks when
    the file with them is present, else the documented earlier measurement.  The step is timed inside a long
    run under the power cap, so the tensor figure is the sustained one."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", 1400.0)), "measured"
    except Exception:
        return 6650.0, 1400.0, "fallback"


def low_rank_dims(wl, i, projection):
    """(r', rows of the projector, elements of one low-rank matrix) of matrix i: the low-rank gradient is
    r' x N under a left projection and M x r' under a right one (short-side rule, M >= N)."""
    _, M, N = wl.shapes[i]
    rp = wl.rank_of(i)
    right = projection == "short_side" and M >= N
    return rp, (N if right else M), rp * (M if right else N)


def byte_model(wl, projection="left", history="fp32", moments="fp32"):
    """Algorithmic bytes per step: every datum moved once (G bf16, W fp32, P bf16, history/m/v fp32).
    With a bf16 history the s - 1 older gradients are 2 bytes each, the current one is written and read in
    fp32, and its bf16 copy is written once.  With bf16 moments m and v are 2 bytes each way instead of 4."""
    tot = stream = 0
    mom = 8 if moments == "bf16" else 16        # m and v, read and written
    for i, (_, M, N) in enumerate(wl.shapes):
        rp, pr, rn = low_rank_dims(wl, i, projection)
        if history == "bf16":
            tot += 10 * M * N + 2 * pr * rp + (2 * wl.s + 8 + mom) * rn
            stream += (2 * wl.s + 4 + mom) * rn  # older slots (bf16) + current (fp32) once, bf16 copy, m and v
        else:
            tot += 10 * M * N + 2 * pr * rp + (4 * wl.s + 4 + mom) * rn
            stream += (4 * wl.s + mom) * rn      # history read once + m, v read and written
    return tot, stream


def flop_model(wl, projection="left"):
    f = 0
    for i, (_, M, N) in enumerate(wl.shapes):
        rp, _, rn = low_rank_dims(wl, i, projection)
        f += 4 * M * N * rp + 4 * wl.s * rn + 12 * rn
    return f


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- oracle arm

class OracleSampler:
    """The fp64 oracle on one matrix of each distinct shape of the workload, with a full history.

    A whole oracle step over the 1.1B shapes takes minutes, so a step is sampled: one oracle step on one
    matrix per distinct shape, scaled by how many matrices have that shape.  Inputs (gradient, projector)
    are made once per shape and kept; every timing starts from a fresh state whose history holds s
    gradients, the steady state of the optimizer."""

    def __init__(self, wl, projection="left", history="fp32", moments="fp32"):
        self.wl, self.projection, self.history, self.moments = wl, projection, history, moments
        self.counts = {}
        for _, M, N in wl.shapes:
            self.counts[(M, N)] = self.counts.get((M, N), 0) + 1
        self.shapes = list(wl.distinct_shapes())          # (index of the first matrix of the shape, M, N)
        self.inputs = {}
        self.seconds = {}                                 # latest time of one oracle step per shape

    def _hyper(self, orc):
        wl = self.wl
        return orc.Hyper(r=wl.r, s=wl.s, T=0, lam=wl.lam, lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps,
                         projection=self.projection, history_bf16=self.history == "bf16",
                         moments_bf16=self.moments == "bf16")

    def time_shape(self, j, seed):
        """One oracle step on matrix shape j (history pre-filled); returns and records its seconds."""
        from oracle import natural_galore as orc
        from paper_2410_16029_b200 import workload as W

        i, M, N = self.shapes[j]
        st = orc.MatrixState(M, N, self._hyper(orc))
        if (M, N) not in self.inputs:
            rng = np.random.default_rng(1234 + j)
            P, _ = np.linalg.qr(rng.standard_normal((N if st.right else M, st.rp)))
            self.inputs[(M, N)] = (P, W.bf16_bits_to_f64(W.gradient_bits(self.wl, i, 1)))
        P, G = self.inputs[(M, N)]
        st.set_subspace(P)
        rng = np.random.default_rng(99 + seed)
        for slot in range(self.wl.s):
            st.slots[slot] = rng.standard_normal(st.m.shape)
        st.count, st.head = self.wl.s, 0
        Wm = np.zeros((M, N))
        t0 = time.perf_counter()
        st.step(Wm, G, auto_refresh=False)
        self.seconds[(M, N)] = time.perf_counter() - t0
        return self.seconds[(M, N)]

    def step_seconds(self):
        """Seconds of one step over every matrix, from the latest time of each shape."""
        return sum(self.seconds[k] * c for k, c in self.counts.items())

    @staticmethod
    def threads():
        try:
            import threadpoolctl
            return max(p["num_threads"] for p in threadpoolctl.threadpool_info())
        except Exception:
            return os.cpu_count()


def oracle_sample(wl, projection="left", history="fp32", moments="fp32"):
    """Time the oracle once on every distinct shape.  Returns (seconds per full step, description, threads)."""
    smp = OracleSampler(wl, projection, history, moments)
    for j in range(len(smp.shapes)):
        smp.time_shape(j, 0)
    desc = (f"one oracle step (full history of {wl.s}) on one matrix of each of the "
            f"{len(smp.counts)} distinct shapes, scaled by the shape counts to the {wl.n_matrices}-matrix step")
    return smp.step_seconds(), desc, smp.threads()


def run_reference(args, wl):
    """The oracle as the reference arm.  The first step times one matrix of every distinct shape; every later
    step times one matrix of one shape (the shapes take turns) and the step's time is put together from the
    latest time of each shape, so that a run of many steps stays within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSampler(wl, args.projection, args.history, args.moments)
    n_shapes = len(smp.shapes)
    times = []
    for k in range(args.warmup + args.steps):
        if k == 0:
            for j in range(n_shapes):
                smp.time_shape(j, k)
        else:
            smp.time_shape(k % n_shapes, k)
        if k >= args.warmup:
            times.append(smp.step_seconds())
    sec = float(np.mean(times))
    val = 1.0 / sec
    desc = (f"per step one oracle step (full history of {wl.s}) on one matrix of one of the {n_shapes} distinct shapes, "
            f"the shapes taking turns (all of them in the first step); the step time is the latest time of each shape "
            f"scaled by the shape counts to the {wl.n_matrices}-matrix step")
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": config_dict(args, wl, wl.n_matrices, False),
           "cpu_baseline": {"value": val, "unit": UNIT, "cores": smp.threads(), "kind": "oracle", "sample": desc},
           "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


# --------------------------------------------------------------------------------------- multi-rank helpers

def rank_workload(wl, rank):
    """Every rank steps its own replica: same shapes and hyper-parameters, its own seed stream."""
    import dataclasses

    return dataclasses.replace(wl, index=wl.index + 100 * rank)


def max_over_ranks(value, device, world):
    """The slowest rank's time: the job is as fast as its slowest replica."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world, steps, ms_total):
    """Whole-job steps/s: all ranks' steps over the slowest rank's time."""
    return world * steps * 1e3 / ms_total


# --------------------------------------------------------------------------------------- CUDA arm

def run_ours(args, wl):
    import torch
    import torch.distributed as dist

    from paper_2410_16029_b200 import workload as W
    from paper_2410_16029_b200.ngalore import NGaLore

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    parts = None
    if args.shard and world > 1:
        # one model over all ranks: each rank keeps the optimizer state of its share of the matrices and steps
        # them; the updated weights of every shard are then broadcast by their owners (inside the timed region)
        import dataclasses

        from paper_2410_16029_b200 import sharding

        full_shapes = [(M, N) for _, M, N in wl.shapes]
        parts = sharding.partition(full_shapes, wl.r, wl.s, world, args.projection)
        wl = dataclasses.replace(wl, shapes=tuple(wl.shapes[i] for i in parts[rank]))
    shapes = [(M, N) for _, M, N in wl.shapes]
    n = len(shapes)
    # The state is created without automatic refreshes: the timed steps are steady-state steps (history ring full,
    # no refresh among them, whatever T is); the refresh is run once before them and timed alone further down.
    opt = NGaLore(shapes, wl.r, wl.s, 0, lam=wl.lam, lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps,
                  wd=wl.wd, seed=1 + rank, projection=args.projection, history_bf16=args.history == "bf16",
                  gram_fusion=args.gram_fusion == "on", moments_bf16=args.moments == "bf16",
                  small_rank_path=args.small_rank_path == "on")
    # seeded synthetic inputs, resident in HBM: a pool of gradient sets cycled through the steps
    wl_rank = rank_workload(wl, rank)
    if parts is not None:
        # weights of the matrices other ranks own, received after each step
        others = {i: torch.empty(full_shapes[i], dtype=torch.float32, device=dev)
                  for k, p in enumerate(parts) if k != rank for i in p}
    pool_sets = pool_size(args, wl)
    pool = [[W.gradient_device(wl_rank, i, k, dev) for i in range(n)] for k in range(pool_sets)]
    Wt = [W.initial_weight_device(wl_rank, i, dev) for i in range(n)]
    Wp = NGaLore.pointer_array(Wt)
    Gp = [NGaLore.pointer_array(g) for g in pool]
    grad_bytes = sum(M * N * 2 for M, N in shapes)
    opt.refresh_subspace(pool[0])

    groups_by_owner, comm = None, None
    if parts is not None:
        Wall = [None] * len(full_shapes)
        for j, i in enumerate(parts[rank]):
            Wall[i] = Wt[j]
        for i, t in others.items():
            Wall[i] = t
        if args.exchange == "overlapped":
            # the weight update in groups, each group on the wire as soon as it is done (sharding.exchange_overlapped)
            opt.set_update_groups(args.update_groups)
            mine_groups = [[parts[rank][j] for j in range(a, b)] for a, b in opt.update_groups()]
            groups_by_owner = [None] * world
            dist.all_gather_object(groups_by_owner, mine_groups)
            comm = torch.cuda.Stream()

    def step(k):
        if groups_by_owner is not None:
            main = torch.cuda.current_stream()
            before = torch.cuda.Event()
            before.record(main)
            comm.wait_event(before)
        opt.step_ptrs(Wp, Gp[k % pool_sets])
        if parts is None:
            return
        if groups_by_owner is None:
            sharding.exchange_updated(Wall, parts)
        else:
            sharding.exchange_overlapped(Wall, groups_by_owner, wait_update=lambda g: opt.stream_wait_update(g, comm),
                                         comm_stream=comm, wire=args.wire)
            torch.cuda.current_stream().wait_stream(comm)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- untimed: fill the history ring (a step with c < s slots held moves fewer bytes than a steady-state one)
    # and show the library every gradient set once, so that no timed step encodes or uploads TMA descriptors
    fill = max(args.warmup, wl.s, pool_sets)
    for k in range(fill):
        step(k)
    barrier()
    assert opt.step_count >= wl.s, "the history ring must be full before the timed region"
    uploads_before = opt.descriptor_uploads

    # ---- launch: one CUDA graph per gradient set (the step's kernel arguments do not change from step to step;
    # only the descriptors of the gradient buffers differ between sets), or plain stream launches
    use_graph = args.launch == "graph" and parts is None
    graphs = None
    if use_graph:
        graphs = []
        for j in range(pool_sets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                opt.step_ptrs(Wp, Gp[j])
            graphs.append(g)
        barrier()

    launches_per_step = [0]

    def timed_step(k):
        if graphs is not None:
            graphs[k % pool_sets].replay()
        else:
            l0 = opt.launch_count
            step(k)
            launches_per_step[0] = opt.launch_count - l0

    if graphs is not None:
        l0 = opt.launch_count
        opt.step_ptrs(Wp, Gp[fill % pool_sets])      # counts the kernels of one step; also one more warm step
        launches_per_step[0] = opt.launch_count - l0
        fill += 1
    for k in range(args.warmup):
        timed_step(fill + k)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    ev[0].record()
    for k in range(args.steps):
        timed_step(fill + args.warmup + k)
        ev[k + 1].record()
    barrier()
    ms_total = ev[0].elapsed_time(ev[-1])
    per_step = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    launches = launches_per_step[0] * args.steps
    clocks = sampler.stop() if rank == 0 else None
    ms_total = max_over_ranks(ms_total, dev, world)
    ms_median = max_over_ranks(float(np.median(per_step)), dev, world)
    ms_step = ms_total / args.steps
    # sharded: the job made args.steps steps of one model; replicas: every rank made args.steps steps of its own
    value = job_throughput(1 if parts is not None else world, args.steps, ms_total)
    assert opt.descriptor_uploads == uploads_before, "a timed step uploaded TMA descriptors"
    done_steps = fill + args.warmup + args.steps

    code, per = opt.poll_status()
    if code != 0:
        raise RuntimeError(f"device status {code}: {per[:8]}...")

    # ---- per-phase kernel times (CUDA events on the launching stream, inside the library)
    opt.set_profiling(True)
    phase = np.zeros(3)
    reps = 10
    for k in range(reps):
        step(done_steps + k)
        phase += np.array([opt.last_phase_ms(p) for p in range(3)])
    phase /= reps
    opt.set_profiling(False)

    # ---- refresh, timed alone
    torch.cuda.synchronize()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    opt.refresh_subspace(pool[0])
    r1.record()
    torch.cuda.synchronize()
    refresh_ms = r0.elapsed_time(r1)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        Wh = [torch.empty((M, N), dtype=torch.float32).pin_memory() for M, N in shapes]
        Gh = [torch.empty((M, N), dtype=torch.bfloat16).pin_memory() for M, N in shapes]
        for i in range(n):
            Wh[i].copy_(Wt[i])
            Gh[i].copy_(pool[0][i])
        opt.step_host(Wh, Gh)          # first call allocates the device staging
        t0 = time.perf_counter()
        e2e_steps = 3
        for _ in range(e2e_steps):
            opt.step_host(Wh, Gh)      # returns after the device-to-host copy of W has finished
        dt = (time.perf_counter() - t0) / e2e_steps
        w_bytes = sum(M * N * 4 for M, N in shapes)
        e2e = {"value": 1.0 / dt, "unit": UNIT, "h2d_bytes_per_step": w_bytes + grad_bytes,
               "d2h_bytes_per_step": w_bytes, "ms_per_step": dt * 1e3, "steps": e2e_steps}
        del Wh, Gh

    # ---- roofline of the dominant kernel and of the whole step
    peak, tensor_peak, peak_kind = measured_peaks()
    tot_bytes, stream_bytes = byte_model(wl, args.projection, args.history, args.moments)
    dims = [low_rank_dims(wl, i, args.projection) for i in range(n)]
    # the library runs the projection with 256-row tiles (tc_project2_kernel) where nearly all of the work has at
    # least 512 output rows and a long K, which of the workloads here are those of rank 512; elsewhere the
    # 128-row tc_gemm_kernel does the same work
    names = ["tc_project2_kernel" if wl.r >= 512 else "tc_gemm_kernel", "fused_stream_kernel", "tc_backproject_kernel"]
    fused_gram = args.gram_fusion == "on" and wl.r >= 512 and args.projection == "left" and args.history == "fp32"
    if fused_gram:
        # phase 0 is then the projection with the Gram row in its epilogue (plus the solves and the plain projection
        # of the matrices that do not take part); the byte split between the phases below is that of the default path
        names[0] = "tc_project_gram_kernel"
    proj_bytes = sum(2 * M * N + 2 * dims[i][1] * dims[i][0] + 4 * dims[i][2] for i, (M, N) in enumerate(shapes))
    back_bytes = sum(8 * M * N + 2 * dims[i][1] * dims[i][0] for i, (M, N) in enumerate(shapes))
    alg = [proj_bytes, stream_bytes, back_bytes]
    if opt.uses_small_rank_path:
        # two bandwidth kernels (every r' <= 8): the first reads the history once for the Gram row, the second owns
        # the moments; there is no separate stream phase
        names = ["sr_project_gram_kernel", "(no stream phase)", "sr_update_kernel"]
        hist_once = sum(4 * wl.s * d[2] for d in dims)
        alg = [proj_bytes + hist_once, 0, back_bytes + sum(16 * d[2] for d in dims)]
    dom = int(np.argmax(phase))
    achieved = alg[dom] / (phase[dom] * 1e-3) / 1e9
    traffic = None
    per_unit = NCU_TRAFFIC_PER_UNIT.get(names[dom])
    if (per_unit is not None and wl.r == 512 and wl.s == 16 and args.projection == "left" and args.history == "fp32"
            and args.moments == "fp32" and not fused_gram):
        units = sum(d[2] for d in dims) if per_unit[0] == "rn" else sum(M * N for M, N in shapes)
        traffic = per_unit[1] * units
    roofline = {"bound": "hbm", "kernel": names[dom], "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_kind": peak_kind,
                "algorithmic_bytes_per_launch": alg[dom], "ms_per_launch": float(phase[dom]),
                "phases_ms": {names[i]: float(phase[i]) for i in range(3)},
                "phases_frac_of_peak": {names[i]: alg[i] / (phase[i] * 1e-3) / 1e9 / peak for i in range(3)
                                        if phase[i] > 1e-6}}
    flops = flop_model(wl, args.projection)
    step_roofline_ms = max(tot_bytes / (peak * 1e9), flops / (tensor_peak * 1e12)) * 1e3
    step_roof = {"bytes_per_step": tot_bytes, "flops_per_step": flops, "roofline_ms": step_roofline_ms,
                 "frac": step_roofline_ms / ms_step, "hbm_peak_gbs": peak, "tensor_peak_tflops": tensor_peak,
                 "peak_kind": peak_kind}

    # ---- the oracle on the host cores, bounded sample
    cpu = None
    if not args.no_cpu:
        sec, desc, threads = oracle_sample(wl, projection=args.projection, history=args.history, moments=args.moments)
        cpu = {"value": 1.0 / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
           "scaling": "strong" if parts is not None else "weak",
           "vs_baseline": None, "dtype": "bf16",
           "dtype_detail": "bf16 (projection) and fp16 (back-projection) GEMM operands, f32 state and accumulation, "
                           "f64 Gram reduction and solve",
           "data": "synthetic",
           "config": config_dict(args, wl, n, parts is not None),
           "launch": "cuda_graph" if use_graph else "stream", "ms_per_step_median": ms_median,
           "exchange": None if parts is None else {"mode": args.exchange, "wire": args.wire,
                                                   "update_groups": args.update_groups},
           "untimed_steps_before": fill + args.warmup, "state_bytes": opt.device_bytes,
           "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
           "step_roofline": step_roof,
           "refresh": {"ms": refresh_ms, "T": wl.T, "amortised_ms_per_step": ms_step + refresh_ms / max(wl.T, 1),
                       "amortised_steps_per_s": (1 if parts is not None else world) * 1e3 / (ms_step + refresh_ms / max(wl.T, 1))},
           "cpu_baseline": cpu}
    print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--pool", type=int, default=0,
                    help="gradient sets resident in HBM, cycled (default s + 1: no gradient repeats inside the history)")
    ap.add_argument("--layers", type=int, default=0,
                    help="keep only the first LAYERS transformer layers of the workload (small case for profiling)")
    ap.add_argument("--projection", default="left", choices=["left", "short_side"],
                    help="left: R = P^T G for every matrix (the paper's form, the headline configuration); "
                         "short_side: matrices with rows >= cols are projected on the right")
    ap.add_argument("--history", default="fp32", choices=["fp32", "bf16"],
                    help="fp32: the ring of low-rank gradients in fp32 (the headline configuration); bf16: every "
                         "stored gradient but the current one in bf16 (reduced-precision state option)")
    ap.add_argument("--moments", default="fp32", choices=["fp32", "bf16"],
                    help="fp32: the Adam moments in fp32 (the headline configuration); bf16: m rounded to nearest and v "
                         "rounded stochastically to bf16 (reduced-precision state option)")
    ap.add_argument("--gram-fusion", default="off", choices=["on", "off"],
                    help="off (the library's default): the Gram tiles run in the stream kernel; on: where the workload "
                         "allows it the new Gram row is formed in the projection's epilogue")
    ap.add_argument("--small-rank-path", default="off", choices=["on", "off"],
                    help="on: where every matrix has r' <= 8 the step runs as two kernels without tensor cores (an "
                         "option of the library, slower than the default as built)")
    ap.add_argument("--shard", action="store_true",
                    help="with --gpus N > 1: one model's matrices split over the ranks (state memory / N, weights "
                         "exchanged after every step) instead of N independent replicas; rank 0's phases and "
                         "roofline then describe its own shard")
    ap.add_argument("--launch", default="graph", choices=["graph", "stream"],
                    help="graph (default): every timed step is one replay of a CUDA graph captured from ngalore_step, one "
                         "graph per gradient set; stream: plain calls of ngalore_step")
    ap.add_argument("--exchange", default="overlapped", choices=["overlapped", "after"],
                    help="with --shard: overlapped (default): the weights are updated in groups and every group is "
                         "broadcast by its owner while the next one is being updated; after: one broadcast per owner "
                         "after the step")
    ap.add_argument("--update-groups", type=int, default=4, help="with --shard --exchange overlapped: groups per rank")
    ap.add_argument("--wire", default="fp32", choices=["fp32", "bf16"],
                    help="with --shard --exchange overlapped: format of the weights on the wire")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2410_16029_b200 import workload as W

    wl = W.WORKLOADS[args.workload]
    if args.layers > 0:
        wl = W.truncated(wl, args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        import __graft_entry__ as entry

        entry.build()
        run_ours(args, wl)


if __name__ == "__main__":
    main()
