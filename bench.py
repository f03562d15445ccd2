#!/usr/bin/env python
"""Benchmark of the gossip-BMUF synchronisation round.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload wikitext103] [--impl gbmuf]

One "step" is one synchronisation round (neighbour draws + the fused gather / average /
block-momentum pass) over all K replicas of the workload, preceded by one synthetic local step
that is launched outside the timed interval (its time is reported separately).  Prints ONE JSON
line.  `--impl reference` times the CPU oracle instead, on a bounded column sample.

Metric: replica-parameters per second per round (K * N / t_round), with the achieved
algorithmic HBM traffic (24 B per replica-parameter for fp32 replicas, 20 B for bf16) against
the measured copy bandwidth of the GPU.

Several GPUs: one process per GPU.  Under a launcher (`python -m torch.distributed.run ...
bench.py --gpus N`) the ranks are taken from the environment; `python bench.py --gpus N` on its
own starts the N rank processes itself.  Either way rank r holds the columns [r*N, (r+1)*N) of
a model N times as wide (weak scaling, no data exchanged: given the counter-based neighbour
draws every column is independent); the process group only serves the barrier around the timed
region, the max-over-ranks time and the gathering of what each rank ran.
`--workload NAME:form=peer` (several ranks only) times the other multi-GPU form: one worker per
rank, each pulling its drawn neighbours' slices from the other ranks' memory.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "replica_params_per_sec_per_gossip_bmuf_round"
UNIT = "replica-params/s"
FALLBACK_HBM_GBS = 6650.0
NVLINK_GBS_PER_DIRECTION = 770.0     # measured peer copy on this machine, per direction and GPU

# DRAM traffic of the fused kernel per replica-parameter from an ncu capture (dram__bytes_read.sum
# + dram__bytes_write.sum divided by the replica-parameters of the captured launch), valid only
# for the kernel source it was taken from (source_sha() below) and for the launch variant and
# theta dtype it was taken with: key = (variant, dtype); 0 fp32 from workload profile16, 1 bf16
# from profile16bf (all K rows in tensor memory); the ring-window figure is from profile64 and
# holds for that ring only (K = 64, p = 5: p / K extra theta row reads).
NCU_TRAFFIC = {"source_sha": "eef893168e51",
               "bytes_per_replica_param": {("tmem", 0): (3.221349e9 + 3.161665e9) / 268435536,
                                           ("tmem", 1): (2.684770e9 + 2.625498e9) / 268435536,
                                           ("tmem-window", 0): (3.311525e9 + 3.161882e9) / 268435776},
               "window_ring": (64, 5)}


def algorithmic_bytes_per_replica_param(dtype: int, mode: int = 0) -> int:
    """theta read once + omega, Delta read + omega, Delta, theta written."""
    th = 4 if dtype == 0 else 2
    return 2 * th if mode == 1 else th + 8 + 8 + th


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def host_info() -> dict:
    """CPU model and core count of the box the oracle is timed on."""
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"cpu_model": model, "nproc": os.cpu_count()}


class ClockSampler:
    """Samples SM and memory clocks, power and throttle reasons with nvidia-smi (a read-only
    query) while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap,clocks.mem")

    def __init__(self, index: int, period_ms: int = 100):
        self.index, self.rows, self.proc, self.period_ms = index, [], None, period_ms

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def window(self, t0: float, t1: float, detail: bool = False) -> dict:
        """Summary of the samples taken in [t0, t1] (wall clock)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        mhz, mem, power, mx, reasons = [], [], [], None, set()
        for ts, line in list(self.rows):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8 or not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            try:
                mhz.append(float(f[0]))
                mx = float(f[1])
                power.append(float(f[2]))
                mem.append(float(f[7]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        out = {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
               "samples": len(mhz), "reasons": sorted(reasons)}
        if detail:
            out["mem_mhz"] = statistics.median(mem) if mem else None
            out["power_w_median"] = statistics.median(power) if power else None
            out["power_w_max"] = max(power) if power else None
            bins = {}
            for v in mhz:                                     # samples binned by SM clock (100 MHz)
                key = f"{int(v // 100) * 100}-{int(v // 100) * 100 + 99}"
                bins[key] = bins.get(key, 0) + 1
            out["samples_by_sm_mhz"] = dict(sorted(bins.items()))
        return out

    def stop(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()


def source_sha() -> str:
    """Fingerprint of the fused kernels' code: the files that hold the barrier / bulk-copy
    primitives and theta traits, the shared-memory-tile kernel (with the averaging division and
    the filter) and the tensor-memory-tile kernel, with comments and white space left out (so that
    rewording a comment does not invalidate the counters taken from the same code)."""
    h = hashlib.sha256()
    for name in ("primitives.cuh", "sync_fused.cuh", "sync_fused_tmem.cuh"):
        with open(os.path.join(ROOT, "paper_1909_09010_b200", "csrc", name), "r") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update("".join(text.split()).encode())
    return h.hexdigest()[:12]


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample(w, cols: int):
    """Oracle state over the first `cols` columns of the workload (a column range is exact)."""
    import oracle
    from paper_1909_09010_b200 import workloads
    cols = min(cols, w.N)
    sh = workloads.shard_columns(w.offsets, 0, cols)
    theta0 = workloads.theta0_numpy(w, cols)
    if w.dtype == 1:
        theta0 = oracle.f32_to_bf16(theta0)
    st = oracle.init(theta0, w.K, dtype=w.dtype)
    oracle.local_perturb(st, w.seed, 0, w.lr or 0.1, w.sigma or 1e-3, 1, elem_base=0)
    return sh, st


def time_oracle_rounds(w, cols: int, rounds: int, first_round: int = 1):
    """Seconds per oracle round (single thread) on the column sample."""
    import oracle
    sh, st = oracle_sample(w, cols)
    times = []
    for r in range(first_round, first_round + rounds):
        oracle.local_perturb(st, w.seed, r, w.lr or 0.1, w.sigma or 1e-3, 1, elem_base=0)
        t0 = time.perf_counter()
        nbr = oracle.sample_neighbors(w.seed, r, w.K, sh.m, w.p, w.q, comp_base=sh.comp_base)
        oracle.sync_round(st, sh.offsets, nbr, w.eta, w.zeta, mode=w.mode)
        times.append(time.perf_counter() - t0)
    return times, w.K * sh.n


def cpu_baseline_entry(args, w) -> dict:
    times, units_cpu = time_oracle_rounds(w, args.ref_cols, args.ref_rounds)
    t = sum(times) / len(times)
    return {"value": units_cpu / t, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"columns [0,{min(args.ref_cols, w.N)}) of {w.name}, K={w.K}, {args.ref_rounds} rounds, "
                      f"{t:.2f} s per round", "host": host_info()}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = args.ref_cols
    times, units = time_oracle_rounds(w, cols, args.warmup + args.steps)
    times = times[args.warmup:]
    t = sum(times) / len(times)
    val = units / t
    sample = f"columns [0,{min(cols, w.N)}) of {w.name}, all K={w.K} replicas, one round per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.dtype == 0 else "bf16-stored/f32", "data": "synthetic",
            "config": {"workload": w.name, "K": w.K, "N": w.N, "components": w.m, "p": w.p,
                       "q": w.q, "eta": w.eta, "zeta": w.zeta, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample, "host": host_info()},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# Ranks: one process per GPU
# ------------------------------------------------------------------------------------------------
class RankCtx:
    """What a leg needs to know about its place among the ranks, and the three things the
    process group is used for: a barrier, the max of a host number over ranks, and gathering
    one small object per rank."""

    def __init__(self, rank: int, world: int, local: int, backend: str | None, device_index: int):
        self.rank, self.world, self.local, self.backend = rank, world, local, backend
        self.device_index = device_index

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, x: float) -> float:
        if self.world == 1:
            return float(x)
        import torch
        import torch.distributed as dist
        dev = f"cuda:{self.device_index}" if self.backend == "nccl" else "cpu"
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def gather(self, obj) -> list:
        if self.world == 1:
            return [obj]
        import torch.distributed as dist
        out = [None] * self.world
        dist.all_gather_object(out, obj)
        return out


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_process(local_rank: int, world: int, port: int, argdict: dict, leg, backend):
    """Entry of a rank process started by launch_ranks."""
    os.environ.update(RANK=str(local_rank), LOCAL_RANK=str(local_rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    args = argparse.Namespace(**argdict)
    run_ranked(args, resolve_workload(args), leg=leg, backend=backend)


def launch_ranks(args, leg=None, backend=None):
    """`--gpus N` without a launcher: start the N rank processes of this node (rank r on cuda:r)
    and wait for them.  Rank 0 prints the line.  `leg` / `backend` let a check run the same
    framing around another leg or over gloo."""
    import torch.multiprocessing as mp
    n = args.gpus
    if leg is None and args.share_device is None:
        import torch
        have = torch.cuda.device_count()
        if have < n:
            raise SystemExit(f"bench.py --gpus {n}: this node has {have} CUDA device(s); "
                             f"refusing to run {n} ranks on fewer GPUs (that would not be a {n}-GPU number)")
    mp.spawn(_rank_process, args=(n, free_port(), vars(args), leg, backend), nprocs=n, join=True)


def run_ranked(args, w, leg=None, backend=None):
    """One rank: set up the process group, run the leg, let rank 0 assemble and print the line."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if leg is None:
        leg = peer_leg if args.form == "peer" else gpu_leg
    if backend is None:
        backend = "gloo" if args.share_device is not None else "nccl"
    device_index = args.share_device if args.share_device is not None else local
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            import torch
            # the communicator log (rank count, transport) goes to stderr; stdout stays one line
            os.environ.setdefault("NCCL_DEBUG", "INFO")
            os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
            os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{device_index}"))
        else:
            dist.init_process_group(backend, rank=rank, world_size=world)
    ctx = RankCtx(rank, world, local, backend if world > 1 else None, device_index)
    try:
        res = leg(args, w, ctx)
        ranks = ctx.gather(res["rank_info"])
        ctx.barrier()
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
    if rank != 0:
        return
    units = res["units_per_rank"] * world * args.steps
    total_s = res["total_sync_s"]                       # max over ranks
    config = dict(res["config"])
    config["ranks"] = ranks
    if args.share_device is not None and world > 1:
        config["note"] = "all ranks share one device: a check of the multi-rank path, not a measurement"
    line = {"metric": METRIC, "value": units / total_s, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_s / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if w.dtype == 0 else "bf16-stored/f32", "data": "synthetic",
            "config": config, "roofline": res.get("roofline"), "clocks": res.get("clocks"),
            "gpu_launches": res.get("gpu_launches", 0), "e2e": res.get("e2e")}
    if res.get("regimes") is not None:
        line["regimes"] = res["regimes"]
    if not args.no_cpu_baseline:
        # the other ranks have left and released their GPUs by now
        line["cpu_baseline"] = cpu_baseline_entry(args, w)
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU leg: K replicas resident in this rank's GPU (the element-range shard of rank r)
# ------------------------------------------------------------------------------------------------
def parallelism_text(form: str, world: int) -> str:
    if form == "peer":
        return (f"one worker per rank x{world}, neighbour slices pulled from peer memory inside the round "
                "kernel, one barrier per round")
    return f"element-range shards x{world}, no collective"


def rank_shard(w, rank: int) -> dict:
    """Rank r's place in the model `world` times as wide: its components keep their global
    index and its columns their global position, so the ranks reproduce the wide model's draws
    and noise."""
    return {"comp_base": rank * w.m, "elem_base": rank * w.N}


def _regime_entry(ms_per_round, bytes_per_round, peak, clocks):
    gbs = bytes_per_round / (ms_per_round / 1e3) / 1e9
    out = {"ms_per_round": ms_per_round, "gbs": gbs, "frac_of_measured": gbs / peak,
           "frac_of_nominal_8TBs": gbs / 8000.0, "clocks": clocks}
    if clocks.get("sm_mhz"):
        out["ms_x_sm_ghz"] = ms_per_round * clocks["sm_mhz"] / 1e3
    return out


def gpu_leg(args, w, ctx: RankCtx) -> dict:
    import torch
    from paper_1909_09010_b200 import binding, build, workloads

    build.build()
    torch.cuda.set_device(ctx.device_index)
    dev = torch.device(f"cuda:{ctx.device_index}")
    rank, world = ctx.rank, ctx.world
    shard = rank_shard(w, rank)

    K, N, ld = w.K, w.N, w.ld
    tdt = torch.float32 if w.dtype == 0 else torch.bfloat16
    theta = torch.empty((K, ld), dtype=tdt, device=dev)
    omega = torch.empty((K, ld), dtype=torch.float32, device=dev)
    delta = torch.empty((K, ld), dtype=torch.float32, device=dev)
    g = binding.Gbmuf(theta, omega, delta, K=K, N=N, ld=ld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta,
                      seed=w.seed, theta_dtype=w.dtype, device=ctx.device_index, mode=w.mode, **shard)
    if args.tuning:
        t = [int(x) for x in args.tuning.split(",")]
        g.set_tuning(*t)
    g.set_partition(w.offsets)
    theta0 = workloads.theta0_torch(w, dev).to(tdt)
    g.init(theta0)
    del theta0
    lr, sigma = w.lr or 0.1, w.sigma or 1e-3
    g.local_perturb(0, lr, sigma, 1)
    grad = accum = clip_mask = None

    def adagrad_buffers():
        # the experiments' optimiser on a fixed synthetic gradient (std 1e-2); the recurrent
        # components (here: those of 1 Mi to 8 Mi elements) form the clipped group
        nonlocal grad, accum, clip_mask
        if grad is None:
            grad = torch.empty((K, ld), dtype=torch.float32, device=dev).normal_(0.0, 1e-2)
            accum = torch.full((K, ld), 0.1, dtype=torch.float32, device=dev)
            sizes = [w.offsets[i + 1] - w.offsets[i] for i in range(w.m)]
            clip_mask = [1 if (1 << 20) <= n <= (1 << 23) else 0 for n in sizes]

    def adagrad_step(step):
        g.local_adagrad(grad, accum, lr, eps=1e-8, clip_norm=10.0, clip_mask=clip_mask)

    def perturb_step(step):
        g.local_perturb(step, lr, sigma, 1)

    if args.local_step == "adagrad":
        adagrad_buffers()
        local_step = adagrad_step
    else:
        local_step = perturb_step
    torch.cuda.synchronize()
    info = g.launch_info()

    def barrier():
        ctx.barrier()
        torch.cuda.synchronize()

    # ---- the timed rounds: events around each round, the local step between them untimed
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    rnd = 1
    for _ in range(args.warmup):
        local_step(rnd)
        g.sync_round(rnd)
        rnd += 1
    barrier()
    sampler = ClockSampler(ctx.device_index).start() if rank == 0 else None
    t_wall0 = time.time()
    for i in range(args.steps):
        a, b, c = ev[i]
        a.record()
        local_step(rnd)                         # the local step: outside the timed interval
        b.record()
        g.sync_round(rnd)                       # set-up kernel + fused kernel
        c.record()
        rnd += 1
    barrier()
    t_wall1 = time.time()
    clocks = sampler.window(t_wall0, t_wall1) if rank == 0 else None
    status = g.device_status()
    sync_ms = [b.elapsed_time(c) for a, b, c in ev]
    pert_ms = [a.elapsed_time(b) for a, b, c in ev]
    total_sync_s = ctx.max_over_ranks(sum(sync_ms) / 1e3)

    if args.save_state:
        # each rank's result after the timed rounds (a check reassembles the wide model from these)
        os.makedirs(args.save_state, exist_ok=True)
        torch.save({"rank": rank, "world": world, "rounds": rnd - 1, **shard,
                    "theta": theta[:, :N].cpu(), "omega": omega[:, :N].cpu(), "delta": delta[:, :N].cpu()},
                   os.path.join(args.save_state, f"rank{rank}.pt"))

    peak, peak_kind = measured_peak()
    bpe = algorithmic_bytes_per_replica_param(w.dtype, w.mode)
    round_bytes = bpe * K * N

    # ---- the same rounds back to back, replayed from one CUDA graph (set-up + fused kernel per
    # round, no local step in between): what a launch-bound small model gains from a graph
    graph_ms = None
    if not args.no_graph:
        gs = torch.cuda.Stream(device=dev)
        gs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(gs):
            g.sync_round(rnd, stream=gs)
            rnd += 1
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gs):
                for i in range(args.steps):
                    g.sync_round(rnd + i, stream=gs)
            rnd += args.steps
            ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph.replay()                      # warm-up replay
            ga.record(gs)
            graph.replay()
            gb.record(gs)
        gs.synchronize()
        torch.cuda.current_stream().wait_stream(gs)
        graph_ms = ga.elapsed_time(gb) / args.steps
        status = status or g.device_status()

    # ---- regimes: how the round behaves over seconds, under the three kinds of neighbour it
    # can have on the GPU -- an ALU-bound local step, nothing (rounds back to back), a
    # bandwidth-bound local step -- with SM / memory clocks and power sampled across each, and a
    # plain device copy sustained the same way as the yardstick.  Rank 0 only.
    regimes = None
    if rank == 0 and not args.no_regimes and args.regime_rounds > 0:
        R = args.regime_rounds
        regimes = {"rounds_each": R, "round_bytes": round_bytes}

        def timed_rounds(step_fn):
            nonlocal rnd
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(R)]
            torch.cuda.synchronize()
            t0 = time.time()
            for a, b in evs:
                if step_fn is not None:
                    step_fn(rnd)
                a.record()
                g.sync_round(rnd)
                b.record()
                rnd += 1
            torch.cuda.synchronize()
            t1 = time.time()
            ms = [a.elapsed_time(b) for a, b in evs]
            return sum(ms) / len(ms), sampler.window(t0, t1, detail=True)

        ms, ck = timed_rounds(perturb_step)
        regimes["separated_by_alu_bound_local_step"] = _regime_entry(ms, round_bytes, peak, ck)
        # back to back: a graph of 50 rounds replayed until R rounds have run
        per_graph = min(50, R)
        gs = torch.cuda.Stream(device=dev)
        gs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(gs):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gs):
                for i in range(per_graph):
                    g.sync_round(rnd + i, stream=gs)
            rnd += per_graph
            graph.replay()
            gs.synchronize()
            ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(1, R // per_graph)
            t0 = time.time()
            ga.record(gs)
            for _ in range(reps):
                graph.replay()
            gb.record(gs)
            gs.synchronize()
            t1 = time.time()
        torch.cuda.current_stream().wait_stream(gs)
        regimes["back_to_back_in_cuda_graph"] = _regime_entry(
            ga.elapsed_time(gb) / (reps * per_graph), round_bytes, peak, sampler.window(t0, t1, detail=True))
        del graph
        free_b = torch.cuda.mem_get_info(dev)[0]
        if grad is not None or free_b > 2 * K * ld * 4 + (4 << 30):
            adagrad_buffers()
            ms, ck = timed_rounds(adagrad_step)
            regimes["separated_by_hbm_bound_local_step"] = _regime_entry(ms, round_bytes, peak, ck)
            # the yardstick sustained the same way: a plain device copy of one [K][ld] fp32 array
            n_copy = 3 * R
            ca, cb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(3):
                accum.copy_(grad)
            torch.cuda.synchronize()
            t0 = time.time()
            ca.record()
            for _ in range(n_copy):
                accum.copy_(grad)
            cb.record()
            torch.cuda.synchronize()
            t1 = time.time()
            copy_bytes = 2 * grad.numel() * 4
            regimes["device_copy_back_to_back"] = _regime_entry(
                ca.elapsed_time(cb) / n_copy, copy_bytes, peak, sampler.window(t0, t1, detail=True))
            regimes["device_copy_back_to_back"]["copies"] = n_copy
        status = status or g.device_status()
        if args.local_step != "adagrad":
            grad = accum = None
            torch.cuda.empty_cache()
    if sampler is not None:
        sampler.stop()

    # ---- a plain device copy of the same size class on this very GPU, as context for the
    # roofline fraction (boxes of one pool differ by a percent or two); the state is no longer
    # needed as a training state after this point
    torch.cuda.synchronize()
    ca, cb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    copy_ms = []
    for _ in range(4):
        ca.record()
        delta.copy_(omega)
        cb.record()
        torch.cuda.synchronize()
        copy_ms.append(ca.elapsed_time(cb))
    copy_gbs_live = 2 * omega.numel() * 4 / (min(copy_ms[1:]) / 1e3) / 1e9

    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(args, w, ctx, dev, theta, omega, delta, rnd, shard)

    # per-launch figures of the fused kernel on this rank (the set-up kernel that shares the
    # event bracket runs for microseconds)
    t_launch = (sum(sync_ms) / len(sync_ms)) / 1e3
    achieved = round_bytes / t_launch / 1e9
    traffic = None
    per_param = NCU_TRAFFIC["bytes_per_replica_param"].get((info.get("variant"), w.dtype))
    if info.get("variant") == "tmem-window" and (K, w.p) != NCU_TRAFFIC["window_ring"]:
        per_param = None
    if per_param is not None and not args.tuning and w.mode == 0 and NCU_TRAFFIC["source_sha"] == source_sha():
        traffic = per_param * K * N
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "algorithmic_bytes_per_replica_param": bpe, "traffic": traffic,
                "device_copy_gbs_on_this_gpu": copy_gbs_live,
                "kernel": "sync_fused_tmem_kernel" if str(info.get("variant")).startswith("tmem") else "sync_fused_kernel"}
    if graph_ms:
        gbs = round_bytes / (graph_ms / 1e3) / 1e9
        roofline["back_to_back"] = {"ms_per_round": graph_ms, "achieved": gbs, "frac": gbs / peak,
                                    "frac_of_nominal_8TBs": gbs / 8000.0,
                                    "what": f"{args.steps} rounds replayed from one CUDA graph, no local step between them"}
    config = {"workload": w.name, "K": K, "N": N, "components": w.m, "p": w.p, "q": w.q,
              "eta": w.eta, "zeta": w.zeta, "mode": "gossip-MA" if w.mode else "gossip-BMUF",
              "replica_params_per_gpu": K * N,
              "parallelism": parallelism_text("resident", world),
              "l2": "inputs_larger_than_l2 (state %.1f GB per GPU)" %
                    ((K * ld * (8 + (4 if w.dtype == 0 else 2))) / 1e9),
              "launch": info, "local_step": args.local_step,
              "local_step_ms": sum(pert_ms) / len(pert_ms),
              "round_plus_local_step_ms": (sum(pert_ms) + sum(sync_ms)) / len(sync_ms),
              "sync_ms_min": min(sync_ms), "sync_ms_max": max(sync_ms),
              "sync_ms_in_cuda_graph": graph_ms, "device_status": status}
    g.destroy()
    return {"units_per_rank": K * N, "total_sync_s": total_sync_s, "config": config,
            "roofline": roofline, "clocks": clocks, "regimes": regimes,
            "gpu_launches": (3 if args.local_step == "perturb" else 5) * args.steps, "e2e": e2e,
            "rank_info": {"rank": rank, "device": ctx.device_index, **shard, "columns": N,
                          "sync_ms": sum(sync_ms) / len(sync_ms)}}


def measure_e2e(args, w, ctx: RankCtx, dev, theta, omega, delta, rnd, shard) -> dict:
    """The same round through the host-memory entry points: replicas in page-locked host arrays,
    host->device and device->host copies of theta, omega and Delta inside the timed call, on a
    bounded column sample so that all ranks together pin at most ~26 GB of host RAM.  Beside it the
    box's own ceiling: the same bytes copied both ways at once with plain pinned copies."""
    import torch
    from paper_1909_09010_b200 import binding, workloads
    K, N = w.K, w.N
    world = ctx.world
    tdt = torch.float32 if w.dtype == 0 else torch.bfloat16
    C = min(N, args.e2e_cols // world // 32 * 32)
    sh = workloads.shard_columns(w.offsets, 0, C)
    cld = workloads.padded_ld(C)
    hth = torch.empty((K, cld), dtype=tdt, pin_memory=True)
    hom = torch.empty((K, cld), dtype=torch.float32, pin_memory=True)
    hde = torch.empty((K, cld), dtype=torch.float32, pin_memory=True)
    hth[:, :C].copy_(theta[:, :C])
    hom[:, :C].copy_(omega[:, :C])
    hde[:, :C].copy_(delta[:, :C])
    torch.cuda.synchronize()
    h = binding.GbmufHost(sh.offsets, K=K, N=C, ld=cld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta,
                          seed=w.seed, theta_dtype=w.dtype, device=ctx.device_index, mode=w.mode,
                          chunk_cols=args.e2e_chunk_cols, row_copies=args.e2e_row_copies, **shard)
    h.sync_round(hth, hom, hde, rnd)                                        # warm-up
    ctx.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(args.e2e_steps):
        h.sync_round(hth, hom, hde, rnd + 1 + i)                            # returns with the result on the host
    ctx.barrier()
    t_e2e = ctx.max_over_ranks(time.perf_counter() - t0)
    h.destroy()
    esz = 4 if w.dtype == 0 else 2
    per_dir = K * C * ((esz + 8) if w.mode == 0 else esz)
    # the ceiling on this machine: the same bytes each way, both directions at once, nothing else
    scratch = [torch.empty((K, cld), dtype=t.dtype, device=dev) for t in (hth, hom, hde)]
    src = [torch.empty((K, cld), dtype=t.dtype, device=dev) for t in (hth, hom, hde)]
    arrays = (0, 1, 2) if w.mode == 0 else (0,)
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    best = None
    for _ in range(3):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        with torch.cuda.stream(s_in):
            for i in arrays:
                scratch[i].copy_((hth, hom, hde)[i], non_blocking=True)
        with torch.cuda.stream(s_out):
            for i in arrays:                     # (writes the host arrays: their contents are no longer needed)
                (hth, hom, hde)[i].copy_(src[i], non_blocking=True)
        s_in.synchronize()
        s_out.synchronize()
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    pad = cld / C
    ceiling = per_dir * pad / best / 1e9
    rate = per_dir / (t_e2e / args.e2e_steps) / 1e9
    del hth, hom, hde, scratch, src
    return {"value": world * K * C * args.e2e_steps / t_e2e, "unit": UNIT,
            "h2d_bytes_per_step": per_dir, "d2h_bytes_per_step": per_dir,
            "steps": args.e2e_steps, "ms_per_step": t_e2e / args.e2e_steps * 1e3,
            "gbs_each_way": rate, "pcie_gbs_each_way_on_this_box": ceiling, "frac": rate / ceiling,
            "sample": f"columns [0,{C}) of {w.name} per GPU, all K={K} replicas, "
                      "page-locked host arrays, gbmuf_host_sync_round (buffers and streams kept across rounds)"}


# ------------------------------------------------------------------------------------------------
# Peer leg: one worker per rank, neighbours' slices pulled from the other ranks' memory
# ------------------------------------------------------------------------------------------------
def peer_leg(args, w, ctx: RankCtx) -> dict:
    import torch
    from paper_1909_09010_b200 import binding, build, peer_ipc, workloads

    if ctx.world < 2:
        raise SystemExit("bench.py: form=peer needs at least two ranks (one worker per rank)")
    build.build()
    torch.cuda.set_device(ctx.device_index)
    dev = torch.device(f"cuda:{ctx.device_index}")
    rank, K = ctx.rank, ctx.world
    N, ld = w.N, w.ld
    p = w.p
    q = min(w.q, min(2 * p, K - 1))
    tdt = torch.float32 if w.dtype == 0 else torch.bfloat16
    theta0 = workloads.theta0_torch(w, dev).to(tdt)
    own = [torch.zeros(ld, dtype=tdt, device=dev), torch.zeros(ld, dtype=tdt, device=dev)]
    own[0][:N].copy_(theta0)
    omega = torch.zeros(ld, dtype=torch.float32, device=dev)
    omega[:N].copy_(theta0.float())
    delta = torch.zeros(ld, dtype=torch.float32, device=dev)
    del theta0
    views = peer_ipc.exchange_buffers(own)
    for r in range(K):                 # touching a peer's memory once lets torch enable peer access
        if r != rank:
            _ = views[r][0][:1].to(dev)
    bufs = [[views[r][b] for r in range(K)] for b in (0, 1)]
    wk = binding.GbmufPeer(rank, bufs, omega, delta, K=K, N=N, ld=ld, p=p, q=q, eta=w.eta, zeta=w.zeta,
                           seed=w.seed, theta_dtype=w.dtype, device=ctx.device_index, mode=w.mode)
    wk.set_partition(w.offsets)
    lr, sigma = w.lr or 0.1, w.sigma or 1e-3

    def barrier():
        torch.cuda.synchronize()
        ctx.barrier()

    cur, rnd = 0, 1

    def local_step(step):
        # this worker's synthetic local step: a seeded input (no method arithmetic), applied in place
        # (the product and the difference are separate tensor operations: each rounds once)
        upd = workloads.replica_noise_torch(w, rank, step, N, dev).mul_(lr * sigma)
        if w.dtype == 0:
            own[cur][:N].sub_(upd)
        else:
            own[cur][:N].copy_((own[cur][:N].float() - upd).to(tdt))

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for _ in range(args.warmup):
        local_step(rnd)
        barrier()                      # everybody's local step is in place before anybody pulls
        wk.sync_round(rnd, cur)
        barrier()                      # everybody's round has finished before the buffers swap roles
        cur, rnd = 1 - cur, rnd + 1
    sampler = ClockSampler(ctx.device_index).start() if rank == 0 else None
    t_wall0 = time.time()
    for i in range(args.steps):
        local_step(rnd)
        barrier()
        a, b = ev[i]
        a.record()
        wk.sync_round(rnd, cur)
        b.record()
        barrier()
        cur, rnd = 1 - cur, rnd + 1
    t_wall1 = time.time()
    clocks = None
    if sampler is not None:
        clocks = sampler.window(t_wall0, t_wall1)
        sampler.stop()
    status = wk.device_status()
    sync_ms = [a.elapsed_time(b) for a, b in ev]
    total_sync_s = ctx.max_over_ranks(sum(sync_ms) / 1e3)
    if args.save_state:
        os.makedirs(args.save_state, exist_ok=True)
        torch.save({"rank": rank, "world": K, "rounds": rnd - 1, "p": p, "q": q,
                    "theta": own[cur][:N].cpu(), "omega": omega[:N].cpu(), "delta": delta[:N].cpu()},
                   os.path.join(args.save_state, f"rank{rank}.pt"))
    esz = 4 if w.dtype == 0 else 2
    # what must move per worker and round: q slices over the links; own theta, omega, Delta read
    # and omega, Delta, theta written in local memory
    link_bytes = q * esz * N
    hbm_bytes = (esz + 8 + 8 + esz) * N if w.mode == 0 else 2 * esz * N
    peak_hbm, kind = measured_peak()
    t_link = link_bytes / (NVLINK_GBS_PER_DIRECTION * 1e9)
    t_hbm = hbm_bytes / (peak_hbm * 1e9)
    shared = args.share_device is not None
    bound = "hbm" if shared or t_hbm >= t_link else "nvlink"
    t_launch = sum(sync_ms) / len(sync_ms) / 1e3
    if bound == "nvlink":
        achieved, peak = link_bytes / t_launch / 1e9, NVLINK_GBS_PER_DIRECTION
    else:
        achieved, peak = (hbm_bytes + (link_bytes if shared else 0)) / t_launch / 1e9, peak_hbm
    roofline = {"bound": bound, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": "measured peer copy per direction on this pool" if bound == "nvlink" else f"of {kind}",
                "link_bytes_per_worker_round": link_bytes, "local_bytes_per_worker_round": hbm_bytes,
                "traffic": None, "kernel": "peer_round_kernel"}
    config = {"workload": w.name, "form": "peer", "K": K, "N": N, "components": w.m, "p": p, "q": q,
              "eta": w.eta, "zeta": w.zeta, "mode": "gossip-MA" if w.mode else "gossip-BMUF",
              "replica_params_per_gpu": N,
              "parallelism": parallelism_text("peer", K),
              "l2": "inputs_larger_than_l2" if N * (esz + 8) > (126 << 20) else "flushed_by_the_local_step_between_rounds",
              "device_status": status}
    wk.destroy()
    ctx.barrier()
    del views, bufs
    return {"units_per_rank": N, "total_sync_s": total_sync_s, "config": config, "roofline": roofline,
            "clocks": clocks, "gpu_launches": 2 * args.steps, "e2e": None,
            "rank_info": {"rank": rank, "device": ctx.device_index, "worker": rank, "columns": N,
                          "sync_ms": sum(sync_ms) / len(sync_ms)}}


# ------------------------------------------------------------------------------------------------
def build_parser() -> argparse.ArgumentParser:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="gbmuf", choices=["gbmuf", "reference"])
    ap.add_argument("--workload", default="wikitext103")
    ap.add_argument("--tuning", default="", help="consumer_threads,tile_elems,theta_stages,ring_slots,flags")
    ap.add_argument("--ref-cols", type=int, default=1 << 23,
                    help="columns of the workload the CPU oracle is timed on")
    ap.add_argument("--ref-rounds", type=int, default=12,
                    help="oracle rounds timed for the cpu_baseline entry (about 20 s of CPU work in all)")
    ap.add_argument("--local-step", default="perturb", choices=["perturb", "adagrad"],
                    help="what moves the replicas between rounds (launched outside the timed interval)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="skip the extra timing of the rounds replayed from one CUDA graph")
    ap.add_argument("--no-regimes", action="store_true",
                    help="skip the seconds-long regimes (round next to an ALU-bound step, back to back, "
                         "next to a bandwidth-bound step, and a sustained device copy) with sampled clocks")
    ap.add_argument("--regime-rounds", type=int, default=200)
    ap.add_argument("--e2e-cols", type=int, default=1 << 27,
                    help="columns (summed over ranks) of the end-to-end host-buffer sample")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-chunk-cols", type=int, default=0, help="columns per chunk (0 = the library's choice)")
    ap.add_argument("--e2e-row-copies", action="store_true", help="K row copies per array and chunk instead of one 2-D copy")
    ap.add_argument("--share-device", type=int, default=None, metavar="D",
                    help="run every rank on cuda:D over gloo: a correctness check of the multi-rank path on a "
                         "box with fewer GPUs than ranks, not a measurement")
    ap.add_argument("--save-state", default="", metavar="DIR",
                    help="each rank writes its theta, omega, Delta after the timed rounds to DIR/rank<r>.pt")
    return ap


def resolve_workload(args):
    from paper_1909_09010_b200 import workloads
    name, _, opts = args.workload.partition(":")           # e.g. sweep:C=64,q=4,eta=0.5 or wikitext103:mode=1
    over, form = {}, "resident"
    for kv in filter(None, opts.split(",")):
        k, v = kv.split("=")
        if k == "form":
            form = v
        else:
            over[k] = float(v) if k == "eta" else int(v)
    if form not in ("resident", "peer"):
        raise SystemExit(f"bench.py: unknown form {form!r}")
    args.form = form
    return workloads.get(name, **over)


def main(argv=None):
    args = build_parser().parse_args(argv)
    w = resolve_workload(args)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        launch_ranks(args)                      # no launcher: start the ranks ourselves
    else:
        run_ranked(args, w)


if __name__ == "__main__":
    main()
