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
"""
from __future__ import annotations

import argparse
import hashlib
import re
import json
import os
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

# DRAM traffic of the fused kernel per replica-parameter from an ncu capture (dram__bytes_read.sum
# + dram__bytes_write.sum divided by the replica-parameters of the captured launch), valid only
# for the kernel source it was taken from (source_sha() below) and for the launch variant and
# theta dtype it was taken with: key = (variant, dtype); 0 fp32 from workload profile16, 1 bf16
# from profile16bf (all K rows in tensor memory); the ring-window figure is from profile64 and
# holds for that ring only (K = 64, p = 5: p / K extra theta row reads).
NCU_TRAFFIC = {"source_sha": "0e09b2d1894a",
               "bytes_per_replica_param": {("tmem", 0): 6.383437e9 / 268435536,
                                           ("tmem", 1): 5.308850e9 / 268435536,
                                           ("tmem-window", 0): 6.469350e9 / 268435776},
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


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        mhz, mx, reasons = [], None, set()
        for ts, line in self.rows:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7 or not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            try:
                mhz.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "samples": len(mhz), "reasons": sorted(reasons)}


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


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = args.ref_cols
    for _ in range(max(args.warmup, 0)):
        pass
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
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU leg
# ------------------------------------------------------------------------------------------------
def run_gpu(args, w):
    import torch
    import torch.distributed as dist
    from paper_1909_09010_b200 import binding, build, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    build.build()
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    # each rank holds the columns [rank*N, (rank+1)*N) of a model `world` times as wide: ranges of
    # columns are independent given the (counter-based) neighbour draws, so no data is exchanged
    K, N, ld = w.K, w.N, w.ld
    tdt = torch.float32 if w.dtype == 0 else torch.bfloat16
    theta = torch.empty((K, ld), dtype=tdt, device=dev)
    omega = torch.empty((K, ld), dtype=torch.float32, device=dev)
    delta = torch.empty((K, ld), dtype=torch.float32, device=dev)
    g = binding.Gbmuf(theta, omega, delta, K=K, N=N, ld=ld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta,
                      seed=w.seed, theta_dtype=w.dtype, device=local, comp_base=rank * w.m,
                      elem_base=rank * N, mode=w.mode)
    if args.tuning:
        t = [int(x) for x in args.tuning.split(",")]
        g.set_tuning(*t)
    g.set_partition(w.offsets)
    theta0 = workloads.theta0_torch(w, dev).to(tdt)
    g.init(theta0)
    del theta0
    lr, sigma = w.lr or 0.1, w.sigma or 1e-3
    g.local_perturb(0, lr, sigma, 1)
    if args.local_step == "adagrad":
        # the experiments' optimiser on a fixed synthetic gradient (std 1e-2); the recurrent
        # components (here: those of 1 Mi to 8 Mi elements) form the clipped group
        grad = torch.empty((K, ld), dtype=torch.float32, device=dev).normal_(0.0, 1e-2)
        accum = torch.full((K, ld), 0.1, dtype=torch.float32, device=dev)
        sizes = [w.offsets[i + 1] - w.offsets[i] for i in range(w.m)]
        clip_mask = [1 if n <= (1 << 23) and n >= (1 << 20) else 0 for n in sizes]

        def local_step(step):
            g.local_adagrad(grad, accum, lr, eps=1e-8, clip_norm=10.0, clip_mask=clip_mask)
    else:
        def local_step(step):
            g.local_perturb(step, lr, sigma, 1)
    torch.cuda.synchronize()
    info = g.launch_info()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
           torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    rnd = 1
    for _ in range(args.warmup):
        local_step(rnd)
        g.sync_round(rnd)
        rnd += 1
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
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
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    status = g.device_status()
    sync_ms = [b.elapsed_time(c) for a, b, c in ev]
    pert_ms = [a.elapsed_time(b) for a, b, c in ev]
    total_sync_s = sum(sync_ms) / 1e3
    tt = torch.tensor([total_sync_s], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    total_sync_s = float(tt.item())

    # ---- the same rounds back to back, replayed from one CUDA graph (set-up + fused kernel per
    # round, no local step in between): what a launch-bound small model gains from a graph
    graph_ms = None
    if not args.no_graph:
        gs = torch.cuda.Stream(device=dev)
        gs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(gs):
            g.sync_round(rnd)
            rnd += 1
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gs):
                for i in range(args.steps):
                    g.sync_round(rnd + i)
            rnd += args.steps
            ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph.replay()                      # warm-up replay
            ga.record(gs)
            graph.replay()
            gb.record(gs)
        gs.synchronize()
        torch.cuda.current_stream().wait_stream(gs)
        graph_ms = ga.elapsed_time(gb) / args.steps
        del graph
        status = status or g.device_status()

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

    # ---- end to end: the same round through the host-buffer entry point (replicas in page-locked
    # host memory; host->device and device->host copies of theta, omega and Delta inside the timed
    # call), on a bounded column sample so that all ranks together pin at most ~26 GB of host RAM
    e2e = None
    if not args.no_e2e:
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
        kw = dict(K=K, N=C, ld=cld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta, seed=w.seed,
                  theta_dtype=w.dtype, device=local, comp_base=rank * w.m, elem_base=rank * N,
                  mode=w.mode)
        binding.sync_round_host(hth, hom, hde, sh.offsets, rnd, **kw)          # warm-up
        barrier()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            binding.sync_round_host(hth, hom, hde, sh.offsets, rnd + 1 + i, **kw)
        barrier()
        t_e2e = time.perf_counter() - t0
        tt = torch.tensor([t_e2e], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        esz = 4 if w.dtype == 0 else 2
        e2e = {"value": world * K * C * args.e2e_steps / float(tt.item()), "unit": UNIT,
               "h2d_bytes_per_step": K * C * (esz + 8), "d2h_bytes_per_step": K * C * (esz + 8),
               "steps": args.e2e_steps, "ms_per_step": float(tt.item()) / args.e2e_steps * 1e3,
               "sample": f"columns [0,{C}) of {w.name} per GPU, all K={K} replicas, "
                         "page-locked host arrays, gbmuf_sync_round_host"}
        del hth, hom, hde

    line = None
    if rank == 0:
        units = world * K * N * args.steps
        value = units / total_sync_s
        peak, peak_kind = measured_peak()
        bpe = algorithmic_bytes_per_replica_param(w.dtype, w.mode)
        # per-launch figures of the fused kernel on this rank (the set-up kernel that shares the
        # event bracket runs for microseconds)
        t_launch = (sum(sync_ms) / len(sync_ms)) / 1e3
        achieved = bpe * K * N / t_launch / 1e9
        traffic = None
        per_param = NCU_TRAFFIC["bytes_per_replica_param"].get((info.get("variant"), w.dtype))
        if info.get("variant") == "tmem-window" and (K, w.p) != NCU_TRAFFIC["window_ring"]:
            per_param = None
        if per_param is not None and not args.tuning and w.mode == 0 and NCU_TRAFFIC["source_sha"] == source_sha():
            traffic = per_param * K * N
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_sync_s / args.steps * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32" if w.dtype == 0 else "bf16-stored/f32", "data": "synthetic",
                "config": {"workload": w.name, "K": K, "N": N, "components": w.m, "p": w.p, "q": w.q,
                           "eta": w.eta, "zeta": w.zeta, "mode": "gossip-MA" if w.mode else "gossip-BMUF",
                           "replica_params_per_gpu": K * N,
                           "parallelism": f"element-range shards x{world}, no collective",
                           "l2": "inputs_larger_than_l2 (state %.1f GB per GPU)" %
                                 ((K * ld * (8 + (4 if w.dtype == 0 else 2))) / 1e9),
                           "launch": info, "local_step": args.local_step,
                           "local_step_ms": sum(pert_ms) / len(pert_ms),
                           "round_plus_local_step_ms": (sum(pert_ms) + sum(sync_ms)) / len(sync_ms),
                           "sync_ms_min": min(sync_ms), "sync_ms_max": max(sync_ms),
                           "sync_ms_in_cuda_graph": graph_ms, "device_status": status},
                "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                             "frac_of_nominal_8TBs": achieved / 8000.0,
                             "algorithmic_bytes_per_replica_param": bpe, "traffic": traffic,
                             "device_copy_gbs_on_this_gpu": copy_gbs_live,
                             "kernel": "sync_fused_tmem_kernel" if str(info.get("variant")).startswith("tmem") else "sync_fused_kernel"},
                "clocks": clocks,
                "gpu_launches": (3 if args.local_step == "perturb" else 5) * args.steps, "e2e": e2e}
        if not args.no_cpu_baseline and world == 1:
            times, units_cpu = time_oracle_rounds(w, args.ref_cols, args.ref_rounds)
            t = sum(times) / len(times)
            line["cpu_baseline"] = {
                "value": units_cpu / t, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"columns [0,{min(args.ref_cols, N)}) of {w.name}, K={K}, {args.ref_rounds} rounds, "
                          f"{t:.2f} s per round"}
    g.destroy()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


def main():
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
    ap.add_argument("--e2e-cols", type=int, default=1 << 27,
                    help="columns (summed over ranks) of the end-to-end host-buffer sample")
    ap.add_argument("--e2e-steps", type=int, default=3)
    args = ap.parse_args()
    from paper_1909_09010_b200 import workloads
    name, _, opts = args.workload.partition(":")           # e.g. sweep:C=64,q=4,eta=0.5 or wikitext103:mode=1
    over = {}
    for kv in filter(None, opts.split(",")):
        k, v = kv.split("=")
        over[k] = float(v) if k == "eta" else int(v)
    w = workloads.get(name, **over)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
