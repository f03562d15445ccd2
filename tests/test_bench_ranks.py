"""`bench.py --gpus N` starts its own N rank processes when no launcher did; this drives that path
on CPU: two gloo ranks, with a stand-in for the GPU leg (these ranks have no GPU), through the
same framing the real legs use -- process group, barrier, max-over-ranks time, gathering of each
rank's shard, rank 0 printing the one line."""
import json
import os
import subprocess
import sys

import pytest

import bench

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def stub_leg(args, w, ctx):
    """What gpu_leg hands back, without touching a GPU: rank r claims r + 0.5 s for its rounds."""
    shard = bench.rank_shard(w, ctx.rank)
    total = ctx.max_over_ranks(0.5 + ctx.rank)
    ctx.barrier()
    return {"units_per_rank": w.K * w.N, "total_sync_s": total,
            "config": {"workload": w.name, "parallelism": bench.parallelism_text("resident", ctx.world)},
            "roofline": None, "clocks": None, "gpu_launches": 0, "e2e": None,
            "rank_info": {"rank": ctx.rank, "device": None, **shard, "columns": w.N}}


def test_gpus_2_without_a_launcher_runs_two_ranks(capfd):
    args = bench.build_parser().parse_args(["--gpus", "2", "--steps", "4", "--warmup", "3",
                                            "--workload", "tiny", "--no-cpu-baseline"])
    w = bench.resolve_workload(args)
    bench.launch_ranks(args, leg=stub_leg, backend="gloo")
    out = capfd.readouterr().out
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["warmup"] == 3
    assert line["config"]["parallelism"] == "element-range shards x2, no collective"
    ranks = line["config"]["ranks"]
    assert [r["rank"] for r in ranks] == [0, 1]
    assert [r["comp_base"] for r in ranks] == [0, w.m]
    assert [r["elem_base"] for r in ranks] == [0, w.N]
    # whole-job value: both ranks' units over the slowest rank's time (1.5 s)
    assert line["value"] == pytest.approx(2 * w.K * w.N * 4 / 1.5)
    assert line["ms_per_step"] == pytest.approx(1.5 / 4 * 1e3)
    assert line["scaling"] == "weak" and line["higher_is_better"] is True


def test_rank_count_must_match_the_launcher(monkeypatch):
    args = bench.build_parser().parse_args(["--gpus", "2", "--workload", "tiny"])
    w = bench.resolve_workload(args)
    monkeypatch.setenv("WORLD_SIZE", "1")
    monkeypatch.setenv("RANK", "0")
    with pytest.raises(SystemExit) as e:
        bench.run_ranked(args, w, leg=stub_leg, backend="gloo")
    assert "--gpus 2" in str(e.value)


def test_more_ranks_than_gpus_is_refused():
    """Without enough CUDA devices `--gpus N` must say so instead of quietly running fewer."""
    import torch
    have = torch.cuda.device_count()
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(have + 2),
                        "--workload", "tiny", "--steps", "1", "--warmup", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode != 0
    assert f"--gpus {have + 2}" in r.stderr and "CUDA device" in r.stderr
    assert not any(l.startswith("{") for l in r.stdout.splitlines())


def test_peer_form_is_parsed_and_needs_ranks():
    args = bench.build_parser().parse_args(["--workload", "tiny:form=peer,q=2"])
    w = bench.resolve_workload(args)
    assert args.form == "peer" and w.q == 2
    assert "one worker per rank x3" in bench.parallelism_text("peer", 3)
    with pytest.raises(SystemExit):
        bench.resolve_workload(bench.build_parser().parse_args(["--workload", "tiny:form=nope"]))


def test_clock_sampler_summarises_a_window():
    """The nvidia-smi sampler's parsing and binning, fed with canned rows (no GPU needed)."""
    s = bench.ClockSampler(0)
    s.proc = object()                                    # pretend the query is running
    row = "{sm}, 1965, {w}, Not Active, Not Active, Not Active, {cap}, 3996"
    s.rows = [(10.0, row.format(sm=1965, w=700.0, cap="Not Active")),
              (10.1, row.format(sm=1740, w=995.5, cap="Active")),
              (10.2, row.format(sm=1725, w=996.0, cap="Active")),
              (10.3, "garbage"),
              (99.0, row.format(sm=500, w=100.0, cap="Not Active"))]      # outside the window
    out = s.window(10.0, 10.25, detail=True)
    assert out["samples"] == 3 and out["sm_mhz"] == 1740.0 and out["sm_max_mhz"] == 1965.0
    assert out["reasons"] == ["sw_power_cap"] and out["mem_mhz"] == 3996.0
    assert out["power_w_max"] == 996.0 and out["samples_by_sm_mhz"] == {"1700-1799": 2, "1900-1999": 1}
    e = bench._regime_entry(17.0, 24 * 4458028400, 6530.0, out)
    assert abs(e["gbs"] - 24 * 4458028400 / 17.0e-3 / 1e9) < 1e-6 and abs(e["ms_x_sm_ghz"] - 17.0 * 1.74) < 1e-9


def test_traffic_constants_name_a_kernel_fingerprint():
    """The DRAM-traffic constants are only applied to the kernel source they were measured on."""
    sha = bench.source_sha()
    assert len(sha) == 12 and all(c in "0123456789abcdef" for c in sha)
    assert set(bench.NCU_TRAFFIC["bytes_per_replica_param"]) == {("tmem", 0), ("tmem", 1), ("tmem-window", 0)}
    for (variant, dtype), b in bench.NCU_TRAFFIC["bytes_per_replica_param"].items():
        alg = bench.algorithmic_bytes_per_replica_param(dtype)
        assert 0.97 * alg < b < 1.03 * alg, (variant, dtype, b)      # measured traffic ~ algorithmic bytes
