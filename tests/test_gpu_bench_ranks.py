"""The multi-rank paths of `bench.py` with the PRODUCT inside the ranks: the bench starts its own
rank processes, every rank runs the CUDA library on its share, and what the ranks leave behind is
compared bit for bit with the CPU oracle's unsharded run.

Only one GPU is available, so all ranks use cuda:0 (`--share-device 0`, gloo between them).  No
kernel of one rank waits for a kernel of another: the ranks meet only at host barriers."""
import json

import numpy as np
import pytest
import torch

import bench
import oracle
from paper_1909_09010_b200 import workloads

pytestmark = pytest.mark.gpu


def _run(argv, capfd):
    args = bench.build_parser().parse_args(argv)
    w = bench.resolve_workload(args)
    bench.launch_ranks(args)
    out = capfd.readouterr().out
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out
    return args, w, json.loads(lines[0])


def test_element_range_shards_as_two_rank_processes(tmp_path, capfd):
    """Rank r = columns [r*N, (r+1)*N) of a model twice as wide, global component / element
    indices through comp_base / elem_base.  Reassembled, the ranks' theta, omega, Delta must
    equal the oracle's run over the wide model."""
    world, W, S = 2, 1, 2
    args, w, line = _run(["--gpus", str(world), "--workload", "tiny", "--steps", str(S), "--warmup", str(W),
                          "--share-device", "0", "--no-graph", "--no-e2e", "--no-cpu-baseline",
                          "--no-regimes", "--save-state", str(tmp_path)], capfd)
    assert line["n_gpus"] == world
    assert line["config"]["parallelism"] == "element-range shards x2, no collective"
    assert [r["comp_base"] for r in line["config"]["ranks"]] == [0, w.m]
    assert [r["elem_base"] for r in line["config"]["ranks"]] == [0, w.N]
    assert line["config"]["device_status"] == 0 and line["value"] > 0

    # the oracle over the wide model: every rank started from the same seeded theta_0
    N, K = w.N, w.K
    theta0 = workloads.theta0_torch(w, torch.device("cuda:0")).cpu().numpy()
    wide_offsets = [r * N + x for r in range(world) for x in w.offsets[:-1]] + [world * N]
    st = oracle.init(np.concatenate([theta0] * world), K)
    lr, sigma = w.lr or 0.1, w.sigma or 1e-3
    oracle.local_perturb(st, w.seed, 0, lr, sigma, 1)
    for rnd in range(1, W + S + 1):
        oracle.local_perturb(st, w.seed, rnd, lr, sigma, 1)
        nbr = oracle.sample_neighbors(w.seed, rnd, K, len(wide_offsets) - 1, w.p, w.q)
        oracle.sync_round(st, wide_offsets, nbr, w.eta, w.zeta)
    for r in range(world):
        got = torch.load(tmp_path / f"rank{r}.pt")
        assert got["rounds"] == W + S and got["comp_base"] == r * w.m and got["elem_base"] == r * N
        cols = slice(r * N, (r + 1) * N)
        for name, ref in (("theta", st.theta), ("omega", st.omega), ("delta", st.delta)):
            a = got[name].numpy()
            assert np.array_equal(a.view(np.uint32), ref[:, cols].view(np.uint32)), f"rank {r} {name}"


@pytest.mark.parametrize("world,q", [(2, 1), (3, 2)])
def test_one_worker_per_rank_through_the_bench(world, q, tmp_path, capfd):
    """form=peer: rank r is worker r; its round kernel pulls the drawn neighbours' slices out of
    the other processes' buffers (mapped through CUDA IPC).  Compared with the oracle's
    K-replica round."""
    W, S = 1, 2
    args, w, line = _run(["--gpus", str(world), "--workload", f"tiny:form=peer,q={q}", "--steps", str(S),
                          "--warmup", str(W), "--share-device", "0", "--no-cpu-baseline",
                          "--save-state", str(tmp_path)], capfd)
    assert line["n_gpus"] == world and line["config"]["form"] == "peer"
    assert f"one worker per rank x{world}" in line["config"]["parallelism"]
    assert line["config"]["device_status"] == 0
    assert line["roofline"]["kernel"] == "peer_round_kernel"
    assert [r["worker"] for r in line["config"]["ranks"]] == list(range(world))

    N, K = w.N, world
    dev = torch.device("cuda:0")
    theta0 = workloads.theta0_torch(w, dev).cpu().numpy()
    st = oracle.init(theta0, K)
    lr, sigma = w.lr or 0.1, w.sigma or 1e-3
    p, qq = w.p, line["config"]["q"]
    assert qq == q
    for rnd in range(1, W + S + 1):
        for k in range(K):                         # the ranks' local steps: the same seeded input
            upd = workloads.replica_noise_torch(w, k, rnd, N, dev).cpu().numpy() * np.float32(lr * sigma)
            st.theta[k, :N] = st.theta[k, :N] - upd
        nbr = oracle.sample_neighbors(w.seed, rnd, K, w.m, p, qq)
        oracle.sync_round(st, w.offsets, nbr, w.eta, w.zeta)
    for r in range(world):
        got = torch.load(tmp_path / f"rank{r}.pt")
        for name, ref in (("theta", st.theta), ("omega", st.omega), ("delta", st.delta)):
            a = got[name].numpy()
            assert np.array_equal(a.view(np.uint32), ref[r, :N].view(np.uint32)), f"worker {r} {name}"
