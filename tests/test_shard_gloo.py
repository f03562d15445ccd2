"""The column-range shard planner on CPU: `workloads.shard_even` cuts the columns between ranks,
and because the path shards with no data exchange, running the round on each share alone must
reassemble to the unsharded result.  Two gloo ranks do that here with the oracle as the round
(these ranks have no GPU): this pins the PLANNER (global component / element indices of a share).
The ranks of the product are covered elsewhere: `test_bench_ranks.py` drives the bench's own rank
launching with two gloo ranks on CPU, and `test_gpu_bench_ranks.py` runs the CUDA library inside
two rank processes and compares the reassembled state with the oracle."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1909_09010_b200 import workloads


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = workloads.get("tiny")
        N, K = 60_011, w.K
        offsets = (0, 7, 20_000, 20_001, 41_111, N)
        theta0 = workloads.theta0_numpy(w, N)
        sh = workloads.shard_even(offsets, world, rank)
        st = oracle.init(theta0[sh.col0:sh.col1].copy(), K)
        for r in (1, 2, 3):
            oracle.local_perturb(st, w.seed, r, 0.1, 0.05, 2, elem_base=sh.col0)
            nbr = oracle.sample_neighbors(w.seed, r, K, sh.m, w.p, w.q, comp_base=sh.comp_base)
            oracle.sync_round(st, sh.offsets, nbr, w.eta, w.zeta)
        # no collective on the data path: results are only gathered here to be checked
        mine = torch.from_numpy(np.stack([st.theta, st.omega, st.delta]))
        sizes = [None] * world
        dist.all_gather_object(sizes, (sh.col0, sh.col1))
        gathered = [None] * world
        dist.all_gather_object(gathered, mine.numpy())
        # bench-style timing reduction: max over ranks
        t = torch.tensor([0.5 + rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert float(t.item()) == 0.5 + world - 1
        if rank == 0:
            full = oracle.init(theta0, K)
            for r in (1, 2, 3):
                oracle.local_perturb(full, w.seed, r, 0.1, 0.05, 2)
                nbr = oracle.sample_neighbors(w.seed, r, K, len(offsets) - 1, w.p, w.q)
                oracle.sync_round(full, offsets, nbr, w.eta, w.zeta)
            cat = np.concatenate(gathered, axis=2)
            assert sizes[0][0] == 0 and sizes[-1][1] == N
            assert all(sizes[i][1] == sizes[i + 1][0] for i in range(world - 1))
            assert np.array_equal(cat[0], full.theta) and np.array_equal(cat[1], full.omega)
            assert np.array_equal(cat[2], full.delta)
            open(os.path.join(out_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_column_shards_reassemble(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert os.path.exists(tmp_path / "ok")


def test_shard_planner_properties():
    for name in ("tiny", "mid", "wikitext103", "longrun"):
        w = workloads.get(name)
        for world in (1, 2, 3, 8):
            prev = 0
            for rank in range(world):
                sh = workloads.shard_even(w.offsets, world, rank)
                assert sh.col0 == prev and sh.col0 % 32 == 0
                prev = sh.col1
                # local offsets map back onto the global component edges inside the range
                glob = [sh.col0 + x for x in sh.offsets]
                inner = [x for x in w.offsets if sh.col0 < x < sh.col1]
                assert glob[1:-1] == inner and glob[0] == sh.col0 and glob[-1] == sh.col1
                assert w.offsets[sh.comp_base] <= sh.col0 < w.offsets[sh.comp_base + 1]
            assert prev == w.N
    sh = workloads.shard_columns((0, 10, 20, 30), 10, 20)
    assert (sh.comp_base, sh.offsets) == (1, (0, 10))
    sl = workloads.edge_slices(workloads.get("wikitext103").offsets, 4096)
    assert sl[0][0] == 0 and sl[-1][1] == workloads.get("wikitext103").N
