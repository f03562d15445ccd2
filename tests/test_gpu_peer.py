"""The one-worker-per-GPU form on ONE GPU: the K workers' buffers all live on cuda:0 and each
worker's round is launched one after the other (no kernel waits for another), which is exactly
what K GPUs would run at the same time because a round only reads the 'current' buffers and only
writes the 'other' ones.  Compared with the CPU oracle's K-replica round."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_09010_b200 import binding
from harness import ATOL, RTOL, random_theta0, to_numpy, from_numpy, tdtype

pytestmark = pytest.mark.gpu


class Emulated:
    def __init__(self, K, offsets, p, q, eta, zeta, dtype, seed, mode=0, periods=None):
        self.K, self.offsets, self.p, self.q, self.eta, self.zeta = K, offsets, p, q, eta, zeta
        self.dtype, self.seed, self.mode, self.periods = dtype, seed, mode, periods
        dev = torch.device("cuda:0")
        N = offsets[-1]
        ld = (N + 31) // 32 * 32
        self.N, self.ld = N, ld
        self.st = oracle.init(random_theta0(N, seed=seed + 1, dtype=dtype), K, ld=ld, dtype=dtype)
        g = np.random.Generator(np.random.PCG64(seed))
        drift = (g.standard_normal((K, N)) * 0.05).astype(np.float32)
        if dtype == 0:
            self.st.theta[:, :N] += drift
        else:
            self.st.theta[:, :N] = oracle.f32_to_bf16(oracle.bf16_to_f32(self.st.theta[:, :N]) + drift)
        # per worker: two theta buffers, omega, Delta -- separate allocations, as on separate GPUs
        self.bufs = [[from_numpy(self.st.theta[k].copy(), dtype, dev) for k in range(K)],
                     [torch.full((ld,), 7.0, dtype=tdtype(dtype), device=dev) for k in range(K)]]
        self.omega = [torch.from_numpy(self.st.omega[k].copy()).to(dev) for k in range(K)]
        self.delta = [torch.from_numpy(self.st.delta[k].copy()).to(dev) for k in range(K)]
        self.workers = []
        for k in range(K):
            w = binding.GbmufPeer(k, self.bufs, self.omega[k], self.delta[k], K=K, N=N, ld=ld, p=p, q=q,
                                  eta=eta, zeta=zeta, seed=seed, mode=mode, theta_dtype=dtype)
            w.set_partition(offsets, periods)
            self.workers.append(w)
        self.cur = 0

    def round(self, rnd, mask=None):
        for w in self.workers:                       # "all GPUs at once": order cannot matter
            w.sync_round(rnd, self.cur, mask)
        torch.cuda.synchronize()                     # stands for the barrier between workers
        for w in self.workers:
            assert w.device_status() == 0
        self.cur = 1 - self.cur
        m = len(self.offsets) - 1
        per = self.periods or [1] * m
        due = [bool(x) for x in mask] if mask is not None else [rnd % h == 0 for h in per]
        nbr = oracle.sample_neighbors(self.seed, rnd, self.K, m, self.p, self.q)
        oracle.sync_round(self.st, self.offsets, nbr, self.eta, self.zeta, mode=self.mode, sync=due)

    def check(self, what):
        N = self.N
        for k in range(self.K):
            got_t = to_numpy(self.bufs[self.cur][k])[:N]
            assert np.array_equal(got_t.view(np.uint8), self.st.theta[k, :N].view(np.uint8)), f"{what}: theta of worker {k}"
            for name, got, ref in (("omega", self.omega[k], self.st.omega[k]), ("delta", self.delta[k], self.st.delta[k])):
                got = got.cpu().numpy()
                assert np.all(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref)), f"{what}: {name} of worker {k}"
                assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), f"{what}: {name} of worker {k}"

    def local_step(self, g):
        noise = (g.standard_normal((self.K, self.N)) * 0.01).astype(np.float32)
        for k in range(self.K):
            cur = self.bufs[self.cur][k]
            if self.dtype == 0:
                cur[:self.N] += torch.from_numpy(noise[k]).to(cur.device)
                self.st.theta[k, :self.N] += noise[k]
            else:
                upd = (cur[:self.N].float() + torch.from_numpy(noise[k]).to(cur.device)).to(torch.bfloat16)
                cur[:self.N] = upd
                self.st.theta[k, :self.N] = upd.view(torch.int16).cpu().numpy().view(np.uint16)

    def close(self):
        for w in self.workers:
            w.destroy()


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("K,offsets,p,q", [
    (4, (0, 1000, 5001, 9000, 20003), 1, 1),
    (8, (0, 7, 4099, 4100, 33000, 70001), 2, 2),
    (16, (0, 40_000, 40_001, 100_005), 3, 2),
    (5, (0, 2049, 6000), 2, 4),
    (1, (0, 3001), 0, 0),
])
def test_peer_rounds_match_oracle(dtype, K, offsets, p, q):
    em = Emulated(K, offsets, p, q, 0.875, 1.0, dtype, seed=K * 7 + q)
    g = np.random.Generator(np.random.PCG64(5))
    try:
        m = len(offsets) - 1
        masks = [None, [i % 2 for i in range(m)], None, [0] * m]
        for r in range(1, 5):
            em.local_step(g)
            em.round(r, masks[r - 1])
            em.check(f"round {r}")
    finally:
        em.close()


def test_peer_periods_and_ma_mode():
    em = Emulated(8, (0, 3000, 3001, 12000, 30011), 2, 2, 0.9, 1.0, 0, seed=3, periods=(1, 2, 3, 2))
    g = np.random.Generator(np.random.PCG64(6))
    try:
        for r in range(1, 7):
            em.local_step(g)
            em.round(r)
            em.check(f"periods round {r}")
    finally:
        em.close()
    em = Emulated(8, (0, 3000, 12000), 2, 2, 0.9, 1.0, 0, seed=4, mode=binding.MODE_MA)
    try:
        for r in (1, 2):
            em.local_step(g)
            em.round(r)
            em.check(f"MA round {r}")
    finally:
        em.close()


def test_peer_argument_errors():
    dev = torch.device("cuda:0")
    bufs = [[torch.zeros(64, device=dev) for _ in range(2)] for _ in range(2)]
    om, de = torch.zeros(64, device=dev), torch.zeros(64, device=dev)
    kw = dict(K=2, N=64, ld=64, p=1, q=1, eta=0.9, zeta=1.0)
    with pytest.raises(binding.GbmufError):
        binding.GbmufPeer(2, bufs, om, de, **kw)                      # rank out of range
    same = [[bufs[0][0], bufs[0][1]], [bufs[0][0], bufs[1][1]]]
    with pytest.raises(binding.GbmufError):
        binding.GbmufPeer(0, same, om, de, **kw)                      # own buffers identical
    w = binding.GbmufPeer(0, bufs, om, de, **kw)
    with pytest.raises(binding.GbmufError) as e:
        w.sync_round(1, 0)
    assert e.value.status == binding.ERR_BAD_STATE
    w.set_partition([0, 10, 64])
    with pytest.raises(binding.GbmufError):
        w.sync_round(1, 2)
    w.destroy()


# ------------------------------------------------------------------------------------------------
# the same thing as separate processes: one worker per process, buffers shared through CUDA IPC,
# a host barrier between rounds.  All processes use cuda:0 here; no kernel waits for another.
# ------------------------------------------------------------------------------------------------
def _peer_process(rank, world, port, out_dir):
    import os
    import torch.distributed as dist
    from paper_1909_09010_b200 import peer_ipc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        K, p, q, eta, seed = world, 1, 2 if world > 2 else 1, 0.9, 17
        offsets = (0, 5001, 5002, 30_000, 70_003)
        N = offsets[-1]
        ld = (N + 31) // 32 * 32
        dev = torch.device("cuda:0")
        st = oracle.init(random_theta0(N, seed=2), K, ld=ld)             # every process: whole oracle
        g = np.random.Generator(np.random.PCG64(9))
        st.theta[:, :N] += (g.standard_normal((K, N)) * 0.05).astype(np.float32)
        own = [torch.from_numpy(st.theta[rank].copy()).to(dev), torch.zeros(ld, device=dev)]
        om = torch.from_numpy(st.omega[rank].copy()).to(dev)
        de = torch.zeros(ld, device=dev)
        views = peer_ipc.exchange_buffers(own)
        bufs = [[views[r][b] for r in range(K)] for b in (0, 1)]
        w = binding.GbmufPeer(rank, bufs, om, de, K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=1.0, seed=seed)
        w.set_partition(offsets)
        cur = 0
        for rnd in (1, 2, 3):
            noise = (g.standard_normal((K, N)) * 0.01).astype(np.float32)
            own[cur][:N] += torch.from_numpy(noise[rank]).to(dev)       # local step on own replica
            st.theta[:, :N] += noise
            torch.cuda.synchronize()
            dist.barrier()                                               # everybody's local step is visible
            mask = None if rnd != 2 else [1, 0, 1, 1]
            w.sync_round(rnd, cur, mask)
            torch.cuda.synchronize()
            assert w.device_status() == 0
            dist.barrier()                                               # everybody's round is finished
            cur = 1 - cur
            nbr = oracle.sample_neighbors(seed, rnd, K, 4, p, q)
            oracle.sync_round(st, offsets, nbr, eta, 1.0, sync=mask)
            assert np.array_equal(own[cur].cpu().numpy()[:N].view(np.uint32), st.theta[rank, :N].view(np.uint32))
            assert np.array_equal(om.cpu().numpy().view(np.uint32), st.omega[rank].view(np.uint32))
            assert np.array_equal(de.cpu().numpy().view(np.uint32), st.delta[rank].view(np.uint32))
        dist.barrier()
        w.destroy()
        del views, bufs
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_peer_processes_share_buffers_over_ipc(world, tmp_path):
    import os
    import socket
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_peer_process, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))
