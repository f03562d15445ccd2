"""Parity at the full sizes of the named workloads, in the launch configuration the bench times.

The oracle cannot hold 50 GB of state, but given the neighbour table every element of a round is
independent and both sides key their random streams by global component / element index, so the
oracle replays the same calls on column ranges: one range around every component edge (plus the
head and the unaligned tail) and a few interior ranges.  On top of that, properties that hold at
any size are checked over the whole state on the device."""
import numpy as np
import pytest
import torch

from paper_1909_09010_b200 import binding, workloads
from harness import Pair, case_of, check_round_every_element, tdtype

pytestmark = pytest.mark.gpu


def _slices(w, width=4096, interior=4):
    sl = workloads.edge_slices(w.offsets, width)
    g = np.random.Generator(np.random.PCG64(w.seed + 99))
    for _ in range(interior):
        a = int(g.integers(0, w.N - width))
        if all(b <= a or a + width <= c for c, b in sl):
            sl.append((a, a + width))
    return sorted(sl)


def _restart_invariant(pr, eta):
    """theta == store(fl(omega + fl(eta * Delta))) over the whole state (two separately rounded
    library operations on the device)."""
    N = pr.case.N
    ok = True
    for k in range(pr.case.K):                       # row by row keeps the temporaries small
        t = pr.delta[k, :N] * np.float32(eta)
        t += pr.omega[k, :N]
        ok = ok and bool(torch.equal(t.to(pr.theta.dtype), pr.theta[k, :N]))
    return ok


@pytest.mark.parametrize("name,over,tuning", [("wikitext103", {}, None), ("longrun", {}, None),
                                              ("sweep", dict(C=256, q=4, eta=0.5), None),
                                              ("sweep", dict(C=64, q=1, eta=0.9), None),
                                              ("sweep", dict(C=4, q=2, eta=0.9), None),
                                              ("sweep", dict(C=4, q=4, eta=0.5), None),
                                              ("sweep", dict(C=16, q=2, eta=0.5), None),
                                              ("sweep", dict(C=16, q=4, eta=0.9), None),
                                              ("wikitext103", {}, dict(flags=8))])
def test_full_size_sampled_parity(name, over, tuning):
    w = workloads.get(name, **over)
    dev = torch.device("cuda:0")
    theta0 = workloads.theta0_torch(w, dev)
    if w.dtype == 1:
        theta0 = theta0.to(torch.bfloat16)
    pr = Pair(case_of(w), theta0, slices=_slices(w), tuning=tuning)
    try:
        info = pr.g.launch_info()
        assert info["grid"] == torch.cuda.get_device_properties(0).multi_processor_count
        pr.compare("after init")
        for r in (1, 2):
            pr.perturb(step=r * w.local_steps, lr=w.lr, sigma=10 * w.sigma, nsteps=w.local_steps)
            pr.check_neighbors(r)
            mask = None if r == 1 else [i % 3 != 1 for i in range(w.m)]
            before = None
            if mask is not None:
                idle = [i for i in range(w.m) if not mask[i]][:4]
                before = [pr.theta[:, w.offsets[i]:w.offsets[i + 1]].double().sum().item() for i in idle]
            pr.sync(r, mask)
            pr.compare(f"round {r}")
            if mask is None:
                assert _restart_invariant(pr, w.eta), "restart point is not omega + eta*Delta"
            else:
                after = [pr.theta[:, w.offsets[i]:w.offsets[i + 1]].double().sum().item() for i in idle]
                assert before == after, "a component that did not take part was modified"
        assert not pr.theta[:, w.N:].any() and not pr.omega[:, w.N:].any()   # padding untouched
    finally:
        pr.close()


# ------------------------------------------------------------------------------------------------
# every element of a full-size launch
# ------------------------------------------------------------------------------------------------
def _full_round_check(w, second_round=True, tuning=None):
    """The first synchronisation from the state the initialisation line leaves (plus seeded local
    steps), and, if asked, a second one with some components idle from the state the first left (momentum and
    global models no longer trivial): all K * N elements of theta, omega and Delta against the
    oracle, in the launch configuration the bench times."""
    dev = torch.device("cuda:0")
    case = case_of(w, mode=w.mode)
    K, N, ld = w.K, w.N, w.ld
    theta0 = workloads.theta0_torch(w, dev).to(tdtype(w.dtype))
    theta = torch.empty((K, ld), dtype=tdtype(w.dtype), device=dev)
    omega = torch.empty((K, ld), dtype=torch.float32, device=dev)
    delta = torch.empty((K, ld), dtype=torch.float32, device=dev)
    g = binding.Gbmuf(theta, omega, delta, K=K, N=N, ld=ld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta,
                      seed=w.seed, theta_dtype=w.dtype, mode=w.mode)
    try:
        if tuning:
            g.set_tuning(**tuning)
        g.set_partition(w.offsets)
        info = g.launch_info()
        assert info["grid"] == torch.cuda.get_device_properties(0).multi_processor_count
        g.init(theta0)
        g.local_perturb(1, w.lr, 10 * w.sigma, w.local_steps)       # the replicas drift apart: G != 0
        pre_theta = theta.clone()
        g.sync_round(1)
        torch.cuda.synchronize()
        assert g.device_status() == 0
        n = check_round_every_element(case, 1, (pre_theta, theta0, None), (theta, omega, delta),
                                      what=f"{w.name} first synchronisation")
        assert n >= K * N // (1 << 26)
        if second_round:
            g.local_perturb(2, w.lr, 10 * w.sigma, w.local_steps)
            pre = (pre_theta.copy_(theta), omega.clone(), delta.clone())
            mask = [i % 5 != 3 for i in range(w.m)]
            g.sync_round(2, mask)
            torch.cuda.synchronize()
            assert g.device_status() == 0
            check_round_every_element(case, 2, pre, (theta, omega, delta), mask=mask,
                                      what=f"{w.name} second synchronisation")
    finally:
        g.destroy()


def test_every_element_of_the_headline_launch():
    """wikitext103 (K = 16, 278.6 M columns, fp32): the launch the bench times, all 4.46 G
    replica-parameters of two rounds."""
    _full_round_check(workloads.get("wikitext103"))


def test_every_element_of_a_long_run_round():
    """The mixed-precision workload (bf16 theta, K = 16, 238.5 M columns, 64 components)."""
    _full_round_check(workloads.get("longrun"), second_round=False)


def test_every_element_of_a_gossip_ma_round():
    """The other branch of Algorithm 1 (theta <- average) at the wikitext103 size: every element
    of one round through the gossip-MA schedule of the shared-memory kernel."""
    _full_round_check(workloads.get("wikitext103", mode=1), second_round=False)


def test_every_element_with_the_shared_memory_tile():
    """The gossip-BMUF round with the theta tile in shared memory (tuning flag bit 3), K = 8
    replicas of the wikitext103 model: every element of one round."""
    _full_round_check(workloads.get("sweep", C=16, q=2, eta=0.9), second_round=False, tuning=dict(flags=8))


def test_every_element_of_a_ring_window_round():
    """64 workers on the ring the paper's rule gives them (p = 5): the ring-window launch over
    1.07 G replica-parameters."""
    n = (1 << 24) + 5
    cuts = tuple(int(x) // 4 * 4 for x in np.linspace(0, n, 17)[:-1]) + (n,)
    w = workloads.get("profile64", offsets=cuts)
    assert w.K * w.N >= 1 << 30
    _full_round_check(w)


# ------------------------------------------------------------------------------------------------
# the whole schedule of a workload at full size, on sampled ranges
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,width,interior", [("wikitext103", 4096, 4), ("longrun", 1024, 2)])
def test_full_size_whole_schedule_sampled(name, width, interior):
    """All rounds the workload is specified with (wikitext103: 20 rounds, one local step each;
    long-run: 100 rounds of 8 local steps each, bf16 theta), at full size in the launch
    configuration the bench times, compared with the oracle after EVERY round on column ranges
    around every component edge plus interior ones: momentum, global models and restart points
    after many rounds, not only after the first two."""
    w = workloads.get(name)
    dev = torch.device("cuda:0")
    theta0 = workloads.theta0_torch(w, dev)
    if w.dtype == 1:
        theta0 = theta0.to(torch.bfloat16)
    pr = Pair(case_of(w), theta0, slices=_slices(w, width=width, interior=interior))
    try:
        for r in range(1, w.rounds + 1):
            pr.perturb(step=r * w.local_steps, lr=w.lr, sigma=w.sigma, nsteps=w.local_steps)
            pr.sync(r)
            pr.compare(f"{name} round {r}")
    finally:
        pr.close()


def test_every_point_of_the_granularity_sweep_at_full_size():
    """All 24 points of the granularity sweep (C in {4, 16, 64, 256} components with non-uniform
    sizes, 1 / 2 / 4 neighbours, eta 0.5 / 0.9; K = 8 replicas of the 279 M-parameter model) in the
    launch configuration the bench times: one synchronisation each after seeded local steps,
    compared with the oracle on column ranges around every component edge (at most 48 of them,
    evenly picked) plus interior ones."""
    dev = torch.device("cuda:0")
    for C, q, eta in workloads.SWEEP_POINTS:
        w = workloads.get("sweep", C=C, q=q, eta=eta)
        sl = workloads.edge_slices(w.offsets, 2048, count=48)
        g = np.random.Generator(np.random.PCG64(1000 + C + q))
        for _ in range(3):
            a = int(g.integers(0, w.N - 2048))
            if all(b <= a or a + 2048 <= c for c, b in sl):
                sl.append((a, a + 2048))
        pr = Pair(case_of(w), workloads.theta0_torch(w, dev), slices=sorted(sl))
        try:
            assert pr.g.launch_info()["grid"] == torch.cuda.get_device_properties(0).multi_processor_count
            pr.perturb(step=1, lr=w.lr, sigma=10 * w.sigma, nsteps=1)
            pr.check_neighbors(1)
            pr.sync(1)
            pr.compare(f"sweep C={C} q={q} eta={eta}")
        finally:
            pr.close()
            del pr
            torch.cuda.empty_cache()
