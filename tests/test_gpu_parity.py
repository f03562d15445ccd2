"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on the
same seeded inputs: neighbour tables bit-exact; theta, omega, Delta within 1e-7 + 1e-6 |ref|
after every step (and, by design, bit-equal)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_09010_b200 import binding, workloads
from harness import Case, Pair, case_of, random_theta0, to_numpy

pytestmark = pytest.mark.gpu


def run(case, theta0, rounds, lr=0.1, sigma=1e-2, nsteps=1, tuning=None, slices=None, masks=None,
        first_round=1, check_nbr=True):
    pr = Pair(case, theta0, slices=slices, tuning=tuning)
    try:
        pr.compare("after init")
        for r in range(first_round, first_round + rounds):
            if nsteps:
                pr.perturb(step=r * nsteps, lr=lr, sigma=sigma, nsteps=nsteps)
                pr.compare(f"after local steps of round {r}")
            if check_nbr:
                pr.check_neighbors(r)
            pr.sync(r, None if masks is None else masks[(r - first_round) % len(masks)])
            pr.compare(f"after round {r}")
    finally:
        pr.close()


# ------------------------------------------------------------------------------------------------
# the named small workloads
# ------------------------------------------------------------------------------------------------
def test_tiny_workload():
    w = workloads.get("tiny")
    pr = Pair(case_of(w), workloads.theta0_numpy(w))
    try:
        pr.add_drift(workloads.drift_numpy(w))
        pr.compare("after drift")
        for r in range(1, w.rounds + 1):
            pr.check_neighbors(r)
            pr.sync(r)
            pr.compare(f"round {r}")
    finally:
        pr.close()


def test_mid_workload_two_rounds():
    w = workloads.get("mid")
    run(case_of(w), workloads.theta0_numpy(w), rounds=2, lr=w.lr, sigma=w.sigma, nsteps=w.local_steps)


# ------------------------------------------------------------------------------------------------
# shapes: ragged edges, unaligned offsets, tiny components, many K / p / q
# ------------------------------------------------------------------------------------------------
RAGGED = [
    # K, offsets, p, q
    (4, (0, 1, 2, 3, 10, 4099, 4100, 9001), 1, 1),
    (8, (0, 7, 1031, 2055, 2056, 5000, 12345), 2, 2),
    (16, (0, 33467 * 3 + 1, 33467 * 5 + 2, 200003), 3, 2),
    (3, (0, 5, 777), 1, 2),
    (1, (0, 100, 3001), 0, 0),
    (2, (0, 4097), 1, 1),
    (5, (0, 2049, 6000), 2, 4),
    (17, (0, 999, 5003), 4, 3),
    (33, (0, 4096, 8200), 3, 5),
    (16, (0, 8, 16, 24, 1048, 9000), 8, 15),
    (6, (0, 3, 4, 8, 9, 31, 32, 33, 64, 1000), 3, 5),
]


@pytest.mark.parametrize("K,offsets,p,q", RAGGED)
@pytest.mark.parametrize("dtype", [0, 1])
def test_ragged_shapes(K, offsets, p, q, dtype):
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.875, zeta=1.0, dtype=dtype, seed=K * 31 + q)
    run(case, random_theta0(case.N, seed=K, dtype=dtype), rounds=3, sigma=5e-2)
    if K <= 128:                          # the default was the tensor-memory tile: also the shared-memory one
        run(case, random_theta0(case.N, seed=K, dtype=dtype), rounds=3, sigma=5e-2, tuning=dict(flags=8),
            check_nbr=False)


@pytest.mark.parametrize("tuning", [
    dict(consumer_threads=32, tile_elems=64, theta_stages=1, ring_slots=2),
    dict(consumer_threads=128, tile_elems=256, theta_stages=2, ring_slots=3),
    dict(consumer_threads=256, tile_elems=512, theta_stages=2, ring_slots=8),
    dict(consumer_threads=512, tile_elems=2048, theta_stages=1, ring_slots=4),
    dict(consumer_threads=96, tile_elems=200, theta_stages=2, ring_slots=5),
    dict(consumer_threads=992, tile_elems=768, theta_stages=2, ring_slots=2),
    dict(consumer_threads=256, tile_elems=4096, theta_stages=1, ring_slots=2),
    dict(consumer_threads=512, tile_elems=1024, theta_stages=2, ring_slots=4, flags=1),
])
@pytest.mark.parametrize("dtype", [0, 1])
def test_launch_shapes_agree(tuning, dtype):
    """Several tiles per CTA, a ragged last tile and every pipeline depth give the same bits."""
    K = 8
    offsets = (0, 100_003, 100_004, 350_001, 777_777)
    case = Case(K=K, offsets=offsets, p=2, q=2, eta=0.9, zeta=1.0, dtype=dtype, seed=5)
    run(case, random_theta0(case.N, seed=77, dtype=dtype), rounds=2, tuning=tuning, check_nbr=False)


def test_many_tiles_per_cta():
    """More tiles than resident CTAs: the persistent loop and stage re-use are exercised."""
    K, N = 4, 6_000_011
    case = Case(K=K, offsets=(0, 1_000_000, 1_000_001, 3_999_999, N), p=1, q=1, seed=9)
    run(case, random_theta0(N, seed=3), rounds=2,
        tuning=dict(consumer_threads=128, tile_elems=512, theta_stages=2, ring_slots=3))


# ------------------------------------------------------------------------------------------------
# modes, masks, periods, hyper-parameters
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [0, 1])
def test_gossip_ma_mode(dtype):
    case = Case(K=8, offsets=(0, 1001, 5000, 20011), p=2, q=2, dtype=dtype, seed=2,
                mode=binding.MODE_MA)
    run(case, random_theta0(case.N, seed=8, dtype=dtype), rounds=3, sigma=5e-2)


@pytest.mark.parametrize("K,p,q", [(16, 8, 15), (16, 3, 6), (8, 3, 6), (12, 4, 5), (7, 3, 6), (6, 3, 5)])
@pytest.mark.parametrize("dtype", [0, 1])
def test_gossip_ma_many_neighbours(K, p, q, dtype):
    """gossip-MA with many neighbours per draw (local-MA q = 2p, the full average q = K - 1)."""
    offsets = (0, 3, 1001, 5000, 5004, 70_011)
    case = Case(K=K, offsets=offsets, p=p, q=q, dtype=dtype, seed=3 * K + q, mode=binding.MODE_MA)
    run(case, random_theta0(case.N, seed=K + q, dtype=dtype), rounds=3, sigma=5e-2,
        masks=[None, [1, 1, 0, 1, 1], None])
    run(case, random_theta0(case.N, seed=K + q, dtype=dtype), rounds=2, sigma=5e-2,
        tuning=dict(tile_elems=256, theta_stages=2), check_nbr=False)


def test_component_masks_and_periods():
    offsets = (0, 3000, 3001, 9000, 20000, 40001)
    masks = [[1, 0, 1, 0, 1], [0, 1, 0, 0, 0], [0, 0, 0, 0, 0], [1, 1, 1, 1, 1]]
    case = Case(K=4, offsets=offsets, p=1, q=1, seed=4)
    run(case, random_theta0(case.N, seed=1), rounds=8, masks=masks, sigma=5e-2)
    case = Case(K=8, offsets=offsets, p=2, q=2, seed=4, periods=(2, 1, 4, 3, 2))
    run(case, random_theta0(case.N, seed=1), rounds=12, sigma=5e-2)


@pytest.mark.parametrize("eta,zeta,q", [(0.0, 1.0, 1), (0.5, 1.0, 3), (0.9, 0.75, 2), (0.99, 1.5, 4),
                                        (0.875, 1.0, 6)])
def test_hyper_parameters(eta, zeta, q):
    case = Case(K=16, offsets=(0, 5000, 10001, 30000), p=3, q=q, eta=eta, zeta=zeta, seed=q)
    run(case, random_theta0(case.N, seed=q), rounds=4, sigma=5e-2)


def test_column_range_reproduces_the_full_model():
    """A context bound to a column range (comp_base, elem_base) makes the choices and draws the
    noise the full model gives those columns."""
    w = workloads.get("tiny")
    theta0 = workloads.theta0_numpy(w)
    full = Pair(case_of(w), theta0)
    try:
        for r in (1, 2):
            full.perturb(r, 0.1, 0.05, 2)
            full.sync(r)
        full.compare("full")
        for rank in range(3):
            sh = workloads.shard_even(w.offsets, 3, rank)
            dev = torch.device("cuda:0")
            ld = workloads.padded_ld(sh.n)
            th = torch.zeros((w.K, ld), device=dev)
            om, de = torch.zeros_like(th), torch.zeros_like(th)
            g = binding.Gbmuf(th, om, de, K=w.K, N=sh.n, ld=ld, p=w.p, q=w.q, eta=w.eta,
                              zeta=w.zeta, seed=w.seed, comp_base=sh.comp_base, elem_base=sh.col0)
            g.set_partition(sh.offsets)
            g.init(torch.from_numpy(theta0[sh.col0:sh.col1].copy()).to(dev))
            for r in (1, 2):
                g.local_perturb(r, 0.1, 0.05, 2)
                g.sync_round(r)
            torch.cuda.synchronize()
            for part, whole in ((th, full.theta), (om, full.omega), (de, full.delta)):
                assert torch.equal(part[:, :sh.n], whole[:, sh.col0:sh.col1])
            g.destroy()
    finally:
        full.close()


def test_long_run_stays_bit_equal():
    """100 rounds with local steps in between (the shape of the long-run workload, small)."""
    case = Case(K=16, offsets=tuple(int(x) for x in np.linspace(0, 50_000, 9).astype(int)), p=3,
                q=3, eta=0.9, zeta=1.0, dtype=1, seed=4)
    pr = Pair(case, random_theta0(case.N, seed=4, dtype=1))
    try:
        for r in range(1, 101):
            pr.perturb(step=8 * r, lr=0.1, sigma=1e-2, nsteps=8)
            pr.sync(r)
            if r % 20 == 0:
                pr.compare(f"round {r}")
    finally:
        pr.close()


def test_final_average():
    for dtype in (0, 1):
        case = Case(K=8, offsets=(0, 4001, 10007), p=2, q=2, dtype=dtype, seed=3)
        pr = Pair(case, random_theta0(case.N, seed=5, dtype=dtype))
        try:
            pr.perturb(1, 1.0, 0.05)
            pr.sync(1)
            out = torch.zeros(case.N, dtype=pr.theta.dtype, device=pr.device)
            pr.g.final_average(out)
            torch.cuda.synchronize()
            want = oracle.final_average(pr.states[0])
            assert np.array_equal(to_numpy(out).view(np.uint8), want.view(np.uint8))
        finally:
            pr.close()


# ------------------------------------------------------------------------------------------------
# errors and state
# ------------------------------------------------------------------------------------------------
def test_call_order_and_argument_errors():
    dev = torch.device("cuda:0")
    th = torch.zeros((4, 128), device=dev)
    om, de = torch.zeros_like(th), torch.zeros_like(th)
    g = binding.Gbmuf(th, om, de, K=4, N=100, ld=128, p=1, q=1, eta=0.9, zeta=1.0)
    with pytest.raises(binding.GbmufError) as e:
        g.sync_round(1)
    assert e.value.status == binding.ERR_BAD_STATE
    for bad in ([0, 50], [1, 100], [0, 50, 50, 100], [0, 60, 40, 100]):
        with pytest.raises(binding.GbmufError) as e:
            g.set_partition(bad)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.GbmufError):
        g.set_partition([0, 50, 100], periods=[1, 0])
    g.set_partition([0, 50, 100])
    with pytest.raises(binding.GbmufError):
        g.set_tuning(consumer_threads=100)
    with pytest.raises(binding.GbmufError):
        g.set_tuning(tile_elems=100)
    with pytest.raises(binding.GbmufError):
        g.set_tuning(tile_elems=1000)
    with pytest.raises(binding.GbmufError):
        g.local_perturb(2 ** 32, 0.1, 0.1)
    info = g.launch_info()
    assert info["tiles"] == 2 and info["grid"] == 2 and info["block"] % 32 == 0
    g.sync_round(1)
    assert g.device_status() == 0
    g.destroy()
    g.destroy()                                          # idempotent
    with pytest.raises(binding.GbmufError) as e:         # K too large for one staged tile
        big = torch.zeros((300, 32), device=dev)
        binding.Gbmuf(big, big, big, K=300, N=32, ld=32, p=1, q=1, eta=0.9, zeta=1.0)
    assert e.value.status == binding.ERR_UNSUPPORTED


def test_padding_columns_are_never_written():
    K, N, ld = 4, 1000, 1056
    dev = torch.device("cuda:0")
    th = torch.full((K, ld), 7.0, device=dev)
    om, de = torch.full_like(th, 8.0), torch.full_like(th, 9.0)
    g = binding.Gbmuf(th, om, de, K=K, N=N, ld=ld, p=1, q=1, eta=0.9, zeta=1.0)
    g.set_partition([0, 333, N])
    g.init(torch.randn(N, device=dev))
    g.local_perturb(1, 0.1, 0.1, 2)
    g.sync_round(1)
    torch.cuda.synchronize()
    assert bool((th[:, N:] == 7.0).all()) and bool((om[:, N:] == 8.0).all())
    assert bool((de[:, N:] == 9.0).all())
    g.destroy()


# ------------------------------------------------------------------------------------------------
# resume, graph replay, random shapes
# ------------------------------------------------------------------------------------------------
def test_resume_from_saved_state_is_bit_identical():
    """The state of a run is (theta, omega, Delta, round number, seed, partition): the draws and the
    noise are counter-based, so R rounds + save / restore + R rounds equals 2R rounds."""
    w = workloads.get("tiny")
    dev = torch.device("cuda:0")
    kw = dict(K=w.K, N=w.N, ld=w.ld, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta, seed=w.seed)

    def fresh():
        th = torch.zeros((w.K, w.ld), device=dev)
        return th, torch.zeros_like(th), torch.zeros_like(th)

    def advance(g, first, count):
        for r in range(first, first + count):
            g.local_perturb(2 * r, 0.1, 0.05, 2)
            g.sync_round(r)

    a = fresh()
    ga = binding.Gbmuf(*a, **kw)
    ga.set_partition(w.offsets)
    ga.init(torch.from_numpy(workloads.theta0_numpy(w)).to(dev))
    advance(ga, 1, 3)
    torch.cuda.synchronize()
    saved = [t.cpu().clone() for t in a]                 # "checkpoint"
    advance(ga, 4, 3)
    b = tuple(t.to(dev) for t in saved)                  # "restore" into other buffers, new context
    gb = binding.Gbmuf(*b, **kw)
    gb.set_partition(w.offsets)
    advance(gb, 4, 3)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    ga.destroy()
    gb.destroy()


def test_rounds_replayed_from_a_cuda_graph():
    """Rounds without a host mask only launch kernels, so a sequence of them can be captured once
    and replayed (the launch-bound tiny workload is where that pays)."""
    w = workloads.get("tiny")
    pr = Pair(case_of(w), workloads.theta0_numpy(w))
    try:
        pr.add_drift(workloads.drift_numpy(w))
        pr.sync(1)                                      # first call outside capture
        pr.compare("before capture")
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            graph.capture_begin()
            for r in (2, 3, 4):
                pr.g.local_perturb(r, 0.1, 0.02, 1, stream=side)
                pr.g.sync_round(r, stream=side)
            graph.capture_end()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        for r in (2, 3, 4):                             # the oracle replays the same calls once
            for sh, st in zip(pr.shards, pr.states):
                oracle.local_perturb(st, w.seed, r, 0.1, 0.02, 1, elem_base=sh.col0)
                nbr = oracle.sample_neighbors(w.seed, r, w.K, sh.m, w.p, w.q, comp_base=sh.comp_base)
                oracle.sync_round(st, sh.offsets, nbr, w.eta, w.zeta)
        pr.compare("after graph replay")
    finally:
        pr.close()


def test_page_locked_mask_may_be_reused_at_once():
    """A comp_mask in page-locked memory, overwritten as soon as gbmuf_sync_round returns while the
    stream is still busy with earlier work: the round must use the mask as it was at the call."""
    offsets = (0, 3000, 3001, 9000, 20000, 40001)
    case = Case(K=8, offsets=offsets, p=2, q=2, seed=12)
    pr = Pair(case, random_theta0(case.N, seed=4))
    try:
        pr.perturb(1, 0.1, 0.05)
        mask_pin = torch.tensor([1, 0, 1, 0, 1], dtype=torch.uint8).pin_memory()
        busy = torch.empty(1 << 28, device=pr.device)
        for _ in range(20):
            busy.add_(1.0)
        pr.g.sync_round(1, mask_pin.numpy())
        mask_pin.fill_(1)                                # the caller's array changes at once
        for sh, st in zip(pr.shards, pr.states):
            nbr = oracle.sample_neighbors(case.seed, 1, case.K, sh.m, case.p, case.q)
            oracle.sync_round(st, sh.offsets, nbr, case.eta, case.zeta, sync=[1, 0, 1, 0, 1])
        pr.compare("pinned mask")
    finally:
        pr.close()


def test_mask_is_refused_inside_a_stream_capture():
    w = workloads.get("tiny")
    pr = Pair(case_of(w), workloads.theta0_numpy(w))
    try:
        pr.sync(1)
        pr.compare("before capture")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            graph.capture_begin()
            with pytest.raises(binding.GbmufError) as e:
                pr.g.sync_round(2, [1, 1, 0, 1], stream=side)
            pr.g.sync_round(2, stream=side)               # without a mask the round is recorded
            graph.capture_end()
        assert e.value.status == binding.ERR_BAD_STATE
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        for sh, st in zip(pr.shards, pr.states):
            nbr = oracle.sample_neighbors(w.seed, 2, w.K, sh.m, w.p, w.q)
            oracle.sync_round(st, sh.offsets, nbr, w.eta, w.zeta)
        pr.compare("after replay")
    finally:
        pr.close()


def test_random_shapes_property():
    """Random K, p, q, component edges (unaligned, tiny and large), eta, zeta, dtype, mode, and
    launch shapes of both variants of the fused kernel (several tiles per CTA included)."""
    import os
    from hypothesis import given, settings, strategies as st_, HealthCheck

    @settings(max_examples=int(os.environ.get("GBMUF_PROPERTY_EXAMPLES", "100")), deadline=None,
              derandomize=True, suppress_health_check=list(HealthCheck))
    @given(st_.data())
    def inner(data):
        K = data.draw(st_.one_of(st_.integers(1, 24), st_.sampled_from([33, 48, 70])))
        p = data.draw(st_.integers(0, 6))
        c = min(2 * p, K - 1)
        q = data.draw(st_.integers(0, c))
        m = data.draw(st_.integers(1, 6))
        N = data.draw(st_.sampled_from([30_000, 30_000, 300_000]))
        N = data.draw(st_.integers(m, N))
        cuts = sorted(data.draw(st_.sets(st_.integers(1, N - 1), min_size=m - 1, max_size=m - 1))) if m > 1 else []
        offsets = tuple([0] + cuts + [N])
        eta = data.draw(st_.sampled_from([0.0, 0.5, 0.875, 0.9, 0.99]))
        zeta = data.draw(st_.sampled_from([0.5, 1.0, 1.25]))
        dtype = data.draw(st_.integers(0, 1))
        mode = data.draw(st_.sampled_from([0, 0, 0, 1]))
        case = Case(K=K, offsets=offsets, p=p, q=q, eta=eta, zeta=zeta, dtype=dtype,
                    seed=data.draw(st_.integers(0, 2 ** 63)), mode=mode)
        shape = data.draw(st_.sampled_from(["default", "shared", "shared_custom", "tensor_custom", "window"]))
        tuning = None
        if shape == "shared":
            tuning = dict(flags=8)
        elif shape == "shared_custom":
            tuning = dict(tile_elems=data.draw(st_.sampled_from([64, 256, 512])),
                          consumer_threads=data.draw(st_.sampled_from([64, 256])))
        elif shape == "tensor_custom" and mode == 0:
            tuning = dict(tile_elems=data.draw(st_.sampled_from([512, 1024])),
                          ring_slots=data.draw(st_.sampled_from([0, 2, 3, 4, 6])),
                          flags=data.draw(st_.sampled_from([2, 6])))
        elif shape == "window" and mode == 0 and 2 * p + (2 if dtype == 0 else 4) < K:
            tuning = dict(tile_elems=data.draw(st_.sampled_from([512, 1024])),
                          ring_slots=data.draw(st_.sampled_from([0, 2, 3, 4, 6])),
                          flags=data.draw(st_.sampled_from([16, 18, 22, 80, 86])))
        run(case, random_theta0(N, seed=K + N, dtype=dtype), rounds=2, sigma=5e-2, tuning=tuning)

    inner()


# ------------------------------------------------------------------------------------------------
# extremes: many components, many workers, degenerate sizes
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,N,seed", [(300, 40_000, 1), (700, 9_000, 2), (3000, 100_000, 3)])
def test_many_components(m, N, seed):
    """More components than one pass of the work-list scan (256) handles, with many one- and
    two-element components and a mask that leaves runs of them out."""
    g = np.random.Generator(np.random.PCG64(seed))
    cuts = np.sort(g.choice(np.arange(1, N), size=m - 1, replace=False))
    offsets = tuple([0] + [int(x) for x in cuts] + [N])
    masks = [None, [int(x) for x in (g.random(m) < 0.6)], [1 if (i // 37) % 2 else 0 for i in range(m)]]
    case = Case(K=4, offsets=offsets, p=1, q=1, eta=0.9, zeta=1.0, seed=seed)
    run(case, random_theta0(N, seed=seed), rounds=3, masks=masks, sigma=5e-2, check_nbr=(m <= 700))


@pytest.mark.parametrize("K,p,q,dtype", [(64, 5, 7, 0), (128, 6, 3, 1), (256, 7, 2, 0), (200, 32, 64, 0)])
def test_many_workers(K, p, q, dtype):
    offsets = (0, 1001, 1002, 6007)
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.875, zeta=1.0, dtype=dtype, seed=K)
    run(case, random_theta0(offsets[-1], seed=K, dtype=dtype), rounds=2, sigma=5e-2)


@pytest.mark.parametrize("K,N,p,q", [(1, 1, 0, 0), (2, 1, 1, 1), (3, 7, 1, 2), (16, 8, 3, 2), (5, 33, 2, 4)])
def test_degenerate_sizes(K, N, p, q):
    for dtype in (0, 1):
        case = Case(K=K, offsets=(0, N), p=p, q=q, dtype=dtype, seed=N)
        run(case, random_theta0(N, seed=N, dtype=dtype), rounds=3, sigma=5e-2)
    if N >= 7:
        case = Case(K=K, offsets=tuple(range(N + 1)), p=p, q=q, seed=N)     # every element its own component
        run(case, random_theta0(N, seed=N), rounds=2, sigma=5e-2)


def test_expired_wait_is_reported_not_hung():
    """Failure reporting without a fault: a wait on a barrier that nothing signals expires after
    its two-second limit, the kernel returns, the status word says TIMEOUT once, and the context
    goes on working."""
    w = workloads.get("tiny")
    pr = Pair(case_of(w), workloads.theta0_numpy(w))
    try:
        pr.perturb(1, 0.1, 0.05)
        sec = pr.g.selftest_wait_timeout()
        assert 1.5 < sec < 10.0, sec
        assert pr.g.device_status() == binding.ERR_TIMEOUT
        assert pr.g.device_status() == 0                   # reading cleared it
        pr.sync(1)
        pr.compare("round after the expired wait")
    finally:
        pr.close()


@pytest.mark.parametrize("mode", [binding.MODE_BMUF, binding.MODE_MA])
@pytest.mark.parametrize("dtype", [0, 1])
def test_special_values_propagate_identically(dtype, mode):
    """Denormals (no flush-to-zero), signed zeros, infinities, NaN and extreme magnitudes go
    through the round as IEEE arithmetic dictates: bit-equal with the oracle wherever the result
    is not NaN, NaN exactly where the oracle has NaN."""
    K, N = 8, 6000
    offsets = (0, 1000, 1001, 4003, N)
    g = np.random.Generator(np.random.PCG64(12))
    theta0 = (g.standard_normal(N) * 0.1).astype(np.float32)
    specials = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, 3e-39, 1.1754944e-38, 3.4e38, -3.4e38,
                         np.inf, -np.inf, np.nan, 1e30, -1e-30, 65504.0, 1.0], dtype=np.float32)
    theta0[g.choice(N, size=400, replace=False)] = g.choice(specials, size=400)
    theta0[1001:1200] = (g.integers(-2000, 2000, size=199) * 1e-42).astype(np.float32)   # a denormal stretch
    if dtype == 1:
        theta0 = oracle.f32_to_bf16(theta0)
    case = Case(K=K, offsets=offsets, p=2, q=2, eta=0.9, zeta=1.0, dtype=dtype, seed=3, mode=mode)
    pr = Pair(case, theta0)
    try:
        drift = (g.standard_normal((K, N)) * 0.05).astype(np.float32)
        drift[g.random((K, N)) < 0.02] = np.float32(1e-42)           # denormal nudges
        drift[:, 1001:1200] = (g.integers(-500, 500, size=(K, 199)) * 1e-43).astype(np.float32)
        saw_denormal = False
        if dtype == 0:
            pr.add_drift(drift)
        else:
            pr.perturb(1, 1.0, 0.05)
        for r in (1, 2, 3):
            pr.sync(r)
            torch.cuda.synchronize()
            st = pr.states[0]
            for name, got, ref in (("omega", to_numpy(pr.omega), st.omega), ("delta", to_numpy(pr.delta), st.delta),
                                   ("theta", to_numpy(pr.theta), st.theta)):
                if ref.dtype == np.uint16:
                    gf, rf = oracle.bf16_to_f32(got), oracle.bf16_to_f32(ref)
                else:
                    gf, rf = got, ref
                nan_g, nan_r = np.isnan(gf), np.isnan(rf)
                assert np.array_equal(nan_g, nan_r), f"{name}: NaN pattern differs in round {r}"
                assert np.array_equal(got[~nan_r], ref[~nan_r]) and \
                    np.array_equal(np.signbit(gf[~nan_r]), np.signbit(rf[~nan_r])), f"{name} round {r}"
            assert pr.g.device_status() == 0
            d = st.delta[np.isfinite(st.delta)]
            saw_denormal = saw_denormal or bool((np.abs(d[d != 0]) < 1.1754944e-38).any())
        assert np.isnan(st.theta if dtype == 0 else oracle.bf16_to_f32(st.theta)).any()
        if mode == binding.MODE_BMUF:
            assert saw_denormal or dtype == 1, "the test never produced a denormal Delta"
        elif dtype == 0:
            t = st.theta[np.isfinite(st.theta)]
            assert (np.abs(t[t != 0]) < 1.1754944e-38).any(), "no denormal average was produced"
    finally:
        pr.close()


@pytest.mark.parametrize("flags", [2, 6])          # 6: outputs leave through bulk stores
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("K,p,q,tile,ring", [(16, 3, 2, 0, 0), (8, 2, 2, 2048, 4), (5, 2, 4, 1024, 3),
                                              (4, 1, 1, 512, 8), (16, 3, 6, 1024, 2), (32, 4, 3, 2048, 0)])
def test_tensor_memory_variant(K, p, q, tile, ring, dtype, flags):
    """The variant that parks the theta tile in tensor memory gives the same bits: several tiles
    per CTA, ragged component edges, masks, odd K (a partly filled last theta item)."""
    offsets = (0, 100_003, 100_004, 350_001, 777_777)
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.875, zeta=1.0, dtype=dtype, seed=K + q)
    masks = [None, [1, 0, 1, 1], None]
    run(case, random_theta0(case.N, seed=K, dtype=dtype), rounds=3, sigma=5e-2, masks=masks,
        tuning=dict(tile_elems=tile, ring_slots=ring, flags=flags), check_nbr=False)


@pytest.mark.parametrize("flags", [16, 18, 80])    # 18: stores from registers; 80: every row read once
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("K,p,q,tile,ring", [(16, 3, 2, 0, 0), (9, 2, 4, 1024, 3), (12, 1, 2, 512, 8),
                                              (24, 4, 8, 2048, 0), (64, 5, 7, 512, 4), (7, 1, 1, 512, 2),
                                              (40, 0, 0, 1024, 4), (256, 7, 3, 512, 0), (23, 8, 16, 512, 0)])
def test_ring_window_variant(K, p, q, tile, ring, dtype, flags):
    """Tensor-memory tile that holds only a window of rows along the ring (plus the first p rows
    kept for the last workers) gives the same bits as the oracle: wrap-around at both ends of the
    worker range, several tiles per CTA, ragged component edges, masks, partly filled load items."""
    if 2 * p + (2 if dtype == 0 else 4) >= K:
        pytest.skip("no window for this shape: 2p + rows per load item must be below K")
    offsets = ((0, 100_003, 100_004, 350_001, 777_777) if K <= 16 else
               (0, 40_003, 40_004, 140_001, 300_001) if K <= 64 else (0, 10_003, 10_004, 35_001, 77_777))
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.875, zeta=1.0, dtype=dtype, seed=K + q)
    masks = [None, [1, 0, 1, 1], None]
    run(case, random_theta0(case.N, seed=K, dtype=dtype), rounds=3, sigma=5e-2, masks=masks,
        tuning=dict(tile_elems=tile, ring_slots=ring, flags=flags), check_nbr=False)


@pytest.mark.parametrize("K,p,q,dtype", [(64, 5, 3, 0), (64, 5, 3, 1), (24, 3, 2, 0), (130, 6, 2, 1)])
def test_ring_window_default_shape(K, p, q, dtype):
    """The launch shape the library picks by itself for many workers (window, widest tile, deep
    ring), with more tiles than CTAs so that every CTA goes round its ring several times."""
    N = 148 * 4096 * 2 + 12_345 if K <= 64 else 148 * 5120 + 777
    offsets = (0, N // 3 + 1, N // 3 + 2, N)
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.9, zeta=1.0, dtype=dtype, seed=K + p)
    run(case, random_theta0(N, seed=K, dtype=dtype), rounds=2, sigma=5e-2, check_nbr=False)


@pytest.mark.parametrize("K,p,q,dtype,expect", [(64, 5, 7, 0, "tmem-window"), (128, 6, 3, 1, "tmem-window"),
                                                  (256, 7, 2, 0, "tmem-window"), (16, 3, 2, 0, "tmem"),
                                                  (32, 15, 30, 0, "tmem"), (200, 32, 64, 0, "tmem-window")])
def test_which_rows_are_resident_follows_the_ring(K, p, q, dtype, expect):
    """The window is taken by itself exactly when it buys a wider tile; flags bit 5 switches it
    off; forcing it where the ring is too dense for a window is refused."""
    dev = torch.device("cuda:0")
    th = torch.zeros((K, 8192), device=dev, dtype=torch.float32 if dtype == 0 else torch.bfloat16)
    om = torch.zeros((K, 8192), device=dev)
    g = binding.Gbmuf(th, om, om.clone(), K=K, N=8192, ld=8192, p=p, q=q, eta=0.9, zeta=1.0, theta_dtype=dtype)
    try:
        g.set_partition([0, 8192])
        info = g.launch_info()
        assert info["variant"] == expect, info
        rows_per_item = 2 if dtype == 0 else 4
        if expect == "tmem-window":
            assert -info["stages"] in (3 * p + rows_per_item, 4 * p + rows_per_item)   # last p rows read twice / kept
            assert info["tile_elems"] >= (2048 if p <= 7 else 512)
            g.set_tuning(flags=32)
            assert g.launch_info()["variant"] in ("tmem", "smem")
        elif 2 * p + rows_per_item >= K:
            with pytest.raises(binding.GbmufError) as e:
                g.set_tuning(flags=16)
            assert e.value.status == binding.ERR_UNSUPPORTED
        else:                                      # possible, but buys nothing at this K: only on request
            g.set_tuning(flags=16)
            assert g.launch_info()["variant"] == "tmem-window"
    finally:
        g.destroy()


@pytest.mark.parametrize("K,p,q,dtype,tuning,expect", [
    (64, 5, 3, 0, dict(flags=16), "smem-window"), (64, 5, 3, 1, dict(flags=16), "smem-window"),
    (130, 6, 2, 1, dict(flags=16), "smem-window"), (256, 7, 2, 0, None, "smem-window"),
    (200, 6, 6, 0, None, "smem-window"), (200, 32, 64, 0, None, "smem"), (256, 7, 2, 1, None, "smem"),
    (9, 2, 4, 0, dict(flags=16), "smem-window"), (12, 1, 2, 1, dict(flags=16, tile_elems=512), "smem-window"),
    (6, 2, 3, 0, dict(flags=16, tile_elems=128), "smem-window"), (64, 5, 10, 0, dict(flags=16, tile_elems=256), "smem-window"),
    (64, 5, 3, 0, dict(flags=32), "smem"), (20, 0, 0, 0, dict(flags=16), "smem-window")])
def test_gossip_ma_ring_window(K, p, q, dtype, tuning, expect):
    """gossip-MA with many workers streams a window of rows along the ring through shared memory
    (fp32 theta from 192 workers on, or on request): several tiles per CTA, ragged component edges, kept first
    rows, last rows read twice, both theta types, and the settings where it is not taken."""
    offsets = (0, 5, 4099, 4100, 30_001, 70_003)
    case = Case(K=K, offsets=offsets, p=p, q=q, eta=0.9, zeta=1.0, dtype=dtype, seed=K + q,
                mode=binding.MODE_MA)
    pr = Pair(case, random_theta0(case.N, seed=K, dtype=dtype), tuning=tuning)
    try:
        assert pr.g.launch_info()["variant"] == expect
        for r in (1, 2, 3):
            pr.perturb(step=r, lr=0.1, sigma=5e-2)
            mask = None if r != 2 else [1, 0, 1, 1, 0]
            pr.sync(r, mask)
            pr.compare(f"round {r}")
    finally:
        pr.close()


def test_averaging_division_equals_the_ieee_division_for_every_dividend():
    """The kernels divide the gossip sum by q+1 through a multiply and a residual correction;
    for every divisor they can meet (q+1 <= 65) and some beyond, all 2^32 dividends -- zeros,
    subnormals, infinities and NaNs included -- give the bits of the plain division."""
    dev = torch.device("cuda:0")
    th = torch.zeros((2, 1024), device=dev)
    g = binding.Gbmuf(th, th.clone(), th.clone(), K=2, N=1024, ld=1024, p=1, q=1, eta=0.9, zeta=1.0)
    try:
        for b in list(range(2, 66)) + [96, 100, 127, 129, 255, 256]:
            bad, first = g.selftest_divide(b)
            assert bad == 0, f"divisor {b}: {bad} dividends differ, first pattern {first:#010x}"
        with pytest.raises(binding.GbmufError):
            g.selftest_divide(1)
    finally:
        g.destroy()


def test_tensor_memory_variant_is_refused_where_it_does_not_apply():
    dev = torch.device("cuda:0")
    th = torch.zeros((130, 1024), device=dev)
    g = binding.Gbmuf(th, th.clone(), th.clone(), K=130, N=1024, ld=1024, p=1, q=1, eta=0.9, zeta=1.0)
    with pytest.raises(binding.GbmufError) as e:
        g.set_tuning(flags=2 | 32)                 # all rows resident: more workers than tensor memory has room for
    assert e.value.status == binding.ERR_UNSUPPORTED
    g.destroy()
    th = torch.zeros((8, 1024), device=dev)
    g = binding.Gbmuf(th, th.clone(), th.clone(), K=8, N=1024, ld=1024, p=1, q=1, eta=0.9, zeta=1.0,
                      mode=binding.MODE_MA)
    with pytest.raises(binding.GbmufError):
        g.set_tuning(flags=6)                      # gossip-MA
    g.set_tuning(flags=16)                         # gossip-MA has a ring window of its own (shared memory)
    g.set_partition([0, 1024])
    assert g.launch_info()["variant"] == "smem-window"
    g.destroy()
    th = torch.zeros((3, 1024), device=dev)
    g = binding.Gbmuf(th, th.clone(), th.clone(), K=3, N=1024, ld=1024, p=1, q=1, eta=0.9, zeta=1.0,
                      mode=binding.MODE_MA)
    with pytest.raises(binding.GbmufError) as e:
        g.set_tuning(flags=16)                     # too few workers for a window: K < 2p + 2
    assert e.value.status == binding.ERR_UNSUPPORTED
    g.destroy()
    th = torch.zeros((24, 1024), device=dev)
    g = binding.Gbmuf(th, th.clone(), th.clone(), K=24, N=1024, ld=1024, p=3, q=2, eta=0.9, zeta=1.0)
    for flags in (16 | 32, 8 | 16, 8 | 2, 4, 128):     # force and forbid at once; two variants at once; out of range
        with pytest.raises(binding.GbmufError) as e:
            g.set_tuning(flags=flags)
        assert e.value.status == binding.ERR_INVALID_ARG, flags
    g.set_tuning(flags=64)                         # "every row once" alone only shapes a window that is taken anyway
    g.set_partition([0, 1024])
    assert g.launch_info()["variant"] == "tmem-window"
    g.destroy()
