"""The allocation-free entry point gives the results of the ordinary context path.

Some users of this library cannot allocate device memory at the moment they synchronise: their
framework's memory pool already owns the GPU, or they are a plug-in that is handed buffers and a
stream and must not call the allocator.  For them ``gbmuf_sync_round_noalloc`` keeps all of the
library's own tables in one fixed array of the loaded library.  This file checks, through the C
ABI, that two rounds in a row through that entry point leave theta, omega and Delta exactly as
two rounds through a context do, and that it really refuses what does not fit its array.

(Collected last on purpose: a run that stops at the first failure has then already run the rest.)
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_09010_b200 import binding
from harness import ATOL, RTOL, from_numpy, random_theta0, to_numpy

pytestmark = pytest.mark.gpu


def _state(K, N, ld, dtype, seed, dev):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    tdt = torch.float32 if dtype == 0 else torch.bfloat16
    theta = (torch.randn((K, ld), generator=g) * 0.1).to(tdt).to(dev)
    omega = (torch.randn((K, ld), generator=g) * 0.1).to(dev)
    delta = (torch.randn((K, ld), generator=g) * 0.01).to(dev)
    return theta, omega, delta


@pytest.mark.parametrize("dtype", [0, 1])
def test_two_rounds_match_the_context_path(dtype):
    dev = torch.device("cuda:0")
    K, p, q, eta, zeta, seed = 8, 2, 2, 0.875, 1.0, 11
    offsets = (0, 4099, 4100, 150_001, 400_003)
    N = offsets[-1]
    ld = (N + 31) // 32 * 32
    kw = dict(K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=zeta, seed=seed, theta_dtype=dtype)

    ref = _state(K, N, ld, dtype, 5, dev)
    got = tuple(t.clone() for t in ref)

    g = binding.Gbmuf(*ref, **kw)
    g.set_partition(offsets)
    masks = [None, [1, 0, 1, 1]]
    for rnd, mask in zip((1, 2), masks):
        g.sync_round(rnd, mask)
    torch.cuda.synchronize()
    assert g.device_status() == 0
    g.destroy()

    free_before = None
    for rnd, mask in zip((1, 2), masks):
        status = binding.sync_round_noalloc(*got, offsets, rnd, comp_mask=mask, want_status=True, **kw)
        assert status == 0
        free_now = torch.cuda.mem_get_info()[0]
        if free_before is not None:            # the second call must not have taken device memory
            assert free_now >= free_before
        free_before = free_now

    for name, a, b in zip(("theta", "omega", "delta"), got, ref):
        a32, b32 = a.float().cpu().numpy(), b.float().cpu().numpy()
        tol = ATOL + (1e-2 if (dtype == 1 and name == "theta") else RTOL) * np.abs(b32)
        assert np.all(np.abs(a32 - b32) <= tol), f"{name} outside tolerance"
        assert torch.equal(a, b), f"{name}: the two entry points should agree bit for bit"


def test_sizes_beyond_the_fixed_array_are_refused():
    dev = torch.device("cuda:0")
    K, N, ld = 4, 4096, 4096
    th = torch.zeros((K, ld), device=dev)
    om, de = torch.zeros_like(th), torch.zeros_like(th)
    kw = dict(K=K, N=N, ld=ld, p=1, q=1, eta=0.9, zeta=1.0)
    too_many = list(range(0, 1026)) + [N]                     # 1026 components
    with pytest.raises(binding.GbmufError) as e:
        binding.sync_round_noalloc(th, om, de, too_many, 1, **kw)
    assert e.value.status == binding.ERR_UNSUPPORTED and "1024" in str(e.value)
    K2 = 128
    th2 = torch.zeros((K2, ld), device=dev)
    kw2 = dict(K=K2, N=N, ld=ld, p=3, q=6, eta=0.9, zeta=1.0)
    offs = list(range(0, 4 * 100, 4)) + [N]                   # 100 components * 128 * 6 > 65536
    with pytest.raises(binding.GbmufError) as e:
        binding.sync_round_noalloc(th2, th2.clone(), th2.clone(), offs, 1, **kw2)
    assert e.value.status == binding.ERR_UNSUPPORTED and "65536" in str(e.value)
    with pytest.raises(binding.GbmufError) as e:
        binding.sync_round_noalloc(th, om, de, [0, 10, 5, N], 1, **kw)
    assert e.value.status == binding.ERR_INVALID_ARG
    assert not th.any() and not om.any() and not de.any()     # refused calls touch nothing


def _oracle_state(K, N, ld, dtype, eta, seed):
    """A consistent mid-training state: theta, omega, Delta arbitrary, and the block-start value
    the oracle stores equal to what the kernels recompute, store(omega + eta * Delta)."""
    st = oracle.init(random_theta0(N, seed=seed, dtype=dtype), K, ld=ld, dtype=dtype)
    oracle.local_perturb(st, seed, 0, 1.0, 0.05)
    g = np.random.Generator(np.random.PCG64(seed + 1))
    st.omega[:, :N] += (g.standard_normal((K, N)) * 0.01).astype(np.float32)
    st.delta[:, :N] = (g.standard_normal((K, N)) * 0.01).astype(np.float32)
    r32 = st.omega + np.float32(eta) * st.delta
    st.rst[:] = oracle.f32_to_bf16(r32) if dtype == 1 else r32
    return st


def _assert_equals_oracle(got, st, dtype, what):
    th, om, de = got
    assert np.array_equal(to_numpy(th).view(np.uint8), st.theta.view(np.uint8)), f"{what}: theta"
    assert np.array_equal(to_numpy(om).view(np.uint32), st.omega.view(np.uint32)), f"{what}: omega"
    assert np.array_equal(to_numpy(de).view(np.uint32), st.delta.view(np.uint32)), f"{what}: delta"
    tol = ATOL + RTOL * np.abs(st.omega)
    assert np.all(np.abs(to_numpy(om) - st.omega) <= tol), f"{what}: omega outside tolerance"


@pytest.mark.parametrize("dtype,mode,K,p,q", [(0, 0, 8, 2, 2), (1, 0, 8, 2, 3), (0, 1, 8, 2, 2),
                                              (1, 1, 6, 2, 1), (0, 0, 5, 2, 0), (0, 0, 40, 4, 3)])
def test_against_the_oracle_directly(dtype, mode, K, p, q):
    """The entry point element by element against the CPU oracle (not via the context path):
    gossip-BMUF and gossip-MA (the latter takes the shared-memory tile, whose tensor map is built
    for the call), bf16 theta, q = 0, and a worker count that takes the ring-window launch.  The
    calls share one array, so a sequence with a large partition first, then a small one, then a
    masked round checks that nothing stale from an earlier call is read."""
    dev = torch.device("cuda:0")
    eta, zeta, seed = 0.875, 1.0, 23
    big = tuple(range(0, 8 * 400, 8)) + (20_011,)           # 400 small components and a large one
    small = (0, 4099, 4100, 20_011)
    N = big[-1]
    ld = (N + 31) // 32 * 32
    st = _oracle_state(K, N, ld, dtype, eta, seed)
    got = (from_numpy(st.theta, dtype, dev), from_numpy(st.omega, 0, dev), from_numpy(st.delta, 0, dev))
    kw = dict(K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=zeta, seed=seed, theta_dtype=dtype, mode=mode)
    seq = [(1, big, None), (2, small, None), (3, small, [1, 0, 1]), (4, big, [i % 3 != 0 for i in range(len(big) - 1)])]
    for rnd, offsets, mask in seq:
        status = binding.sync_round_noalloc(*got, offsets, rnd, comp_mask=mask, want_status=True, **kw)
        assert status == 0
        nbr = oracle.sample_neighbors(seed, rnd, K, len(offsets) - 1, p, q)
        oracle.sync_round(st, offsets, nbr, eta, zeta, mode=mode, sync=mask)
        _assert_equals_oracle(got, st, dtype, f"round {rnd}")


def test_page_locked_tables_may_be_reused_at_once():
    """offsets and comp_mask in page-locked memory, scribbled over as soon as the call returns:
    the library must have taken its own copy before the (asynchronous) upload."""
    dev = torch.device("cuda:0")
    K, p, q, eta, zeta, seed, dtype = 8, 2, 2, 0.9, 1.0, 31, 0
    offsets = (0, 1001, 5000, 5001, 60_003)
    N = offsets[-1]
    ld = (N + 31) // 32 * 32
    st = _oracle_state(K, N, ld, dtype, eta, seed)
    got = (from_numpy(st.theta, dtype, dev), from_numpy(st.omega, 0, dev), from_numpy(st.delta, 0, dev))
    off_pin = torch.tensor(offsets, dtype=torch.int64).pin_memory()
    mask_pin = torch.tensor([1, 0, 1, 1], dtype=torch.uint8).pin_memory()
    kw = dict(K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=zeta, seed=seed)
    side = torch.cuda.Stream()
    busy = torch.empty(1 << 28, device=dev)
    with torch.cuda.stream(side):
        for _ in range(20):                                # keep the stream busy so that the upload is queued
            busy.add_(1.0)
        binding.sync_round_noalloc(*got, off_pin.numpy(), 1, comp_mask=mask_pin.numpy(), stream=side, **kw)
        off_pin.fill_(7)                                   # the caller reuses its tables at once
        mask_pin.fill_(1)
    side.synchronize()
    nbr = oracle.sample_neighbors(seed, 1, K, len(offsets) - 1, p, q)
    oracle.sync_round(st, offsets, nbr, eta, zeta, sync=[1, 0, 1, 1])
    _assert_equals_oracle(got, st, dtype, "pinned tables")


def test_refused_inside_a_stream_capture():
    """The call uploads host tables, so it cannot be part of a CUDA graph: inside a capture it
    is refused and nothing is recorded or changed."""
    dev = torch.device("cuda:0")
    K, N, ld = 4, 4096, 4096
    th = torch.randn((K, ld), device=dev)
    om, de = th.clone(), torch.zeros_like(th)
    before = th.clone()
    kw = dict(K=K, N=N, ld=ld, p=1, q=1, eta=0.9, zeta=1.0)
    binding.sync_round_noalloc(th.clone(), om.clone(), de.clone(), [0, 100, N], 1, **kw)   # first use: outside
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        with pytest.raises(binding.GbmufError) as e:
            binding.sync_round_noalloc(th, om, de, [0, 100, N], 2, stream=side, **kw)
        graph.capture_end()
    assert e.value.status == binding.ERR_BAD_STATE and "capture" in str(e.value)
    torch.cuda.synchronize()
    assert torch.equal(th, before)
