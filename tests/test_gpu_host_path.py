"""The host-buffer entry point (replicas in host memory, streamed through the GPU in column
chunks) against the CPU oracle and against the resident-replica path."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_09010_b200 import binding
from harness import ATOL, RTOL, random_theta0

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,chunk,pinned", [(0, 4096, True), (0, 1024, False), (1, 2048, True),
                                                (0, 0, True)])
@pytest.mark.parametrize("K,p,q", [(8, 2, 2), (40, 4, 3)])      # 40 workers: ring-window launch shape
def test_host_round_matches_oracle(dtype, chunk, pinned, K, p, q):
    eta, zeta, seed = 0.9, 1.0, 21
    offsets = (0, 1000, 1001, 4096, 9999, 20001, 50003)
    N = offsets[-1]
    ld = N + 13                                           # host arrays need no padding rule
    st = oracle.init(random_theta0(N, seed=3, dtype=dtype), K, ld=ld, dtype=dtype)
    oracle.local_perturb(st, seed, 0, 1.0, 0.05)
    st.omega[:, :N] += np.float32(0.01)
    st.delta[:, :N] = (np.random.Generator(np.random.PCG64(1)).standard_normal((K, N)) * 0.01).astype(np.float32)
    st.rst[:] = st.theta                                   # block-start value consistent with ...
    if dtype == 0:                                         # ... omega + eta*Delta is what the GPU recomputes
        st.rst[:, :N] = st.omega[:, :N] + np.float32(eta) * st.delta[:, :N]
    else:
        st.rst[:, :N] = oracle.f32_to_bf16(st.omega[:, :N] + np.float32(eta) * st.delta[:, :N])

    def host(a, tdt):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).clone()
        if a.dtype == np.uint16:
            t = t.view(torch.bfloat16)
        return t.pin_memory() if pinned else t

    th, om, de = host(st.theta, dtype), host(st.omega, 0), host(st.delta, 0)
    masks = [None, [1, 0, 1, 1, 0, 1]]
    for rnd, mask in zip((1, 2), masks):
        binding.sync_round_host(th, om, de, offsets, rnd, K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=zeta,
                                seed=seed, theta_dtype=dtype, comp_mask=mask, chunk_cols=chunk)
        nbr = oracle.sample_neighbors(seed, rnd, K, len(offsets) - 1, p, q)
        oracle.sync_round(st, offsets, nbr, eta, zeta, sync=mask)
        got_t = th.view(torch.int16).numpy().view(np.uint16) if dtype == 1 else th.numpy()
        for name, got, ref in (("omega", om.numpy(), st.omega), ("delta", de.numpy(), st.delta)):
            assert np.all(np.abs(got - ref) <= ATOL + RTOL * np.abs(ref)), name
            assert np.array_equal(got.view(np.uint32), ref.view(np.uint32)), name
        assert np.array_equal(got_t.view(np.uint8), st.theta.view(np.uint8)), "theta"


@pytest.mark.parametrize("dtype,mode,row_copies", [(0, 0, False), (1, 0, True), (0, 1, True)])
def test_host_handle_over_several_rounds(dtype, mode, row_copies):
    """The handle form: chunk buffers, streams and chunk tables made once and used for four
    rounds (masks changing from round to round), against the oracle after every round."""
    K, p, q, eta, zeta, seed = 8, 2, 2, 0.875, 1.0, 5
    offsets = (0, 1000, 1001, 4096, 9999, 20001, 50003)
    N = offsets[-1]
    ld = N + 5
    st = oracle.init(random_theta0(N, seed=9, dtype=dtype), K, ld=ld, dtype=dtype)
    oracle.local_perturb(st, seed, 0, 1.0, 0.05)

    def host(a):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).clone()
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).pin_memory()

    th, om, de = host(st.theta), host(st.omega), host(st.delta)
    h = binding.GbmufHost(offsets, K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=zeta, seed=seed,
                          theta_dtype=dtype, mode=mode, chunk_cols=2048, row_copies=row_copies)
    try:
        masks = [None, [1, 0, 1, 1, 0, 1], [0, 0, 0, 0, 0, 0], [0, 1, 0, 0, 1, 0]]
        for rnd, mask in enumerate(masks, start=1):
            h.sync_round(th, om if mode == 0 else None, de if mode == 0 else None, rnd, mask)
            nbr = oracle.sample_neighbors(seed, rnd, K, len(offsets) - 1, p, q)
            oracle.sync_round(st, offsets, nbr, eta, zeta, mode=mode, sync=mask)
            got_t = th.view(torch.int16).numpy().view(np.uint16) if dtype == 1 else th.numpy()
            assert np.array_equal(got_t.view(np.uint8), st.theta.view(np.uint8)), f"theta, round {rnd}"
            assert np.array_equal(om.numpy().view(np.uint32), st.omega.view(np.uint32)), f"omega, round {rnd}"
            assert np.array_equal(de.numpy().view(np.uint32), st.delta.view(np.uint32)), f"delta, round {rnd}"
    finally:
        h.destroy()


def test_host_handle_many_chunks_of_the_default_size():
    """Five chunks of the default 2,097,152 columns rotate through the three buffer sets (every
    set is re-used), two rounds, the second with a mask that leaves whole chunks untouched;
    every element against the oracle."""
    K, p, q, eta, zeta, seed = 8, 2, 2, 0.9, 1.0, 77
    N = (1 << 23) + 5
    offsets = (0, 1 << 21, (1 << 21) + 3, 3 << 21, (3 << 21) + 1000, N)
    st = oracle.init(random_theta0(N, seed=4), K)
    oracle.local_perturb(st, seed, 0, 1.0, 0.05)
    th = torch.from_numpy(st.theta).clone().pin_memory()
    om = torch.from_numpy(st.omega).clone().pin_memory()
    de = torch.from_numpy(st.delta).clone().pin_memory()
    h = binding.GbmufHost(offsets, K=K, N=N, ld=N, p=p, q=q, eta=eta, zeta=zeta, seed=seed)
    try:
        for rnd, mask in ((1, None), (2, [0, 1, 1, 0, 1])):
            h.sync_round(th, om, de, rnd, mask)
            nbr = oracle.sample_neighbors(seed, rnd, K, len(offsets) - 1, p, q)
            oracle.sync_round(st, offsets, nbr, eta, zeta, sync=mask)
            for name, got, ref in (("theta", th, st.theta), ("omega", om, st.omega), ("delta", de, st.delta)):
                assert np.array_equal(got.numpy().view(np.uint32), ref.view(np.uint32)), f"{name}, round {rnd}"
    finally:
        h.destroy()


def test_host_round_argument_errors():
    K, N = 4, 1000
    th = torch.zeros((K, N))
    kw = dict(K=K, N=N, ld=N, p=1, q=1, eta=0.9, zeta=1.0)
    with pytest.raises(binding.GbmufError) as e:
        binding.sync_round_host(th, th.clone(), th.clone(), [0, 500, N], 1, chunk_cols=100, **kw)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.GbmufError):
        binding.sync_round_host(th, th.clone(), th.clone(), [0, 500, 400, N], 1, **kw)
    with pytest.raises(binding.GbmufError):
        binding.sync_round_host(th, th.clone(), th.clone(), [0, N], 1, **dict(kw, q=3))
