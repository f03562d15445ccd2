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

from paper_1909_09010_b200 import binding
from harness import ATOL, RTOL

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
