"""The Adagrad local step with gradient-norm clipping (the optimiser of the paper's experiments)
on the GPU against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_09010_b200 import binding
from harness import ATOL, RTOL, random_theta0, to_numpy, from_numpy

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("K,offsets,mask", [
    (4, (0, 1000, 5001, 9000, 20003), [0, 1, 1, 0]),          # one merged run, unaligned edges
    (3, (0, 7, 4099, 4100, 10000, 30001), [1, 0, 1, 0, 1]),   # three separate runs
    (2, (0, 50_000), [1]),                                    # everything clipped
    (5, (0, 64, 10_007), None),                               # no clipping
    (8, (0, 100_000, 100_003, 333_333, 500_003), [0, 1, 1, 0]),   # every CTA goes round its ring of slots
    (1, (0, 5), None),                                        # shorter than one 16-byte piece
])
def test_adagrad_step_matches_oracle(dtype, K, offsets, mask):
    dev = torch.device("cuda:0")
    N = offsets[-1]
    ld = (N + 31) // 32 * 32
    st = oracle.init(random_theta0(N, seed=K, dtype=dtype), K, ld=ld, dtype=dtype)
    g = np.random.Generator(np.random.PCG64(K + 100))
    accum = np.zeros((K, ld), dtype=np.float32)
    accum[:, :N] = 0.1
    theta = from_numpy(st.theta, dtype, dev)
    om, de = torch.zeros((K, ld), device=dev), torch.zeros((K, ld), device=dev)
    acc_dev = torch.from_numpy(accum.copy()).to(dev)
    ctx = binding.Gbmuf(theta, om, de, K=K, N=N, ld=ld, p=1 if K > 2 else 0, q=0, eta=0.9, zeta=1.0,
                        theta_dtype=dtype)
    ctx.set_partition(offsets)
    ranges = []
    if mask is not None:
        ranges = [(offsets[i], offsets[i + 1]) for i in range(len(mask)) if mask[i]]
    for step in range(3):
        grad = np.zeros((K, ld), dtype=np.float32)
        scale = [3.0, 0.02, 1.0][step]                       # above, below and near the threshold
        grad[:, :N] = (g.standard_normal((K, N)) * scale).astype(np.float32)
        grad_dev = torch.from_numpy(grad).to(dev)
        lr = 0.1 * 0.9 ** step
        ctx.local_adagrad(grad_dev, acc_dev, lr, eps=1e-8, clip_norm=10.0, clip_mask=mask)
        oracle.local_adagrad(st, grad, accum, lr, eps=1e-8, clip_norm=10.0, ranges=ranges)
        torch.cuda.synchronize()
        got_a = acc_dev.cpu().numpy()
        assert np.all(np.abs(got_a - accum) <= ATOL + RTOL * np.abs(accum))
        assert np.array_equal(got_a.view(np.uint32), accum.view(np.uint32)), "accumulator not bit-equal"
        got_t = to_numpy(theta)
        if dtype == 0:
            assert np.all(np.abs(got_t - st.theta) <= ATOL + RTOL * np.abs(st.theta))
        assert np.array_equal(got_t.view(np.uint8), st.theta.view(np.uint8)), "theta not bit-equal"
    ctx.destroy()


def test_adagrad_random_shapes_property():
    """Random worker counts, row lengths (several chunks per CTA included), clip groups, theta type
    and step sizes: accumulator and theta bit-equal with the oracle, padding untouched."""
    import os
    from hypothesis import given, settings, strategies as st_, HealthCheck

    @settings(max_examples=int(os.environ.get("GBMUF_PROPERTY_EXAMPLES", "30")), deadline=None,
              derandomize=True, suppress_health_check=list(HealthCheck))
    @given(st_.data())
    def inner(data):
        dev = torch.device("cuda:0")
        K = data.draw(st_.integers(1, 12))
        m = data.draw(st_.integers(1, 7))
        N = data.draw(st_.integers(m, data.draw(st_.sampled_from([5_000, 60_000, 700_000]))))
        cuts = sorted(data.draw(st_.sets(st_.integers(1, N - 1), min_size=m - 1, max_size=m - 1))) if m > 1 else []
        offsets = tuple([0] + cuts + [N])
        dtype = data.draw(st_.integers(0, 1))
        mask = data.draw(st_.one_of(st_.none(), st_.lists(st_.integers(0, 1), min_size=m, max_size=m)))
        clip = data.draw(st_.sampled_from([10.0, 0.5, 0.0]))
        gscale = data.draw(st_.sampled_from([3.0, 0.02, 1.0]))
        lr = data.draw(st_.sampled_from([0.1, 0.081, 1e-3]))
        ld = (N + 31) // 32 * 32
        st = oracle.init(random_theta0(N, seed=K + N, dtype=dtype), K, ld=ld, dtype=dtype)
        g = np.random.Generator(np.random.PCG64(N))
        accum = np.zeros((K, ld), dtype=np.float32)
        accum[:, :N] = 0.1
        grad = np.zeros((K, ld), dtype=np.float32)
        grad[:, :N] = (g.standard_normal((K, N)) * gscale).astype(np.float32)
        theta = from_numpy(st.theta, dtype, dev)
        om, de = torch.zeros((K, ld), device=dev), torch.zeros((K, ld), device=dev)
        acc_dev, grad_dev = torch.from_numpy(accum.copy()).to(dev), torch.from_numpy(grad).to(dev)
        ctx = binding.Gbmuf(theta, om, de, K=K, N=N, ld=ld, p=0, q=0, eta=0.9, zeta=1.0, theta_dtype=dtype)
        try:
            ctx.set_partition(offsets)
            ranges = [(offsets[i], offsets[i + 1]) for i in range(m) if mask and mask[i]] if clip > 0 else []
            for _ in range(2):
                ctx.local_adagrad(grad_dev, acc_dev, lr, eps=1e-8, clip_norm=clip, clip_mask=mask)
                oracle.local_adagrad(st, grad, accum, lr, eps=1e-8, clip_norm=clip, ranges=ranges)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            assert np.array_equal(acc_dev.cpu().numpy().view(np.uint32), accum.view(np.uint32))
            assert np.array_equal(to_numpy(theta).view(np.uint8), st.theta.view(np.uint8))
        finally:
            ctx.destroy()

    inner()


def test_adagrad_then_sync_round_full_step():
    """Algorithm 1's loop body with the experiments' optimiser: local Adagrad step, then the
    gossip-BMUF round every second step, both sides replaying the same calls."""
    dev = torch.device("cuda:0")
    K, p, q, eta = 8, 2, 2, 0.9
    offsets = (0, 3000, 7001, 12000)
    N, ld = 12000, 12000
    st = oracle.init(random_theta0(N, seed=2), K, ld=ld)
    theta = torch.from_numpy(st.theta.copy()).to(dev)
    om, de = torch.from_numpy(st.omega.copy()).to(dev), torch.zeros((K, ld), device=dev)
    accum = np.full((K, ld), 0.1, dtype=np.float32)
    acc_dev = torch.from_numpy(accum.copy()).to(dev)
    ctx = binding.Gbmuf(theta, om, de, K=K, N=N, ld=ld, p=p, q=q, eta=eta, zeta=1.0, seed=5)
    ctx.set_partition(offsets)
    g = np.random.Generator(np.random.PCG64(7))
    for t in range(1, 7):
        grad = g.standard_normal((K, ld)).astype(np.float32)
        ctx.local_adagrad(torch.from_numpy(grad).to(dev), acc_dev, 0.1, clip_norm=10.0, clip_mask=[0, 1, 0])
        oracle.local_adagrad(st, grad, accum, 0.1, clip_norm=10.0, ranges=[(3000, 7001)])
        if t % 2 == 0:                                        # sync period H = 2
            ctx.sync_round(t)
            nbr = oracle.sample_neighbors(5, t, K, 3, p, q)
            oracle.sync_round(st, offsets, nbr, eta, 1.0)
    torch.cuda.synchronize()
    assert np.array_equal(theta.cpu().numpy().view(np.uint32), st.theta.view(np.uint32))
    assert np.array_equal(om.cpu().numpy().view(np.uint32), st.omega.view(np.uint32))
    assert np.array_equal(de.cpu().numpy().view(np.uint32), st.delta.view(np.uint32))
    ctx.destroy()


def test_adagrad_argument_errors():
    dev = torch.device("cuda:0")
    th = torch.zeros((2, 64), device=dev)
    ctx = binding.Gbmuf(th, th.clone(), th.clone(), K=2, N=64, ld=64, p=0, q=0, eta=0.9, zeta=1.0)
    m = np.ones(1, dtype=np.uint8)                            # a mask before set_partition
    rc = binding.lib().gbmuf_local_adagrad(ctx._h, th.data_ptr(), th.data_ptr(), 0.1, 0.0, 10.0,
                                           m.ctypes.data, None)
    assert rc == binding.ERR_BAD_STATE
    ctx.set_partition(list(range(0, 65, 1)))                 # 64 components
    with pytest.raises(binding.GbmufError) as e:             # 32 separate runs
        ctx.local_adagrad(th, th.clone(), 0.1, clip_norm=10.0, clip_mask=[i % 2 for i in range(64)])
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.GbmufError):
        ctx.local_adagrad(None, th, 0.1)
    ctx.destroy()
