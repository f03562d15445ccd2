"""Pins of the oracle's synthetic local step (the stand-in for theta <- theta - alpha g)."""
import numpy as np

F32 = np.float32


def test_noise_moments(oracle):
    """z is a centred, unit-variance sum of four 16-bit uniforms (Irwin-Hall, n=4):
    mean 0, variance 1, kurtosis 3 - 6/(5*4) = 2.7, support |z| <= sqrt(12)."""
    K, N = 4, 500_000
    st = oracle.init(np.zeros(N, dtype=F32), K)
    oracle.local_perturb(st, seed=123, step=7, lr=1.0, sigma=1.0)
    z = -st.theta.astype(np.float64).ravel()
    assert abs(z.mean()) < 4.0 / np.sqrt(z.size)
    assert abs(z.var() - 1.0) < 0.01
    assert abs((z ** 4).mean() / z.var() ** 2 - 2.7) < 0.02
    assert np.abs(z).max() <= np.sqrt(12.0) + 1e-6
    assert abs(np.mean(np.abs(z) < 1.0) - 0.6826) < 0.02            # close to a normal's 68 %
    # no correlation between the two elements of a pair, between workers, between neighbours
    zz = z.reshape(K, N)
    assert abs(np.mean(zz[:, 0::2] * zz[:, 1::2])) < 0.005
    assert abs(np.mean(zz[0] * zz[1])) < 0.006
    assert abs(np.mean(zz[:, :-2] * zz[:, 2:])) < 0.005


def test_scale_is_lr_times_sigma(oracle):
    N = 200_000
    st = oracle.init(np.full(N, 0.25, dtype=F32), 2)
    oracle.local_perturb(st, seed=5, step=0, lr=0.1, sigma=1e-3)
    d = st.theta.astype(np.float64) - 0.25
    assert abs(d.std() / 1e-4 - 1.0) < 0.01 and abs(d.mean()) < 1e-6


def test_steps_compose_and_are_keyed(oracle):
    N = 1001
    a = oracle.init(np.linspace(-1, 1, N).astype(F32), 3, ld=1024)
    b, c, d = a.copy(), a.copy(), a.copy()
    oracle.local_perturb(a, seed=9, step=4, lr=0.1, sigma=0.5, nsteps=3)
    for s in (4, 5, 6):
        oracle.local_perturb(b, seed=9, step=s, lr=0.1, sigma=0.5)
    assert np.array_equal(a.theta, b.theta)
    assert not a.theta[:, N:].any()
    oracle.local_perturb(c, seed=9, step=5, lr=0.1, sigma=0.5, nsteps=3)      # other steps
    oracle.local_perturb(d, seed=10, step=4, lr=0.1, sigma=0.5, nsteps=3)     # other seed
    assert not np.array_equal(a.theta, c.theta) and not np.array_equal(a.theta, d.theta)
    assert not np.array_equal(a.theta[0], a.theta[1])                          # per worker
    e = oracle.init(np.linspace(-1, 1, N).astype(F32), 3, ld=1024)
    oracle.local_perturb(e, seed=9, step=4, lr=0.1, sigma=0.5, nsteps=0)
    assert np.array_equal(e.theta[:, :N], np.tile(np.linspace(-1, 1, N).astype(F32), (3, 1)))


def test_noise_is_a_function_of_the_global_element_index(oracle):
    """A column range processed on its own (elem_base = its first column) gets the noise the
    full run gives those columns -- odd starts included."""
    N = 300
    full = oracle.init(np.zeros(N, dtype=F32), 2)
    oracle.local_perturb(full, seed=77, step=1, lr=1.0, sigma=1.0, nsteps=2)
    for c0, c1 in ((0, 10), (7, 120), (101, 300)):
        part = oracle.init(np.zeros(c1 - c0, dtype=F32), 2)
        oracle.local_perturb(part, seed=77, step=1, lr=1.0, sigma=1.0, nsteps=2, elem_base=c0)
        assert np.array_equal(part.theta, full.theta[:, c0:c1])


def test_bf16_theta_is_rounded_after_every_step(oracle):
    import torch
    N = 4096
    x0 = oracle.f32_to_bf16((np.random.Generator(np.random.PCG64(3)).standard_normal(N) * 0.1)
                            .astype(F32))
    st = oracle.init(x0, 2, dtype=1)
    ref = oracle.State(2, N, N, 0, oracle.bf16_to_f32(st.theta), st.omega, st.delta,
                       oracle.bf16_to_f32(st.rst))
    oracle.local_perturb(st, seed=1, step=0, lr=0.1, sigma=0.05, nsteps=2)
    for s in (0, 1):
        oracle.local_perturb(ref, seed=1, step=s, lr=0.1, sigma=0.05)
        r = torch.from_numpy(ref.theta).to(torch.bfloat16)
        ref.theta[:] = r.float().numpy()
    assert np.array_equal(oracle.bf16_to_f32(st.theta), ref.theta)
