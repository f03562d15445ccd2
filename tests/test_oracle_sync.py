"""Pins of the oracle's synchronisation round (Algorithm 1: gossip average, block delta,
block momentum, global-model update, restart point) against closed forms, float64 brute
force, exact rational brute force and invariants."""
from fractions import Fraction

import numpy as np
import pytest

F32 = np.float32


def ulp(x):
    return np.spacing(np.abs(np.asarray(x, dtype=np.float32)))


def make_state(oracle, K, N, seed, ld=None, dtype=0, spread=0.05):
    g = np.random.Generator(np.random.PCG64(seed))
    theta0 = (g.standard_normal(N) * 0.1).astype(F32)
    if dtype == 1:
        theta0 = oracle.f32_to_bf16(theta0)
    st = oracle.init(theta0, K, ld=ld, dtype=dtype)
    drift = (g.standard_normal((K, N)) * spread).astype(F32)
    if dtype == 0:
        st.theta[:, :N] += drift
    else:
        st.theta[:, :N] = oracle.f32_to_bf16(oracle.bf16_to_f32(st.theta[:, :N]) + drift)
    return st, g


def all_others(K, m):
    return np.array([[[j for j in range(K) if j != k]] * m for k in range(K)], dtype=np.int32)


# -------------------------------------------------------------------------------------------
# gossip average
# -------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K,p,q", [(4, 1, 1), (8, 2, 2), (16, 3, 2), (8, 2, 3), (16, 3, 6)])
def test_average_is_the_row_stochastic_mixing_matrix(oracle, K, p, q):
    """theta_bar = A_i theta with A_i[k][k] = A_i[k][k_j] = 1/(q+1): float64 brute force."""
    N, off = 96, [0, 17, 40, 96]
    st, _ = make_state(oracle, K, N, seed=K * 100 + q)
    before = st.theta.astype(np.float64).copy()
    nbr = oracle.sample_neighbors(5, 1, K, 3, p, q)
    oracle.sync_round(st, off, nbr, 0.9, 1.0, mode=oracle.MODE_MA)
    for i in range(3):
        A = np.zeros((K, K))
        for k in range(K):
            A[k, k] = 1.0 / (q + 1)
            for j in nbr[k, i]:
                A[k, j] += 1.0 / (q + 1)
        assert np.allclose(A.sum(axis=1), 1.0)
        want = A @ before[:, off[i]:off[i + 1]]
        got = st.theta[:, off[i]:off[i + 1]]
        scale = ulp(np.abs(before[:, off[i]:off[i + 1]]).max())
        assert np.max(np.abs(got - want)) <= 2 * scale


def test_identical_replicas_are_a_fixed_point(oracle):
    """Equal replicas, Delta = 0, restart = theta: the whole round is the identity, exactly,
    when q+1 is a power of two (the sum (q+1)x is exact)."""
    for K, p, q in [(4, 1, 1), (8, 2, 3), (8, 2, 1)]:
        g = np.random.Generator(np.random.PCG64(1))
        theta0 = (g.standard_normal(200) * 0.1).astype(F32)
        st = oracle.init(theta0, K)
        ref = st.copy()
        nbr = oracle.sample_neighbors(0, 1, K, 2, p, q)
        gout = oracle.sync_round(st, [0, 77, 200], nbr, 0.9, 1.0, want_g=True)
        for a, b in [(st.theta, ref.theta), (st.omega, ref.omega), (st.delta, ref.delta),
                     (st.rst, ref.rst)]:
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
        assert not gout.any()
    # q+1 = 3: the average may move by at most one ulp
    st = oracle.init(theta0, 8)
    nbr = oracle.sample_neighbors(0, 1, 8, 1, 2, 2)
    oracle.sync_round(st, [0, 200], nbr, 0.0, 1.0, mode=oracle.MODE_MA)
    assert np.all(np.abs(st.theta - theta0[None]) <= ulp(theta0)[None])


# -------------------------------------------------------------------------------------------
# closed forms of the whole round
# -------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K", [4, 5, 8])
def test_all_workers_as_neighbours_is_classic_bmuf(oracle, K):
    """Neighbour set = everybody else: theta_bar is the full mean (Simple MA's averaging line)
    and the round is the classic block-momentum update with Nesterov restart, here restated in
    float64 from the mean."""
    N, eta, zeta = 64, 0.9, 1.0
    st, g = make_state(oracle, K, N, seed=K)
    th = st.theta.astype(np.float64)
    om, de, rs = st.omega.astype(np.float64), st.delta.astype(np.float64), st.rst.astype(np.float64)
    nbr = all_others(K, 1)
    for rnd in range(6):
        oracle.sync_round(st, [0, N], nbr, eta, zeta)
        mean = th.mean(axis=0, keepdims=True)
        G = mean - rs
        de = np.float64(F32(eta)) * de + zeta * G
        om = om + de
        th = om + np.float64(F32(eta)) * de
        rs = th.copy()
        tol = 1e-6 * (rnd + 1)
        assert np.allclose(st.theta, th, rtol=tol, atol=tol * 0.1)
        assert np.allclose(st.omega, om, rtol=tol, atol=tol * 0.1)
        assert np.allclose(st.delta, de, rtol=tol, atol=tol * 0.1)
        # all workers agree up to summation order
        assert np.max(np.abs(st.theta - st.theta[0:1])) <= 4 * ulp(np.abs(st.theta).max())
        step = (g.standard_normal((K, N)) * 0.01).astype(F32)
        st.theta += step
        th = st.theta.astype(np.float64)            # local steps are inputs, not under test
        om, de = st.omega.astype(np.float64), st.delta.astype(np.float64)
        rs = st.rst.astype(np.float64)


def test_full_neighbour_set_through_the_ring_sampler(oracle):
    """Same closed form, but with the neighbour table produced by the sampler: p >= K/2 and
    q = K-1 make every draw a permutation of all other workers."""
    K, N = 6, 40
    st, _ = make_state(oracle, K, N, seed=3)
    nbr = oracle.sample_neighbors(8, 2, K, 1, 3, K - 1)
    mean = st.theta.astype(np.float64).mean(axis=0)
    oracle.sync_round(st, [0, N], nbr, 0.0, 1.0, mode=oracle.MODE_MA)
    assert np.max(np.abs(st.theta - mean[None])) <= 3 * ulp(np.abs(mean).max())


def test_eta_zero_zeta_one_is_model_averaging(oracle):
    """eta=0, zeta=1: Delta=G, omega and theta both land on theta_bar (gossip-MA branch)."""
    K, N, p, q = 8, 120, 2, 2
    st, g = make_state(oracle, K, N, seed=21)
    ma = st.copy()
    for rnd in range(1, 5):
        nbr = oracle.sample_neighbors(4, rnd, K, 2, p, q)
        oracle.sync_round(st, [0, 50, N], nbr, 0.0, 1.0)
        oracle.sync_round(ma, [0, 50, N], nbr, 0.0, 1.0, mode=oracle.MODE_MA)
        scale = ulp(np.abs(ma.theta).max())
        assert np.max(np.abs(st.theta - ma.theta)) <= 2 * scale
        assert np.array_equal(st.theta, st.omega)
        step = (g.standard_normal((K, N)) * 0.01).astype(F32)
        st.theta += step
        ma.theta[:] = st.theta
    # in MA mode omega, Delta and the restart slot are never touched
    assert np.array_equal(ma.delta, np.zeros_like(ma.delta))


def test_filter_geometric_series_exact(oracle):
    """K=1, no neighbours, a constant block delta g fed every round:
    Delta_n = zeta g (1-eta^n)/(1-eta), omega_n = theta_0 + sum Delta_j, theta_n = omega_n + eta Delta_n.
    With eta=1/2, g=1, theta_0=0 every quantity is a dyadic rational, so fp32 must be exact."""
    st = oracle.init(np.zeros(4, dtype=F32), K=1)
    nbr = np.zeros((1, 1, 0), dtype=np.int32)
    eta, zeta, gval = Fraction(1, 2), Fraction(1), Fraction(1)
    om_sum = Fraction(0)
    for n in range(1, 16):
        st.theta[:] = st.rst + F32(1.0)                   # the local steps moved theta by g
        G = oracle.sync_round(st, [0, 4], nbr, 0.5, 1.0, want_g=True)
        d = zeta * gval * (1 - eta ** n) / (1 - eta)
        om_sum += d
        assert np.all(G == 1.0)
        assert np.all(st.delta == float(d))
        assert np.all(st.omega == float(om_sum))
        assert np.all(st.theta == float(om_sum + eta * d))
        assert np.array_equal(st.rst, st.theta)


def test_filter_geometric_series_general(oracle):
    eta, zeta, gval = 0.9, 0.75, 0.013
    st = oracle.init(np.full(3, 0.2, dtype=F32), K=1)
    nbr = np.zeros((1, 1, 0), dtype=np.int32)
    om = float(F32(0.2))
    e32, z32 = float(F32(eta)), float(F32(zeta))
    for n in range(1, 40):
        before = st.rst.astype(np.float64)
        st.theta[:] = st.rst + F32(gval)
        g_eff = (st.theta.astype(np.float64) - before)[0, 0]      # what fp32 made of g
        if n == 1:
            d = z32 * g_eff
        else:
            d = e32 * d + z32 * g_eff
        om += d
        oracle.sync_round(st, [0, 3], nbr, eta, zeta)
        assert abs(st.delta[0, 0] - d) <= 2e-6 * abs(d)
        assert abs(st.omega[0, 0] - om) <= 2e-6 * abs(om)
        assert abs(st.theta[0, 0] - (om + e32 * d)) <= 2e-6 * abs(om + e32 * d)
    # limit: Delta -> zeta g / (1 - eta)
    assert abs(st.delta[0, 0] - z32 * gval / (1 - e32)) < 0.02 * z32 * gval / (1 - e32) + 1e-3


# -------------------------------------------------------------------------------------------
# exact rational brute force on tiny inputs (all values dyadic, all fp32 operations exact)
# -------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K,p,q,eta,zeta", [(4, 1, 1, 0.5, 1.0), (4, 2, 3, 0.25, 2.0),
                                             (3, 1, 1, 0.5, 0.5), (2, 1, 1, 0.75, 1.0)])
def test_tiny_integer_brute_force(oracle, K, p, q, eta, zeta):
    N, off, rounds = 24, [0, 5, 6, 24], 3
    g = np.random.Generator(np.random.PCG64(K * 7 + q))
    theta0 = g.integers(-64, 64, size=N).astype(F32)
    st = oracle.init(theta0, K)
    th = [[Fraction(int(theta0[e])) for e in range(N)] for _ in range(K)]
    om = [row[:] for row in th]
    rs = [row[:] for row in th]
    de = [[Fraction(0)] * N for _ in range(K)]
    fe, fz = Fraction(eta), Fraction(zeta)
    for rnd in range(1, rounds + 1):
        bump = g.integers(-32, 32, size=(K, N)).astype(F32)
        st.theta += bump
        for k in range(K):
            for e in range(N):
                th[k][e] += Fraction(int(bump[k, e]))
        nbr = oracle.sample_neighbors(1, rnd, K, 3, p, q)
        sync = [1, 1, 1] if rnd != 2 else [1, 0, 1]
        oracle.sync_round(st, off, nbr, eta, zeta, sync=sync)
        snap = [row[:] for row in th]
        for k in range(K):
            for i in range(3):
                if not sync[i]:
                    continue
                for e in range(off[i], off[i + 1]):
                    avg = (snap[k][e] + sum(snap[int(j)][e] for j in nbr[k, i])) / (q + 1)
                    G = avg - rs[k][e]
                    de[k][e] = fe * de[k][e] + fz * G
                    om[k][e] = om[k][e] + de[k][e]
                    th[k][e] = om[k][e] + fe * de[k][e]
                    rs[k][e] = th[k][e]
        for name, got, want in (("theta", st.theta, th), ("omega", st.omega, om),
                                ("delta", st.delta, de), ("rst", st.rst, rs)):
            w = np.array([[float(x) for x in row] for row in want])
            assert all(Fraction(float(F32(float(x)))) == x for row in want for x in row), \
                "test input left the exactly representable range"
            assert np.array_equal(got[:, :N].astype(np.float64), w), (name, rnd)


# -------------------------------------------------------------------------------------------
# invariants
# -------------------------------------------------------------------------------------------
def test_restart_point_invariant_and_recomputability(oracle):
    """After every round theta == fl(omega + fl(eta Delta)) bit for bit, and the stored
    block-start value equals theta: the next round's "theta_{t-H}" can be recomputed from
    omega and Delta alone."""
    K, N, p, q, eta = 8, 333, 2, 2, 0.875
    st, g = make_state(oracle, K, N, seed=5, ld=352)
    off = [0, 100, 101, 333]
    for rnd in range(1, 6):
        nbr = oracle.sample_neighbors(6, rnd, K, 3, p, q)
        oracle.sync_round(st, off, nbr, eta, 1.0)
        recomputed = st.omega + F32(eta) * st.delta
        assert np.array_equal(recomputed.view(np.uint32)[:, :N], st.theta.view(np.uint32)[:, :N])
        assert np.array_equal(st.rst.view(np.uint32), st.theta.view(np.uint32))
        assert not st.theta[:, N:].any() and not st.omega[:, N:].any()   # padding untouched
        st.theta[:, :N] += (g.standard_normal((K, N)) * 0.01).astype(F32)


def test_result_does_not_depend_on_worker_order(oracle):
    """All neighbour reads see the round's input replicas (every term of the averaging line
    carries the same step index), so the processing order of workers cannot matter."""
    K, N, p, q = 8, 150, 2, 2
    base, _ = make_state(oracle, K, N, seed=9)
    nbr = oracle.sample_neighbors(2, 1, K, 2, p, q)
    outs = []
    for order in (None, list(range(K))[::-1], [3, 7, 0, 5, 1, 6, 2, 4]):
        st = base.copy()
        oracle.sync_round(st, [0, 64, N], nbr, 0.9, 1.0, order=order)
        outs.append(st)
    for st in outs[1:]:
        for a, b in ((st.theta, outs[0].theta), (st.omega, outs[0].omega),
                     (st.delta, outs[0].delta)):
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_unsynced_components_are_untouched(oracle):
    K, N = 4, 90
    st, _ = make_state(oracle, K, N, seed=13)
    ref = st.copy()
    nbr = oracle.sample_neighbors(2, 1, K, 3, 1, 1)
    oracle.sync_round(st, [0, 30, 60, 90], nbr, 0.9, 1.0, sync=[1, 0, 1])
    for a, b in ((st.theta, ref.theta), (st.omega, ref.omega), (st.delta, ref.delta),
                 (st.rst, ref.rst)):
        assert np.array_equal(a[:, 30:60], b[:, 30:60])
        assert not np.array_equal(a[:, :30], b[:, :30])
        assert not np.array_equal(a[:, 60:], b[:, 60:])


def test_first_round_block_delta_is_against_theta0(oracle):
    """Before any sync the block-start value is theta_0 (the initialisation line)."""
    K, N = 4, 32
    theta0 = np.linspace(-1, 1, N).astype(F32)
    st = oracle.init(theta0, K)
    assert np.array_equal(st.rst, np.tile(theta0, (K, 1)))
    assert np.array_equal(st.omega, np.tile(theta0, (K, 1))) and not st.delta.any()
    st.theta += F32(0.5)                                   # every replica moved by +0.5
    nbr = oracle.sample_neighbors(0, 1, K, 1, 1, 1)
    G = oracle.sync_round(st, [0, N], nbr, 0.9, 1.0, want_g=True)
    assert np.allclose(G, 0.5, atol=1e-6)
    assert np.allclose(st.delta, 0.5, atol=1e-6)
    assert np.allclose(st.omega, theta0[None] + 0.5, atol=1e-6)
    assert np.allclose(st.theta, theta0[None] + 0.5 + 0.9 * 0.5, atol=1e-6)


# -------------------------------------------------------------------------------------------
# bf16 storage of theta
# -------------------------------------------------------------------------------------------
def test_bf16_rounding_matches_library_conversion(oracle):
    import torch
    g = np.random.Generator(np.random.PCG64(17))
    x = np.concatenate([(g.standard_normal(20000) * 10.0 ** g.integers(-30, 30, 20000)).astype(F32),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, np.inf, -np.inf,
                                  3.3895314e38, 1e-40, -1e-45], dtype=F32)])
    # exact ties: bf16 keeps 8 significant bits; x = (2n+1) * 2^-8 scaled
    ties = ((np.arange(256, 512, dtype=np.float64) * 2 + 1) / 512).astype(F32)
    x = np.concatenate([x, ties, -ties])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16(x), want)
    back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(oracle.bf16_to_f32(want).view(np.uint32), back.view(np.uint32))


def test_bf16_theta_round_is_fp32_round_then_rounded(oracle):
    """bf16 replicas: widen exactly, do the fp32 round, round theta to nearest even on store;
    omega and Delta stay fp32.  Checked against the fp32 oracle run on the widened inputs with
    the block-start value taken from the bf16 run."""
    import torch
    K, N, p, q, eta = 4, 100, 1, 1, 0.9
    st, g = make_state(oracle, K, N, seed=31, dtype=1)
    wide = oracle.State(K, N, N, 0, oracle.bf16_to_f32(st.theta), st.omega.copy(), st.delta.copy(),
                        oracle.bf16_to_f32(st.rst))
    nbr = oracle.sample_neighbors(1, 1, K, 1, p, q)
    oracle.sync_round(st, [0, N], nbr, eta, 1.0)
    oracle.sync_round(wide, [0, N], nbr, eta, 1.0)
    assert np.array_equal(st.omega, wide.omega) and np.array_equal(st.delta, wide.delta)
    want = torch.from_numpy(wide.theta).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(st.theta, want)
    assert np.array_equal(st.rst, st.theta)
    # the bf16 restart point is the rounded fl(omega + fl(eta Delta))
    rec = torch.from_numpy(st.omega + F32(eta) * st.delta).to(torch.bfloat16).view(torch.int16)
    assert np.array_equal(st.theta, rec.numpy().view(np.uint16))


# -------------------------------------------------------------------------------------------
# final model (return line of Algorithm 1)
# -------------------------------------------------------------------------------------------
def test_final_average(oracle):
    K, N = 8, 77
    st, _ = make_state(oracle, K, N, seed=2, ld=96)
    got = oracle.final_average(st)
    want = st.theta[:, :N].astype(np.float64).mean(axis=0)
    assert np.max(np.abs(got - want)) <= 4 * ulp(np.abs(st.theta).max())
    # identical replicas: exact for K=2 (x+x is exact), within rounding of the running sum else
    same2 = oracle.init(st.theta[0, :N].copy(), 2)
    assert np.array_equal(oracle.final_average(same2), st.theta[0, :N])
    same8 = oracle.init(st.theta[0, :N].copy(), 8)
    assert np.all(np.abs(oracle.final_average(same8) - st.theta[0, :N]) <= 2 * ulp(st.theta[0, :N]))
