"""Pins of the oracle's Adagrad local step with gradient-norm clipping (the optimiser of the
paper's experiments, Section 3.2) against library routines and closed forms."""
import numpy as np
import torch

F32 = np.float32


def _setup(oracle, K, N, seed, ld=None):
    g = np.random.Generator(np.random.PCG64(seed))
    ld = ld or N
    st = oracle.init((g.standard_normal(N) * 0.1).astype(F32), K, ld=ld)
    grad = np.zeros((K, ld), dtype=F32)
    grad[:, :N] = g.standard_normal((K, N)).astype(F32)
    accum = np.full((K, ld), 0.1, dtype=F32)
    return st, grad, accum, g


def test_matches_library_adagrad_without_clipping(oracle):
    K, N, lr, eps = 3, 500, 0.1, 1e-10
    st, grad, accum, g = _setup(oracle, K, N, 1)
    params = [torch.nn.Parameter(torch.from_numpy(st.theta[k].copy())) for k in range(K)]
    opt = torch.optim.Adagrad(params, lr=lr, lr_decay=0.0, initial_accumulator_value=0.1, eps=eps)
    for step in range(5):
        grad[:, :N] = (g.standard_normal((K, N)) * (1 + step)).astype(F32)
        for k in range(K):
            params[k].grad = torch.from_numpy(grad[k].copy())
        opt.step()
        oracle.local_adagrad(st, grad, accum, lr, eps=eps)
        for k in range(K):
            want = params[k].detach().numpy()
            assert np.allclose(st.theta[k], want, rtol=2e-6, atol=1e-7)
            assert np.allclose(accum[k], opt.state[params[k]]["sum"].numpy(), rtol=1e-6)


def test_constant_gradient_closed_form(oracle):
    """a_n = a_0 + n g^2, theta_n = theta_0 - lr * sum_j g / sqrt(a_0 + j g^2)."""
    st = oracle.init(np.zeros(4, dtype=F32), 1)
    grad = np.full((1, 4), 0.5, dtype=F32)
    accum = np.full((1, 4), 0.1, dtype=F32)
    want = 0.0
    for n in range(1, 30):
        oracle.local_adagrad(st, grad, accum, 0.1)
        want -= 0.1 * 0.5 / np.sqrt(float(F32(0.1)) + n * 0.25)
        assert abs(accum[0, 0] - (float(F32(0.1)) + n * 0.25)) < 1e-5
        assert abs(st.theta[0, 0] - want) < 2e-6 * n


def test_clipping_is_global_norm_clipping_of_the_group(oracle):
    K, N = 2, 400
    ranges = [(50, 120), (300, 390)]
    st, grad, accum, g = _setup(oracle, K, N, 2, ld=416)
    grad[0] *= 3.0                                   # worker 0: norm far above the threshold
    grad[1] *= 0.01                                  # worker 1: far below
    idx = np.r_[50:120, 300:390]
    norms = np.sqrt((grad[:, idx].astype(np.float64) ** 2).sum(axis=1))
    assert norms[0] > 10.0 > norms[1]
    a0 = accum.copy()
    oracle.local_adagrad(st, grad, accum, 0.1, clip_norm=10.0, ranges=ranges)
    geff = np.sqrt(np.maximum(accum - a0, 0))        # |g'| recovered from the accumulator
    inside = np.zeros(416, dtype=bool)
    inside[idx] = True
    # worker 0: inside the ranges the gradient was scaled to norm 10, outside it is untouched
    assert abs(np.sqrt((geff[0, inside].astype(np.float64) ** 2).sum()) - 10.0) < 1e-3
    assert np.allclose(geff[0, ~inside][:N - idx.size], np.abs(grad[0, ~inside][:N - idx.size]), rtol=1e-3, atol=1e-4)
    # worker 1: nothing is scaled
    assert np.allclose(geff[1, :N], np.abs(grad[1, :N]), rtol=2e-3, atol=1e-4)
    # against the library's clip on worker 0's group (its formula adds 1e-6 to the norm)
    p = torch.nn.Parameter(torch.zeros(idx.size))
    p.grad = torch.from_numpy(grad[0, idx].copy())
    torch.nn.utils.clip_grad_norm_([p], 10.0)
    assert np.allclose(geff[0, idx], np.abs(p.grad.numpy()), rtol=1e-3, atol=1e-4)
    assert not accum[:, N:].any() or np.all(accum[:, N:] == a0[:, N:])     # padding untouched
    assert np.array_equal(accum[:, N:], a0[:, N:]) and not st.theta[:, N:].any()


def test_clip_off_and_empty_ranges_are_the_plain_step(oracle):
    st, grad, accum, _ = _setup(oracle, 2, 100, 3)
    a, b, c = st.copy(), st.copy(), st.copy()
    acc = [accum.copy() for _ in range(3)]
    oracle.local_adagrad(a, grad, acc[0], 0.1, clip_norm=0.0, ranges=[(0, 100)])
    oracle.local_adagrad(b, grad, acc[1], 0.1, clip_norm=10.0, ranges=[])
    oracle.local_adagrad(c, grad, acc[2], 0.1, clip_norm=1e9, ranges=[(0, 100)])
    assert np.array_equal(a.theta, b.theta) and np.array_equal(a.theta, c.theta)


def test_bf16_theta_is_rounded_on_store(oracle):
    g = np.random.Generator(np.random.PCG64(9))
    x0 = oracle.f32_to_bf16((g.standard_normal(256) * 0.1).astype(F32))
    st = oracle.init(x0, 2, dtype=1)
    wide = oracle.State(2, 256, 256, 0, oracle.bf16_to_f32(st.theta), st.omega, st.delta,
                        oracle.bf16_to_f32(st.rst))
    grad = g.standard_normal((2, 256)).astype(F32)
    a1, a2 = np.full((2, 256), 0.1, dtype=F32), np.full((2, 256), 0.1, dtype=F32)
    oracle.local_adagrad(st, grad, a1, 0.1)
    oracle.local_adagrad(wide, grad, a2, 0.1)
    want = torch.from_numpy(wide.theta).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(st.theta, want) and np.array_equal(a1, a2)
