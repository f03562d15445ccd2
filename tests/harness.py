"""Shared machinery of the GPU parity tests: drives the CUDA library (through its C ABI binding)
and the CPU oracle side by side on the same seeded inputs and compares after every step.

The oracle never receives anything the CUDA path produced: it starts from the same theta_0 and
replays the same calls on its own state (whole model, or column ranges of it -- exact, because
with the neighbour table fixed every element is independent and both sides key their random
streams by global component / element index)."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import oracle
from paper_1909_09010_b200 import binding, workloads

# tolerance of the parity bar: |gpu - ref| <= ATOL + RTOL * |ref| per element (fp32 state);
# bf16-stored theta: 1e-2 relative.  The design target is bit equality, also asserted.
RTOL, ATOL = 1e-6, 1e-7
BF16_RTOL = 1e-2


@dataclass
class Case:
    K: int
    offsets: tuple
    p: int
    q: int
    eta: float = 0.9
    zeta: float = 1.0
    dtype: int = 0
    seed: int = 0
    mode: int = 0
    periods: tuple | None = None
    ld: int | None = None

    @property
    def N(self):
        return int(self.offsets[-1])

    @property
    def m(self):
        return len(self.offsets) - 1


def case_of(w: workloads.Workload, **over) -> Case:
    c = Case(K=w.K, offsets=w.offsets, p=w.p, q=w.q, eta=w.eta, zeta=w.zeta, dtype=w.dtype,
             seed=w.seed)
    for k, v in over.items():
        setattr(c, k, v)
    return c


def tdtype(dtype):
    return torch.float32 if dtype == 0 else torch.bfloat16


def to_numpy(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_numpy(a: np.ndarray, dtype, device) -> torch.Tensor:
    if dtype == 1:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)
    return torch.from_numpy(a.copy()).to(device)


class Pair:
    """GPU context + oracle state(s) over the same case."""

    def __init__(self, case: Case, theta0: np.ndarray | torch.Tensor, slices=None, tuning=None,
                 device="cuda:0"):
        self.case, self.device = case, torch.device(device)
        K, N = case.K, case.N
        self.ld = case.ld or workloads.padded_ld(N)
        dt = tdtype(case.dtype)
        self.theta = torch.zeros((K, self.ld), dtype=dt, device=self.device)
        self.omega = torch.zeros((K, self.ld), dtype=torch.float32, device=self.device)
        self.delta = torch.zeros((K, self.ld), dtype=torch.float32, device=self.device)
        self.g = binding.Gbmuf(self.theta, self.omega, self.delta, K=K, N=N, ld=self.ld, p=case.p,
                               q=case.q, eta=case.eta, zeta=case.zeta, seed=case.seed,
                               mode=case.mode, theta_dtype=case.dtype,
                               device=self.device.index or 0)
        if tuning:
            self.g.set_tuning(**tuning)
        self.g.set_partition(case.offsets, case.periods)
        if isinstance(theta0, np.ndarray):
            theta0_dev = from_numpy(theta0, case.dtype, self.device)
        else:
            theta0_dev = theta0
        self.theta0_dev = theta0_dev
        self.g.init(theta0_dev)
        # oracle side: one State per column range
        self.slices = slices or [(0, N)]
        self.shards, self.states = [], []
        for a, b in self.slices:
            sh = workloads.shard_columns(case.offsets, a, b)
            t0 = to_numpy(theta0_dev[a:b]) if not isinstance(theta0, np.ndarray) else theta0[a:b]
            ld = self.ld if (a, b) == (0, N) else None
            self.shards.append(sh)
            self.states.append(oracle.init(np.ascontiguousarray(t0), K, ld=ld, dtype=case.dtype))

    # ---------------------------------------------------------------- the same calls on both sides
    def perturb(self, step, lr, sigma, nsteps=1):
        self.g.local_perturb(step, lr, sigma, nsteps)
        for sh, st in zip(self.shards, self.states):
            oracle.local_perturb(st, self.case.seed, step, lr, sigma, nsteps, elem_base=sh.col0)

    def add_drift(self, drift: np.ndarray):
        """theta^k += drift[k] (fp32 replicas), an input both sides receive."""
        assert self.case.dtype == 0
        self.theta[:, :self.case.N] += torch.from_numpy(drift).to(self.device)
        for (a, b), st in zip(self.slices, self.states):
            st.theta[:, :b - a] += drift[:, a:b]

    def due(self, rnd, mask=None):
        if mask is not None:
            return [bool(x) for x in mask]
        per = self.case.periods or [1] * self.case.m
        return [rnd % h == 0 for h in per]

    def sync(self, rnd, mask=None):
        c = self.case
        self.g.sync_round(rnd, mask)
        due = self.due(rnd, mask)
        for sh, st in zip(self.shards, self.states):
            nbr = oracle.sample_neighbors(c.seed, rnd, c.K, sh.m, c.p, c.q, comp_base=sh.comp_base)
            flags = due[sh.comp_base:sh.comp_base + sh.m]
            oracle.sync_round(st, sh.offsets, nbr, c.eta, c.zeta, mode=c.mode, sync=flags)

    def check_neighbors(self, rnd):
        c = self.case
        got = self.g.get_neighbors(rnd)
        want = oracle.sample_neighbors(c.seed, rnd, c.K, c.m, c.p, c.q)
        assert got.dtype == np.int32 and got.shape == want.shape
        assert np.array_equal(got, want), f"neighbour table differs in round {rnd}"

    # ---------------------------------------------------------------- comparison
    def compare(self, what="", exact=True):
        torch.cuda.synchronize(self.device)
        assert self.g.device_status() == 0
        c = self.case
        for (a, b), st in zip(self.slices, self.states):
            whole = (a, b) == (0, c.N)
            cols = slice(0, self.ld) if whole else slice(a, b)
            got_t = to_numpy(self.theta[:, cols])
            got_o = to_numpy(self.omega[:, cols])
            got_d = to_numpy(self.delta[:, cols])
            for name, got, ref in (("omega", got_o, st.omega), ("delta", got_d, st.delta)):
                bad = np.abs(got.astype(np.float64) - ref) > ATOL + RTOL * np.abs(ref)
                assert not bad.any(), f"{what} {name} cols[{a},{b}): {int(bad.sum())} outside tolerance"
                if exact:
                    ne = got.view(np.uint32) != ref.view(np.uint32)
                    assert not ne.any(), f"{what} {name} cols[{a},{b}): {int(ne.sum())} not bit-equal"
            if c.dtype == 0:
                bad = np.abs(got_t.astype(np.float64) - st.theta) > ATOL + RTOL * np.abs(st.theta)
                assert not bad.any(), f"{what} theta cols[{a},{b}): {int(bad.sum())} outside tolerance"
                if exact:
                    ne = got_t.view(np.uint32) != st.theta.view(np.uint32)
                    assert not ne.any(), f"{what} theta cols[{a},{b}): {int(ne.sum())} not bit-equal"
            else:
                gf, rf = oracle.bf16_to_f32(got_t), oracle.bf16_to_f32(st.theta)
                bad = np.abs(gf.astype(np.float64) - rf) > 1e-7 + BF16_RTOL * np.abs(rf)
                assert not bad.any(), f"{what} bf16 theta cols[{a},{b}): {int(bad.sum())} outside tolerance"
                if exact:
                    assert np.array_equal(got_t, st.theta), f"{what} bf16 theta cols[{a},{b}) not bit-equal"

    def close(self):
        self.g.destroy()


def random_theta0(N, seed, dtype=0, sigma=0.1):
    g = np.random.Generator(np.random.PCG64(seed))
    x = (g.standard_normal(N, dtype=np.float32) * np.float32(sigma)).astype(np.float32)
    return oracle.f32_to_bf16(x) if dtype == 1 else x


# ------------------------------------------------------------------------------------------------
# one whole round of a large state, every element, checked slice by slice
# ------------------------------------------------------------------------------------------------
def check_round_every_element(case: Case, rnd, pre, post, mask=None, width=None, threads=None,
                              what=""):
    """Compares one synchronisation round over the WHOLE state with the oracle, bit for bit.

    `pre` = (theta, omega, delta) device tensors as they were before the round, `post` the same
    after it.  In `pre`, omega may be a 1-D tensor [N] that stands for K identical rows and delta
    may be None for zeros (the state right after the initialisation line of Algorithm 1).  The
    columns are cut into ranges of `width` (default: 2^26 replica-parameters per range); each range goes to the host, the oracle runs the round
    on it alone (exact: with the neighbour table fixed every column is independent, and the draws
    are keyed by the global component index), and the result must equal the same range of
    `post`.  The block-start value the oracle stores is what the previous synchronisation left:
    store(fl(omega + fl(eta * Delta))) of the pre-round values.  Ranges are checked by a few
    threads (the oracle releases the interpreter while it computes)."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    K, N = case.K, case.N
    th0, om0, de0 = pre
    th1, om1, de1 = post
    per = case.periods or [1] * case.m
    due = [bool(x) for x in mask] if mask is not None else [rnd % h == 0 for h in per]
    eta32 = np.float32(case.eta)

    def host(t, a, b):
        return to_numpy(t[:, a:b])

    def one(rng):
        a, b = rng
        n = b - a
        sh = workloads.shard_columns(case.offsets, a, b)
        theta = np.ascontiguousarray(host(th0, a, b))
        if om0.dim() == 1:
            row = to_numpy(om0[a:b])
            row = oracle.bf16_to_f32(row) if row.dtype == np.uint16 else row
            omega = np.ascontiguousarray(np.broadcast_to(row.astype(np.float32), (K, n)))
        else:
            omega = np.ascontiguousarray(host(om0, a, b))
        delta = np.zeros((K, n), dtype=np.float32) if de0 is None else np.ascontiguousarray(host(de0, a, b))
        r32 = omega + eta32 * delta                       # two roundings, as the filter wrote it
        rst = oracle.f32_to_bf16(r32) if case.dtype == 1 else r32
        st = oracle.State(K, n, n, case.dtype, theta, omega, delta, np.ascontiguousarray(rst))
        nbr = oracle.sample_neighbors(case.seed, rnd, K, sh.m, case.p, case.q, comp_base=sh.comp_base)
        oracle.sync_round(st, sh.offsets, nbr, case.eta, case.zeta, mode=case.mode,
                          sync=due[sh.comp_base:sh.comp_base + sh.m])
        bad = []
        for name, got, ref in (("theta", host(th1, a, b), st.theta), ("omega", host(om1, a, b), st.omega),
                               ("delta", host(de1, a, b), st.delta)):
            if case.mode == 1 and name != "theta":
                continue
            ne = got.view(np.uint8) != ref.view(np.uint8)
            if ne.any():
                bad.append(f"{what} {name} cols[{a},{b}): {int(ne.any(axis=0).sum() if ne.ndim == 2 else ne.sum())} "
                           "columns not bit-equal")
        return bad

    width = width or max(1 << 12, ((1 << 26) // K) // 32 * 32)
    ranges = [(a, min(N, a + width)) for a in range(0, N, width)]
    threads = threads or max(1, min(6, (os.cpu_count() or 2) - 1))
    problems = []
    with ThreadPoolExecutor(max_workers=threads) as pool:
        for bad in pool.map(one, ranges):
            problems += bad
    assert not problems, "; ".join(problems[:5])
    return len(ranges)
