"""Parity at the full sizes of the named workloads, in the launch configuration the bench times.

The oracle cannot hold 50 GB of state, but given the neighbour table every element of a round is
independent and both sides key their random streams by global component / element index, so the
oracle replays the same calls on column ranges: one range around every component edge (plus the
head and the unaligned tail) and a few interior ranges.  On top of that, properties that hold at
any size are checked over the whole state on the device."""
import numpy as np
import pytest
import torch

from paper_1909_09010_b200 import workloads
from harness import Pair, case_of

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
