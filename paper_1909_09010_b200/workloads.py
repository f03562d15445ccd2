"""Synthetic workloads: LSTM-LM-shaped parameter layouts, their component partitions, seeded
input generators and the element-range shard planner.

This module holds none of the method's arithmetic (no averaging, no block-momentum filter, no
neighbour sampling, no noise generator).  It only says how large things are, where component
boundaries fall and how the seeded starting values are drawn, so that the CUDA library, the CPU
checker and the bench can all be fed the same inputs.

Flat layout of one replica: ``[embedding | LSTM_1 | ... | LSTM_L | softmax W | softmax b]`` with
embedding V*h, each LSTM layer 4h*2h weights + 4h biases, softmax h*V + V.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np

F32, BF16 = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    K: int                 # workers n
    vocab: int
    hidden: int
    layers: int
    p: int                 # symmetric degree of the ring
    q: int                 # gossip neighbours
    eta: float
    zeta: float
    dtype: int             # storage type of theta
    seed: int
    rounds: int
    local_steps: int       # synthetic local steps before each round
    lr: float
    sigma: float           # std of the synthetic gradient noise
    offsets: tuple = field(repr=False, default=())
    drift_sigma: float = 0.0   # one-off per-replica drift added before the first round
    init_sigma: float = 0.1
    mode: int = 0          # 0 gossip-BMUF, 1 gossip-MA (Algorithm 1's other branch)

    @property
    def N(self) -> int:
        return int(self.offsets[-1])

    @property
    def m(self) -> int:
        return len(self.offsets) - 1

    @property
    def ld(self) -> int:
        return padded_ld(self.N)


def padded_ld(N: int) -> int:
    """Row stride: N rounded up to a multiple of 32 elements (rows start 128-byte aligned)."""
    return max(32, (N + 31) // 32 * 32)


def lstm_lm_layout(vocab: int, hidden: int, layers: int):
    """Sizes of the named blocks of the flat parameter vector, in order."""
    blocks = [("emb", vocab * hidden)]
    for l in range(layers):
        blocks.append((f"lstm{l + 1}", 4 * hidden * 2 * hidden + 4 * hidden))
    blocks.append(("softmax", hidden * vocab + vocab))
    return blocks


def _starts(blocks):
    out, at = {}, 0
    for name, n in blocks:
        out[name] = (at, at + n)
        at += n
    return out, at


def _even_row_shards(begin: int, rows: int, row_len: int, shards: int, end: int):
    """Cut `rows` rows of `row_len` into `shards` near-equal runs of whole rows; the last shard
    runs to `end` (so a trailing bias joins it)."""
    base, extra = divmod(rows, shards)
    cuts, at = [], begin
    for s in range(shards):
        cuts.append(at)
        at += (base + (1 if s < extra else 0)) * row_len
    return cuts, end


def partition_tiny():
    blocks = lstm_lm_layout(1000, 128, 2)
    off, at = [0], 0
    for _, n in blocks:
        at += n
        off.append(at)
    return tuple(off)


def partition_mid():
    """Each of emb / LSTM1 / LSTM2 / softmax cut into two contiguous row blocks (halves rounded
    to whole rows; biases ride with the second half)."""
    V, h = 10000, 512
    st, N = _starts(lstm_lm_layout(V, h, 2))
    cuts = []
    for name, rows, row_len in (("emb", V, h), ("lstm1", 4 * h, 2 * h), ("lstm2", 4 * h, 2 * h),
                                ("softmax", V, h)):
        b, e = st[name]
        c, _ = _even_row_shards(b, rows, row_len, 2, e)
        cuts += c
    return tuple(cuts + [N])


def partition_wikitext103():
    """16 components shaped like the paper's split (Section 3.2): 8 even row shards of the
    embedding, the two recurrent layers as one group each, and 6 near-equal softmax blocks
    (edges at multiples of 4 elements; the last block takes the remainder and the bias)."""
    V, h = 267735, 512
    st, N = _starts(lstm_lm_layout(V, h, 2))
    cuts, _ = _even_row_shards(st["emb"][0], V, h, 8, st["emb"][1])
    cuts += [st["lstm1"][0], st["lstm2"][0]]
    b, e = st["softmax"]
    blk = ((e - b) // 6) // 4 * 4
    cuts += [b + j * blk for j in range(6)]
    return tuple(cuts + [N])


def partition_sweep(C: int):
    """Embedding whole, softmax whole, each LSTM layer cut into (C-2)/2 components: 64 KB
    (16,384-element) slices followed by one remainder."""
    assert C >= 4 and C % 2 == 0
    V, h = 267735, 512
    st, N = _starts(lstm_lm_layout(V, h, 2))
    per = (C - 2) // 2
    cuts = [st["emb"][0]]
    for name in ("lstm1", "lstm2"):
        b, e = st[name]
        assert (per - 1) * 16384 < e - b
        cuts += [b + j * 16384 for j in range(per)]
    cuts.append(st["softmax"][0])
    return tuple(cuts + [N])


def partition_longrun():
    """64 components: embedding in 24 even row shards, each of 4 LSTM layers in 4 gate-row
    blocks (the bias rides with the last), softmax in 24 even row shards (bias with the last)."""
    V, h, L = 100000, 1024, 4
    st, N = _starts(lstm_lm_layout(V, h, L))
    cuts, _ = _even_row_shards(st["emb"][0], V, h, 24, st["emb"][1])
    for l in range(L):
        b, e = st[f"lstm{l + 1}"]
        c, _ = _even_row_shards(b, 4 * h, 2 * h, 4, e)
        cuts += c
    c, _ = _even_row_shards(st["softmax"][0], V, h, 24, st["softmax"][1])
    cuts += c
    return tuple(cuts + [N])


def get(name: str, **over) -> Workload:
    """The named workload.  ``sweep`` takes C=, q=, eta= overrides."""
    if name == "tiny":
        w = Workload("tiny", K=4, vocab=1000, hidden=128, layers=2, p=1, q=1, eta=0.9, zeta=1.0,
                     dtype=F32, seed=0, rounds=3, local_steps=0, lr=0.0, sigma=0.0,
                     offsets=partition_tiny(), drift_sigma=0.01)
    elif name == "mid":
        w = Workload("mid", K=8, vocab=10000, hidden=512, layers=2, p=2, q=2, eta=0.9, zeta=1.0,
                     dtype=F32, seed=1, rounds=10, local_steps=4, lr=0.1, sigma=1e-3,
                     offsets=partition_mid())
    elif name == "wikitext103":
        w = Workload("wikitext103", K=16, vocab=267735, hidden=512, layers=2, p=3, q=2, eta=0.875,
                     zeta=1.0, dtype=F32, seed=2, rounds=20, local_steps=1, lr=0.1, sigma=1e-3,
                     offsets=partition_wikitext103())
    elif name == "sweep":
        C = over.pop("C", 16)
        w = Workload(f"sweep_C{C}", K=8, vocab=267735, hidden=512, layers=2, p=2,
                     q=over.pop("q", 2), eta=over.pop("eta", 0.9), zeta=1.0, dtype=F32, seed=3,
                     rounds=5, local_steps=1, lr=0.1, sigma=1e-3, offsets=partition_sweep(C))
    elif name == "longrun":
        w = Workload("longrun", K=16, vocab=100000, hidden=1024, layers=4, p=3, q=3, eta=0.9,
                     zeta=1.0, dtype=BF16, seed=4, rounds=100, local_steps=8, lr=0.1, sigma=1e-3,
                     offsets=partition_longrun())
    elif name == "profile16":
        # the wikitext-103-shaped replica set cut down to 2^24+5 columns (3.2 GB of state): the
        # case profiler captures run on
        n = (1 << 24) + 5
        cuts = tuple(int(x) // 4 * 4 for x in np.linspace(0, n, 17)[:-1]) + (n,)
        w = Workload("profile16", K=16, vocab=0, hidden=0, layers=0, p=3, q=2, eta=0.875, zeta=1.0,
                     dtype=F32, seed=2, rounds=4, local_steps=1, lr=0.1, sigma=1e-3, offsets=cuts)
    elif name == "profile16bf":
        # the long-run mixed-precision replica set (bf16 theta) cut down to 2^24+5 columns
        n = (1 << 24) + 5
        cuts = tuple(int(x) // 8 * 8 for x in np.linspace(0, n, 65)[:-1]) + (n,)
        w = Workload("profile16bf", K=16, vocab=0, hidden=0, layers=0, p=3, q=3, eta=0.9, zeta=1.0,
                     dtype=BF16, seed=4, rounds=4, local_steps=1, lr=0.1, sigma=1e-3, offsets=cuts)
    elif name == "profile64":
        # 64 workers on the ring the paper's rule gives them (p = log2(64) - 1 = 5), 2^22+5 columns
        # (3.2 GB of state): the many-worker case profiler captures run on
        n = (1 << 22) + 5
        cuts = tuple(int(x) // 4 * 4 for x in np.linspace(0, n, 17)[:-1]) + (n,)
        w = Workload("profile64", K=64, vocab=0, hidden=0, layers=0, p=5, q=2, eta=0.875, zeta=1.0,
                     dtype=F32, seed=2, rounds=4, local_steps=1, lr=0.1, sigma=1e-3, offsets=cuts)
    else:
        raise KeyError(name)
    return replace(w, **over) if over else w


SWEEP_POINTS = [(C, q, eta) for C in (4, 16, 64, 256) for q in (1, 2, 4) for eta in (0.5, 0.9)]


# ------------------------------------------------------------------------------------------------
# seeded starting values
# ------------------------------------------------------------------------------------------------
def theta0_numpy(w: Workload, n: int | None = None) -> np.ndarray:
    """theta_0 ~ N(0, init_sigma^2) i.i.d., fp32, from a PCG64 stream keyed by the seed."""
    n = w.N if n is None else n
    g = np.random.Generator(np.random.PCG64(w.seed))
    return (g.standard_normal(n, dtype=np.float32) * np.float32(w.init_sigma)).astype(np.float32)


def drift_numpy(w: Workload, n: int | None = None) -> np.ndarray:
    """Per-replica drift [K][n] ~ N(0, drift_sigma^2), fp32 (tiny workload only)."""
    n = w.N if n is None else n
    g = np.random.Generator(np.random.PCG64([w.seed, 0xD21F7]))
    return (g.standard_normal((w.K, n), dtype=np.float32) * np.float32(w.drift_sigma)).astype(
        np.float32)


def theta0_torch(w: Workload, device, n: int | None = None):
    """theta_0 drawn on `device` with a seeded torch generator (large workloads)."""
    import torch
    n = w.N if n is None else n
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    t = torch.empty(n, dtype=torch.float32, device=device)
    t.normal_(0.0, w.init_sigma, generator=g)
    return t


def replica_noise_torch(w: Workload, k: int, step: int, n: int, device):
    """Standard-normal input noise [n] for worker k's local step `step`, drawn on `device` from a
    torch generator seeded by (workload seed, k, step).  Used where each worker is a process of
    its own and applies its local step with library tensor operations; a checker that wants the
    same input calls this with the same arguments on the same kind of device."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((w.seed * 1_000_003 + k) * 1_000_003 + step)
    t = torch.empty(n, dtype=torch.float32, device=device)
    t.normal_(0.0, 1.0, generator=g)
    return t


# ------------------------------------------------------------------------------------------------
# element-range shards: given the neighbour table every element is independent, so a column
# range [c0, c1) of all K replicas can be processed on its own as long as components keep their
# global index and elements keep their global position.
# ------------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Shard:
    col0: int              # first global column
    col1: int              # one past the last
    comp_base: int         # global index of the first component that intersects the range
    offsets: tuple         # local offsets (relative to col0) of the intersecting components

    @property
    def n(self) -> int:
        return self.col1 - self.col0

    @property
    def m(self) -> int:
        return len(self.offsets) - 1


def shard_columns(offsets, col0: int, col1: int) -> Shard:
    """Partition of the column range [col0, col1) induced by the global `offsets`."""
    offsets = [int(x) for x in offsets]
    N = offsets[-1]
    assert 0 <= col0 < col1 <= N
    first = max(i for i in range(len(offsets) - 1) if offsets[i] <= col0)
    local, i = [0], first
    while offsets[i + 1] < col1:
        local.append(offsets[i + 1] - col0)
        i += 1
    local.append(col1 - col0)
    return Shard(col0, col1, first, tuple(local))


def shard_even(offsets, world: int, rank: int, align: int = 32) -> Shard:
    """Rank `rank`'s share when the columns are cut into `world` near-equal contiguous ranges
    whose interior edges fall on multiples of `align` elements."""
    N = int(offsets[-1])
    edges = [min(N, (N * r // world + align - 1) // align * align) for r in range(world)] + [N]
    assert edges[rank] < edges[rank + 1], "more ranks than aligned column groups"
    return shard_columns(offsets, edges[rank], edges[rank + 1])


def edge_slices(offsets, width: int, count: int | None = None):
    """Column ranges of about `width` elements centred on component edges (plus the head and the
    unaligned tail): the places where a sliced check of a large workload should look."""
    N = int(offsets[-1])
    marks = sorted(set(int(x) for x in offsets))
    out = []
    for x in marks:
        a = max(0, min(N - width, x - width // 2))
        b = min(N, a + width)
        if not out or a >= out[-1][1]:
            out.append((a, b))
        elif b > out[-1][1]:
            out[-1] = (out[-1][0], b)
    if count is not None and len(out) > count:
        idx = np.linspace(0, len(out) - 1, count).round().astype(int)
        out = [out[i] for i in sorted(set(idx))]
    return out
