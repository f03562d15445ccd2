"""Pins of the oracle's ring topology (Definition 1) and neighbour sampler (Algorithm 1,
the neighbour-choice line)."""
import itertools

import numpy as np
import pytest

PAPER_SETTINGS = [(4, 1, 1), (8, 2, 2), (16, 3, 2)]          # (n, p, q) of Section 3.3


def ring_distance(a, b, K):
    d = abs(a - b) % K
    return min(d, K - d)


@pytest.mark.parametrize("K,p,q", PAPER_SETTINGS)
def test_candidate_list_is_definition_1(oracle, K, p, q):
    for k in range(K):
        want = [(k - d) % K for d in range(1, p + 1)] + [(k + d) % K for d in range(1, p + 1)]
        assert oracle.candidate_list(k, K, p) == want
        assert len(set(want)) == 2 * p


def test_candidate_list_wraps_without_duplicates(oracle):
    # 2p > K-1: the ring closes on itself; every other node once, never the node itself
    assert sorted(oracle.candidate_list(0, 4, 2)) == [1, 2, 3]
    assert sorted(oracle.candidate_list(2, 5, 2)) == [0, 1, 3, 4]
    assert sorted(oracle.candidate_list(1, 3, 5)) == [0, 2]
    assert oracle.candidate_list(0, 1, 3) == []
    assert oracle.candidate_list(0, 2, 1) == [1]


@pytest.mark.parametrize("K,p,q", PAPER_SETTINGS + [(8, 2, 4), (16, 3, 6), (5, 2, 3), (16, 3, 5)])
def test_draw_invariants(oracle, K, p, q):
    for rnd in range(50):
        nbr = oracle.sample_neighbors(7, rnd, K, 5, p, q)
        assert nbr.shape == (K, 5, q)
        for k in range(K):
            for i in range(5):
                row = nbr[k, i].tolist()
                assert len(set(row)) == q                       # distinct
                assert k not in row                             # never itself
                assert all(1 <= ring_distance(k, j, K) <= p for j in row)


@pytest.mark.parametrize("K,p", [(4, 1), (8, 2), (16, 3), (4, 2), (7, 3)])
def test_q_equal_to_all_neighbours_selects_them_all(oracle, K, p):
    """local-BMUF / local-MA: with q = 2p every neighbour takes part, whatever the seed."""
    c = len(oracle.candidate_list(0, K, p))
    for seed in (0, 1, 2 ** 63 + 5):
        nbr = oracle.sample_neighbors(seed, 3, K, 2, p, c)
        for k in range(K):
            for i in range(2):
                assert sorted(nbr[k, i].tolist()) == sorted(oracle.candidate_list(k, K, p))


def test_q_above_candidate_count_is_rejected(oracle):
    with pytest.raises(ValueError):
        oracle.sample_neighbors(0, 0, 4, 1, 1, 3)
    with pytest.raises(ValueError):
        oracle.sample_neighbors(0, 0, 4, 1, 2, 4)


def test_deterministic_and_keyed_by_every_index(oracle):
    a = oracle.sample_neighbors(11, 5, 16, 16, 3, 2)
    assert np.array_equal(a, oracle.sample_neighbors(11, 5, 16, 16, 3, 2))
    assert not np.array_equal(a, oracle.sample_neighbors(12, 5, 16, 16, 3, 2))        # seed
    assert not np.array_equal(a, oracle.sample_neighbors(11, 6, 16, 16, 3, 2))        # round
    assert not np.array_equal(a, oracle.sample_neighbors(11 + 2 ** 32, 5, 16, 16, 3, 2))   # seed hi
    assert not np.array_equal(a, oracle.sample_neighbors(11, 5 + 2 ** 32, 16, 16, 3, 2))   # round hi
    # different components draw independently: columns are not all the same
    assert any(not np.array_equal(a[:, 0], a[:, i]) for i in range(1, 16))
    # relative picks differ between workers too
    rel = (a - np.arange(16)[:, None, None]) % 16
    assert any(not np.array_equal(rel[0], rel[k]) for k in range(1, 16))


def test_component_index_is_global(oracle):
    full = oracle.sample_neighbors(3, 9, 8, 10, 2, 2)
    part = oracle.sample_neighbors(3, 9, 8, 4, 2, 2, comp_base=5)
    assert np.array_equal(part, full[:, 5:9])


def _chi2(counts, expected):
    counts = np.asarray(counts, dtype=np.float64)
    return float(((counts - expected) ** 2 / expected).sum())


def test_ordered_pairs_are_uniform(oracle):
    """K=16, p=3, q=2: each of the 6*5 ordered pairs of distinct neighbours equally likely."""
    K, p, q, R = 16, 3, 2, 12000
    cand = oracle.candidate_list(4, K, p)
    pairs = {pr: 0 for pr in itertools.permutations(cand, 2)}
    for rnd in range(R):
        nbr = oracle.sample_neighbors(2024, rnd, K, 1, p, q)
        pairs[tuple(nbr[4, 0].tolist())] += 1
    # 29 degrees of freedom: P(chi2 > 70) < 3e-5
    assert _chi2(list(pairs.values()), R / 30) < 70.0
    # marginal: each candidate is chosen with probability q/c
    marg = {c_: 0 for c_ in cand}
    for (a, b), n in pairs.items():
        marg[a] += n
        marg[b] += n
    assert max(abs(v / R - q / 6) for v in marg.values()) < 0.02


@pytest.mark.parametrize("K,p,q", [(4, 1, 1), (5, 2, 2), (5, 2, 3), (5, 2, 4), (4, 2, 2)])
def test_small_cases_every_ordered_tuple_equally_often(oracle, K, p, q):
    """Brute force on tiny candidate sets: all c!/(c-q)! ordered tuples occur, uniformly."""
    cand = oracle.candidate_list(0, K, p)
    tuples = {t: 0 for t in itertools.permutations(cand, q)}
    R = 400 * len(tuples)
    for rnd in range(R):
        # many components per call: each (round, component) is its own draw
        nbr = oracle.sample_neighbors(99, rnd, K, 1, p, q)
        tuples[tuple(nbr[0, 0].tolist())] += 1
    assert min(tuples.values()) > 0
    df = len(tuples) - 1
    assert _chi2(list(tuples.values()), R / len(tuples)) < df + 6 * np.sqrt(2 * df) + 10


def test_draws_beyond_four_use_further_blocks(oracle):
    """q > 4 needs a second Philox block; the first four picks must not change with q."""
    a = oracle.sample_neighbors(5, 1, 16, 3, 3, 4)
    b = oracle.sample_neighbors(5, 1, 16, 3, 3, 6)
    assert np.array_equal(a, b[:, :, :4])
    for k in range(16):
        assert sorted(b[k, 0].tolist()) == sorted(oracle.candidate_list(k, 16, 3))
