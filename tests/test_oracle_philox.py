"""Pins of the oracle's Philox4x32-10 and of the two streams built on it, against the
generator's published known-answer vectors."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_known_answer_vectors(oracle):
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


def test_counter_and_key_words_all_matter(oracle):
    base = [int(x) for x in oracle.philox4x32_10([1, 2, 3, 4], [5, 6])]
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        assert [int(x) for x in oracle.philox4x32_10(c, [5, 6])] != base
    for pos in range(2):
        k = [5, 6]
        k[pos] ^= 1
        assert [int(x) for x in oracle.philox4x32_10([1, 2, 3, 4], k)] != base


def test_sampler_stream_worked_example(oracle):
    """With seed = 'SAMP' << 32 the sampler's key is (0,0); round 0, component 0, worker 0 gives
    the all-zero counter, whose output is the first published vector.  Worked by hand for
    K=16, p=3 (candidates 15,14,13,1,2,3), q=2:
      j=0: u=0x6627e8d5, floor(u*6/2^32)=2 -> swap slots 0,2 -> pick 13
      j=1: u=0xe169c58d, floor(u*5/2^32)=4 -> swap slots 1,5 -> pick 3"""
    words = _kat()[0][2]
    assert (words[0] * 6) >> 32 == 2 and (words[1] * 5) >> 32 == 4
    nbr = oracle.sample_neighbors(0x53414D50 << 32, 0, 16, 1, 3, 2)
    assert nbr[0, 0].tolist() == [13, 3]
    # third and fourth draws continue with words 2 and 3 of the same block
    #   after two swaps the list is 13,3,15,1,2,14
    #   j=2: u=0xbc57ac4c, floor(u*4/2^32)=2 -> slot 4 (value 2);  j=3: u=0x9b00dbd8, floor(u*3/2^32)=1
    #   -> slot 4, which now holds 15
    assert (words[2] * 4) >> 32 == 2 and (words[3] * 3) >> 32 == 1
    nbr4 = oracle.sample_neighbors(0x53414D50 << 32, 0, 16, 1, 3, 4)
    assert nbr4[0, 0].tolist() == [13, 3, 2, 15]


def test_perturb_stream_worked_example(oracle):
    """With seed = 'PERT' << 32 the noise key is (0,0); elements 0 and 1 of worker 0 at step 0
    share the all-zero counter.  Element 0 sums the halves of words 0,1, element 1 those of
    words 2,3; z = (sum - 131070) / sqrt((2^32-1)/3)."""
    words = _kat()[0][2]
    halves = lambda a, b: (a & 0xFFFF) + (a >> 16) + (b & 0xFFFF) + (b >> 16)
    s0, s1 = halves(words[0], words[1]), halves(words[2], words[3])
    assert (s0, s1) == (194034, 188283)
    c = np.float32(1.0 / np.sqrt((2.0 ** 32 - 1) / 3.0))
    want = [-(np.float32(s0 - 131070) * c), -(np.float32(s1 - 131070) * c)]
    st = oracle.init(np.zeros(2, dtype=np.float32), K=1)
    oracle.local_perturb(st, seed=0x50455254 << 32, step=0, lr=1.0, sigma=1.0)
    assert st.theta[0].tolist() == [float(want[0]), float(want[1])]
    assert abs(st.theta[0, 0] + 62964 / 37837.2272) < 1e-5
