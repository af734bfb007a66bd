"""Pins of the oracle's comparison permutations (absmax order, zigzag dealing) and their statistic (CPU only)."""
import numpy as np

from paper_2601_22347_b200 import inputs


def test_chan_abs_max_is_the_column_maximum(oracle):
    bits, _ = inputs.student_t_outliers(37, 256, 3.0, 4, 100.0, seed=1)
    ref = np.abs(inputs.bf16_to_f64(bits)).max(axis=0)
    assert np.array_equal(oracle.chan_abs_max(bits), ref)
    one = np.zeros((3, 32), np.float32); one[1, 5] = -7.0
    got = oracle.chan_abs_max(inputs.f32_to_bf16_bits(one))
    assert got[5] == 7.0 and got.sum() == 7.0


def test_absmax_order_by_hand_and_against_a_library_sort(oracle):
    stat = np.array([3.0, 9.0, 1.0, 9.0, 0.0, 4.0])
    assert oracle.absmax_perm(stat).tolist() == [1, 3, 5, 0, 2, 4]          # equal values: lower channel first
    rng = np.random.default_rng(2)
    s = rng.exponential(size=500)
    s[rng.integers(0, 500, 40)] = s[0]
    ref = np.argsort(-s, kind="stable")
    assert np.array_equal(oracle.absmax_perm(s), ref)


def test_zigzag_by_hand(oracle):
    # d = 8, b = 2 -> 4 blocks; visiting order 7 6 5 4 | 3 2 1 0 by value
    stat = np.arange(8, dtype=np.float64)
    perm = oracle.zigzag_perm(stat, 2)
    # round 0 goes to blocks 0,1,2,3; round 1 comes back 3,2,1,0: block j = (7 - j, j)
    assert perm.tolist() == [7, 0, 6, 1, 5, 2, 4, 3]
    # three rounds: the third goes forward again
    stat = np.arange(6, dtype=np.float64)
    assert oracle.zigzag_perm(stat, 3).tolist() == [5, 2, 1, 4, 3, 0]


def test_zigzag_invariants(oracle):
    rng = np.random.default_rng(3)
    d, b = 512, 16
    s = rng.exponential(size=d) * np.where(rng.random(d) < 0.05, 50.0, 1.0)
    perm = oracle.zigzag_perm(s, b)
    assert sorted(perm.tolist()) == list(range(d))
    n = d // b
    rank = np.empty(d, np.int64)
    rank[np.argsort(-s, kind="stable")] = np.arange(d)
    blocks = perm.reshape(n, b)
    # slot r of every block holds a channel of round r (ranks r n .. r n + n - 1), each round once per block
    assert np.array_equal(rank[blocks] // n, np.tile(np.arange(b), (n, 1)))
    # within a round the ranks run forwards over the blocks in even rounds, backwards in odd ones
    assert np.array_equal(rank[blocks[:, 0]], np.arange(n))
    assert np.array_equal(rank[blocks[:, 1]], 2 * n - 1 - np.arange(n))
    # pairs of rounds balance: rank sums of rounds 0 and 1 are the same for every block
    assert len(set((rank[blocks[:, 0]] + rank[blocks[:, 1]]).tolist())) == 1
    # the largest block maximum sum is no larger than under the absmax order, which packs the largest together
    am = oracle.absmax_perm(s).reshape(n, b)
    assert s[blocks].sum(axis=1).max() <= s[am].sum(axis=1).max()
