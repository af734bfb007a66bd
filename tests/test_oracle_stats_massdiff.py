"""Pins for the oracle's calibration statistic and the greedy mass-diffusion permutation.

Checked against: direct numpy reductions, the identities the block proposition and its
corollary state, brute force over all block assignments on tiny inputs, and the
algorithm's own invariants (valid permutation, full blocks, running sums).
"""
import itertools

import numpy as np
import pytest

from paper_2601_22347_b200 import inputs


def test_stats_match_numpy_reductions(oracle):
    w, _ = inputs.gaussian_outliers(32, 256, 4, 50.0, seed=21)
    perm = inputs.random_perm(256, 22)
    x = np.abs(inputs.bf16_to_f64(w))
    for b in (16, 64):
        cas, blm, tmx = oracle.block_l1_stats(w, perm, b)
        assert np.allclose(cas, x.sum(axis=0), rtol=1e-14)          # original channel order
        L = x[:, perm].reshape(32, 256 // b, b).sum(axis=2)          # ||(x P)_{j}||_1
        assert np.allclose(blm, L.mean(axis=0), rtol=1e-14)
        assert np.allclose(tmx, L.max(axis=1), rtol=1e-14)
        # total mass is the same however it is sliced
        assert np.isclose(cas.sum(), blm.sum() * 32, rtol=1e-12)


def test_corollary_block_size_growth(oracle):
    """Z(b;X) = max_j ||X_{j}||_1 / sqrt(b) satisfies Z(k b') <= sqrt(k) Z(b')."""
    w, _ = inputs.student_t_outliers(64, 512, 3.0, 8, 100.0, seed=23)
    Z = {b: oracle.block_l1_stats(w, None, b)[2] / np.sqrt(b) for b in (16, 32, 64, 128)}
    for bp in (16, 32, 64):
        for b in (32, 64, 128):
            if b > bp:
                assert np.all(Z[b] <= np.sqrt(b / bp) * Z[bp] * (1 + 1e-12))


def test_delta_lies_between_one_over_b_and_one(oracle):
    """delta_{j} = ||X_{j}||_1 / (b ||X_{j}||_inf) is in [1/b, 1]; the bound of the block
    proposition, max_j ||X_{j}||_1/sqrt(b), dominates the rotated row's max."""
    w, _ = inputs.laplace_outliers(16, 512, 2, 200.0, seed=24)
    x = np.abs(inputs.bf16_to_f64(w))
    for b in (16, 128):
        tmx = oracle.block_l1_stats(w, None, b)[2]
        blk = x.reshape(16, 512 // b, b)
        j = blk.sum(axis=2).argmax(axis=1)
        inf = blk.max(axis=2)[np.arange(16), j]
        delta = tmx / (b * inf)
        assert np.all((delta >= 1 / b - 1e-15) & (delta <= 1 + 1e-15))
        y = oracle.rotate(w, None, b)
        assert np.all(np.abs(y).max(axis=1) <= tmx / np.sqrt(b) * (1 + 1e-12))


def block_objective(a, perm, b):
    return a[perm].reshape(-1, b).sum(axis=1).max()


def test_massdiff_is_a_permutation_with_full_blocks(oracle):
    rng = np.random.default_rng(31)
    a = rng.exponential(size=256)
    perm = oracle.massdiff_perm(a, 16)
    assert sorted(perm.tolist()) == list(range(256))


def test_massdiff_hand_example(oracle):
    # masses 9 8 7 6 5 4 3 2 (already sorted), b = 4, two blocks
    # 9->B0, 8->B1, 7->B1(8<9), 6->B0(9<15), 5->B0(15=15 tie: lower index), 4->B1(15<20),
    # 3->B1(19<20; B1 now full), 2->B0
    a = np.array([9, 8, 7, 6, 5, 4, 3, 2], np.float64)
    perm = oracle.massdiff_perm(a, 4)
    assert perm.tolist() == [0, 3, 4, 7, 1, 2, 5, 6]


def test_massdiff_sort_is_descending_with_stable_ties(oracle):
    a = np.array([1, 5, 5, 1, 5, 1, 1, 5], np.float64)
    perm = oracle.massdiff_perm(a, 2)     # 4 blocks; the four 5s open the four blocks in index order
    assert perm.reshape(4, 2)[:, 0].tolist() == [1, 2, 4, 7]
    assert perm.reshape(4, 2)[:, 1].tolist() == [0, 3, 5, 6]


@pytest.mark.parametrize("b", [2, 4])
def test_massdiff_against_brute_force_optimum(oracle, b):
    rng = np.random.default_rng(32)
    d = 8
    worst_gap = 0.0
    for _ in range(20):
        a = rng.exponential(size=d) * np.where(rng.random(d) < 0.25, 20.0, 1.0)
        greedy = block_objective(a, oracle.massdiff_perm(a, b), b)
        best = min(block_objective(a, np.array(p), b) for p in itertools.permutations(range(d)))
        assert greedy >= best - 1e-12
        # the paper claims no ratio; 4/3 is the classical bound of this greedy without the
        # capacity constraint, used here only as a sanity ceiling
        assert greedy <= best * 1.5
        worst_gap = max(worst_gap, greedy / best)
    assert worst_gap < 1.5


def test_massdiff_beats_identity_and_random_on_adjacent_outliers(oracle):
    w, ch = inputs.gaussian_outliers(64, 512, 0, 1.0, seed=33)
    x = inputs.bf16_bits_to_f32(w)
    x[:, 32:40] *= 60.0                       # eight adjacent outlier channels: one block holds them all
    w = inputs.f32_to_bf16_bits(x)
    b = 32
    cas, blm_id, tmx_id = oracle.block_l1_stats(w, None, b)
    perm = oracle.massdiff_perm(cas, b)
    _, blm_md, tmx_md = oracle.block_l1_stats(w, perm, b)
    _, blm_rn, tmx_rn = oracle.block_l1_stats(w, inputs.random_perm(512, 34), b)
    assert blm_md.max() < blm_id.max() and blm_md.max() <= blm_rn.max()
    assert tmx_md.mean() < tmx_id.mean()
    # the greedy's running sums are the per-block means recomputed under the returned perm
    assert np.allclose(cas[perm].reshape(-1, b).sum(axis=1) / 64, blm_md, rtol=1e-12)
    # balancing block l1 mass lowers the post-rotation range the quantiser sees
    y_id = oracle.rotate(w, None, b)
    y_md = oracle.rotate(w, perm, b)
    assert np.abs(y_md).max(axis=1).mean() < np.abs(y_id).max(axis=1).mean()
