"""Pins for the oracle's per-token diagnostics (the quantities behind the paper's figures on delta, on the
block bound and on the bound versus the quantization error).

Checked against: hand-computed small cases, closed forms (one-hot rows, rows of H), the inequalities of the two
propositions and of Sec. 3, and a second derivation composed from other oracle calls plus numpy.
"""
import numpy as np
import scipy.linalg

from paper_2601_22347_b200 import inputs


def bits_of(a):
    bits = inputs.f32_to_bf16_bits(np.asarray(a, np.float32))
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), np.asarray(a, np.float32))
    return bits


def test_hand_computed_two_by_two(oracle):
    # x = (3, 1), b = 2: y = (4, 2)/sqrt(2); step = y0/7; y1/step = 3.5 rounds to 4 (even): error = step/2
    out = oracle.token_diagnostics(bits_of([[3.0, 1.0]]), None, 2)[0]
    s = (4 / np.sqrt(2)) / 7
    assert np.allclose(out, [3.0, 4.0, 4.0, 4 / np.sqrt(2), s / 2], rtol=1e-14)
    # same row through the swap permutation: y = (4, -2)/sqrt(2); -3.5 rounds to -4: the same error
    out = oracle.token_diagnostics(bits_of([[3.0, 1.0]]), np.array([1, 0], np.int32), 2)[0]
    assert np.allclose(out, [3.0, 4.0, 4.0, 4 / np.sqrt(2), s / 2], rtol=1e-14)
    # b = 1: no rotation; y = x; 1/(3/7) = 2.33 -> 2: error |1 - 6/7|
    out = oracle.token_diagnostics(bits_of([[3.0, 1.0]]), None, 1)[0]
    assert np.allclose(out, [3.0, 4.0, 3.0, 3.0, 1 - 6 / 7], rtol=1e-13)


def test_one_hot_rows_and_rows_of_h(oracle):
    d, b = 256, 32
    x = np.zeros((3, d), np.float32)
    x[0, 77] = -2.5                       # one-hot: every |y| in its block is 2.5/sqrt(b): codes +-7, no error
    H = scipy.linalg.hadamard(b)
    x[1, 64:96] = 0.5 * H[5]              # a row of H in block 2: y = 0.5 sqrt(b) e_5: bound attained, no error
    out = oracle.token_diagnostics(bits_of(x), None, b)
    assert np.allclose(out[0], [2.5, 2.5, 2.5, 2.5 / np.sqrt(b), 0.0], atol=1e-13)
    assert np.allclose(out[1], [0.5, 16.0, 16.0, 0.5 * np.sqrt(b), 0.0], atol=1e-13)
    assert np.isclose(out[1, 3], out[1, 2] / np.sqrt(b))          # equality in the block proposition
    assert np.array_equal(out[2], np.zeros(5))                     # zero row


def test_inequalities_of_the_propositions(oracle):
    w, _ = inputs.laplace_outliers(48, 1024, 4, 200.0, seed=61)
    d = 1024
    for b, perm in ((16, None), (64, inputs.random_perm(d, 62)), (1024, None)):
        o = oracle.token_diagnostics(w, perm, b)
        delta = o[:, 1] / (d * o[:, 0])
        assert np.all((delta >= 1 / d) & (delta <= 1))                              # delta in [1/d, 1]
        assert np.all(o[:, 3] <= o[:, 2] / np.sqrt(b) * (1 + 1e-12))                # ||y||_inf <= max_j ||x_j||_1 / sqrt(b)
        assert np.all(o[:, 2] / b >= o[:, 0] / b * (1 - 1e-12))                     # normalised bound >= 1/b
        assert np.all(o[:, 4] <= np.sqrt(d) * (o[:, 3] / 7) / 2 * (1 + 1e-12))      # Sec. 3: error <= sqrt(d) step / 2
        if b == d:
            assert np.allclose(o[:, 2], o[:, 1], rtol=1e-14)                        # one block: its l1 is the row's
            assert np.all(o[:, 3] <= delta * np.sqrt(d) * o[:, 0] * (1 + 1e-12))    # full-vector proposition


def test_second_derivation_from_other_calls(oracle):
    w, _ = inputs.student_t_outliers(40, 512, 3.0, 4, 100.0, seed=63)
    perm = inputs.random_perm(512, 64)
    b = 32
    o = oracle.token_diagnostics(w, perm, b)
    x = np.abs(inputs.bf16_to_f64(w))
    assert np.allclose(o[:, 0], x.max(axis=1), rtol=0) and np.allclose(o[:, 1], x.sum(axis=1), rtol=1e-14)
    assert np.allclose(o[:, 2], oracle.block_l1_stats(w, perm, b)[2], rtol=1e-14)
    r = oracle.rotate_quantize(w, perm, b, 0, 0, want_y=True)
    y = r["y"]
    assert np.allclose(o[:, 3], np.abs(y).max(axis=1), rtol=0)
    codes = r["codes"]
    lo, hi = (codes & 0xF).astype(np.int64), (codes >> 4).astype(np.int64)
    q = np.stack([lo, hi], axis=2).reshape(codes.shape[0], -1)
    q = np.where(q >= 8, q - 16, q)                                                  # two's complement nibbles
    s64 = np.abs(y).max(axis=1) / 7
    err = np.sqrt(((y - s64[:, None] * q) ** 2).sum(axis=1))
    assert np.allclose(o[:, 4], err, rtol=1e-12)
