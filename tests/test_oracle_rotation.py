"""Pins for the oracle's permutation gather and block Hadamard rotation.

Each test checks the oracle against something other than itself: the paper's stated
properties of R (Notation paragraph), the hand expansion of H_2 / H_4, scipy's Sylvester
construction, the block proposition's per-coordinate bound, and orthonormality.
"""
import numpy as np
import pytest
import scipy.linalg

from paper_2601_22347_b200 import inputs


def bits(a):
    """float array -> bf16 bit patterns; asserts the values are exactly representable."""
    a = np.asarray(a, np.float32)
    h = inputs.f32_to_bf16_bits(a)
    assert np.array_equal(inputs.bf16_bits_to_f32(h), a), "test input not bf16-exact"
    return h


@pytest.mark.parametrize("b", [1, 2, 4, 16, 32, 64, 128, 2048, 4096])
def test_hadamard_orthogonal_and_unit_columns(oracle, b):
    H = oracle.hadamard_pm1(b).astype(np.float64)   # +-1 sums up to 4096 are exact in double
    assert np.all(np.abs(H) == 1)                                  # entries +-1 -> |R_ki| = 1/sqrt(b)
    assert np.array_equal(H @ H.T, b * np.eye(b))                  # R R^T = I exactly
    assert np.array_equal(H, H.T)
    R = H / np.sqrt(b)
    assert np.allclose(np.linalg.norm(R, axis=0), 1.0, atol=1e-12)  # ||R_i||_2 = 1
    assert np.allclose(np.abs(R).max(axis=0), 1 / np.sqrt(b))       # ||R_i||_inf = 1/sqrt(b)


@pytest.mark.parametrize("b", [2, 4, 16, 128, 1024])
def test_hadamard_is_scipy_sylvester(oracle, b):
    assert np.array_equal(oracle.hadamard_pm1(b), scipy.linalg.hadamard(b).astype(np.int8))


def test_rotate_hand_expanded_b2_b4(oracle):
    x = np.array([[1.5, -0.25, 3.0, 7.0, -2.0, 0.5, 0.125, -9.0]], np.float32)
    y2 = oracle.rotate(bits(x), None, 2)
    e2 = np.empty(8)
    for j in range(4):
        x0, x1 = float(x[0, 2 * j]), float(x[0, 2 * j + 1])
        e2[2 * j:2 * j + 2] = [(x0 + x1) / np.sqrt(2), (x0 - x1) / np.sqrt(2)]
    assert np.allclose(y2[0], e2, rtol=0, atol=1e-15)
    y4 = oracle.rotate(bits(x), None, 4)
    e4 = np.empty(8)
    for j in range(2):
        x0, x1, x2, x3 = [float(v) for v in x[0, 4 * j:4 * j + 4]]
        e4[4 * j:4 * j + 4] = [(x0 + x1 + x2 + x3) / 2, (x0 - x1 + x2 - x3) / 2,
                               (x0 + x1 - x2 - x3) / 2, (x0 - x1 - x2 + x3) / 2]
    assert np.array_equal(y4[0], e4)  # /2 is exact


@pytest.mark.parametrize("b", [16, 64])
def test_rotate_basis_and_constant_inputs(oracle, b):
    H = scipy.linalg.hadamard(b)
    x = np.zeros((b, 2 * b), np.float32)
    for k in range(b):
        x[k, b + k] = 1.0                       # e_k placed in the second block
    y = oracle.rotate(bits(x), None, b)
    assert np.all(y[:, :b] == 0)
    assert np.allclose(y[:, b:], H / np.sqrt(b), atol=1e-15)   # row k of R
    c = np.full((1, 2 * b), 3.0, np.float32)
    yc = oracle.rotate(bits(c), None, b)
    expect = np.zeros(2 * b); expect[0] = expect[b] = 3.0 * np.sqrt(b)
    assert np.allclose(yc[0], expect, atol=1e-13)


@pytest.mark.parametrize("b", [16, 32, 128, 512])
def test_rotate_matches_library_matmul(oracle, b):
    w = inputs.gaussian_outliers(6, 1024, 4, 50.0, seed=11)[0]
    x = inputs.bf16_to_f64(w)
    y = oracle.rotate(w, None, b)
    R = scipy.linalg.hadamard(b) / np.sqrt(b)
    ref = (x.reshape(6, 1024 // b, b) @ R).reshape(6, 1024)
    assert np.allclose(y, ref, rtol=0, atol=1e-11 * np.abs(ref).max())


@pytest.mark.parametrize("b", [16, 128, 1024])
def test_rotate_preserves_block_l2_and_obeys_l1_bound(oracle, b):
    w = inputs.student_t_outliers(8, 2048, 3.0, 16, 100.0, seed=5)[0]
    x = inputs.bf16_to_f64(w).reshape(8, 2048 // b, b)
    y = oracle.rotate(w, None, b).reshape(8, 2048 // b, b)
    # orthonormal block-diagonal rotation: per-block l2 norm is unchanged
    assert np.allclose(np.linalg.norm(y, axis=2), np.linalg.norm(x, axis=2), rtol=1e-12)
    # proof of the block proposition: |X_{j} R_i| <= ||X_{j}||_1 / sqrt(b)
    bound = np.abs(x).sum(axis=2, keepdims=True) / np.sqrt(b)
    assert np.all(np.abs(y) <= bound * (1 + 1e-12))


def test_l1_bound_is_attained_by_a_hadamard_row(oracle):
    b = 32
    H = scipy.linalg.hadamard(b).astype(np.float32)
    y = oracle.rotate(bits(H[5:6] * 2.0), None, b)
    # x = 2 * (row 5 of H): coordinate 5 collects every term with the same sign
    assert y[0, 5] == pytest.approx(2.0 * b / np.sqrt(b), rel=1e-15)
    assert np.allclose(np.delete(y[0], 5), 0, atol=1e-13)


def test_rotation_is_an_involution_on_dyadic_inputs(oracle):
    b = 16  # sqrt(b) = 4: small integers stay exactly representable through both passes
    rng = np.random.default_rng(3)
    x = rng.integers(-8, 9, size=(4, 64)).astype(np.float32) * 4.0
    y = oracle.rotate(bits(x), None, b)
    assert np.array_equal(y, np.round(y * 4) / 4)
    back = oracle.rotate(bits(y.astype(np.float32)), None, b)
    assert np.array_equal(back, x.astype(np.float64))


def test_full_vector_is_the_one_block_case(oracle):
    w = inputs.laplace_outliers(3, 256, 2, 200.0, seed=9)[0]
    full = oracle.rotate(w, None, 256)
    x = inputs.bf16_to_f64(w)
    ref = x @ (scipy.linalg.hadamard(256) / 16.0)
    assert np.allclose(full, ref, rtol=0, atol=1e-10)
    # full-vector bound ||XR||_inf <= ||X||_1 / sqrt(d)
    assert np.all(np.abs(full).max(axis=1) <= np.abs(x).sum(axis=1) / 16.0 * (1 + 1e-12))


def test_permutation_is_a_gather(oracle):
    d = 64
    x = np.arange(d, dtype=np.float32)[None, :]            # x_c = c
    perm = np.random.default_rng(1).permutation(d).astype(np.int32)
    y = oracle.rotate(bits(x), perm, 1)                     # b = 1: the rotation is the identity
    assert np.array_equal(y[0], perm.astype(np.float64))    # (XP)_i = X_{pi(i)}
    inv = np.argsort(perm).astype(np.int32)
    y2 = oracle.rotate(bits(y.astype(np.float32)), inv, 1)
    assert np.array_equal(y2[0], x[0].astype(np.float64))   # perm then inverse = identity


def test_permutation_changes_block_membership(oracle):
    # swapping two channels across a block boundary moves their mass between blocks
    b, d = 4, 8
    x = np.array([[8, 0, 0, 0, 0, 0, 0, 0]], np.float32)
    perm = np.array([4, 1, 2, 3, 0, 5, 6, 7], np.int32)     # slot 4 now reads channel 0
    y = oracle.rotate(bits(x), perm, b)
    assert np.array_equal(y[0], [0, 0, 0, 0, 4, 4, 4, 4])


def test_rejects_bad_arguments(oracle):
    w = np.zeros((1, 48), np.uint16)
    with pytest.raises(RuntimeError):
        oracle.rotate(w, None, 32)            # 48 % 32 != 0
    with pytest.raises(RuntimeError):
        oracle.rotate(w, None, 12)            # not a power of two
    with pytest.raises(RuntimeError):
        oracle.rotate(w, np.full(48, 48, np.int32), 16)   # perm out of range


def test_op_count_table():
    """d*log2(b) add/sub per token reproduces the paper's printed block-rotation counts."""
    import os
    from paper_2601_22347_b200.roofline import butterfly_add_sub_per_token
    here = os.path.dirname(__file__)
    rows = [l.split() for l in open(os.path.join(here, "golden", "hadamard_op_counts.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 16
    for _, d, b, ops in rows:
        assert butterfly_add_sub_per_token(int(d), int(b)) == int(ops)


# ------------------------------------------------------------------ full-vector rotation of a non-power-of-2 dimension

def _paley2_by_kron(q: int) -> np.ndarray:
    """Textbook form of Paley's second construction, by another route than the oracle's loops: Euler's criterion
    for the quadratic character and H = S (x) [[1, 1], [1, -1]] + I (x) [[1, -1], [-1, -1]]."""
    chi = [0] + [1 if pow(a, (q - 1) // 2, q) == 1 else -1 for a in range(1, q)]
    S = np.zeros((q + 1, q + 1), np.int64)
    S[0, 1:] = 1
    S[1:, 0] = 1
    for i in range(q):
        for j in range(q):
            S[1 + i, 1 + j] = chi[(i - j) % q]
    return np.kron(S, np.array([[1, 1], [1, -1]])) + np.kron(np.eye(q + 1, dtype=np.int64), np.array([[1, -1], [-1, -1]]))


@pytest.mark.parametrize("n", [12, 28, 36, 60, 76])
def test_base_matrix_is_hadamard(oracle, n):
    """What the mathematics fixes about the base matrix of order 4t (the paper does not print its own)."""
    H = oracle.hadamard_base(n).astype(np.int64)
    assert set(np.unique(H).tolist()) == {-1, 1}
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))
    assert np.array_equal(H.T @ H, n * np.eye(n, dtype=np.int64))
    assert np.array_equal(H, H.T)
    assert np.array_equal(H, _paley2_by_kron(n // 2 - 1))


@pytest.mark.parametrize("n", [8, 20, 44, 52, 14, 3])
def test_orders_without_a_base_matrix_are_refused(oracle, n):
    with pytest.raises(Exception):
        oracle.hadamard_base(n)


@pytest.mark.parametrize("d", [48, 112, 3072, 1216])
def test_non_po2_matrix_is_sylvester_kron_base(oracle, d):
    """H_d = H_{2^k'} (x) H_{4t}: k' butterfly stages over strides of 4t, rotations of 4t ADJACENT inputs."""
    import scipy.linalg
    t = d
    while t % 2 == 0:
        t //= 2
    n = 4 * t
    H = oracle.hadamard_pm1(d).astype(np.int64)
    assert np.array_equal(H, np.kron(scipy.linalg.hadamard(d // n).astype(np.int64), oracle.hadamard_base(n).astype(np.int64)))
    if d <= 1216:
        assert np.array_equal(H @ H.T, d * np.eye(d, dtype=np.int64))


def test_non_po2_rotation_closed_forms(oracle):
    rng = np.random.default_rng(41)
    for d in (48, 112, 3072):
        x = rng.standard_normal((5, d)).astype(np.float32)
        bits = inputs.f32_to_bf16_bits(x)
        xb = inputs.bf16_to_f64(bits)
        y = oracle.rotate(bits, None, d)
        H = oracle.hadamard_pm1(d).astype(np.float64)
        np.testing.assert_allclose(y, xb @ H / np.sqrt(d), rtol=0, atol=1e-12 * np.abs(xb).sum(axis=1).max())
        # orthogonal and (H symmetric) an involution; the full-vector bound of Sec. 3
        np.testing.assert_allclose((y * y).sum(axis=1), (xb * xb).sum(axis=1), rtol=1e-12)
        np.testing.assert_allclose(y @ H / np.sqrt(d), xb, atol=1e-12 * np.abs(xb).sum(axis=1).max())
        assert (np.abs(y).max(axis=1) <= np.abs(xb).sum(axis=1) / np.sqrt(d) * (1 + 1e-12)).all()
        # a unit vector returns a row of H
        e = np.zeros((1, d), np.float32)
        e[0, 17] = 1.0
        np.testing.assert_array_equal(oracle.rotate(inputs.f32_to_bf16_bits(e), None, d)[0] * np.sqrt(d), H[17])
    # a permutation is applied before the rotation
    p = inputs.random_perm(112, 5)
    bits = inputs.f32_to_bf16_bits(rng.standard_normal((2, 112)).astype(np.float32))
    np.testing.assert_array_equal(oracle.rotate(bits, p, 112), oracle.rotate(bits[:, p], None, 112))
    with pytest.raises(Exception):
        oracle.rotate(bits, None, 56)             # a non-power-of-2 block inside a longer row


def test_non_po2_op_count_table():
    """The three add/sub counts of the paper's Table "non-po2-ops" for its five dimensions."""
    import os
    from paper_2601_22347_b200.roofline import full_vector_add_sub_per_token, non_po2_factors
    here = os.path.dirname(__file__)
    rows = [l.split() for l in open(os.path.join(here, "golden", "non_po2_op_counts.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 5

    def printed(v):
        return "%.2fM" % (v / 1e6) if v >= 1e6 else "%.2fK" % (v / 1e3)

    for _, d, kp, n, dense, mixed, ours in rows:
        assert non_po2_factors(int(d)) == (int(kp), int(n))
        assert tuple(printed(v) for v in full_vector_add_sub_per_token(int(d))) == (dense, mixed, ours)
    assert non_po2_factors(4096) is None
