"""Pins for the oracle's INT4 and MXFP4 quantisers and the nibble packing.

Checked against: the paper's step size and worst-case error bound (Sec. 3), a library
round-half-even (numpy.rint / torch.round), exact ties built by hand, the OCP E2M1 value
grid searched by brute force, and the exponent field of the IEEE encoding.
"""
import numpy as np
import pytest
import torch

from paper_2601_22347_b200 import inputs

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def unpack(codes):
    """packed [T, d/2] -> nibbles [T, 2*(d/2)]; low nibble is the even index."""
    lo = codes & 0xF
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def int4_value(nib):
    return np.where(nib >= 8, nib.astype(np.int64) - 16, nib.astype(np.int64))


def e2m1_value(nib):
    return np.where(nib & 8, -1.0, 1.0) * GRID[nib & 7]


def rand_y(T, d, seed, outlier=50.0):
    rng = np.random.default_rng(seed)
    y = rng.standard_normal((T, d))
    y[:, rng.choice(d, 3, replace=False)] *= outlier
    return y


# ------------------------------------------------------------------ packing

def test_pack_round_trip_all_byte_values(oracle):
    # a row whose 512 nibbles enumerate every (low, high) pair = every byte value
    d = 512
    want = np.array([[k & 0xF, k >> 4] for k in range(256)], np.int64).reshape(-1)  # nibble values
    vals = np.where(want >= 8, want - 16, want).astype(np.float64)                 # as signed codes
    y = vals[None, :].copy()
    y[0, 0] = 0.0
    y[0, 15 * 2 + 1] = 0  # keep one zero; make the max exactly 7 so that s = 1
    y = np.clip(y, -7, 7)
    codes, scales = oracle.quantize_int4(y, 0)
    assert scales[0, 0] == 1.0
    nib = unpack(codes)[0]
    assert np.array_equal(int4_value(nib), y[0].astype(np.int64))
    # byte k = code[2k] | code[2k+1] << 4
    assert np.array_equal(codes[0], (nib[0::2] | (nib[1::2] << 4)).astype(np.uint8))
    assert codes[0, 1] == ((1 & 0xF) | (0 << 4))


def test_low_nibble_is_even_index(oracle):
    y = np.zeros((1, 32)); y[0, 0] = 7.0; y[0, 1] = -7.0; y[0, 2] = 3.0
    codes, _ = oracle.quantize_int4(y, 0)
    assert codes[0, 0] == (7 | (9 << 4))     # -7 -> two's complement nibble 0b1001
    assert codes[0, 1] == 3


# ------------------------------------------------------------------ INT4

@pytest.mark.parametrize("group", [0, 128, 32])
def test_int4_step_size_and_error_bound(oracle, group):
    T, d = 16, 1024
    y = rand_y(T, d, 1)
    codes, scales, pre = oracle.quantize_int4(y, group, want_pre=True)
    g = d if group == 0 else group
    q = int4_value(unpack(codes)).reshape(T, d // g, g)
    yr = y.reshape(T, d // g, g)
    amax = np.abs(yr).max(axis=2)
    # s = ||X||_inf / (2^{q-1} - 1), stored as binary32
    assert np.array_equal(scales, (amax / 7.0).astype(np.float32))
    assert q.min() >= -7 and q.max() <= 7            # -8 is never produced with this step
    # the element that attains the max gets +-7
    am = np.abs(yr).argmax(axis=2)
    assert np.all(np.abs(np.take_along_axis(q, am[..., None], 2)) == 7)
    s = amax[..., None] / 7.0
    err = np.abs(yr - q * s)
    assert np.all(err <= s / 2 * (1 + 1e-12))        # round-to-nearest: |err| <= s/2
    # paper's bound: ||X - Q(X)||_2 <= sqrt(d)/(2^q - 2) * ||X||_inf  (per scale range)
    l2 = np.sqrt((err ** 2).sum(axis=2))
    assert np.all(l2 <= np.sqrt(g) / 14.0 * amax * (1 + 1e-12))
    # same codes from a library round-half-even
    ref = np.rint(yr / s).astype(np.int64)
    assert np.array_equal(q, ref)
    assert np.array_equal(torch.round(torch.from_numpy(yr / s)).numpy().astype(np.int64), q)
    assert np.allclose(pre.reshape(yr.shape), yr / s, rtol=1e-15)


def test_int4_ties_round_to_even(oracle):
    # max = 7 => s = 1 exactly; then every k + 0.5 is an exact tie
    y = np.array([[7.0, 0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, -0.5, -1.5, -2.5, -3.5, -4.5, -5.5, -6.5, 0.0]
                  + [0.0] * 16])
    codes, scales = oracle.quantize_int4(y, 0)
    q = int4_value(unpack(codes))[0, :16]
    assert scales[0, 0] == 1.0
    assert list(q) == [7, 0, 2, 2, 4, 4, 6, 6, 0, -2, -2, -4, -4, -6, -6, 0]


def test_int4_zero_range(oracle):
    y = np.zeros((2, 256)); y[1, 128:] = rand_y(1, 128, 2)[0]
    codes, scales = oracle.quantize_int4(y, 128)
    assert scales[0, 0] == 0 and scales[0, 1] == 0 and scales[1, 0] == 0 and scales[1, 1] > 0
    assert not codes[0].any() and not codes[1, :64].any() and codes[1, 64:].any()


def test_int4_group_ranges_are_contiguous(oracle):
    y = np.ones((1, 64)); y[0, 32:] = 100.0; y[0, 5] = -2.0
    codes, scales = oracle.quantize_int4(y, 32)
    assert np.allclose(scales[0], [2.0 / 7, 100.0 / 7])
    q = int4_value(unpack(codes))[0]
    assert q[5] == -7 and np.all(q[32:] == 7) and q[0] == 4   # 1/(2/7) = 3.5 -> 4 (even)


# ------------------------------------------------------------------ MXFP4

def brute_e2m1(v):
    """nearest grid magnitude by exhaustive search; ties -> even index; saturate at 6."""
    out = np.empty(v.shape, np.int64)
    flat = np.abs(v).ravel()
    for n, m in enumerate(flat):
        dist = np.abs(GRID - min(m, 6.0))
        best = np.flatnonzero(dist == dist.min())
        k = best[0] if len(best) == 1 else [i for i in best if i % 2 == 0][0]
        out.ravel()[n] = k
    return out


def test_mxfp4_scale_is_exponent_field_minus_two(oracle):
    T, d = 8, 512
    y = rand_y(T, d, 3) * np.exp2(np.random.default_rng(4).integers(-20, 20, size=(T, 1)))
    codes, e8m0, pre = oracle.quantize_mxfp4(y, want_pre=True)
    amax = np.abs(y.reshape(T, d // 32, 32)).max(axis=2)
    # independent derivation: biased exponent straight from the IEEE double encoding
    expo = ((amax.view(np.uint64) >> 52) & 0x7FF).astype(np.int64) - 1023
    assert np.array_equal(e8m0.astype(np.int64), expo - 2 + 127)
    scaled = amax / np.exp2(expo - 2)
    assert np.all((scaled >= 4) & (scaled < 8))       # "rounded down to a power of two"
    # shared scale never exceeds amax/4 and is a power of two (E8M0 has no mantissa)
    assert np.allclose(np.abs(pre).reshape(T, d // 32, 32).max(axis=2), scaled)


def test_mxfp4_elements_are_nearest_grid_points(oracle):
    T, d = 4, 256
    y = rand_y(T, d, 5, outlier=8.0)
    codes, e8m0, pre = oracle.quantize_mxfp4(y, want_pre=True)
    nib = unpack(codes)
    assert np.array_equal(nib & 7, brute_e2m1(pre))
    assert np.array_equal((nib >> 3).astype(bool), np.signbit(y))
    E = e8m0.astype(np.int64) - 127
    deq = e2m1_value(nib).reshape(T, d // 32, 32) * np.exp2(E)[..., None]
    yr = y.reshape(T, d // 32, 32)
    # inside the representable range the error is at most half the local grid spacing (<= 1 at the top)
    inside = np.abs(pre).reshape(yr.shape) <= 6
    assert np.all(np.abs(deq - yr)[inside] <= 1.0 * np.exp2(E)[..., None].repeat(32, 2)[inside] + 0)
    # values in (6, 8) * 2^E saturate to 6
    sat = np.abs(pre) > 6
    assert sat.any()
    assert np.all((nib & 7)[sat] == 7)


def test_mxfp4_tie_midpoints_go_to_even_code(oracle):
    # amax = 4 => E = 0, so v = y; midpoints of the grid are exact ties
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    want = [0, 2, 2, 4, 4, 6, 6]                     # even code index of the two neighbours
    row = [4.0] + mids + [-m for m in mids] + [7.0 * 0] + [0.0] * 16
    y = np.array([row])
    assert y.shape[1] == 32
    codes, e8m0 = oracle.quantize_mxfp4(y)
    nib = unpack(codes)[0]
    assert e8m0[0, 0] == 127
    assert list(nib[1:8]) == want
    assert list(nib[8:15]) == [8 | w for w in want]   # sign kept, also when the magnitude rounds to 0
    assert nib[0] == 6                                 # 4.0 -> index 6


def test_mxfp4_saturation_and_sign(oracle):
    y = np.zeros((1, 32)); y[0, :6] = [7.9, -7.0, 6.0, 6.5, -0.1, 5.1]
    codes, e8m0 = oracle.quantize_mxfp4(y)
    nib = unpack(codes)[0]
    assert e8m0[0, 0] == 127                          # floor(log2 7.9) - 2 = 0
    assert list(nib[:6]) == [7, 15, 7, 7, 8, 7]       # (6,8) saturates; -0.1 -> -0


def test_mxfp4_zero_group_and_clamp(oracle):
    y = np.zeros((1, 96)); y[0, 32] = 1e-45; y[0, 64] = 3e38
    codes, e8m0 = oracle.quantize_mxfp4(y)
    assert e8m0[0, 0] == 0 and not codes[0, :16].any()
    assert e8m0[0, 1] == 0                            # exponent below -127 clamps to code 0
    assert e8m0[0, 2] == 127 - 2 + 127                # floor(log2 3e38) = 127


def test_whole_path_composes_rotate_then_quantize(oracle):
    w = inputs.config1(T=4)
    y = oracle.rotate(w.x, None, 16)
    c1, s1 = oracle.quantize_int4(y, 0)
    r = oracle.rotate_quantize(w.x, None, 16, oracle.FMT_INT4, 0, want_y=True)
    assert np.array_equal(r["codes"], c1) and np.array_equal(r["scales"], s1) and np.array_equal(r["y"], y)
    c2, e2 = oracle.quantize_mxfp4(y)
    r2 = oracle.rotate_quantize(w.x, None, 16, oracle.FMT_MXFP4, 32)
    assert np.array_equal(r2["codes"], c2) and np.array_equal(r2["scales"], e2)


def test_constructed_ties_through_the_rotation(oracle):
    """H is an involution: feed x = y* H_16 / 4 with y* dyadic, get y* back exactly, and
    the codes must round the exact .5 values to even."""
    import scipy.linalg
    ystar = np.array([7, 0.5, 1.5, 2.5, -3.5, 4.5, -5.5, 6.5, 0, 1, -2, 3, -0.5, -1.5, 0.25, 0.75])
    x = (ystar @ scipy.linalg.hadamard(16)) / 4.0
    xb = inputs.f32_to_bf16_bits(np.tile(x.astype(np.float32), 2)[None, :])
    assert np.array_equal(inputs.bf16_to_f64(xb)[0, :16], x)
    r = oracle.rotate_quantize(xb, None, 16, oracle.FMT_INT4, 0, want_y=True)
    assert np.array_equal(r["y"][0, :16], ystar)
    q = int4_value(unpack(r["codes"]))[0, :16]
    assert list(q) == [7, 0, 2, 2, -4, 4, -6, 6, 0, 1, -2, 3, 0, -2, 0, 1]


# ------------------------------------------------------------------ FP4 with a per-token scale

E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def _fp4_unpack(codes):
    lo, hi = codes & 0xF, codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def test_fp4_per_token_scale_is_row_max_over_seven_and_values_sit_on_the_grid(oracle):
    rng = np.random.default_rng(71)
    y = rng.standard_normal((40, 256)) * np.exp2(rng.integers(-20, 20, size=(40, 1)))
    y[3] = 0.0
    codes, scales, pre = oracle.quantize_fp4(y, want_pre=True)
    a = np.abs(y).max(axis=1)
    assert np.array_equal(scales[:, 0], (a / 7.0).astype(np.float32))
    nib = _fp4_unpack(codes)
    mag = E2M1_VALUES[nib & 7]
    s = (a / 7.0)[:, None]
    # the element that attains the maximum maps to 7 and saturates to the largest magnitude
    assert np.all(mag[np.arange(40), np.abs(y).argmax(axis=1)][a > 0] == 6.0)
    # every element: nearest grid value, error at most half the local spacing (a full step in the 6..7 band)
    v = np.abs(pre)
    err = np.abs(v - mag)
    spacing = np.where(v < 2, 0.5, np.where(v < 4, 1.0, 2.0))
    assert np.all(err[v <= 6] <= spacing[v <= 6] / 2 + 1e-12)
    assert np.all(err[v > 6] <= 1.0 + 1e-12)
    # signs are the input's, also for zeros
    assert np.array_equal((nib >> 3).astype(bool), np.signbit(y))
    assert scales[3, 0] == 0.0 and not (nib[3] & 7).any()
    del s


def test_fp4_midpoints_go_to_the_even_code(oracle):
    # s = 1 when the row maximum is 7: the midpoints themselves are the scaled values
    y = np.array([[7.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, 6.5]])
    codes, scales = oracle.quantize_fp4(y)
    nib = _fp4_unpack(codes)[0]
    assert scales[0, 0] == 1.0
    assert (nib & 7).tolist() == [7, 0, 2, 2, 4, 4, 6, 6, 0, 2, 2, 4, 4, 6, 6, 7]
    assert (nib >> 3).tolist() == [0] * 8 + [1] * 7 + [0]


def test_fp4_agrees_with_the_mx_quantiser_when_the_scale_is_a_power_of_two(oracle):
    # a row of 32 whose maximum is 7 * 2^k has step 2^k under both quantisers (E = floor(log2(7 * 2^k)) - 2 = k)
    rng = np.random.default_rng(72)
    for k in (-9, 0, 5):
        y = rng.uniform(-6.9, 6.9, size=(25, 32)) * 2.0 ** k
        y[:, 0] = 7.0 * 2.0 ** k
        c4, s4 = oracle.quantize_fp4(y)
        cm, em = oracle.quantize_mxfp4(y)
        assert np.array_equal(c4, cm)
        assert np.all(s4 == np.float32(2.0 ** k)) and np.all(em.astype(int) - 127 == k)


def test_fp4_whole_path_is_rotation_then_quantiser(oracle):
    from paper_2601_22347_b200 import inputs
    bits, _ = inputs.gaussian_outliers(9, 256, 2, 50.0, seed=73)
    perm = inputs.random_perm(256, 74)
    out = oracle.rotate_quantize(bits, perm, 32, oracle.FMT_FP4, 0, want_y=True)
    c, s = oracle.quantize_fp4(out["y"])
    assert np.array_equal(out["codes"], c) and np.array_equal(out["scales"], s)


# ------------------------------------------------------------------ asymmetric INT4, per token

def test_asym_int4_range_extremes_and_round_trip(oracle):
    rng = np.random.default_rng(81)
    y = rng.standard_normal((60, 512)) * np.exp2(rng.integers(-12, 12, size=(60, 1))) + rng.standard_normal((60, 1)) * 3
    y[4] = 2.5            # constant row
    y[5] = 0.0
    codes, sz, pre = oracle.quantize_int4_asym(y, want_pre=True)
    nib = _fp4_unpack(codes).astype(np.int64)
    mx, mn = y.max(axis=1), y.min(axis=1)
    s = (mx - mn) / 15.0
    assert np.array_equal(sz[:, 0], s.astype(np.float32))
    assert nib.min() >= 0 and nib.max() <= 15
    live = s > 0
    rows = np.arange(60)
    assert np.all(nib[rows, y.argmin(axis=1)][live] == 0)            # the minimum is the first level
    assert np.all(nib[rows, y.argmax(axis=1)][live] >= 14)           # the maximum the last (15, or 14 at a tie)
    z = sz[:, 1].astype(np.float64)
    assert np.all(z == np.rint(z))
    deq = s[:, None] * (nib + z[:, None])
    assert np.all(np.abs(y - deq)[live] <= s[live][:, None] * (0.5 + 1e-9))   # half a step, as in Sec. 3
    assert not nib[4].any() and not nib[5].any() and sz[4, 0] == 0 and sz[5, 1] == 0
    order = np.argsort(y, axis=1)                                    # codes are monotone in the value
    assert np.all(np.diff(np.take_along_axis(nib, order, axis=1), axis=1) >= 0)


def test_asym_int4_is_equivariant_under_power_of_two_scaling_and_even_step_shifts(oracle):
    rng = np.random.default_rng(82)
    base = rng.integers(-40, 41, size=(20, 64)).astype(np.float64)     # small integers: exact in every step below
    base[:, 0], base[:, 1] = -44.0, 46.0                               # range 90 -> s = 6, min / s = -7.33 (no tie)
    c0, sz0 = oracle.quantize_int4_asym(base)
    assert np.all(sz0[:, 0] == 6.0) and np.all(sz0[:, 1] == -7.0)
    for k in (-7, 3):
        c, sz = oracle.quantize_int4_asym(base * 2.0 ** k)
        assert np.array_equal(c, c0) and np.all(sz[:, 0] == np.float32(6.0 * 2.0 ** k)) and np.array_equal(sz[:, 1], sz0[:, 1])
    for shift in (-4, 2):                       # whole even numbers of steps keep every tie's parity: only z moves
        c, sz = oracle.quantize_int4_asym(base + 6.0 * shift)
        assert np.array_equal(c, c0) and np.array_equal(sz[:, 1], sz0[:, 1] + shift)


def test_asym_int4_rounds_half_to_even(oracle):
    # s = 1: min 0, max 15; values k + 1/2 go to the even integer
    y = np.array([[0.0, 15.0, 0.5, 1.5, 2.5, 3.5, 13.5, 14.5, 7.49, 7.51, 4.0, 4.0, 4.0, 4.0, 4.0, 4.0]])
    c, sz = oracle.quantize_int4_asym(y)
    nib = _fp4_unpack(c)[0].tolist()
    assert sz[0].tolist() == [1.0, 0.0]
    assert nib[:10] == [0, 15, 0, 2, 2, 4, 14, 14, 7, 8]
