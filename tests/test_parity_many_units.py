"""Parity with the oracle on calls long enough that every warp group of the persistent kernel processes
many units: the shared-memory ring wraps, the stage parities flip, the double-buffered code staging is
reused, and the deferred scale records fill up and are served in the middle of the run (not only in the
kernel's tail).  The GPU runs the whole call, the oracle a sample of rows including the first and last.

The number of units a warp group sees follows from the launch arithmetic of the library, restated in
`units_per_group` below; every case asserts that it is at least MIN_UNITS, so a later change of the grid
cannot hollow these tests out unnoticed.
"""
import numpy as np
import pytest
import torch

from paper_2601_22347_b200 import inputs

from parity import compare_quantized

pytestmark = pytest.mark.gpu

FMT = {"int4": 0, "mxfp4": 1, "fp4": 3, "int4_asym": 4}
SMS = 148                # CTAs of the persistent kernel: one per SM of a B200
WARPS_PER_CTA = 16
SEG = 1024               # elements of a warp's segment
MIN_UNITS = 40


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2601_22347_b200 import binding, build
    build.build()
    binding.load()
    return binding


@pytest.fixture(autouse=True)
def clean_error_word(B):
    B.perq_device_error_clear()
    yield
    assert B.perq_device_error() == 0


def units_per_group(T, d, b, fmt, group, permuted):
    """Units (rows, or 1024-element segments) that the busiest warp group of the persistent kernel handles.
    A unit is a whole row when the warps of a row are coupled (per-token scales, a permutation, a block that
    spans the row), else a single segment; a CTA holds 16 // G groups of G warps.  (The records of deferred
    scales are served when 32 have gathered, 16 in the lean per-token kernel.)"""
    assert d % SEG == 0
    segs = d // SEG
    per_token = fmt in ("fp4", "int4_asym") or (fmt == "int4" and group in (0, d))
    G = segs if (per_token or permuted or (b == d and b > 128)) else 1
    if fmt in ("int4", "fp4") and per_token and not permuted and b <= 128 and segs in (2, 4, 8):
        G = segs // 2        # the lean per-token kernel: a warp owns two adjacent segments of a row
    units = T * segs // G
    if fmt == "mxfp4" and not permuted and b <= 128 and segs % 2 == 0:
        units //= 2          # the lean MXFP4 kernel: a warp's unit is two adjacent segments
    groups_per_cta = WARPS_PER_CTA // G
    grid = min((units + groups_per_cta - 1) // groups_per_cta, SMS)
    return -(-units // (grid * groups_per_cta))


def rows_for(d, b, fmt, group, permuted, want=MIN_UNITS):
    """Smallest multiple of 1024 rows that gives every group at least `want` units."""
    T = 1024
    while units_per_group(T, d, b, fmt, group, permuted) < want:
        T += 1024
    return T


def tiled(bits, T):
    """T rows made of the base rows, each repetition rotated by one more row so that a given base row
    meets different warps and ring stages."""
    n = bits.shape[0]
    idx = (np.arange(T) + (np.arange(T) // n)) % n
    return bits[idx]


def check_sampled(B, oracle, name, bits, perm, b, fmt, group, seed, n_rows=48, want=MIN_UNITS, exempt_zero=False):
    T, d = bits.shape
    upg = units_per_group(T, d, b, fmt, group, perm is not None)
    assert upg >= want, "only %d units per group" % upg
    x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    p = None if perm is None else torch.from_numpy(perm).cuda()
    codes, scales = B.perq_rotate_quantize(x, p, b, FMT[fmt], group)
    torch.cuda.synchronize()
    rows = np.sort(np.random.default_rng(seed).choice(T, n_rows, replace=False))
    rows[0], rows[-1] = 0, T - 1
    ora = oracle.rotate_quantize(bits[rows], perm, b, FMT[fmt], group, want_pre=True)
    rows_t = torch.from_numpy(rows).cuda()
    rep = compare_quantized(fmt, codes[rows_t].cpu().numpy(), scales[rows_t].cpu().numpy(), ora)
    print("%s T=%d d=%d b=%d %s g=%d perm=%s: %d units per group, %d rows checked, %d tie-window exemptions"
          % (name, T, d, b, fmt, group, perm is not None, upg, n_rows, rep["code_mismatch_exempt"]))
    if exempt_zero:
        assert rep["code_mismatch_exempt"] == 0
    return rep


def base_rows(kind, d, seed, n=1024):
    if kind == "laplace":       # a few outlier channels: the row maximum sits in the same warp for every row
        return inputs.laplace_outliers(n, d, max(1, d // 1024), 200.0, seed)[0]
    if kind == "student":
        return inputs.student_t_outliers(n, d, 3.0, max(2, d // 256), 100.0, seed)[0]
    if kind == "gauss":         # no outliers: the maximum moves between the warps of a row
        return inputs.gaussian_outliers(n, d, 0, 1.0, seed)[0]
    raise ValueError(kind)


# ------------------------------------------------------------------ asymmetric INT4 per token

@pytest.mark.parametrize("d,b,perm,kind", [(4096, 32, False, "laplace"), (1024, 16, False, "student"),
                                           (8192, 128, False, "gauss"), (2048, 32, True, "laplace"),
                                           (8192, 64, True, "student")])
def test_asymmetric_int4_many_rows_per_group(B, oracle, d, b, perm, kind):
    bits = base_rows(kind, d, 11000 + d + b)
    x = inputs.bf16_bits_to_f32(bits)
    x[7] = np.abs(x[7]) + 0.25           # an all-positive row
    x[9] = 0.0                           # a constant row
    bits = inputs.f32_to_bf16_bits(x)
    T = rows_for(d, b, "int4_asym", 0, perm, want=72)      # two flushes of 32 records and a tail
    p = inputs.random_perm(d, 11001) if perm else None
    check_sampled(B, oracle, "asym-long", tiled(bits, T), p, b, "int4_asym", 0, 11002 + d, want=72,
                  exempt_zero=True)


# ------------------------------------------------------------------ blocks of 256, 512 and 1024

@pytest.mark.parametrize("fmt,group", [("int4", 0), ("mxfp4", 32)])
@pytest.mark.parametrize("b", [256, 512, 1024])
@pytest.mark.parametrize("d", [4096, 8192])
def test_long_blocks_many_units_per_group(B, oracle, d, b, fmt, group):
    bits = base_rows("laplace" if b != 512 else "gauss", d, 12000 + d + b)
    bits[5] = 0
    T = rows_for(d, b, fmt, group, False)
    check_sampled(B, oracle, "long-b", tiled(bits, T), None, b, fmt, group, 12001 + b, n_rows=32)


# ------------------------------------------------------------------ permuted MXFP4 / FP4

@pytest.mark.parametrize("fmt,group", [("mxfp4", 32), ("fp4", 0)])
@pytest.mark.parametrize("d,b", [(2048, 32), (8192, 128)])
def test_permuted_e2m1_many_rows_per_group(B, oracle, d, b, fmt, group):
    bits = base_rows("student", d, 13000 + d + b)
    bits[3] = 0
    T = rows_for(d, b, fmt, group, True)
    check_sampled(B, oracle, "perm-e2m1", tiled(bits, T), inputs.random_perm(d, 13001), b, fmt, group, 13002 + d)


# ------------------------------------------------------------------ per-128 scales with short blocks (deferred records)

@pytest.mark.parametrize("b", [16, 32])
def test_per_128_short_blocks_many_units_per_group(B, oracle, b):
    d = 4096
    bits = base_rows("laplace", d, 14000 + b)
    bits[2, 128:640] = 0
    T = rows_for(d, b, "int4", 128, False)
    check_sampled(B, oracle, "g128-short", tiled(bits, T), None, b, "int4", 128, 14001 + b)


# ------------------------------------------------------------------ per-token INT4 / FP4: the 32-record flush

@pytest.mark.parametrize("fmt", ["int4", "fp4"])
@pytest.mark.parametrize("d,b,kind", [(4096, 32, "laplace"), (1024, 16, "laplace"), (2048, 128, "gauss"),
                                      (14336, 64, "laplace")])
def test_per_token_many_rows_per_group(B, oracle, d, b, fmt, kind):
    bits = base_rows(kind, d, 15000 + d + b)
    bits[4] = 0
    T = rows_for(d, b, fmt, 0, False, want=72)
    check_sampled(B, oracle, "token-long", tiled(bits, T), None, b, fmt, 0, 15001 + d, want=72)


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("mxfp4", 32)])
def test_full_vector_many_rows_per_group(B, oracle, fmt, group):
    d = 4096
    bits = base_rows("laplace", d, 16000)
    bits[6] = 0
    T = rows_for(d, d, fmt, group, False)
    check_sampled(B, oracle, "full-long", tiled(bits, T), None, d, fmt, group, 16001, n_rows=16)


# ------------------------------------------------------------------ the workloads at their stated sizes

@pytest.mark.parametrize("b", [16, 32, 64, 128, 2048])
def test_config2_at_full_T(B, oracle, b):
    w = inputs.config2(T=4096, b=b)
    check_sampled(B, oracle, "cfg2", w.x, w.perm, b, w.fmt, w.group, 17000 + b, n_rows=48 if b <= 128 else 16, want=1)


def test_config3_at_full_T_with_the_massdiff_permutation(B, oracle):
    w = inputs.config3(T=4096)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    chan, _, _ = B.perq_block_l1_stats(x, None, w.b, want=("chan",))
    torch.cuda.synchronize()
    perm = B.perq_massdiff_perm(chan.cpu().numpy(), w.b)
    assert np.array_equal(perm, oracle.massdiff_perm(chan.cpu().numpy().astype(np.float64), w.b))
    check_sampled(B, oracle, "cfg3", w.x, perm, w.b, w.fmt, w.group, 17100, n_rows=32, want=1)


@pytest.mark.parametrize("b", [32, 128])
def test_config5_at_T_16384(B, oracle, b):
    base = inputs.config5(T=1024, b=b)
    check_sampled(B, oracle, "cfg5", tiled(base.x, 16384), base.perm, b, base.fmt, base.group, 17200 + b, n_rows=24)


# ------------------------------------------------------------------ flat-spectrum blocks: the error model's worst case

def _quadratic_sign_sequence(log2b):
    """(-1)^(x1 x2 + x2 x3 + ... ) over the bits of the index: the Rudin-Shapiro signs.  For an even number
    of bits the sequence is bent (every Walsh-Hadamard coefficient has magnitude sqrt(b)), for an odd number
    the coefficients are 0 or sqrt(2 b): the rotated block is as flat as a +-1 block can be, so the l1 norm
    of the inputs is as large as it gets against the largest rotated value."""
    n = np.arange(1 << log2b)
    acc = np.zeros_like(n)
    for i in range(log2b - 1):
        acc ^= (n >> i) & (n >> (i + 1)) & 1
    return 1.0 - 2.0 * acc


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32), ("fp4", 0), ("int4_asym", 0)])
@pytest.mark.parametrize("b", [16, 32, 64, 128, 1024])
def test_flat_spectrum_blocks(B, oracle, b, fmt, group):
    """x_k = s_k m_k with s a bent / Rudin-Shapiro sign pattern and m_k a random bf16 in [1, 2): every partial
    sum of the butterfly is as large as the outputs, so fp32 rounding errors are as large, relative to the
    block's largest output, as they can be.  Some blocks are scaled by powers of two, a few are plain noise."""
    d, T = 4096, 96
    rng = np.random.default_rng(18000 + b)
    s = _quadratic_sign_sequence(int(np.log2(b)))
    m = 1.0 + rng.integers(0, 128, size=(T, d)) / 128.0                 # every bf16 value in [1, 2)
    x = (m.reshape(T, d // b, b) * s[None, None, :])
    x *= np.exp2(rng.integers(-3, 4, size=(T, d // b, 1)))             # block magnitudes over 7 binades
    flip = rng.random((T, d // b, 1)) < 0.25
    x = np.where(flip, -x, x)
    x = x.reshape(T, d)
    x[::7] = rng.standard_normal((len(range(0, T, 7)), d))              # plain rows in between
    bits = inputs.f32_to_bf16_bits(x.astype(np.float32))
    ora = oracle.rotate_quantize(bits, None, b, FMT[fmt], group, want_pre=True)
    xd = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    codes, scales = B.perq_rotate_quantize(xd, None, b, FMT[fmt], group)
    torch.cuda.synchronize()
    rep = compare_quantized(fmt, codes.cpu().numpy(), scales.cpu().numpy(), ora)
    print("flat b=%d %s g=%d: %d tie-window exemptions" % (b, fmt, group, rep["code_mismatch_exempt"]))
    # the same blocks through a permutation (the gathered row is the constructed one)
    if b <= 128:
        perm = inputs.random_perm(d, 18001)
        pb = np.empty_like(bits)
        pb[:, perm] = bits
        codes, scales = B.perq_rotate_quantize(torch.from_numpy(pb.view(np.int16)).cuda().view(torch.bfloat16),
                                               torch.from_numpy(perm).cuda(), b, FMT[fmt], group)
        torch.cuda.synchronize()
        compare_quantized(fmt, codes.cpu().numpy(), scales.cpu().numpy(), ora)


def test_random_asymmetric_rows_need_no_exemption(B, oracle):
    """On random data no code of the asymmetric quantiser may differ from the oracle's at all."""
    for d, b, seed in ((4096, 32, 19000), (2048, 128, 19001), (1536, 16, 19002)):
        bits, _ = inputs.student_t_outliers(300, d, 3.0, 8, 100.0, seed)
        x = inputs.bf16_bits_to_f32(bits)
        x[::5] += 40.0                       # rows far from symmetric: large |y / s|
        bits = inputs.f32_to_bf16_bits(x)
        ora = oracle.rotate_quantize(bits, None, b, FMT["int4_asym"], 0, want_pre=True)
        xd = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        codes, scales = B.perq_rotate_quantize(xd, None, b, FMT["int4_asym"], 0)
        torch.cuda.synchronize()
        rep = compare_quantized("int4_asym", codes.cpu().numpy(), scales.cpu().numpy(), ora)
        assert rep["code_mismatch_exempt"] == 0
