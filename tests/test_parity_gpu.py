"""Parity of the CUDA path (called through the C ABI) with the CPU oracle, on a B200."""
import numpy as np
import pytest
import torch

from paper_2601_22347_b200 import inputs

from parity import compare_quantized, compare_rotated, unpack_nibbles, int4_values

pytestmark = pytest.mark.gpu

FMT = {"int4": 0, "mxfp4": 1, "fp4": 3, "int4_asym": 4}


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2601_22347_b200 import binding, build
    build.build()
    binding.load()
    return binding


@pytest.fixture(autouse=True)
def clean_error_word(B):
    """Every test starts from a cleared device error word and must leave it clear."""
    B.perq_device_error_clear()
    yield
    assert B.perq_device_error() == 0


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def run_gpu(B, w: inputs.Workload, x_dev=None):
    x = to_dev(w.x) if x_dev is None else x_dev
    perm = None if w.perm is None else torch.from_numpy(w.perm).cuda()
    codes, scales = B.perq_rotate_quantize(x, perm, w.b, FMT[w.fmt], w.group)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy()


def check(B, oracle, w: inputs.Workload, rows=None):
    """Full comparison when rows is None, else the GPU runs everything and the oracle the sampled rows."""
    codes, scales = run_gpu(B, w)
    xs = w.x if rows is None else w.x[rows]
    ora = oracle.rotate_quantize(xs, w.perm, w.b, FMT[w.fmt], w.group, want_pre=True)
    if rows is not None:
        codes, scales = codes[rows], scales[rows]
    rep = compare_quantized(w.fmt, codes, scales, ora)
    print("%s T=%d d=%d b=%d %s g=%d: %d elements, %d tie-window exemptions, scale ulp max %d"
          % (w.name, w.T, w.d, w.b, w.fmt, w.group, rep["elements"], rep["code_mismatch_exempt"],
             rep["scale_ulp_max"]))
    return rep


# ------------------------------------------------------------------ the five workloads

def test_config1_full(B, oracle):
    check(B, oracle, inputs.config1())


@pytest.mark.parametrize("b", [16, 32, 64, 128, 2048])
def test_config2(B, oracle, b):
    check(B, oracle, inputs.config2(T=768 if b <= 128 else 96, b=b))


def test_config3_with_massdiff_permutation(B, oracle):
    w = inputs.config3(T=320)
    x = to_dev(w.x)
    chan, _, _ = B.perq_block_l1_stats(x, None, w.b, want=("chan",))
    torch.cuda.synchronize()
    w.perm = B.perq_massdiff_perm(chan.cpu().numpy(), w.b)
    assert sorted(w.perm.tolist()) == list(range(w.d))
    status = B.perq_validate_perm(torch.from_numpy(w.perm).cuda())
    assert int(status.item()) == 0
    check(B, oracle, w)
    # the permutation does what it is for: it lowers the largest per-block l1 mass
    _, blk_id, _ = B.perq_block_l1_stats(x, None, w.b, want=("block",))
    _, blk_md, _ = B.perq_block_l1_stats(x, torch.from_numpy(w.perm).cuda(), w.b, want=("block",))
    assert float(blk_md.max()) < float(blk_id.max())


@pytest.mark.parametrize("fmt", ["int4", "mxfp4"])
@pytest.mark.parametrize("b", [16, 32, 128, 4096])
def test_config4_full_size_sampled(B, oracle, b, fmt):
    w = inputs.config4(T=16384, b=b, fmt=fmt)
    rows = np.sort(np.random.default_rng(4).choice(w.T, 96 if b < 4096 else 24, replace=False))
    rows[0], rows[-1] = 0, w.T - 1
    check(B, oracle, w, rows=rows)


@pytest.mark.parametrize("T", [1, 16, 128])
@pytest.mark.parametrize("b", [16, 32, 64, 128])
def test_config5_small_T(B, oracle, T, b):
    check(B, oracle, inputs.config5(T=T, b=b))


def test_config5_large_T_sampled(B, oracle):
    w = inputs.config5(T=1024, b=128)
    rows = np.sort(np.random.default_rng(5).choice(w.T, 64, replace=False))
    check(B, oracle, w, rows=rows)


# ------------------------------------------------------------------ the tensor-core fast path, every variant

@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32)])
@pytest.mark.parametrize("b", [16, 32, 64, 128])
@pytest.mark.parametrize("d,T", [(1024, 67), (2048, 301), (4096, 130), (8192, 45)])
def test_fast_path_matrix(B, oracle, d, T, b, fmt, group):
    bits, _ = inputs.student_t_outliers(T, d, 3.0, max(2, d // 256), 100.0, seed=1000 + d + b)
    bits[3] = 0                                   # an all-zero row in the middle of a CTA's work
    bits[5, 128:384] = 0                          # zero groups / zero MX blocks
    check(B, oracle, inputs.Workload("fast", bits, None, b, fmt, group, 0))


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32)])
def test_fast_path_many_units_per_warp(B, oracle, fmt, group):
    # enough rows that every warp of every CTA goes round its ring several times
    w = inputs.config4(T=16384, b=64, fmt=fmt)
    w.group = group
    rows = np.sort(np.random.default_rng(6).choice(w.T, 80, replace=False))
    rows[0], rows[-1] = 0, w.T - 1
    check(B, oracle, w, rows=rows)
    assert B.perq_device_error() == 0


def test_fast_path_exact_ties(B, oracle):
    import scipy.linalg
    H = scipy.linalg.hadamard(16)
    rng = np.random.default_rng(18)
    rows = []
    for _ in range(24):
        blocks = []
        for j in range(64):
            ystar = rng.integers(-13, 14, size=16) * 0.5
            ystar[rng.integers(0, 16)] = 7.0 if j == 0 else ystar[0]
            blocks.append((ystar @ H) / 4.0)
        rows.append(np.concatenate(blocks))
    x = np.array(rows, np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    rep = check(B, oracle, inputs.Workload("fast-ties", bits, None, 16, "int4", 0, 0))
    assert rep["code_mismatch_exempt"] == 0
    rep = check(B, oracle, inputs.Workload("fast-ties-g", bits, None, 16, "int4", 128, 0))
    assert rep["code_mismatch_exempt"] == 0
    rep = check(B, oracle, inputs.Workload("fast-ties-mx", inputs.f32_to_bf16_bits(x * 0.5), None, 16, "mxfp4", 32, 0))
    assert rep["code_mismatch_exempt"] == 0


# ------------------------------------------------------------------ rotated values (debug format)

@pytest.mark.parametrize("d,b,perm", [(2048, 16, False), (2048, 128, True), (4096, 4096, False),
                                      (14336, 64, True), (8192, 32, False), (2048, 2048, True),
                                      (3072, 3072, False), (14336, 14336, True), (9728, 9728, False)])
def test_rotated_values(B, oracle, d, b, perm):
    bits, _ = inputs.laplace_outliers(48, d, 4, 200.0, seed=77 + d + b)
    p = inputs.random_perm(d, 78) if perm else None
    x = to_dev(bits)
    y, _ = B.perq_rotate_quantize(x, None if p is None else torch.from_numpy(p).cuda(), b, B.PERQ_FMT_F32_DEBUG, 0)
    torch.cuda.synchronize()
    rep = compare_rotated(y.cpu().numpy(), oracle.rotate(bits, p, b), b)
    print("rotated d=%d b=%d: max %.2e rms %.2e of block max" % (d, b, rep["max_rel_to_block_max"], rep["rms_rel"]))


# ------------------------------------------------------------------ edge cases

def test_empty_and_tiny_T(B, oracle):
    x = torch.empty((0, 2048), dtype=torch.bfloat16, device="cuda")
    codes, scales = B.perq_rotate_quantize(x, None, 16, 0, 0)
    assert codes.shape == (0, 1024) and scales.shape == (0, 1)
    for T in (1, 3):
        w = inputs.config1(T=T, variant=T)
        check(B, oracle, w)
        w.fmt, w.group = "mxfp4", 32
        check(B, oracle, w)


def test_zero_rows_and_zero_groups(B, oracle):
    w = inputs.config2(T=8, b=32)
    w.x[1] = 0
    w.x[2, :] = 0
    w.x[3, 256:512] = 0           # two whole groups of 128 (under the identity permutation)
    w.perm = None
    check(B, oracle, w)
    w.fmt, w.group = "mxfp4", 32
    check(B, oracle, w)
    codes, scales = run_gpu(B, w)
    assert not codes[1].any() and not scales[1].any()


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32), ("fp4", 0), ("int4_asym", 0)])
@pytest.mark.parametrize("d,b", [(4096, 32), (2048, 16), (8192, 64), (3072, 128)])
def test_padded_rows_and_padded_channels(B, oracle, d, b, fmt, group):
    """Zero rows (padding tokens) and all-zero blocks (padding channels) between dense rows: exact zeros take the
    code +0 and the scale of an empty range, through the persistent kernels' main loops (many rows per group)."""
    T = 640
    bits, _ = inputs.laplace_outliers(T, d, 4, 200.0, seed=11)
    bits[::3] = 0                                  # every third row
    bits[:, 2 * b:3 * b] = 0                       # one Hadamard block of every row
    bits[5::7, d // 2:] = 0                        # the second half of some rows
    bits[:, 7] = 0                                 # one zero channel inside a dense block
    w = inputs.Workload(name="padded", x=bits, perm=None, b=b, fmt=fmt, group=group, seed=11)
    check(B, oracle, w)
    codes, scales = run_gpu(B, w)
    assert not codes[0].any()
    if fmt != "int4_asym":
        assert not scales[0].any()


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("mxfp4", 32), ("fp4", 0)])
def test_padding_does_not_slow_a_call_down(B, fmt, group):
    """Exact zeros must stay on the fast path of the rounding test: a call on padded rows may not take several
    times as long as the same call on dense rows (an E2M1 zero flagged for its sign goes to the exact path)."""
    T, d, b = 4096, 4096, 32
    dense, _ = inputs.laplace_outliers(T, d, 4, 200.0, seed=12)
    padded = dense.copy()
    padded[::2] = 0
    padded[:, 64:96] = 0

    def timed(bits):
        x = to_dev(bits)
        oc, os_ = B.alloc_outputs(T, d, FMT[fmt], group, x.device)
        for _ in range(3):
            B.perq_rotate_quantize(x, None, b, FMT[fmt], group, out_codes=oc, out_scales=os_)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            B.perq_rotate_quantize(x, None, b, FMT[fmt], group, out_codes=oc, out_scales=os_)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 20

    t_dense, t_padded = timed(dense), timed(padded)
    print("%s: dense %.1f us, padded %.1f us" % (fmt, 1e3 * t_dense, 1e3 * t_padded))
    assert t_padded < 2.5 * t_dense


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32), ("fp4", 0), ("int4_asym", 0)])
@pytest.mark.parametrize("d,T,perm", [(3072, 40, False), (14336, 6, False), (9728, 5, True), (6144, 300, False), (12288, 9, True)])
def test_full_vector_rotation_of_rows_that_are_not_a_power_of_two(B, oracle, d, T, perm, fmt, group):
    """b = d = 2^k' * 4t (Appendix A.1: Llama-3-8B's 14336 = 2^9 * 28, Qwen3's 3072 / 6144 / 12288 = 2^k' * 12 and
    9728 = 2^7 * 76): base-matrix rotations of adjacent inputs, then butterflies, every format."""
    bits, _ = inputs.laplace_outliers(T, d, 4, 200.0, seed=500 + d)
    bits[1] = 0
    if T > 3:
        bits[3, : d // 2] = 0
    w = inputs.Workload("non-po2 full vector", bits, inputs.random_perm(d, 9) if perm else None, d, fmt, group, 0)
    check(B, oracle, w)


def test_single_huge_outlier_and_basis_rows(B, oracle):
    d = 2048
    x = np.zeros((6, d), np.float32)
    x[0, 77] = 3.0e4                      # one nonzero: every output of its block has the same magnitude
    x[1, 5] = 1.0
    x[1, 1029] = -2.5
    x[2] = 1.0                            # constant row: all mass lands on the first coordinate of each block
    x[3] = np.random.default_rng(1).standard_normal(d) * 1e-3
    x[3, 100] = 6.0e4
    x[4] = np.random.default_rng(2).standard_normal(d)
    x[4, 1000:1016] = 0
    x[5, ::2] = 1.0
    x[5, 1::2] = -1.0
    bits = inputs.f32_to_bf16_bits(x)
    for b in (16, 128, 2048):
        for fmt, g in (("int4", 0), ("int4", 128), ("mxfp4", 32)):
            check(B, oracle, inputs.Workload("edge", bits, None, b, fmt, g, 0))


def test_constructed_exact_ties(B, oracle):
    """Rows built so that the rotated values are exact k + 1/2 multiples of the step: the
    CUDA path has to resolve them like exact arithmetic does (round half to even)."""
    import scipy.linalg
    H = scipy.linalg.hadamard(16)
    rng = np.random.default_rng(8)
    rows = []
    for _ in range(32):
        blocks = []
        for j in range(8):
            ystar = rng.integers(-13, 14, size=16) * 0.5          # halves in [-6.5, 6.5]
            ystar[rng.integers(0, 16)] = 7.0 if j == 0 else ystar[0]
            blocks.append((ystar @ H) / 4.0)
        rows.append(np.concatenate(blocks))
    x = np.array(rows, np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    w = inputs.Workload("ties", bits, None, 16, "int4", 0, 0)
    rep = check(B, oracle, w)
    assert rep["code_mismatch_exempt"] == 0          # exact ties are not approximated: they must match
    ora = oracle.rotate_quantize(bits, None, 16, 0, 0, want_pre=True)
    assert (np.abs(ora["pre"] - np.floor(ora["pre"])) == 0.5).sum() > 500
    # the same rows scaled so that MX midpoints are hit: amax 7 -> E = 0, halves/quarters are midpoints
    w2 = inputs.Workload("ties-mx", inputs.f32_to_bf16_bits(x * 0.5), None, 16, "mxfp4", 32, 0)
    rep2 = check(B, oracle, w2)
    assert rep2["code_mismatch_exempt"] == 0


def test_mx_saturation_band(B, oracle):
    """Values in (6, 8) * 2^E must saturate to the largest E2M1 magnitude."""
    d = 64
    x = np.zeros((4, d), np.float32)
    x[:, 0] = [7.5 * 4, 6.5 * 4, 7.0 * 4, 4.0 * 4]     # with b = 16 a lone entry spreads as x/4 over its block
    bits = inputs.f32_to_bf16_bits(x)
    w = inputs.Workload("sat", bits, None, 16, "mxfp4", 32, 0)
    check(B, oracle, w)
    codes, scales = run_gpu(B, w)
    nib = unpack_nibbles(codes)
    assert np.all(nib[:3, :16] == 7) and np.all(nib[3, :16] == 6)


@pytest.mark.parametrize("kind", ["reversal", "interleave", "random"])
def test_permutations(B, oracle, kind):
    d = 2048
    if kind == "reversal":
        perm = np.arange(d - 1, -1, -1, dtype=np.int32)
    elif kind == "interleave":
        perm = np.arange(d, dtype=np.int32).reshape(32, 64).T.reshape(-1).copy()
    else:
        perm = inputs.random_perm(d, 99)
    w = inputs.config2(T=64, b=64)
    w.perm = perm
    check(B, oracle, w)


def test_group_smaller_than_block_and_other_groups(B, oracle):
    for b, g in ((128, 32), (2048, 64), (16, 8), (64, 256), (32, 1024)):
        w = inputs.config2(T=32, b=b)
        w.group = g
        check(B, oracle, w)


def test_outputs_are_deterministic_and_stay_inside_their_buffers(B):
    w = inputs.config2(T=200, b=128)
    x = to_dev(w.x)
    perm = torch.from_numpy(w.perm).cuda()
    cb, sb = B.perq_out_sizes(w.T, w.d, 0, 128)
    guard = 4096
    bufc = torch.full((cb + guard,), 0xA5, dtype=torch.uint8, device="cuda")
    bufs = torch.full((sb + guard,), 0x5A, dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        bufc.fill_(0xA5); bufs.fill_(0x5A)
        B.perq_rotate_quantize(x, perm, 128, 0, 128, out_codes=bufc, out_scales=bufs)
        torch.cuda.synchronize()
        assert bool((bufc[cb:] == 0xA5).all()) and bool((bufs[sb:] == 0x5A).all())
        outs.append((bufc[:cb].clone(), bufs[:sb].clone()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_row_sharding_gives_identical_bytes(B):
    """Rows are independent: running two halves separately (as two ranks would) must
    reproduce the unsharded call byte for byte."""
    w = inputs.config4(T=512, b=32, fmt="mxfp4")
    x = to_dev(w.x)
    c_all, s_all = B.perq_rotate_quantize(x, None, 32, 1, 32)
    c0, s0 = B.perq_rotate_quantize(x[:200].contiguous(), None, 32, 1, 32)
    c1, s1 = B.perq_rotate_quantize(x[200:].contiguous(), None, 32, 1, 32)
    torch.cuda.synchronize()
    assert torch.equal(torch.cat([c0, c1]), c_all) and torch.equal(torch.cat([s0, s1]), s_all)


def test_host_buffer_entry_point(B, oracle):
    w = inputs.config1(T=64)
    xh = torch.from_numpy(w.x.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    ws = torch.empty(B.perq_host_workspace_bytes(w.T, w.d, 0, 0), dtype=torch.uint8, device="cuda")
    codes = torch.empty((w.T, w.d // 2), dtype=torch.uint8).pin_memory()
    scales = torch.empty((w.T, 1), dtype=torch.float32).pin_memory()
    B.perq_rotate_quantize_host(xh, None, 16, 0, 0, codes, scales, ws)
    ora = oracle.rotate_quantize(w.x, None, 16, 0, 0, want_pre=True)
    compare_quantized("int4", codes.numpy(), scales.numpy(), ora)


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("mxfp4", 32), ("int4", 128)])
def test_host_entry_point_in_chunks_matches_the_device_entry_point(B, fmt, group):
    """From 4096 rows on, the host-buffer call works in chunks of rows with the two copy
    directions overlapped; its bytes must equal those of one device call."""
    T, d, b = 5001, 2048, 32
    bits, _ = inputs.student_t_outliers(T, d, 3.0, 8, 100.0, seed=7000)
    f = FMT[fmt]
    x = to_dev(bits)
    codes_d, scales_d = B.perq_rotate_quantize(x, None, b, f, group)
    torch.cuda.synchronize()
    xh = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    ws = torch.empty(B.perq_host_workspace_bytes(T, d, f, group), dtype=torch.uint8, device="cuda")
    codes_h = torch.empty_like(codes_d, device="cpu").pin_memory()
    scales_h = torch.empty_like(scales_d, device="cpu").pin_memory()
    for _ in range(2):
        codes_h.zero_(); scales_h.zero_()
        B.perq_rotate_quantize_host(xh, None, b, f, group, codes_h, scales_h, ws)
        assert torch.equal(codes_h, codes_d.cpu()) and torch.equal(scales_h, scales_d.cpu())


def test_invalid_permutation_is_reported_not_faulted(B):
    d = 2048
    bad = inputs.random_perm(d, 3)
    bad[10] = bad[11]
    assert int(B.perq_validate_perm(torch.from_numpy(bad).cuda()).item()) == 2
    bad2 = inputs.random_perm(d, 3)
    bad2[0] = d + 5
    bad2[1] = -1
    st = int(B.perq_validate_perm(torch.from_numpy(bad2).cuda()).item())
    assert st & 1
    # out-of-range entries are clamped by the main kernel: it must finish without an error
    w = inputs.config2(T=16, b=32)
    x = to_dev(w.x)
    B.perq_rotate_quantize(x, torch.from_numpy(bad2).cuda(), 32, 0, 128)
    torch.cuda.synchronize()


# ------------------------------------------------------------------ statistic

@pytest.mark.parametrize("T,d,b,perm", [(320, 8192, 32, True), (1000, 2048, 16, False), (37, 14336, 128, True),
                                        (5, 4096, 4096, False), (700, 4096, 8, True)])
def test_block_l1_stats(B, oracle, T, d, b, perm):
    bits, _ = inputs.swiglu_outliers(T, d, 32, 30.0, seed=300 + T)
    p = inputs.random_perm(d, 301) if perm else None
    x = to_dev(bits)
    pd = None if p is None else torch.from_numpy(p).cuda()
    chan, block, token = B.perq_block_l1_stats(x, pd, b)
    chan2, block2, token2 = B.perq_block_l1_stats(x, pd, b)
    torch.cuda.synchronize()
    assert torch.equal(chan, chan2) and torch.equal(block, block2) and torch.equal(token, token2)
    cas, blm, tmx = oracle.block_l1_stats(bits, p, b)
    # fp32 accumulation in a fixed order: 1e-5 relative covers T up to a few thousand rows
    assert np.allclose(chan.cpu().numpy(), cas, rtol=1e-5, atol=0)
    assert np.allclose(block.cpu().numpy(), blm, rtol=1e-5, atol=0)
    assert np.allclose(token.cpu().numpy(), tmx, rtol=1e-5, atol=0)
    # only some outputs requested
    only_tok = B.perq_block_l1_stats(x, pd, b, want=("token",))
    torch.cuda.synchronize()
    assert only_tok[0] is None and only_tok[1] is None and torch.equal(only_tok[2], token)


# ------------------------------------------------------------------ fast-kernel variants added later: permuted, full-vector

@pytest.mark.parametrize("fmt,group", [("int4", 0), ("int4", 128), ("mxfp4", 32)])
@pytest.mark.parametrize("d,T,b", [(1024, 70, 16), (2048, 333, 32), (4096, 150, 64), (8192, 40, 128), (14336, 20, 32)])
def test_permuted_fast_path_matrix(B, oracle, d, T, b, fmt, group):
    bits, _ = inputs.student_t_outliers(T, d, 3.0, max(2, d // 256), 100.0, seed=2000 + d + b)
    bits[2] = 0
    bits[4, 64:320] = 0
    perm = inputs.random_perm(d, 2001 + d)
    check(B, oracle, inputs.Workload("perm-fast", bits, perm, b, fmt, group, 0))
    assert B.perq_device_error() == 0


@pytest.mark.parametrize("fmt,group", [("int4", 0), ("mxfp4", 32)])
@pytest.mark.parametrize("d,T", [(1024, 40), (2048, 64), (4096, 24), (8192, 12)])
def test_full_vector_fast_path(B, oracle, d, T, fmt, group):
    bits, _ = inputs.laplace_outliers(T, d, 4, 200.0, seed=3000 + d)
    bits[1] = 0
    bits[3, : d // 2] = 0
    check(B, oracle, inputs.Workload("full-fast", bits, None, d, fmt, group, 0))
    assert B.perq_device_error() == 0


def test_rows_with_several_maximum_candidates(B, oracle):
    """Rows whose largest rotated magnitude is attained (exactly) in several places -- in one
    warp's segment, in several segments, in every block -- take the paths that resolve the
    exact maximum at once and combine it across the warps of a row."""
    d = 4096
    rng = np.random.default_rng(31)
    x = (rng.standard_normal((12, d)) * 0.01).astype(np.float32)
    x[0, 5] = 300.0;  x[0, 5 + 1024] = 300.0                 # equal outliers in two segments
    x[1, 7] = -300.0; x[1, 7 + 32] = 300.0                   # and in two blocks of one segment
    x[2, :] = 0.0;    x[2, 100] = 64.0                       # a lone entry: every output of its block ties
    x[3, :] = 0.0;    x[3, 0::1024] = 8.0                    # one per segment, identical
    x[4, :] = 1.0                                            # constant row: first output of every block
    x[5, :] = 0.0;    x[5, 2049] = 1.0; x[5, 3] = -1.0
    x[6, 9] = 300.0;  x[6, 9 + 2048] = 300.0; x[6, 9 + 3072] = -300.0
    bits = inputs.f32_to_bf16_bits(x)
    for b in (16, 32, 128, 256, 1024, 4096):
        for fmt, g in (("int4", 0), ("int4", 128), ("mxfp4", 32)):
            if b == 4096 and g == 128:
                continue
            check(B, oracle, inputs.Workload("multi-cand", bits, None, b, fmt, g, 0))
    p = inputs.random_perm(d, 32)
    for b in (32, 128):
        for fmt, g in (("int4", 0), ("int4", 128), ("mxfp4", 32)):
            check(B, oracle, inputs.Workload("multi-cand-perm", bits, p, b, fmt, g, 0))
    assert B.perq_device_error() == 0


def test_exact_ties_through_the_permuted_and_full_vector_paths(B, oracle):
    """Constructed exact rounding ties (see test_constructed_exact_ties) must also be resolved like
    exact arithmetic when the row goes through the permutation gather, and for whole-row blocks."""
    import scipy.linalg
    rng = np.random.default_rng(28)
    # b = 16 blocks of a d = 2048 row, then scattered by the inverse of a permutation
    H = scipy.linalg.hadamard(16)
    rows = []
    for _ in range(16):
        blocks = []
        for j in range(128):
            ystar = rng.integers(-13, 14, size=16) * 0.5
            ystar[rng.integers(0, 16)] = 7.0 if j == 0 else ystar[0]
            blocks.append((ystar @ H) / 4.0)
        rows.append(np.concatenate(blocks))
    xp = np.array(rows, np.float32)                      # the permuted row the kernel should see
    perm = inputs.random_perm(2048, 29)
    x = np.empty_like(xp)
    x[:, perm] = xp                                      # x[perm[i]] = xp[i]
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    for fmt, g, scale in (("int4", 0, 1.0), ("int4", 128, 1.0), ("mxfp4", 32, 0.5)):
        rep = check(B, oracle, inputs.Workload("ties-perm", inputs.f32_to_bf16_bits(x * np.float32(scale)), perm, 16, fmt, g, 0))
        assert rep["code_mismatch_exempt"] == 0
    # whole-row block, d = 1024 (sqrt(d) = 32): rotated values are small half-integers, maximum 7
    H = scipy.linalg.hadamard(1024)
    rows = []
    for _ in range(6):
        ystar = rng.integers(-13, 14, size=1024) * 0.5
        ystar[rng.integers(0, 1024)] = 7.0
        rows.append((ystar @ H) / 32.0)
    x = np.array(rows, np.float64)
    bits = inputs.f32_to_bf16_bits(x.astype(np.float32))
    if np.array_equal(inputs.bf16_to_f64(bits), x):      # representable in bf16: exact ties survive the cast
        rep = check(B, oracle, inputs.Workload("ties-full", bits, None, 1024, "int4", 0, 0))
        assert rep["code_mismatch_exempt"] == 0
    else:                                                # otherwise still a valid parity case
        check(B, oracle, inputs.Workload("ties-full", bits, None, 1024, "int4", 0, 0))


def test_permuted_path_many_rows_per_group(B, oracle):
    # enough rows that every group goes round its three-stage ring many times, and the deferred
    # scale records fill and are served in the middle of the run
    w = inputs.config2(T=16384, b=32)
    w.group = 0
    rows = np.sort(np.random.default_rng(7).choice(w.T, 64, replace=False))
    rows[0], rows[-1] = 0, w.T - 1
    check(B, oracle, w, rows=rows)
    w = inputs.config5(T=2048, b=64)
    rows = np.sort(np.random.default_rng(8).choice(w.T, 24, replace=False))
    check(B, oracle, w, rows=rows)
    assert B.perq_device_error() == 0


@pytest.mark.parametrize("d,b,T,perm", [(4096, 256, 40, False), (8192, 512, 24, True), (8192, 2048, 16, False),
                                        (4096, 1024, 24, True), (14336, 2048, 6, True), (8192, 512, 150, False),
                                        (4096, 1024, 70, False), (2048, 1024, 301, False), (1024, 256, 67, False)])
def test_intermediate_block_sizes(B, oracle, d, b, T, perm):
    """Block sizes between 128 and d (the paper's block-size sweep goes 16 ... 2048 at d = 8192)."""
    bits, _ = inputs.gaussian_outliers(T, d, 8, 50.0, seed=4000 + d + b)
    p = inputs.random_perm(d, 4001) if perm else None
    for fmt, g in (("int4", 0), ("int4", 128), ("mxfp4", 32)):
        check(B, oracle, inputs.Workload("mid-b", bits, p, b, fmt, g, 0))


def test_randomised_shapes_and_modes(B, oracle):
    """A seeded sweep over shapes, block sizes, formats, groups, permutations and value
    distributions (including rows scaled far up and down), every case held to the oracle."""
    rng = np.random.default_rng(2601)
    ds = [256, 1024, 1536, 2048, 3072, 4096, 6144, 8192, 14336]
    n_cases = 40
    for case in range(n_cases):
        d = int(rng.choice(ds))
        bs = [b for b in (16, 32, 64, 128, 256, 512, 1024, 2048, 4096, 8192) if b <= d and d % b == 0]
        b = int(rng.choice(bs))
        fmt, g = [("int4", 0), ("int4", 128), ("int4", 32), ("mxfp4", 32)][int(rng.integers(0, 4))]
        if fmt == "int4" and g and d % g:
            g = 0
        T = int(rng.integers(1, 40))
        kind = int(rng.integers(0, 3))
        seed = 5000 + case
        if kind == 0:
            bits, _ = inputs.gaussian_outliers(T, d, int(rng.integers(0, 9)), 50.0, seed)
        elif kind == 1:
            bits, _ = inputs.student_t_outliers(T, d, 3.0, int(rng.integers(0, 17)), 100.0, seed)
        else:
            bits, _ = inputs.laplace_outliers(T, d, int(rng.integers(0, 5)), 200.0, seed)
        # rows at very different magnitudes (exact powers of two keep the values bf16)
        scale = np.exp2(rng.integers(-30, 31, size=(T, 1))).astype(np.float32)
        bits = inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(bits) * scale)
        perm = inputs.random_perm(d, seed + 1) if rng.random() < 0.5 else None
        check(B, oracle, inputs.Workload("fuzz%d" % case, bits, perm, b, fmt, g, seed))
    assert B.perq_device_error() == 0


@pytest.mark.parametrize("d,T", [(3072, 90), (6144, 70), (12288, 30), (14336, 33)])
def test_per_token_scales_for_rows_of_any_number_of_segments(B, oracle, d, T):
    bits, _ = inputs.laplace_outliers(T, d, 6, 200.0, seed=6000 + d)
    bits[5] = 0
    for b in (16, 128):
        check(B, oracle, inputs.Workload("token-anyG", bits, None, b, "int4", 0, 0))
    check(B, oracle, inputs.Workload("token-anyG-perm", bits, inputs.random_perm(d, 6001), 32, "int4", 0, 0))
    assert B.perq_device_error() == 0


# ------------------------------------------------------------------ E2M1 with a per-token scale

@pytest.mark.parametrize("perm", [False, True])
@pytest.mark.parametrize("d,T,b", [(1024, 67, 16), (2048, 301, 32), (4096, 130, 64), (8192, 45, 128), (6144, 40, 32),
                                   (1536, 33, 32), (4096, 20, 4096), (4096, 24, 512)])
def test_fp4_per_token(B, oracle, d, T, b, perm):
    bits, _ = inputs.student_t_outliers(T, d, 3.0, max(2, d // 256), 100.0, seed=8000 + d + b)
    bits[3] = 0
    bits[5, 128:384] = 0
    p = inputs.random_perm(d, 8001) if perm else None
    check(B, oracle, inputs.Workload("fp4", bits, p, b, "fp4", 0, 0))
    assert B.perq_device_error() == 0


def test_fp4_exact_midpoints_and_saturation(B, oracle):
    import scipy.linalg
    H = scipy.linalg.hadamard(16)
    rng = np.random.default_rng(88)
    rows = []
    for _ in range(24):
        blocks = []
        for j in range(64):
            ystar = rng.integers(-26, 27, size=16) * 0.25          # quarters in [-6.5, 6.5]: every midpoint occurs
            ystar[rng.integers(0, 16)] = 7.0 if j == 0 else ystar[0]
            blocks.append((ystar @ H) / 4.0)
        rows.append(np.concatenate(blocks))
    x = np.array(rows, np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    rep = check(B, oracle, inputs.Workload("fp4-ties", bits, None, 16, "fp4", 0, 0))
    assert rep["code_mismatch_exempt"] == 0
    rep = check(B, oracle, inputs.Workload("fp4-ties-perm", bits, inputs.random_perm(1024, 89), 16, "fp4", 0, 0))
    w = inputs.config4(T=16384, b=32, fmt="fp4")
    w.group = 0
    rows_ = np.sort(np.random.default_rng(9).choice(w.T, 64, replace=False))
    check(B, oracle, w, rows=rows_)


# ------------------------------------------------------------------ asymmetric INT4 per token

@pytest.mark.parametrize("perm", [False, True])
@pytest.mark.parametrize("d,T,b", [(1024, 40, 16), (2048, 100, 32), (4096, 60, 128), (8192, 20, 64), (1536, 33, 32),
                                   (2048, 12, 2048), (14336, 9, 32)])
def test_asymmetric_int4_per_token(B, oracle, d, T, b, perm):
    bits, _ = inputs.student_t_outliers(T, d, 3.0, max(2, d // 256), 100.0, seed=9000 + d + b)
    x = inputs.bf16_bits_to_f32(bits)
    x[1] += 3.0                      # a row whose range is far from symmetric
    x[2] = 0.0                       # constant rows: step 0
    x[3] = 1.5
    bits = inputs.f32_to_bf16_bits(x)
    p = inputs.random_perm(d, 9001) if perm else None
    check(B, oracle, inputs.Workload("asym", bits, p, b, "int4_asym", 0, 0))


def test_asymmetric_int4_exact_ties(B, oracle):
    import scipy.linalg
    H = scipy.linalg.hadamard(16)
    rng = np.random.default_rng(98)
    rows = []
    for _ in range(16):
        blocks = []
        for j in range(64):
            ystar = rng.integers(-13, 17, size=16) * 0.5           # halves in [-6.5, 8]
            if j == 0:
                ystar[0], ystar[1] = -7.0, 8.0                     # range 15 -> step 1, zero point -7
            blocks.append((ystar @ H) / 4.0)
        rows.append(np.concatenate(blocks))
    x = np.array(rows, np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    rep = check(B, oracle, inputs.Workload("asym-ties", bits, None, 16, "int4_asym", 0, 0))
    assert rep["code_mismatch_exempt"] == 0


def _asym_constructed_rows():
    """Rows built in the rotated domain (H_16 is an involution up to the factor 16), every input exactly a
    bf16 value: blocks are redrawn until they are."""
    import scipy.linalg
    H = scipy.linalg.hadamard(16)
    rng = np.random.default_rng(99)
    nblk = 256

    def representable(xb):
        xb = xb.astype(np.float32)
        return np.array_equal(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(xb)), xb)

    def block(draw, fix=None):
        for _ in range(1000):
            yb = draw().astype(np.float64)
            if fix:
                for pos, val in fix.items():
                    yb[pos] = val
            xb = (yb @ H) / 4.0
            if representable(xb):
                return xb
        raise AssertionError("no representable block found")

    def row(draw, fixes):
        return np.concatenate([block(draw, fixes.get(j)) for j in range(nblk)])

    rows = []
    # (a) even integers, min -26, max 34: step 4, min / step = -6.5 is a tie (zero point -6), v = y / 4 in halves
    rows.append(row(lambda: rng.integers(-12, 17, size=16) * 2.0, {3: {5: -26.0}, 200: {9: 34.0}}))
    # (b) all positive: multiples of 4 in [4, 64]: step 4, zero point 1
    rows.append(row(lambda: rng.integers(1, 17, size=16) * 4.0, {0: {0: 4.0}, 255: {15: 64.0}}))
    # (c) the same extremes in every 1024-element segment (64 blocks each), twice in one slot
    fixes = {}
    for seg in range(4):
        fixes[64 * seg + 7] = {2: 24.0, 3: 24.0}
        fixes[64 * seg + 40] = {12: -36.0}
        fixes[64 * seg + 41] = {1: -36.0}
    rows.append(row(lambda: rng.integers(-10, 11, size=16) * 1.0, fixes))
    # (d) constant rotated row
    rows.append(row(lambda: np.full(16, 2.0), {}))
    # (e) random even integers: codes in halves of the step whenever the range is 60
    for _ in range(4):
        rows.append(row(lambda: rng.integers(-15, 16, size=16) * 2.0, {1: {0: -30.0}, 2: {0: 30.0}}))
    x = np.array(rows, np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), x)
    return bits


def test_asymmetric_int4_constructed_rows(B, oracle):
    """A zero point that is an exact tie, an all-positive row, extremes repeated in every segment, a constant
    rotated row, and rows full of exact rounding ties; also through a permutation."""
    bits = _asym_constructed_rows()
    d = bits.shape[1]
    for perm in (None, inputs.random_perm(d, 991)):
        pb = bits
        if perm is not None:      # so that the gathered row is the constructed one: pb[:, perm[i]] = bits[:, i]
            pb = np.empty_like(bits)
            pb[:, perm] = bits
        rep = check(B, oracle, inputs.Workload("asym-constructed", pb, perm, 16, "int4_asym", 0, 0))
        assert rep["code_mismatch_exempt"] == 0


@pytest.mark.parametrize("d,b", [(1024, 32), (2048, 64), (4096, 32), (8192, 128), (6144, 16), (14336, 64), (15360, 32)])
def test_asymmetric_int4_persistent_kernel_shapes(B, oracle, d, b):
    bits, _ = inputs.laplace_outliers(150, d, max(1, d // 1024), 200.0, seed=9100 + d)
    x = inputs.bf16_bits_to_f32(bits)
    x[5] = np.abs(x[5]) + 0.5            # an all-positive row
    x[6] = 0.0
    bits = inputs.f32_to_bf16_bits(x)
    check(B, oracle, inputs.Workload("asym-shapes", bits, None, b, "int4_asym", 0, 0))


# ------------------------------------------------------------------ per-token diagnostics

@pytest.mark.parametrize("d,b,perm", [(1024, 16, False), (2048, 32, True), (4096, 128, False), (4096, 4096, False),
                                      (8192, 32, True), (1536, 64, True), (14336, 128, False)])
def test_token_diagnostics(B, oracle, d, b, perm):
    """fp32 on the device against fp64 definitions: 2e-5 relative (the sums run over up to 14336 fp32 terms; a
    code that flips at a near tie changes the error norm by less than the tie distance)."""
    T = 70
    bits, _ = inputs.laplace_outliers(T, d, max(1, d // 1024), 200.0, seed=9300 + d + b)
    x = inputs.bf16_bits_to_f32(bits)
    x[3] = 0.0                              # a zero row
    x[4] = 0.0
    x[4, 17] = -3.0                         # a one-hot row: no quantization error
    bits = inputs.f32_to_bf16_bits(x)
    p = inputs.random_perm(d, 9301) if perm else None
    ora = oracle.token_diagnostics(bits, p, b)
    got = B.perq_token_diagnostics(to_dev(bits), None if p is None else torch.from_numpy(p).cuda(), b)
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    assert np.array_equal(got[3], np.zeros(5))
    scale = np.maximum(np.abs(ora[:, 3:4]), 1e-30)
    assert np.allclose(got[:, :4], ora[:, :4], rtol=2e-5, atol=0)
    assert np.all(np.abs(got[:, 4] - ora[:, 4]) <= 2e-5 * ora[:, 4] + 1e-6 * scale[:, 0])
    assert got[4, 4] <= 1e-6 * got[4, 3]


# ------------------------------------------------------------------ Algorithm 1 on the device

@pytest.mark.parametrize("d,b", [(256, 16), (2048, 32), (8192, 32), (4096, 4096), (14336, 128), (1000, 8), (96, 1)])
def test_massdiff_on_the_device_matches_the_oracle(B, oracle, d, b):
    rng = np.random.default_rng(4100 + d + b)
    a = (rng.exponential(size=d) * np.where(rng.random(d) < 0.05, 40.0, 1.0)).astype(np.float32)
    a[rng.integers(0, d, 16)] = a[0]                     # equal masses: the index decides
    a[rng.integers(0, d, 4)] = 0.0
    ref = oracle.massdiff_perm(a.astype(np.float64), b)
    got = B.perq_massdiff_perm_device(torch.from_numpy(a).cuda(), b)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), ref)


def test_calibration_pass_stays_on_the_device(B, oracle):
    """statistic -> permutation -> permuted rotate+quantize without a host copy, against the oracle's chain."""
    w = inputs.config3(T=96)
    x = to_dev(w.x)
    chan, _, _ = B.perq_block_l1_stats(x, None, 32, want=("chan",))
    perm = B.perq_massdiff_perm_device(chan, 32)
    codes, scales = B.perq_rotate_quantize(x, perm, 32, FMT["mxfp4"], 32)
    torch.cuda.synchronize()
    cas, _, _ = oracle.block_l1_stats(w.x, None, 32)
    # the device sums are fp32: feed the oracle's greedy the same fp32 masses, then compare everything after it
    assert np.allclose(chan.cpu().numpy(), cas, rtol=1e-5)
    ref_perm = oracle.massdiff_perm(chan.cpu().numpy().astype(np.float64), 32)
    assert np.array_equal(perm.cpu().numpy(), ref_perm)
    ora = oracle.rotate_quantize(w.x, ref_perm, 32, FMT["mxfp4"], 32, want_pre=True)
    compare_quantized("mxfp4", codes.cpu().numpy(), scales.cpu().numpy(), ora)


@pytest.mark.parametrize("T,d", [(1, 64), (37, 2048), (4096, 8192), (1000, 14336), (5, 32768)])
def test_chan_abs_max_and_the_comparison_permutations(B, oracle, T, d):
    bits, _ = inputs.student_t_outliers(T, d, 3.0, max(1, d // 512), 100.0, seed=9500 + d)
    got = B.perq_chan_abs_max(to_dev(bits))
    torch.cuda.synchronize()
    ref = oracle.chan_abs_max(bits)
    assert np.array_equal(got.cpu().numpy().astype(np.float64), ref)        # a maximum of bf16 magnitudes: exact
    b = 32
    assert np.array_equal(B.perq_zigzag_perm(got.cpu().numpy(), b), oracle.zigzag_perm(ref, b))
    assert np.array_equal(B.perq_absmax_perm(got.cpu().numpy()), oracle.absmax_perm(ref))
