"""The gated-activation entry point (h = Swish(gate) * up, then rotate + quantize) against the oracle's chain."""
import numpy as np
import pytest
import torch

from paper_2601_22347_b200 import inputs

from parity import compare_quantized

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
    B.perq_device_error_clear()
    yield
    assert B.perq_device_error() == 0


def dev(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def projections(T, d, seed, n_out=8):
    """gate ~ N(0, 2^2), up ~ N(0, 1), a few channels of both scaled up (the shape of a gated MLP's two
    projections before the activation)."""
    rng = np.random.default_rng(seed)
    g = rng.standard_normal((T, d)) * 2.0
    u = rng.standard_normal((T, d))
    ch = rng.choice(d, n_out, replace=False)
    g[:, ch] *= 4.0
    u[:, ch] *= 20.0
    return inputs.f32_to_bf16_bits(g.astype(np.float32)), inputs.f32_to_bf16_bits(u.astype(np.float32))


def check(B, oracle, gate, up, b, fmt, group, rows=None):
    codes, scales = B.perq_swiglu_rotate_quantize(dev(gate), dev(up), None, b, FMT[fmt], group)
    torch.cuda.synchronize()
    codes, scales = codes.cpu().numpy(), scales.cpu().numpy()
    if rows is not None:
        gate, up, codes, scales = gate[rows], up[rows], codes[rows], scales[rows]
    h = oracle.swiglu(gate, up)
    ora = oracle.rotate_quantize(h, None, b, FMT[fmt], group, want_pre=True)
    rep = compare_quantized(fmt, codes, scales, ora)
    print("swiglu T=%d d=%d b=%d %s g=%d: %d tie-window exemptions" % (gate.shape[0], gate.shape[1], b, fmt, group,
                                                                      rep["code_mismatch_exempt"]))
    return h


@pytest.mark.parametrize("fmt,group", [("mxfp4", 32), ("int4", 128), ("int4", 0)])
@pytest.mark.parametrize("d,T,b", [(1024, 67, 16), (2048, 301, 32), (4096, 130, 64), (8192, 45, 128), (3072, 50, 32)])
def test_swiglu_matches_the_oracle_chain(B, oracle, d, T, b, fmt, group):
    gate, up = projections(T, d, 21000 + d + b)
    gate[3] = 0                                   # Swish(0) = 0: an all-zero row of h
    up[5, 128:384] = 0                            # zero groups
    check(B, oracle, gate, up, b, fmt, group)


def test_swiglu_equals_the_plain_entry_point_on_a_materialised_h(B, oracle):
    """Byte for byte: the codes and scales of the fused call are those of perq_rotate_quantize on the stored h."""
    T, d, b = 400, 4096, 32
    gate, up = projections(T, d, 22000)
    h = oracle.swiglu(gate, up)
    for fmt, group in (("mxfp4", 32), ("int4", 128), ("int4", 0)):
        c1, s1 = B.perq_swiglu_rotate_quantize(dev(gate), dev(up), None, b, FMT[fmt], group)
        c2, s2 = B.perq_rotate_quantize(dev(h), None, b, FMT[fmt], group)
        torch.cuda.synchronize()
        assert torch.equal(c1, c2)
        if fmt == "mxfp4":
            assert torch.equal(s1, s2)
        else:      # fp32 scales: the same exact maximum through two kernels, one more rounding of a constant at most
            a, bb = s1.cpu().numpy().view(np.int32).astype(np.int64), s2.cpu().numpy().view(np.int32).astype(np.int64)
            assert np.abs(a - bb).max() <= 1


def test_swiglu_special_values(B, oracle):
    """Arguments where the fp32 evaluation of the activation is not trusted (far out, zeros, tiny results) and
    products that land exactly on a bf16 rounding tie."""
    d = 1024
    g = np.zeros((6, d), np.float32)
    u = np.ones((6, d), np.float32)
    rng = np.random.default_rng(23)
    g[0] = np.linspace(-120.0, 120.0, d)                    # beyond +-80 the exponential leaves the fp32 range
    u[0] = rng.standard_normal(d) * 3.0
    g[1] = rng.standard_normal(d) * 1e-10                   # Swish(g) ~ g / 2: tiny, the products still normal numbers
    u[1] = rng.standard_normal(d) * 1e-10
    g[2] = rng.standard_normal(d) * 1e-3
    u[2] = 1e-30
    g[3] = 96.0                                             # Swish(96) = 96 exactly in fp64
    u[3] = 1.0 + rng.integers(0, 128, d) / 128.0            # 96 * u: nine significant bits, half of them exact ties
    g[4] = rng.standard_normal(d) * 8.0
    u[4] = 0.0
    g[5] = rng.standard_normal(d) * 30.0
    u[5] = rng.standard_normal(d) * 100.0
    gate, up = inputs.f32_to_bf16_bits(g), inputs.f32_to_bf16_bits(u)
    for fmt, group in (("mxfp4", 32), ("int4", 128), ("int4", 0)):
        check(B, oracle, gate, up, 16, fmt, group)


def test_swiglu_long_call_sampled(B, oracle):
    """The benchmark's shape: every warp goes round its two-stage ring many times."""
    T, d, b = 4096, 8192, 32
    gate, up = projections(1024, d, 24000, n_out=32)
    idx = (np.arange(T) + np.arange(T) // 1024) % 1024
    gate, up = gate[idx], up[(idx * 7 + 3) % 1024]
    rows = np.unique(np.concatenate([[0, T - 1], np.random.default_rng(24).choice(T, 30, replace=False)]))
    check(B, oracle, gate, up, b, "mxfp4", 32, rows=rows)
    check(B, oracle, gate, up, b, "int4", 0, rows=rows)


def test_swiglu_combinations_outside_its_coverage_are_refused(B):
    x = torch.zeros((4, 2048), dtype=torch.bfloat16, device="cuda")
    lib = B.load()
    import ctypes as C
    codes = torch.zeros((4, 1024), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    perm = torch.arange(2048, dtype=torch.int32, device="cuda")

    def call(perm_ptr, d, b, fmt, group):
        return lib.perq_swiglu_rotate_quantize(x.data_ptr(), x.data_ptr(), perm_ptr, 4, d, b, fmt, group, codes.data_ptr(),
                                               scales.data_ptr(), None)
    assert call(perm.data_ptr(), 2048, 32, 1, 32) == 10          # a permutation
    assert call(None, 2048, 256, 1, 32) == 10                    # a block longer than 128
    assert call(None, 2048, 32, 3, 0) == 10                      # FP4 with a per-token scale
    assert call(None, 2048, 32, 0, 64) == 10                     # INT4 groups other than 128
    assert call(None, 1536, 32, 1, 32) == 10                     # rows that are not whole 1024-element segments
    assert call(None, 2048, 48, 1, 32) == 3                      # plain argument errors keep their codes
    assert call(None, 2048, 32, 1, 32) == 0
