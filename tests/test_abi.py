"""Host-side checks that need no GPU: the library loads, exports what the header declares,
validates arguments before touching CUDA, and its host-only entry points work."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_22347_b200 import build, binding
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "perq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(perq_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for required in ("perq_rotate_quantize", "perq_block_l1_stats", "perq_out_sizes", "perq_validate_perm",
                     "perq_massdiff_perm", "perq_status_string", "perq_version", "perq_rotate_quantize_host"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), "libperq.so does not export %s" % name


def test_version_and_status_strings(lib):
    from paper_2601_22347_b200 import binding
    assert binding.perq_version() >= 100
    seen = set()
    for code in range(0, 10):
        s = binding.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert binding.status_string(1234) == "unknown status"


def test_out_sizes(lib):
    from paper_2601_22347_b200 import binding as B
    assert B.perq_out_sizes(16384, 4096, B.PERQ_FMT_INT4, 0) == (16384 * 2048, 16384 * 4)
    assert B.perq_out_sizes(4096, 2048, B.PERQ_FMT_INT4, 128) == (4096 * 1024, 4096 * 16 * 4)
    assert B.perq_out_sizes(4096, 8192, B.PERQ_FMT_MXFP4, 32) == (4096 * 4096, 4096 * 256)
    assert B.perq_out_sizes(3, 64, B.PERQ_FMT_F32_DEBUG, 0) == (3 * 64 * 4, 0)
    assert B.perq_out_sizes(0, 64, B.PERQ_FMT_INT4, 0) == (0, 0)
    assert B.perq_out_sizes(16384, 4096, B.PERQ_FMT_FP4, 0) == (16384 * 2048, 16384 * 4)
    assert B.perq_out_sizes(16384, 4096, B.PERQ_FMT_INT4_ASYM, 0) == (16384 * 2048, 16384 * 8)


def test_argument_validation_happens_before_any_launch(lib):
    """Every rejected call returns before the library touches the CUDA runtime, so these
    run on a machine without a GPU.  Pointers are fake but 16-byte aligned."""
    from paper_2601_22347_b200 import binding as B
    p = C.c_void_p(0x1000)
    call = lambda x, perm, T, d, b, fmt, g, oc, os_: lib.perq_rotate_quantize(x, perm, T, d, b, fmt, g, oc, os_, None)
    assert call(p, None, -1, 4096, 32, 0, 0, p, p) == 2          # T < 0
    assert call(p, None, 4, 4100, 32, 0, 0, p, p) == 2           # d % 32
    assert call(p, None, 4, 65536, 32, 0, 0, p, p) == 2          # d too large
    assert call(p, None, 4, 4096, 8, 0, 0, p, p) == 3            # b not allowed
    assert call(p, None, 4, 4096, 24, 0, 0, p, p) == 3           # b not a power of two
    assert call(p, None, 4, 4096, 8192, 0, 0, p, p) == 3         # b larger than d
    assert call(p, None, 4, 12288, 8192, 0, 0, p, p) == 3        # b does not divide d
    assert call(p, None, 4, 5120, 5120, 0, 0, p, p) == 3         # 2^8 * 20: no base matrix of order 20
    assert call(p, None, 4, 14336, 28, 0, 0, p, p) == 3          # a base-matrix block only as the whole row
    assert call(p, None, 4, 14336, 7168, 0, 0, p, p) == 3
    assert call(p, None, 0, 14336, 14336, 0, 0, p, p) == 0       # 2^9 * 28 as the whole row: accepted (T == 0)
    assert call(p, None, 0, 9728, 9728, 1, 32, p, p) == 0        # 2^7 * 76
    assert call(p, None, 0, 3072, 3072, 3, 0, p, p) == 0         # 2^8 * 12
    assert call(p, None, 4, 4096, 32, 0, 12, p, p) == 4          # group % 8
    assert call(p, None, 4, 4096, 32, 0, 24, p, p) == 4          # group does not divide d
    assert call(p, None, 4, 4096, 32, 1, 64, p, p) == 4          # MX group must be 32
    assert call(p, None, 4, 4096, 32, 7, 0, p, p) == 5           # format
    assert call(p, None, 4, 4096, 32, 3, 128, p, p) == 4         # FP4 has one scale per token
    assert call(None, None, 4, 4096, 32, 0, 0, p, p) == 1        # null x
    assert call(p, None, 4, 4096, 32, 0, 0, p, None) == 1        # null scales
    assert call(C.c_void_p(0x1004), None, 4, 4096, 32, 0, 0, p, p) == 6   # misaligned
    assert call(p, C.c_void_p(0x1008), 4, 4096, 32, 0, 0, p, p) == 6      # misaligned perm
    assert call(p, None, 0, 4096, 32, 0, 0, p, p) == 0           # T == 0: nothing to do
    n = C.c_size_t(0)
    assert lib.perq_block_l1_stats_workspace_bytes(4096, 8192, 24, C.byref(n)) == 3
    assert lib.perq_block_l1_stats(p, None, 16, 4096, 32, p, None, None, None, 0, None) == 9   # no workspace
    assert lib.perq_rotate_quantize_host(p, None, 4, 4096, 32, 0, 0, p, p, None, 0, None) == 9
    assert lib.perq_validate_perm(None, 16, p, None) == 1


def test_token_diagnostics_validation(lib):
    f = lib.perq_token_diagnostics
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    fake = C.c_void_p(0x1000)
    assert f(None, None, 4, 2048, 32, fake, None) == 1
    assert f(fake, None, 4, 2048, 32, None, None) == 1
    assert f(fake, None, 4, 2050, 32, fake, None) == 2
    assert f(fake, None, 4, 2048, 8, fake, None) == 3          # blocks of at least 16
    assert f(fake, None, 4, 3072, 3072, fake, None) == 3       # power-of-two blocks only
    assert f(C.c_void_p(0x1008), None, 4, 2048, 32, fake, None) == 6
    assert f(fake, None, 0, 2048, 32, fake, None) == 0          # T = 0: nothing to do


def test_device_massdiff_validation(lib):
    f = lib.perq_massdiff_perm_device
    f.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    fake = C.c_void_p(0x1000)
    assert f(None, 256, 16, fake, fake, 1024, None) == 1
    assert f(fake, 0, 16, fake, fake, 1024, None) == 2
    assert f(fake, 256, 24, fake, fake, 1024, None) == 3
    assert f(fake, 8192, 1, fake, fake, 32768, None) == 3       # more than 4096 blocks
    assert f(fake, 256, 16, fake, fake, 1023, None) == 9         # workspace too small
    assert f(fake, 256, 16, fake, None, 0, None) == 9


def test_host_massdiff_matches_oracle(lib, oracle):
    from paper_2601_22347_b200 import binding as B
    rng = np.random.default_rng(41)
    for d, b in ((256, 16), (512, 32), (8192, 32), (2048, 2048), (64, 1)):
        a = (rng.exponential(size=d) * np.where(rng.random(d) < 0.05, 40.0, 1.0)).astype(np.float32)
        a[rng.integers(0, d, 8)] = a[0]                     # force some equal masses
        mine = B.perq_massdiff_perm(a, b)
        ref = oracle.massdiff_perm(a.astype(np.float64), b)
        assert sorted(mine.tolist()) == list(range(d))
        assert np.array_equal(mine, ref)


def test_host_massdiff_hand_example(lib):
    from paper_2601_22347_b200 import binding as B
    assert B.perq_massdiff_perm(np.array([9, 8, 7, 6, 5, 4, 3, 2], np.float32), 4).tolist() == [0, 3, 4, 7, 1, 2, 5, 6]
    with pytest.raises(B.PerqError):
        B.perq_massdiff_perm(np.ones(10, np.float32), 4)


def test_comparison_permutations_match_the_oracle(oracle):
    from paper_2601_22347_b200 import binding as B
    rng = np.random.default_rng(77)
    for d, b in ((256, 16), (2048, 32), (96, 8), (64, 64)):
        s = (rng.exponential(size=d) * np.where(rng.random(d) < 0.05, 40.0, 1.0)).astype(np.float32)
        s[rng.integers(0, d, 8)] = s[0]
        assert np.array_equal(B.perq_absmax_perm(s), oracle.absmax_perm(s.astype(np.float64)))
        assert np.array_equal(B.perq_zigzag_perm(s, b), oracle.zigzag_perm(s.astype(np.float64), b))
    with pytest.raises(RuntimeError):
        B.perq_zigzag_perm(np.ones(10, np.float32), 4)
