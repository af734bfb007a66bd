"""ctypes wrapper around the CPU oracle (oracle/perq_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module;
the CUDA library and its Python binding never do.  `build()` compiles the C file with gcc
into `oracle/libperq_oracle.so` (rebuilt when the source is newer).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "perq_oracle.c")
_LIB = os.path.join(_HERE, "libperq_oracle.so")
_lib = None

FMT_INT4 = 0
FMT_MXFP4 = 1
FMT_FP4 = 3
FMT_INT4_ASYM = 4


def build(force: bool = False) -> str:
    """Compile the oracle.  -ffp-contract=off and no fast-math: plain IEEE double."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
             "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.perq_oracle_num_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError("%s failed with oracle status %d" % (what, rc))


def num_threads() -> int:
    return int(_load().perq_oracle_num_threads())


def hadamard_pm1(b: int) -> np.ndarray:
    H = np.empty((b, b), np.int8)
    _check(_load().perq_oracle_hadamard_pm1(C.c_int32(b), _p(H)), "hadamard_pm1")
    return H


def hadamard_base(n: int) -> np.ndarray:
    """Base matrix of order n = 4t of the non-power-of-2 rotation (Appendix A.1; Paley's second construction)."""
    H = np.empty((n, n), np.int8)
    _check(_load().perq_oracle_hadamard_base(C.c_int32(n), _p(H)), "hadamard_base")
    return H


def _x(x):
    x = np.ascontiguousarray(x, dtype=np.uint16)
    assert x.ndim == 2
    return x


def _perm(perm):
    return None if perm is None else np.ascontiguousarray(perm, dtype=np.int32)


def rotate(x, perm, b: int) -> np.ndarray:
    """y = (x P) R~ in fp64; x is uint16 bf16 bits [T, d]."""
    x = _x(x); perm = _perm(perm)
    T, d = x.shape
    y = np.empty((T, d), np.float64)
    _check(_load().perq_oracle_rotate(_p(x), _p(perm), C.c_int64(T), C.c_int32(d), C.c_int32(b), _p(y)),
           "rotate")
    return y


def quantize_int4(y, group: int, want_pre: bool = False):
    y = np.ascontiguousarray(y, dtype=np.float64)
    T, d = y.shape
    ng = 1 if group == 0 else d // group
    codes = np.empty((T, d // 2), np.uint8)
    scales = np.empty((T, ng), np.float32)
    pre = np.empty((T, d), np.float64) if want_pre else None
    _check(_load().perq_oracle_quantize_int4(_p(y), C.c_int64(T), C.c_int32(d), C.c_int32(group),
                                             _p(codes), _p(scales), _p(pre)), "quantize_int4")
    return (codes, scales, pre) if want_pre else (codes, scales)


def quantize_mxfp4(y, want_pre: bool = False):
    y = np.ascontiguousarray(y, dtype=np.float64)
    T, d = y.shape
    codes = np.empty((T, d // 2), np.uint8)
    e8m0 = np.empty((T, d // 32), np.uint8)
    pre = np.empty((T, d), np.float64) if want_pre else None
    _check(_load().perq_oracle_quantize_mxfp4(_p(y), C.c_int64(T), C.c_int32(d), _p(codes), _p(e8m0),
                                              _p(pre)), "quantize_mxfp4")
    return (codes, e8m0, pre) if want_pre else (codes, e8m0)


def quantize_fp4(y, want_pre: bool = False):
    """E2M1 elements with one fp32 scale per token (row maximum over 7)."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    T, d = y.shape
    codes = np.empty((T, d // 2), np.uint8)
    scales = np.empty((T, 1), np.float32)
    pre = np.empty((T, d), np.float64) if want_pre else None
    _check(_load().perq_oracle_quantize_fp4(_p(y), C.c_int64(T), C.c_int32(d), _p(codes), _p(scales), _p(pre)),
           "quantize_fp4")
    return (codes, scales, pre) if want_pre else (codes, scales)


def quantize_int4_asym(y, want_pre: bool = False):
    """Asymmetric per-token INT4: codes 0..15, (scale, integer zero point) per token."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    T, d = y.shape
    codes = np.empty((T, d // 2), np.uint8)
    sz = np.empty((T, 2), np.float32)
    pre = np.empty((T, d), np.float64) if want_pre else None
    _check(_load().perq_oracle_quantize_int4_asym(_p(y), C.c_int64(T), C.c_int32(d), _p(codes), _p(sz), _p(pre)),
           "quantize_int4_asym")
    return (codes, sz, pre) if want_pre else (codes, sz)


def rotate_quantize(x, perm, b: int, fmt: int, group: int, want_y: bool = False, want_pre: bool = False):
    """The whole path.  Returns dict(codes, scales[, y][, pre])."""
    x = _x(x); perm = _perm(perm)
    T, d = x.shape
    codes = np.empty((T, d // 2), np.uint8)
    if fmt == FMT_INT4:
        scales = np.empty((T, 1 if group == 0 else d // group), np.float32)
    elif fmt == FMT_FP4:
        scales = np.empty((T, 1), np.float32)
    elif fmt == FMT_INT4_ASYM:
        scales = np.empty((T, 2), np.float32)
    else:
        scales = np.empty((T, d // 32), np.uint8)
    y = np.empty((T, d), np.float64) if want_y else None
    pre = np.empty((T, d), np.float64) if want_pre else None
    _check(_load().perq_oracle_rotate_quantize(_p(x), _p(perm), C.c_int64(T), C.c_int32(d), C.c_int32(b),
                                               C.c_int32(fmt), C.c_int32(group), _p(codes), _p(scales),
                                               _p(y), _p(pre)), "rotate_quantize")
    out = {"codes": codes, "scales": scales}
    if want_y:
        out["y"] = y
    if want_pre:
        out["pre"] = pre
    return out


def swiglu(gate, up) -> np.ndarray:
    """h = Swish(gate) * up in fp64, rounded once to bf16 (round to nearest even); bf16 bit patterns in and out."""
    gate = _x(gate); up = _x(up)
    assert gate.shape == up.shape
    T, d = gate.shape
    h = np.empty((T, d), np.uint16)
    _check(_load().perq_oracle_swiglu(_p(gate), _p(up), C.c_int64(T), C.c_int32(d), _p(h)), "swiglu")
    return h


def block_l1_stats(x, perm, b: int):
    """Returns (chan_abs_sum[d], block_l1_mean[d/b], token_max_block_l1[T]) in fp64."""
    x = _x(x); perm = _perm(perm)
    T, d = x.shape
    cas = np.empty(d, np.float64)
    blm = np.empty(d // b, np.float64)
    tmx = np.empty(T, np.float64)
    _check(_load().perq_oracle_block_l1_stats(_p(x), _p(perm), C.c_int64(T), C.c_int32(d), C.c_int32(b),
                                              _p(cas), _p(blm), _p(tmx)), "block_l1_stats")
    return cas, blm, tmx


def token_diagnostics(x, perm, b: int) -> np.ndarray:
    """[T, 5] fp64: ||x||_inf, ||x||_1, max block l1 (under perm), ||y||_inf, ||y - Q(y)||_2 per token."""
    x = _x(x); perm = _perm(perm)
    T, d = x.shape
    out = np.empty((T, 5), np.float64)
    _check(_load().perq_oracle_token_diagnostics(_p(x), _p(perm), C.c_int64(T), C.c_int32(d), C.c_int32(b), _p(out)),
           "token_diagnostics")
    return out


def massdiff_perm(chan_abs_sum, b: int) -> np.ndarray:
    a = np.ascontiguousarray(chan_abs_sum, dtype=np.float64)
    d = a.shape[0]
    perm = np.empty(d, np.int32)
    _check(_load().perq_oracle_massdiff_perm(_p(a), C.c_int32(d), C.c_int32(b), _p(perm)), "massdiff_perm")
    return perm


def chan_abs_max(x) -> np.ndarray:
    """max_t |x[t, c]| per channel, fp64."""
    x = _x(x)
    T, d = x.shape
    out = np.empty(d, np.float64)
    _check(_load().perq_oracle_chan_abs_max(_p(x), C.c_int64(T), C.c_int32(d), _p(out)), "chan_abs_max")
    return out


def absmax_perm(stat) -> np.ndarray:
    a = np.ascontiguousarray(stat, dtype=np.float64)
    perm = np.empty(a.shape[0], np.int32)
    _check(_load().perq_oracle_absmax_perm(_p(a), C.c_int32(a.shape[0]), _p(perm)), "absmax_perm")
    return perm


def zigzag_perm(stat, b: int) -> np.ndarray:
    a = np.ascontiguousarray(stat, dtype=np.float64)
    perm = np.empty(a.shape[0], np.int32)
    _check(_load().perq_oracle_zigzag_perm(_p(a), C.c_int32(a.shape[0]), C.c_int32(b), _p(perm)), "zigzag_perm")
    return perm
