"""Thin ctypes binding of libperq.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/perq.h for what
each computes).  torch is used for device memory and streams; all arithmetic of the path
happens inside the CUDA library.  There is no CPU fallback: if the library cannot be
loaded, importing this module's functions raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

PERQ_FMT_INT4 = 0
PERQ_FMT_MXFP4 = 1
PERQ_FMT_F32_DEBUG = 2
PERQ_FMT_FP4 = 3
PERQ_FMT_INT4_ASYM = 4
FMT_BY_NAME = {"int4": PERQ_FMT_INT4, "mxfp4": PERQ_FMT_MXFP4, "f32": PERQ_FMT_F32_DEBUG, "fp4": PERQ_FMT_FP4,
               "int4_asym": PERQ_FMT_INT4_ASYM}

PERQ_OK = 0

_lib = None


class PerqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


def load() -> C.CDLL:
    """Load libperq.so from the package directory (never builds implicitly)."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError("%s not found: run `python -m paper_2601_22347_b200.build` "
                               "(or __graft_entry__.build()) first" % path)
        lib = C.CDLL(path)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        lib.perq_rotate_quantize.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, vp, vp]
        lib.perq_swiglu_rotate_quantize.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, vp]
        lib.perq_swiglu_rotate_quantize.restype = C.c_int
        lib.perq_rotate_quantize_host.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        lib.perq_host_workspace_bytes.argtypes = [i64, i32, i32, i32, C.POINTER(sz)]
        lib.perq_out_sizes.argtypes = [i64, i32, i32, i32, C.POINTER(sz), C.POINTER(sz)]
        lib.perq_block_l1_stats.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp, sz, vp]
        lib.perq_block_l1_stats_static.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp]
        lib.perq_block_l1_stats_workspace_bytes.argtypes = [i64, i32, i32, C.POINTER(sz)]
        lib.perq_token_diagnostics.argtypes = [vp, vp, i64, i32, i32, vp, vp]
        lib.perq_validate_perm.argtypes = [vp, i32, vp, vp]
        lib.perq_massdiff_perm.argtypes = [vp, i32, i32, vp]
        lib.perq_massdiff_perm_device.argtypes = [vp, i32, i32, vp, vp, sz, vp]
        lib.perq_chan_abs_max.argtypes = [vp, i64, i32, vp, vp]
        lib.perq_absmax_perm.argtypes = [vp, i32, vp]
        lib.perq_zigzag_perm.argtypes = [vp, i32, i32, vp]
        for name in ("perq_chan_abs_max", "perq_absmax_perm", "perq_zigzag_perm"):
            getattr(lib, name).restype = C.c_int
        lib.perq_device_error.argtypes = [C.POINTER(C.c_uint32)]
        lib.perq_device_error.restype = C.c_int
        lib.perq_device_error_clear.argtypes = []
        lib.perq_device_error_clear.restype = C.c_int
        lib.perq_status_string.argtypes = [C.c_int]
        lib.perq_status_string.restype = C.c_char_p
        lib.perq_version.restype = C.c_int
        for name in ("perq_rotate_quantize", "perq_rotate_quantize_host", "perq_host_workspace_bytes",
                     "perq_out_sizes", "perq_block_l1_stats", "perq_block_l1_stats_static",
                     "perq_block_l1_stats_workspace_bytes",
                     "perq_token_diagnostics", "perq_validate_perm", "perq_massdiff_perm", "perq_massdiff_perm_device"):
            getattr(lib, name).restype = C.c_int
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().perq_status_string(int(status)).decode()


def perq_version() -> int:
    return int(load().perq_version())


def _check(rc: int, where: str):
    if rc != PERQ_OK:
        raise PerqError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def perq_out_sizes(T: int, d: int, fmt: int, group: int):
    cb, sb = C.c_size_t(0), C.c_size_t(0)
    _check(load().perq_out_sizes(T, d, fmt, group, C.byref(cb), C.byref(sb)), "perq_out_sizes")
    return int(cb.value), int(sb.value)


def alloc_outputs(T: int, d: int, fmt: int, group: int, device):
    """Device buffers of the right shape for one call (torch owns the memory)."""
    if fmt == PERQ_FMT_F32_DEBUG:
        return torch.empty((T, d), dtype=torch.float32, device=device), None
    codes = torch.empty((T, d // 2), dtype=torch.uint8, device=device)
    if fmt == PERQ_FMT_FP4:
        scales = torch.empty((T, 1), dtype=torch.float32, device=device)
    elif fmt == PERQ_FMT_INT4_ASYM:
        scales = torch.empty((T, 2), dtype=torch.float32, device=device)
    elif fmt == PERQ_FMT_INT4:
        scales = torch.empty((T, 1 if group == 0 else d // group), dtype=torch.float32, device=device)
    else:
        scales = torch.empty((T, d // 32), dtype=torch.uint8, device=device)
    return codes, scales


def perq_rotate_quantize(x: torch.Tensor, perm: Optional[torch.Tensor], b: int, fmt: int, group: int = 0,
                         out_codes: Optional[torch.Tensor] = None, out_scales: Optional[torch.Tensor] = None,
                         stream=None):
    """x: bf16 CUDA tensor [T, d] (contiguous); perm: int32 CUDA tensor [d] or None."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    assert perm is None or (perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous())
    T, d = x.shape
    if out_codes is None:
        out_codes, out_scales = alloc_outputs(T, d, fmt, group, x.device)
    rc = load().perq_rotate_quantize(_ptr(x), _ptr(perm), T, d, b, fmt, group, _ptr(out_codes), _ptr(out_scales),
                                     _stream(stream))
    _check(rc, "perq_rotate_quantize")
    return out_codes, out_scales


def perq_swiglu_rotate_quantize(gate: torch.Tensor, up: torch.Tensor, perm: Optional[torch.Tensor], b: int, fmt: int,
                                group: int = 0, out_codes: Optional[torch.Tensor] = None,
                                out_scales: Optional[torch.Tensor] = None, stream=None):
    """gate, up: bf16 CUDA tensors [T, d] (contiguous); perm must be None."""
    for t in (gate, up):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 2 and t.is_contiguous()
    assert gate.shape == up.shape
    T, d = gate.shape
    if out_codes is None:
        out_codes, out_scales = alloc_outputs(T, d, fmt, group, gate.device)
    rc = load().perq_swiglu_rotate_quantize(_ptr(gate), _ptr(up), _ptr(perm), T, d, b, fmt, group, _ptr(out_codes),
                                            _ptr(out_scales), _stream(stream))
    _check(rc, "perq_swiglu_rotate_quantize")
    return out_codes, out_scales


def perq_host_workspace_bytes(T: int, d: int, fmt: int, group: int) -> int:
    n = C.c_size_t(0)
    _check(load().perq_host_workspace_bytes(T, d, fmt, group, C.byref(n)), "perq_host_workspace_bytes")
    return int(n.value)


def perq_rotate_quantize_host(x_host: torch.Tensor, perm: Optional[torch.Tensor], b: int, fmt: int, group: int,
                              out_codes_host: torch.Tensor, out_scales_host: Optional[torch.Tensor],
                              workspace: torch.Tensor, stream=None):
    """x_host / outputs: CPU tensors (pinned for asynchronous copies); workspace: CUDA uint8 tensor."""
    assert not x_host.is_cuda and x_host.dtype == torch.bfloat16 and x_host.is_contiguous()
    T, d = x_host.shape
    rc = load().perq_rotate_quantize_host(_ptr(x_host), _ptr(perm), T, d, b, fmt, group, _ptr(out_codes_host),
                                          _ptr(out_scales_host), _ptr(workspace), workspace.numel(),
                                          _stream(stream))
    _check(rc, "perq_rotate_quantize_host")
    return out_codes_host, out_scales_host


def perq_block_l1_stats_workspace_bytes(T: int, d: int, b: int) -> int:
    n = C.c_size_t(0)
    _check(load().perq_block_l1_stats_workspace_bytes(T, d, b, C.byref(n)), "perq_block_l1_stats_workspace_bytes")
    return int(n.value)


def perq_block_l1_stats(x: torch.Tensor, perm: Optional[torch.Tensor], b: int, want=("chan", "block", "token"),
                        workspace: Optional[torch.Tensor] = None, stream=None):
    """Returns (chan_abs_sum[d], block_l1_mean[d/b], token_max_block_l1[T]); entries not in `want` are None."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    T, d = x.shape
    if workspace is None:
        workspace = torch.empty(max(16, perq_block_l1_stats_workspace_bytes(T, d, b)), dtype=torch.uint8,
                                device=x.device)
    chan = torch.empty(d, dtype=torch.float32, device=x.device) if "chan" in want else None
    block = torch.empty(d // b, dtype=torch.float32, device=x.device) if "block" in want else None
    token = torch.empty(T, dtype=torch.float32, device=x.device) if "token" in want else None
    rc = load().perq_block_l1_stats(_ptr(x), _ptr(perm), T, d, b, _ptr(chan), _ptr(block), _ptr(token),
                                    _ptr(workspace), workspace.numel(), _stream(stream))
    _check(rc, "perq_block_l1_stats")
    return chan, block, token


def perq_block_l1_stats_static(x: torch.Tensor, perm: Optional[torch.Tensor], b: int, chan: Optional[torch.Tensor],
                               block: Optional[torch.Tensor], token: Optional[torch.Tensor], stream=None):
    """perq_block_l1_stats with the library's built-in scratch array instead of a workspace.

    The caller passes the output tensors (any may be None); nothing is allocated here or in
    the library.  Shapes whose partial sums do not fit the built-in array raise PerqError
    (status 9).  Calls that may overlap on the GPU must not share a device: they would race
    on the one scratch array."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    T, d = x.shape
    rc = load().perq_block_l1_stats_static(_ptr(x), _ptr(perm), T, d, b, _ptr(chan), _ptr(block), _ptr(token),
                                           _stream(stream))
    _check(rc, "perq_block_l1_stats_static")
    return chan, block, token


def perq_token_diagnostics(x: torch.Tensor, perm: Optional[torch.Tensor], b: int, out: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    """[T, 5] fp32: ||x||_inf, ||x||_1, largest block l1 under perm, ||y||_inf, ||y - Q(y)||_2 per token."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    assert perm is None or (perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous())
    T, d = x.shape
    if out is None:
        out = torch.empty((T, 5), dtype=torch.float32, device=x.device)
    _check(load().perq_token_diagnostics(_ptr(x), _ptr(perm), T, d, b, _ptr(out), _stream(stream)),
           "perq_token_diagnostics")
    return out


def perq_validate_perm(perm: torch.Tensor, stream=None) -> torch.Tensor:
    """Returns a 1-element int32 CUDA tensor: 0 valid, bit0 out of range, bit1 duplicate."""
    assert perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous()
    status = torch.empty(1, dtype=torch.int32, device=perm.device)
    _check(load().perq_validate_perm(_ptr(perm), perm.numel(), _ptr(status), _stream(stream)), "perq_validate_perm")
    return status


def perq_device_error() -> int:
    """Device-side error word of the current device (0 = none); synchronises."""
    v = C.c_uint32(0)
    _check(load().perq_device_error(C.byref(v)), "perq_device_error")
    return int(v.value)


def perq_device_error_clear() -> None:
    """Zeroes the device-side error word of the current device; synchronises."""
    _check(load().perq_device_error_clear(), "perq_device_error_clear")


def perq_massdiff_perm_device(chan_abs_sum: torch.Tensor, b: int, perm: Optional[torch.Tensor] = None,
                              workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """chan_abs_sum: fp32 CUDA tensor [d]; returns the int32 CUDA permutation [d] (nothing is synchronised)."""
    assert chan_abs_sum.is_cuda and chan_abs_sum.dtype == torch.float32 and chan_abs_sum.is_contiguous()
    d = chan_abs_sum.numel()
    if perm is None:
        perm = torch.empty(d, dtype=torch.int32, device=chan_abs_sum.device)
    if workspace is None:
        workspace = torch.empty(d * 4, dtype=torch.uint8, device=chan_abs_sum.device)
    _check(load().perq_massdiff_perm_device(_ptr(chan_abs_sum), d, b, _ptr(perm), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)),
           "perq_massdiff_perm_device")
    return perm


def perq_chan_abs_max(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """x: bf16 CUDA tensor [T, d]; returns fp32 CUDA tensor [d] (nothing is synchronised)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    T, d = x.shape
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=x.device)
    _check(load().perq_chan_abs_max(_ptr(x), T, d, _ptr(out), _stream(stream)), "perq_chan_abs_max")
    return out


def perq_absmax_perm(chan_abs_max_host: np.ndarray) -> np.ndarray:
    """Host only.  float32 [d] numpy array in, int32 [d] out."""
    a = np.ascontiguousarray(chan_abs_max_host, dtype=np.float32)
    perm = np.empty(a.shape[0], np.int32)
    _check(load().perq_absmax_perm(a.ctypes.data_as(C.c_void_p), a.shape[0], perm.ctypes.data_as(C.c_void_p)), "perq_absmax_perm")
    return perm


def perq_zigzag_perm(chan_abs_max_host: np.ndarray, b: int) -> np.ndarray:
    """Host only.  float32 [d] numpy array in, int32 [d] out."""
    a = np.ascontiguousarray(chan_abs_max_host, dtype=np.float32)
    perm = np.empty(a.shape[0], np.int32)
    _check(load().perq_zigzag_perm(a.ctypes.data_as(C.c_void_p), a.shape[0], b, perm.ctypes.data_as(C.c_void_p)), "perq_zigzag_perm")
    return perm


def perq_massdiff_perm(chan_abs_sum_host: np.ndarray, b: int) -> np.ndarray:
    """Host only.  chan_abs_sum_host: float32 [d] numpy array; returns int32 [d]."""
    a = np.ascontiguousarray(chan_abs_sum_host, dtype=np.float32)
    perm = np.empty(a.shape[0], np.int32)
    rc = load().perq_massdiff_perm(a.ctypes.data_as(C.c_void_p), a.shape[0], b, perm.ctypes.data_as(C.c_void_p))
    _check(rc, "perq_massdiff_perm")
    return perm
