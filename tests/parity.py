"""Comparison of the CUDA path's outputs with the oracle's, under the stated tolerances.

Tolerances (written here once, used by every parity test):
  * rotated fp32 values: |y_gpu - y_oracle| <= 1e-5 * max|y_oracle| over the element's
    Hadamard block;
  * INT4 scales: within 1 fp32 ulp of the oracle's; MXFP4 scale bytes: bit-exact;
  * codes: bit-exact, except that a code may differ by one step where the oracle's
    pre-rounding value lies within 1e-6 (in code units) of a rounding tie.  Such elements
    are counted and returned, everything else is a failure.
"""
from __future__ import annotations

import numpy as np

E2M1_MIDPOINTS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
TIE_WINDOW = 1e-6


def unpack_nibbles(codes: np.ndarray) -> np.ndarray:
    lo = codes & 0xF
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def int4_values(nib: np.ndarray) -> np.ndarray:
    n = nib.astype(np.int64)
    return np.where(n >= 8, n - 16, n)


def ulp_distance_f32(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Distance in units of the last place between non-negative float32 arrays."""
    ai = np.ascontiguousarray(a, np.float32).view(np.int32).astype(np.int64)
    bi = np.ascontiguousarray(b, np.float32).view(np.int32).astype(np.int64)
    return np.abs(ai - bi)


def compare_quantized(fmt: str, gpu_codes, gpu_scales, ora: dict) -> dict:
    """`ora` is the oracle's rotate_quantize(..., want_pre=True) result.  Raises AssertionError
    on any out-of-tolerance difference; returns counters."""
    gpu_codes = np.asarray(gpu_codes)
    gpu_scales = np.asarray(gpu_scales).reshape(ora["scales"].shape)
    assert gpu_codes.shape == ora["codes"].shape
    report = {"elements": int(gpu_codes.size) * 2, "code_mismatch_exempt": 0, "scale_ulp_max": 0}
    if fmt == "int4_asym":
        ulp = ulp_distance_f32(np.abs(gpu_scales[:, 0]), np.abs(ora["scales"][:, 0]))
        report["scale_ulp_max"] = int(ulp.max()) if ulp.size else 0
        assert report["scale_ulp_max"] <= 1, "asymmetric INT4 step differs by %d ulp" % report["scale_ulp_max"]
        assert np.array_equal(gpu_scales[:, 1], ora["scales"][:, 1]), "zero points differ"
    elif fmt in ("int4", "fp4"):
        ulp = ulp_distance_f32(gpu_scales, ora["scales"])
        report["scale_ulp_max"] = int(ulp.max()) if ulp.size else 0
        assert report["scale_ulp_max"] <= 1, "%s scale differs by %d ulp" % (fmt, report["scale_ulp_max"])
    else:
        bad = np.flatnonzero(gpu_scales.ravel() != ora["scales"].ravel())
        assert bad.size == 0, "E8M0 mismatch at %s: gpu %s oracle %s" % (
            bad[:5], gpu_scales.ravel()[bad[:5]], ora["scales"].ravel()[bad[:5]])
    diff = gpu_codes != ora["codes"]
    if diff.any():
        g = unpack_nibbles(gpu_codes)
        o = unpack_nibbles(ora["codes"])
        idx = np.nonzero(g != o)
        pre = ora["pre"][idx]
        if fmt == "int4_asym":
            step = np.abs(g[idx].astype(np.int64) - o[idx].astype(np.int64))
            near = np.abs(np.abs(pre - np.floor(pre)) - 0.5) < TIE_WINDOW
        elif fmt == "int4":
            step = np.abs(int4_values(g[idx]) - int4_values(o[idx]))
            near = np.abs(np.abs(pre - np.floor(pre)) - 0.5) < TIE_WINDOW
        else:
            same_sign = (g[idx] & 8) == (o[idx] & 8)
            step = np.where(same_sign, np.abs((g[idx] & 7).astype(np.int64) - (o[idx] & 7).astype(np.int64)), 99)
            near = np.abs(np.abs(pre)[:, None] - E2M1_MIDPOINTS[None, :]).min(axis=1) < TIE_WINDOW
        bad = ~((step == 1) & near)
        if bad.any():
            k = np.flatnonzero(bad)[:8]
            raise AssertionError(
                "%d code mismatches outside the tie window; first at (row, col) %s: gpu %s oracle %s pre %s"
                % (int(bad.sum()), list(zip(idx[0][k], idx[1][k])), g[idx][k], o[idx][k], pre[k]))
        report["code_mismatch_exempt"] = int(near.sum())
    return report


def compare_rotated(y_gpu: np.ndarray, y_oracle: np.ndarray, b: int) -> dict:
    T, d = y_oracle.shape
    ref = np.abs(y_oracle).reshape(T, d // b, b).max(axis=2, keepdims=True)
    err = np.abs(y_gpu.astype(np.float64) - y_oracle).reshape(T, d // b, b)
    rel = np.where(ref > 0, err / np.where(ref > 0, ref, 1), err)
    worst = float(rel.max()) if rel.size else 0.0
    assert worst <= 1e-5, "rotated values off by %.3g relative to the block max" % worst
    return {"max_rel_to_block_max": worst, "rms_rel": float(np.sqrt((rel ** 2).mean())) if rel.size else 0.0}
