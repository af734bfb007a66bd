"""Algorithmic work model of the rotate+quantize path (bytes and add/sub per token).

Pure integer bookkeeping used by the benchmark to turn a measured time into effective
bandwidth; it contains none of the method's arithmetic.
"""
from __future__ import annotations


def butterfly_add_sub_per_token(d: int, b: int) -> int:
    """A block Hadamard rotation with power-of-two block size b over d channels costs
    d*log2(b) additions/subtractions (Appendix A, remark on compute requirements)."""
    assert b >= 1 and (b & (b - 1)) == 0 and d % b == 0
    return d * (b.bit_length() - 1)


def scale_bytes_per_token(d: int, fmt: str, group: int) -> int:
    if fmt == "int4":
        return 4 * (1 if group == 0 else d // group)
    if fmt == "mxfp4":
        return d // 32
    if fmt == "fp4":
        return 4
    if fmt == "int4_asym":
        return 8           # step and zero point, fp32 each
    raise ValueError(fmt)


def algorithmic_bytes_per_token(d: int, fmt: str, group: int) -> int:
    """bf16 row in (2d) + packed 4-bit codes out (d/2) + scales out."""
    return 2 * d + d // 2 + scale_bytes_per_token(d, fmt, group)


def non_po2_factors(d: int):
    """d = 2^k' * 4t with t the largest odd factor of d (Appendix A.1); None when d is a power of two or has
    fewer than two factors of two beside t."""
    t = d
    while t % 2 == 0:
        t //= 2
    if t == 1 or d % (4 * t) != 0:
        return None
    return (d // (4 * t)).bit_length() - 1, 4 * t


def full_vector_add_sub_per_token(d: int):
    """Add/sub counts of a full-vector rotation of a non-power-of-2 dimension (Appendix A.1): the dense product
    d (d - 1), k' butterfly stages plus dense 4t-dimensional products d (k' + 4t - 1), and the appendix's
    decomposition d (k' + t + 2)."""
    kp, n = non_po2_factors(d)
    return d * (d - 1), d * (kp + n - 1), d * (kp + n // 4 + 2)
