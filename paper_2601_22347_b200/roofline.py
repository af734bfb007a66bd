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
