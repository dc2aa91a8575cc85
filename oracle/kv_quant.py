"""4-bit group-wise quantisation of stored K/V rows — TEST INFRASTRUCTURE (oracle side).

The paper reports that the eviction policy is compatible with 4-bit quantisation (Q3 of its question
section and the appendix on throughput with quantisation) but does not specify a quantiser.  This file
defines the one the oracle uses, step by step in fp32 so that the integer codes are the same on every
implementation that follows the same steps (parity unpinned against the paper: there is nothing printed
to pin it to; the pins in the tests are mathematical — error bound, idempotence, end points, constants).

A row of d channels is cut into groups of 32 consecutive channels.  Per group, with all arithmetic in
IEEE fp32 (round to nearest even):
    zero  = min of the group                         (an input value, exact)
    scale = bf16_round((max - zero) / 15)            ; a constant group gets scale = 1
    code  = clamp(rint((x - zero) / scale), 0, 15)   ; division, not multiplication by a reciprocal
    x_hat = zero + code * scale                      ; code * scale is exact (4 x 8 bits), one rounding
Stored per row: d/2 bytes of codes, then per group scale and zero as bf16 (zero is one of the bf16 inputs;
for fp32 inputs it is rounded to bf16 first and the codes are taken against the rounded value).
"""
import numpy as np

GROUP = 32


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even), returned as fp32.  Finite inputs only."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def quantize_rows(x):
    """x: [..., d] with d a multiple of 32.  Returns (codes uint8 [..., d], scale f32 [..., d/32], zero f32 [..., d/32])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    d = x.shape[-1]
    assert d % GROUP == 0
    g = x.reshape(x.shape[:-1] + (d // GROUP, GROUP))
    zero = bf16_round(g.min(axis=-1))
    mx = g.max(axis=-1)
    scale = bf16_round(((mx - zero) / np.float32(15.0)).astype(np.float32))
    scale = np.where(scale > 0, scale, np.float32(1.0)).astype(np.float32)
    t = ((g - zero[..., None]).astype(np.float32) / scale[..., None]).astype(np.float32)
    codes = np.clip(np.rint(t), 0, 15).astype(np.uint8)
    return codes.reshape(x.shape), scale, zero


def dequantize_rows(codes, scale, zero):
    d = codes.shape[-1]
    g = codes.reshape(codes.shape[:-1] + (d // GROUP, GROUP)).astype(np.float32)
    prod = (g * scale[..., None]).astype(np.float32)  # exact: 4-bit code times 8-bit mantissa
    return (zero[..., None] + prod).astype(np.float32).reshape(codes.shape)


def qdq(x):
    """What a stored row reads back as."""
    return dequantize_rows(*quantize_rows(x))
