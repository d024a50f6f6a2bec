"""Comparison of a bf16 GEMM output with the fp64 reference, in units of bf16 steps.  Test infrastructure only.

The layer's output is bf16(acc * ts_x * ts_w) (Eq. 8 with fp32 accumulation).  Rounding to bf16 alone
moves a value by up to 2^-9 of its magnitude, so a comparison in relative error mixes the output format's
rounding with what the kernel itself contributes (the order of its fp32 additions).  Counting in bf16 steps
separates the two: if the kernel's fp32 value is within `slack` of the reference, its rounding can differ
from bf16(reference) only where the reference lies within `slack` of a rounding boundary (the midpoint
of two neighbouring bf16 values), and then by one step.
"""
import numpy as np


def _ordinal(bits):
    """bf16 bit patterns -> integers ordered like the values (+0 and -0 both 0)."""
    b = bits.astype(np.int64)
    mag = b & 0x7FFF
    return np.where(b & 0x8000, -mag, mag)


def _from_ordinal(o):
    """Inverse of _ordinal for finite values -> float64."""
    mag = np.abs(o).astype(np.uint32) << 16
    v = mag.view(np.float32).astype(np.float64)
    return np.where(o < 0, -v, v)


def bf16_bits_rne(ref):
    """float64 -> bf16 bit patterns, one rounding to nearest even (finite values in bf16's normal range)."""
    ref = np.asarray(ref, dtype=np.float64)
    # A first guess through fp32 (two roundings), then the nearest of the guess and its two neighbours by
    # distance in fp64, ties to the even mantissa: that undoes the rare double-rounding cases.
    f = ref.astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    o = _ordinal(r)
    cand = np.stack([o - 1, o, o + 1])
    vals = _from_ordinal(cand)
    dist = np.abs(vals - ref[None])
    best = dist.min(axis=0)
    # among equidistant candidates take the even mantissa (ordinal parity = mantissa LSB parity)
    pick = np.full(ref.shape, 1, dtype=np.int64)
    for i in (0, 2):
        better = (dist[i] < dist[1]) | ((dist[i] == dist[1]) & (cand[i] % 2 == 0) & (cand[1] % 2 != 0))
        better &= dist[i] == best
        pick = np.where(better, i, pick)
    o = np.take_along_axis(cand, pick[None], axis=0)[0]
    mag = np.abs(o).astype(np.uint16)
    neg = (o < 0) | ((o == 0) & np.signbit(ref))
    return np.where(neg, mag | 0x8000, mag).astype(np.uint16)


def bf16_step_report(y_bits, ref, slack):
    """y_bits: uint16 bf16 patterns of the kernel's output; ref: float64 reference; slack: absolute
    accumulation allowance.  Returns a dict:
       exact      fraction of outputs equal to bf16(ref)
       max_steps  largest distance from bf16(ref) in bf16 steps
       off_clear  number of outputs that differ from bf16(ref) although ref is further than `slack`
                  from every rounding boundary (must be 0)
       near       fraction of outputs whose reference is within `slack` of a boundary
    """
    y_bits = np.asarray(y_bits, dtype=np.uint16)
    ref = np.asarray(ref, dtype=np.float64)
    want = bf16_bits_rne(ref)
    oy, ow = _ordinal(y_bits), _ordinal(want)
    steps = np.abs(oy - ow)
    lo_mid = (_from_ordinal(ow) + _from_ordinal(ow - 1)) / 2
    hi_mid = (_from_ordinal(ow) + _from_ordinal(ow + 1)) / 2
    to_boundary = np.minimum(np.abs(ref - lo_mid), np.abs(ref - hi_mid))
    near = to_boundary <= slack
    return {"exact": float((steps == 0).mean()), "max_steps": int(steps.max()),
            "off_clear": int(((steps != 0) & ~near).sum()), "near": float(near.mean()),
            "steps": steps, "near_mask": near}
