"""Quantizer primitives of Sec. 3.1 (Eq. 1, Eq. 2) and the group parameters of Eq. 6.

Test infrastructure only; see the package docstring.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
MIN_SCALE = F32(1e-8)


# --------------------------------------------------------------------------- Eq. 1
def linear_quantize(x, s, z, b):
    """Eq. 1, left half, in fp64: clamp(round(x / s) + z, 0, 2^b - 1).

    Rounding is half-to-even (the paper does not name the tie rule).
    """
    q = np.rint(np.asarray(x, dtype=np.float64) / np.asarray(s, dtype=np.float64)) + z
    return np.clip(q, 0, 2 ** b - 1).astype(np.int64)


def linear_dequantize(q, s, z):
    """Eq. 1, right half: s * (x_q - z)."""
    return np.asarray(s, dtype=np.float64) * (np.asarray(q, dtype=np.float64) - z)


# --------------------------------------------------------------------------- Eq. 2
def log_quantize(x, s, b):
    """Eq. 2, left half, in fp64: clamp(round(-log2(x / s)), 0, 2^b - 1).

    x = 0 gives -log2(0) = +inf, which clamps to the last code; there is no
    separate "zero" level (the paper defines none).
    """
    x = np.asarray(x, dtype=np.float64)
    with np.errstate(divide="ignore"):
        t = -np.log2(x / np.asarray(s, dtype=np.float64))
    return np.clip(np.rint(t), 0, 2 ** b - 1).astype(np.int64)


def log_dequantize(q, s):
    """Eq. 2, right half: s * 2^(-x_q), exact (a shift of the exponent)."""
    return np.ldexp(np.asarray(s, dtype=np.float64), -np.asarray(q, dtype=np.int64))


# --------------------------------------------------------------------------- Eq. 6
def group_params(lo, hi, b):
    """Eq. 6 for one group: scale from the group's range, zero-point from its minimum.

    Readings (the paper leaves these open):
      * the denominator is 2^b as printed, not 2^b - 1;
      * Eq. 1 adds an integer z after rounding while Eq. 6 gives z_k = min x, a
        real number: the integer zero-point is Z = round(-min x / s), so that
        x = min x maps to code 0;
      * a constant group (hi == lo) gets the floor scale 1e-8;
      * arithmetic is IEEE fp32, in this order: s = (hi - lo) * 2^-b,
        inv_s = 1 / s, Z = rint(clamp(-lo * inv_s, -2^30, 2^30)); the clamp only
        matters for a constant group far from zero, where it keeps Z an int32.
    Returns (s, inv_s, Z) as (float32, float32, int).
    """
    lo = F32(lo)
    hi = F32(hi)
    s = F32(F32(hi - lo) * F32(2.0 ** -b))
    if not s > MIN_SCALE:
        s = MIN_SCALE
    inv_s = F32(F32(1.0) / s)
    Z = int(np.rint(np.clip(F32(-lo * inv_s), F32(-2.0 ** 30), F32(2.0 ** 30))))
    return s, inv_s, Z


def group_params_array(lo, hi, b):
    """`group_params` element-wise over arrays; returns float32, float32, int32 arrays."""
    lo = np.asarray(lo, dtype=F32)
    hi = np.asarray(hi, dtype=F32)
    s = ((hi - lo).astype(F32) * F32(2.0 ** -b)).astype(F32)
    s = np.where(s > MIN_SCALE, s, MIN_SCALE).astype(F32)
    inv_s = (F32(1.0) / s).astype(F32)
    Z = np.rint(np.clip((-lo * inv_s).astype(F32), F32(-2.0 ** 30), F32(2.0 ** 30))).astype(np.int32)
    return s, inv_s, Z


def quantize_canonical_f32(x, inv_s, Z, b):
    """Eq. 1 in the fp32 operation order that fixes the integer code.

    Floating point decides an integer here, so the decision is taken in one
    stated precision: t = x * inv_s (one rounded fp32 multiply),
    u = rint(t) + float(Z), q = min(max(u, 0), 2^b - 1) with NaN -> 0.
    `inv_s` and `Z` broadcast against `x`.
    """
    L = F32(2 ** b - 1)
    t = (np.asarray(x, dtype=F32) * np.asarray(inv_s, dtype=F32)).astype(F32)
    u = (np.rint(t) + np.asarray(Z).astype(F32)).astype(F32)
    q = np.fmin(np.fmax(u, F32(0.0)), L)
    return q.astype(np.int32)
