"""Oracle for the sketch matrix S ("Gaussian v1"), numpy only.  TEST INFRASTRUCTURE.

The paper names its random-projection compressor (Section 5, experimental
setup; Appendix A.1) but does not define a generator, so the generator is a
frozen specification of this library.  It is restated here from that
specification, step by step, with one numpy operation per rounding step:

    S[i, j] = z(seed, i, j) * fp32(1/sqrt(r)),   z iid ~ N(0, 1)
    =>  E[S S^T] = I      (the unbiasedness premise of Theorem 3.2(a))

1. Bits: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) with
   key = (seed mod 2^32, seed div 2^32) and counter = (i, j div 4, 0, kind).
   The four output words x0..x3 belong to columns 4q..4q+3 of row i:
   (x0, x1) make the pair (4q, 4q+1) and (x2, x3) the pair (4q+2, 4q+3).
2. Box-Muller in binary32 using only +, -, * (each a separate round-to-nearest-even
   step: no fused multiply-add, no division, no square root, no libm) and moves
   between integer and float bit patterns, so that the same straight-line
   sequence runs at full rate on GPU ALUs and in numpy:
       u     = ((xa >> 9) + 0.5) * 2^-23                   in (0, 1), exact
       rho   = sqrt(-2 ln u)      ln by atanh series with a Newton reciprocal,
                                  sqrt as w * rsqrt(w) with a Newton rsqrt
       oct   = xb >> 29;  a = ((xb >> 6) & 0x7FFFFF) * 2^-23   in [0, 1), exact
       theta = (oct + a) * pi/4, evaluated as a reflection into [0, pi/4]
       z(4q or 4q+2) = rho * cos(theta),  z(next column) = rho * sin(theta)
3. Scale by fp32(1/sqrt(r)) (the double-precision value rounded once).
4. For the bf16 data path the operand is that value rounded to bfloat16 with
   round-to-nearest-even.

The values depend on (seed, kind, i, j) only, never on d_in, r's tiling or on
who asks, so the forward pass and the reconstruction see identical bits.
"""
from __future__ import annotations

import numpy as np

_M32 = np.uint64(0xFFFFFFFF)
# Philox4x32 round multipliers and Weyl key increments (Salmon et al. 2011, Sec. 3.3).
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)

_F = np.float32


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox4x32 on arrays of 32-bit words held in uint64.

    One round maps (c0, c1, c2, c3) to (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2),
    hi(M0*c0) ^ c3 ^ k1, lo(M0*c0)); the key is advanced by the Weyl constants
    between rounds.  Returns the four output words as uint64 arrays < 2^32.
    """
    c0, c1, c2, c3, k0, k1 = (np.asarray(v, dtype=np.uint64) & _M32 for v in (c0, c1, c2, c3, k0, k1))
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(c0, c1, c2, c3, k0, k1)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & _M32
            k1 = (k1 + _PHILOX_W1) & _M32
        p0 = _PHILOX_M0 * c0  # < 2^64, no overflow
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _M32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _M32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return c0, c1, c2, c3


def _as_float(bits):
    return np.asarray(bits, dtype=np.uint32).view(np.float32)


def _as_bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def _reciprocal(d):
    """1/d for d in [1.70, 2.42]: linear start (relative error < 1.8e-2), three Newton steps y <- y*(2 - d*y)."""
    y = _F(0.99259) - _F(0.24264) * d
    for _ in range(3):
        y = y * (_F(2.0) - d * y)
    return y


def _rsqrt(w):
    """1/sqrt(w) for positive normal w: bit-shift start (relative error < 3.5e-2), three Newton steps
    y <- y*(1.5 - (0.5*w)*(y*y))."""
    y = _as_float(np.uint32(0x5F3759DF) - (_as_bits(w) >> np.uint32(1)))
    h = _F(0.5) * w
    for _ in range(3):
        y = y * (_F(1.5) - h * (y * y))
    return y


def _ln_unit_interval(u):
    """Natural log of binary32 u in (0, 1).

    u = mant * 2^e with mant in [1, 2); if mant > sqrt(2) (mantissa field above
    0x3504F3) use mant/2 and e+1, so mant in (0.7071, 1.4143).  Then with
    t = (mant-1)/(mant+1):  ln mant = 2*(t + t^3/3 + ... + t^11/11), Horner in
    t^2, and ln u = e*ln2 + ln mant.  The exponent becomes a float through the
    bit pattern of 1.5*2^23 + e (exact).
    """
    bits = _as_bits(u)
    frac = bits & np.uint32(0x7FFFFF)
    upper = frac > np.uint32(0x3504F3)
    mant = _as_float(np.where(upper, np.uint32(0x3F000000), np.uint32(0x3F800000)) | frac)
    e_plus_127 = (bits >> np.uint32(23)) + upper.astype(np.uint32)            # in [103, 127]
    e_f = _as_float(np.uint32(0x4B400000 - 127) + e_plus_127) - _F(12582912.0)
    one = _F(1.0)
    t = (mant - one) * _reciprocal(mant + one)
    t2 = t * t
    p = _F(1.0 / 11.0)
    for c in (_F(1.0 / 9.0), _F(1.0 / 7.0), _F(1.0 / 5.0), _F(1.0 / 3.0), _F(1.0)):
        p = p * t2
        p = p + c
    ln_mant = (_F(2.0) * t) * p
    return e_f * _F(np.log(2.0)) + ln_mant


def _sincos_octant(a):
    """sin and cos of y = a*fp32(pi/4), a in [0, 1]: Taylor series, Horner in y^2."""
    y = a * _F(np.pi / 4.0)
    y2 = y * y
    s = _F(1.0 / 362880.0)
    for c in (_F(-1.0 / 5040.0), _F(1.0 / 120.0), _F(-1.0 / 6.0), _F(1.0)):
        s = s * y2
        s = s + c
    s = s * y
    c_ = _F(-1.0 / 3628800.0)
    for c in (_F(1.0 / 40320.0), _F(-1.0 / 720.0), _F(1.0 / 24.0), _F(-0.5), _F(1.0)):
        c_ = c_ * y2
        c_ = c_ + c
    return s, c_


def gaussian_pair(xa, xb):
    """Map two 32-bit words to two independent standard normals (binary32).

    Box-Muller: radius from xa, angle from xb.  The angle's octant (top three
    bits of xb) decides which of +-sin y, +-cos y is the cosine and which the
    sine of theta = (oct + a)*pi/4; odd octants use the reflected offset 1-a.
    """
    xa = np.asarray(xa, dtype=np.uint64).astype(np.uint32)
    xb = np.asarray(xb, dtype=np.uint64).astype(np.uint32)
    # u = (2n+1) * 2^-24 with n = xa >> 9: the float 1.n minus (1 - 2^-24), exact
    u = _as_float(np.uint32(0x3F800000) | (xa >> np.uint32(9))) - _as_float(np.uint32(0x3F7FFFFF))
    w = _F(-2.0) * _ln_unit_interval(u)
    rho = w * _rsqrt(w)

    octant = (xb >> np.uint32(29)).astype(np.int64)
    a = _as_float(np.uint32(0x3F800000) | ((xb >> np.uint32(6)) & np.uint32(0x7FFFFF))) - _F(1.0)
    a = np.where(octant & 1, _F(1.0) - a, a)
    sin_y, cos_y = _sincos_octant(a)

    # theta = k*pi/2 +- y : octants 1,2,5,6 exchange the roles of sin y and cos y
    swap = np.isin(octant, (1, 2, 5, 6))
    cos_t = np.where(swap, sin_y, cos_y)
    sin_t = np.where(swap, cos_y, sin_y)
    cos_t = np.where(np.isin(octant, (2, 3, 4, 5)), -cos_t, cos_t)  # cos < 0 on (pi/2, 3pi/2)
    sin_t = np.where(octant >= 4, -sin_t, sin_t)                    # sin < 0 on (pi, 2pi)
    return rho * cos_t, rho * sin_t


def standard_normal_block(seed: int, n_rows: int, n_cols: int, kind: int = 0, row0: int = 0):
    """z(seed, i, j) for row0 <= i < row0+n_rows, 0 <= j < n_cols, as binary32."""
    if n_cols % 4:
        raise ValueError("n_cols must be a multiple of 4 (one Philox call covers 4 columns)")
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    i = np.arange(row0, row0 + n_rows, dtype=np.uint64)[:, None]
    q = np.arange(n_cols // 4, dtype=np.uint64)[None, :]
    x0, x1, x2, x3 = philox4x32_10(i, q, 0, kind, seed & 0xFFFFFFFF, seed >> 32)
    z = np.empty((n_rows, n_cols), dtype=np.float32)
    z[:, 0::4], z[:, 1::4] = gaussian_pair(x0, x1)
    z[:, 2::4], z[:, 3::4] = gaussian_pair(x2, x3)
    return z


def sketch(seed: int, d_in: int, r: int, kind: int = 0):
    """The d_in x r sketch S in binary32: z * fp32(1/sqrt(r)); E[S S^T] = I."""
    scale = _F(1.0 / np.sqrt(np.float64(r)))
    return standard_normal_block(seed, d_in, r, kind) * scale


def round_to_bf16(x):
    """Round binary32 to the nearest bfloat16 (ties to even); returned as binary32."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return rounded.astype(np.uint32).view(np.float32)


def sketch_for_dtype(seed: int, d_in: int, r: int, dtype: str, kind: int = 0):
    """S as the data path of `dtype` ("f32" or "bf16") uses it, promoted to float64."""
    s = sketch(seed, d_in, r, kind)
    if dtype == "bf16":
        s = round_to_bf16(s)
    elif dtype != "f32":
        raise ValueError(dtype)
    return s.astype(np.float64)
