"""Reproducible float32 elementary functions, built only from IEEE-754 operations.

Two steps of the rollout path turn floating point into integers that must agree bit
for bit between this oracle and the GPU: the seeded normal weights and the sampler's
quantised probabilities.  libm and CUDA's math library differ in the last ulp, so the
project defines ln, sin/cos(2*pi*k/2^24) and exp as short polynomial recipes that use
nothing but float32 add, multiply, divide and sqrt, each rounded to nearest-even and
never fused.  Every operation below is a separate numpy float32 operation, which is
exactly that.  (The polynomials are plain Taylor / atanh series; accuracy ~1e-7.)
"""
import numpy as np

F = np.float32


def _c(x):
    """float32 constant from a double expression (one rounding, double -> float)."""
    return np.float32(x)


_SQRT2 = _c(1.41421356237309504880)
_LN2 = _c(0.69314718055994530942)
_HALF_PI = _c(1.57079632679489661923)


def ln_unit(u):
    """Natural log of float32 u in (0, 1], u normal.  Series: ln m = 2 atanh((m-1)/(m+1))."""
    u = np.asarray(u, dtype=F)
    bits = u.view(np.uint32)
    e = (bits >> np.uint32(23)).astype(np.int32) - np.int32(127)
    m = ((bits & np.uint32(0x007FFFFF)) | np.uint32(0x3F800000)).view(F)
    big = m > _SQRT2
    m = np.where(big, m * F(0.5), m).astype(F)
    e = np.where(big, e + np.int32(1), e).astype(np.int32)
    f = (m - F(1.0)).astype(F)
    s = (f / (F(2.0) + f)).astype(F)
    z = (s * s).astype(F)
    t = _c(1.0 / 11.0)
    for k in (9.0, 7.0, 5.0, 3.0, 1.0):
        t = ((t * z).astype(F) + _c(1.0 / k)).astype(F)
    lnm = ((F(2.0) * s).astype(F) * t).astype(F)
    return ((e.astype(F) * _LN2).astype(F) + lnm).astype(F)


_SIN_C = [_c(1.0 / 6227020800.0), _c(-1.0 / 39916800.0), _c(1.0 / 362880.0), _c(-1.0 / 5040.0),
          _c(1.0 / 120.0), _c(-1.0 / 6.0), _c(1.0)]
_COS_C = [_c(-1.0 / 87178291200.0), _c(1.0 / 479001600.0), _c(-1.0 / 3628800.0), _c(1.0 / 40320.0),
          _c(-1.0 / 720.0), _c(1.0 / 24.0), _c(-0.5), _c(1.0)]


def sincos_turn24(k24):
    """(sin, cos) of the angle 2*pi*k24/2^24, k24 integer in [0, 2^24).

    The quadrant is taken exactly from the top two bits; the remainder maps to
    x in [0, pi/2) where Taylor polynomials in x^2 are evaluated by Horner's rule.
    """
    k24 = np.asarray(k24, dtype=np.uint32)
    q = (k24 >> np.uint32(22)).astype(np.int32)
    r = (k24 & np.uint32(0x3FFFFF)).astype(F)
    x = ((r * _c(2.0 ** -22)).astype(F) * _HALF_PI).astype(F)
    x2 = (x * x).astype(F)
    ps = _SIN_C[0]
    for c in _SIN_C[1:]:
        ps = ((ps * x2).astype(F) + c).astype(F)
    s = (x * ps).astype(F)
    pc = _COS_C[0]
    for c in _COS_C[1:]:
        pc = ((pc * x2).astype(F) + c).astype(F)
    c_ = pc
    sin = np.where(q == 0, s, np.where(q == 1, c_, np.where(q == 2, -s, -c_))).astype(F)
    cos = np.where(q == 0, c_, np.where(q == 1, -s, np.where(q == 2, -c_, s))).astype(F)
    return sin, cos


_LOG2E = _c(1.44269504088896340736)
_LN2_HI = np.uint32(0x3F317200).view(F)            # 0.693145751953125, 15 significant bits
_LN2_LO = _c(0.69314718055994530942 - 0.693145751953125)
_EXP_C = [_c(1.0 / 5040.0), _c(1.0 / 720.0), _c(1.0 / 120.0), _c(1.0 / 24.0), _c(1.0 / 6.0), _c(0.5),
          _c(1.0), _c(1.0)]
EXP_CUTOFF = F(-24.0)


def exp_nonpos(x):
    """exp(x) for float32 x <= 0; returns exactly 0 below EXP_CUTOFF (= -24)."""
    x = np.asarray(x, dtype=F)
    dead = x < EXP_CUTOFF
    xs = np.where(dead, F(0.0), x).astype(F)
    n = np.rint((xs * _LOG2E).astype(F)).astype(F)           # round half to even
    r = (xs - (n * _LN2_HI).astype(F)).astype(F)
    r = (r - (n * _LN2_LO).astype(F)).astype(F)
    p = _EXP_C[0]
    for c in _EXP_C[1:]:
        p = ((p * r).astype(F) + c).astype(F)
    scale = ((n.astype(np.int32) + np.int32(127)).astype(np.uint32) << np.uint32(23)).view(F)
    out = (p * scale).astype(F)
    return np.where(dead, F(0.0), out).astype(F)


def to_bf16_bits(x):
    """float32 -> bfloat16 bit pattern (uint16), round to nearest even.  Finite inputs."""
    b = np.asarray(x, dtype=F).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    return ((b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(h):
    return (np.asarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(F)


def round_bf16(x):
    return from_bf16_bits(to_bf16_bits(x))
