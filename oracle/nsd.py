"""NSD quantizer oracle (test infrastructure): Python face of `nsd_oracle.c`.

Follows Section 3.1 Eq. (nsd) and Algorithm 1 of the dithered-backprop paper; the readings
taken where the paper is silent are listed at the top of `nsd_oracle.c`.
"""
import ctypes
from fractions import Fraction

import numpy as np

from . import build as _build

_lib = ctypes.CDLL(_build.build())
_lib.oracle_splitmix64_at.restype = ctypes.c_uint64
_lib.oracle_splitmix64_at.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
_lib.oracle_dither_u.restype = ctypes.c_float
_lib.oracle_dither_u.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
_lib.oracle_mean_std.restype = None
_lib.oracle_mean_std.argtypes = [ctypes.c_void_p, ctypes.c_int64,
                                 ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
_lib.oracle_nsd_codes.restype = ctypes.c_int64
_lib.oracle_nsd_codes.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64, ctypes.c_float,
                                  ctypes.c_uint64, ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64)]
_lib.oracle_nsd_codes_literal_f64.restype = ctypes.c_int64
_lib.oracle_nsd_codes_literal_f64.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64,
                                              ctypes.c_float, ctypes.c_uint64, ctypes.c_void_p]

_MASK64 = (1 << 64) - 1


def _f32(x):
    a = np.ascontiguousarray(x, dtype=np.float32)
    return a


def splitmix64_at(seed: int, c: int) -> int:
    """Output number c (0-based) of the SplitMix64 sequence started at `seed`."""
    return int(_lib.oracle_splitmix64_at(seed & _MASK64, c & _MASK64))


def dither_u(seed: int, i: int) -> float:
    """u_i in (0,1): the dither nu_i of Eq. (nsd) is (u_i - 1/2) * Delta."""
    return float(_lib.oracle_dither_u(seed & _MASK64, i & _MASK64))


def derive_layer_seed(seed: int, layer: int) -> int:
    """Seed of layer `layer` in a multi-layer backward pass: output `layer` of the
    SplitMix64 sequence started at `seed` (layers draw independent dither, Eq. (qdz))."""
    return splitmix64_at(seed, layer)


def mean_std(x) -> tuple:
    """Population mean and standard deviation in fp64 (Algorithm 1, std line)."""
    a = _f32(x).ravel()
    m = ctypes.c_double()
    s = ctypes.c_double()
    _lib.oracle_mean_std(a.ctypes.data, a.size, ctypes.byref(m), ctypes.byref(s))
    return m.value, s.value


def step_size(x, s: float) -> np.float32:
    """Delta = s * sigma (Algorithm 1), rounded once to fp32."""
    _, sd = mean_std(x)
    return np.float32(float(np.float32(s)) * sd)


def nsd_codes(x, seed: int, Delta, index_base: int = 0):
    """Integer codes q of Eq. (nsd) (x~ = q * Delta) -> (codes int8 like x, nnz, nsat)."""
    a = _f32(x)
    codes = np.empty(a.shape, dtype=np.int8)
    nsat = ctypes.c_int64()
    nnz = _lib.oracle_nsd_codes(a.ctypes.data, a.size, seed & _MASK64,
                                ctypes.c_float(float(Delta)), index_base & _MASK64,
                                codes.ctypes.data, ctypes.byref(nsat))
    return codes, int(nnz), int(nsat.value)


def nsd_codes_literal_f64(x, seed: int, Delta, index_base: int = 0):
    """Eq. (nsd) evaluated as printed, in fp64, with nu = (u - 1/2) * Delta."""
    a = _f32(x)
    codes = np.empty(a.shape, dtype=np.int32)
    _lib.oracle_nsd_codes_literal_f64(a.ctypes.data, a.size, seed & _MASK64,
                                      ctypes.c_float(float(Delta)), index_base & _MASK64,
                                      codes.ctypes.data)
    return codes


def _splitmix64_py(seed: int, c: int) -> int:
    """SplitMix64 output c in Python integers (independent of the C routine)."""
    z = (seed + (c + 1) * 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _round_to_f32(fr: Fraction) -> Fraction:
    """Round an exact rational to the nearest fp32 (ties to even), returned as a rational.
    Pure integer arithmetic; normal range only (enough for the small pinning cases)."""
    if fr == 0:
        return Fraction(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    # a in [2^e, 2^(e+1)); fp32 spacing there is 2^(e-23)
    if e < -126:
        e = -126                      # subnormal spacing 2^-149
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (fl & 1)):
        fl += 1
    return sign * fl * ulp


def nsd_codes_exact_python(x, seed: int, Delta, index_base: int = 0):
    """The same decision as `nsd_codes`, in exact rational arithmetic (tiny inputs only):
    round32(x * round32(1/Delta) + u), then floor, then saturation."""
    a = _f32(x).ravel()
    D = Fraction(float(np.float32(Delta)))
    out = np.zeros(a.size, dtype=np.int8)
    if D <= 0:
        return out.reshape(np.shape(x))
    inv = _round_to_f32(1 / D)
    for i in range(a.size):
        r = _splitmix64_py(seed & _MASK64, (index_base + i) >> 1)
        h = (r >> 32) if ((index_base + i) & 1) else (r & 0xFFFFFFFF)
        u = Fraction(2 * (h >> 9) + 1, 1 << 24)
        t = _round_to_f32(Fraction(float(a[i])) * inv + u)
        q = t.numerator // t.denominator      # floor
        out[i] = max(-127, min(127, q))
    return out.reshape(np.shape(x))
