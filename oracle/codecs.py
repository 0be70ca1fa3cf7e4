"""Number formats the oracle needs: bfloat16 and FP8 E4M3 (finite-only variant).

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it shares no code with the CUDA library.

The paper fixes no rounding points for the expert FFN; the reading taken here
is that the SwiGLU activation and the layer output are each rounded once to
bfloat16 with round-to-nearest-even, and that FP8 tensors are E4M3 with the
largest finite magnitude 448, no infinities, codes 0x7F/0xFF = NaN, conversion
by round-to-nearest-even with saturation.

Everything works on numpy arrays; bf16 values travel as uint16 bit patterns and
E4M3 values as uint8 bit patterns, so no library float type decides a rounding.
"""
from __future__ import annotations

import numpy as np


def bf16_decode(bits) -> np.ndarray:
    """uint16 bit patterns -> the exact values as float64."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def bf16_rne(v) -> np.ndarray:
    """float64 values -> bfloat16 bit patterns (uint16), round to nearest even,
    straight from binary64 (no intermediate binary32 rounding)."""
    v = np.asarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.float64)
    a = np.abs(v)
    with np.errstate(over="ignore", invalid="ignore"):
        # normal bf16 range: keep 8 significant bits (1 implicit + 7 stored)
        _, ex = np.frexp(a)                      # a = m * 2**ex, m in [0.5, 1)
        ex = np.maximum(ex, -125)                # below 2**-126 the quantum stays 2**-133
        quantum = np.ldexp(1.0, ex - 8)
        q = np.rint(a / quantum) * quantum       # np.rint rounds half to even
    out[...] = np.copysign(q, v)
    big = q >= np.ldexp(1.0, 128)                # rounds past the largest finite bf16
    out[big] = np.copysign(np.inf, v[big])
    out[np.isnan(v)] = np.nan
    f32 = out.astype(np.float32)                 # exact: out is representable in bf16
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_round(v) -> np.ndarray:
    """float64 -> nearest bfloat16 value, returned as float64."""
    return bf16_decode(bf16_rne(v))


# --- FP8 E4M3 (bias 7, 3 mantissa bits, max 448, no inf) ----------------------

def _e4m3_table() -> np.ndarray:
    t = np.empty(256, dtype=np.float64)
    for code in range(256):
        s = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            t[code] = np.nan
        elif e == 0:
            t[code] = s * m * 2.0 ** -9          # subnormals: m/8 * 2**-6
        else:
            t[code] = s * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return t


E4M3_VALUES = _e4m3_table()
E4M3_MAX = 448.0


def e4m3_decode(codes) -> np.ndarray:
    return E4M3_VALUES[np.asarray(codes, dtype=np.uint8)]


def e4m3_rne_sat(v) -> np.ndarray:
    """float64 (finite) -> E4M3 codes (uint8): round to nearest even, then
    saturate to +-448.  NaN codes are never produced for finite input."""
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    _, ex = np.frexp(a)
    ex = np.maximum(ex, -5)                      # below 2**-6 the quantum stays 2**-9
    quantum = np.ldexp(1.0, ex - 4)              # 4 significant bits
    q = np.minimum(np.rint(a / quantum) * quantum, E4M3_MAX)
    # encode q (exactly representable) into bits
    m, e2 = np.frexp(q)                          # q = m * 2**e2, m in [0.5,1)
    is_sub = q < 2.0 ** -6
    exp_field = np.where(is_sub, 0, e2 - 1 + 7).astype(np.int64)
    man_field = np.where(is_sub, np.rint(q * 2.0 ** 9), np.rint((m * 2.0 - 1.0) * 8.0)).astype(np.int64)
    code = (exp_field << 3) | man_field
    code = np.where(q == 0.0, 0, code)
    sign = (np.signbit(v)).astype(np.int64) << 7
    return (code | sign).astype(np.uint8)
