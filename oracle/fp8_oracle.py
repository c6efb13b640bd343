"""Float64 CPU checker for the 8-bit (E4M3) storage of the expanded shared-prefix cache.

TEST INFRASTRUCTURE ONLY (imported by the tests, never by the library or its binding; shares no
code with them).

The paper evaluates its method in 16-bit precision and only *assumes* 8-bit weights and caches
in its memory-footprint analysis (Section 4, "HBM Footprint", Fig. 5); it does not say how an 8-bit
cache is encoded.  The reading taken here, which the library follows:

* format: OCP 8-bit floating point E4M3 ("fn" variant): 1 sign, 4 exponent (bias 7), 3 mantissa
  bits, no infinities, 0x7f / 0xff are NaN, largest finite value 448, subnormals m * 2^-9;
* rounding: to nearest, ties to the even code, saturating at +-448;
* scale: one power of two per head and per tensor (K_nope, V): the smallest 2^e with
  amax / 2^e <= 448 (amax over the head's real tokens; 1 if the head is all zero);
* what is encoded: the expanded K_nope / V *as the 16-bit path stores them*, i.e. the exact
  up-projection rounded to bfloat16 (round to nearest even), then encoded.  Rope keys, the
  per-request latent cache and all queries stay 16-bit.

Attention itself is the definition of `mla_oracle.mla_decode`, taken over the decoded values: the
codes are data, the arithmetic after decoding is exact.

Pins (tests/test_oracle_pins.py): the 256-entry decode table against the format's closed forms
(1.0 = 0x38, 448 = 0x7e, 2^-6 = 0x08, 2^-9 = 0x01, 254 finite codes, symmetric in the sign bit);
encode(decode(c)) = c for every finite code; ties at hand-computed midpoints; a brute-force
nearest-value search over the table on random inputs; torch's CPU float8_e4m3fn cast inside the
finite range; the scale rule at exact powers of two; round-trip relative error <= 2^-4 for normal
values.
"""
from __future__ import annotations

from typing import Iterable, Optional, Sequence, Tuple

import numpy as np

from . import mla_oracle as _def

E4M3_MAX = 448.0


def e4m3_decode_table() -> np.ndarray:
    """Value of each of the 256 codes (NaN for 0x7f and 0xff)."""
    t = np.empty(256, dtype=np.float64)
    for c in range(256):
        e, m = (c >> 3) & 0xF, c & 7
        if e == 15 and m == 7:
            v = np.nan
        elif e == 0:
            v = m * 2.0 ** -9
        else:
            v = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[c] = -v if c & 0x80 else v
    return t


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """Round float64 values to E4M3 codes: nearest, ties to even, saturating; NaN -> 0x7f."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    sign = np.where(np.signbit(x), 0x80, 0).astype(np.int64)
    a = np.minimum(a, E4M3_MAX)                       # saturate (also +-inf)
    code = np.zeros(x.shape, dtype=np.int64)
    sub = a < 2.0 ** -6                               # below the smallest normal: fixed step 2^-9
    code[sub] = np.rint(a[sub] * 2.0 ** 9).astype(np.int64)      # 8 = the smallest normal, by construction
    nrm = ~sub & ~np.isnan(a)
    mant, ex = np.frexp(a[nrm])                       # a = mant * 2^ex, mant in [0.5, 1)
    e = ex - 1
    q = np.rint((mant * 2.0 - 1.0) * 8.0).astype(np.int64)      # np.rint rounds halves to even
    carry = q == 8
    e = e + carry
    q = np.where(carry, 0, q)
    c = ((e + 7) << 3) | q
    code[nrm] = np.minimum(c, 0x7E)
    code[np.isnan(a)] = 0x7F
    return (code | sign).astype(np.uint8)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to bfloat16 (nearest even) through float32, returned as float64."""
    u = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def pow2_scale(amax: float) -> float:
    """Smallest power of two s with amax / s <= 448 (1 for amax = 0)."""
    if not amax > 0.0:
        return 1.0
    mant, ex = np.frexp(amax / E4M3_MAX)              # amax / 448 = mant * 2^ex, mant in [0.5, 1)
    return float(2.0 ** (ex - 1 if mant == 0.5 else ex))


def encode_head(x_h: np.ndarray) -> Tuple[np.ndarray, float]:
    """One head's expanded tensor [L, D] (exact) -> (codes uint8 [L, D], scale)."""
    xb = bf16_round(x_h)
    s = pow2_scale(float(np.max(np.abs(xb))) if xb.size else 0.0)
    return e4m3_encode(xb / s), s


def roundtrip_head(x_h: np.ndarray) -> np.ndarray:
    """The values the attention sees for one head: decode(encode(x)) * scale."""
    codes, s = encode_head(x_h)
    return e4m3_decode_table()[codes] * s


def mla_decode_fp8_shared(q_nope: np.ndarray, q_pe: np.ndarray,
                          ckv_shared: np.ndarray, kpe_shared: np.ndarray,
                          ckv_suffix: Sequence[np.ndarray], kpe_suffix: Sequence[np.ndarray],
                          w_uk: np.ndarray, w_uv: np.ndarray, scale: float,
                          pairs: Optional[Iterable[Tuple[int, int]]] = None):
    """`mla_oracle.mla_decode` with the shared prefix's expanded K_nope and V stored in E4M3.

    Same arguments and results.  Only the decompressed keys/values of the *shared* tokens pass
    through encode/decode; everything else is the definition.
    """
    B, H, _ = q_nope.shape
    D_v = w_uv.shape[1]
    out = np.full((B, H, D_v), np.nan, dtype=np.float64)
    lse = np.full((B, H), np.nan, dtype=np.float64)
    if pairs is None:
        by_head = {h: list(range(B)) for h in range(H)}
    else:
        by_head = {}
        for b, h in pairs:
            by_head.setdefault(int(h), []).append(int(b))
    for h, bs in sorted(by_head.items()):
        Ks = roundtrip_head(_def.decompress_head(ckv_shared, w_uk[h]))
        Vs = roundtrip_head(_def.decompress_head(ckv_shared, w_uv[h]))
        for b in bs:
            Kn = _def.decompress_head(ckv_suffix[b], w_uk[h])
            Vn = _def.decompress_head(ckv_suffix[b], w_uv[h])
            K = np.concatenate([Ks, Kn], axis=0)
            V = np.concatenate([Vs, Vn], axis=0)
            R = np.concatenate([kpe_shared, kpe_suffix[b]], axis=0)
            out[b, h], lse[b, h] = _def.attend(q_nope[b, h], q_pe[b, h], K, R, V, scale)
    return out, lse
