"""Pins of the E4M3 checker (oracle/fp8_oracle.py) to things other than itself: the format's closed
forms, hand-computed ties, a brute-force nearest-value search, torch's CPU cast, and the reduction
of the 8-bit-cache operator to the plain definition when every value is exactly representable."""
import math

import numpy as np
import pytest
import torch

from oracle import fp8_oracle as F
from oracle import mla_oracle as O


def test_decode_table_closed_forms():
    t = F.e4m3_decode_table()
    assert t[0x00] == 0.0 and t[0x80] == 0.0 and math.copysign(1.0, t[0x80]) == -1.0
    assert t[0x38] == 1.0 and t[0x39] == 1.125 and t[0x40] == 2.0
    assert t[0x7E] == 448.0 and t[0x08] == 2.0 ** -6 and t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF])
    fin = t[~np.isnan(t)]
    assert fin.size == 254 and np.max(fin) == 448.0 and np.min(fin) == -448.0
    assert np.array_equal(t[:0x7F], -t[0x80:0xFF])
    assert np.all(np.diff(t[:0x7F]) > 0)                      # codes of one sign are ordered like their values


def test_encode_inverts_decode_on_every_finite_code():
    t = F.e4m3_decode_table()
    codes = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=np.uint8)
    assert np.array_equal(F.e4m3_encode(t[codes]), codes)


def test_ties_go_to_the_even_code_and_large_values_saturate():
    enc = lambda v: int(F.e4m3_encode(np.array([v]))[0])
    assert enc(1.0625) == 0x38            # halfway 1.0 (mantissa 0) .. 1.125 (1): even is 0
    assert enc(1.1875) == 0x3A            # halfway 1.125 (1) .. 1.25 (2): even is 2
    assert enc(-1.1875) == 0xBA
    assert enc(2.0 ** -10) == 0x00        # halfway 0 .. 2^-9
    assert enc(3 * 2.0 ** -10) == 0x02    # halfway 2^-9 .. 2^-8
    assert enc(15 * 2.0 ** -10) == 0x08   # halfway largest subnormal .. smallest normal: even is the normal
    assert enc(1.9375) == 0x40            # halfway 1.875 (7) .. 2.0 (next exponent, mantissa 0)
    assert enc(447.9) == 0x7E and enc(1e9) == 0x7E and enc(-1e9) == 0xFE and enc(float("inf")) == 0x7E
    assert enc(float("nan")) == 0x7F


def test_encode_matches_brute_force_nearest_value():
    t = F.e4m3_decode_table()
    cand = np.array([c for c in range(0x7F)], dtype=np.int64)      # non-negative finite codes, ascending values
    r = np.random.default_rng(3)
    x = np.concatenate([r.standard_normal(4000) * 3.0, r.standard_normal(2000) * 0.01, r.uniform(-448, 448, 2000),
                        r.standard_normal(500) * 2.0 ** -8])
    got = F.e4m3_encode(x)
    for xi, gi in zip(x, got):
        a = abs(xi)
        d = np.abs(t[cand] - a)
        best = np.flatnonzero(d == d.min())
        c = int(best[0]) if best.size == 1 else int([b for b in best if b % 2 == 0][0])   # tie: even code
        assert int(gi) == (c | (0x80 if xi < 0 else 0)), (xi, gi, c)


def test_encode_matches_torch_cast_inside_the_finite_range():
    r = np.random.default_rng(4)
    x = np.concatenate([r.standard_normal(20000) * 5.0, r.uniform(-448, 448, 20000), r.standard_normal(5000) * 1e-2,
                        np.arange(-64, 65) * 2.0 ** -10])
    x = x.astype(np.float32).astype(np.float64)               # torch casts from float32
    want = torch.from_numpy(x.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = F.e4m3_encode(x)
    nz = x != 0                                               # the sign of a rounded-to-zero value is kept by both
    assert np.array_equal(got[nz], want[nz])


def test_bf16_round_matches_torch():
    r = np.random.default_rng(5)
    x = np.concatenate([r.standard_normal(20000), r.standard_normal(2000) * 1e-20, r.standard_normal(2000) * 1e20,
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -1.0 - 2.0 ** -8])])   # ties
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(F.bf16_round(x), want)


def test_scale_rule():
    assert F.pow2_scale(0.0) == 1.0
    assert F.pow2_scale(448.0) == 1.0 and F.pow2_scale(448.0001) == 2.0 and F.pow2_scale(447.0) == 1.0
    assert F.pow2_scale(224.0) == 0.5 and F.pow2_scale(224.5) == 1.0
    assert F.pow2_scale(3.5) == 2.0 ** -7 and F.pow2_scale(3.6) == 2.0 ** -6
    r = np.random.default_rng(6)
    for a in np.exp(r.uniform(-20, 20, 200)):
        s = F.pow2_scale(a)
        assert a / s <= 448.0 < a / (s / 2) and math.log2(s) == round(math.log2(s))


def test_roundtrip_error_bound():
    """Normal values: relative error of decode(encode(x)) at most 2^-4 (half a step of a 3-bit mantissa)."""
    r = np.random.default_rng(7)
    x = r.standard_normal((64, 32)) * 4.0
    y = F.roundtrip_head(x)
    xb = F.bf16_round(x)
    s = F.pow2_scale(np.max(np.abs(xb)))
    normal = np.abs(xb) >= s * 2.0 ** -6
    assert np.all(np.abs(y - xb)[normal] <= np.abs(xb)[normal] * 2.0 ** -4 * (1 + 1e-12))
    assert np.all(np.abs(y - xb)[~normal] <= s * 2.0 ** -10)  # subnormal range: half of the fixed step


def test_fp8_operator_reduces_to_the_definition_on_representable_values():
    """If every expanded K and V value is an E4M3 value times one power of two, encoding is lossless and the
    operator equals the plain definition: pins the wiring of mla_decode_fp8_shared (which tensors pass
    through the codec, and that nothing else changes)."""
    r = np.random.default_rng(8)
    B, H, Ls, Dn, Dr, Dv, Dl = 2, 3, 7, 4, 2, 3, 4
    # one-hot up-projections and latents made of small E4M3 values: K = selected latent entries, exactly
    grid = F.e4m3_decode_table()[np.array([0x30, 0x34, 0x38, 0x3C, 0x40, 0xB8, 0xB4, 0x28])]
    ckv_s = r.choice(grid, size=(Ls, Dl))
    w_uk = np.zeros((H, Dn, Dl))
    w_uv = np.zeros((H, Dv, Dl))
    for h in range(H):
        for i in range(Dn):
            w_uk[h, i, (i + h) % Dl] = 1.0
        for i in range(Dv):
            w_uv[h, i, (i + 2 * h) % Dl] = -2.0                # a power-of-two factor keeps values representable
    d = dict(q_nope=r.standard_normal((B, H, Dn)), q_pe=r.standard_normal((B, H, Dr)), ckv_shared=ckv_s,
             kpe_shared=r.standard_normal((Ls, Dr)), ckv_suffix=[r.standard_normal((n, Dl)) for n in (3, 0)],
             kpe_suffix=[r.standard_normal((n, Dr)) for n in (3, 0)], w_uk=w_uk, w_uv=w_uv, scale=0.4)
    args = (d["q_nope"], d["q_pe"], d["ckv_shared"], d["kpe_shared"], d["ckv_suffix"], d["kpe_suffix"], d["w_uk"],
            d["w_uv"], d["scale"])
    o1, l1 = O.mla_decode(*args)
    o2, l2 = F.mla_decode_fp8_shared(*args)
    assert np.allclose(o1, o2, rtol=0, atol=1e-14) and np.allclose(l1, l2, rtol=0, atol=1e-14)


def test_fp8_operator_only_touches_the_shared_prefix():
    """Generic inputs: with an empty shared prefix the two operators agree exactly; with one, they differ by no
    more than the perturbation bound of the codec (and do differ)."""
    r = np.random.default_rng(9)
    B, H, Dn, Dr, Dv, Dl = 2, 2, 8, 4, 8, 16
    mk = lambda Ls: (r.standard_normal((B, H, Dn)), r.standard_normal((B, H, Dr)), r.standard_normal((Ls, Dl)),
                     r.standard_normal((Ls, Dr)), [r.standard_normal((n, Dl)) for n in (5, 9)],
                     [r.standard_normal((n, Dr)) for n in (5, 9)], r.standard_normal((H, Dn, Dl)) / 4,
                     r.standard_normal((H, Dv, Dl)) / 4, 0.3)
    a = mk(0)
    o1, l1 = O.mla_decode(*a)
    o2, l2 = F.mla_decode_fp8_shared(*a)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    a = mk(40)
    o1, l1 = O.mla_decode(*a)
    o2, l2 = F.mla_decode_fp8_shared(*a)
    err = np.max(np.abs(o1 - o2))
    assert 0 < err < 0.25 and np.max(np.abs(l1 - l2)) < 0.25
