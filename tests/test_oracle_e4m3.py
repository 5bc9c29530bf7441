"""Pins for the oracle's software e4m3 codec and block quantizer (App. E.2 semantics)."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O

FINITE = [c for c in range(256) if (c & 0x7F) != 0x7F]


def test_decode_table_against_format_definition():
    # OCP e4m3fn: bias 7, subnormal quantum 2^-9, max 448, no infinity, S.1111.111 = NaN
    d = O.e4m3_decode(np.arange(256, dtype=np.uint8))
    assert d[0x00] == 0.0 and d[0x80] == 0.0 and math.copysign(1, d[0x80]) == -1
    assert d[0x01] == 2.0 ** -9 and d[0x07] == 7 * 2.0 ** -9
    assert d[0x08] == 2.0 ** -6 and d[0x38] == 1.0 and d[0x3C] == 1.5
    assert d[0x7E] == 448.0 and d[0xFE] == -448.0 and d[0x77] == 240.0
    assert math.isnan(d[0x7F]) and math.isnan(d[0xFF])
    pos = d[:0x7F]
    assert np.all(np.diff(pos) > 0)
    assert np.array_equal(d[0x80:0xFF], -pos)
    # library special case: torch's own decode of the same bytes
    t = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    fin = np.array(FINITE)
    assert np.array_equal(t[fin], d[fin])


def test_encode_roundtrip_all_codes():
    codes = np.array(FINITE, dtype=np.uint8)
    vals = O.e4m3_decode(codes).astype(np.float32)
    assert np.array_equal(O.e4m3_encode(vals), codes)   # includes -0 -> 0x80


def test_midpoints_round_to_even_and_neighbours():
    d = O.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    for c in range(0x7E):
        lo, hi = d[c], d[c + 1]
        mid = np.float32((lo + hi) / 2)          # exact in fp32
        assert float(mid) == (lo + hi) / 2
        even = c if c % 2 == 0 else c + 1
        assert O.e4m3_encode([mid])[0] == even
        assert O.e4m3_encode([-mid])[0] == (even | 0x80)
        assert O.e4m3_encode([np.nextafter(mid, np.float32(np.inf))])[0] == c + 1
        assert O.e4m3_encode([np.nextafter(mid, np.float32(0))])[0] == c


def test_saturation_and_specials():
    enc = lambda v: int(O.e4m3_encode([np.float32(v)])[0])
    assert enc(448) == 0x7E and enc(449) == 0x7E and enc(463.9) == 0x7E
    assert enc(464) == 0x7E and enc(465) == 0x7E and enc(1e30) == 0x7E and enc(np.inf) == 0x7E
    assert enc(-1e30) == 0xFE and enc(-np.inf) == 0xFE
    assert enc(np.nan) == 0x7F
    assert enc(2.0 ** -10) == 0x00                      # tie between 0 and 2^-9 -> even (0)
    assert enc(np.nextafter(np.float32(2.0 ** -10), np.float32(1))) == 0x01
    assert enc(3 * 2.0 ** -10) == 0x02                  # tie between 1 and 2 quanta -> 2
    assert enc(15 * 2.0 ** -10) == 0x08                 # tie between 7 quanta and 2^-6 -> 2^-6
    assert enc(1e-30) == 0x00 and enc(-1e-30) == 0x80


def test_encode_matches_library_cast_in_range():
    # library special case: torch's CPU cast is RNE and agrees wherever no saturation is involved
    rng = np.random.default_rng(0)
    parts = [rng.uniform(-448, 448, 200000), rng.standard_normal(200000),
             rng.standard_normal(200000) * 2.0 ** -7, rng.uniform(-0.02, 0.02, 100000),
             rng.uniform(-2 ** -8, 2 ** -8, 100000)]
    y = np.concatenate(parts).astype(np.float32)
    want = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(O.e4m3_encode(y), want)


def test_encode_is_nearest_by_brute_force():
    # definition: the nearest representable value, ties to the even code
    d = O.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    rng = np.random.default_rng(3)
    y = np.abs(np.concatenate([rng.uniform(0, 448, 3000), rng.uniform(0, 0.05, 3000)])).astype(np.float32)
    got = O.e4m3_encode(y)
    for v, g in zip(y, got):
        dist = np.abs(d - float(v))
        best = np.flatnonzero(dist == dist.min())
        want = best[0] if len(best) == 1 else [b for b in best if b % 2 == 0][0]
        assert g == want


@pytest.mark.parametrize("blk", [32, 128])
def test_quantizer_definition_fp32_scale(blk):
    # scale = amax/448 in fp32, cast RNE, rescale (App. E.2); checked against a direct numpy restatement
    rng = np.random.default_rng(5)
    X = rng.standard_normal((8, 4 * blk)).astype(np.float32)
    codes, scales, _ = O.quant_rows(X, blk)
    Xb = X.reshape(8, 4, blk)
    amax = np.abs(Xb).max(axis=2)
    assert np.array_equal(scales, (amax / np.float32(448)).astype(np.float32))
    inv = (np.float32(448) / amax).astype(np.float32)
    y = (Xb * inv[:, :, None]).astype(np.float32)
    want = torch.from_numpy(y.reshape(8, -1)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    # torch does not saturate above 464 but y <= 448(1+2^-23) here, so the casts agree
    assert np.array_equal(codes, want)
    # every non-zero block carries a +-448 code
    assert np.all((codes.reshape(8, 4, blk) & 0x7F).max(axis=2) == 0x7E)
    # the B-side quantizer is the same map applied along the other axis
    cT, sT, _ = O.quant_cols(np.ascontiguousarray(X.T), blk)
    assert np.array_equal(cT.T, codes) and np.array_equal(sT.T, scales)


def test_quantizer_power_of_two_homogeneity():
    # App. E.2: a power-of-two rescale leaves the codes bit-identical and scales the scales
    rng = np.random.default_rng(6)
    X = rng.standard_normal((16, 256)).astype(np.float32)
    c0, s0, _ = O.quant_rows(X, 32)
    for k in (-20, -3, 1, 7, 30):
        f = np.float32(2.0 ** k)
        c1, s1, _ = O.quant_rows(X * f, 32)
        assert np.array_equal(c0, c1)
        assert np.array_equal(s1, s0 * f)


def test_minimum_scale_clamp_engages_between_1e12_and_1e13():
    # App. E.2: Q(cx) = cQ(x) holds for factors down to 1e-12 and breaks at 1e-13
    rng = np.random.default_rng(7)
    X = (rng.random((64, 256), dtype=np.float32) * 2 - 1).astype(np.float32)
    X[:, ::32] = np.sign(X[:, ::32]) * np.float32(0.999)     # every block has amax just below 1
    c0, s0, _ = O.quant_rows(X, 32)
    base = O.dequant_rows(c0, s0, 32)
    dev = {}
    for f in (1e-3, 1e-9, 1.25e-12, 1e-13):
        c1, s1, _ = O.quant_rows((X * np.float32(f)).astype(np.float32), 32)
        d = O.dequant_rows(c1, s1, 32) / f
        dev[f] = np.linalg.norm(d - base) / np.linalg.norm(base)
    assert dev[1e-3] < 2e-3 and dev[1e-9] < 2e-3 and dev[1.25e-12] < 2e-3
    assert dev[1e-13] > 1e-2
    # all-zero block: codes zero, scale is the clamped one
    cz, sz, _ = O.quant_rows(np.zeros((1, 32), np.float32), 32)
    assert not cz.any() and sz[0, 0] == np.float32(1e-12) / np.float32(448)


def test_ue8m0_scale_is_smallest_power_of_two_not_below_amax_over_448():
    rng = np.random.default_rng(8)
    X = (rng.standard_normal((32, 256)) * 10.0 ** rng.uniform(-6, 6, (32, 1))).astype(np.float32)
    X[0, :32] = 0
    X[1, :32] = np.float32(448.0)           # exactly a power of two scale: e = 0
    X[2, :32] = np.float32(448.0 * 4)       # e = 2
    codes, scales, e8 = O.quant_rows(X, 32, mode=O.SCALE_UE8M0)
    amax = np.maximum(np.abs(X.reshape(32, 8, 32)).max(axis=2), np.float32(1e-12))
    s0 = (amax / np.float32(448)).astype(np.float32).astype(np.float64)
    assert np.array_equal(scales.astype(np.float64), 2.0 ** (e8.astype(np.int32) - 127))
    assert np.all(scales >= s0) and np.all(scales / 2 < s0)
    assert e8[1, 0] == 127 and e8[2, 0] == 129
    # no saturation can occur: |x| / scale <= 448
    deq = O.dequant_rows(codes, scales, 32)
    assert np.all(np.abs(deq - X) <= np.abs(X) * 2.0 ** -4 + scales.repeat(32, axis=1) * 2.0 ** -10)
