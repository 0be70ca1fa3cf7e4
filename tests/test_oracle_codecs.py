"""Pins for the oracle's number formats: exhaustive round trips, hand-computed
ties, and agreement with torch's own bf16 / float8_e4m3fn conversions."""
import numpy as np
import torch

from oracle import codecs


def test_bf16_all_codes_round_trip():
    b = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        v = codecs.bf16_decode(b)
    finite = np.isfinite(v)
    assert np.array_equal(codecs.bf16_rne(v[finite]), b[finite])
    assert np.isinf(codecs.bf16_decode(codecs.bf16_rne(np.array([1e39]))))[0]


def test_bf16_ties_to_even_by_hand():
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: even mantissa (1.0) wins
    assert codecs.bf16_round(np.array([1 + 2.0 ** -8]))[0] == 1.0
    # 1 + 3*2^-8 is halfway between 1+2^-7 (odd) and 1+2^-6 (even)
    assert codecs.bf16_round(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    # just above / below the tie
    assert codecs.bf16_round(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1 + 2.0 ** -7
    assert codecs.bf16_round(np.array([1 + 2.0 ** -8 - 2.0 ** -40]))[0] == 1.0
    # a value whose binary32 rounding would land on a tie (double rounding trap)
    v = 1 + 2.0 ** -8 + 2.0 ** -30
    assert codecs.bf16_round(np.array([v]))[0] == 1 + 2.0 ** -7
    assert codecs.bf16_round(np.array([-v]))[0] == -(1 + 2.0 ** -7)
    # subnormal quantum 2^-133
    assert codecs.bf16_round(np.array([2.0 ** -133 * 2.5]))[0] == 2.0 ** -133 * 2


def test_bf16_matches_torch_on_binary32_values():
    rng = np.random.default_rng(0)
    f = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = codecs.bf16_rne(f.astype(np.float64))
    assert np.array_equal(got, want)


def test_e4m3_codes_round_trip_and_constants():
    codes = np.arange(256, dtype=np.uint8)
    v = codecs.e4m3_decode(codes)
    ok = ~np.isnan(v)
    assert set(codes[~ok].tolist()) == {0x7F, 0xFF}
    back = codecs.e4m3_rne_sat(v[ok])
    # -0 and +0 keep their sign bit
    assert np.array_equal(back, codes[ok])
    assert np.nanmax(v) == 448.0
    assert np.min(v[(v > 0)]) == 2.0 ** -9


def test_e4m3_rounding_and_saturation():
    enc = lambda x: codecs.e4m3_decode(codecs.e4m3_rne_sat(np.array([x])))[0]
    assert enc(1000.0) == 448.0 and enc(-1e9) == -448.0
    assert enc(464.0) == 448.0            # would round to 480 without saturation? no: tie -> even = 448
    assert enc(1.0625) == 1.0             # tie between 1.0 and 1.125 -> even mantissa
    assert enc(1.1875) == 1.25            # tie between 1.125 (odd) and 1.25 (even)
    assert enc(2.0 ** -10) == 0.0         # tie between 0 and 2^-9 -> even (0)
    assert enc(3 * 2.0 ** -10) == 2.0 ** -8


def test_e4m3_matches_torch():
    rng = np.random.default_rng(1)
    f = (rng.standard_normal(100000) * np.exp(rng.uniform(-8, 5.5, 100000))).astype(np.float32)
    f = np.clip(f, -448, 448)
    want = torch.from_numpy(f).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = codecs.e4m3_rne_sat(f.astype(np.float64))
    assert np.array_equal(got, want)
