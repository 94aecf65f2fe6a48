"""Pins for the oracle's FP8 E4M3 quantiser (O6): the format's published
constants, hand-worked roundings, round trips of every code, torch's
float8_e4m3fn conversion as the library special case."""
import numpy as np
import pytest
import torch

from oracle import lt_oracle as O


def test_format_constants():
    t = O.e4m3_values()
    assert t[0x00] == 0.0 and t[0x80] == 0.0 and np.signbit(t[0x80])
    assert t[0x7E] == 448.0 and t[0xFE] == -448.0                  # largest finite
    assert np.isnan(t[0x7F]) and np.isnan(t[0xFF])                 # the only NaNs; no infinities
    assert t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9       # subnormals
    assert t[0x08] == 2.0 ** -6                                    # smallest normal
    assert t[0x38] == 1.0 and t[0x39] == 1.125 and t[0x40] == 2.0
    fin = t[:0x7F]
    assert np.all(np.diff(fin) > 0)                                # codes 0..126 increase strictly
    assert np.sum(~np.isnan(t)) == 254


def test_hand_worked_roundings_and_saturation():
    q = lambda x, s=1.0: O.quantize_e4m3(np.array([x]), s)
    assert q(0.3)[1][0] == 0.3125                                  # between 0.28125 and 0.3125
    assert q(1.0625)[1][0] == 1.0                                  # tie 1.0 / 1.125 -> even mantissa (1.0)
    assert q(1.1875)[1][0] == 1.25                                 # tie 1.125 / 1.25 -> even mantissa (1.25)
    assert q(-17.0)[1][0] == -16.0                                 # tie -16 / -18 -> even
    assert q(1000.0)[1][0] == 448.0 and q(-1e9)[1][0] == -448.0    # saturation, never NaN
    assert q(464.0)[1][0] == 448.0
    assert q(2.0 ** -10)[1][0] == 0.0                              # tie 0 / 2^-9 -> even (zero)
    assert q(1.5 * 2.0 ** -9)[1][0] == 2.0 ** -8                   # tie 2^-9 / 2^-8 -> even code 2
    assert q(float("nan"))[0][0] == 0x7F
    assert q(-0.0)[0][0] == 0x80
    # the scale divides before rounding and multiplies after
    c, v = q(6.0, 2.0)
    assert c[0] == O.quantize_e4m3(np.array([3.0]), 1.0)[0][0] and v[0] == 6.0
    assert q(0.3, 0.5)[1][0] == 0.3125                             # 0.6 -> 0.625 -> 0.3125


def test_every_code_round_trips_and_midpoints_break_to_even():
    t = O.e4m3_values()
    for code in range(256):
        if np.isnan(t[code]):
            continue
        c, v = O.quantize_e4m3(np.array([t[code]]), 1.0)
        assert v[0] == t[code] and (c[0] == code or t[code] == 0.0)
    for code in range(0, 0x7E):
        mid = (t[code] + t[code + 1]) / 2                          # exactly representable in float32
        c = O.quantize_e4m3(np.array([mid]), 1.0)[0][0]
        assert c == (code if code % 2 == 0 else code + 1)


def test_against_torch_float8_conversion():
    """Library special case: torch's float8_e4m3fn cast (round to nearest even)
    inside the finite range, where it and the saturating definition coincide."""
    g = np.random.default_rng(5)
    x = np.concatenate([g.standard_normal(4000) * 3, g.standard_normal(2000) * 100, g.uniform(-448, 448, 2000),
                        g.standard_normal(1000) * 1e-2, np.array([447.9, -447.9, 0.0, 2.0 ** -9, 2.0 ** -10 * 1.01])])
    x = x[np.abs(x) <= 448].astype(np.float32)
    for scale in (1.0, 0.37, 4.0):
        c, v = O.quantize_e4m3(x, scale)
        y = torch.from_numpy((x / np.float32(scale)).astype(np.float32))
        keep = (y.abs() <= 448).numpy()
        ref = y.to(torch.float8_e4m3fn).to(torch.float64).numpy() * float(np.float32(scale))
        assert np.array_equal(v[keep], ref[keep])
