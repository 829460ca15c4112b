"""Pins for the oracle's number formats: every encoder is checked against the
definition of round-to-nearest-even (brute force over all representable values),
not against a second copy of its own formula."""
import math

import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc

# value tables written from the format definitions (Section 2.1: E2M1 max 6; E4M3 max normal 448)
E2M1_MAG = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def e4m3_value(code: int) -> float:
    s, e, m = code >> 7, (code >> 3) & 15, code & 7
    v = m * 2.0 ** -9 if e == 0 else (1 + m / 8) * 2.0 ** (e - 7)
    return -v if s else v


def brute_nearest(a: float, grid):
    """Index of the grid value nearest to a >= 0; ties go to the even index; saturating."""
    best, best_d = None, None
    for i, g in enumerate(grid):
        d = abs(a - g)
        if best is None or d < best_d or (d == best_d and i % 2 == 0):
            best, best_d = i, d
    return best


def f32(x):
    return float(np.float32(x))


def test_e4m3_decode_all_codes():
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue  # NaN pattern, never produced
        assert orc.e4m3_decode(c) == e4m3_value(c)
    assert orc.e4m3_decode(0x7E) == 448.0
    assert orc.e4m3_decode(0x38) == 1.0
    assert orc.e4m3_decode(0x01) == 2.0 ** -9


def test_e4m3_roundtrip_all_codes():
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue
        assert orc.e4m3_encode(e4m3_value(c)) == c


def test_e4m3_known_codes():
    known = {1.0: 0x38, 0.5: 0x30, 448.0: 0x7E, 2.0 ** -6: 0x08, 2.0 ** -9: 0x01, 432.0: 0x7E, 431.9: 0x7D,
             1000.0: 0x7E, 2.0 ** -10: 0x00, 2.0 ** -10 * 1.01: 0x01, 0.0: 0x00}
    for x, c in known.items():
        assert orc.e4m3_encode(x) == c, x
        assert orc.e4m3_encode(-x) == (c | 0x80), x


def test_e4m3_encode_bruteforce_sweep():
    grid = [e4m3_value(c) for c in range(127)]  # nonnegative finite values, ascending with the code
    assert grid == sorted(grid)
    pts = []
    for i in range(126):
        lo, hi = grid[i], grid[i + 1]
        mid = (lo + hi) / 2
        for x in (lo, mid, hi, lo + (hi - lo) * 0.3, lo + (hi - lo) * 0.7):
            x = f32(x)
            pts += [x, float(np.nextafter(np.float32(x), np.float32(np.inf))),
                    float(np.nextafter(np.float32(x), np.float32(-np.inf)))]
    rng = np.random.default_rng(0)
    pts += [f32(v) for v in np.abs(rng.standard_normal(4000)) * 50]
    pts += [f32(v) for v in np.abs(rng.standard_normal(2000)) * 0.01]
    pts += [449.0, 463.9, 464.0, 480.0, 1e6, 1e30]
    for x in pts:
        if x < 0:
            continue
        assert orc.e4m3_encode(x) == brute_nearest(x, grid), x
        assert orc.e4m3_encode(-x) == brute_nearest(x, grid) | 0x80


def test_e4m3_matches_torch_cast_in_range():
    # library routine: torch's float8_e4m3fn cast is round-to-nearest-even inside the finite range
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * 3, rng.standard_normal(5000) * 0.02,
                        rng.uniform(-440, 440, 5000)]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([orc.e4m3_encode(float(v)) for v in x], np.uint8)
    # torch keeps the sign of a value that rounds to zero, as the oracle does
    assert np.array_equal(got, ref)


def test_e2m1_decode_and_roundtrip():
    for c in range(16):
        v = E2M1_MAG[c & 7] * (-1 if c & 8 else 1)
        assert orc.e2m1_decode(c) == v
        if c != 8:
            assert orc.e2m1_encode(v) == c
    assert orc.e2m1_encode(-0.0) == 8
    assert orc.e2m1_encode(-0.1) == 8  # sign survives rounding to zero


def test_e2m1_tie_table():
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for x, v in ties.items():
        assert orc.e2m1_decode(orc.e2m1_encode(x)) == v, x
        assert orc.e2m1_decode(orc.e2m1_encode(-x)) == -v, x
    assert orc.e2m1_decode(orc.e2m1_encode(7.0)) == 6.0
    assert orc.e2m1_decode(orc.e2m1_encode(1e9)) == 6.0


def test_e2m1_encode_bruteforce_sweep():
    pts = []
    for i in range(7):
        lo, hi = E2M1_MAG[i], E2M1_MAG[i + 1]
        for x in (lo, (lo + hi) / 2, hi, lo + 0.3 * (hi - lo), lo + 0.71 * (hi - lo)):
            x = f32(x)
            pts += [x, float(np.nextafter(np.float32(x), np.float32(np.inf))),
                    float(np.nextafter(np.float32(x), np.float32(-np.inf)))]
    rng = np.random.default_rng(2)
    pts += [f32(v) for v in np.abs(rng.standard_normal(5000)) * 3]
    pts += [6.5, 100.0]
    for x in pts:
        if x < 0:
            continue
        assert orc.e2m1_encode(x) == brute_nearest(x, E2M1_MAG), x
        assert orc.e2m1_encode(-x) == brute_nearest(x, E2M1_MAG) | 8


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000), rng.standard_normal(2000) * 1e-3,
                        np.array([1.00390625, 1.01171875, 0.0, -0.0, 3.0])]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.uint16).numpy()
    got = np.array([orc.f32_to_bf16(float(v)) for v in x], np.uint16)
    assert np.array_equal(got, ref)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: even mantissa wins
    assert orc.f32_to_bf16(1.00390625) == 0x3F80
    assert orc.f32_to_bf16(1.01171875) == 0x3F82
