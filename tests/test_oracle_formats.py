"""Pins for the oracle's number formats (Section 2 ExMy formats; Section 3 cast FP4 -> FP8).

Nothing here re-types the oracle's rounding formula: values come from hand-typed tables of the
format definitions (tests/golden), from torch's own float8_e4m3fn conversion, or from a brute-force
nearest-value search over a decoded table.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                out.append(line.split())
    return out


E2M1_TABLE = [(int(c, 2), float(v)) for c, v in _rows("e2m1_codes.txt")]


def test_e2m1_all_16_codes_decode():
    assert len(E2M1_TABLE) == 16
    for code, val in E2M1_TABLE:
        got = oracle.e2m1_decode(code)
        assert got == val and math.copysign(1, got) == math.copysign(1, val), (code, got, val)
    mags = sorted({abs(v) for _, v in E2M1_TABLE})
    assert mags == [0, 0.5, 1, 1.5, 2, 3, 4, 6]


def test_e2m1_encode_is_inverse_on_all_codes():
    for code, val in E2M1_TABLE:
        assert oracle.e2m1_encode(val) == code  # -0.0 keeps its sign bit: code 0b1000


def test_e2m1_rounding_table():
    for s_in, s_out in _rows("e2m1_rounding.txt"):
        v, want = float(s_in), float(s_out)
        assert oracle.e2m1_decode(oracle.e2m1_encode(v)) == want, (v, want)
        assert oracle.e2m1_decode(oracle.e2m1_encode(-v)) == -want, (v, want)
        assert oracle.e2m1_encode(-v) == (oracle.e2m1_encode(v) | 0x8)


def _nearest_even(v, table):
    """Brute force: nearest magnitude of `table` [(code, value)...]; ties -> even code; saturating."""
    a = abs(v)
    best = None
    for code, val in table:
        d = abs(a - val)
        if best is None or d < best[0] or (d == best[0] and code % 2 == 0 and best[1] % 2 == 1):
            best = (d, code)
    return best[1]


def test_e2m1_encode_brute_force_and_monotone():
    pos = [(c, v) for c, v in E2M1_TABLE if c < 8]
    xs = np.concatenate([np.linspace(-8, 8, 6401), np.random.default_rng(0).normal(0, 2.5, 4000)]).astype(np.float32)
    prev = None
    for v in np.sort(xs):
        code = oracle.e2m1_encode(float(v))
        want = _nearest_even(float(v), pos) | (0x8 if np.signbit(v) else 0)
        assert code == want, (v, code, want)
        val = oracle.e2m1_decode(code)
        if prev is not None:
            assert val >= prev
        prev = val


def test_e4m3_landmarks_and_torch_decode():
    for c, v in _rows("e4m3_landmarks.txt"):
        got = oracle.e4m3_decode(int(c, 16))
        assert got == float(v) and math.copysign(1, got) == math.copysign(1, float(v)), (c, got, v)
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for c in range(256):
        got = oracle.e4m3_decode(c)
        if c in (0x7F, 0xFF):
            assert math.isnan(got) and math.isnan(ref[c])
        else:
            assert got == ref[c], (c, got, ref[c])
    assert oracle.e4m3_decode(0x7E) == 448.0  # the largest finite value


def test_e4m3_rounding_table_and_saturation():
    for s_in, s_code in _rows("e4m3_rounding.txt"):
        assert oracle.e4m3_encode(float(s_in)) == int(s_code, 16), (s_in, s_code)
    assert oracle.e4m3_encode(float("nan")) & 0x7F == 0x7F


def test_e4m3_idempotent_on_all_codes():
    for c in range(256):
        if c & 0x7F == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) == c


def test_e4m3_encode_matches_torch_for_every_bf16_input():
    bits = np.arange(65536, dtype=np.uint32)
    x = (bits << 16).astype(np.uint32).view(np.float32)
    for scale in (1.0, 0.37, 3.0, 448.0 / 20.5, 1.0 / 1024):
        v = (x * np.float32(scale)).astype(np.float32)
        ok = np.isfinite(v) & (np.abs(v) <= 448.0)
        vv = v[ok]
        ref = torch.from_numpy(vv.copy()).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        got = np.array([oracle.e4m3_encode(float(t)) for t in vv], dtype=np.uint8)
        bad = np.nonzero(got != ref)[0]
        assert bad.size == 0, (scale, vv[bad[:5]], got[bad[:5]], ref[bad[:5]])
        # above the range everything saturates to the largest finite code, sign kept
        big = v[np.isfinite(v) & (np.abs(v) > 448.0)][::97]
        for t in big:
            assert oracle.e4m3_encode(float(t)) == (0xFE if t < 0 else 0x7E)


def test_e4m3_encode_brute_force_nearest():
    table = [(c, oracle.e4m3_decode(c)) for c in range(0x7F)]  # decode is pinned above
    rng = np.random.default_rng(1)
    xs = np.concatenate([rng.normal(0, 30, 1500), rng.normal(0, 0.01, 1500), rng.uniform(-460, 460, 1500)])
    for v in xs.astype(np.float32):
        want = _nearest_even(float(v), table) | (0x80 if np.signbit(v) else 0)
        assert oracle.e4m3_encode(float(v)) == want, v


def test_shift_is_multiply_exactly():
    """Section 3, 'Casting the FP4 to FP8': with power-of-two scale ratios the cast is a shift."""
    for code in range(16):
        for d in range(0, 6):
            w8 = oracle.widen(code, d)
            assert oracle.e4m3_decode(w8) == oracle.e2m1_decode(code) * 2.0 ** -d, (code, d)
            if code & 7:  # non-zero magnitude: the shift only lowers the exponent field
                assert w8 == oracle.widen(code, 0) - (d << 3)
                assert (w8 >> 3) & 0xF >= 1, "stays a normal number"
            else:
                assert w8 == (0x80 if code & 8 else 0)
    # one more step would leave the normal range for the smallest non-zero magnitude
    assert (oracle.widen(1, 6) >> 3) & 0xF == 0
    # the unshifted cast keeps sign, and maps the 8 magnitudes onto E4M3 codes of equal value
    for code, val in E2M1_TABLE:
        assert oracle.e4m3_decode(oracle.widen(code, 0)) == val
