"""Pins for the oracle's number formats and rounding (CPU only).

The oracle rounds by exhaustive search over the value grid.  Here it is checked against
things that are not itself: the closed-form value tables, an independent
"sorted midpoints" rounding routine, and torch's own float8_e4m3fn cast.
"""
import os

import numpy as np
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _e4m3_closed_form(code: int) -> float:
    s, e, m = (code >> 7) & 1, (code >> 3) & 15, code & 7
    if e == 15 and m == 7:
        return float("nan")
    v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
    return -v if s else v


def test_e2m1_table_matches_closed_form_and_fixture():
    line = [l for l in open(os.path.join(GOLDEN, "e2m1_values.txt")) if not l.startswith("#")][0]
    mags = [float(t) for t in line.split()]
    for code in range(16):
        e, m = (code & 7) >> 1, code & 1
        closed = 0.5 * m if e == 0 else (1 + m / 2.0) * 2.0 ** (e - 1)
        assert mags[code & 7] == closed
        want = -closed if code & 8 else closed
        assert oracle.e2m1_value(code) == want


def test_e4m3_table_matches_closed_form_and_torch():
    codes = torch.arange(256, dtype=torch.uint8)
    lib_vals = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for c in range(256):
        v = oracle.e4m3_value(c)
        w = _e4m3_closed_form(c)
        if np.isnan(w):
            assert c in (0x7F, 0xFF) and np.isnan(v) and np.isnan(lib_vals[c])
        else:
            assert v == w == lib_vals[c]
    assert oracle.e4m3_value(0x7E) == 448.0
    assert oracle.e4m3_value(0x01) == 2.0 ** -9
    # 126 positive finite non-zero codes
    assert sum(1 for c in range(1, 0x7F) if oracle.e4m3_value(c) > 0) == 126


def test_encode_decode_roundtrip_every_code():
    for c in range(16):
        assert oracle.e2m1_encode(oracle.e2m1_value(c)) == c or (c & 7) == 0
    # signed zeros keep their sign
    assert oracle.e2m1_encode(0.0) == 0 and oracle.e2m1_encode(-0.0) == 8
    assert oracle.e4m3_encode(0.0) == 0 and oracle.e4m3_encode(-0.0) == 0x80
    for c in range(256):
        if c in (0x7F, 0xFF):
            continue
        assert oracle.e4m3_encode(oracle.e4m3_value(c)) == c


def _round_by_midpoints(x: np.ndarray, grid: np.ndarray) -> np.ndarray:
    """Independent rounding: magnitude code = number of midpoints below |x|, a value
    exactly on a midpoint goes to the neighbour with the even code; saturating."""
    a = np.abs(x.astype(np.float64))
    mid = (grid[:-1] + grid[1:]) / 2.0
    lo = np.searchsorted(mid, a, side="left")     # midpoints strictly below a
    hi = np.searchsorted(mid, a, side="right")    # midpoints <= a
    code = np.where(lo == hi, lo, np.where(lo % 2 == 0, lo, hi))
    return code.astype(np.int64)


def _all_finite_bf16() -> np.ndarray:
    bits = np.arange(65536, dtype=np.uint32)
    f = (bits << 16).view(np.float32)
    return f[np.isfinite(f)]


def test_e2m1_rounding_exhaustive_vs_midpoints():
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], np.float64)
    x = _all_finite_bf16()
    for scale in (1.0, 0.75, 3.0, 1.0 / 3.0):
        xs = (x * np.float32(scale)).astype(np.float32)
        want = _round_by_midpoints(xs, grid) | (np.signbit(xs).astype(np.int64) << 3)
        got = np.array([oracle.e2m1_encode(float(v)) for v in xs])
        assert np.array_equal(got, want)
    # every midpoint goes to the even code, above the maximum saturates
    for lo in range(7):
        mid = (grid[lo] + grid[lo + 1]) / 2
        assert oracle.e2m1_encode(mid) == (lo if lo % 2 == 0 else lo + 1)
    assert oracle.e2m1_encode(1e9) == 7 and oracle.e2m1_encode(-1e9) == 15


def test_e4m3_rounding_exhaustive_vs_midpoints_and_torch():
    grid = np.array([_e4m3_closed_form(c) for c in range(0x7F)], np.float64)
    x = _all_finite_bf16()
    for scale in (1.0, 1.0 / 7.0, 5.0):
        xs = (x * np.float32(scale)).astype(np.float32)
        xs = xs[np.isfinite(xs)]
        want = _round_by_midpoints(xs, grid) | (np.signbit(xs).astype(np.int64) << 7)
        got = np.array([oracle.e4m3_encode(float(v)) for v in xs])
        assert np.array_equal(got, want)
        # library special case: inside the finite range torch's cast is the same rounding
        inr = np.abs(xs) <= 448.0
        tcast = torch.from_numpy(xs[inr]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        assert np.array_equal(got[inr], tcast.astype(np.int64))
    for lo in range(0x7E):
        mid = (grid[lo] + grid[lo + 1]) / 2
        assert oracle.e4m3_encode(mid) == (lo if lo % 2 == 0 else lo + 1)
    assert oracle.e4m3_encode(1e9) == 0x7E and oracle.e4m3_encode(-1e9) == 0xFE
    assert oracle.e4m3_encode(449.0) == 0x7E and oracle.e4m3_encode(464.0) == 0x7E
