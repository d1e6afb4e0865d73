"""Pins of the oracle's quantization mappings and nearest-entry rule (CPU only).

Each test ties the oracle to something other than itself: constants the paper prints, tables
worked by hand from App. E.2, exact rational arithmetic, or brute force.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import lpmm_oracle_np as onp
from conftest import read_golden

CONST = read_golden("paper_constants.txt")
TABLES = read_golden("de_tables_4bit.txt")


def _frac_list(key):
    return [Fraction(s) for s in TABLES[key]]


@pytest.mark.parametrize("impl", [oracle, onp])
def test_linear_map_closed_form_and_printed_minimum(impl):
    T = impl.linear_map(4)
    assert len(T) == int(CONST["entries_4bit"][0])
    assert [Fraction(float(t)) for t in T] == [Fraction(i + 1, 16) for i in range(16)]
    assert float(T.min()) == float(CONST["linear_smallest"][0])      # Sec. 4.1 prints 0.0625
    assert not np.any(T == 0)                                         # zero is excluded
    T3 = impl.linear_map(3)
    assert [Fraction(float(t)) for t in T3] == [Fraction(i + 1, 8) for i in range(8)]


@pytest.mark.parametrize("impl", [oracle, onp])
def test_de0_smallest_matches_printed_value(impl):
    T = impl.de_map(4, False, True)      # unsigned, zero removed: the DE-0 variant of Sec. 4.1
    assert len(T) == 15
    assert round(float(T.min()), 4) == float(CONST["de0_smallest_4dp"][0])
    # without the 0...01 -> 1 corner case the smallest entry would be 0.00055, not 0.0033
    assert float(T.min()) > 0.003


@pytest.mark.parametrize("impl", [oracle, onp])
def test_de_fraction_cells(impl):
    lo, hi = float(CONST["fraction_lo"][0]), float(CONST["fraction_hi"][0])
    for F in range(0, 7):
        fr = [Fraction(impl.de_fraction(F, k)).limit_denominator(10 ** 9) for k in range(2 ** F)]
        assert all(lo <= f <= hi for f in fr)
        width = Fraction(9, 10) / 2 ** F
        for k, f in enumerate(fr):   # midpoint of the k-th of 2^F equal cells of [0.1, 1]
            assert f == Fraction(1, 10) + width * k + width / 2


@pytest.mark.parametrize("impl", [oracle, onp])
def test_signed_de_table_against_hand_worked_fractions(impl):
    T = impl.de_map(4, True, False)
    want = _frac_list("signed")
    assert len(T) == 16 and len(want) == 16
    assert np.all(np.diff(T) > 0)                                     # sorted, increasing, distinct
    for t, f in zip(T, want):
        assert np.float32(float(f)) == t                             # rational rounded to binary32
    vals = set(float(t) for t in T)
    for s in CONST["signed_has"]:
        assert float(s) in vals
    for s in CONST["signed_lacks"]:
        assert float(s) not in vals
    pos = sorted(t for t in T if t > 0 and t != 1.0)
    neg = sorted(-t for t in T if t < 0)
    assert pos == neg and len(pos) == 7                               # mirror image except +1


@pytest.mark.parametrize("impl", [oracle, onp])
def test_unsigned_de_table_against_hand_worked_fractions(impl):
    T = impl.de_map(4, False, False)
    want = _frac_list("unsigned")
    assert len(T) == 16
    for t, f in zip(T, want):
        assert np.float32(float(f)) == t


@pytest.mark.parametrize("impl", [oracle, onp])
def test_de_8bit_structure(impl):
    # b = 8 signed (the 8-bit optimizer's map): 256 entries, contains 0 and +1, lacks -1, and
    # for each exponent E there are 2^(6-E) magnitudes in [0.1, 1] * 10^-E.
    T = impl.de_map(8, True, False)
    assert len(T) == 256 and np.all(np.diff(T) > 0)
    assert 0.0 in T and 1.0 in T and -1.0 not in T
    mags = np.array(sorted(t for t in T if 0 < t < 1.0), dtype=np.float64)
    for E in range(7):
        lo, hi = 0.1 * 10.0 ** -E, 1.0 * 10.0 ** -E
        assert np.sum((mags > lo) & (mags < hi)) == 2 ** (6 - E)


def _exact_nearest(T, x):
    best, bd = 0, abs(Fraction(float(x)) - Fraction(float(T[0])))
    for i in range(1, len(T)):
        d = abs(Fraction(float(x)) - Fraction(float(T[i])))
        if d < bd:
            best, bd = i, d
    return best


def _probe_points(T):
    pts = [np.float32(v) for v in (-2.0, -1.0, -0.0, 0.0, 1.0, 1.5, 1e-30, -1e-30, 1e-45)]
    for a, b in zip(T[:-1], T[1:]):
        mid = np.float32((float(a) + float(b)) / 2)
        p = mid
        for _ in range(6):
            p = np.nextafter(p, np.float32(-np.inf), dtype=np.float32)
        for _ in range(13):
            pts.append(np.float32(p))
            p = np.nextafter(p, np.float32(np.inf), dtype=np.float32)
    pts += list(T)
    rng = np.random.default_rng(5)
    pts += list(rng.uniform(-1.1, 1.1, 500).astype(np.float32))
    return np.array(pts, dtype=np.float32)


@pytest.mark.parametrize("which", ["de_signed", "linear", "de_unsigned"])
def test_nearest_is_exact_argmin_with_first_minimiser(which):
    T = {"de_signed": oracle.de_map(4, True), "linear": oracle.linear_map(4),
         "de_unsigned": oracle.de_map(4, False)}[which]
    pts = _probe_points(T)
    want = np.array([_exact_nearest(T, x) for x in pts], dtype=np.uint8)
    got_c = np.array([oracle.nearest(T, x) for x in pts], dtype=np.uint8)
    got_np = onp.nearest(T, pts)
    assert np.array_equal(got_c, want)
    assert np.array_equal(got_np, want)


def test_nearest_tie_goes_to_lower_index():
    T = oracle.linear_map(4)
    for i in range(15):
        mid = np.float32((2 * i + 3) / 32.0)       # exactly representable midpoint of T[i], T[i+1]
        assert oracle.nearest(T, mid) == i
        assert oracle.nearest(T, np.nextafter(mid, np.float32(2), dtype=np.float32)) == i + 1
    assert oracle.nearest(T, 0.0) == 0 and oracle.nearest(T, -5.0) == 0 and oracle.nearest(T, 7.0) == 15


def test_reciprocal_rule():
    tiny = float(np.finfo(np.float32).tiny)
    assert oracle.rcp(0.0) == 0.0
    assert oracle.rcp(tiny / 2) == 0.0                                 # denormal scale counts as zero
    assert oracle.rcp(tiny) == float(np.float32(1.0) / np.float32(tiny))
    assert oracle.rcp(3.0) == float(np.float32(1.0) / np.float32(3.0))
    s = np.array([0.0, tiny / 2, tiny, 3.0, 1e30], np.float32)
    assert np.array_equal(onp.rcp(s), np.array([oracle.rcp(float(x)) for x in s], np.float32))


def test_bf16_rounding_is_nearest_even():
    # worked cases: exact values, ties to even in both directions, just off a tie, binade and infinity carries, zeros
    cases = [(0x3F800000, 0x3F80), (0x3F808000, 0x3F80), (0x3F818000, 0x3F82), (0x3F808001, 0x3F81), (0x3F807FFF, 0x3F80),
             (0x3FFF8000, 0x4000), (0x7F7FFFFF, 0x7F80), (0x7F800000, 0x7F80), (0x80000000, 0x8000), (0x00000000, 0x0000),
             (0x00008000, 0x0000), (0x00018000, 0x0002), (0xBF818000, 0xBF82), (0x7FC00001, 0x7FFF), (0xFF800001, 0x7FFF)]
    x = np.array([c[0] for c in cases], np.uint32).view(np.float32)
    assert list(oracle.f32_to_bf16_bits(x)) == [c[1] for c in cases]
    # a library routine on random data (finite values of every magnitude)
    import torch
    rng = np.random.default_rng(0)
    r = (rng.standard_normal(200000) * np.exp(rng.uniform(-80, 80, 200000))).astype(np.float32)
    want = torch.from_numpy(r).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16_bits(r), want)
    # and it inverts the exact widening
    back = oracle.bf16_bits_to_f32(want)
    assert np.array_equal(oracle.f32_to_bf16_bits(back), want)
