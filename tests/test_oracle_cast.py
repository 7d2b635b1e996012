"""Pins for the oracle's fp32 -> bf16 cast (D5): the hand table, an exhaustive sweep against a
definition by exact arithmetic, torch's CPU conversion, monotonicity and the half-ulp bound."""
import numpy as np
import torch

import oracle


def _exact_value(bits):
    """Exact real value of fp32 patterns as float64; an all-ones exponent with zero mantissa is read
    as 2**128, the value the format's next binade would start at (what rounding measures against)."""
    bits = bits.astype(np.uint64)
    e = ((bits >> 23) & 0xFF).astype(np.int64)
    m = (bits & 0x7FFFFF).astype(np.float64)
    sub = e == 0
    mag = np.where(sub, np.ldexp(m, -149), np.ldexp(m + 8388608.0, (e - 150).astype(np.int32)))
    return np.where((bits >> 31) & 1 == 1, -mag, mag)


def _nearest_even_definition(u):
    """Independent statement: the two bf16 neighbours of x are lo = u with the low half cleared and
    hi = lo + one unit in bit 16; take the nearer in exact arithmetic, the one with an even bit 16 on
    a tie.  Non-NaN inputs only."""
    u = u.astype(np.uint64)
    lo = u & 0xFFFF0000
    hi = lo + 0x10000
    x, vlo, vhi = _exact_value(u), _exact_value(lo), _exact_value(hi & 0xFFFFFFFF)
    dlo, dhi = np.abs(x - vlo), np.abs(vhi - x)
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (((lo >> 16) & 1) == 1))
    return (np.where(pick_hi, hi, lo) >> 16).astype(np.uint16)


def test_hand_table(golden):
    rows = golden("cast_rne.txt")
    assert len(rows) >= 20
    for r in rows:
        assert oracle.cast_bf16(int(r[0], 16)) == int(r[1], 16), r


def test_exhaustive_high_halves_against_exact_definition():
    highs = np.arange(1 << 16, dtype=np.uint32) << 16
    for low in (0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF):
        u = highs | np.uint32(low)
        nan = (u & 0x7FFFFFFF) > 0x7F800000
        got = oracle.cast_bf16_array(u)
        want = _nearest_even_definition(u[~nan])
        assert np.array_equal(got[~nan], want)
        assert (got[nan] == 0x7FFF).all()


def test_random_patterns_against_torch_cpu():
    rng = np.random.default_rng(7)
    u = rng.integers(0, 1 << 32, size=300_000, dtype=np.uint64).astype(np.uint32)
    u[:100_000] = (u[:100_000] & 0xFFFF0000) | 0x8000  # forced ties
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    t = torch.from_numpy(u.view(np.float32).copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.cast_bf16_array(u)
    assert np.array_equal(got[~nan], t[~nan])
    tn = t[nan]
    assert (((tn & 0x7F80) == 0x7F80) & ((tn & 0x7F) != 0)).all()  # torch also yields a NaN there


def test_monotone_and_half_ulp_bound():
    rng = np.random.default_rng(11)
    u = np.sort(rng.integers(0, 0x7F800000, size=200_000, dtype=np.uint64).astype(np.uint32))
    b = oracle.cast_bf16_array(u)
    assert (np.diff(b.astype(np.int64)) >= 0).all()  # positive patterns order like their values
    normal = (u >= 0x00800000) & (u < 0x7F7F8000)
    x = _exact_value(u[normal])
    back = _exact_value(b[normal].astype(np.uint32) << 16)
    e = np.floor(np.log2(x))
    assert (np.abs(x - back) <= np.ldexp(1.0, (e - 8).astype(np.int32))).all()


def test_widen_is_exact_and_cast_is_its_left_inverse():
    b = np.arange(1 << 16, dtype=np.uint32)
    nan = ((b & 0x7F80) == 0x7F80) & ((b & 0x7F) != 0)
    for x in b[~nan][::37]:
        w = oracle.widen_bf16(int(x))
        assert w == int(x) << 16
        assert oracle.cast_bf16(w) == int(x)
