"""Brute force over all 65536 bf16 bit patterns: the integer facts the bf16 top-k / top-p kernel
relies on when it counts logits per exact value (a restatement in numpy, not the kernel's code).

* the 16-bit order key (sign set: all bits flipped; sign clear: sign bit set) sorts bf16 values in
  IEEE total order, so "key >= T" is "value >= threshold" with -0 < +0;
* two keys packed in one 32-bit word can be subtracted from a packed reference in one operation as
  long as the reference is at or above both: no half borrows from the other;
* the keys from 16 down through zero to -16 are fewer than the 35840 counters of the histogram, and
  a reference one step above the row maximum reaches values far below any logit that carries mass.
"""
import numpy as np

BITS = np.arange(65536, dtype=np.uint32)
VALS = (BITS << 16).astype(np.uint32).view(np.float32)
FINITE_OR_INF = ~np.isnan(VALS)
VALS64 = np.where(FINITE_OR_INF, VALS, 0).astype(np.float64)     # NaN patterns are masked out wherever values are used
COUNTERS = 35840


def key16(bits):
    bits = bits.astype(np.uint32)
    return np.where(bits & 0x8000, ~bits & 0xFFFF, bits | 0x8000).astype(np.uint32)


def test_key_order_is_the_total_order_of_the_values():
    k = key16(BITS)
    assert len(np.unique(k)) == 65536                      # a bijection
    sel = np.flatnonzero(FINITE_OR_INF)
    order = np.argsort(k[sel], kind="stable")
    v = VALS64[sel][order]
    assert np.all(np.diff(v) >= 0)                          # ascending keys = ascending values
    # the only equal neighbours are -0 and +0, in that order
    eq = np.flatnonzero(np.diff(v) == 0)
    assert len(eq) == 1
    b = BITS[sel][order]
    assert b[eq[0]] == 0x8000 and b[eq[0] + 1] == 0x0000


def test_keys_from_a_packed_word_by_sign_spreading():
    # sign of each half spread over the half, or-ed with the sign bits, xor-ed onto the word
    rng = np.random.default_rng(7)
    lo = rng.integers(0, 65536, 200000, dtype=np.uint32)
    hi = rng.integers(0, 65536, 200000, dtype=np.uint32)
    w = (hi << 16) | lo
    spread = np.where(lo & 0x8000, 0xFFFF, 0).astype(np.uint32) | (np.where(hi & 0x8000, 0xFFFF, 0).astype(np.uint32) << 16)
    k2 = w ^ (spread | 0x80008000)
    assert np.array_equal(k2 & 0xFFFF, key16(lo))
    assert np.array_equal(k2 >> 16, key16(hi))


def test_packed_subtraction_needs_no_borrow_below_the_reference():
    rng = np.random.default_rng(8)
    ref = rng.integers(1, 65536, 200000, dtype=np.uint32)
    a = (rng.random(200000) * (ref + 1)).astype(np.uint32)          # keys <= ref
    b = (rng.random(200000) * (ref + 1)).astype(np.uint32)
    d2 = (ref * 0x10001 - ((b << 16) | a)) & 0xFFFFFFFF
    assert np.array_equal(d2 & 0xFFFF, ref - a)
    assert np.array_equal(d2 >> 16, ref - b)


def test_the_counters_reach_far_below_any_logit_with_mass():
    k = key16(BITS).astype(np.int64)
    v = VALS64
    finite = np.isfinite(VALS)
    between = finite & (v >= -16.0) & (v <= 16.0)
    assert between.sum() < COUNTERS                                   # 33.5 k keys from -16 to 16
    # a row maximum anywhere from 1e-3 to 1e4: the lowest value inside the counters lies more than
    # ten thousand logit units under the maximum (mass 2^-44 is reached after 31 at temperature 1)
    for mx in (1e-3, 0.5, 13.0, 100.0, 1e4):
        top = k[finite & (v <= mx)].max() + 1                          # reference: one step above the maximum's key
        lowest_key = top - (COUNTERS - 1)
        lowest_val = v[finite][np.argmin(np.abs(k[finite] - lowest_key))]
        assert lowest_val < mx - 1e4
    # an all-negative row: the counters reach the bottom of the format
    top = k[finite & (v <= -1e-3)].max() + 1
    assert top - (COUNTERS - 1) <= k[finite].min()
