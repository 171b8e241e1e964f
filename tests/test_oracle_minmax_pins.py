"""Pins of the CPU checker's (min, max) nearest-rounding codec variant against things other than
itself: exact rational arithmetic, closed forms on dyadic grids, the defining properties of a
uniform nearest-level quantizer (error bound, monotonicity, end points, best neighbour), Python
big-integer packing, and numpy for ranges and sums.  Everything here runs on the CPU."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import mqg_oracle as O

ALL_BITS = list(range(1, 9))


def _rng(seed):
    return np.random.default_rng(seed)


def _quant(x, bits, bucket):
    codes, ranges = O.quantize_minmax(x, bits, bucket)
    q = O.unpack(codes, x.size, bits)
    return codes, ranges, q


# ------------------------------------------------------------------ ranges
@pytest.mark.parametrize("n,bucket", [(1, 4), (7, 4), (1000, 256), (513, 512), (64, 64)])
def test_ranges_are_numpy_min_and_max_per_bucket(n, bucket):
    x = _rng(n).standard_normal(n).astype(np.float32)
    r = O.bucket_ranges(x, bucket)
    nb = (n + bucket - 1) // bucket
    assert r.size == 2 * nb
    for k in range(nb):
        part = x[k * bucket:(k + 1) * bucket]          # the last bucket is simply shorter
        assert r[2 * k] == part.min() and r[2 * k + 1] == part.max()


def test_zero_of_either_sign_is_stored_as_plus_zero():
    x = np.array([-0.0, 0.0, -0.0, -0.0], np.float32)
    r = O.bucket_ranges(x, 4)
    assert r.view(np.uint32).tolist() == [0, 0]
    x = np.array([-0.0, -1.0, -0.0, -2.0], np.float32)      # hi is a negative zero
    r = O.bucket_ranges(x, 4)
    assert r[0] == -2.0 and r.view(np.uint32)[1] == 0


# ------------------------------------------------------------------ closed forms
@pytest.mark.parametrize("bits", ALL_BITS)
def test_values_on_a_dyadic_grid_are_coded_and_restored_exactly(bits):
    L = (1 << bits) - 1
    lo, step = np.float32(-4.0), np.float32(2.0 ** -3)
    j = _rng(bits).permutation(np.concatenate([np.arange(L + 1), np.arange(L + 1)]))
    x = (lo + j.astype(np.float32) * step).astype(np.float32)     # exact: small integers times 2^-3
    # hi - lo = L * step is exact, L / (L * step) = 8 is exact, so t = j + 1/2 exactly
    _, ranges, q = _quant(x, bits, x.size)
    assert ranges.tolist() == [float(lo), float(lo + L * step)]
    assert np.array_equal(q, j.astype(np.uint8))
    assert np.array_equal(O.dequantize_minmax(q, bits, x.size, ranges), x)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_end_points(bits):
    L = (1 << bits) - 1
    x = _rng(10 + bits).standard_normal(512).astype(np.float32) * np.float32(1e-3)
    _, ranges, q = _quant(x, bits, 512)
    lo, hi = ranges
    assert q[np.argmin(x)] == 0 and q[np.argmax(x)] == L
    xhat = O.dequantize_minmax(q, bits, 512, ranges)
    assert xhat[np.argmin(x)] == lo                                   # fma(0, step, lo) = lo, bit for bit
    assert abs(float(xhat[np.argmax(x)]) - float(hi)) <= 2.0 ** -21 * (float(hi) - float(lo))


@pytest.mark.parametrize("bits", [1, 3, 8])
def test_constant_and_nearly_constant_buckets(bits):
    for c in (np.float32(0.37), np.float32(-1e-20), np.float32(0.0)):
        x = np.full(100, c, np.float32)
        codes, ranges, q = _quant(x, bits, 64)
        assert not q.any() and not codes.any()
        assert np.array_equal(O.dequantize_minmax(q, bits, 64, ranges), x)
    # a spread below 2^-96 counts as constant: every element decodes to lo
    x = np.array([1e-30, 1.5e-30, 1.2e-30, 1e-30], np.float32)
    assert float(x.max()) - float(x.min()) < 2.0 ** -96
    _, ranges, q = _quant(x, bits, 4)
    assert not q.any()
    assert np.array_equal(O.dequantize_minmax(q, bits, 4, ranges), np.full(4, x.min(), np.float32))
    # just above the threshold the bucket is coded normally
    x = np.array([0.0, 2.0 ** -95], np.float32)
    _, ranges, q = _quant(x, bits, 2)
    assert q.tolist() == [0, (1 << bits) - 1]


# ------------------------------------------------------------------ properties of nearest rounding
@pytest.mark.parametrize("bits", ALL_BITS)
def test_error_is_at_most_half_a_step_and_no_neighbour_is_closer(bits):
    L = (1 << bits) - 1
    n, bucket = 4096, 512
    x = (_rng(20 + bits).standard_normal(n) * 3e-4).astype(np.float32)
    _, ranges, q = _quant(x, bits, bucket)
    xhat = O.dequantize_minmax(q, bits, bucket, ranges).astype(np.float64)
    lo = np.repeat(ranges[0::2].astype(np.float64), bucket)[:n]
    hi = np.repeat(ranges[1::2].astype(np.float64), bucket)[:n]
    step = (hi - lo) / L
    err = np.abs(xhat - x.astype(np.float64))
    assert (err <= 0.5 * step * (1 + 2.0 ** -18)).all()
    # the chosen level is the best one: its neighbours are not closer (up to fp32 rounding of the grid)
    qf = q.astype(np.float64)
    for dq in (-1.0, 1.0):
        ok = (qf + dq >= 0) & (qf + dq <= L)
        other = np.abs(lo + (qf + dq) * step - x.astype(np.float64))
        assert (err[ok] <= other[ok] + step[ok] * 2.0 ** -18).all()
    assert q.max() <= L


@pytest.mark.parametrize("bits", [1, 2, 5, 8])
def test_codes_are_monotone_in_the_value(bits):
    x = np.sort((_rng(30 + bits).standard_normal(2000) * 0.01).astype(np.float32))
    _, _, q = _quant(x, bits, x.size)
    assert (np.diff(q.astype(np.int32)) >= 0).all()
    assert q[0] == 0 and q[-1] == (1 << bits) - 1


@pytest.mark.parametrize("bits", ALL_BITS)
def test_against_exact_rational_arithmetic_on_small_buckets(bits):
    """The ideal code is floor((x - lo) L / (hi - lo) + 1/2) over the rationals; the fp32 pipeline
    (three roundings before the floor) may only differ when the exact value sits within 2^-19 L of
    a half-integer boundary."""
    L = (1 << bits) - 1
    rng = _rng(40 + bits)
    checked = agree = 0
    for trial in range(60):
        n = int(rng.integers(2, 17))
        x = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 2)).astype(np.float32)
        _, ranges, q = _quant(x, bits, n)
        lo, hi = Fraction(float(ranges[0])), Fraction(float(ranges[1]))
        if hi == lo:
            continue
        for xi, qi in zip(x, q):
            t = (Fraction(float(xi)) - lo) * L / (hi - lo) + Fraction(1, 2)
            ideal = min(L, int(t // 1))
            checked += 1
            if int(qi) == ideal:
                agree += 1
            else:
                frac = t - (t // 1)
                dist = min(frac, 1 - frac)                # distance of t to the nearest integer
                assert abs(int(qi) - ideal) == 1 and dist < Fraction(L, 1 << 19), (xi, qi, ideal)
    assert checked > 300 and agree >= checked - 3


def _nearest_f32(t):
    """The float32 nearest to the rational t (ties to even), by exact comparison."""
    c = np.float32(float(t))
    cands = [c, np.nextafter(c, np.float32(-np.inf)), np.nextafter(c, np.float32(np.inf))]
    best = min(cands, key=lambda v: (abs(Fraction(float(v)) - t), int(v.view(np.uint32)) & 1))
    return best


# (bits, hi, x): buckets [0, hi, x] where rounding the product d * inv before adding 1/2 gives code 1
# but the single rounding of the fused multiply-add gives code 0 (found by a search over random
# ranges for products just below 1/2 - 2^-25)
FUSED_CASES = [
    (6, 1.0539307594299316, 0.008364529348909855),
    (3, 1.6523691415786743, 0.11802636086940765),
    (8, 1.2345101833343506, 0.002420607954263687),
    (5, 1.8976776599884033, 0.03060770221054554),
    (6, 1.060802698135376, 0.008419068530201912),
    (8, 1.8796511888504028, 0.0036855903454124928),
]


@pytest.mark.parametrize("bits,hi,xv", FUSED_CASES)
def test_scaled_offset_is_rounded_once(bits, hi, xv):
    """t = d * inv + 1/2 is rounded once (a fused multiply-add): the expected code comes from exact
    rational arithmetic followed by one rounding to float32; rounding the product first would
    give the other code on these inputs."""
    f32 = np.float32
    L = (1 << bits) - 1
    x = np.array([0.0, hi, xv], f32)
    assert float(x[1]) == hi and float(x[2]) == xv           # the literals are float32 values
    _, ranges, q = _quant(x, bits, 3)
    assert ranges.tolist() == [0.0, hi]
    inv = f32(f32(L) / f32(hi))                              # one IEEE division
    exact = Fraction(xv) * Fraction(float(inv)) + Fraction(1, 2)
    once = int(np.floor(_nearest_f32(exact)))
    twice = int(np.floor(f32(_nearest_f32(Fraction(xv) * Fraction(float(inv))) + f32(0.5))))
    assert once != twice
    assert q.tolist() == [0, L, once]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_restored_value_is_rounded_once(bits):
    """x^ = q * step + lo with a single rounding: checked against exact rational arithmetic."""
    L = (1 << bits) - 1
    x = (_rng(90 + bits).standard_normal(600) * 0.37).astype(np.float32)
    _, ranges, q = _quant(x, bits, 200)
    xhat = O.dequantize_minmax(q, bits, 200, ranges)
    differs_if_rounded_twice = 0
    for i in range(x.size):
        lo, hi = np.float32(ranges[2 * (i // 200)]), np.float32(ranges[2 * (i // 200) + 1])
        step = np.float32(np.float32(hi - lo) / np.float32(L))               # two IEEE operations
        exact = Fraction(int(q[i])) * Fraction(float(step)) + Fraction(float(lo))
        assert xhat[i] == _nearest_f32(exact)
        twice = np.float32(_nearest_f32(Fraction(int(q[i])) * Fraction(float(step))) + lo)
        differs_if_rounded_twice += int(twice != xhat[i])
    assert differs_if_rounded_twice > 0 or bits == 2


@pytest.mark.parametrize("bits", [1, 4, 8])
def test_values_outside_the_given_range_saturate(bits):
    """Encoding against a range that does not cover the data (a caller's own range) clamps."""
    L = (1 << bits) - 1
    x = np.array([-50.0, -1.0, 0.0, 0.5, 1.0, 3.0, 300.0], np.float32)
    ranges = np.array([-1.0, 1.0], np.float32)
    q = O.encode_minmax(x, bits, x.size, ranges)
    assert q[0] == 0 and q[1] == 0 and q[4] == L and q[5] == L and q[6] == L
    assert 0 <= q[2] <= L and q[2] <= q[3] <= L


# ------------------------------------------------------------------ packing and the server side
@pytest.mark.parametrize("bits", [1, 3, 8])
def test_codes_are_packed_least_significant_bit_first(bits):
    n = 77
    x = _rng(50 + bits).standard_normal(n).astype(np.float32)
    codes, ranges, q = _quant(x, bits, 32)
    big = 0
    for i, qi in enumerate(q):
        big |= int(qi) << (i * bits)
    words = [(big >> (32 * k)) & 0xFFFFFFFF for k in range(codes.size)]
    assert codes.tolist() == words
    assert np.array_equal(q, O.encode_minmax(x, bits, 32, O.bucket_ranges(x, 32)))


@pytest.mark.parametrize("bits", [2, 4, 7])
def test_sum_runs_in_worker_order_and_update_is_one_fma(bits):
    n, bucket, W = 300, 128, 3
    xs = [(_rng(60 + w).standard_normal(n) * 10.0 ** (w - 1)).astype(np.float32) for w in range(W)]
    enc = [O.quantize_minmax(x, bits, bucket) for x in xs]
    xh = [O.dequantize_minmax(O.unpack(c, n, bits), bits, bucket, r) for c, r in enc]
    acc = O.dequant_accumulate_minmax([c for c, _ in enc], [r for _, r in enc], bits, n, bucket)
    want = (xh[0] + xh[1]) + xh[2]                         # float32, left to right
    assert np.array_equal(acc, want)
    other = xh[0] + (xh[1] + xh[2])
    assert not np.array_equal(want, other)                 # the order is observable on this input
    acc2 = O.dequant_accumulate_minmax([c for c, _ in enc], [r for _, r in enc], bits, n, bucket, acc=acc)
    assert np.array_equal(acc2, ((acc + xh[0]) + xh[1]) + xh[2])
    p0 = _rng(70).standard_normal(n).astype(np.float32)
    p, got_acc = O.server_step_minmax([c for c, _ in enc], [r for _, r in enc], bits, n, bucket, p0.copy(), 0.125,
                                      want_acc=True)
    assert np.array_equal(got_acc, acc)
    exact = p0.astype(np.float64) - 0.125 * acc.astype(np.float64)      # exact in double: lr is 2^-3
    assert np.array_equal(p, exact.astype(np.float32))


def test_bf16_input_is_widened_exactly():
    bits16 = _rng(80).integers(0, 1 << 16, 500).astype(np.uint16)
    bits16 = bits16[((bits16 >> 7) & 0xFF) < 0xF0]                      # no inf / nan, no huge values
    wide = (bits16.astype(np.uint32) << 16).view(np.float32)
    wide = np.clip(wide, -1e30, 1e30)
    keep = np.abs(wide) < 1e30
    c1, r1 = O.quantize_minmax(bits16[keep], 4, 64, dtype="bf16")
    c2, r2 = O.quantize_minmax(wide[keep], 4, 64)
    assert np.array_equal(c1, c2) and np.array_equal(r1.view(np.uint32), r2.view(np.uint32))
