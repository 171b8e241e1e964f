"""Pins of the CPU checker's 1-bit error-feedback variant against things other than itself: small
cases worked out by hand, the conservation law of error feedback on exactly representable data,
numpy means on integer data, inputs built so that another summation order gives another float,
exact rational arithmetic for the roundings, and the separately pinned (min, max) de-quantizer
acting as the receiver.  Everything here runs on the CPU."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import mqg_oracle as O
from tests.exact import f32_to_fraction, round_to_f32

F = np.float32


def _rng(seed):
    return np.random.default_rng(seed)


def _run(g, e, bucket):
    codes, ranges, e2 = O.quantize_1bit_ef(g, e, bucket)
    q = O.unpack(codes, g.size, 1)
    return codes, ranges, e2, q


# ------------------------------------------------------------------ worked by hand
def test_four_elements_by_hand():
    # v = g: classes {3, 1} and {-1, -3}: pos = 2, neg = -2, r = 4; x^ = +-2; e = v - x^
    codes, ranges, e2, q = _run(np.array([3, -1, 1, -3], F), np.zeros(4, F), 4)
    assert q.tolist() == [1, 0, 1, 0] and codes.tolist() == [0b0101]
    assert ranges.tolist() == [-2.0, 2.0]
    assert e2.tolist() == [1.0, 1.0, -1.0, -1.0]


def test_the_old_residual_is_added_before_the_sign_is_taken():
    # g = [1, 1], e = [-3, 1]: v = [-2, 2] -> q = [0, 1], neg = -2, pos = 2, nothing left over
    codes, ranges, e2, q = _run(np.array([1, 1], F), np.array([-3, 1], F), 2)
    assert q.tolist() == [0, 1] and ranges.tolist() == [-2.0, 2.0] and e2.tolist() == [0.0, 0.0]


def test_zero_counts_as_non_negative_and_one_sided_buckets():
    codes, ranges, e2, q = _run(np.array([0.0, -0.0, 4.0, 2.0], F), np.zeros(4, F), 4)
    assert q.tolist() == [1, 1, 1, 1]
    assert ranges.tolist() == [0.0, 1.5]                      # empty class -> 0; mean of (0, 0, 4, 2)
    assert e2.tolist() == [-1.5, -1.5, 2.5, 0.5]
    codes, ranges, e2, q = _run(np.array([-1.0, -2.0, -6.0], F), np.zeros(3, F), 8)
    assert q.tolist() == [0, 0, 0] and ranges.tolist() == [-3.0, 0.0] and e2.tolist() == [2.0, 1.0, -3.0]


def test_all_zero_bucket_is_constant():
    codes, ranges, e2, q = _run(np.zeros(40, F), np.zeros(40, F), 32)
    assert not codes.any() and ranges.view(np.uint32).tolist() == [0, 0, 0, 0] and not e2.any()
    assert not np.signbit(e2).any()


def test_a_spread_below_the_threshold_is_constant_and_the_codes_are_cleared():
    v = np.array([1e-30, -1e-30, 2e-30, -2e-30], F)
    codes, ranges, e2, q = _run(v, np.zeros(4, F), 4)
    assert not codes.any()                                     # r = 3e-30 < 2^-96
    neg = ranges[0]
    assert neg == F(F(-1e-30) + F(-2e-30)) / F(2) and np.array_equal(e2, v - neg)


# ------------------------------------------------------------------ conservation
@pytest.mark.parametrize("bucket", [32, 96, 256, 1000])
def test_what_is_sent_plus_the_new_residual_is_the_gradient_plus_the_old_one(bucket):
    # small multiples of 2^-6 with class counts that divide their sums (means are made exact by using
    # two values per class), so every operation is exact and the law holds bit for bit
    n = 1000
    rng = _rng(bucket)
    sign = rng.integers(0, 2, n) * 2 - 1
    g = (sign * 5 * 2.0 ** -6).astype(F)
    e = np.zeros(n, F)
    sent_total = np.zeros(n, np.float64)
    for it in range(6):
        codes, ranges, e2 = O.quantize_1bit_ef(g, e, bucket)
        xhat = O.dequantize_minmax(O.unpack(codes, n, 1), 1, bucket, ranges)
        assert np.array_equal(xhat.astype(np.float64) + e2, g.astype(np.float64) + e)
        sent_total += xhat
        e = e2
    assert np.array_equal(sent_total + e, 6 * g.astype(np.float64))


def test_conservation_holds_within_rounding_on_real_valued_data():
    n, bucket = 5000, 512
    g = _rng(1).laplace(0, 1e-4, n).astype(F)
    e = np.zeros(n, F)
    total = np.zeros(n, np.float64)
    for it in range(8):
        codes, ranges, e2 = O.quantize_1bit_ef(g, e, bucket)
        xhat = O.dequantize_minmax(O.unpack(codes, n, 1), 1, bucket, ranges)
        # one rounding in v = g + e and one in e' = v - x^
        v = g.astype(np.float64) + e
        assert np.all(np.abs(xhat + e2.astype(np.float64) - v) <= 2.0 ** -23 * (np.abs(v) + np.abs(xhat)) + 1e-45)
        total += xhat
        e = e2
    # the running sum of what was sent follows the running sum of the gradients up to the residual
    assert np.all(np.abs(total + e - 8 * g.astype(np.float64)) <= 1e-9)


# ------------------------------------------------------------------ the means
@pytest.mark.parametrize("n,bucket", [(64, 64), (1000, 256), (513, 512), (70, 32)])
def test_means_against_numpy_on_integer_data(n, bucket):
    v = _rng(n).integers(-50, 51, n).astype(F)               # sums are exact in any order
    codes, ranges, e2, q = _run(v, np.zeros(n, F), bucket)
    for k in range((n + bucket - 1) // bucket):
        part = v[k * bucket:(k + 1) * bucket]
        pos, neg = part[part >= 0], part[part < 0]
        want_pos = F(F(pos.sum()) / F(pos.size)) if pos.size else F(0)
        want_neg = F(F(neg.sum()) / F(neg.size)) if neg.size else F(0)
        assert ranges[2 * k] == want_neg and ranges[2 * k + 1] == want_pos
        assert np.array_equal(q[k * bucket:(k + 1) * bucket], (part >= 0).astype(np.uint8))


def test_class_sums_run_left_to_right_inside_a_row_and_pairwise_over_rows():
    # one row: 2^24 then 31 ones (each tie rounds back) against the ones first (-> 2^24 + 32)
    v = np.ones(32, F); v[0] = 2.0 ** 24
    assert _run(v, np.zeros(32, F), 32)[1][1] == F(2.0 ** 24 / 32)
    v = np.ones(32, F); v[31] = 2.0 ** 24
    assert _run(v, np.zeros(32, F), 32)[1][1] == F((2.0 ** 24 + 32) / 32)
    # four rows with sums 2^24, 1, 1, 1: pairwise (2^24 + 1 -> 2^24) + (1 + 1) = 2^24 + 2
    v = np.zeros(128, F); v[0] = 2.0 ** 24; v[32] = v[64] = v[96] = 1
    assert _run(v, np.zeros(128, F), 128)[1][1] == F((2.0 ** 24 + 2) / 128)
    # the same for the negative class, which skips the non-negative elements of its rows
    v = np.full(128, 7.0, F); v[0] = -2.0 ** 24; v[32] = v[64] = v[96] = -1
    r = _run(v, np.zeros(128, F), 128)[1]
    assert r[0] == F(-(2.0 ** 24 + 2) / 4) and r[1] == F(7.0)
    # partners are neighbours: rows (2^24, 1, 0, 0, 0, 1, 0, 0) -> 2^24, not 2^24 + 2
    v = np.zeros(256, F); v[0] = 2.0 ** 24; v[32] = 1; v[160] = 1
    assert _run(v, np.zeros(256, F), 256)[1][1] == F(2.0 ** 24 / 256)


def _exact(g, e, bucket):
    """E1..E5 with Fractions and one correct rounding per named operation."""
    rnd = lambda x: Fraction(round_to_f32(x))
    n = len(g)
    v = [rnd(f32_to_fraction(a) + f32_to_fraction(b)) for a, b in zip(g, e)]
    ranges, res = [], []
    for b0 in range(0, n, bucket):
        part = v[b0:b0 + bucket]
        means = []
        for cls in (0, 1):
            rows = []
            for r0 in range(0, len(part), 32):
                a = Fraction(0)
                for x in part[r0:r0 + 32]:
                    if (x >= 0) == bool(cls):
                        a = rnd(a + x)
                rows.append(a)
            while len(rows) & (len(rows) - 1):
                rows.append(Fraction(0))
            while len(rows) > 1:
                rows = [rnd(rows[2 * j] + rows[2 * j + 1]) for j in range(len(rows) // 2)]
            c = sum(1 for x in part if (x >= 0) == bool(cls))
            means.append(rnd(rows[0] / c) if c else Fraction(0))
        neg, pos = means
        r = rnd(pos - neg)
        ranges += [float(neg), float(pos)]
        for x in part:
            xhat = neg if (r < Fraction(2) ** -96 or x < 0) else rnd(r + neg)
            res.append(float(rnd(x - xhat)))
    return np.array(ranges, F), np.array(res, F)


@pytest.mark.parametrize("n,bucket,scale", [(7, 8, 1.0), (40, 32, 1e-3), (100, 64, 1e3), (300, 96, 1e-4)])
def test_ranges_and_residual_match_exact_rationals_rounded_once_per_operation(n, bucket, scale):
    rng = _rng(n)
    g = (rng.standard_normal(n) * scale).astype(F)
    e = (rng.standard_normal(n) * scale * 0.3).astype(F)
    codes, ranges, e2, q = _run(g, e, bucket)
    want_ranges, want_e = _exact(g, e, bucket)
    assert np.array_equal(ranges, want_ranges)
    assert np.array_equal(e2, want_e)
    assert np.array_equal(q, ((g + e) >= 0).astype(np.uint8))


# ------------------------------------------------------------------ receiver, packing, formats
def test_the_minmax_receiver_reconstructs_the_value_the_residual_was_taken_against():
    n, bucket = 3000, 256
    g = _rng(4).standard_normal(n).astype(F)
    e = (_rng(5).standard_normal(n) * 0.1).astype(F)
    codes, ranges, e2, q = _run(g, e, bucket)
    xhat = O.dequantize_minmax(q, 1, bucket, ranges)
    v = (g + e).astype(F)
    assert np.array_equal(e2, (v - xhat).astype(F))
    # and the server sum of several such workers is the ordinary ordered sum
    acc = O.dequant_accumulate_minmax([codes, codes], [ranges, ranges], 1, n, bucket)
    assert np.array_equal(acc, (xhat + xhat).astype(F))


def test_codes_are_the_packed_sign_bits():
    n = 1000
    g = _rng(6).standard_normal(n).astype(F)
    codes, ranges, e2, q = _run(g, np.zeros(n, F), 128)
    big = sum(int(b) << i for i, b in enumerate((g >= 0).astype(int)))
    assert codes.tobytes() == big.to_bytes(4 * ((n + 31) // 32), "little")


def test_bf16_gradient_is_widened_first():
    x16 = (_rng(8).integers(0, 1 << 16, 300).astype(np.uint16) & np.uint16(0xBFFF)) | np.uint16(0x3000)
    x16[::3] |= np.uint16(0x8000)
    e = (_rng(9).standard_normal(300) * 0.01).astype(F)
    a = O.quantize_1bit_ef(x16, e, 64, dtype="bf16")
    b = O.quantize_1bit_ef(O.widen_bf16(x16), e, 64)
    assert all(np.array_equal(u, w) for u, w in zip(a, b))


def test_error_feedback_makes_the_time_average_converge():
    # a constant gradient sent with one bit: the mean of what the receiver gets tends to the gradient
    n, bucket, T = 256, 256, 400
    g = _rng(10).standard_normal(n).astype(F)
    e = np.zeros(n, F)
    total = np.zeros(n, np.float64)
    for it in range(T):
        codes, ranges, e = O.quantize_1bit_ef(g, e, bucket)
        total += O.dequantize_minmax(O.unpack(codes, n, 1), 1, bucket, ranges)
    assert np.abs(total / T - g).max() <= np.abs(e).max() / T + 1e-5
    # inside a class the residuals cancel: the class mean takes out exactly the class's total
    v_last = g.astype(np.float64) + 0          # (checked on a fresh step with zero residual)
    codes, ranges, e1 = O.quantize_1bit_ef(g, np.zeros(n, F), bucket)
    assert abs(e1[g >= 0].astype(np.float64).sum()) <= 1e-4 and abs(e1[g < 0].astype(np.float64).sum()) <= 1e-4
