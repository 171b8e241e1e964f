"""Pins of the CPU checker's L2-norm scale variant against things other than itself: closed forms
where every partial sum is exact, inputs built so that a different summation order or an unfused
square yields a different float, exact rational arithmetic with one correct rounding per named
operation, the error bound of the sum against double precision, and the properties the encode
relies on (no element exceeds its scale).  Everything here runs on the CPU."""
from fractions import Fraction
import math

import numpy as np
import pytest

from oracle import mqg_oracle as O
from tests.exact import f32_to_fraction, round_to_f32

F = np.float32


def _rng(seed):
    return np.random.default_rng(seed)


def _rows(values):
    """A bucket whose row r (32 elements) is [values[r], 0, 0, ...]."""
    x = np.zeros(32 * len(values), F)
    x[::32] = values
    return x


# ------------------------------------------------------------------ closed forms, exact sums
@pytest.mark.parametrize("x,S", [
    ([3, 4], 25), ([1, 2, 2], 9), ([2, 3, 6], 49), ([1, 4, 8], 81), ([2, 10, 11], 225),
    ([1] * 31, 31), ([1] * 32, 32), ([1] * 33, 33), ([2] * 1000, 4000), ([3] * 8191, 9 * 8191),
])
def test_small_integers_sum_exactly(x, S):
    # every partial sum is an integer below 2^24, so no rounding happens in any order
    x = np.array(x, F)
    assert O.sumsq_tree(x) == F(S)
    r = math.isqrt(S)
    if r * r == S:
        assert O.bucket_norms(x, x.size)[0] == F(r)


@pytest.mark.parametrize("e", [-40, -13, 0, 7, 30])
def test_scaling_by_a_power_of_two_scales_the_sum_by_its_square(e):
    x = _rng(e + 100).standard_normal(700).astype(F)
    S = O.sumsq_tree(x)
    assert O.sumsq_tree(x * F(2.0 ** e)) == F(float(S) * 4.0 ** e)
    assert O.bucket_norms(x * F(2.0 ** e), 700)[0] == F(float(O.bucket_norms(x, 700)[0]) * 2.0 ** e)


def test_sign_and_trailing_zeros_do_not_matter():
    x = _rng(5).standard_normal(100).astype(F)
    S = O.sumsq_tree(x)
    assert O.sumsq_tree(-x) == S
    for pad in (1, 28, 29, 500, 5000):                    # zeros add exactly at every level
        assert O.sumsq_tree(np.concatenate([x, np.zeros(pad, F)])) == S


# ------------------------------------------------------------------ the order of the sum
def test_rows_are_summed_left_to_right():
    # 4096^2 = 2^24, then 31 ones: each 2^24 + 1 is a tie that rounds back to 2^24
    x = np.ones(32, F)
    x[0] = 4096
    assert O.sumsq_tree(x) == F(2.0 ** 24)
    # ones first: 31, then 31 + 2^24 is a tie between 2^24 + 30 and 2^24 + 32 -> even -> + 32
    x = np.ones(32, F)
    x[31] = 4096
    assert O.sumsq_tree(x) == F(2.0 ** 24 + 32)


def test_square_and_add_are_fused():
    # a = 2^-24 after element 0; x1^2 = 1 + 2^-11 + 2^-24 exactly.  Fused: 1 + 2^-11 + 2^-23
    # (representable).  A rounded square (tie -> 1 + 2^-11) plus 2^-24 is again a tie -> 1 + 2^-11.
    x = np.array([2.0 ** -12, 1 + 2.0 ** -12], F)
    assert O.sumsq_tree(x) == F(1 + 2.0 ** -11 + 2.0 ** -23)


def test_row_sums_are_combined_pairwise_not_in_sequence():
    # row sums 2^24, 1, 1, 1: pairs (2^24 + 1 -> 2^24) + (1 + 1) = 2^24 + 2; in sequence: 2^24
    assert O.sumsq_tree(_rows([4096, 1, 1, 1])) == F(2.0 ** 24 + 2)
    # the pairs are adjacent rows: (1 + 1) + (2^24 + 1 -> 2^24) against (1 + 2^24) + (1 + 1)
    assert O.sumsq_tree(_rows([1, 1, 4096, 1])) == F(2.0 ** 24 + 2)
    assert O.sumsq_tree(_rows([1, 4096, 1, 1])) == F(2.0 ** 24 + 2)
    # three levels: ((2^24 + 1) + (1 + 1)) + ((1 + 1) + (1 + 1)) = (2^24 + 2) + 4
    assert O.sumsq_tree(_rows([4096, 1, 1, 1, 1, 1, 1, 1])) == F(2.0 ** 24 + 6)
    # a leaf count that is not a power of two is padded with zeros: rows (2^24, 1, 1) ->
    # (2^24 + 1 -> 2^24) + (1 + 0) -> tie -> 2^24
    assert O.sumsq_tree(_rows([4096, 1, 1])) == F(2.0 ** 24)
    # eight rows, partners are neighbours at every level: (2^24 + 1 -> 2^24) and, in the other
    # half, (0 + 1); pairing row j with row j + 4 would add the two ones first and give 2^24 + 2
    assert O.sumsq_tree(_rows([4096, 1, 0, 0, 0, 1, 0, 0])) == F(2.0 ** 24)
    # five rows: the fifth meets the first four only at the root: (1+1)+(1+1) = 4, 4 + 2^24
    assert O.sumsq_tree(_rows([1, 1, 1, 1, 4096])) == F(2.0 ** 24 + 4)


def test_a_row_is_32_elements_counted_from_the_start_of_the_bucket():
    # elements 0..31 form row 0 and 32..63 row 1: with 2^12 at index 0 and ones behind it the ones
    # of row 0 vanish one by one, those of row 1 add up to 32 first
    x = np.ones(64, F)
    x[0] = 4096
    assert O.sumsq_tree(x) == F(2.0 ** 24 + 32)
    # in a later bucket the rows start at the bucket's first element
    y = np.concatenate([np.ones(96, F), x])
    s = O.bucket_norms(y, 96)
    assert s[0] == F(math.sqrt(96)) and s.size == 2
    assert s[1] == F(math.sqrt(2.0 ** 24 + 32))          # 64 elements: the last bucket is shorter


# ------------------------------------------------------------------ exact rational arithmetic
def _exact_tree(x):
    """N1/N2 with Fractions, one correct rounding (tests.exact) per fused multiply-add and per sum."""
    rows = []
    for r0 in range(0, len(x), 32):
        a = Fraction(0)
        for v in x[r0:r0 + 32]:
            fv = f32_to_fraction(v)
            a = Fraction(round_to_f32(fv * fv + a))
        rows.append(a)
    while len(rows) & (len(rows) - 1):
        rows.append(Fraction(0))
    while len(rows) > 1:
        rows = [Fraction(round_to_f32(rows[2 * j] + rows[2 * j + 1])) for j in range(len(rows) // 2)]
    return float(rows[0])


@pytest.mark.parametrize("n,scale", [(1, 1.0), (5, 1e-4), (32, 1.0), (33, 3e-3), (100, 1e3), (257, 1e-4),
                                     (700, 1.0)])
def test_sum_matches_exact_rationals_rounded_once_per_operation(n, scale):
    x = (_rng(n).standard_normal(n) * scale).astype(F)
    assert float(O.sumsq_tree(x)) == _exact_tree(x)


def test_root_is_correctly_rounded():
    for seed in range(20):
        x = (_rng(seed).standard_normal(40 + seed) * 10.0 ** (seed % 7 - 4)).astype(F)
        S = Fraction(float(O.sumsq_tree(x)))
        s = float(O.bucket_norms(x, x.size)[0])
        below, above = float(np.nextafter(F(s), F(0))), float(np.nextafter(F(s), F(np.inf)))
        lo_mid, hi_mid = (Fraction(s) + Fraction(below)) / 2, (Fraction(s) + Fraction(above)) / 2
        assert lo_mid * lo_mid <= S <= hi_mid * hi_mid          # s is the float nearest to sqrt(S)


# ------------------------------------------------------------------ against double precision
@pytest.mark.parametrize("n", [31, 2048, 8192, 100_000])
def test_norm_is_close_to_the_double_precision_norm(n):
    x = _rng(n).laplace(0.0, 1e-4, n).astype(F)
    s = float(O.bucket_norms(x, n)[0])
    ref = math.sqrt(float(np.sum(x.astype(np.float64) ** 2)))
    depth = 32 + max(1, math.ceil(math.log2((n + 31) // 32))) + 1       # roundings on any path
    assert abs(s - ref) <= depth * 2.0 ** -24 * ref


@pytest.mark.parametrize("n,bucket", [(1000, 256), (513, 512), (4096, 1024), (70, 32)])
def test_one_norm_per_bucket_last_bucket_shorter(n, bucket):
    x = _rng(n).standard_normal(n).astype(F)
    s = O.bucket_norms(x, bucket)
    nb = (n + bucket - 1) // bucket
    assert s.size == nb
    for k in range(nb):
        assert s[k] == O.bucket_norms(x[k * bucket:(k + 1) * bucket], bucket)[0]
        ref = math.sqrt(float(np.sum(x[k * bucket:(k + 1) * bucket].astype(np.float64) ** 2)))
        assert abs(float(s[k]) - ref) <= 2.0 ** -18 * ref


# ------------------------------------------------------------------ what the encode relies on
def test_no_element_exceeds_its_scale():
    rng = _rng(77)
    cases = [rng.standard_normal(300).astype(F) * F(10.0 ** e) for e in (-30, -20, -10, 0, 10)]
    one_hot = np.zeros(64, F); one_hot[17] = F(1.2345678)            # sqrt(fl(x^2)) = |x| exactly
    cases.append(one_hot)
    for e in range(-60, -40):                                        # squares near the subnormals
        v = np.zeros(40, F); v[3] = F((1 + 2.0 ** -23) * 2.0 ** e); v[9] = F(2.0 ** -48)
        cases.append(v)
    for x in cases:
        s = O.bucket_norms(x, x.size)[0]
        assert s == 0 or float(np.abs(x).max()) <= float(s)


def test_flush_is_decided_on_the_sum_of_squares():
    x = np.zeros(50, F)
    x[7] = F(2.0 ** -48)                                             # S = 2^-96: kept
    assert O.bucket_norms(x, 50)[0] == F(2.0 ** -48)
    x[7] = np.nextafter(F(2.0 ** -48), F(0))                         # S just below 2^-96: flushed
    assert O.bucket_norms(x, 50)[0] == 0
    codes, scales = O.quantize_l2(x, 4, 50, seed=1)
    assert scales[0] == 0 and not codes.any()
    x[:] = 0
    assert O.bucket_norms(x, 50)[0] == 0 and np.signbit(O.bucket_norms(x, 50)[0]) == False  # noqa: E712


# ------------------------------------------------------------------ the codec around the scale
@pytest.mark.parametrize("bits", [1, 3, 4, 8])
def test_quantize_l2_is_the_main_codec_with_the_norm_as_scale(bits):
    n, bucket = 1000, 256
    x = _rng(bits).laplace(0.0, 1e-4, n).astype(F)
    codes, scales = O.quantize_l2(x, bits, bucket, seed=9, worker=2, step=5, elem_offset=64)
    assert np.array_equal(scales, O.bucket_norms(x, bucket))
    h = O.draw_h(9, 2, 5, 64, n)
    q = O.encode(x, bits, bucket, scales, h)
    assert np.array_equal(codes, O.pack(q, bits))
    L = (1 << bits) - 1
    assert q.max() <= L
    # decoding with the ordinary de-quantizer stays within one grid step of the input
    xhat = O.dequantize(q, bits, bucket, scales)
    step = 2 * np.repeat(scales, bucket)[:n].astype(np.float64) / L
    assert np.all(np.abs(xhat.astype(np.float64) - x) < step * (1 + 1e-6))


def test_quantize_l2_is_unbiased():
    n, bits = 64, 4
    x = _rng(3).standard_normal(n).astype(F) * F(1e-3)
    s = O.bucket_norms(x, n)
    acc = np.zeros(n, np.float64)
    seeds = 1500
    for seed in range(seeds):
        codes, sc = O.quantize_l2(x, bits, n, seed=seed)
        acc += O.dequantize(O.unpack(codes, n, bits), bits, n, sc)
    step = 2 * float(s[0]) / ((1 << bits) - 1)
    assert np.all(np.abs(acc / seeds - x) <= 5 * (step / 2) / math.sqrt(seeds))


def test_bf16_input_is_widened_first():
    x16 = (_rng(8).integers(0, 1 << 16, 300).astype(np.uint16) & np.uint16(0xBFFF)) | np.uint16(0x3000)
    x16 &= np.uint16(0xBFFF)                                          # finite, moderate exponents
    x = O.widen_bf16(x16)
    c16, s16 = O.quantize_l2(x16, 5, 64, seed=4, dtype="bf16")
    c32, s32 = O.quantize_l2(x, 5, 64, seed=4)
    assert np.array_equal(c16, c32) and np.array_equal(s16, s32)


def test_segments_are_buckets_with_word_aligned_streams():
    x = _rng(12).standard_normal(500).astype(F)
    seg_off = np.array([0, 37, 37, 300, 500], np.uint64)
    bits = 3
    words = [O.code_words(int(seg_off[j + 1] - seg_off[j]), bits) for j in range(4)]
    code_off = np.concatenate([[0], np.cumsum(words)]).astype(np.uint64)
    codes, scales = O.quantize_segments_l2(x, seg_off, code_off, bits, seed=21, worker=1, step=2, elem_offset=8)
    for j in range(4):
        a, b = int(seg_off[j]), int(seg_off[j + 1])
        if a == b:
            assert scales[j] == 0
            continue
        c, s = O.quantize_l2(x[a:b], bits, b - a, seed=21, worker=1, step=2, elem_offset=8 + a)
        assert np.array_equal(codes[int(code_off[j]):int(code_off[j + 1])], c) and scales[j] == s[0]
