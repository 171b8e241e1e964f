"""Pins for the CPU checker (oracle/): what the paper and the mathematics fix,
checked without reference to the checker's own formulas.

The paper (Section 3.2, Algorithm 1) fixes: the server result is the sum/mean of the
de-quantized worker gradients, the update is w - eta*g, K is an integer number of
bits.  The codec reading adds: codes in [0, 2^K-1], exact bit packing, exactness on
the grid, unbiased stochastic rounding.  Each test below names the property."""
import math
import os
import subprocess
import sys
from fractions import Fraction

import numpy as np
import pytest

from oracle import mqg_oracle as O
from tests.exact import f32_bits, f32_to_fraction, round_to_f32

ALL_BITS = list(range(1, 9))


# ---------------------------------------------------------------- packing (R9)
@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("n", [0, 1, 7, 31, 32, 33, 1000])
def test_pack_is_little_endian_big_integer(bits, n):
    rng = np.random.default_rng(100 * bits + n)
    q = rng.integers(0, 1 << bits, n, dtype=np.uint8)
    big = 0
    for i, v in enumerate(q.tolist()):
        big |= v << (i * bits)
    nbytes = 4 * ((n * bits + 31) // 32)
    expect = big.to_bytes(nbytes, "little")
    words = O.pack(q, bits)
    assert words.astype("<u4").tobytes() == expect
    assert np.array_equal(O.unpack(words, n, bits), q)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_pack_extremes_and_padding(bits):
    L = (1 << bits) - 1
    for n in (1, 5, 37):
        q = np.full(n, L, np.uint8)
        words = O.pack(q, bits)
        total = int.from_bytes(words.astype("<u4").tobytes(), "little")
        assert total == (1 << (n * bits)) - 1          # all ones, pad bits zero
        assert np.array_equal(O.unpack(words, n, bits), q)


# ---------------------------------------------------------------- scale (R2, R3)
def test_scale_is_bucket_max_abs():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(4096 + 100).astype(np.float32)
    s = O.bucket_scales(x, 512)
    full = np.abs(x[:4096]).reshape(-1, 512).max(1)
    assert np.array_equal(s[:8], full)
    assert s[8] == np.abs(x[4096:]).max()
    assert s.size == 9


def test_scale_flush_threshold():
    tiny = np.float32(2.0 ** -96)
    below = np.nextafter(tiny, np.float32(0))
    x = np.zeros(96, np.float32)
    x[0:32] = below
    x[32] = -tiny
    s = O.bucket_scales(x, 32)
    assert s[0] == 0.0 and s[1] == tiny and s[2] == 0.0
    h = np.arange(96, dtype=np.uint16) * 600
    for bits in ALL_BITS:
        q = O.encode(x, bits, 32, s, h)
        assert not q[:32].any() and not q[64:].any()
        xh = O.dequantize(q, bits, 32, s)
        assert not xh[:32].any() and not np.signbit(xh[:32]).any()


# ---------------------------------------------------------------- range
@pytest.mark.parametrize("bits", ALL_BITS)
def test_codes_stay_in_range_on_adversarial_inputs(bits):
    L = (1 << bits) - 1
    fmax = np.finfo(np.float32).max
    cases = []
    for s in (1.0, 3.0, 1e-30, 2.0 ** -96, 1e30, fmax, 0.1, 1.0 / 3.0, 7e-5):
        s = np.float32(s)
        row = [s, -s, 0.0, -0.0, s * np.float32(0.5), np.nextafter(s, np.float32(0)),
               -np.nextafter(s, np.float32(0)), np.float32(1e-45), np.float32(-1e-45)]
        cases.append(np.array(row + [0.0] * (16 - len(row)), np.float32))
    x = np.concatenate(cases)
    s = O.bucket_scales(x, 16)
    for hval in (0, 1, 32767, 32768, 65534, 65535):
        q = O.encode(x, bits, 16, s, np.full(x.size, hval, np.uint16))
        assert q.max() <= L
        # x = +s encodes to L and x = -s to 0, whatever the draw
        for k in range(len(cases)):
            if 0 < s[k] < 1e38:
                assert q[16 * k] == L and q[16 * k + 1] == 0


# ---------------------------------------------------------------- grid exactness
@pytest.mark.parametrize("bits", ALL_BITS)
def test_dyadic_grid_is_a_fixed_point(bits):
    L = (1 << bits) - 1
    rng = np.random.default_rng(bits)
    for e in (-20, -3, 0, 5):
        s = np.float32(L * 2.0 ** e)
        q0 = rng.integers(0, L + 1, 256, dtype=np.uint8)
        q0[0], q0[1] = L, 0                      # make max|x| = s
        grid = ((2.0 * q0.astype(np.float64) - L) * 2.0 ** e).astype(np.float32)
        assert np.array_equal(grid.astype(np.float64), (2.0 * q0 - L) * 2.0 ** e)
        sc = O.bucket_scales(grid, 256)
        assert sc[0] == s
        assert np.array_equal(O.dequantize(q0, bits, 256, sc), grid)
        for hval in (0, 12345, 65535):
            q = O.encode(grid, bits, 256, sc, np.full(256, hval, np.uint16))
            assert np.array_equal(q, q0)


# ---------------------------------------------------------------- rounding rule
def _exact_t(x, s, L):
    return f32_to_fraction(x) * L / (2 * f32_to_fraction(s)) + Fraction(L, 2)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_round_up_probability_over_all_65536_draws(bits):
    """For a fixed element the number of draws that round up must be the number of
    h with (h+1/2)/2^16 below frac(t): E[q] = t to within 2^-17 plus fp32 error."""
    L = (1 << bits) - 1
    rng = np.random.default_rng(40 + bits)
    s = np.float32(0.0371)
    xs = rng.uniform(-0.0371, 0.0371, 12).astype(np.float32)
    h = np.arange(65536, dtype=np.uint16)
    for xv in xs:
        x = np.full(65537, xv, np.float32)
        x[0] = s                                 # pins the bucket scale
        sc = O.bucket_scales(x, 65537)
        assert sc[0] == s
        hh = np.concatenate([[0], h]).astype(np.uint16)
        q = O.encode(x, bits, 65537, sc, hh)[1:].astype(np.int64)
        t = _exact_t(xv, s, L)
        lo = math.floor(t)
        assert set(np.unique(q)).issubset({lo - 1, lo, lo + 1})
        mean_q = Fraction(int(q.sum()), 65536)
        # fp32 error of t: a few ulp at magnitude L
        tol = Fraction(1, 2 ** 17) + 4 * Fraction(L, 2 ** 23)
        assert abs(mean_q - t) <= tol, (float(mean_q), float(t))
        # monotone in h: small draws round up, large ones do not
        ups = (q == q.max()) if q.max() != q.min() else None
        if ups is not None:
            first_down = np.argmin(ups)
            assert ups[:first_down].all() and not ups[first_down:].any()


def test_t_carries_one_fused_rounding():
    """R4/R5 name two roundings: inv = fl(L/(2s)) and t = fl(x*inv + L/2).  For K = 8
    the unit in the last place of t (2^-16 above 128) is as coarse as the draw grid,
    so the exact number of round-ups over all 65,536 draws reveals t to the last bit.
    Inputs are chosen, with exact rationals, where a two-rounding t would differ."""
    bits, L = 8, 255
    s = np.float32(0.0371)
    inv = round_to_f32(Fraction(L) / (2 * f32_to_fraction(s)))
    rng = np.random.default_rng(77)
    picked = []
    for xv in rng.uniform(0.001, 0.0371, 4000).astype(np.float32):
        prod = f32_to_fraction(xv) * Fraction(inv)
        fused = round_to_f32(prod + Fraction(L, 2))
        unfused = round_to_f32(Fraction(round_to_f32(prod)) + Fraction(L, 2))
        if fused != unfused and fused >= 128 and math.floor(fused) == math.floor(unfused):
            picked.append((xv, fused))
        if len(picked) == 4:
            break
    assert len(picked) == 4
    h = np.concatenate([[0], np.arange(65536)]).astype(np.uint16)
    for xv, t in picked:
        x = np.full(65537, xv, np.float32)
        x[0] = s
        sc = O.bucket_scales(x, 65537)
        q = O.encode(x, bits, 65537, sc, h)[1:].astype(np.int64)
        r = Fraction(t) - math.floor(t)
        # number of h in [0, 65536) with (h + 1/2) / 65536 < r
        want_ups = max(0, min(65536, math.ceil(r * 65536 - Fraction(1, 2))))
        assert int((q == math.floor(t) + 1).sum()) == want_ups


def test_one_bit_is_stochastic_sign():
    """K = 1: the code is 1 with probability (x + s) / (2 s) (closed form)."""
    s = np.float32(0.5)
    h = np.arange(65536, dtype=np.uint16)
    for xv in (-0.5, -0.25, 0.0, 0.125, 0.3, 0.4999):
        x = np.full(65536 + 1, xv, np.float32)
        x[0] = s
        sc = O.bucket_scales(x, x.size)
        q = O.encode(x, 1, x.size, sc, np.concatenate([[0], h]).astype(np.uint16))[1:]
        p = (float(np.float32(xv)) + 0.5) / 1.0
        assert abs(q.mean() - p) <= 2.0 ** -16
        xh = O.dequantize(q, 1, q.size, sc)
        assert set(np.unique(xh)).issubset({-0.5, 0.5})


@pytest.mark.parametrize("bits", ALL_BITS)
def test_error_bounds_nearest_and_stochastic(bits):
    """With the mid draw the codec is textbook nearest-level quantization on [-s, s]
    (error <= half a step); with any draw the error stays below one step."""
    L = (1 << bits) - 1
    rng = np.random.default_rng(7 * bits)
    x = (rng.standard_normal(8192) * 1e-3).astype(np.float32)
    sc = O.bucket_scales(x, 512)
    step = np.repeat(2.0 * sc.astype(np.float64) / L, 512)
    slack = 8 * np.spacing(np.repeat(sc, 512)).astype(np.float64)
    q = O.encode(x, bits, 512, sc, np.full(x.size, 32767, np.uint16))
    err = np.abs(O.dequantize(q, bits, 512, sc).astype(np.float64) - x)
    assert (err <= 0.5 * step * (1 + 2.0 ** -15) + slack).all()
    for seed in range(3):
        hh = O.draw_h(seed, 0, 0, 0, x.size)
        q = O.encode(x, bits, 512, sc, hh)
        err = np.abs(O.dequantize(q, bits, 512, sc).astype(np.float64) - x)
        assert (err < step + slack).all()


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_unbiased_over_many_seeds(bits):
    """Mean of the de-quantized value over S seeds tends to x (stochastic rounding is
    unbiased): per element within 5 sigma, grand mean much tighter."""
    L = (1 << bits) - 1
    S, n = 2048, 64
    rng = np.random.default_rng(bits)
    x = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    acc = np.zeros(n, np.float64)
    for seed in range(S):
        codes, sc = O.quantize(x, bits, n, seed=seed, worker=1, step=2)
        acc += O.dequantize(O.unpack(codes, n, bits), bits, n, sc)
    mean = acc / S
    step = 2.0 * float(sc[0]) / L
    sigma = 0.5 * step / math.sqrt(S)              # sd of a Bernoulli step is <= step/2
    assert np.abs(mean - x).max() <= 5 * sigma + 1e-9
    assert abs((mean - x).mean()) <= 5 * sigma / math.sqrt(n) + step * 2.0 ** -16


# ---------------------------------------------------------------- brute force, n <= 16
def _ref_scale(xs):
    return max(abs(f32_to_fraction(v)) for v in xs)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_brute_force_small_vectors(bits):
    L = (1 << bits) - 1
    rng = np.random.default_rng(900 + bits)
    for trial in range(6):
        n = int(rng.integers(1, 17))
        W = int(rng.integers(1, 5))
        xs = [(rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 1)).astype(np.float32)
              for _ in range(W)]
        lr = np.float32(rng.uniform(0.01, 1.0))
        p0 = rng.standard_normal(n).astype(np.float32)
        codes, scales, qs = [], [], []
        for w in range(W):
            c, sc = O.quantize(xs[w], bits, n, seed=trial, worker=w, step=3)
            s_exact = _ref_scale(xs[w])
            assert f32_to_fraction(sc[0]) == s_exact
            q = O.unpack(c, n, bits)
            # every code is one of the two integers around the exact t
            for i in range(n):
                t = _exact_t(xs[w][i], sc[0], L)
                assert abs(Fraction(int(q[i])) - t) < 1 + Fraction(1, 10 ** 4)
                assert 0 <= q[i] <= L
            big = sum(int(v) << (i * bits) for i, v in enumerate(q.tolist()))
            assert c.astype("<u4").tobytes() == big.to_bytes(4 * ((n * bits + 31) // 32), "little")
            codes.append(c), scales.append(sc), qs.append(q)
        # exact-rational server step, one rounding per named operation
        acc_ref = []
        for i in range(n):
            tot = None
            for w in range(W):
                hstep = round_to_f32(f32_to_fraction(scales[w][0]) / L)
                xh = round_to_f32(Fraction(2 * int(qs[w][i]) - L) * Fraction(hstep))
                tot = xh if tot is None else round_to_f32(Fraction(tot) + Fraction(xh))
            acc_ref.append(tot)
        p_ref = [round_to_f32(f32_to_fraction(p0[i]) - f32_to_fraction(lr) * Fraction(acc_ref[i]))
                 for i in range(n)]
        p = p0.copy()
        p, acc = O.server_step(codes, scales, bits, n, n, p, float(lr), want_acc=True)
        assert [f32_bits(float(v)) for v in acc] == [f32_bits(v) for v in acc_ref]
        assert [f32_bits(float(v)) for v in p] == [f32_bits(v) for v in p_ref]
        acc2 = O.dequant_accumulate(codes, scales, bits, n, n)
        assert np.array_equal(acc2, acc)


# ---------------------------------------------------------------- special cases of the server step
@pytest.mark.parametrize("bits", [1, 3, 8])
def test_identical_workers_sum_exactly(bits):
    n, B = 2048 + 17, 256
    x = (np.random.default_rng(1).standard_normal(n) * 1e-2).astype(np.float32)
    c, sc = O.quantize(x, bits, B, seed=9)
    xh = O.dequantize(O.unpack(c, n, bits), bits, B, sc)
    for W in (1, 2, 3, 4, 8):
        acc = O.dequant_accumulate([c] * W, [sc] * W, bits, n, B)
        if W <= 2:
            assert np.array_equal(acc, np.float32(W) * xh)  # x and x + x are exact
        # worker-ordered sum, one rounding per addition: a double holds the sum of two
        # floats of like magnitude exactly, so rounding it to float32 is that one rounding
        want = xh.copy()
        for _ in range(W - 1):
            want = (want.astype(np.float64) + xh.astype(np.float64)).astype(np.float32)
        assert np.array_equal(acc, want)
    p = np.zeros(n, np.float32)
    O.server_step([c], [sc], bits, n, B, p, 1.0)
    assert np.array_equal(p, -xh)                            # W = 1, lr = 1: w - x^
    base = np.full(n, 1.5, np.float32)
    out = O.dequant_accumulate([c], [sc], bits, n, B, acc=base)
    assert np.array_equal(out, base + xh)


def test_apply_is_a_single_rounding():
    rng = np.random.default_rng(5)
    p = rng.standard_normal(4096).astype(np.float32)
    g = rng.standard_normal(4096).astype(np.float32)
    lr = np.float32(0.1)
    want = (p.astype(np.float64) - np.float64(lr) * g.astype(np.float64)).astype(np.float32)
    got = O.apply(p.copy(), g, float(lr))
    # double arithmetic holds the 48-bit product exactly; the only inexact step is the
    # addition, whose double rounding can differ from a fused one in ~2^-29 of the cases
    assert (got != want).mean() < 1e-3
    assert np.abs(got.astype(np.float64) - want).max() <= np.spacing(np.abs(want)).max()
    unfused = p - lr * g
    assert (got != unfused).any()                # a two-rounding update would differ


# ---------------------------------------------------------------- bf16 widening (R1)
def test_bf16_widening_is_exact():
    import torch
    bits16 = np.arange(0, 65536, dtype=np.uint16)
    got = O.widen_bf16(bits16)
    ref = torch.from_numpy(bits16.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.array_equal(got.view(np.uint32), bits16.astype(np.uint32) << 16)


# ---------------------------------------------------------------- Philox (R7)
_TRITON_PROBE = r'''
import os, sys, json
os.environ["TRITON_INTERPRET"] = "1"
import numpy as np, torch, triton, triton.language as tl

@triton.jit
def k(out_ptr, c_ptr, N: tl.constexpr):
    o = tl.arange(0, N)
    c0 = tl.load(c_ptr + o); c1 = tl.load(c_ptr + N + o)
    c2 = tl.load(c_ptr + 2 * N + o); c3 = tl.load(c_ptr + 3 * N + o)
    k0 = tl.load(c_ptr + 4 * N + o); k1 = tl.load(c_ptr + 5 * N + o)
    a, b, c, d = tl.philox_impl(c0, c1, c2, c3, k0, k1, 10)
    tl.store(out_ptr + o, a); tl.store(out_ptr + N + o, b)
    tl.store(out_ptr + 2 * N + o, c); tl.store(out_ptr + 3 * N + o, d)

N = 64
inp = np.load(sys.argv[1])
out = torch.zeros(4 * N, dtype=torch.uint32)
k[(1,)](out, torch.from_numpy(inp.reshape(-1)), N)
np.save(sys.argv[2], out.numpy().reshape(4, N))
'''


def test_philox_matches_an_independent_library(tmp_path):
    """Philox4x32-10 of the checker against Triton's own implementation run by its
    CPU interpreter (an independent statement of the published generator)."""
    pytest.importorskip("triton")
    rng = np.random.default_rng(11)
    N = 64
    inp = rng.integers(0, 2 ** 32, (6, N), dtype=np.uint64).astype(np.uint32)
    inp[:, 0] = 0                       # all-zero counter and key
    inp[:, 1] = 0xFFFFFFFF              # all-ones counter and key
    inp[:, 2] = [1, 0, 0, 0, 0, 0]
    a, b = tmp_path / "in.npy", tmp_path / "out.npy"
    np.save(a, inp)
    script = tmp_path / "probe.py"
    script.write_text(_TRITON_PROBE)
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, str(script), str(a), str(b)], env=env,
                       capture_output=True, text=True, timeout=600)
    # Triton is importable here, so its interpreter not running is a failure, not a skip: without this
    # test the generator would silently lose its independent pin
    assert r.returncode == 0, "Triton's CPU interpreter did not run: " + r.stderr[-600:]
    ref = np.load(b)
    for j in range(N):
        got = O.philox4x32_10(inp[0:4, j], inp[4:6, j])
        assert np.array_equal(got, ref[:, j]), j


def _philox_python(ctr, key):
    """Restatement with Python integers (a cross-check, not a pin)."""
    c = list(ctr)
    k = list(key)
    for r in range(10):
        if r:
            k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
    return c


def test_draw_layout_counter_key_and_field():
    """Element g uses half (g&1) of word ((g&7)>>1) of the block with counter
    (lo(g>>3), hi(g>>3), worker, step) and key (lo(seed), hi(seed))."""
    seed = 0x1234567890ABCDEF
    off = (1 << 35) + 5                              # crosses 32 bits of the block index
    h = O.draw_h(seed, 6, 77, off, 40)
    for i in range(40):
        g = off + i
        blk = g >> 3
        y = _philox_python([blk & 0xFFFFFFFF, blk >> 32, 6, 77],
                           [seed & 0xFFFFFFFF, seed >> 32])
        e = g & 7
        assert h[i] == (y[e >> 1] >> (16 * (e & 1))) & 0xFFFF
    # an offset only shifts the stream
    assert np.array_equal(O.draw_h(seed, 6, 77, 0, 64)[24:], O.draw_h(seed, 6, 77, 24, 40))


def test_draw_statistics_and_stream_separation():
    n = 1 << 20
    h = O.draw_h(0, 0, 0, 0, n).astype(np.int64)
    assert abs(h.mean() - 32767.5) < 5 * 65536 / math.sqrt(12 * n)
    counts = np.bincount(h >> 8, minlength=256)
    chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
    assert 150 < chi2 < 380                          # 255 dof
    base = O.draw_h(0, 0, 0, 0, 4096)
    for other in (O.draw_h(1, 0, 0, 0, 4096), O.draw_h(0, 1, 0, 0, 4096),
                  O.draw_h(0, 0, 1, 0, 4096), O.draw_h(1 << 32, 0, 0, 0, 4096)):
        assert (other == base).mean() < 0.01


# ---------------------------------------------------------------- composition
@pytest.mark.parametrize("bits", [2, 5])
def test_quantize_is_the_composition_of_its_steps(bits):
    n, B = 5000, 512
    x = (np.random.default_rng(2).standard_normal(n) * 1e-3).astype(np.float32)
    codes, sc = O.quantize(x, bits, B, seed=4, worker=2, step=9, elem_offset=4096)
    sc2 = O.bucket_scales(x, B)
    h = O.draw_h(4, 2, 9, 4096, n)
    q = O.encode(x, bits, B, sc2, h)
    assert np.array_equal(sc, sc2) and np.array_equal(codes, O.pack(q, bits))
    # a bucket can be checked in isolation through elem_offset
    c1, s1 = O.quantize(x[1024:1536], bits, B, seed=4, worker=2, step=9, elem_offset=4096 + 1024)
    assert s1[0] == sc[2]
    assert np.array_equal(O.unpack(c1, 512, bits), q[1024:1536])


def test_segments_are_buckets_with_word_aligned_streams():
    sizes = [96, 1000, 7, 0, 4096, 33]
    seg = np.zeros(len(sizes) + 1, np.uint64)
    seg[1:] = np.cumsum(sizes)
    rng = np.random.default_rng(8)
    x = rng.standard_normal(int(seg[-1])).astype(np.float32)
    for bits in (3, 8):
        coff = np.zeros(len(sizes) + 1, np.uint64)
        coff[1:] = np.cumsum([(s * bits + 31) // 32 for s in sizes])
        codes, sc = O.quantize_segments(x, seg, coff, bits, seed=1, worker=3, step=0, elem_offset=64)
        for j, s in enumerate(sizes):
            if s == 0:
                assert sc[j] == 0
                continue
            lo = int(seg[j])
            c, s1 = O.quantize(x[lo:lo + s], bits, s, seed=1, worker=3, step=0, elem_offset=64 + lo)
            assert s1[0] == sc[j] == np.abs(x[lo:lo + s]).max()
            assert np.array_equal(codes[int(coff[j]):int(coff[j + 1])], c)
        p = rng.standard_normal(x.size).astype(np.float32)
        p2 = p.copy()
        O.server_step_segments([codes, codes], [sc, sc], bits, seg, coff, p, 0.25)
        for j, s in enumerate(sizes):
            lo = int(seg[j])
            if s:
                O.server_step([codes[int(coff[j]):]] * 2, [sc[j:j + 1]] * 2, bits, s, s,
                              p2[lo:lo + s], 0.25)
        assert np.array_equal(p, p2)


# ---------------------------------------------------------------- downlink re-quantization
@pytest.mark.parametrize("bits", [1, 2, 5, 8])
def test_requantize_is_mean_then_quantize_and_fixes_grid_points(bits):
    L = (1 << bits) - 1
    n, B, W = 3000, 512, 4
    rng = np.random.default_rng(60 + bits)
    xs = [(rng.standard_normal(n) * 1e-3).astype(np.float32) for _ in range(W)]
    enc = [O.quantize(x, bits, B, 11, worker=w) for w, x in enumerate(xs)]
    codes, scales = [e[0] for e in enc], [e[1] for e in enc]
    c2, s2 = O.server_requantize(codes, scales, bits, n, B, 0.25, seed=11, worker=99, step=4)
    mean = (O.dequant_accumulate(codes, scales, bits, n, B).astype(np.float64) * 0.25).astype(np.float32)
    want_c, want_s = O.quantize(mean, bits, B, 11, worker=99, step=4)
    assert np.array_equal(c2, want_c) and np.array_equal(s2, want_s)
    assert np.array_equal(s2, O.bucket_scales(mean, B))
    # one worker whose scale is L * 2^e decodes onto its own grid: re-quantizing the "mean" of
    # that single worker returns its codes and scale, whatever the draws
    q0 = rng.integers(0, L + 1, 512, dtype=np.uint8)
    q0[0], q0[1] = L, 0
    sc = np.array([L * 2.0 ** -9], np.float32)
    c1 = O.pack(q0, bits)
    for seed in (0, 5):
        c3, s3 = O.server_requantize([c1], [sc], bits, 512, 512, 1.0, seed=seed, worker=7)
        assert np.array_equal(c3, c1) and s3[0] == sc[0]
