"""Parity of the CUDA path (through the C ABI binding) with the CPU checker, element by
element on the same seeded inputs.

Bars: packed codes and scales bit-exact (the benchmark spec allows elements within one ulp
of a rounding threshold to differ, at most 1e-6 of n; none are expected because both
sides perform the same IEEE operations, and the count is asserted to be 0); accumulated
gradients and updated parameters bit-exact as well, with max relative error <= 1e-6
asserted separately as the stated bar."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, max_rel_err, to_dev

pytestmark = pytest.mark.gpu
ALL_BITS = list(range(1, 9))


@pytest.fixture(autouse=True)
def no_kernel_wait_gave_up():
    yield
    assert mqg.mqg_device_timeouts() == 0, "a kernel's bounded wait ran out"


def gpu_quantize(x, bits, bucket, seed, worker=0, step=0, elem_offset=0, bf16=False):
    n = x.size
    if bf16:
        g = to_dev(x.view(np.int16)).view(torch.bfloat16)
    else:
        g = to_dev(x)
    codes = Guarded(mqg.mqg_code_words(n, bits), torch.int32)
    scales = Guarded(mqg.mqg_num_buckets(n, bucket), torch.float32)
    mqg.mqg_quantize(g, n, bits, bucket, seed, codes.view, scales.view, worker, step, elem_offset)
    torch.cuda.synchronize()
    codes.check_guards(), scales.check_guards()
    return codes.numpy(np.uint32), scales.numpy(np.float32)


def assert_quantize_parity(x, bits, bucket, seed, worker=0, step=0, elem_offset=0, bf16=False):
    c_gpu, s_gpu = gpu_quantize(x, bits, bucket, seed, worker, step, elem_offset, bf16)
    c_ref, s_ref = O.quantize(x, bits, bucket, seed, worker, step, elem_offset,
                              dtype="bf16" if bf16 else "f32")
    assert bits_equal(s_gpu, s_ref) == 0, "scales differ"
    bad_words = int((c_gpu != c_ref).sum())
    if bad_words:
        q_gpu, q_ref = O.unpack(c_gpu, x.size, bits), O.unpack(c_ref, x.size, bits)
        idx = np.nonzero(q_gpu != q_ref)[0]
        raise AssertionError("%d codes differ (first at %s: gpu %s, ref %s), %d words"
                             % (idx.size, idx[:5], q_gpu[idx[:5]], q_ref[idx[:5]], bad_words))
    return c_ref, s_ref


# ------------------------------------------------------------------ quantize + pack
@pytest.mark.parametrize("bits", ALL_BITS)
def test_quantize_config1_shape(bits):
    """n = 2^20, N(0, 1e-3), bucket 512, Philox seed 0 (the small configuration)."""
    x = wl.normal(1 << 20, 1e-3, config=1, worker=1)
    assert_quantize_parity(x, bits, 512, seed=0, worker=1)


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("n,bucket", [
    (1, 32), (7, 32), (31, 32), (32, 32), (33, 32), (511, 512), (513, 512), (8192 + 5, 2048),
    (3 * 8192 + 2048 + 64, 2048), (20000, 4096), (100_003, 8192), (9000, 96), (70_000, 1056),
    (5000, 10_000), (40, 64),
])
def test_quantize_shapes_and_ragged_tails(bits, n, bucket):
    x = wl.normal(n, 3e-3, config=11, worker=bits)
    assert_quantize_parity(x, bits, bucket, seed=n, worker=3, step=bits)


@pytest.mark.parametrize("bits", [1, 3, 4, 7, 8])
@pytest.mark.parametrize("elem_offset", [8, 4096, (1 << 35) + 64, 3, 2049, (1 << 40) + 5,
                                         (1 << 35) - 16, (1 << 35) - 8 * 4 * 5 - 8, (1 << 35) - 13])
def test_quantize_elem_offset(bits, elem_offset):
    """Offsets that are block-aligned or not, beyond 32 bits, and whose Philox block index
    crosses 2^32 inside a row and between rows."""
    x = wl.normal(10_000, 1e-3, config=12, worker=0)
    assert_quantize_parity(x, bits, 512, seed=0xFEDCBA9876543210, worker=5, step=17,
                           elem_offset=elem_offset)


@pytest.mark.parametrize("bits", [1, 2, 5, 8])
@pytest.mark.parametrize("n,bucket", [(100_000, 16384), (50_000, 50_000), (70_001, 1 << 20),
                                      (9001, 9001), (3 * 32768 + 77, 32768)])
def test_quantize_buckets_larger_than_a_tile(bits, n, bucket):
    x = wl.laplace(n, 1e-4, config=13, worker=1)
    assert_quantize_parity(x, bits, bucket, seed=5, worker=2)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_quantize_bf16_heavy_tailed_with_zeros(bits):
    xb = wl.student_t_bf16(200_000 + 13, config=5, worker=2, zero_frac=0.01)
    assert (xb == 0).sum() > 100
    assert_quantize_parity(xb, bits, 4096, seed=5, worker=2, bf16=True)
    assert_quantize_parity(xb[:70_000], bits, 32768, seed=5, worker=2, bf16=True)


@pytest.mark.parametrize("bits", [1, 4, 7])
def test_quantize_degenerate_values(bits):
    n, B = 4096, 512
    x = wl.normal(n, 1.0, config=14)
    x[0:512] = 0.0                                     # an all-zero bucket
    x[512:1024] = np.float32(1e-30)                    # below the flush limit
    x[1024:1536] = np.float32(2.0 ** -96)              # exactly at the limit
    x[1536:2048] *= np.float32(1e-38)                  # denormal products
    x[2048:2560] = np.float32(-3.25)                   # constant bucket: every x = -s
    x[2560] = np.float32(1e30)                         # one huge value
    c, s = assert_quantize_parity(x, bits, B, seed=1)
    assert s[0] == 0 and s[1] == 0 and s[2] == np.float32(2.0 ** -96)
    q = O.unpack(c, n, bits)
    assert not q[:1024].any() and not q[2048:2560].any()


def test_quantize_is_a_pure_function_of_its_arguments():
    x = wl.normal(50_000, 1e-3, config=15)
    a = gpu_quantize(x, 3, 512, seed=9, worker=1, step=2)
    b = gpu_quantize(x, 3, 512, seed=9, worker=1, step=2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    for kw in (dict(seed=10, worker=1, step=2), dict(seed=9, worker=2, step=2),
               dict(seed=9, worker=1, step=3)):
        c = gpu_quantize(x, 3, 512, **kw)
        assert (c[0] != a[0]).mean() > 0.3


def test_zero_elements_is_a_no_op():
    e = torch.zeros(0, device="cuda")
    ei = torch.zeros(0, dtype=torch.int32, device="cuda")
    mqg.mqg_quantize(e, 0, 4, 512, 0, ei, e)
    mqg.mqg_server_step([ei], [e], 1, 4, 0, 512, e, 0.1)
    mqg.mqg_dequant_accumulate([ei], [e], 1, 4, 0, e, 512)
    mqg.mqg_apply(e, e, 0.1, 0)
    torch.cuda.synchronize()


# ------------------------------------------------------------------ server side
def oracle_workers(xs, bits, bucket, seed):
    out = [O.quantize(x, bits, bucket, seed, worker=w) for w, x in enumerate(xs)]
    return [c for c, _ in out], [s for _, s in out]


def run_server(codes, scales, bits, n, bucket, params, lr, want_acc):
    dc = [to_dev(c.view(np.int32)) for c in codes]
    ds = [to_dev(s) for s in scales]
    p = Guarded(n, torch.float32, fill=params)
    acc = Guarded(n, torch.float32) if want_acc else None
    mqg.mqg_server_step(dc, ds, len(dc), bits, n, bucket, p.view, lr, acc.view if want_acc else None)
    torch.cuda.synchronize()
    p.check_guards()
    if want_acc:
        acc.check_guards()
    return p.numpy(np.float32), (acc.numpy(np.float32) if want_acc else None)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_server_step_config1(bits):
    """W = 4, n = 2^20, bucket 512, params N(0, 0.05), lr 0.1: one full step."""
    n, W, B = 1 << 20, 4, 512
    xs = [wl.normal(n, 1e-3, config=1, worker=w) for w in range(W)]
    codes, scales = oracle_workers(xs, bits, B, seed=0)
    p0 = wl.params(n, 0.05, config=1)
    p_ref, acc_ref = O.server_step(codes, scales, bits, n, B, p0.copy(), 0.1, want_acc=True)
    p, acc = run_server(codes, scales, bits, n, B, p0, 0.1, True)
    assert max_rel_err(acc, acc_ref) <= 1e-6 and max_rel_err(p, p_ref) <= 1e-6
    assert bits_equal(acc, acc_ref) == 0 and bits_equal(p, p_ref) == 0


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("n,bucket,W", [(1, 32, 1), (33, 32, 2), (8192 + 5, 2048, 3),
                                        (100_003, 4096, 5), (9000, 96, 2), (5000, 10_000, 4),
                                        (3 * 32768 + 77, 32768, 2), (65_536 + 31, 512, 32),
                                        # buckets shorter than a 32-row tile that still take the TMA-fed kernel
                                        # (16, 24, 28, 30, 31 rows) and one that does not (20 rows)
                                        (40_000 + 5, 768, 3), (50_000, 896, 2), (33_333, 960, 2),
                                        (70_001, 992, 3), (30_000, 640, 2),
                                        # buckets of 8, 4, 2, 1 rows: TMA-fed for few workers, else the general kernel
                                        (50_000 + 3, 256, 8), (50_000, 256, 20), (40_000 + 7, 128, 8),
                                        (40_000, 64, 4), (30_000, 32, 2), (30_000 + 1, 32, 3)])
def test_server_step_shapes(bits, n, bucket, W):
    xs = [wl.normal(n, 2e-3, config=21, worker=w) for w in range(W)]
    xs[0][: min(n, 40)] = 0.0
    if n >= bucket:
        xs[W - 1][:bucket] = 0.0                       # a flushed bucket on one worker
    codes, scales = oracle_workers(xs, bits, bucket, seed=bits)
    p0 = wl.params(n, 0.05, config=21)
    lr = 0.1 / W
    p_ref, acc_ref = O.server_step(codes, scales, bits, n, bucket, p0.copy(), lr, want_acc=True)
    p, acc = run_server(codes, scales, bits, n, bucket, p0, lr, True)
    assert bits_equal(acc, acc_ref) == 0 and bits_equal(p, p_ref) == 0
    p2, _ = run_server(codes, scales, bits, n, bucket, p0, lr, False)
    assert bits_equal(p2, p_ref) == 0


@pytest.mark.parametrize("bits", [1, 3, 4, 6, 8])
@pytest.mark.parametrize("n,B", [(50_000 + 9, 512), (300_000 + 9, 2048), (8 * 4096 * 33, 4096), (70_000, 1 << 20)])
def test_dequant_accumulate_then_apply_equals_fused(bits, n, B):
    W = 4
    xs = [wl.laplace(n, 1e-4, config=22, worker=w) for w in range(W)]
    codes, scales = oracle_workers(xs, bits, B, seed=3)
    dc = [to_dev(c.view(np.int32)) for c in codes]
    ds = [to_dev(s) for s in scales]
    acc = Guarded(n, torch.float32)
    mqg.mqg_dequant_accumulate(dc, ds, W, bits, n, acc.view, B)
    torch.cuda.synchronize()
    acc.check_guards()
    acc_ref = O.dequant_accumulate(codes, scales, bits, n, B)
    assert bits_equal(acc.numpy(np.float32), acc_ref) == 0
    # continue the sum from an existing accumulator (two halves of the workers)
    acc2 = Guarded(n, torch.float32)
    mqg.mqg_dequant_accumulate(dc[:2], ds[:2], 2, bits, n, acc2.view, B)
    mqg.mqg_dequant_accumulate(dc[2:], ds[2:], 2, bits, n, acc2.view, B, add_into_acc=True)
    torch.cuda.synchronize()
    acc2.check_guards()
    assert bits_equal(acc2.numpy(np.float32), acc_ref) == 0
    # apply
    p0 = wl.params(n, 0.05, config=22)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_apply(p.view, acc.view, 0.025, n)
    torch.cuda.synchronize()
    p.check_guards()
    p_ref = O.apply(p0.copy(), acc_ref, 0.025)
    assert bits_equal(p.numpy(np.float32), p_ref) == 0
    p_fused, _ = run_server(codes, scales, bits, n, B, p0, 0.025, False)
    assert bits_equal(p_fused, p_ref) == 0


@pytest.mark.parametrize("n", [1, 3, 4, 5, 1023, 1 << 16])
def test_apply_tails(n):
    rng = np.random.default_rng(n)
    p0 = rng.standard_normal(n).astype(np.float32)
    g = rng.standard_normal(n).astype(np.float32)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_apply(p.view, to_dev(g), 0.3, n)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), O.apply(p0.copy(), g, 0.3)) == 0


# ------------------------------------------------------------------ per-layer segments
def _segments(sizes, bits):
    seg = np.zeros(len(sizes) + 1, np.uint64)
    seg[1:] = np.cumsum(sizes)
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum([O.code_words(s, bits) for s in sizes])
    return seg, coff


@pytest.mark.parametrize("bits", ALL_BITS)
def test_segments_quantize_and_server(bits):
    sizes = [96, 1000, 7, 0, 34_848, 33, 20_000, 256, 8192, 8193, 1]
    W = 3
    seg, coff = _segments(sizes, bits)
    n = int(seg[-1])
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(W)]
    refs = [O.quantize_segments(x, seg, coff, bits, seed=3, worker=w, step=1, elem_offset=64)
            for w, x in enumerate(xs)]
    for w, x in enumerate(xs):
        codes = Guarded(int(coff[-1]), torch.int32)
        scales = Guarded(len(sizes), torch.float32)
        mqg.mqg_quantize_segments(to_dev(x), seg, coff, bits, 3, codes.view, scales.view,
                                  worker=w, step=1, elem_offset=64)
        torch.cuda.synchronize()
        codes.check_guards(), scales.check_guards()
        assert bits_equal(scales.numpy(np.float32), refs[w][1]) == 0
        got = codes.numpy(np.uint32)
        for j, s in enumerate(sizes):       # words between streams are not part of the result
            lo = int(coff[j])
            nw = O.code_words(s, bits)
            assert np.array_equal(got[lo:lo + nw], refs[w][0][lo:lo + nw]), (w, j)
    codes = [r[0] for r in refs]
    scales = [r[1] for r in refs]
    p0 = wl.params(n, 0.05, config=3)
    p_ref, acc_ref = O.server_step_segments(codes, scales, bits, seg, coff, p0.copy(), 0.05,
                                            want_acc=True)
    p = Guarded(n, torch.float32, fill=p0)
    acc = Guarded(n, torch.float32)
    mqg.mqg_server_step_segments([to_dev(c.view(np.int32)) for c in codes],
                                 [to_dev(s) for s in scales], W, bits, seg, coff, p.view, 0.05,
                                 acc.view)
    torch.cuda.synchronize()
    p.check_guards(), acc.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0
    assert bits_equal(acc.numpy(np.float32), acc_ref) == 0


@pytest.mark.parametrize("bits", [1, 3, 8])
def test_segments_long_segments_take_their_own_launches(bits):
    """Segments of a million elements and more go to the TMA-fed kernel when their buffers are
    16-byte aligned (the second one here, ragged length included) and stay in the table-driven
    launch otherwise (the fourth one starts on an odd word); both must match the checker."""
    sizes = [128, (1 << 20) + 37, 5, (1 << 20) + 64, 100]
    W = 3
    seg, coff = _segments(sizes, bits)
    n = int(seg[-1])
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(W)]
    xs[1][128:128 + (1 << 20) + 37] = np.float32(1e-30)     # a long segment whose maximum is flushed to 0
    refs = [O.quantize_segments(x, seg, coff, bits, seed=5, worker=w) for w, x in enumerate(xs)]
    codes, scales = [r[0] for r in refs], [r[1] for r in refs]
    for w in (0, 1):                                        # the quantizer routes long segments too
        dc = Guarded(int(coff[-1]), torch.int32)
        ds = Guarded(len(sizes), torch.float32)
        mqg.mqg_quantize_segments(to_dev(xs[w]), seg, coff, bits, 5, dc.view, ds.view, worker=w)
        torch.cuda.synchronize()
        dc.check_guards(), ds.check_guards()
        assert bits_equal(ds.numpy(np.float32), scales[w]) == 0
        got = dc.numpy(np.uint32)
        for j, sz in enumerate(sizes):
            lo, nw = int(coff[j]), O.code_words(sz, bits)
            assert np.array_equal(got[lo:lo + nw], codes[w][lo:lo + nw]), (w, j)
    assert scales[1][1] == 0 and scales[0][1] > 0
    p0 = wl.params(n, 0.05, config=3)
    p_ref, _ = O.server_step_segments(codes, scales, bits, seg, coff, p0.copy(), 0.05)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_segments([to_dev(c.view(np.int32)) for c in codes], [to_dev(s) for s in scales],
                                 W, bits, seg, coff, p.view, 0.05)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0
    assert mqg.mqg_device_timeouts() == 0


def test_segments_more_long_segments_than_one_server_launch_holds():
    """18 long segments (16 per launch of the segment server kernel; a segment is long from 32,768 elements
    on) between short ones, ragged lengths."""
    bits, W = 5, 2
    sizes = []
    for j in range(18):                  # multiples of 128 elements keep every segment's buffers 16-byte aligned
        sizes += [((1 << 20) if j % 2 == 0 else (1 << 15)) + 128 * j, 128 * (1 + j % 3)]
    sizes[-2] += 7                       # the last long segment ends with a ragged row
    sizes[-1] = 45
    seg, coff = _segments(sizes, bits)
    n = int(seg[-1])
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(W)]
    refs = [O.quantize_segments(x, seg, coff, bits, seed=6, worker=w) for w, x in enumerate(xs)]
    codes, scales = [r[0] for r in refs], [r[1] for r in refs]
    p0 = wl.params(n, 0.05, config=3)
    p_ref, _ = O.server_step_segments(codes, scales, bits, seg, coff, p0.copy(), 0.05)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_segments([to_dev(c.view(np.int32)) for c in codes], [to_dev(s) for s in scales],
                                 W, bits, seg, coff, p.view, 0.05)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0


def test_segments_more_than_one_launch_chunk():
    rng = np.random.default_rng(0)
    sizes = [int(v) for v in rng.integers(0, 600, 150)]
    bits = 5
    seg, coff = _segments(sizes, bits)
    x = wl.layered(sizes, config=31)
    c_ref, s_ref = O.quantize_segments(x, seg, coff, bits, seed=8)
    codes = Guarded(int(coff[-1]), torch.int32)
    scales = Guarded(len(sizes), torch.float32)
    mqg.mqg_quantize_segments(to_dev(x), seg, coff, bits, 8, codes.view, scales.view)
    torch.cuda.synchronize()
    codes.check_guards(), scales.check_guards()
    assert bits_equal(scales.numpy(np.float32), s_ref) == 0
    assert np.array_equal(codes.numpy(np.uint32), c_ref)     # streams are back to back here


# ------------------------------------------------------------------ downlink: server re-quantization
@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("n,bucket,W", [(40, 64, 1), (8192 + 5, 2048, 3), (100_003, 4096, 4), (9000, 96, 2),
                                        (5000, 10_000 - 1808, 5), (65_536 + 31, 512, 8),
                                        # whole rows, power-of-two buckets: the warp-pipelined kernel (buckets
                                        # held by two warps, four warps, one warp, parts of a warp; short last
                                        # buckets; worker counts that do not fill a code stage; 32 workers)
                                        ((1 << 17) + 64, 2048, 8), ((1 << 17) + 5 * 1024, 4096, 3), (99_968, 1024, 5),
                                        (32_768 + 64, 256, 8), (16_384 + 32, 32, 2), (22_400, 64, 4),
                                        (1 << 15, 2048, 32), ((1 << 16) + 2048 + 32, 2048, 9), (1 << 16, 2048, 1)])
def test_server_requantize(bits, n, bucket, W):
    xs = [wl.normal(n, 2e-3, config=41, worker=w) for w in range(W)]
    if n >= bucket:
        for x in xs:
            x[:bucket] = 0.0                            # a bucket whose mean is exactly zero
    codes, scales = oracle_workers(xs, bits, bucket, seed=bits)
    c_ref, s_ref = O.server_requantize(codes, scales, bits, n, bucket, 1.0 / W, seed=bits, worker=1000, step=3)
    out_c = Guarded(mqg.mqg_code_words(n, bits), torch.int32)
    out_s = Guarded(mqg.mqg_num_buckets(n, bucket), torch.float32)
    mqg.mqg_server_requantize([to_dev(c.view(np.int32)) for c in codes], [to_dev(s) for s in scales], W, bits,
                              n, bucket, 1.0 / W, bits, out_c.view, out_s.view, worker=1000, step=3)
    torch.cuda.synchronize()
    out_c.check_guards(), out_s.check_guards()
    assert bits_equal(out_s.numpy(np.float32), s_ref) == 0
    assert np.array_equal(out_c.numpy(np.uint32), c_ref)
    # the worker side of the downlink: de-quantize the broadcast and update (W = 1)
    p0 = wl.params(n, 0.05, config=41)
    p_ref, _ = O.server_step([c_ref], [s_ref], bits, n, bucket, p0.copy(), 0.1)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step([out_c.view], [out_s.view], 1, bits, n, bucket, p.view, 0.1)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0


def test_server_requantize_rejects_large_buckets():
    e = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(mqg.MqgError):
        mqg.mqg_server_requantize([e], [e.view(torch.float32)], 1, 4, 100_000, 16384, 1.0, 0, e, e.view(torch.float32))
