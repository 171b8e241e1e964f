"""Parity of the (min, max) nearest-rounding codec variant (CUDA, through the C ABI binding)
with the CPU checker, element by element on the same seeded inputs: packed codes and ranges bit
for bit, sums and parameters bit for bit (the stated bar for floating point is 1e-6 relative;
both sides perform the same IEEE operations, so equality is asserted)."""
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


def gpu_quantize(x, bits, bucket, bf16=False):
    n = x.size
    g = to_dev(x.view(np.int16)).view(torch.bfloat16) if bf16 else to_dev(x)
    codes = Guarded(mqg.mqg_code_words(n, bits), torch.int32)
    ranges = Guarded(2 * mqg.mqg_num_buckets(n, bucket), torch.float32)
    mqg.mqg_quantize_minmax(g, n, bits, bucket, codes.view, ranges.view)
    torch.cuda.synchronize()
    codes.check_guards(), ranges.check_guards()
    return codes, ranges


def assert_quantize_parity(x, bits, bucket, bf16=False):
    codes, ranges = gpu_quantize(x, bits, bucket, bf16)
    c_ref, r_ref = O.quantize_minmax(x, bits, bucket, dtype="bf16" if bf16 else "f32")
    assert bits_equal(ranges.numpy(np.float32), r_ref) == 0, "ranges differ"
    c_gpu = codes.numpy(np.uint32)
    if not np.array_equal(c_gpu, c_ref):
        q_gpu, q_ref = O.unpack(c_gpu, x.size, bits), O.unpack(c_ref, x.size, bits)
        idx = np.nonzero(q_gpu != q_ref)[0]
        raise AssertionError("%d codes differ (first at %s: gpu %s, ref %s)"
                             % (idx.size, idx[:5], q_gpu[idx[:5]], q_ref[idx[:5]]))
    return codes, ranges, c_ref, r_ref


@pytest.mark.parametrize("bits", ALL_BITS)
def test_quantize_small_configuration(bits):
    """n = 2^20, N(0, 1e-3), bucket 512: whole tiles of the one-pass kernel, shuffle buckets."""
    assert_quantize_parity(wl.normal(1 << 20, 1e-3, config=1, worker=2), bits, 512)


@pytest.mark.parametrize("bits", [1, 3, 4, 8])
@pytest.mark.parametrize("n,bucket", [
    (3 * 4096 * 7 + 2048 + 37, 2048),     # several tiles, ragged last tile and ragged last row
    (300_000 + 9, 4096),                  # the largest bucket of the one-pass kernel
    (40_000, 96),                         # buckets of three rows
    (2048, 2048), (2049, 1024),           # smallest one-pass shapes
    (1, 32), (31, 32), (33, 32), (1000, 256),      # below the one-pass kernel: general kernels
    (100_000, 16384), (70_001, 1 << 20), (50_000, 50_000), (65_536 + 32, 8192),   # big buckets: two passes
])
def test_quantize_shapes(bits, n, bucket):
    x = wl.laplace(n, 2e-3, config=2, worker=n % 7)
    assert_quantize_parity(x, bits, bucket)


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_quantize_one_sided_and_constant_buckets(bits):
    """All-positive and all-negative buckets (zero padding must not widen the range), constant
    buckets, buckets of zeros of both signs, a spread below the flush threshold."""
    n, bucket = 8192 + 2048 + 13, 2048
    x = np.abs(wl.normal(n, 1.0, config=1, worker=3)) + np.float32(0.5)
    x[2048:4096] *= np.float32(-1.0)
    x[4096:6144] = np.float32(0.25)
    x[6144:8192] = np.where(np.arange(2048) % 2 == 0, np.float32(0.0), np.float32(-0.0))
    x[8192:10240] = np.float32(1e-30) + np.float32(1e-31) * (np.arange(2048) % 3).astype(np.float32)
    assert_quantize_parity(x.astype(np.float32), bits, bucket)
    assert_quantize_parity(x[: 8192 + 2048 + 5].astype(np.float32), bits, 1 << 20)


@pytest.mark.parametrize("bits", [1, 4, 7])
def test_quantize_bf16(bits):
    x = wl.student_t_bf16(200_000 + 24, config=5, worker=1)
    assert_quantize_parity(x, bits, 2048, bf16=True)
    assert_quantize_parity(x[:70_001], bits, 1 << 20, bf16=True)


def encode_workers(xs, bits, bucket):
    enc = [O.quantize_minmax(x, bits, bucket) for x in xs]
    return [c for c, _ in enc], [r for _, r in enc]


@pytest.mark.parametrize("bits", ALL_BITS)
@pytest.mark.parametrize("n,bucket,W", [
    (300_000 + 9, 2048, 8),     # the TMA kernel, ragged last row
    (8 * 4096 * 5, 4096, 3),    # whole tiles
    (40_000, 96, 2),            # small buckets: the general kernel
    (33, 32, 2), (1, 32, 1),
    (70_000, 1 << 20, 5),       # a single bucket
    (50_000 + 3, 512, 6), (40_000 + 5, 768, 3), (50_000, 256, 8), (40_000 + 7, 128, 3), (30_000, 32, 2),
])
def test_server_step_and_accumulate(bits, n, bucket, W):
    xs = [wl.laplace(n, 10.0 ** (-3 + (w % 3)), config=2, worker=w) for w in range(W)]
    codes, ranges = encode_workers(xs, bits, bucket)
    dcodes, dranges = [to_dev(c.view(np.int32)) for c in codes], [to_dev(r) for r in ranges]
    p0 = wl.params(n, 0.05, config=2)
    lr = 0.1 / W

    acc_ref = O.dequant_accumulate_minmax(codes, ranges, bits, n, bucket)
    acc = Guarded(n, torch.float32)
    mqg.mqg_dequant_accumulate_minmax(dcodes, dranges, W, bits, n, acc.view, bucket)
    torch.cuda.synchronize()
    acc.check_guards()
    assert max_rel_err(acc.numpy(np.float32), acc_ref) <= 1e-6
    assert bits_equal(acc.numpy(np.float32), acc_ref) == 0

    acc2_ref = O.dequant_accumulate_minmax(codes, ranges, bits, n, bucket, acc=acc_ref)
    mqg.mqg_dequant_accumulate_minmax(dcodes, dranges, W, bits, n, acc.view, bucket, add_into_acc=True)
    torch.cuda.synchronize()
    acc.check_guards()
    assert bits_equal(acc.numpy(np.float32), acc2_ref) == 0

    p_ref, _ = O.server_step_minmax(codes, ranges, bits, n, bucket, p0.copy(), lr)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_minmax(dcodes, dranges, W, bits, n, bucket, p.view, lr)
    torch.cuda.synchronize()
    p.check_guards()
    assert max_rel_err(p.numpy(np.float32), p_ref) <= 1e-6
    assert bits_equal(p.numpy(np.float32), p_ref) == 0

    p2 = Guarded(n, torch.float32, fill=p0)
    acc_out = Guarded(n, torch.float32)
    mqg.mqg_server_step_minmax(dcodes, dranges, W, bits, n, bucket, p2.view, lr, acc_out.view)
    torch.cuda.synchronize()
    p2.check_guards(), acc_out.check_guards()
    assert bits_equal(p2.numpy(np.float32), p_ref) == 0
    assert bits_equal(acc_out.numpy(np.float32), acc_ref) == 0


@pytest.mark.parametrize("bits", [2, 8])
def test_quantize_then_server_round_trip_on_device(bits):
    """Codes and ranges written by the CUDA quantizer feed the CUDA server directly."""
    n, bucket, W = 1_000_000 + 40, 2048, 4
    xs = [wl.normal(n, 1e-3, config=1, worker=w) for w in range(W)]
    outs = [gpu_quantize(x, bits, bucket) for x in xs]
    codes, ranges = encode_workers(xs, bits, bucket)
    p0 = wl.params(n, 0.05, config=1)
    p_ref, _ = O.server_step_minmax(codes, ranges, bits, n, bucket, p0.copy(), 0.025)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_minmax([c.view for c, _ in outs], [r.view for _, r in outs], W, bits, n, bucket, p.view, 0.025)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0


def test_argument_errors_and_empty_input():
    n = 4096
    g = to_dev(wl.normal(n, 1.0, config=1, worker=0))
    c = torch.zeros(mqg.mqg_code_words(n, 4), dtype=torch.int32, device="cuda")
    r = torch.zeros(2 * mqg.mqg_num_buckets(n, 512) + 1, dtype=torch.float32, device="cuda")
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_minmax(g, n, 0, 512, c, r)
    assert e.value.status == mqg.MQG_ERR_BITS
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_minmax(g, n, 4, 48, c, r)
    assert e.value.status == mqg.MQG_ERR_INVALID
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_minmax(g, n, 4, 512, c, r[1:])
    assert e.value.status == mqg.MQG_ERR_ALIGN
    mqg.mqg_quantize_minmax(g, 0, 4, 512, c, r)
    mqg.mqg_server_step_minmax([c], [r], 1, 4, 0, 512, g, 0.1)


def assert_workers_parity(xs, bits, bucket, bf16=False):
    """mqg_quantize_workers_minmax (one launch for all workers) against the CPU checker, worker by worker."""
    W, n = len(xs), xs[0].size
    gs = [to_dev(x.view(np.int16)).view(torch.bfloat16) if bf16 else to_dev(x) for x in xs]
    codes = [Guarded(mqg.mqg_code_words(n, bits), torch.int32) for _ in range(W)]
    ranges = [Guarded(2 * mqg.mqg_num_buckets(n, bucket), torch.float32) for _ in range(W)]
    mqg.mqg_quantize_workers_minmax(gs, W, n, bits, bucket, [c.view for c in codes], [r.view for r in ranges])
    torch.cuda.synchronize()
    for w in range(W):
        codes[w].check_guards(), ranges[w].check_guards()
        c_ref, r_ref = O.quantize_minmax(xs[w], bits, bucket, dtype="bf16" if bf16 else "f32")
        assert bits_equal(ranges[w].numpy(np.float32), r_ref) == 0, "worker %d: ranges differ" % w
        assert np.array_equal(codes[w].numpy(np.uint32), c_ref), "worker %d: codes differ" % w


@pytest.mark.parametrize("bits", ALL_BITS)
def test_workers_in_one_launch(bits):
    """Four workers, bucket 2048, ragged last tile and ragged last row (its padding must not widen a range)."""
    n = 5 * 4096 * 9 + 2048 + 21
    xs = [wl.laplace(n, 1e-4, config=2, worker=w) + np.float32(1e-4 * w) for w in range(4)]
    assert_workers_parity(xs, bits, 2048)


@pytest.mark.parametrize("bits", [1, 4, 7])
@pytest.mark.parametrize("n,bucket", [
    (300_000 + 9, 4096), (70_000, 512), (40_000, 96),       # four warps; 16-row shuffles; a shape of W calls
    (1 << 20, 1024), (33, 32),
])
def test_workers_shapes(bits, n, bucket):
    xs = [wl.normal(n, 1e-3, config=1, worker=10 + w) for w in range(3)]
    xs[1][: min(n, bucket)] = np.float32(0.25)              # a constant bucket: every code 0
    assert_workers_parity(xs, bits, bucket)


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_workers_bf16(bits):
    n = 3 * 4096 * 11 + 4096
    xs = [wl.student_t_bf16(n, config=5, worker=w) for w in range(2)]
    assert_workers_parity(xs, bits, 4096, bf16=True)
