"""Parity of the 1-bit error-feedback variant (CUDA, through the C ABI binding) with the CPU
checker, element by element on the same seeded inputs: sign codes, class means and the residual
bit for bit over several iterations (the residual of one iteration is the input of the next),
then the (min, max) variant's server step with one bit on those outputs, bit for bit (the stated
bar for floating point is 1e-6 relative; both sides perform the same IEEE operations in the same
order, so equality is asserted)."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, to_dev

pytestmark = pytest.mark.gpu


def gpu_step(g_dev, res, n, bucket):
    codes = Guarded(mqg.mqg_code_words(n, 1), torch.int32)
    ranges = Guarded(2 * mqg.mqg_num_buckets(n, bucket), torch.float32)
    mqg.mqg_quantize_1bit_ef(g_dev, res.view, n, bucket, codes.view, ranges.view)
    torch.cuda.synchronize()
    codes.check_guards(), ranges.check_guards(), res.check_guards()
    return codes, ranges


def assert_parity(g, e0, bucket, iterations=1, bf16=False):
    n = g.size
    g_dev = to_dev(g.view(np.int16)).view(torch.bfloat16) if bf16 else to_dev(g)
    res = Guarded(n, torch.float32, fill=e0)
    e_ref = e0.copy()
    out = None
    for it in range(iterations):
        codes, ranges = gpu_step(g_dev, res, n, bucket)
        c_ref, r_ref, e_ref = O.quantize_1bit_ef(g, e_ref, bucket, dtype="bf16" if bf16 else "f32")
        assert bits_equal(ranges.numpy(np.float32), r_ref) == 0, "class means differ (iteration %d)" % it
        assert np.array_equal(codes.numpy(np.uint32), c_ref), "codes differ (iteration %d)" % it
        assert bits_equal(res.numpy(np.float32), e_ref) == 0, "residual differs (iteration %d)" % it
        out = (codes, ranges, c_ref, r_ref)
    return out


@pytest.mark.parametrize("n,bucket", [
    (1 << 20, 512),                          # buckets of 16 rows: lane shuffles
    (3 * 4096 * 7 + 2048 + 37, 2048),        # two warps per bucket, ragged last tile and row
    (300_000 + 9, 4096), (65_536 + 32, 8192),
    (40_000, 96), (9_000, 3072), (50_000, 5 * 32), (33_000, 7 * 32 * 4),
    (2048, 2048), (2049, 1024), (1, 32), (31, 32), (33, 32), (1000, 256), (64, 32),
    (5000, 8192), (8192, 8192), (8191, 1 << 20), (37, 100),
])
def test_shapes_three_iterations(n, bucket):
    g = wl.laplace(n, 1e-4, config=2, worker=n % 5)
    assert_parity(g, np.zeros(n, np.float32), bucket, iterations=3)


def test_special_buckets():
    """All-positive and all-negative buckets, zeros of both signs, an all-zero bucket, a spread
    below the flush threshold, values spread over many binades, a non-zero starting residual."""
    n, bucket = 6 * 2048 + 77, 2048
    rng = np.random.default_rng(9)
    g = (rng.standard_normal(n) * np.exp2(rng.integers(-12, 12, n))).astype(np.float32)
    g[:2048] = np.abs(g[:2048]) + np.float32(0.5)
    g[2048:4096] = -np.abs(g[2048:4096]) - np.float32(0.5)
    g[4096:6144] = np.where(np.arange(2048) % 2 == 0, np.float32(0.0), np.float32(-0.0))
    g[6144:8192] = np.float32(1e-30) * (np.arange(2048) % 3 - 1).astype(np.float32)
    e0 = (rng.standard_normal(n) * 0.25).astype(np.float32)
    e0[4096:8192] = 0.0
    assert_parity(g, e0, bucket, iterations=2)
    assert_parity(np.zeros(5000, np.float32), np.zeros(5000, np.float32), 1024)


def test_bf16_gradient():
    g = wl.student_t_bf16(200_000 + 24, config=5, worker=1)
    assert_parity(g, np.zeros(g.size, np.float32), 2048, iterations=2, bf16=True)


def test_buckets_above_the_one_pass_limit_and_bad_buffers_are_rejected():
    n = 20_000
    g = to_dev(wl.normal(n, 1.0))
    res = torch.zeros(n, dtype=torch.float32, device="cuda")
    codes = torch.zeros(mqg.mqg_code_words(n, 1), dtype=torch.int32, device="cuda")
    ranges = torch.zeros(4, dtype=torch.float32, device="cuda")
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_1bit_ef(g, res, n, 16_384, codes, ranges)
    assert e.value.status == mqg.MQG_ERR_INVALID
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_1bit_ef(g, res[1:], n - 1, 1 << 20, codes, ranges)
    assert e.value.status in (mqg.MQG_ERR_ALIGN, mqg.MQG_ERR_INVALID)


def test_server_step_of_several_workers_and_conservation():
    """W workers, T iterations: the (min, max) server step with one bit applies exactly what the
    checker applies, and per worker the sent values plus the residual add up to the gradients."""
    n, bucket, W, T, lr = 100_000 + 19, 2048, 3, 3, 0.1 / 3
    gs = [wl.laplace(n, 1e-4, config=2, worker=w) for w in range(W)]
    g_dev = [to_dev(g) for g in gs]
    res = [Guarded(n, torch.float32, fill=np.zeros(n, np.float32)) for _ in range(W)]
    e_ref = [np.zeros(n, np.float32) for _ in range(W)]
    p0 = wl.params(n, 0.05, config=2)
    p = Guarded(n, torch.float32, fill=p0)
    p_ref = p0.copy()
    sent = [np.zeros(n, np.float64) for _ in range(W)]
    for it in range(T):
        dev_c, dev_r, ref_c, ref_r = [], [], [], []
        for w in range(W):
            codes, ranges = gpu_step(g_dev[w], res[w], n, bucket)
            c, r, e_ref[w] = O.quantize_1bit_ef(gs[w], e_ref[w], bucket)
            assert np.array_equal(codes.numpy(np.uint32), c) and bits_equal(ranges.numpy(np.float32), r) == 0
            dev_c.append(codes.view), dev_r.append(ranges.view), ref_c.append(c), ref_r.append(r)
            sent[w] += O.dequantize_minmax(O.unpack(c, n, 1), 1, bucket, r)
        mqg.mqg_server_step_minmax(dev_c, dev_r, W, 1, n, bucket, p.view, lr)
        torch.cuda.synchronize()
        p.check_guards()
        p_ref, _ = O.server_step_minmax(ref_c, ref_r, 1, n, bucket, p_ref, lr)
        assert bits_equal(p.numpy(np.float32), p_ref) == 0
    for w in range(W):
        assert bits_equal(res[w].numpy(np.float32), e_ref[w]) == 0
        drift = np.abs(sent[w] + e_ref[w] - T * gs[w].astype(np.float64))
        assert drift.max() <= 1e-9                     # roundings only: nothing is forgotten
