"""Parity of the L2-norm scale variant (CUDA, through the C ABI binding) with the CPU checker,
element by element on the same seeded inputs: scales (a fixed-order fp32 sum of squares and one
square root) and packed codes bit for bit, then the ordinary server step on those outputs bit
for bit (the stated bar for floating point is 1e-6 relative; both sides perform the same IEEE
operations in the same order, so equality is asserted)."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, to_dev

pytestmark = pytest.mark.gpu
ALL_BITS = list(range(1, 9))


@pytest.fixture(autouse=True)
def no_kernel_wait_gave_up():
    yield
    assert mqg.mqg_device_timeouts() == 0, "a kernel's bounded wait ran out"


def assert_quantize_parity(x, bits, bucket, bf16=False, **key):
    n = x.size
    g = to_dev(x.view(np.int16)).view(torch.bfloat16) if bf16 else to_dev(x)
    codes = Guarded(mqg.mqg_code_words(n, bits), torch.int32)
    scales = Guarded(mqg.mqg_num_buckets(n, bucket), torch.float32)
    mqg.mqg_quantize_l2(g, n, bits, bucket, key.get("seed", 0), codes.view, scales.view,
                        worker=key.get("worker", 0), step=key.get("step", 0),
                        elem_offset=key.get("elem_offset", 0))
    torch.cuda.synchronize()
    codes.check_guards(), scales.check_guards()
    c_ref, s_ref = O.quantize_l2(x, bits, bucket, key.get("seed", 0), worker=key.get("worker", 0),
                                 step=key.get("step", 0), elem_offset=key.get("elem_offset", 0),
                                 dtype="bf16" if bf16 else "f32")
    assert bits_equal(scales.numpy(np.float32), s_ref) == 0, "scales differ"
    c_gpu = codes.numpy(np.uint32)
    if not np.array_equal(c_gpu, c_ref):
        q_gpu, q_ref = O.unpack(c_gpu, n, bits), O.unpack(c_ref, n, bits)
        idx = np.nonzero(q_gpu != q_ref)[0]
        raise AssertionError("%d codes differ (first at %s: gpu %s, ref %s)"
                             % (idx.size, idx[:5], q_gpu[idx[:5]], q_ref[idx[:5]]))
    return c_ref, s_ref


@pytest.mark.parametrize("bits", ALL_BITS)
def test_quantize_small_configuration(bits):
    """n = 2^20, N(0, 1e-3), bucket 512: buckets of 16 rows (lane shuffles)."""
    assert_quantize_parity(wl.normal(1 << 20, 1e-3, config=1, worker=2), bits, 512, seed=0, worker=2)


@pytest.mark.parametrize("bits", [1, 3, 4, 8])
@pytest.mark.parametrize("n,bucket", [
    (3 * 4096 * 7 + 2048 + 37, 2048),     # two warps per bucket, ragged last tile and row
    (300_000 + 9, 4096), (65_536 + 32, 8192),      # four and eight warps per bucket
    (40_000, 96), (9_000, 3072),          # three rows / three warps per bucket: zero-padded trees
    (50_000, 5 * 32), (33_000, 7 * 32 * 4),        # 5 rows (level-by-level path), 28 rows
    (2048, 2048), (2049, 1024), (1, 32), (31, 32), (33, 32), (1000, 256), (64, 32),
    (5000, 8192), (8192, 8192), (8191, 1 << 20), (37, 100),      # a single (ragged) bucket
])
def test_quantize_shapes(bits, n, bucket):
    x = wl.laplace(n, 2e-3, config=2, worker=n % 7)
    assert_quantize_parity(x, bits, bucket, seed=n, worker=3, step=bits)


@pytest.mark.parametrize("bits", [2, 7])
def test_quantize_where_the_summation_order_shows(bits):
    """Values spread over many binades, so that another order of the same additions rounds
    differently; a one-hot bucket (s = |x| exactly); zero and sub-threshold buckets."""
    n, bucket = 6 * 2048, 2048
    rng = np.random.default_rng(123)
    x = (rng.standard_normal(n) * np.exp2(rng.integers(-12, 12, n))).astype(np.float32)
    x[2048:4096] = 0.0
    x[2048 + 77] = np.float32(-1.2345678)
    x[4096:6144] = 0.0
    x[6144:8192] = np.float32(1e-30)                     # sum of squares below 2^-96: flushed
    x[8192:10240] = np.float32(2.0 ** -50)               # 2048 * 2^-100 = 2^-89: kept
    c_ref, s_ref = assert_quantize_parity(x, bits, bucket, seed=5)
    assert s_ref[1] == np.float32(1.2345678) and s_ref[2] == 0 and s_ref[3] == 0 and s_ref[4] > 0


@pytest.mark.parametrize("bits", [1, 4, 7])
def test_quantize_bf16(bits):
    x = wl.student_t_bf16(200_000 + 24, config=5, worker=1)
    assert_quantize_parity(x, bits, 2048, bf16=True, seed=2)
    assert_quantize_parity(x[:8001], bits, 1 << 20, bf16=True, seed=2)


def test_element_offsets():
    x = wl.normal(10_000, 1e-2, config=1, worker=5)
    assert_quantize_parity(x, 5, 1024, seed=11, worker=1, step=2, elem_offset=12_345)       # not a multiple of 8
    assert_quantize_parity(x, 5, 1024, seed=11, worker=1, step=2, elem_offset=8 * 12_345)   # block-aligned
    assert_quantize_parity(x, 2, 4096, seed=(1 << 40) + 3, worker=7, step=9, elem_offset=(1 << 36) + 64)


def test_buckets_above_the_one_pass_limit_are_rejected():
    x = to_dev(wl.normal(20_000, 1.0))
    codes = torch.zeros(mqg.mqg_code_words(20_000, 4), dtype=torch.int32, device="cuda")
    scales = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_l2(x, 20_000, 4, 16_384, 0, codes, scales)
    assert e.value.status == mqg.MQG_ERR_INVALID


@pytest.mark.parametrize("bits", [1, 4, 6])
def test_server_step_on_l2_scaled_buffers(bits):
    """The variant's outputs feed the ordinary fused server step."""
    n, bucket, W, lr = 150_000 + 19, 2048, 4, 0.1 / 4
    xs = [wl.laplace(n, 1e-4, config=2, worker=w) for w in range(W)]
    dev_c, dev_s, ref_c, ref_s = [], [], [], []
    for w, x in enumerate(xs):
        codes = torch.zeros(mqg.mqg_code_words(n, bits), dtype=torch.int32, device="cuda")
        scales = torch.zeros(mqg.mqg_num_buckets(n, bucket), dtype=torch.float32, device="cuda")
        mqg.mqg_quantize_l2(to_dev(x), n, bits, bucket, 7, codes, scales, worker=w)
        c, s = O.quantize_l2(x, bits, bucket, 7, worker=w)
        dev_c.append(codes), dev_s.append(scales), ref_c.append(c), ref_s.append(s)
    p0 = wl.params(n, 0.05, config=2)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step(dev_c, dev_s, W, bits, n, bucket, p.view, lr)
    torch.cuda.synchronize()
    p.check_guards()
    p_ref, _ = O.server_step(ref_c, ref_s, bits, n, bucket, p0.copy(), lr)
    assert bits_equal(p.numpy(np.float32), p_ref) == 0


# ------------------------------------------------------------------ per-layer norm (segments)
def _segments(sizes, bits):
    seg = np.zeros(len(sizes) + 1, np.uint64)
    seg[1:] = np.cumsum(sizes)
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum([O.code_words(s, bits) for s in sizes])
    return seg, coff


def segments_parity(sizes, bits, x, ws_extra=0, **key):
    seg, coff = _segments(sizes, bits)
    need = mqg.mqg_l2_workspace_floats(seg)
    assert need == sum((s + 8191) // 8192 for s in sizes)
    codes = Guarded(int(coff[-1]), torch.int32)
    scales = Guarded(len(sizes), torch.float32)
    ws = Guarded(need + ws_extra, torch.float32)
    mqg.mqg_quantize_segments_l2(to_dev(x), seg, coff, bits, key.get("seed", 0), codes.view, scales.view,
                                 ws.view, worker=key.get("worker", 0), step=key.get("step", 0),
                                 elem_offset=key.get("elem_offset", 0))
    torch.cuda.synchronize()
    codes.check_guards(), scales.check_guards(), ws.check_guards()
    c_ref, s_ref = O.quantize_segments_l2(x, seg, coff, bits, key.get("seed", 0), worker=key.get("worker", 0),
                                          step=key.get("step", 0), elem_offset=key.get("elem_offset", 0))
    assert bits_equal(scales.numpy(np.float32), s_ref) == 0, "scales differ"
    got = codes.numpy(np.uint32)
    for j, s in enumerate(sizes):           # words between streams are not part of the result
        lo, nw = int(coff[j]), O.code_words(s, bits)
        assert np.array_equal(got[lo:lo + nw], c_ref[lo:lo + nw]), j
    return seg, coff, c_ref, s_ref


@pytest.mark.parametrize("bits", ALL_BITS)
def test_segments_quantize(bits):
    # one tile, exactly one tile, one tile and a row, 3 / 5 / 13 tiles (zero-padded trees), empty
    sizes = [96, 1000, 7, 0, 34_848, 33, 20_000, 256, 8192, 8193, 1, 5 * 8192 - 3, 100_000]
    x = wl.layered(sizes, config=3, worker=1)
    segments_parity(sizes, bits, x, seed=3, worker=1, step=1, elem_offset=64)


@pytest.mark.parametrize("bits", [3, 8])
def test_segments_long_segments_encode_in_their_own_launches(bits):
    """Segments of a million elements and more with 16-byte aligned buffers (the second one here,
    ragged length included) are encoded by the TMA-fed kernel, the others (the fourth starts on an
    odd word) by the table-driven launch; scales and codes must match the checker either way."""
    sizes = [128, (1 << 20) + 37, 5, (1 << 20) + 64, 100]
    x = wl.layered(sizes, config=3, worker=2)
    x[128 + (1 << 20) + 37 + 5:128 + (1 << 20) + 37 + 5 + 4096] = 0.0
    segments_parity(sizes, bits, x, seed=6, worker=2, step=1)


def test_segments_more_than_one_launch_chunk_and_a_dirty_workspace():
    rng = np.random.default_rng(0)
    sizes = [int(v) for v in rng.integers(0, 30_000, 150)]
    x = wl.layered(sizes, config=31)
    segments_parity(sizes, 5, x, ws_extra=5, seed=8)       # the workspace starts as poison


def test_segments_server_step_on_l2_scaled_buffers():
    sizes, bits, W = [4096 * 9 + 5, 300, 70_000], 3, 3
    seg, coff = _segments(sizes, bits)
    n = int(seg[-1])
    refs = []
    for w in range(W):
        x = wl.layered(sizes, config=3, worker=w)
        refs.append(segments_parity(sizes, bits, x, seed=4, worker=w)[2:])
    p0 = wl.params(n, 0.05, config=3)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_segments([to_dev(c.view(np.int32)) for c, _ in refs], [to_dev(s) for _, s in refs],
                                 W, bits, seg, coff, p.view, 0.05)
    torch.cuda.synchronize()
    p.check_guards()
    p_ref, _ = O.server_step_segments([c for c, _ in refs], [s for _, s in refs], bits, seg, coff,
                                      p0.copy(), 0.05)
    assert bits_equal(p.numpy(np.float32), p_ref) == 0


def test_segments_workspace_too_small_is_rejected():
    sizes = [20_000, 9_000]
    seg, coff = _segments(sizes, 4)
    x = to_dev(wl.layered(sizes, config=3))
    codes = torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda")
    scales = torch.zeros(2, dtype=torch.float32, device="cuda")
    ws = torch.zeros(4, dtype=torch.float32, device="cuda")          # 3 + 2 needed
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_segments_l2(x, seg, coff, 4, 0, codes, scales, ws)
    assert e.value.status == mqg.MQG_ERR_INVALID and "workspace" in str(e.value)


def test_alexnet_shaped_layers_one_norm_per_tensor():
    """The layered workload (16 tensors, 61 M elements): scales of every tensor bit for bit (the
    largest tensor folds 4608 tile sums), codes on the small tensors and on sampled words."""
    sizes = [int(np.prod(s)) for s in wl.ALEXNET_SHAPES]
    bits = 4
    x = wl.layered(sizes, config=3, worker=0)
    seg, coff = _segments(sizes, bits)
    codes = torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda")
    scales = torch.zeros(len(sizes), dtype=torch.float32, device="cuda")
    ws = torch.zeros(mqg.mqg_l2_workspace_floats(seg), dtype=torch.float32, device="cuda")
    mqg.mqg_quantize_segments_l2(to_dev(x), seg, coff, bits, 9, codes, scales, ws)
    torch.cuda.synchronize()
    s_ref = np.array([O.bucket_norms(x[int(seg[j]):int(seg[j + 1])], sizes[j])[0] for j in range(len(sizes))])
    assert bits_equal(scales.cpu().numpy(), s_ref) == 0
    got = codes.cpu().numpy().view(np.uint32)
    for j in (0, 1, 2, 15, 10):             # whole tensors up to 37.7 M elements would take minutes: sample
        a, b = int(seg[j]), int(seg[j + 1])
        m = min(b - a, 64 * 1024)
        h = O.draw_h(9, 0, 0, a, m)
        q = O.encode(x[a:a + m], bits, b - a, s_ref[j:j + 1], h)
        words = O.pack(q, bits)
        full = (m * bits) // 32
        assert np.array_equal(got[int(coff[j]):int(coff[j]) + full], words[:full]), j


def assert_workers_parity(xs, bits, bucket, bf16=False, seed=0, first_worker=0, step=0, elem_offset=0):
    """mqg_quantize_workers_l2 (one launch for all workers) against the CPU checker, worker by worker."""
    W, n = len(xs), xs[0].size
    gs = [to_dev(x.view(np.int16)).view(torch.bfloat16) if bf16 else to_dev(x) for x in xs]
    codes = [Guarded(mqg.mqg_code_words(n, bits), torch.int32) for _ in range(W)]
    scales = [Guarded(mqg.mqg_num_buckets(n, bucket), torch.float32) for _ in range(W)]
    mqg.mqg_quantize_workers_l2(gs, W, n, bits, bucket, seed, [c.view for c in codes], [s.view for s in scales],
                                first_worker=first_worker, step=step, elem_offset=elem_offset)
    torch.cuda.synchronize()
    for w in range(W):
        codes[w].check_guards(), scales[w].check_guards()
        c_ref, s_ref = O.quantize_l2(xs[w], bits, bucket, seed, worker=first_worker + w, step=step,
                                     elem_offset=elem_offset, dtype="bf16" if bf16 else "f32")
        assert bits_equal(scales[w].numpy(np.float32), s_ref) == 0, "worker %d: scales differ" % w
        assert np.array_equal(codes[w].numpy(np.uint32), c_ref), "worker %d: codes differ" % w


@pytest.mark.parametrize("bits", ALL_BITS)
def test_workers_in_one_launch(bits):
    """Four workers, bucket 2048 (two warps per bucket), ragged last tile and row."""
    n = 5 * 4096 * 9 + 2048 + 21
    xs = [wl.laplace(n, 1e-4, config=2, worker=w) for w in range(4)]
    assert_workers_parity(xs, bits, 2048, seed=7, first_worker=3, step=bits)


@pytest.mark.parametrize("bits", [1, 4, 7])
@pytest.mark.parametrize("n,bucket", [
    (300_000 + 9, 4096), (70_000, 512), (40_000, 96),       # four warps; 16-row shuffles; a shape of W launches
    (1 << 20, 1024), (33, 32),
])
def test_workers_shapes(bits, n, bucket):
    xs = [wl.normal(n, 1e-3, config=1, worker=10 + w) for w in range(3)]
    assert_workers_parity(xs, bits, bucket, seed=n, step=2)


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_workers_bf16_and_offset_draws(bits):
    n = 3 * 4096 * 11 + 4096
    xs = [wl.student_t_bf16(n, config=5, worker=w) for w in range(2)]
    assert_workers_parity(xs, bits, 4096, bf16=True, seed=5, first_worker=1, elem_offset=8 * 12345)
