"""mqg_quantize_workers: W workers' gradients in one call.  Worker w's codes and scales must be
bit-identical to the CPU checker's quantize of that gradient with worker id first_worker + w
(the paper's Quantize(g_p, K) of Algorithm 1 applied per worker p), for shapes the one-launch
kernel takes and for shapes it hands to per-worker launches."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def no_kernel_wait_gave_up():
    yield
    assert mqg.mqg_device_timeouts() == 0, "a kernel's bounded wait ran out"


def run_workers(xs, bits, bucket, seed, first_worker, step, elem_offset, bf16=False):
    n, W = xs[0].size, len(xs)
    if bf16:
        grads = [to_dev(x.view(np.int16)).view(torch.bfloat16) for x in xs]
    else:
        grads = [to_dev(x) for x in xs]
    codes = [Guarded(mqg.mqg_code_words(n, bits), torch.int32) for _ in xs]
    scales = [Guarded(mqg.mqg_num_buckets(n, bucket), torch.float32) for _ in xs]
    mqg.mqg_quantize_workers(grads, W, n, bits, bucket, seed, [c.view for c in codes],
                             [s.view for s in scales], first_worker, step, elem_offset)
    torch.cuda.synchronize()
    for c, s in zip(codes, scales):
        c.check_guards(), s.check_guards()
    return [c.numpy(np.uint32) for c in codes], [s.numpy(np.float32) for s in scales]


def assert_workers_parity(xs, bits, bucket, seed, first_worker=0, step=0, elem_offset=0, bf16=False):
    cs, ss = run_workers(xs, bits, bucket, seed, first_worker, step, elem_offset, bf16)
    for w, x in enumerate(xs):
        c_ref, s_ref = O.quantize(x, bits, bucket, seed, first_worker + w, step, elem_offset,
                                  dtype="bf16" if bf16 else "f32")
        assert bits_equal(ss[w], s_ref) == 0, "worker %d: scales differ" % w
        assert int((cs[w] != c_ref).sum()) == 0, "worker %d: codes differ" % w


@pytest.mark.parametrize("bits", list(range(1, 9)))
def test_workers_one_launch_shape(bits):
    """Several tiles per worker, ragged last tile and ragged last row, W = 3."""
    n = 3 * 4096 * 7 + 2048 + 37
    xs = [wl.normal(n, 1e-3, config=1, worker=w) for w in range(3)]
    assert_workers_parity(xs, bits, 2048, seed=5, first_worker=2, step=9)


@pytest.mark.parametrize("bits", [1, 4, 7])
@pytest.mark.parametrize("n,bucket,W", [
    (1 << 20, 512, 8),            # shuffle buckets, whole tiles only
    (300_000 + 9, 4096, 5),       # the largest bucket of the one-launch kernel
    (2048, 2048, 2),              # one tile per worker
    (40_000, 96, 4),              # buckets of three rows: tiles of 126 rows
    (100_000, 1 << 20, 3),        # a single bucket above a tile: per-worker launches
    (1000, 256, 6),               # below the one-launch kernel's minimum: per-worker launches
    (70_001, 8192, 2),            # 256-row buckets: per-worker launches
])
def test_workers_shapes(bits, n, bucket, W):
    xs = [wl.laplace(n, 2e-3, config=2, worker=w) for w in range(W)]
    assert_workers_parity(xs, bits, bucket, seed=77, first_worker=0, step=3)


@pytest.mark.parametrize("elem_offset", [8, (1 << 35) + 64, 3])
def test_workers_elem_offset(elem_offset):
    n = 50_000
    xs = [wl.normal(n, 1.0, config=1, worker=w) for w in range(4)]
    assert_workers_parity(xs, 3, 1024, seed=123, first_worker=7, step=1, elem_offset=elem_offset)


@pytest.mark.parametrize("bits", [2, 8])
def test_workers_bf16(bits):
    n = 200_000 + 24
    xs = [wl.student_t_bf16(n, config=5, worker=w) for w in range(3)]
    assert_workers_parity(xs, bits, 2048, seed=1, first_worker=1, step=2, bf16=True)


def test_workers_max_count_and_single():
    n = 8192
    xs = [wl.normal(n, 1e-2, config=1, worker=w) for w in range(mqg.MQG_MAX_WORKERS)]
    assert_workers_parity(xs, 4, 512, seed=9)
    assert_workers_parity(xs[:1], 4, 512, seed=9, first_worker=5)


def test_workers_argument_errors():
    n = 4096
    g = [to_dev(wl.normal(n, 1.0, config=1, worker=0)) for _ in range(2)]
    c = [torch.zeros(mqg.mqg_code_words(n, 4), dtype=torch.int32, device="cuda") for _ in range(2)]
    s = [torch.zeros(mqg.mqg_num_buckets(n, 512), dtype=torch.float32, device="cuda") for _ in range(2)]
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_workers(g, 2, n, 9, 512, 0, c, s)
    assert e.value.status == mqg.MQG_ERR_BITS
    many = mqg.MQG_MAX_WORKERS + 1
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_workers(g * many, 2 * many, n, 4, 512, 0, c * many, s * many)
    assert e.value.status == mqg.MQG_ERR_TOO_MANY_WORKERS
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_workers([g[0], g[1][1:]], 2, n - 1, 4, 512, 0, c, s)
    assert e.value.status == mqg.MQG_ERR_ALIGN
    mqg.mqg_quantize_workers(g, 2, 0, 4, 512, 0, c, s)      # nothing to do
