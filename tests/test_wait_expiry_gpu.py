"""The give-up path of the kernels' bounded barrier waits, exercised without faulting or hanging
anything: with the library's test hook the kernels arm their barriers for the bytes of a staging
copy but never issue the copy, and poll only 1024 times.  Nothing is in flight, the wait simply runs
out: every CTA (or warp) counts it, waits once more (bounded) for the copies it believes it has
issued, and returns without writing its outputs.  The host then sees MQG_ERR_TIMEOUT from
mqg_check_timeouts, and the next ordinary calls are bit-exact again."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl

pytestmark = pytest.mark.gpu

N, W, B, BITS, LR = 1 << 20, 4, 2048, 4, 0.025
SENTINEL = 0x5A5A5A5A


def _buffers():
    codes = [torch.full((mqg.mqg_code_words(N, BITS),), SENTINEL, dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.full((mqg.mqg_num_buckets(N, B),), -7.0, dtype=torch.float32, device="cuda") for _ in range(W)]
    return codes, scales


def _expect_timeout():
    with pytest.raises(mqg.MqgError) as err:
        mqg.mqg_check_timeouts(reset=True)
    assert err.value.status == mqg.MQG_ERR_TIMEOUT
    assert mqg.mqg_device_timeouts() == 0          # the call above cleared the counter
    assert mqg.mqg_check_timeouts(reset=True) == 0


def test_waits_run_out_are_counted_and_the_next_calls_are_exact():
    xs = [wl.normal(N, 1e-3, config=1, worker=w) for w in range(W)]
    grads = [torch.from_numpy(x).cuda() for x in xs]
    p0 = wl.params(N, 0.05, config=1)
    assert mqg.mqg_check_timeouts(reset=True) == 0

    # codes for the server case, written in normal operation
    good_codes, good_scales = _buffers()
    for w in range(W):
        mqg.mqg_quantize(grads[w], N, BITS, B, 3, good_codes[w], good_scales[w], worker=w)
    torch.cuda.synchronize()

    try:
        mqg.mqg_test_wait_override(1024, True)

        # one-worker quantize kernel: every CTA gives up on its first tile, nothing is written
        codes, scales = _buffers()
        mqg.mqg_quantize(grads[0], N, BITS, B, 3, codes[0], scales[0], worker=0)
        _expect_timeout()
        assert bool((codes[0] == SENTINEL).all()) and bool((scales[0] == -7.0).all())

        # the batched quantize kernel (its walk over several workers' tiles)
        mqg.mqg_quantize_workers(grads, W, N, BITS, B, 3, codes, scales, first_worker=0)
        _expect_timeout()
        assert all(bool((c == SENTINEL).all()) for c in codes)

        # the fused server kernel: every warp gives up waiting for its first parameter tile
        params = torch.from_numpy(p0.copy()).cuda()
        mqg.mqg_server_step(good_codes, good_scales, W, BITS, N, B, params, LR)
        _expect_timeout()
        assert np.array_equal(params.cpu().numpy().view(np.uint32), p0.view(np.uint32))
    finally:
        mqg.mqg_test_wait_override(0, False)

    # normal operation again, bit for bit
    codes, scales = _buffers()
    mqg.mqg_quantize_workers(grads, W, N, BITS, B, 3, codes, scales, first_worker=0)
    ref_codes, ref_scales = [], []
    for w in range(W):
        c_ref, s_ref = O.quantize(xs[w], BITS, B, 3, worker=w)
        assert np.array_equal(codes[w].cpu().numpy().view(np.uint32), c_ref)
        assert np.array_equal(scales[w].cpu().numpy(), s_ref)
        ref_codes.append(c_ref), ref_scales.append(s_ref)
    params = torch.from_numpy(p0.copy()).cuda()
    mqg.mqg_server_step(codes, scales, W, BITS, N, B, params, LR)
    p_ref, _ = O.server_step(ref_codes, ref_scales, BITS, N, B, p0.copy(), LR)
    assert np.array_equal(params.cpu().numpy().view(np.uint32), p_ref.view(np.uint32))
    assert mqg.mqg_check_timeouts(reset=True) == 0
