"""mqg_quantize_segments_l2_static: the per-layer L2-norm quantizer for callers that cannot hand
the library a workspace (all device memory already owned by one pool, no allocation allowed on a
latency-critical path, or a host that only permits launches on the buffers it supplies).  Its
partial sums live in an array inside the library image, shared by every call on the device.

Checked here, through the C ABI: two calls in a row (the second on other data and a smaller table,
so that it finds the first call's leftovers in the array) give bit for bit what
mqg_quantize_segments_l2 gives with a caller workspace; the size limit is enforced before anything
is launched; the calls leave the amount of free device memory unchanged.  This file is collected
last on purpose, so that a run that stops at the first failure has run every other test before."""
import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, to_dev

pytestmark = pytest.mark.gpu
BITS = 5


def _segments(sizes):
    seg = np.zeros(len(sizes) + 1, np.uint64)
    seg[1:] = np.cumsum(sizes)
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum([O.code_words(s, BITS) for s in sizes])
    return seg, coff


def _with_workspace(x, seg, coff, seed):
    codes = Guarded(int(coff[-1]), torch.int32)
    scales = Guarded(len(seg) - 1, torch.float32)
    ws = torch.empty(mqg.mqg_l2_workspace_floats(seg), dtype=torch.float32, device="cuda")
    mqg.mqg_quantize_segments_l2(x, seg, coff, BITS, seed, codes.view, scales.view, ws, worker=1, step=2)
    torch.cuda.synchronize()
    return codes.numpy(np.uint32), scales.numpy(np.float32)


def _outputs(seg, coff):
    return Guarded(int(coff[-1]), torch.int32), Guarded(len(seg) - 1, torch.float32)


def _static(x, seg, coff, seed, codes, scales):
    mqg.mqg_quantize_segments_l2_static(x, seg, coff, BITS, seed, codes.view, scales.view, worker=1, step=2)
    torch.cuda.synchronize()


def _read(codes, scales):
    codes.check_guards(), scales.check_guards()
    return codes.numpy(np.uint32), scales.numpy(np.float32)


def _same(got, want, sizes, coff):
    assert bits_equal(got[1], want[1]) == 0, "scales differ"
    for j, s in enumerate(sizes):           # words between two streams belong to neither
        lo, nw = int(coff[j]), O.code_words(s, BITS)
        assert np.array_equal(got[0][lo:lo + nw], want[0][lo:lo + nw]), "codes of segment %d differ" % j


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    first = [300_000, 7, 8192, 0, 70_001, 8193, 40_000]            # 37 + 1 + 1 + 9 + 2 + 5 partial sums
    second = [50_000, 999, 123_457]                                # fewer: stale sums stay behind them
    xs = [to_dev(wl.layered(first, config=3, worker=0)), to_dev(wl.layered(second, config=3, worker=1))]
    tables = [_segments(first), _segments(second)]
    want = [_with_workspace(xs[k], *tables[k], seed=10 + k) for k in range(2)]

    out = [_outputs(*tables[k]) for k in range(2)]                # every buffer exists before the calls
    _static(xs[0], *tables[0], 10, *out[0])                        # also the call that looks up the address
    free_before = torch.cuda.mem_get_info()[0]
    _static(xs[1], *tables[1], 11, *out[1])
    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
    got0, got1 = _read(*out[0]), _read(*out[1])
    _same(got0, want[0], first, tables[0][1])
    _same(got1, want[1], second, tables[1][1])
    # and the oracle agrees with both entry points on the scales
    ref = O.quantize_segments_l2(xs[1].cpu().numpy(), *tables[1], BITS, 11, worker=1, step=2)
    assert bits_equal(got1[1], ref[1]) == 0
    assert mqg.mqg_device_timeouts() == 0


def test_a_table_beyond_the_built_in_array_is_rejected_before_any_launch():
    limit = mqg.MQG_L2_STATIC_WORKSPACE_FLOATS
    # limit + 1 one-element segments need limit + 1 partial sums; nothing is read or launched, so
    # small buffers suffice
    nseg = limit + 1
    seg = np.arange(nseg + 1, dtype=np.uint64)
    coff = np.arange(nseg + 1, dtype=np.uint64)
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    codes = Guarded(64, torch.int32)
    scales = Guarded(64, torch.float32)
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_segments_l2_static(x, seg, coff, BITS, 0, codes.view, scales.view)
    assert e.value.status == mqg.MQG_ERR_INVALID
    assert str(limit) in str(e.value) and str(limit + 1) in str(e.value)
    torch.cuda.synchronize()
    codes.check_guards(), scales.check_guards()
    assert (codes.numpy(np.uint32) == 0x7FC0DEAD).all(), "something was written"
    # exactly at the limit the table is accepted (here: rejected later, for a reason of its own)
    seg2 = np.zeros(3, np.uint64); seg2[1] = 8192 * (limit - 1); seg2[2] = seg2[1] + 1
    coff2 = np.array([0, 1, 1], np.uint64)                          # too few code words: a table error
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_segments_l2_static(x, seg2, coff2, BITS, 0, codes.view, scales.view)
    assert "built-in" not in str(e.value)
