"""mqg_quantize_segments_workers (several workers' layered gradients, one scale per segment, three
launches for all of them) against the CPU checker, worker by worker and bit for bit, with guard
words around every output.  Covers short segments only, long segments that become entries of the
bulk-copy part (ragged lengths, a flushed one), long segments that do not qualify (odd word
offset), more than 64 (worker, long segment) pairs and more than 64 segments (several launches),
bf16 input, worker ids and offsets, and the AlexNet-shaped and Section 4.1 layouts."""
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


def _segments(sizes, bits, gaps=None):
    seg = np.zeros(len(sizes) + 1, np.uint64)
    seg[1:] = np.cumsum(sizes)
    words = [O.code_words(s, bits) + (gaps[j] if gaps else 0) for j, s in enumerate(sizes)]
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum(words)
    return seg, coff


def _check(xs, sizes, seg, coff, bits, seed, first_worker=0, step=0, elem_offset=0, bf16=False):
    W = len(xs)
    if bf16:
        grads = [to_dev(x.view(np.int16)).view(torch.bfloat16) for x in xs]
    else:
        grads = [to_dev(x) for x in xs]
    codes = [Guarded(int(coff[-1]), torch.int32) for _ in range(W)]
    scales = [Guarded(len(sizes), torch.float32) for _ in range(W)]
    mqg.mqg_quantize_segments_workers(grads, W, seg, coff, bits, seed, [c.view for c in codes],
                                      [s.view for s in scales], first_worker=first_worker, step=step,
                                      elem_offset=elem_offset)
    torch.cuda.synchronize()
    out = []
    for w in range(W):
        codes[w].check_guards(), scales[w].check_guards()
        c_ref, s_ref = O.quantize_segments(xs[w], seg, coff, bits, seed=seed, worker=first_worker + w, step=step,
                                           elem_offset=elem_offset, dtype="bf16" if bf16 else "f32")
        assert bits_equal(scales[w].numpy(np.float32), s_ref) == 0, w
        got = codes[w].numpy(np.uint32)
        for j, sz in enumerate(sizes):          # words between streams are not part of the result
            lo, nw = int(coff[j]), O.code_words(sz, bits)
            assert np.array_equal(got[lo:lo + nw], c_ref[lo:lo + nw]), (w, j)
        out.append((c_ref, s_ref))
    return out


@pytest.mark.parametrize("bits", range(1, 9))
def test_short_segments_only(bits):
    sizes = [96, 1000, 7, 0, 34_848, 33, 20_000, 256, 8192, 8193, 1, 40_000]
    seg, coff = _segments(sizes, bits)
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(3)]
    _check(xs, sizes, seg, coff, bits, seed=3, first_worker=2, step=1, elem_offset=64)


@pytest.mark.parametrize("bits", [1, 3, 4, 8])
def test_long_and_short_segments(bits):
    """Entries of the bulk-copy part (second and sixth segment; ragged lengths; one flushed to zero),
    a long segment that does not qualify (its codes start on an odd word) and short ones."""
    sizes = [128, (1 << 20) + 37, 5, (1 << 20) + 64, 100, (1 << 20) + 4096 * 3 + 31]
    gaps = [0, 0, 0, 1, 2, 0]            # the 4th segment's stream starts at an odd word for odd widths
    seg, coff = _segments(sizes, bits, gaps)
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(3)]
    xs[1][128:128 + (1 << 20) + 37] = np.float32(1e-30)     # below the flush limit
    refs = _check(xs, sizes, seg, coff, bits, seed=5)
    assert refs[1][1][1] == 0 and refs[0][1][1] > 0


def test_more_pairs_than_one_launch_holds_and_more_segments_than_one_table():
    """12 workers x 6 long segments = 72 (worker, long segment) pairs (64 per launch; a segment is an
    entry from 32,768 elements on) and 150 short segments (64 per table)."""
    rng = np.random.default_rng(1)
    sizes = [1 << 20, 1 << 15, (1 << 20) + 32, (1 << 15) + 4096 + 7, 1 << 16, 40_000 - 32] + \
        [int(v) for v in rng.integers(0, 600, 150)]
    bits = 5
    seg, coff = _segments(sizes, bits)
    xs = [wl.layered(sizes, config=31, worker=w) for w in range(12)]
    _check(xs, sizes, seg, coff, bits, seed=8, elem_offset=1 << 33)


@pytest.mark.parametrize("bits", [2, 7])
def test_bf16_input(bits):
    sizes = [1000, (1 << 20) + 96, 300, 77]
    seg, coff = _segments(sizes, bits)
    xs = [wl.f32_to_bf16_bits(wl.layered(sizes, config=3, worker=w)) for w in range(2)]
    _check(xs, sizes, seg, coff, bits, seed=9, bf16=True)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_alexnet_shaped_layered_gradient_all_workers(bits):
    """The layered configuration at full size: 16 tensors, 60,965,224 elements, W = 8 (sampled
    comparison would hide nothing here: the checker encodes a worker in a few seconds, so two of the
    eight workers are checked in full and the launch covers all eight)."""
    seg, sizes = wl.alexnet_segments()
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum([O.code_words(s, bits) for s in sizes])
    W = 8
    grads = [to_dev(wl.layered(sizes, config=3, worker=w)) for w in range(W)]
    codes = [torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(len(sizes), dtype=torch.float32, device="cuda") for _ in range(W)]
    mqg.mqg_quantize_segments_workers(grads, W, seg, coff, bits, 11, codes, scales, step=4)
    torch.cuda.synchronize()
    for w in (0, 7):
        x = wl.layered(sizes, config=3, worker=w)
        c_ref, s_ref = O.quantize_segments(x, seg, coff, bits, seed=11, worker=w, step=4)
        assert bits_equal(scales[w].cpu().numpy(), s_ref) == 0
        assert np.array_equal(codes[w].cpu().numpy().view(np.uint32), c_ref), w
    # every other worker against the one-worker entry point of the library
    for w in range(1, 7):
        c1 = torch.zeros_like(codes[w])
        s1 = torch.zeros_like(scales[w])
        mqg.mqg_quantize_segments(grads[w], seg, coff, bits, 11, c1, s1, worker=w, step=4)
        assert torch.equal(c1, codes[w]) and torch.equal(s1.view(torch.int32), scales[w].view(torch.int32)), w


def test_rejects_bad_arguments():
    seg, coff = _segments([64, 64], 4)
    g = [torch.zeros(128, device="cuda")]
    c = [torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda")]
    s = [torch.zeros(2, device="cuda")]
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_segments_workers(g, 1, seg, coff, 9, 0, c, s)
    assert e.value.status == mqg.MQG_ERR_BITS
    bad = coff.copy()
    bad[1] = 1                                     # too few words for the first segment
    with pytest.raises(mqg.MqgError) as e:
        mqg.mqg_quantize_segments_workers(g, 1, seg, bad, 4, 0, c, s)
    assert e.value.status == mqg.MQG_ERR_INVALID
    lib = mqg.raw_library()
    assert lib.mqg_quantize_segments_workers(None, 33, 2, None, None, 4, 0, None, None, 0, 0, 0, 0, None) \
        == mqg.MQG_ERR_TOO_MANY_WORKERS
