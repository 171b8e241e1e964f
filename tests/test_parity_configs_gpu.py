"""Parity on the remaining workload shapes: the AlexNet-shaped layered gradient with one scale
per tensor and the paper's own CNN with its two large matrices quantized (both full size, every
element checked), and the 10^9-element bf16 stress shape (checked on
sampled buckets, which `elem_offset` lets the CPU checker compute in isolation)."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import paper_1804_08066_b200 as mqg
from oracle import mqg_oracle as O
from paper_1804_08066_b200 import workloads as wl
from tests.gpu_util import Guarded, bits_equal, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_alexnet_layers_one_scale_per_tensor(bits):
    seg, sizes = wl.alexnet_segments()
    assert int(seg[-1]) == 60_965_224 and len(sizes) == 16
    coff = np.zeros(len(sizes) + 1, np.uint64)
    coff[1:] = np.cumsum([O.code_words(s, bits) for s in sizes])
    n, W = int(seg[-1]), 2
    xs = [wl.layered(sizes, config=3, worker=w) for w in range(W)]
    with ThreadPoolExecutor(W) as ex:
        refs = list(ex.map(lambda w: O.quantize_segments(xs[w], seg, coff, bits, seed=3, worker=w, step=bits),
                           range(W)))
    dcodes, dscales = [], []
    for w in range(W):
        codes = Guarded(int(coff[-1]), torch.int32)
        scales = Guarded(len(sizes), torch.float32)
        mqg.mqg_quantize_segments(to_dev(xs[w]), seg, coff, bits, 3, codes.view, scales.view, worker=w, step=bits)
        torch.cuda.synchronize()
        codes.check_guards(), scales.check_guards()
        assert bits_equal(scales.numpy(np.float32), refs[w][1]) == 0
        assert np.array_equal(codes.numpy(np.uint32), refs[w][0])      # streams are back to back
        assert np.array_equal(refs[w][1], [np.abs(xs[w][int(seg[j]):int(seg[j + 1])]).max() for j in range(16)])
        dcodes.append(codes), dscales.append(scales)
    p0 = wl.params(n, 0.05, config=3)
    p_ref, _ = O.server_step_segments([r[0] for r in refs], [r[1] for r in refs], bits, seg, coff, p0.copy(), 0.05)
    p = Guarded(n, torch.float32, fill=p0)
    mqg.mqg_server_step_segments([c.view for c in dcodes], [s.view for s in dscales], W, bits, seg, coff, p.view, 0.05)
    torch.cuda.synchronize()
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0
    assert mqg.mqg_device_timeouts() == 0


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_paper_cnn_two_fc_layers_quantized_rest_uncompressed(bits):
    """The paper's own model (Section 4.1): the two large fully connected matrices (16,072,704
    elements, one scale each) go through quantize -> server step; the other tensors are applied
    uncompressed, worker by worker.  Full size, every element checked."""
    seg, total = wl.paper_cnn_layout()
    nq = int(seg[-1])
    assert nq == 16_072_704 and total == 16_224_586
    coff = np.zeros(3, np.uint64)
    coff[1:] = np.cumsum([O.code_words(int(seg[j + 1] - seg[j]), bits) for j in range(2)])
    W, lr = 3, 0.2 / 3
    xs = [wl.paper_cnn_gradient(worker=w) for w in range(W)]
    with ThreadPoolExecutor(W) as ex:
        refs = list(ex.map(lambda w: O.quantize_segments(xs[w][:nq], seg, coff, bits, seed=6, worker=w, step=1),
                           range(W)))
    p0 = wl.params(total, 0.05, config=6)
    p_ref = p0.copy()
    head = np.ascontiguousarray(p_ref[:nq])
    O.server_step_segments([r[0] for r in refs], [r[1] for r in refs], bits, seg, coff, head, lr)
    p_ref[:nq] = head
    tail = np.ascontiguousarray(p_ref[nq:])
    for w in range(W):
        O.apply(tail, xs[w][nq:], lr)
    p_ref[nq:] = tail

    grads = [to_dev(x) for x in xs]
    dcodes, dscales = [], []
    for w in range(W):
        codes = Guarded(int(coff[-1]), torch.int32)
        scales = Guarded(2, torch.float32)
        mqg.mqg_quantize_segments(grads[w], seg, coff, bits, 6, codes.view, scales.view, worker=w, step=1)
        dcodes.append(codes), dscales.append(scales)
    p = Guarded(total, torch.float32, fill=p0)
    mqg.mqg_server_step_segments([c.view for c in dcodes], [s.view for s in dscales], W, bits, seg, coff, p.view, lr)
    for w in range(W):
        mqg.mqg_apply(p.view[nq:], grads[w][nq:], lr, total - nq)
    torch.cuda.synchronize()
    for w in range(W):
        dcodes[w].check_guards(), dscales[w].check_guards()
        assert bits_equal(dscales[w].numpy(np.float32), refs[w][1]) == 0
        assert np.array_equal(dcodes[w].numpy(np.uint32), refs[w][0])
    p.check_guards()
    assert bits_equal(p.numpy(np.float32), p_ref) == 0
    assert mqg.mqg_device_timeouts() == 0


def _student_t_bf16_on_device(n, seed):
    """Student-t(3) * 1e-4 with 0.1 % exact zeros, rounded to bf16, generated on the GPU in chunks."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    step = 1 << 26
    for lo in range(0, n, step):
        m = min(step, n - lo)
        z = torch.randn(m, generator=g, device="cuda")
        c = torch.randn(3, m, generator=g, device="cuda").square_().sum(0).div_(3.0).sqrt_()
        x = z.div_(c).mul_(1e-4)
        x[torch.rand(m, generator=g, device="cuda") < 1e-3] = 0.0
        out[lo:lo + m] = x.to(torch.bfloat16)
    return out


@pytest.mark.parametrize("bits", [1, 3, 8])
def test_billion_element_bf16_stress_sampled(bits):
    free, _ = torch.cuda.mem_get_info()
    n, B, W = 1_000_000_000, 4096, 16
    if free < 40e9:
        pytest.skip("needs 40 GB of free device memory")
    grad = _student_t_bf16_on_device(n, seed=1804080665)
    nb = mqg.mqg_num_buckets(n, B)
    assert nb == 244_141 and n - (nb - 1) * B == 2560
    rng = np.random.default_rng(bits)
    sample = np.unique(np.concatenate([[0, 1, nb - 2, nb - 1, (1 << 29) // B - 1, (1 << 29) // B],
                                       rng.integers(0, nb, 300)]))
    # two of the sixteen workers are encoded (one gradient buffer serves all: distinct worker
    # ids still give distinct codes); the server step then runs with W = 16 over those two
    workers = [0, W - 1]
    codes = {w: torch.empty(mqg.mqg_code_words(n, bits), dtype=torch.int32, device="cuda") for w in workers}
    scales = {w: torch.empty(nb, dtype=torch.float32, device="cuda") for w in workers}
    for w in workers:
        mqg.mqg_quantize(grad, n, bits, B, 5, codes[w], scales[w], worker=w, step=9)
    torch.cuda.synchronize()
    wpb = B * bits // 32                                   # words per full bucket
    host = {}
    for k in sample.tolist():
        lo, hi = k * B, min(n, (k + 1) * B)
        xb = grad[lo:hi].view(torch.int16).cpu().numpy().view(np.uint16)
        for w in workers:
            c_ref, s_ref = O.quantize(xb, bits, B, 5, worker=w, step=9, elem_offset=lo, dtype="bf16")
            got_c = codes[w][k * wpb:k * wpb + c_ref.size].cpu().numpy().view(np.uint32)
            assert scales[w][k].item() == s_ref[0], (k, w)
            assert np.array_equal(got_c, c_ref), (k, w)
            host[(k, w)] = (c_ref, s_ref)
    assert (grad[:1 << 24] == 0).sum().item() > 1000        # the exact zeros are there

    params = torch.full((n,), 0.25, dtype=torch.float32, device="cuda")
    order = [workers[i % 2] for i in range(W)]
    mqg.mqg_server_step([codes[w] for w in order], [scales[w] for w in order], W, bits, n, B, params, 0.01)
    torch.cuda.synchronize()
    for k in sample.tolist():
        lo, hi = k * B, min(n, (k + 1) * B)
        p_ref = np.full(hi - lo, 0.25, np.float32)
        O.server_step([host[(k, w)][0] for w in order], [host[(k, w)][1] for w in order], bits, hi - lo, B, p_ref, 0.01)
        assert bits_equal(params[lo:hi].cpu().numpy(), p_ref) == 0, k
    assert mqg.mqg_device_timeouts() == 0


@pytest.mark.parametrize("bits", [3, 8])
def test_batched_bf16_bucket_4096_four_workers(bits):
    """The stress shape's kernel instantiation (bf16 input widened in the kernel, bucket 4096) in the
    batched launch, 4 workers x (2^26 + 2560) elements (16,385 buckets per worker, the last one short),
    every element of every worker against the CPU checker."""
    from concurrent.futures import ThreadPoolExecutor
    n, B, W = (1 << 26) + 2560, 4096, 4
    with ThreadPoolExecutor(W) as ex:
        xs = list(ex.map(lambda w: wl.student_t_bf16(n, config=5, worker=w), range(W)))
        refs = list(ex.map(lambda w: O.quantize(xs[w], bits, B, 6, worker=10 + w, step=2, elem_offset=1 << 20,
                                                dtype="bf16"), range(W)))
    grads = [to_dev(x.view(np.int16)).view(torch.bfloat16) for x in xs]
    codes = [Guarded(mqg.mqg_code_words(n, bits), torch.int32) for _ in range(W)]
    scales = [Guarded(mqg.mqg_num_buckets(n, B), torch.float32) for _ in range(W)]
    mqg.mqg_quantize_workers(grads, W, n, bits, B, 6, [c.view for c in codes], [s.view for s in scales],
                             first_worker=10, step=2, elem_offset=1 << 20)
    torch.cuda.synchronize()
    for w in range(W):
        codes[w].check_guards(), scales[w].check_guards()
        assert bits_equal(scales[w].numpy(np.float32), refs[w][1]) == 0, w
        assert np.array_equal(codes[w].numpy(np.uint32), refs[w][0]), w
    assert mqg.mqg_device_timeouts() == 0
