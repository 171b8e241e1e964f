"""The other workloads of the benchmark specification, measured after bench.py's timed region and
reported in its JSON line under `configs`: the small launch-bound case (`configs[0]`), the layered
AlexNet-shaped gradient with one scale per tensor (`configs[2]`) and the stress shape (`configs[4]`:
10^9 bf16 elements, 16 workers), and the end-to-end training loop with the host bit selector (`configs[3]`:
the share of an iteration spent inside the library).  The headline numbers (`value`, `roofline`) stay those of
`configs[1]`; nothing here changes them.

Every kernel is timed as GROUP launches back to back between one pair of CUDA events on torch's
current stream (the stream the library is given), REPS groups: `us` is the median group's time
per launch, `us_best` the best group's.  Inputs of a launch are larger than L2 or rotate over
buffer sets, as stated per entry.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

PHILOX_SEED = 2
# executed instructions per element of quantize_tma / quantize_workers_kernel<K, bf16> (ncu, smsp__inst_executed:
# profiles/per_width_counters_small_cases.md)
BF16_QUANTIZE_INST_PER_ELEM = 14.3


def _time_groups(torch, stream, launch, group, reps, warm=2):
    for i in range(warm):
        launch(i)
    out, i = [], warm
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(group):
            launch(i)
            i += 1
        e1.record(stream)
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) * 1e3 / group)          # us per launch
    return float(np.median(out)), float(min(out))


def _entry(us, best, nbytes, peak):
    return {"us": us, "us_best": best, "moved_gbs": nbytes / us / 1e3,
            "frac_of_measured_peak": nbytes / us / 1e3 / peak, "frac_of_8tbs": nbytes / us / 1e3 / 8000.0,
            "algorithmic_bytes": nbytes}


def _ptrs(tensors):
    return (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def small_case(torch, mqg, lib, check, peak):
    """configs[0]: n = 2^20 fp32 per worker, W = 4, N(0, 1e-3), bucket 512, K in {1, 2, 4, 8}.
    4 MiB per gradient: both launches are bound by launch latency, so the entry carries times and
    rates but no roofline claim."""
    from paper_1804_08066_b200 import workloads as wl
    n, W, B, lr = 1 << 20, 4, 512, 0.1 / 4
    stream = torch.cuda.current_stream()
    sptr = C.c_void_p(stream.cuda_stream)
    grads = [torch.from_numpy(wl.normal(n, 1e-3, config=1, worker=w)).cuda() for w in range(W)]
    params = torch.from_numpy(wl.params(n, 0.05, config=1)).cuda()
    gtab = _ptrs(grads)
    rows = []
    for b in (1, 2, 4, 8):
        codes = [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(W)]
        scales = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
        ctab, stab = _ptrs(codes), _ptrs(scales)
        q = _time_groups(torch, stream, lambda i: check(lib.mqg_quantize_workers(
            gtab, W, n, b, B, 0, ctab, stab, 0, 0, i, 0, sptr)), 8, 5)
        s = _time_groups(torch, stream, lambda i: check(lib.mqg_server_step(
            ctab, stab, W, b, n, B, params.data_ptr(), lr, None, sptr)), 8, 5)
        qb = W * (4 * n + 4 * mqg.mqg_code_words(n, b) + 4 * mqg.mqg_num_buckets(n, B))
        sb = 8 * n + W * (4 * mqg.mqg_code_words(n, b) + 4 * mqg.mqg_num_buckets(n, B))
        rows.append({"bits": b, "quantize_all_workers": _entry(q[0], q[1], qb, peak),
                     "server_step": _entry(s[0], s[1], sb, peak)})
    return {"workload": "configs[0]: n=1,048,576 fp32 per worker, W=4, iid N(0,1e-3), bucket 512, bits 1,2,4,8, "
                        "Philox seed 0, params N(0,0.05), lr 0.1/W",
            "note": "launch-bound (16 MiB of gradients per step, resident in L2): times and rates are reported, "
                    "no roofline claim is made for this size",
            "launches": "one mqg_quantize_workers launch for the 4 workers, one mqg_server_step launch",
            "per_bits": rows}


def layered_case(torch, mqg, lib, check, peak):
    """configs[2]: the AlexNet-shaped layered gradient (16 tensors, 60,965,224 fp32 elements), one
    scale per tensor, W = 8, K in {2, 4, 8}.  The quantizer reads the gradient twice (scale pass,
    encode pass): 8 + K/8 bytes per element; the fused server step moves W K/8 + 8."""
    from paper_1804_08066_b200 import workloads as wl
    W, lr = 8, 0.1 / 8
    stream = torch.cuda.current_stream()
    sptr = C.c_void_p(stream.cuda_stream)
    seg, sizes = wl.alexnet_segments()
    n, nseg = int(seg[-1]), len(sizes)
    seg_c = seg.ctypes.data_as(C.c_void_p)
    grads = [torch.from_numpy(wl.layered(sizes, config=3, worker=w)).cuda() for w in range(W)]
    gtab = _ptrs(grads)
    params = [torch.from_numpy(wl.params(n, 0.05, config=3)).cuda() for _ in range(3)]
    rows = []
    for b in (2, 4, 8):
        coff = np.concatenate([[0], np.cumsum([mqg.mqg_code_words(sz, b) for sz in sizes])]).astype(np.uint64)
        coff_c = coff.ctypes.data_as(C.c_void_p)
        words = int(coff[-1])
        code_sets = [[torch.zeros(words, dtype=torch.int32, device="cuda") for _ in range(W)] for _ in range(3)]
        scales = [torch.zeros(nseg, dtype=torch.float32, device="cuda") for _ in range(W)]
        ctabs = [_ptrs(cs) for cs in code_sets]
        stab = _ptrs(scales)

        def quantize(i):
            check(lib.mqg_quantize_segments_workers(gtab, W, nseg, seg_c, coff_c, b, PHILOX_SEED, ctabs[i % 3],
                                                    stab, 0, 0, i, 0, sptr))

        for r in range(3):
            quantize(r)                     # every code set holds valid codes
        q = _time_groups(torch, stream, quantize, 4, 5)

        def server(i):
            check(lib.mqg_server_step_segments(ctabs[i % 3], stab, W, b, nseg, seg_c, coff_c,
                                               params[i % 3].data_ptr(), lr, None, sptr))

        s = _time_groups(torch, stream, server, 8, 5)
        qb = W * (8 * n + 4 * words + 4 * nseg)
        sb = 8 * n + W * (4 * words + 4 * nseg)
        rows.append({"bits": b, "quantize_all_workers": _entry(q[0], q[1], qb, peak),
                     "quantize_us_per_worker": q[0] / W,
                     "server_step": _entry(s[0], s[1], sb, peak)})
        del code_sets, ctabs
    return {"workload": "configs[2]: AlexNet-shaped layered gradient, 16 tensors, 60,965,224 fp32 elements, layer "
                        "sigma log-uniform in [1e-5,1e-2], one scale per tensor, W=8, bits 2,4,8",
            "launches": "one mqg_quantize_segments_workers call for the 8 workers (scale pass + encode pass), one "
                        "mqg_server_step_segments call",
            "l2": "1.95 GB of gradients per quantize call; three rotating sets of code buffers and parameters",
            "bytes_per_element": "quantize 8 + K/8 (two reads), server W K/8 + 8",
            "per_bits": rows}


def stress_case(torch, mqg, lib, check, peak):
    """configs[4]: n = 10^9 bf16 elements widened in the kernel, W = 16, Student-t(3) x 1e-4 with 0.1 % exact
    zeros, bucket 4096, K = 1..8.  One gradient buffer serves all 16 worker ids (the draws differ by
    worker id, so the 16 code streams differ); codes for the widest K are allocated once and reused.
    The values are drawn on the device (same distribution as the parity tests' host generator, another
    stream of random numbers): 10^9 draws on the host would take longer than the rest of the benchmark."""
    n, W, B, lr = 1_000_000_000, 16, 4096, 0.1 / 16
    stream = torch.cuda.current_stream()
    sptr = C.c_void_p(stream.cuda_stream)
    need = 2 * n + W * 4 * mqg.mqg_code_words(n, 8) + W * 4 * mqg.mqg_num_buckets(n, B) + 4 * n
    free, total = torch.cuda.mem_get_info()
    if free < need + (8 << 30):
        return {"workload": "configs[4]: n=1e9 bf16, W=16", "skipped": "needs %.1f GB of device memory, %.1f GB free"
                % (need / 1e9, free / 1e9)}
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1804080665)
    grad = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        z = torch.randn(m, device="cuda", generator=gen)
        chi = (torch.randn(3, m, device="cuda", generator=gen) ** 2).sum(0) / 3.0
        t = z / chi.sqrt() * 1e-4
        t[torch.rand(m, device="cuda", generator=gen) < 1e-3] = 0.0
        grad[lo:lo + m] = t.to(torch.bfloat16)
        del z, chi, t
    codes = [torch.zeros(mqg.mqg_code_words(n, 8), dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
    params = torch.zeros(n, dtype=torch.float32, device="cuda")
    gtab, ctab, stab = _ptrs([grad] * W), _ptrs(codes), _ptrs(scales)
    rows = []
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    sm_mhz = float(getattr(props, "clock_rate", 1965000)) / 1e3                  # the device's maximum SM clock
    issue_peak = props.multi_processor_count * 4 * sm_mhz / 1e3                  # schedulers x GHz
    for b in range(1, 9):
        q = _time_groups(torch, stream, lambda i: check(lib.mqg_quantize_workers(
            gtab, W, n, b, B, PHILOX_SEED, ctab, stab, 1, 0, i, 0, sptr)), 2, 5, warm=1)
        s = _time_groups(torch, stream, lambda i: check(lib.mqg_server_step(
            ctab, stab, W, b, n, B, params.data_ptr(), lr, None, sptr)), 2, 5, warm=1)
        words, nb = mqg.mqg_code_words(n, b), mqg.mqg_num_buckets(n, B)
        qb = W * (2 * n + 4 * words + 4 * nb)
        sb = 8 * n + W * (4 * words + 4 * nb)
        row = {"bits": b, "quantize_all_workers": _entry(q[0], q[1], qb, peak),
               "quantize_us_per_worker": q[0] / W, "server_step": _entry(s[0], s[1], sb, peak)}
        row["quantize_all_workers"]["fp32_equivalent_grad_gbs"] = W * 4 * n / q[0] / 1e3
        # the ceiling this kernel actually runs against: warp instructions issued per second (14.3 executed
        # instructions per element, from the ncu counters of the bf16 instantiation) against one instruction
        # per cycle and scheduler at the maximum SM clock
        row["quantize_all_workers"]["issue_rate"] = {
            "bound": "alu", "instructions_per_element": BF16_QUANTIZE_INST_PER_ELEM,
            "achieved": W * n * BF16_QUANTIZE_INST_PER_ELEM / 32 / q[0] / 1e3, "peak": issue_peak,
            "unit": "G warp-instructions/s", "frac": W * n * BF16_QUANTIZE_INST_PER_ELEM / 32 / q[0] / 1e3 / issue_peak}
        rows.append(row)
    timeouts = mqg.mqg_device_timeouts()
    del grad, codes, scales, params
    torch.cuda.empty_cache()
    return {"workload": "configs[4]: n=1,000,000,000 bf16 (widened in the kernel), W=16, Student-t(3) x 1e-4 with "
                        "0.1% exact zeros, bucket 4096, bits 1..8",
            "footprint_bytes": need,
            "shared_gradient": "one 2 GB gradient buffer is read under all 16 worker ids (distinct draws per id); "
                               "code buffers sized for K=8 serve every K",
            "launches": "one mqg_quantize_workers launch (16 x 2 GB read), one mqg_server_step launch; groups of 2 "
                        "launches, 5 groups",
            "l2": "inputs far larger than L2",
            "device_timeouts": timeouts,
            "per_bits": rows}


def loop_case():
    """`configs[3]`: the whole loop (model gradients -> quantize -> fused server step -> host selector) with the
    paper's selector; what is reported is the share of an iteration spent in the library's two calls."""
    from paper_1804_08066_b200.train_loop import run
    r = run(iters=40, workers=4, selector="sarsa", seed=1)
    return {"workload": "configs[3]: 5-layer CNN (3x3 conv 32-64-128, FC 2048-256-10) on synthetic 32x32x3 images, "
                        "batch 128 per worker, W=4, bucket 2048, host SARSA selector picks the bits from the losses; "
                        "40 iterations",
            "note": "the model, its autograd and the selector are the harness's; the library is the codec and the "
                    "server step (one mqg_quantize per worker, one mqg_server_step per iteration)",
            "parameters": r["parameters"], "libmqgrad_ms_per_iter": r["libmqgrad_ms_per_iter"],
            "iteration_ms": r["iteration_ms"], "libmqgrad_share_pct": r["libmqgrad_share_pct"],
            "bits_chosen_first_last": [r["bits_chosen"][0], r["bits_chosen"][-1]],
            "first_loss": r["first_loss"], "last_loss": r["last_loss"],
            "uplink_bytes_per_iter": r["uplink_bytes_per_iter"], "uplink_bytes_fp32": r["uplink_bytes_fp32"],
            "paper_table3_share_pct": r["paper_table3_share_pct"]}


def run_all(torch, mqg, lib, check, peak):
    out = {}
    for name, fn in (("config0_small", small_case), ("config2_layered", layered_case), ("config4_stress", stress_case)):
        out[name] = fn(torch, mqg, lib, check, peak)
        torch.cuda.synchronize()
    out["config3_loop"] = loop_case()
    torch.cuda.synchronize()
    return out
