#!/usr/bin/env python
"""Benchmark of the MQGrad hot path on B200: quantize+pack and unpack+accumulate+update.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (the configuration the headline metric is quoted on): one flat gradient of
n = 25,000,000 fp32 per worker, W = 8 simulated workers, iid Laplace(0, 1e-4), bucket 2048,
bit widths 1..8.  One step = one pass of the whole path for every bit width: the quantize phase
(per bit width one mqg_quantize_workers launch over all W gradients, 800 MB; or, with
--quantize-launch per-worker, W mqg_quantize launches of 100 MB each) followed by 8 fused server
launches (each reads W code buffers and updates its own 100 MB parameter replica), so every
launch reads inputs that have been evicted from L2 (> 1.7 GB cycles between reuses).

Prints ONE JSON line (rank 0).  `value` is GB/s of fp32 gradient through the whole path
(8 * W * 4n bytes per step / step time) with all inputs resident in HBM; `e2e` is the same
metric with the gradients starting in pinned host memory and the updated parameters read
back, copies inside the timed region; `roofline` describes the dominant kernel (the quantize
kernel) and `roofline_server` the fused server kernel, both from events at the phase boundaries
inside the timed region; `per_bits` lists both kernels for every bit width, each timed on its own
after the timed region (groups of 8 launches back to back on rotating buffers after a short idle,
i.e. with the SM clock at its maximum: median and best group; 20 launches each between its own
events; and `*_sustained`, the same launch after a quarter of a second of itself back to back,
when the board's power limit has lowered the clock); `cpu_baseline` is the scalar CPU
checker timed on a bounded sample of the same workload.

--impl reference times the CPU checker alone (rank 0 only).
With --gpus N > 1 (under torchrun) every rank runs an independent replica of the workload
on its own GPU; there is no data-path collective.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

N_ELEMS = 25_000_000
N_WORKERS = 8
BUCKET = 2048
ALL_BITS = list(range(1, 9))
LAPLACE_SCALE = 1e-4
LR = 0.1 / N_WORKERS
PHILOX_SEED = 2
METRIC = "quantize+pack and dequant+accumulate+update GB/s (fp32 grad) per bit width; % HBM peak"
UNIT = "GB/s of fp32 gradient through quantize+pack -> unpack+accumulate+update"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per element and bit width, from the ncu captures on small
# cases summarised in profiles/per_width_counters_small_cases.md (quantize_workers_kernel: 4 x 8,388,608
# elements; server_tma_kernel: n = 2^25, W = 8; both bucket 2048).  DRAM traffic grows in proportion to the
# elements, so a launch's traffic is the figure times its elements.  Writes are partly still in L2 when a
# kernel ends, hence less than the algorithmic bytes (4 + K/8 and 8 + W K/8 per element).
QUANTIZE_DRAM_BYTES_PER_ELEM = {1: 4.0744, 2: 4.1027, 3: 4.151, 4: 4.1934, 5: 4.229, 6: 4.2763, 7: 4.3382, 8: 4.3993}
SERVER_DRAM_BYTES_PER_ELEM = {1: 7.2455, 2: 8.2828, 3: 9.3616, 4: 10.404, 5: 11.6736, 6: 12.7431, 7: 13.8224, 8: 14.858}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def quantize_bytes(n, bits, bucket):
    """Algorithmic bytes of one quantize launch: read fp32, write codes and scales."""
    return 4 * n + 4 * ((n * bits + 31) // 32) + 4 * ((n + bucket - 1) // bucket)


def requantize_bytes(n, bits, bucket, W):
    """Algorithmic bytes of one downlink launch: W code streams and scale arrays in, one of each out."""
    return (W + 1) * quantize_bytes(n, bits, bucket) - (W + 1) * 4 * n


def server_bytes(n, bits, bucket, W):
    """Algorithmic bytes of one fused server launch: W code streams + W scale arrays + params r/w."""
    return W * (4 * ((n * bits + 31) // 32) + 4 * ((n + bucket - 1) // bucket)) + 8 * n


# --------------------------------------------------------------------------------------
# clocks: sampled with NVML while the timed region runs (read-only queries)
# --------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
        0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
        0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = device_index
            if visible:
                ids = [v for v in visible.split(",") if v.strip() != ""]
                if device_index < len(ids) and ids[device_index].strip().isdigit():
                    phys = int(ids[device_index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "sm_mhz_min": float(min(self.samples)), "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------------------
# CPU checker leg (the oracle as it stands; bench.py is one of the few places allowed to run it)
# --------------------------------------------------------------------------------------
def oracle_pass(grads, n_s, bits_list, threads):
    """One pass of the whole path on the first n_s elements of every worker, on the CPU checker.
    Bit widths are independent and run on `threads` host threads.  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import mqg_oracle as O

    def one(bits):
        codes, scales = [], []
        for w, g in enumerate(grads):
            c, s = O.quantize(g[:n_s], bits, BUCKET, PHILOX_SEED, worker=w)
            codes.append(c), scales.append(s)
        p = np.zeros(n_s, np.float32)
        O.server_step(codes, scales, bits, n_s, BUCKET, p, LR)
        return float(p[0])

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(one, bits_list))
    return time.perf_counter() - t0


def host_threads():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def make_grads(n, workers):
    from concurrent.futures import ThreadPoolExecutor

    from paper_1804_08066_b200 import workloads as wl
    with ThreadPoolExecutor(max_workers=min(workers, host_threads())) as ex:
        return list(ex.map(lambda w: wl.laplace(n, LAPLACE_SCALE, config=2, worker=w), range(workers)))


def cpu_baseline(grads, target_seconds=20.0):
    cores = host_threads()
    threads = max(1, min(cores, len(ALL_BITS)))
    probe = 32 * BUCKET
    t = oracle_pass(grads, probe, ALL_BITS, threads)
    per_elem = t / probe
    n_s = int(target_seconds / threads / max(per_elem, 1e-12))     # ~target_seconds of CPU work
    n_s = max(BUCKET, min(N_ELEMS // BUCKET * BUCKET, n_s // BUCKET * BUCKET))
    secs = oracle_pass(grads, n_s, ALL_BITS, threads)
    gbs = len(ALL_BITS) * len(grads) * 4 * n_s / secs / 1e9
    # the same checker on ONE host thread (the definition's own speed), on a sample 1/32 the size
    n_1 = max(BUCKET, n_s // 32 // BUCKET * BUCKET)
    secs_1 = oracle_pass(grads, n_1, ALL_BITS, 1)
    gbs_1 = len(ALL_BITS) * len(grads) * 4 * n_1 / secs_1 / 1e9
    return {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "first %d of %d elements of each of %d workers, bits 1..8, one pass in %.2f s"
                      % (n_s, N_ELEMS, len(grads), secs),
            "single_thread": {"value": gbs_1, "cores": 1,
                              "sample": "first %d elements of each of %d workers, bits 1..8, one pass in %.2f s"
                                        % (n_1, len(grads), secs_1)}}, n_s


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    t_budget = 150.0
    n_probe = 16 * BUCKET
    grads = make_grads(max(n_probe, 2_000_000), N_WORKERS)
    cores = host_threads()
    threads = max(1, min(cores, len(ALL_BITS)))
    t = oracle_pass(grads, n_probe, ALL_BITS, threads)
    per_elem = t / n_probe
    total_steps = args.steps + args.warmup
    n_s = int(t_budget / max(total_steps, 1) / max(per_elem, 1e-12))
    n_s = max(BUCKET, min(grads[0].size // BUCKET * BUCKET, n_s // BUCKET * BUCKET))
    for _ in range(args.warmup):
        oracle_pass(grads, n_s, ALL_BITS, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(grads, n_s, ALL_BITS, threads)
    dt = time.perf_counter() - t0
    gbs = args.steps * len(ALL_BITS) * N_WORKERS * 4 * n_s / dt / 1e9
    sample = ("each step = first %d of %d elements of each of %d workers, bits 1..8"
              % (n_s, N_ELEMS, N_WORKERS))
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": workload_config(),
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def slowest_rank_ms(ms, dist, device):
    """Elapsed time of the job = the slowest rank's (every rank runs an independent replica)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(world, grad_bytes_per_rank_step, ms_per_step):
    """Aggregate throughput of `world` replicas that each push grad_bytes per step."""
    return world * grad_bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def workload_config():
    return {"workload": "configs[1]: flat ResNet-50-sized gradient, n=25,000,000 fp32 per worker, W=8, "
                        "iid Laplace(0,1e-4), bucket 2048, bits 1..8",
            "n": N_ELEMS, "workers": N_WORKERS, "bucket": BUCKET, "bits": ALL_BITS,
            "l2": "inputs larger than L2: every launch reads buffers last touched > 1.7 GB of traffic ago",
            "multi_gpu": "replicas only"}


# --------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------
def run_ours(args):
    import torch

    import paper_1804_08066_b200 as mqg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libmqgrad has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    n, W, B = N_ELEMS, N_WORKERS, BUCKET
    lib = mqg.raw_library()
    host_grads = make_grads(n, W)
    pinned = [torch.from_numpy(g).pin_memory() for g in host_grads]
    grads = [p.cuda(non_blocking=True) for p in pinned]
    from paper_1804_08066_b200 import workloads as wl
    params0 = torch.from_numpy(wl.params(n, 0.05, config=2)).cuda()
    params = {b: params0.clone() for b in ALL_BITS}
    codes = {b: [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(W)]
             for b in ALL_BITS}
    scales = {b: [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
              for b in ALL_BITS}
    host_params = torch.empty(n, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    sptr = C.c_void_p(stream.cuda_stream)
    code_tab = {b: (C.c_void_p * W)(*[t.data_ptr() for t in codes[b]]) for b in ALL_BITS}
    scale_tab = {b: (C.c_void_p * W)(*[t.data_ptr() for t in scales[b]]) for b in ALL_BITS}

    def check(rc):
        if rc != 0:
            raise RuntimeError("libmqgrad: %d %s" % (rc, mqg.mqg_last_error()))

    grad_tab = (C.c_void_p * W)(*[t.data_ptr() for t in grads])
    batched = args.quantize_launch == "batched"

    def quantize_per_worker(b, step_no):
        for w in range(W):
            check(lib.mqg_quantize(grads[w].data_ptr(), n, b, B, PHILOX_SEED, codes[b][w].data_ptr(),
                                   scales[b][w].data_ptr(), 0, w, step_no, 0, sptr))

    def quantize_batched(b, step_no):
        check(lib.mqg_quantize_workers(grad_tab, W, n, b, B, PHILOX_SEED, code_tab[b], scale_tab[b], 0, 0,
                                       step_no, 0, sptr))

    quantize_all = quantize_batched if batched else quantize_per_worker
    q_launches = 1 if batched else W       # quantize launches per bit width

    def server(b):
        check(lib.mqg_server_step(code_tab[b], scale_tab[b], W, b, n, B, params[b].data_ptr(), LR,
                                  None, sptr))

    def step(step_no, phases=None):
        """One pass of the whole path.  `phases`: three events per step (start, quantize phase done,
        server phase done); launches inside a phase run back to back."""
        if phases is not None:
            p0 = torch.cuda.Event(enable_timing=True)
            p0.record(stream)
        for b in ALL_BITS:
            quantize_all(b, step_no)
        if phases is not None:
            p1 = torch.cuda.Event(enable_timing=True)
            p1.record(stream)
        for b in ALL_BITS:
            server(b)
        if phases is not None:
            p2 = torch.cuda.Event(enable_timing=True)
            p2.record(stream)
            phases.append((p0, p1, p2))

    # The read-back of the updated parameters runs on its own stream, so that it shares the (full-duplex)
    # host link with the next bit width's gradient upload instead of waiting in front of it.
    d2h_stream = torch.cuda.Stream()

    def e2e_step(step_no):
        for b in ALL_BITS:
            for w in range(W):
                grads[w].copy_(pinned[w], non_blocking=True)
                check(lib.mqg_quantize(grads[w].data_ptr(), n, b, B, PHILOX_SEED, codes[b][w].data_ptr(),
                                       scales[b][w].data_ptr(), 0, w, step_no, 0, sptr))
            server(b)
            updated = torch.cuda.Event()
            updated.record(stream)
            d2h_stream.wait_event(updated)
            with torch.cuda.stream(d2h_stream):
                host_params.copy_(params[b], non_blocking=True)
        stream.wait_stream(d2h_stream)             # the step ends when its last result is on the host

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        return slowest_rank_ms(ms, dist, "cuda")

    # ---- device-resident timing
    for i in range(args.warmup):
        step(i)
    phases = []
    barrier()
    with ClockSampler(local_rank) as clocks:
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_begin.record(stream)
        for i in range(args.steps):
            step(args.warmup + i, phases=phases)
        t_end.record(stream)
        barrier()
    total_ms = max_over_ranks(t_begin.elapsed_time(t_end))
    ms_per_step = total_ms / args.steps
    grad_bytes_per_step = len(ALL_BITS) * W * 4 * n
    value = whole_job_gbs(world, grad_bytes_per_step, ms_per_step)
    q_phase_s = float(np.mean([p0.elapsed_time(p1) for p0, p1, _ in phases])) * 1e-3
    s_phase_s = float(np.mean([p1.elapsed_time(p2) for _, p1, p2 in phases])) * 1e-3

    # ---- per bit width: each kernel timed on its own, K by K.  A group is GROUP launches of the same
    # kernel back to back between one pair of events (as they run inside a step: no event between two
    # launches), on rotating buffer sets so that no launch finds its inputs in L2; `us` is the median
    # over REPS groups of the group's time per launch, `us_best` the best group.  `single` figures are
    # SINGLES launches each between its own pair of events (an event after every launch keeps the next
    # one from being set up while it runs, so these are a few microseconds longer).
    # Power.  A launch sequence that runs for more than a few tens of milliseconds is held at the board's
    # power limit: the SM clock falls from its maximum to 1650 - 1800 MHz (seen with 5 ms samples; the
    # limit is often not reported as a reason) and kernels bound by instruction issue slow down with it.
    # Both regimes are reported: `*_us` after IDLE_S seconds of idle (clock at its maximum, the regime the
    # copy-rate denominator was measured in), `*_us_sustained` after SUSTAIN_S seconds of the same launch
    # back to back.
    GROUP, REPS, SINGLES = 8, 5, 20
    IDLE_S, SUSTAIN_S = 0.4, 0.25

    def time_sustained(launch, est_ms):
        warm = max(GROUP, int(SUSTAIN_S * 1e3 / max(est_ms, 1e-3)))
        count = GROUP * REPS
        for i in range(warm):
            launch(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(count):
            launch(warm + i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    def time_groups(launch):
        torch.cuda.synchronize()
        time.sleep(IDLE_S)
        for i in range(2):
            launch(i)
        out, i = [], 2
        for _ in range(REPS):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(GROUP):
                launch(i)
                i += 1
            e1.record(stream)
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / GROUP)
        return out

    def time_singles(launch):
        pairs = []
        for i in range(SINGLES):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            launch(i)
            e1.record(stream)
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        return [e0.elapsed_time(e1) for e0, e1 in pairs]

    q_ms, s_ms, q_single, s_single, q_sust, s_sust = {}, {}, {}, {}, {}, {}
    for b in ALL_BITS:
        q_ms[b] = time_groups(lambda i: quantize_all(b, i))
        q_single[b] = time_singles(lambda i: quantize_all(b, 100 + i))
        q_sust[b] = time_sustained(lambda i: quantize_all(b, 200 + i), float(np.median(q_ms[b])))
        # three sets of this width's code buffers, every parameter replica in turn: 2 launches
        # (> 450 MB of traffic) lie between two uses of a code set, 7 between two uses of a replica
        sets = [code_tab[b]]
        keep = []
        for _ in range(2):
            cp = [t.clone() for t in codes[b]]
            keep.append(cp)
            sets.append((C.c_void_p * W)(*[t.data_ptr() for t in cp]))

        def server_rot(i):
            check(lib.mqg_server_step(sets[i % 3], scale_tab[b], W, b, n, B,
                                      params[ALL_BITS[i % len(ALL_BITS)]].data_ptr(), LR, None, sptr))

        s_ms[b] = time_groups(server_rot)
        s_single[b] = time_singles(server_rot)
        s_sust[b] = time_sustained(server_rot, float(np.median(s_ms[b])))
        del keep, sets
    torch.cuda.synchronize()

    # the other way of launching the quantize phase, timed on its own for comparison
    other = quantize_per_worker if batched else quantize_batched
    other_ms = {}
    for b in ALL_BITS:
        for i in range(3):
            other(b, i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            other(b, 3 + i)
        e1.record(stream)
        torch.cuda.synchronize()
        other_ms[b] = e0.elapsed_time(e1) / args.steps
    if batched:                            # leave the codes as the timed path writes them
        for b in ALL_BITS:
            quantize_all(b, args.warmup + args.steps - 1)
        torch.cuda.synchronize()

    peak, peak_kind = measured_hbm_peak()
    per_bits = []
    q_bytes_total = q_time_total = 0.0
    s_bytes_total = s_time_total = 0.0
    for b in ALL_BITS:
        tq = float(np.median(q_ms[b])) / W * 1e-3          # per worker's gradient
        ts = float(np.median(s_ms[b])) * 1e-3
        qb, sb = quantize_bytes(n, b, B), server_bytes(n, b, B, W)
        q_bytes_total += qb * W; q_time_total += tq * W
        s_bytes_total += sb; s_time_total += ts
        per_bits.append({
            "bits": b,
            "quantize_us": tq * 1e6, "quantize_grad_gbs": 4 * n / tq / 1e9, "quantize_moved_gbs": qb / tq / 1e9,
            "quantize_frac_of_measured": qb / tq / 1e9 / peak, "quantize_frac_of_8tbs": qb / tq / 1e9 / NOMINAL_HBM_GBS,
            "server_us": ts * 1e6, "server_grad_gbs": 4 * n * W / ts / 1e9, "server_moved_gbs": sb / ts / 1e9,
            "server_frac_of_measured": sb / ts / 1e9 / peak, "server_frac_of_8tbs": sb / ts / 1e9 / NOMINAL_HBM_GBS,
            "quantize_us_sustained": q_sust[b] / W * 1e3,
            "quantize_frac_of_measured_sustained": qb / (q_sust[b] / W * 1e-3) / 1e9 / peak,
            "server_us_sustained": s_sust[b] * 1e3,
            "server_frac_of_measured_sustained": sb / (s_sust[b] * 1e-3) / 1e9 / peak,
            "quantize_us_best": min(q_ms[b]) / W * 1e3,
            "quantize_us_single_median": float(np.median(q_single[b])) / W * 1e3,
            "quantize_us_single_best": min(q_single[b]) / W * 1e3,
            "server_us_best": min(s_ms[b]) * 1e3,
            "server_us_single_median": float(np.median(s_single[b])) * 1e3,
            "server_us_single_best": min(s_single[b]) * 1e3,
            "quantize_dram_traffic": QUANTIZE_DRAM_BYTES_PER_ELEM[b] * n, "quantize_algorithmic_bytes": qb,
            "server_dram_traffic": SERVER_DRAM_BYTES_PER_ELEM[b] * n, "server_algorithmic_bytes": sb,
            "wire_bytes_per_worker": mqg.mqg_wire_bytes(n, b, B),
            ("quantize_us_per_worker_launches" if batched else "quantize_us_one_launch"): other_ms[b] / W * 1e3,
        })
    # the roofline figures come from the timed region: bytes of a phase / its duration
    q_achieved = q_bytes_total / q_phase_s / 1e9
    s_achieved = s_bytes_total / s_phase_s / 1e9
    q_time_total, s_time_total = q_phase_s, s_phase_s
    q_kernel = "quantize_workers_kernel" if batched else "quantize_tma_kernel"
    q_per_launch = W if batched else 1     # gradients one launch encodes
    roofline = {"kernel": "%s (all bit widths, %d launches per step, %d gradient(s) of n per launch)"
                          % (q_kernel, len(ALL_BITS) * q_launches, q_per_launch),
                "bound": "hbm", "achieved": q_achieved, "peak": peak, "peak_kind": peak_kind + " copy rate",
                "unit": "GB/s", "frac": q_achieved / peak,
                "avg_launch_us": q_phase_s / (len(ALL_BITS) * q_launches) * 1e6,
                "traffic": float(np.mean([QUANTIZE_DRAM_BYTES_PER_ELEM[b] for b in ALL_BITS])) * n * q_per_launch,
                "traffic_note": "dram read+write bytes per launch, mean over the eight bit widths of the phase "
                                "(`per_bits[].quantize_dram_traffic` has each width), from the ncu captures of "
                                "profiles/per_width_counters_small_cases.md scaled to the elements of one launch; "
                                "algorithmic bytes of a launch, same mean: %d"
                                % int(np.mean([quantize_bytes(n, b, B) for b in ALL_BITS]) * q_per_launch),
                "time_share_of_step": q_time_total / (q_time_total + s_time_total)}
    roofline_server = {"kernel": "server_tma_kernel (fused step, all bit widths, %d launches per step)" % len(ALL_BITS),
                       "bound": "hbm", "achieved": s_achieved, "peak": peak, "peak_kind": peak_kind + " copy rate",
                       "unit": "GB/s", "frac": s_achieved / peak,
                       "avg_launch_us": s_phase_s / len(ALL_BITS) * 1e6,
                       "traffic": float(np.mean([SERVER_DRAM_BYTES_PER_ELEM[b] for b in ALL_BITS])) * n,
                       "traffic_note": "dram read+write bytes per launch, mean over the eight bit widths (each "
                                       "width: `per_bits[].server_dram_traffic`), same source; algorithmic: %d"
                                       % int(np.mean([server_bytes(n, b, B, W) for b in ALL_BITS]))}

    # ---- the downlink (outside `value`): the server re-quantizes the mean for the broadcast.  ALU-bound:
    # per element 4 W + 13 lane operations (per worker 1 extract + 3 fp for the decode and sum; mean, max,
    # 5 of Philox, 5 of the encode, 1 pack) against 148 SMs x 128 lanes x the SM clock.
    down_codes = torch.zeros(mqg.mqg_code_words(n, max(ALL_BITS)), dtype=torch.int32, device="cuda")
    down_scales = torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda")

    def downlink(b, step_no):
        check(lib.mqg_server_requantize(code_tab[b], scale_tab[b], W, b, n, B, C.c_float(1.0 / W), PHILOX_SEED,
                                        down_codes.data_ptr(), down_scales.data_ptr(), W, step_no, sptr))

    down_steps = max(3, min(args.steps, 20))
    for b in ALL_BITS:
        downlink(b, 0)
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record(stream)
    for i in range(down_steps):
        for b in ALL_BITS:                 # every K reads its own 8 code buffers: 900 MB between reuses
            downlink(b, 1 + i)
    d1.record(stream)
    torch.cuda.synchronize()
    down_us = d0.elapsed_time(d1) * 1e3 / (down_steps * len(ALL_BITS))
    sm_clock_hz = (clocks.summary().get("sm_mhz") or 1965.0) * 1e6
    alu_peak = 148 * 128 * sm_clock_hz / 1e9
    alu_achieved = (4 * W + 13) * n / (down_us * 1e-6) / 1e9
    downlink_line = {"kernel": "requantize_warp_kernel (mqg_server_requantize, all bit widths, not part of `value`)",
                     "avg_launch_us": down_us, "grad_gbs": 4 * n * W / (down_us * 1e-6) / 1e9,
                     "roofline": {"bound": "alu", "achieved": alu_achieved, "peak": alu_peak,
                                  "unit": "G lane-op/s", "frac": alu_achieved / alu_peak, "traffic": None,
                                  "peak_kind": "148 SMs x 128 lanes x sampled SM clock",
                                  "ops_per_element": 4 * W + 13}}

    # ---- codec variant (outside `value`): (min, max) range with nearest rounding, same workload; bytes per
    # element as the main codec plus 4 / B for the second float of a range.  The quantize phase is one
    # mqg_quantize_workers_minmax launch per bit width for all workers; one launch per worker is timed beside it.
    mm_ranges = [torch.zeros(2 * mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
    mm_tab = (C.c_void_p * W)(*[t.data_ptr() for t in mm_ranges])
    mm_steps = max(3, min(args.steps, 20))

    def mm_quantize_per_worker(b):
        for w in range(W):
            check(lib.mqg_quantize_minmax(grads[w].data_ptr(), n, b, B, codes[b][w].data_ptr(),
                                          mm_ranges[w].data_ptr(), 0, sptr))

    def mm_quantize(b):
        check(lib.mqg_quantize_workers_minmax(grad_tab, W, n, b, B, code_tab[b], mm_tab, 0, sptr))

    def mm_server(b):
        check(lib.mqg_server_step_minmax(code_tab[b], mm_tab, W, b, n, B, params[b].data_ptr(), LR, None, sptr))

    for b in ALL_BITS:
        mm_quantize_per_worker(b)
    torch.cuda.synchronize()
    time.sleep(0.4)
    mm_quantize_per_worker(1)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for i in range(mm_steps):
        for b in ALL_BITS:
            mm_quantize_per_worker(b)
    p1.record(stream)
    torch.cuda.synchronize()
    mm_pw_s = p0.elapsed_time(p1) * 1e-3 / mm_steps
    for b in ALL_BITS:
        mm_quantize(b)
    torch.cuda.synchronize()
    time.sleep(0.4)
    mm_quantize(1)
    mm_events = []
    for i in range(mm_steps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record(stream)
        for b in ALL_BITS:
            mm_quantize(b)
        ev[1].record(stream)
        for b in ALL_BITS:
            mm_server(b)
        ev[2].record(stream)
        mm_events.append(ev)
    torch.cuda.synchronize()
    mm_q_s = float(np.mean([e[0].elapsed_time(e[1]) for e in mm_events])) * 1e-3
    mm_s_s = float(np.mean([e[1].elapsed_time(e[2]) for e in mm_events])) * 1e-3
    extra = 4 * mqg.mqg_num_buckets(n, B)
    mm_q_bytes = sum(W * (quantize_bytes(n, b, B) + extra) for b in ALL_BITS)
    mm_s_bytes = sum(server_bytes(n, b, B, W) + W * extra for b in ALL_BITS)
    variant_minmax = {
        "codec": "(min, max) range per bucket, nearest rounding (mqg_quantize_workers_minmax: one launch per bit "
                 "width for all workers / mqg_server_step_minmax); not part of `value`",
        "quantize": {"avg_launch_us": mm_q_s / len(ALL_BITS) * 1e6, "launches_per_step": len(ALL_BITS),
                     "us_per_gradient": mm_q_s / (len(ALL_BITS) * W) * 1e6,
                     "us_per_gradient_one_launch_per_worker": mm_pw_s / (len(ALL_BITS) * W) * 1e6,
                     "roofline": {"bound": "hbm", "achieved": mm_q_bytes / mm_q_s / 1e9, "peak": peak, "unit": "GB/s",
                                  "frac": mm_q_bytes / mm_q_s / 1e9 / peak, "traffic": None}},
        "server": {"avg_launch_us": mm_s_s / len(ALL_BITS) * 1e6, "launches_per_step": len(ALL_BITS),
                   "roofline": {"bound": "hbm", "achieved": mm_s_bytes / mm_s_s / 1e9, "peak": peak, "unit": "GB/s",
                                "frac": mm_s_bytes / mm_s_s / 1e9 / peak, "traffic": None}},
    }
    # ---- codec variant (outside `value`): L2-norm scale; only the quantizer differs (bytes per element as the
    # main codec), the server step is the main codec's.  Timed both ways of launching, as the main codec: one
    # mqg_quantize_workers_l2 launch per bit width for all workers, and one mqg_quantize_l2 launch per worker.
    def l2_quantize(b, step_no):
        for w in range(W):
            check(lib.mqg_quantize_l2(grads[w].data_ptr(), n, b, B, PHILOX_SEED, codes[b][w].data_ptr(),
                                      scales[b][w].data_ptr(), 0, w, step_no, 0, sptr))

    def l2_quantize_batched(b, step_no):
        check(lib.mqg_quantize_workers_l2(grad_tab, W, n, b, B, PHILOX_SEED, code_tab[b], scale_tab[b], 0, 0,
                                          step_no, 0, sptr))

    def l2_time(fn):
        for b in ALL_BITS:
            fn(b, 0)
        torch.cuda.synchronize()
        time.sleep(0.4)
        fn(1, 0)
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record(stream)
        for i in range(mm_steps):
            for b in ALL_BITS:
                fn(b, 1 + i)
        l1.record(stream)
        torch.cuda.synchronize()
        return l0.elapsed_time(l1) * 1e-3 / mm_steps

    l2_pw_s = l2_time(l2_quantize)
    l2_q_s = l2_time(l2_quantize_batched)
    l2_q_bytes = sum(W * quantize_bytes(n, b, B) for b in ALL_BITS)
    variant_l2 = {
        "codec": "L2-norm scale per bucket, fixed summation tree (mqg_quantize_workers_l2: one launch per bit "
                 "width for all workers; server step as the main codec); not part of `value`",
        "quantize": {"avg_launch_us": l2_q_s / len(ALL_BITS) * 1e6, "launches_per_step": len(ALL_BITS),
                     "us_per_gradient": l2_q_s / (len(ALL_BITS) * W) * 1e6,
                     "us_per_gradient_one_launch_per_worker": l2_pw_s / (len(ALL_BITS) * W) * 1e6,
                     "roofline": {"bound": "hbm", "achieved": l2_q_bytes / l2_q_s / 1e9, "peak": peak, "unit": "GB/s",
                                  "frac": l2_q_bytes / l2_q_s / 1e9 / peak, "traffic": None}},
    }
    # ---- codec variant (outside `value`): one bit with error feedback; the quantizer reads the gradient and
    # the residual and writes the residual back (12 + 1/8 + 8/B bytes per element); the server step is the
    # (min, max) variant's with one bit
    ef_res = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(W)]

    def ef_quantize():
        for w in range(W):
            check(lib.mqg_quantize_1bit_ef(grads[w].data_ptr(), ef_res[w].data_ptr(), n, B,
                                           codes[1][w].data_ptr(), mm_ranges[w].data_ptr(), 0, sptr))

    ef_quantize()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(mm_steps):
        ef_quantize()
    f1.record(stream)
    torch.cuda.synchronize()
    ef_s = f0.elapsed_time(f1) * 1e-3 / mm_steps
    ef_bytes = W * (12 * n + 4 * mqg.mqg_code_words(n, 1) + 8 * mqg.mqg_num_buckets(n, B))
    variant_1bit_ef = {
        "codec": "one bit per element with error feedback (mqg_quantize_1bit_ef; server step = the (min, max) "
                 "variant's with bits = 1); not part of `value`",
        "quantize": {"avg_launch_us": ef_s / W * 1e6, "launches_per_step": W,
                     "roofline": {"bound": "hbm", "achieved": ef_bytes / ef_s / 1e9, "peak": peak, "unit": "GB/s",
                                  "frac": ef_bytes / ef_s / 1e9 / peak, "traffic": None}},
    }
    del ef_res
    # put the codes back as the main codec writes them (the end-to-end leg re-quantizes anyway)
    for b in ALL_BITS:
        quantize_all(b, 0)
    torch.cuda.synchronize()

    # ---- end to end from pinned host buffers
    e2e_steps = max(1, min(args.steps, 3))
    e2e_step(0)
    barrier()
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record(stream)
    for i in range(e2e_steps):
        e2e_step(1 + i)
    b1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(b0.elapsed_time(b1)) / e2e_steps
    e2e = {"value": whole_job_gbs(world, grad_bytes_per_step, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": grad_bytes_per_step, "d2h_bytes_per_step": len(ALL_BITS) * 4 * n,
           "ms_per_step": e2e_ms, "steps": e2e_steps}

    # ---- the other workloads of the specification (single-GPU run only; outside `value`)
    other_configs = None
    if rank == 0 and world == 1 and not args.no_configs:
        import bench_configs
        torch.cuda.empty_cache()
        other_configs = bench_configs.run_all(torch, mqg, lib, check, peak)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu, _ = cpu_baseline(host_grads)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(), quantize_launch=args.quantize_launch),
            "clocks": clocks.summary(), "e2e": e2e,
            "gpu_launches": args.steps * len(ALL_BITS) * (q_launches + 1),
            "roofline": roofline, "roofline_server": roofline_server, "downlink": downlink_line,
            "variant_minmax": variant_minmax, "variant_l2": variant_l2,
            "variant_1bit_ef": variant_1bit_ef,
            "per_bits": per_bits,
            "per_bits_note": "`*_us`: groups of launches after 0.4 s of idle (SM clock at its maximum); "
                             "`*_us_sustained`: after 0.25 s of the same launch back to back, when the board's "
                             "power limit has lowered the SM clock (1650-1800 MHz seen)",
        }
        if other_configs is not None:
            line["configs"] = other_configs
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_single_kernel(args):
    """A few launches of one kernel on a small case (inputs still larger than L2), for profiler
    captures and quick timing: python bench.py --kernel quantize|quantize_workers|server|requantize|quantize_l2|onebit
    --bits B [--n N]."""
    import torch

    import paper_1804_08066_b200 as mqg
    from paper_1804_08066_b200 import workloads as wl

    torch.cuda.set_device(0)
    n, W, B, b = args.n, args.workers, args.bucket, args.bits
    rot = 3                                    # rotate buffer sets so launches never re-read L2
    stream = torch.cuda.current_stream()
    if args.kernel == "quantize" and args.dtype == "bf16":
        # the stress shape's input type: heavy-tailed bf16 values widened in the kernel
        grads = [torch.from_numpy(wl.student_t_bf16(n, config=5, worker=w).view(np.int16)).cuda().view(torch.bfloat16)
                 for w in range(rot)]
        codes = [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(rot)]
        scales = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize(grads[i % rot], n, b, B, PHILOX_SEED, codes[i % rot],
                                            scales[i % rot], worker=i % rot, step=i)
        nbytes = quantize_bytes(n, b, B) - 2 * n
    elif args.kernel == "quantize":
        grads = [torch.from_numpy(wl.laplace(n, LAPLACE_SCALE, config=2, worker=w)).cuda() for w in range(rot)]
        codes = [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(rot)]
        scales = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize(grads[i % rot], n, b, B, PHILOX_SEED, codes[i % rot],
                                            scales[i % rot], worker=i % rot, step=i)
        nbytes = quantize_bytes(n, b, B)
    elif args.kernel == "quantize_segments":
        # the layered AlexNet-shaped gradient (16 tensors, one scale per tensor): two passes over the gradient
        sizes = [int(np.prod(sh)) for sh in wl.ALEXNET_SHAPES]
        n = sum(sizes)
        seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
        coff = np.concatenate([[0], np.cumsum([mqg.mqg_code_words(sz, b) for sz in sizes])]).astype(np.uint64)
        grads = [torch.from_numpy(wl.layered(sizes, config=3, worker=w)).cuda() for w in range(rot)]
        codes = [torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda") for _ in range(rot)]
        scales = [torch.zeros(len(sizes), dtype=torch.float32, device="cuda") for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize_segments(grads[i % rot], seg, coff, b, PHILOX_SEED, codes[i % rot],
                                                     scales[i % rot], worker=i % rot, step=i)
        nbytes = 8 * n + 4 * int(coff[-1])
    elif args.kernel == "quantize_segments_workers":
        # the layered gradient of W workers in one call (three launches)
        sizes = [int(np.prod(sh)) for sh in wl.ALEXNET_SHAPES]
        n = sum(sizes)
        seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
        coff = np.concatenate([[0], np.cumsum([mqg.mqg_code_words(sz, b) for sz in sizes])]).astype(np.uint64)
        rot = 2
        grads = [torch.from_numpy(wl.layered(sizes, config=3, worker=w)).cuda() for w in range(W)]
        codes = [[torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda") for _ in range(W)] for _ in range(rot)]
        scales = [[torch.zeros(len(sizes), dtype=torch.float32, device="cuda") for _ in range(W)] for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize_segments_workers(grads, W, seg, coff, b, PHILOX_SEED, codes[i % rot],
                                                             scales[i % rot], first_worker=0, step=i)
        nbytes = W * (8 * n + 4 * int(coff[-1]))
    elif args.kernel == "server_segments":
        # fused server step on the layered gradient (per-layer scale), W workers
        sizes = [int(np.prod(sh)) for sh in wl.ALEXNET_SHAPES]
        n = sum(sizes)
        seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
        coff = np.concatenate([[0], np.cumsum([mqg.mqg_code_words(sz, b) for sz in sizes])]).astype(np.uint64)
        g = torch.from_numpy(wl.layered(sizes, config=3, worker=0)).cuda()
        codes = [[torch.zeros(int(coff[-1]), dtype=torch.int32, device="cuda") for _ in range(W)] for _ in range(rot)]
        scales = [[torch.zeros(len(sizes), dtype=torch.float32, device="cuda") for _ in range(W)] for _ in range(rot)]
        for r in range(rot):
            for w in range(W):
                mqg.mqg_quantize_segments(g, seg, coff, b, PHILOX_SEED, codes[r][w], scales[r][w], worker=w, step=r)
        params = [torch.from_numpy(wl.params(n, 0.05, config=3)).cuda() for _ in range(rot)]
        launch = lambda i: mqg.mqg_server_step_segments(codes[i % rot], scales[i % rot], W, b, seg, coff,
                                                        params[i % rot], LR)
        nbytes = 8 * n + W * 4 * int(coff[-1])
    elif args.kernel == "quantize_l2":
        grads = [torch.from_numpy(wl.laplace(n, LAPLACE_SCALE, config=2, worker=w)).cuda() for w in range(rot)]
        codes = [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(rot)]
        scales = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize_l2(grads[i % rot], n, b, B, PHILOX_SEED, codes[i % rot],
                                               scales[i % rot], worker=i % rot, step=i)
        nbytes = quantize_bytes(n, b, B)
    elif args.kernel == "onebit":
        b = 1
        grads = [torch.from_numpy(wl.laplace(n, LAPLACE_SCALE, config=2, worker=w)).cuda() for w in range(rot)]
        resid = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(rot)]
        codes = [torch.zeros(mqg.mqg_code_words(n, 1), dtype=torch.int32, device="cuda") for _ in range(rot)]
        ranges = [torch.zeros(2 * mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize_1bit_ef(grads[i % rot], resid[i % rot], n, B, codes[i % rot],
                                                    ranges[i % rot])
        nbytes = 12 * n + 4 * mqg.mqg_code_words(n, 1) + 8 * mqg.mqg_num_buckets(n, B)
    elif args.kernel == "quantize_workers":
        # W gradients of n elements per launch; two buffer sets, each far larger than L2
        rot = 2
        grads = [[torch.from_numpy(wl.laplace(n, LAPLACE_SCALE, config=2, worker=w + W * r)).cuda()
                  for w in range(W)] for r in range(rot)]
        codes = [[torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(W)]
                 for _ in range(rot)]
        scales = [[torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
                  for _ in range(rot)]
        launch = lambda i: mqg.mqg_quantize_workers(grads[i % rot], W, n, b, B, PHILOX_SEED, codes[i % rot],
                                                    scales[i % rot], first_worker=0, step=i)
        nbytes = W * quantize_bytes(n, b, B)
    else:
        if args.kernel == "requantize":
            rot = 6                                # 8 code buffers of n * bits / 8 bytes per set
        g = torch.from_numpy(wl.laplace(n, LAPLACE_SCALE, config=2, worker=0)).cuda()
        codes = [[torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(W)]
                 for _ in range(rot)]
        scales = [[torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(W)]
                  for _ in range(rot)]
        for r in range(rot):
            for w in range(W):
                mqg.mqg_quantize(g, n, b, B, PHILOX_SEED, codes[r][w], scales[r][w], worker=w, step=r)
        if args.kernel == "requantize":
            out_c = [torch.zeros(mqg.mqg_code_words(n, b), dtype=torch.int32, device="cuda") for _ in range(rot)]
            out_s = [torch.zeros(mqg.mqg_num_buckets(n, B), dtype=torch.float32, device="cuda") for _ in range(rot)]
            launch = lambda i: mqg.mqg_server_requantize(codes[i % rot], scales[i % rot], W, b, n, B, 1.0 / W,
                                                         PHILOX_SEED, out_c[i % rot], out_s[i % rot],
                                                         worker=W, step=i)
            nbytes = requantize_bytes(n, b, B, W)
        else:
            params = [torch.from_numpy(wl.params(n, 0.05, config=2)).cuda() for _ in range(rot)]
            launch = lambda i: mqg.mqg_server_step(codes[i % rot], scales[i % rot], W, b, n, B,
                                                   params[i % rot], LR)
            nbytes = server_bytes(n, b, B, W)
    torch.cuda.synchronize()
    # two warm-up launches, then all launches back to back between one pair of events
    for i in range(2):
        launch(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.launches):
        launch(2 + i)
    e1.record(stream)
    torch.cuda.synchronize()
    avg = e0.elapsed_time(e1) * 1e-3 / args.launches
    peak, kind = measured_hbm_peak()
    line = {"kernel": args.kernel, "bits": b, "n": n, "workers": W, "bucket": B,
            "launches": args.launches, "avg_us": avg * 1e6, "algorithmic_bytes": nbytes,
            "avg_gbs": nbytes / avg / 1e9, "frac_of_%s_peak" % kind: nbytes / avg / 1e9 / peak}
    if args.clock_trace > 0:
        line["clock_trace"] = clock_trace(torch, stream, launch, avg, args.clock_trace)
    print(json.dumps(line))
    return 0


def clock_trace(torch, stream, launch, est_s, seconds):
    """The same launch back to back for `seconds` after one second of idle, an event every few launches and
    the SM clock, the board power and the throttle reasons read through NVML every 5 ms: shows the time per
    launch following the clock down once the board's power limit acts.  Returns rows of 25 ms."""
    import pynvml
    pynvml.nvmlInit()
    h = pynvml.nvmlDeviceGetHandleByIndex(torch.cuda.current_device())
    samples, stop = [], threading.Event()

    def sample():
        while not stop.is_set():
            samples.append((time.perf_counter(), pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM),
                            pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0,
                            int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))))
            stop.wait(0.005)

    torch.cuda.synchronize()
    time.sleep(1.0)
    per_mark = max(1, int(0.005 / est_s))          # an event about every 5 ms of launches
    marks = max(2, int(seconds / (per_mark * est_s)))
    th = threading.Thread(target=sample, daemon=True)
    th.start()
    t0 = time.perf_counter()
    events = [torch.cuda.Event(enable_timing=True)]
    events[0].record(stream)
    i = 0
    for _ in range(marks):
        for _ in range(per_mark):
            launch(i)
            i += 1
        events.append(torch.cuda.Event(enable_timing=True))
        events[-1].record(stream)
    torch.cuda.synchronize()
    stop.set()
    th.join()
    at = [events[0].elapsed_time(e) for e in events]               # ms since the first launch
    rows, width = [], 25.0
    for lo in np.arange(0.0, at[-1], width):
        seg = [(at[j + 1] - at[j]) / per_mark for j in range(marks) if lo <= at[j] < lo + width]
        smp = [x for x in samples if lo <= (x[0] - t0) * 1e3 < lo + width]
        if seg:
            rows.append({"ms": [float(lo), float(lo + width)], "us_per_launch": float(np.median(seg)) * 1e3,
                         "sm_mhz": sorted({x[1] for x in smp}), "power_w_max": max([x[2] for x in smp], default=None),
                         "reasons": sorted({hex(x[3]) for x in smp})})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the other workloads of the specification (`configs` in the JSON line)")
    ap.add_argument("--quantize-launch", choices=["batched", "per-worker"], default="batched",
                    help="the step's quantize phase: one mqg_quantize_workers launch per bit width for all "
                         "workers' gradients, or one mqg_quantize launch per worker")
    ap.add_argument("--kernel", choices=["quantize", "quantize_workers", "server", "requantize", "quantize_l2", "onebit",
                             "quantize_segments", "quantize_segments_workers", "server_segments"],
                    default=None,
                    help="run a few launches of one kernel on a small case instead of the benchmark")
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--dtype", choices=["f32", "bf16"], default="f32", help="gradient type of --kernel quantize")
    ap.add_argument("--n", type=int, default=1 << 25)
    ap.add_argument("--workers", type=int, default=N_WORKERS)
    ap.add_argument("--bucket", type=int, default=BUCKET)
    ap.add_argument("--launches", type=int, default=6)
    ap.add_argument("--clock-trace", type=float, default=0.0, metavar="SECONDS",
                    help="with --kernel: then run the launch back to back for SECONDS and report time per launch, "
                         "SM clock and board power in rows of 25 ms")
    args = ap.parse_args()
    if args.kernel is not None:
        return run_single_kernel(args)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
