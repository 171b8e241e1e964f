"""The whole MQGrad loop on one GPU with simulated workers (Algorithm 1 end to end):

    python -m paper_1804_08066_b200.train_loop [--iters 60] [--workers 4] [--selector window|sarsa]

A small CNN (3x3 convolutions 3-32-64-128, two fully connected layers) is trained on synthetic
32x32x3 images (ten fixed Gaussian class means plus unit noise), batch 128 per worker.  Every
iteration each worker's flat gradient goes through mqg_quantize, the server pass
mqg_server_step updates the shared flat parameter vector, and the host selector picks the next
bit width from the losses.  The model and its autograd belong to this harness; the library is
only the codec.  Prints one JSON line with the share of iteration time spent inside libmqgrad
(the paper's Table 3 reports 4.1-13.3 % for quantize + de-quantize + MDP on its CPU clusters).
"""
from __future__ import annotations

import argparse
import json
import time

import torch
import torch.nn as nn
import torch.nn.functional as F

import paper_1804_08066_b200 as mqg
from paper_1804_08066_b200.selector import SarsaBitSelector, WindowQSelector

BUCKET = 2048
# Table 3 of the paper: smallest and largest share of training time (%) spent in quantize +
# de-quantize + MDP over its two CPU clusters and five methods; quoted as context in the report.
PAPER_TABLE_3_RANGE_PERCENT = (4.11, 13.3)


class SmallCnn(nn.Module):
    def __init__(self):
        super().__init__()
        self.c1 = nn.Conv2d(3, 32, 3, padding=1)
        self.c2 = nn.Conv2d(32, 64, 3, padding=1)
        self.c3 = nn.Conv2d(64, 128, 3, padding=1)
        self.f1 = nn.Linear(128 * 4 * 4, 256)
        self.f2 = nn.Linear(256, 10)

    def forward(self, x):
        x = F.max_pool2d(F.relu(self.c1(x)), 2)
        x = F.max_pool2d(F.relu(self.c2(x)), 2)
        x = F.max_pool2d(F.relu(self.c3(x)), 2)
        return self.f2(F.relu(self.f1(x.flatten(1))))


def flatten_parameters(model):
    """Re-seat every parameter as a view into one flat fp32 vector (the shared parameters w)."""
    n = sum(p.numel() for p in model.parameters())
    flat = torch.zeros(n, dtype=torch.float32, device="cuda")
    off = 0
    for p in model.parameters():
        flat[off:off + p.numel()].copy_(p.data.reshape(-1))
        p.data = flat[off:off + p.numel()].view_as(p.data)
        off += p.numel()
    return flat


def run(iters=60, workers=4, batch=128, lr=0.05, selector="window", seed=0):
    torch.manual_seed(seed)
    model = SmallCnn().cuda()
    flat = flatten_parameters(model)
    n = flat.numel()
    gen = torch.Generator(device="cuda").manual_seed(seed + 1)
    means = torch.randn(10, 3, 32, 32, generator=gen, device="cuda")
    sel = WindowQSelector(seed=seed) if selector == "window" else SarsaBitSelector(seed=seed)
    codes = [torch.zeros(mqg.mqg_code_words(n, 8), dtype=torch.int32, device="cuda") for _ in range(workers)]
    scales = [torch.zeros(mqg.mqg_num_buckets(n, BUCKET), dtype=torch.float32, device="cuda") for _ in range(workers)]
    bits, lib_ms, total_ms, wire = (1 if selector == "window" else 2), 0.0, 0.0, 0
    losses, chosen = [], []
    last_ms = 1.0
    for m in range(iters):
        t0 = time.perf_counter()
        torch.cuda.synchronize()
        grads, loss_sum = [], 0.0
        for w in range(workers):
            y = torch.randint(0, 10, (batch,), generator=gen, device="cuda")
            x = means[y] + torch.randn(batch, 3, 32, 32, generator=gen, device="cuda")
            model.zero_grad(set_to_none=True)
            loss = F.cross_entropy(model(x), y)
            loss.backward()
            grads.append(torch.cat([p.grad.reshape(-1) for p in model.parameters()]))
            loss_sum += float(loss.detach())
        loss_m = loss_sum / workers
        bits = sel.step(m, loss_m, last_ms)                       # server MDP: loss in, width out
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for w in range(workers):
            mqg.mqg_quantize(grads[w], n, bits, BUCKET, seed, codes[w], scales[w], worker=w, step=m)
        mqg.mqg_server_step(codes, scales, workers, bits, n, BUCKET, flat, lr / workers)
        e1.record()
        torch.cuda.synchronize()
        lib_ms += e0.elapsed_time(e1)
        last_ms = (time.perf_counter() - t0) * 1e3
        total_ms += last_ms
        wire += workers * mqg.mqg_wire_bytes(n, bits, BUCKET)
        losses.append(loss_m), chosen.append(bits)
    assert mqg.mqg_device_timeouts() == 0
    return {"iters": iters, "workers": workers, "parameters": n, "selector": selector,
            "first_loss": losses[0], "last_loss": losses[-1], "bits_chosen": chosen,
            "libmqgrad_ms_per_iter": lib_ms / iters, "iteration_ms": total_ms / iters,
            "libmqgrad_share_pct": 100.0 * lib_ms / total_ms,
            "uplink_bytes_per_iter": wire / iters, "uplink_bytes_fp32": 4 * n * workers,
            "paper_table3_share_pct": "%g-%g (CPU clusters, quantize + de-quantize + MDP)"
                                      % PAPER_TABLE_3_RANGE_PERCENT}


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=60)
    ap.add_argument("--workers", type=int, default=4)
    ap.add_argument("--selector", default="window", choices=["window", "sarsa"])
    a = ap.parse_args()
    print(json.dumps(run(a.iters, a.workers, selector=a.selector)))
