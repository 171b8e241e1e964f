"""The values the paper itself prints (tests/golden/, each file cites its passage) against the host
components that are supposed to carry them: the selector's defaults, the synthetic stand-in for the
paper's network, and the context numbers of the end-to-end loop."""
import inspect
import os

import numpy as np

from paper_1804_08066_b200 import selector, workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _pairs(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_selector_defaults_are_the_papers_settings():
    g = _pairs("section_4_1_settings.txt")
    d = {k: v.default for k, v in inspect.signature(selector.SarsaBitSelector.__init__).parameters.items()
         if v.default is not inspect.Parameter.empty}
    assert d["bits_min"] == g["bits_min"] and d["bits_max"] == g["bits_max"]
    assert d["bits_max"] - d["bits_min"] + 1 == g["bit_levels"] == g["q_outputs"]
    assert d["period"] == g["period_T"] == g["q_inputs"]
    assert d["hidden"] == g["q_hidden"]
    assert d["epsilon"] == g["epsilon"] and d["lr"] == g["eta"] and d["alpha"] == g["alpha"]
    assert d["reward_scale"] == g["gamma_reward_scale"]
    sel = selector.SarsaBitSelector()
    assert sel.net.num_parameters() == int(g["q_inputs"] * g["q_hidden"] + g["q_hidden"]
                                           + g["q_hidden"] * g["q_outputs"] + g["q_outputs"])


def test_paper_network_shapes_and_quantized_share():
    quantized, uncompressed, share = [], [], None
    for line in open(os.path.join(GOLDEN, "section_4_1_model_shapes.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "quantized_share_percent":
            share = float(f[1])
            continue
        (quantized if f[1] == "q" else uncompressed).append(tuple(int(v) for v in f[2:]))
    assert quantized == list(wl.PAPER_CNN_QUANTIZED)
    weights_only = [s for s in wl.PAPER_CNN_UNCOMPRESSED if len(s) > 1]
    assert uncompressed == weights_only                       # the stand-in adds only the bias vectors
    nq = sum(int(np.prod(s)) for s in quantized)
    total = nq + sum(int(np.prod(s)) for s in wl.PAPER_CNN_UNCOMPRESSED)
    assert nq == 16_072_704
    assert abs(100.0 * nq / total - share) < 0.15             # "about 99.2%"


def test_table_3_is_what_the_loop_quotes_as_context():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table_3_time_share.txt")) if l[0] != "#"]
    values = [float(v) for r in rows for v in r[1:]]
    assert len(rows) == 2 and len(values) == 10
    assert min(values) == 4.11 and max(values) == 13.3        # the range the loop's report cites
    from paper_1804_08066_b200 import train_loop
    lo, hi = train_loop.PAPER_TABLE_3_RANGE_PERCENT
    assert (lo, hi) == (min(values), max(values))
