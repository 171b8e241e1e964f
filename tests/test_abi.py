"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, sizes helpers are right, and argument validation rejects
bad calls before anything is launched."""
import ctypes as C
import os
import re

import pytest

import paper_1804_08066_b200 as mqg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "mqgrad.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mqg_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "mqg_quantize" in names and "mqg_server_step" in names and len(names) >= 11
    lib = C.CDLL(mqg.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name
        assert hasattr(mqg, name), "binding lacks " + name


def test_size_helpers():
    assert mqg.mqg_code_words(0, 5) == 0
    assert mqg.mqg_code_words(1, 1) == 1
    assert mqg.mqg_code_words(32, 3) == 3
    assert mqg.mqg_code_words(33, 3) == 4
    assert mqg.mqg_code_words(25_000_000, 3) == 2_343_750
    assert mqg.mqg_code_words(1_000_000_000, 8) == 250_000_000
    assert mqg.mqg_num_buckets(25_000_000, 2048) == 12_208
    assert mqg.mqg_num_buckets(1_000_000_000, 4096) == 244_141
    assert mqg.mqg_wire_bytes(1_048_576, 4, 512) == 4 * 131_072 + 4 * 2048
    assert mqg.mqg_version() >= 100


def test_validation_rejects_bad_arguments_without_launching():
    lib = mqg.raw_library()
    fake = C.c_void_p(0x10000)            # aligned, never dereferenced: validation fails first
    odd = C.c_void_p(0x10004)
    # bits
    for bits in (0, 9, -1):
        assert lib.mqg_quantize(fake, 64, bits, 32, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_BITS
        assert "bits" in mqg.mqg_last_error()
    # bucket
    assert lib.mqg_quantize(fake, 64, 4, 0, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    assert lib.mqg_quantize(fake, 64, 4, 48, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    # null and misaligned buffers
    assert lib.mqg_quantize(None, 64, 4, 32, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    assert lib.mqg_quantize(odd, 64, 4, 32, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_ALIGN
    assert lib.mqg_quantize(fake, 64, 4, 32, 0, odd, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_ALIGN
    assert lib.mqg_quantize(fake, 64, 4, 32, 0, fake, fake, 7, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    # n == 0 is a no-op, even with null buffers
    assert lib.mqg_quantize(None, 0, 4, 32, 0, None, None, 0, 0, 0, 0, None) == mqg.MQG_OK
    assert lib.mqg_apply(None, None, 0.1, 0, None) == mqg.MQG_OK
    # workers
    tab = (C.c_void_p * 2)(0x10000, 0x20000)
    assert lib.mqg_server_step(tab, tab, 0, 4, 64, 32, fake, 0.1, None, None) == mqg.MQG_ERR_TOO_MANY_WORKERS
    assert lib.mqg_server_step(tab, tab, 33, 4, 64, 32, fake, 0.1, None, None) == mqg.MQG_ERR_TOO_MANY_WORKERS
    missing = (C.c_void_p * 2)(0x10000, None)        # a worker's buffer never arrived
    assert lib.mqg_server_step(missing, tab, 2, 4, 64, 32, fake, 0.1, None, None) == mqg.MQG_ERR_INVALID
    assert "worker 1" in mqg.mqg_last_error()
    assert lib.mqg_server_step(tab, tab, 2, 4, 64, 32, None, 0.1, None, None) == mqg.MQG_ERR_INVALID
    assert lib.mqg_server_step(tab, tab, 2, 4, 64, 32, odd, 0.1, None, None) == mqg.MQG_ERR_ALIGN
    assert lib.mqg_dequant_accumulate(tab, tab, 2, 4, 64, None, 32, 0, None) == mqg.MQG_ERR_INVALID
    assert lib.mqg_apply(fake, odd, 0.1, 8, None) == mqg.MQG_ERR_ALIGN
    # segment tables
    seg = (C.c_uint64 * 3)(0, 100, 50)
    cof = (C.c_uint64 * 3)(0, 13, 26)
    assert lib.mqg_quantize_segments(fake, 2, seg, cof, 4, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    seg = (C.c_uint64 * 3)(0, 100, 200)
    cof = (C.c_uint64 * 3)(0, 12, 25)                # 100 * 4 bits need 13 words
    assert lib.mqg_quantize_segments(fake, 2, seg, cof, 4, 0, fake, fake, 0, 0, 0, 0, None) == mqg.MQG_ERR_INVALID
    assert "segment 0" in mqg.mqg_last_error()


def test_binding_refuses_cpu_tensors():
    import torch
    g = torch.zeros(64)
    with pytest.raises(TypeError):
        mqg.mqg_quantize(g, 64, 4, 32, 0, torch.zeros(8, dtype=torch.int32), torch.zeros(2))
