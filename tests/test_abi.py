"""Host-side checks of the C ABI: the library loads, exports everything the header
declares, and validates arguments before touching a device (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(bitnet_a48_\w+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(a48):
    lib = a48.lib()
    declared = _declared()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared == set(a48.EXPORTS), "binding's export list and the header disagree"


def test_status_strings(a48):
    assert a48.status_string(0) == "ok"
    assert "aligned" in a48.status_string(3)
    assert a48.status_string(1234) == "unknown status"


def test_argument_validation_needs_no_device(a48):
    lib = a48.lib()
    null, p = ctypes.c_void_p(0), ctypes.c_void_p(4096)
    odd = ctypes.c_void_p(4100)
    st = null
    assert lib.bitnet_a48_quant_int4(null, 4, 64, 1e-5, p, p, st) == 1
    assert lib.bitnet_a48_quant_int4(p, 0, 64, 1e-5, p, p, st) == 2
    assert lib.bitnet_a48_quant_int4(p, 4, 1 << 21, 1e-5, p, p, st) == 2
    assert lib.bitnet_a48_quant_int4(odd, 4, 64, 1e-5, p, p, st) == 3
    assert lib.bitnet_a48_topk_quant_int8(p, 4, 64, 0, 1e-5, p, p, null, st) == 1
    assert lib.bitnet_a48_topk_quant_int8(p, 4, 64, 65, 1e-5, p, p, null, st) == 1
    assert lib.bitnet_a48_topk_quant_int8(p, 4, 64, 8, 1e-5, p, p, odd, st) == 3
    out = ctypes.c_void_p(0)
    assert lib.bitnet_a48_pack_ternary(null, 8, 8, 1e-5, 0, ctypes.byref(out), st) == 1
    assert lib.bitnet_a48_pack_ternary(p, 8, 8, 1e-5, 64, ctypes.byref(out), st) == 1
    assert lib.bitnet_a48_pack_ternary(p, -1, 8, 1e-5, 0, ctypes.byref(out), st) == 2
    assert lib.bitnet_a48_linear(null, p, p, 1, 0, p, null, null, 0, st) == 1
    assert lib.bitnet_a48_block_forward(null, p, 1, 1, 0, null, null, p, p, 0, st) == 1
    assert lib.bitnet_a48_weight_free(null) is None  # freeing NULL is a no-op


def test_no_cpu_fallback(a48):
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for machines without a GPU")
    lib = a48.lib()
    p = ctypes.c_void_p(4096)
    assert lib.bitnet_a48_quant_int4(p, 4, 64, 1e-5, p, p, ctypes.c_void_p(0)) == 5  # BITNET_A48_ERR_CUDA
