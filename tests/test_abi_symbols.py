"""The C-ABI library loads and exports every symbol the header declares (no GPU work)."""

import ctypes
import os
import re

import pytest

from paper_2504_08838_b200 import binding as sd2

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(sd2_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported():
    L = sd2.lib()
    decl = declared_symbols()
    assert decl, "no declarations found"
    assert decl == set(sd2.EXPORTS), decl ^ set(sd2.EXPORTS)
    for name in decl:
        assert getattr(L, name) is not None


def test_status_strings():
    assert sd2.status_string(0) == "ok"
    seen = {sd2.status_string(s) for s in range(-7, 1)}
    assert len(seen) == 8
    assert sd2.status_string(-99) == "unknown status"


def test_null_and_dead_handles_are_refused_without_a_gpu():
    L = sd2.lib()
    assert L.sd2_free(None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_free(ctypes.c_void_p(0x1234)) == sd2.SD2_ERR_INVALID_ARG      # never a live handle
    assert L.sd2_info(ctypes.c_void_p(0x1234), None, None, None, None, None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_spmm(None, None, None, 1, None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_blob_free(None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_block_step(None, None, None, 1, None, None) == sd2.SD2_ERR_INVALID_ARG


def test_device_entry_points_fail_loudly_without_a_device():
    import numpy as np
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    W = np.zeros((4, 8), np.uint16)
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_compress(W, None)
    assert e.value.status in (sd2.SD2_ERR_CUDA, sd2.SD2_ERR_ALLOC)
