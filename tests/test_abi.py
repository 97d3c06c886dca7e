"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU work)."""
import ctypes
import os
import re

import paper_2012_09849_b200 as hts
from paper_2012_09849_b200 import build as hb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "hts.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hts_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = hb.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    names = _declared()
    assert "hts_policy_step" in names and "hts_gae" in names and len(names) >= 12
    for n in names:
        assert hasattr(L, n), f"{n} is declared in hts.h but not exported"
    assert sorted(hts.EXPORTS) == names, "python binding and header disagree"
    for n in names:
        assert callable(getattr(hts, n)), f"binding lacks {n}"


def test_status_strings_and_launch_counter_without_gpu():
    assert hts.hts_status_string(0) == "HTS_OK"
    assert hts.hts_status_string(1) == "HTS_ERR_INVALID_ARG"
    assert hts.hts_status_string(6) == "HTS_ERR_UNSUPPORTED"
    assert hts.hts_launch_count() >= 0
    assert hts.hts_last_cuda_error() == "" or isinstance(hts.hts_last_cuda_error(), str)


def test_host_side_validation_needs_no_device():
    L = hts.lib()
    # NULL pointers and bad hyper-parameters are refused before any CUDA call
    assert L.hts_gae(None, None, None, None, 0.99, 0.95, 4, 4, None, None, None) == 1
    assert L.hts_gae(8, 16, 24, 32, float("nan"), 0.95, 4, 4, 40, 48, None) == 1
    assert L.hts_gae(8, 16, 24, 32, 0.99, 1.5, 4, 4, 40, 48, None) == 1
    assert L.hts_gae(8, 16, 24, 32, 0.99, 0.95, 0, 4, 40, 48, None) == 1
    assert L.hts_policy_create(None, None) == 1
    d = hts.hts_net_desc(4, 84, 84, 0, 1, 16)
    out = ctypes.c_void_p()
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 1       # zero actions
    d = hts.hts_net_desc(4, 83, 84, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2       # H not a multiple of 4
    d = hts.hts_net_desc(4, 12, 12, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2       # too small for the conv stack
    # shape limits of the tensor-core (bf16) kernels are checked at create time, before any device call
    d = hts.hts_net_desc(4, 84, 256, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2       # wider than the resident conv2 tile allows
    d = hts.hts_net_desc(4, 536, 252, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2       # first hidden grid over 2048 positions
    d = hts.hts_net_desc(3, 84, 84, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2       # bf16 contexts take 4, 8 or 16 channels
    d = hts.hts_net_desc(12, 84, 84, 6, 1, 16)
    assert L.hts_policy_create(ctypes.byref(d), ctypes.byref(out)) == 2
