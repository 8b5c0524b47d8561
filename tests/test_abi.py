"""CPU-side checks of the C-ABI boundary: the library builds for sm_100a, loads,
exports every function the header declares, and its host-only helpers agree
with the oracle.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2604_08971_b200 as sentry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sentry.build()
    return sentry.load_library()


def _declared_functions():
    names = []
    for fname in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", fname)).read()
        names += re.findall(r"SENTRY_API\s+[\w\s\*]+?\b(sentry_\w+)\s*\(", text)
    return names


def test_header_functions_are_exported(lib):
    names = _declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), "libsentry.so does not export %s" % n
    assert set(sentry.EXPORTS) <= set(names)


def test_num_active_queries_agrees_with_oracle(lib):
    for c in (1, 3, 5, 8):
        for T in list(range(0, 3000)) + [4095, 4096, 8103, 8104, 22026, 22027, 32768, 65535]:
            assert sentry.num_active_queries(T, c) == oracle.num_active(T, c), (T, c)
    assert sentry.num_active_queries(128, 5) == 25  # the paper's worked example (Section 4.4)


def test_status_strings(lib):
    assert sentry.status_string(0) == "ok"
    assert "workspace" in sentry.status_string(-4)
    assert sentry.status_string(-99) == "unknown status"


def test_host_side_argument_checks_need_no_gpu(lib):
    # null context / descriptors are rejected before any CUDA call
    assert lib.sentry_gate_select(None, None, 1, 1, None, 0, 1, None, None, 0, None) == -1
    assert lib.sentry_attend_fwd(None, None, *([None] * 8), 0, None, None, None, None) == -1
    assert lib.sentry_ffn_fwd(None, None, *([None] * 9)) == -1
    assert lib.sentry_set_workspace(None, None, 0) == -1
    assert lib.sentry_destroy(None) == -1
    # workspace bound is defined for valid descriptors and has a floor
    a = sentry.AttendDesc(64, 1024, 8, 2, 32, 4, sentry.SENTRY_BF16, 5, 0)
    f = sentry.FfnDesc(64, 1024, 256, 1024, 512, 1, sentry.SENTRY_BF16)
    floor = lib.sentry_workspace_bytes(None, None)
    assert floor >= 1 << 20
    wa = lib.sentry_workspace_bytes(ctypes.byref(a), None)
    wf = lib.sentry_workspace_bytes(None, ctypes.byref(f))
    assert wa >= 64 * 4 * 1024 * 4 and wf >= 2 * 512 * 256 * 2
    assert lib.sentry_workspace_bytes(ctypes.byref(a), ctypes.byref(f)) == max(wa, wf)


def test_create_without_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    h = ctypes.c_void_p()
    assert lib.sentry_create(ctypes.byref(h), 0) == -5 and not h.value
    with pytest.raises(RuntimeError):
        sentry.Sentry(0)
