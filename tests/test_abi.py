"""The C-ABI library: it loads, exports every symbol the header declares, and rejects bad
arguments on the host before anything is launched (no GPU needed: validation comes first)."""
import ctypes
import os
import re

import pytest

from paper_2510_26771_b200 import build as stamp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def st():
    stamp_build.build()
    from paper_2510_26771_b200 import binding
    binding.lib()
    return binding


def test_header_symbols_are_exported(st):
    header = open(os.path.join(ROOT, "include", "stamp.h")).read()
    declared = set(re.findall(r"^\s*(?:int|const char\*)\s+(stamp_\w+)\s*\(", header, flags=re.M))
    assert declared, "no declarations found"
    assert declared == set(st.EXPORTS)
    lib = st.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(st):
    assert st.status_string(0) == "ok"
    assert "wait" in st.status_string(5)
    assert st.status_string(99) == "unknown status"


def test_config_struct_matches_header(st):
    assert ctypes.sizeof(st.StampConfig) == 48      # twelve int32 fields
    header = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "stamp.h")).read()
    body = header[header.index("typedef struct {"):header.index("} stamp_config;")]
    names = re.findall(r"int32_t\s+(\w+);", body)
    assert names == [n for n, _ in st.StampConfig._fields_]


def test_host_side_validation(st):
    lib = st.lib()
    c = st.make_config(st.T_HAAR, 0, 0, 64)
    out = ctypes.c_size_t(0)
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 2048, 4096, 11008, ctypes.byref(out)) == 0
    assert out.value > 2048 * 4096
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 2048, 4096, 11008, None) == 1          # null out
    assert lib.stamp_workspace_bytes(None, 1, 2048, 4096, 11008, ctypes.byref(out)) == 1         # null cfg
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 0, 2048, 4096, 11008, ctypes.byref(out)) == 1
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 2048, 4000, 11008, ctypes.byref(out)) == 2   # K % 128
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 2000, 4096, 11008, ctypes.byref(out)) == 2   # L not 2^j
    assert lib.stamp_workspace_bytes(ctypes.byref(c), 1, 2048, 4096, 11004, ctypes.byref(out)) == 2   # N % 8
    bad = st.make_config(st.T_HAAR, 256, 9, 16)                                                   # levels > log2(block)
    assert lib.stamp_workspace_bytes(ctypes.byref(bad), 1, 2048, 4096, 1024, ctypes.byref(out)) == 2
    bad = st.make_config(st.T_HAAR, 0, 0, 4096)                                                   # k_hi > block
    assert lib.stamp_workspace_bytes(ctypes.byref(bad), 1, 2048, 4096, 1024, ctypes.byref(out)) == 1
    bad = st.make_config(st.T_HAAR, 0, 0, 64, bits_lo=3)
    assert lib.stamp_workspace_bytes(ctypes.byref(bad), 1, 2048, 4096, 1024, ctypes.byref(out)) == 2
    bad = st.make_config(7)
    assert lib.stamp_workspace_bytes(ctypes.byref(bad), 1, 2048, 4096, 1024, ctypes.byref(out)) == 1
    # entry points: null tensors and a missing / short workspace are refused before any launch
    null = ctypes.c_void_p(0)
    assert lib.stamp_quantize(ctypes.byref(c), null, 1, 1, 2048, 4096, null, null, null, null, ctypes.c_size_t(0),
                              null) == 1
    fake = ctypes.c_void_p(4096)  # never dereferenced: the workspace check fails first
    assert lib.stamp_quantize(ctypes.byref(c), fake, 1, 1, 2048, 4096, fake, fake, fake, null, ctypes.c_size_t(0),
                              null) == 3
    assert lib.stamp_quantize(ctypes.byref(c), fake, 1, 1, 2048, 4096, fake, fake, fake, fake, ctypes.c_size_t(16),
                              null) == 3
    assert lib.stamp_linear_fused(ctypes.byref(c), fake, 5, fake, 0, fake, null, 1, 2048, 4096, 1024, fake, 0, fake,
                                  ctypes.c_size_t(1 << 40), null) == 1                          # bad dtype
    assert lib.stamp_last_device_status(null, None) == 1
