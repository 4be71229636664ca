"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

from paper_2603_14303_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "semanticache.h")).read()
    return re.findall(r"SC_API\s+[\w\s\*]+?\b(sc_\w+)\s*\(", text)


def test_header_symbols_are_exported(lib):
    names = _declared()
    assert len(names) >= 8 and {"sc_chunk", "sc_compress", "sc_decode_attn"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(binding.EXPORTS)
    assert b"sm_100a" in lib.sc_version()


def test_host_side_validation_needs_no_gpu(lib):
    a, b = ctypes.c_int32(), ctypes.c_int32()
    assert lib.sc_chunk_bounds(2, 1000, ctypes.byref(a), ctypes.byref(b)) == binding.SC_OK
    assert a.value == 2000 and b.value == 2 * 8 + 1
    assert lib.sc_chunk_bounds(-1, 5, None, None) == binding.SC_ERR_INVALID_ARG
    assert lib.sc_chunk_workspace_bytes(1, 2048) >= 12
    assert lib.sc_compress_workspace_bytes(1, 8, 2048) >= 3 * 4 * 8 * 2048
    assert lib.sc_decode_workspace_bytes(1, 32, 8, 128, 2048) > 0
    # null output pointers / bad sizes are rejected before any CUDA call
    assert lib.sc_chunk(None, 1, 8, None, 0, 256, None, 8, None, None, None, 3, None, None, 0, None, None) \
        == binding.SC_ERR_INVALID_ARG
    prm = binding._GscParams(0.7, 256, 0)
    st = binding._Strides(0, 0, 128)
    assert lib.sc_compress(None, None, st, 7, 1, 8, 16, 128, None, None, None, None, None, 3, ctypes.byref(prm),
                           None, None, None, 16, 1, None, None, 0, None, None) == binding.SC_ERR_UNSUPPORTED
    assert lib.sc_decode_attn(None, 0, 1, 30, 8, 128, None, None, None, 0, None, 0.0, 0, None, None, 0, None,
                              None) == binding.SC_ERR_INVALID_ARG  # Hq % Hkv != 0
    ap = lambda dt, B, max_len, k: lib.sc_append(k, k, dt, B, 8, 128, None, None, 0, max_len, 0.7, None, None, None, 64,
                                                 None, None, None, None, None)
    assert ap(0, 1, 300, None) == binding.SC_ERR_INVALID_ARG       # max_chunk_len beyond SC_MAX_CHUNK_LEN
    assert ap(5, 1, 256, None) == binding.SC_ERR_UNSUPPORTED      # unknown dtype
    assert ap(0, 1, 256, None) == binding.SC_ERR_INVALID_ARG       # null tensors
    assert ap(0, 0, 256, None) == binding.SC_OK                    # nothing to do


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libsemanticache.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
