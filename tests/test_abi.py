"""The C ABI on a machine without a GPU: the library loads and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "odb.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(odb_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported_and_bound():
    import __graft_entry__ as g
    g.build()
    from paper_2511_21759_b200 import binding as B
    lib = B.lib()
    names = _declared()
    assert "odb_refresh_prefill" in names and "odb_block_decode_step" in names and "odb_unmask_accept" in names
    for n in names:
        assert hasattr(lib, n), n
        assert n in B.SIGNATURES, f"{n} declared in odb.h but not bound"
    assert sorted(B.SIGNATURES) == names


def test_pure_host_calls_work_without_gpu():
    from paper_2511_21759_b200 import binding as B
    lib = B.lib()
    assert lib.odb_status_string(0) == b"ok" and lib.odb_status_string(B.ODB_ERR_TIMEOUT) == b"device-side wait timed out"
    cfg = B.odb_config(32, 4096, 32, 128, 12288, 126464, 126336, 126081, 500000.0, 1e-5, 1, 768, 32, 4, 1)
    kv = lib.odb_kv_bytes(ctypes.byref(cfg))
    assert kv == 32 * 2 * 768 * 4096 * 2                              # 0.5 MiB per token
    assert lib.odb_workspace_bytes(ctypes.byref(cfg)) > 0
    # weights once + K/V once: 14.995 GB + 16 KiB per key and layer
    b = lib.odb_step_algorithmic_bytes(ctypes.byref(cfg), 736)
    weights = 32 * 218103808 * 2 + 126464 * 4096 * 2
    assert b == weights + 32 * 736 * 16384
    bad = B.odb_config(32, 4096, 32, 96, 12288, 126464, 126336, 126081, 500000.0, 1e-5, 1, 768, 32, 4, 1)
    assert lib.odb_kv_bytes(ctypes.byref(bad)) == 0                   # head_dim 96 unsupported
    out = ctypes.c_void_p()
    assert lib.odb_model_create(ctypes.byref(bad), None, ctypes.byref(out)) == B.ODB_ERR_SHAPE
    assert lib.odb_model_create(ctypes.byref(cfg), None, ctypes.byref(out)) == B.ODB_ERR_ARG


def test_struct_layouts_match_header():
    from paper_2511_21759_b200 import binding as B
    assert ctypes.sizeof(B.odb_config) == 17 * 4
    assert ctypes.sizeof(B.odb_decode_params) == 9 * 4
    assert ctypes.sizeof(B.odb_result) == (3 + 5 + 3 + 128) * 4
    assert ctypes.sizeof(B.odb_weights) == 9 * ctypes.sizeof(ctypes.c_void_p)
