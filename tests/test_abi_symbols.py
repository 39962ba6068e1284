"""CPU-only checks of the boundary: the library builds for sm_100a, loads, and exports every
symbol the header declares (no compute call is made without a GPU)."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_loads_and_exports_all_declared_symbols():
    from paper_2308_04623_b200 import build
    build.build()
    import paper_2308_04623_b200 as ssd
    lib = ssd.lib()
    header = open(os.path.join(ROOT, "include", "ssd.h")).read()
    declared = set(re.findall(r"\b(ssd_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(ssd.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings_and_null_arguments():
    import ctypes as C
    import paper_2308_04623_b200 as ssd
    lib = ssd.lib()
    assert lib.ssd_strerror(0) == b"ok"
    for code in range(-9, 0):
        assert lib.ssd_strerror(code) not in (b"ok", b"unknown status")
    assert lib.ssd_strerror(-100) == b"unknown status"
    out = C.c_void_p()
    assert lib.ssd_create(None, 0, None, C.byref(out)) == ssd.SSD_ERR_BAD_ARG
    assert lib.ssd_kv_reset(None) == ssd.SSD_ERR_BAD_ARG
    assert lib.ssd_verify_tree(None, None, None, 1, None, None) == ssd.SSD_ERR_BAD_ARG
    assert lib.ssd_kv_commit(None, None, None, 1) == ssd.SSD_ERR_BAD_ARG
    lib.ssd_destroy(None)
    lib.ssd_kv_destroy(None)


def test_unsupported_shapes_are_refused_before_touching_a_device():
    import ctypes as C
    import paper_2308_04623_b200 as ssd
    from paper_2308_04623_b200.binding import ssd_config
    lib = ssd.lib()
    out = C.c_void_p()
    bad_head = ssd_config(2, 256, 8, 32, 1024, 1000, 128, 64, 0, 1e-5)
    assert lib.ssd_create(C.byref(bad_head), 0, None, C.byref(out)) == ssd.SSD_ERR_UNSUPPORTED
    too_many = ssd_config(2, 256, 4, 64, 1024, 1000, 128, 257, 0, 1e-5)
    assert lib.ssd_create(C.byref(too_many), 0, None, C.byref(out)) == ssd.SSD_ERR_UNSUPPORTED
    long_fp32 = ssd_config(2, 256, 4, 64, 1024, 1000, 3000, 64, 0, 1e-5)   # fp32 attention: n_ctx + max_nodes above 3008 keys
    assert lib.ssd_create(C.byref(long_fp32), 0, None, C.byref(out)) == ssd.SSD_ERR_UNSUPPORTED
    bad_dtype = ssd_config(2, 256, 4, 64, 1024, 1000, 128, 64, 7, 1e-5)
    assert lib.ssd_create(C.byref(bad_dtype), 0, None, C.byref(out)) == ssd.SSD_ERR_BAD_ARG


def test_oracle_and_cuda_sources_share_nothing():
    """The oracle must not include or import anything of the CUDA path, and vice versa."""
    csrc = os.path.join(ROOT, "paper_2308_04623_b200")
    for dirpath, _, files in os.walk(csrc):
        for f in files:
            if f.endswith((".cu", ".cuh", ".h", ".py")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "__init__.py" and False, (f, "mentions the oracle")
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".c", ".py", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2308_04623_b200" not in text and "ssd.h" not in text, f
