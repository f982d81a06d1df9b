"""The C-ABI library loads, exports every symbol the public header declares, and rejects bad
arguments on the host before touching a device.  No GPU needed."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_09316_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dsla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsla_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert {"dsla_prefill", "dsla_decode_step", "dsla_state_alloc", "dsla_state_free"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dsla.h but not exported"


def test_binding_covers_every_symbol(lib):
    import paper_2506_09316_b200 as dsla
    for n in declared_symbols():
        assert callable(getattr(dsla, n)), n


def test_status_strings(lib):
    lib.dsla_status_string.restype = ctypes.c_char_p
    got = [lib.dsla_status_string(i).decode() for i in range(6)]
    assert got == ["DSLA_OK", "DSLA_ERR_INVALID_ARG", "DSLA_ERR_UNSUPPORTED", "DSLA_ERR_CUDA", "DSLA_ERR_OOM",
                   "DSLA_ERR_TIMEOUT"]


def test_sizes_and_host_side_rejections(lib):
    from paper_2506_09316_b200 import binding as b
    assert b.dsla_state_bytes(128, 32, 128, 128) == 128 * 2 * 32 * 128 * 128 * 4
    assert b.dsla_state_bytes(0, 32, 128, 128) == 0 and b.dsla_state_bytes(1, 1, -1, 128) == 0
    h = ctypes.c_void_p()
    f = lib.dsla_state_alloc
    f.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                  ctypes.c_void_p, ctypes.c_size_t]
    assert f(None, 1, 1, 64, 64, None, 0) == b.DSLA_ERR_INVALID_ARG
    assert f(ctypes.byref(h), 0, 1, 64, 64, None, 0) == b.DSLA_ERR_INVALID_ARG
    assert f(ctypes.byref(h), 1, 1, 48, 48, None, 0) == b.DSLA_ERR_UNSUPPORTED
    assert f(ctypes.byref(h), 1, 1, 64, 128, None, 0) == b.DSLA_ERR_UNSUPPORTED
    assert f(ctypes.byref(h), 1, 1, 64, 64, ctypes.c_void_p(256), 8) == b.DSLA_ERR_INVALID_ARG   # too small
    assert f(ctypes.byref(h), 1, 1, 64, 64, ctypes.c_void_p(260), 1 << 20) == b.DSLA_ERR_INVALID_ARG  # misaligned
    # prefill / decode with a NULL state or NULL args never reach a launch
    a = b.dsla_prefill_args()
    assert lib.dsla_prefill(None, None, None) == b.DSLA_ERR_INVALID_ARG
    a.N, a.T, a.T_total, a.max_seqlen, a.H, a.d_k, a.d_v, a.chunk = 1, 8, 8, 8, 2, 64, 64, 64
    assert b._lib.dsla_prefill(ctypes.byref(a), None, None) == b.DSLA_ERR_INVALID_ARG
    a.d_k = a.d_v = 96
    assert b._lib.dsla_prefill(ctypes.byref(a), None, None) == b.DSLA_ERR_UNSUPPORTED
    a.d_k = a.d_v = 64
    a.chunk = 48
    assert b._lib.dsla_prefill(ctypes.byref(a), None, None) == b.DSLA_ERR_UNSUPPORTED
    a.chunk, a.T_total = 64, 9
    assert b._lib.dsla_prefill(ctypes.byref(a), None, None) == b.DSLA_ERR_INVALID_ARG      # N*T != T_total
    a.T_total, a.dtype = 8, 7
    assert b._lib.dsla_prefill(ctypes.byref(a), None, None) == b.DSLA_ERR_INVALID_ARG
    assert b._lib.dsla_prefill_workspace_bytes(None) == 0
    d = b.dsla_decode_args()
    assert b._lib.dsla_decode_step(ctypes.byref(d), None, None) == b.DSLA_ERR_INVALID_ARG
    assert b._lib.dsla_decode_step(None, None, None) == b.DSLA_ERR_INVALID_ARG
    assert b._lib.dsla_state_free(None) == b.DSLA_OK
    assert b._lib.dsla_state_zero(None, None, 0, None) == b.DSLA_ERR_INVALID_ARG
    assert b.dsla_launch_count() == 0


def test_product_package_does_not_import_the_checker():
    """Nothing under the CUDA package may import, load or name the CPU checker."""
    pkg = os.path.join(ROOT, "paper_2506_09316_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text, f"{fn} mentions the checker"
