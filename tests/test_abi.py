"""The C-ABI shared library on a machine without a GPU: it loads, exports every function that
include/sparq.h declares, names its status codes, and rejects what the host can see before it
touches the device."""
import ctypes
import os
import re

import pytest

from paper_2312_04985_b200 import build, sparq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return sparq.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sparq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"^\s*(?:const\s+char\*|int|size_t)\s+(\w+)\s*\(", text, flags=re.M)))


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert {"sparq_cache_append", "sparq_cache_build", "sparq_decode", "dense_decode", "dense_decode_static",
            "sparq_step_host", "sparq_status_string"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(sparq.EXPORTS)          # the binding wraps exactly the header's surface


def test_status_strings(lib):
    codes = {0: "SPARQ_OK", 1: "SPARQ_ERR_NULL_POINTER", 2: "SPARQ_ERR_BAD_SHAPE", 3: "SPARQ_ERR_BAD_RK",
             4: "SPARQ_ERR_WORKSPACE", 5: "SPARQ_ERR_TOO_LONG", 6: "SPARQ_ERR_CUDA", 7: "SPARQ_ERR_STATIC_SCRATCH",
             8: "SPARQ_ERR_ALIGNMENT", 9: "SPARQ_ERR_BAD_OPTION",
             16: "SPARQ_DEV_BAD_SEQ_LEN", 17: "SPARQ_DEV_CACHE_FULL", 18: "SPARQ_DEV_TIMEOUT"}
    for code, name in codes.items():
        assert sparq.status_string(code) == name
    assert sparq.status_string(999) == "SPARQ_UNKNOWN_STATUS"


def test_host_visible_errors_need_no_device(lib):
    one = ctypes.c_void_p(16)            # never dereferenced: every call below is refused before any launch
    n = None
    # null pointers
    assert lib.sparq_decode(n, one, one, one, one, one, 1, 1, 1, 128, 8, 1, 1, one, n, n, n, n, 0, n, n) == sparq.ERR_NULL_POINTER
    assert lib.dense_decode(one, n, one, one, 1, 1, 1, 128, 8, one, n, 0, n, n) == sparq.ERR_NULL_POINTER
    assert lib.dense_decode_static(one, one, one, one, 1, 1, 1, 128, 8, n, n, n) == sparq.ERR_NULL_POINTER
    assert lib.sparq_cache_append(one, one, one, one, one, one, one, n, 1, 1, 128, 8, n, n) == sparq.ERR_NULL_POINTER
    assert lib.sparq_cache_build(one, one, one, one, n, one, 1, 1, 128, 8, n, n) == sparq.ERR_NULL_POINTER
    # the host-buffer step: k_new and v_new may be NULL only together (then q_host is the packed buffer)
    step = lambda q, kn, vn, out: lib.sparq_step_host(q, kn, vn, one, one, one, one, one, one, 1, 1, 1, 128, 8, 1, 1, out, n, 0, n, n)
    assert step(one, n, one, one) == sparq.ERR_NULL_POINTER
    assert step(one, one, n, one) == sparq.ERR_NULL_POINTER
    assert step(n, n, n, one) == sparq.ERR_NULL_POINTER
    assert step(one, n, n, n) == sparq.ERR_NULL_POINTER
    assert step(one, n, n, one) == sparq.ERR_WORKSPACE          # packed form accepted; refused next for its missing staging area
    # shapes: d != 128, Hq not a multiple of Hkv, S_max not a multiple of 8, B < 1
    for B, Hq, Hkv, d, S in ((1, 1, 1, 64, 8), (1, 3, 2, 128, 8), (1, 1, 1, 128, 12), (0, 1, 1, 128, 8)):
        assert lib.sparq_decode(one, one, one, one, one, one, B, Hq, Hkv, d, S, 1, 1, one, n, n, n, n, 0, n, n) == sparq.ERR_BAD_SHAPE
        assert lib.dense_decode(one, one, one, one, B, Hq, Hkv, d, S, one, n, 0, n, n) == sparq.ERR_BAD_SHAPE
    # r and k ranges
    for r, k in ((0, 1), (129, 1), (4, -1), (4, sparq.K_MAX + 1)):
        assert lib.sparq_decode(one, one, one, one, one, one, 1, 1, 1, 128, 8, r, k, one, n, n, n, n, 0, n, n) == sparq.ERR_BAD_RK
    # settings of sparq_decode_opt: unknown temperature, window out of range; its other checks are sparq_decode's
    opt = lambda tau, realloc, window, q=one, r=1: lib.sparq_decode_opt(
        q, one, one, one, one, one, 1, 1, 1, 128, 8, r, 1, tau, realloc, window, one, n, n, n, n, 0, n, n)
    for tau, window in ((3, 0), (-1, 0), (0, -1), (0, sparq.K_MAX + 1)):
        assert opt(tau, 1, window) == sparq.ERR_BAD_OPTION
    assert opt(2, 0, 5, q=n) == sparq.ERR_NULL_POINTER
    assert opt(2, 0, 5, r=0) == sparq.ERR_BAD_RK
    gopt = lambda tau, window: lib.sparq_decode_grouped_opt(
        one, one, one, one, one, one, 1, 2, 1, 128, 8, 1, 1, tau, 1, window, one, n, n, n, one, 1 << 20, n, n)
    for tau, window in ((3, 0), (0, -1), (0, sparq.K_MAX + 1)):
        assert gopt(tau, window) == sparq.ERR_BAD_OPTION
    # a tensor pointer that is not 16-byte aligned (the kernels would fault on it)
    odd = ctypes.c_void_p(24)
    assert lib.sparq_decode(one, one, odd, one, one, one, 1, 1, 1, 128, 8, 1, 1, one, n, n, n, n, 0, n, n) == sparq.ERR_ALIGNMENT
    assert lib.sparq_decode(one, one, one, one, one, one, 1, 1, 1, 128, 8, 1, 1, one, n, n, n, odd, 64, n, n) == sparq.ERR_ALIGNMENT
    assert lib.sparq_cache_append(odd, one, one, one, one, one, one, one, 1, 1, 128, 8, n, n) == sparq.ERR_ALIGNMENT
    assert lib.sparq_cache_build(one, one, one, one, odd, one, 1, 1, 128, 8, n, n) == sparq.ERR_ALIGNMENT
    assert lib.dense_decode(one, one, one, one, 1, 1, 1, 128, 8, odd, n, 0, n, n) == sparq.ERR_ALIGNMENT
    assert lib.sparq_decode_grouped(one, one, one, one, one, one, 1, 2, 1, 128, 8, 1, 1, 1, odd, n, n, n, one, 1 << 20, n, n) == sparq.ERR_ALIGNMENT
    assert lib.sparq_decode_1xk(one, odd, one, one, one, 1, 1, 1, 128, 8, 1, 1, one, n, n, n, one, 1 << 20, n, n) == sparq.ERR_ALIGNMENT
    # dense_decode: a split plan without a workspace; the static variant: a plan beyond its built-in scratch
    assert sparq.dense_workspace_bytes(1, 32, 32, 128, 4096) == 32 * 16 * 130 * 4   # 16 splits of 256 positions
    assert lib.dense_decode(one, one, one, one, 1, 32, 32, 128, 4096, one, n, 0, n, n) == sparq.ERR_WORKSPACE
    assert lib.dense_decode_static(one, one, one, one, 2, 1024, 32, 128, 4096, one, n, n) == sparq.ERR_STATIC_SCRATCH
    assert sparq.sparq_workspace_bytes(64, 32, 32, 128, 4096, 32, 128) == 0
    assert sparq.sparq_step_host_staging_bytes(2, 4, 2, 128, 64, 4, 8) == (2 * 2 * 4 * 128 + 2 * 2 * 2 * 128) * 2 + 64   # + decode workspace


def test_binding_refuses_cpu_tensors():
    import torch
    t = torch.zeros(1, 1, 128, dtype=torch.float16)
    with pytest.raises(ValueError):
        sparq.sparq_decode(t, t.view(1, 1, 1, 128), t.view(1, 1, 128, 1), t.view(1, 1, 1, 128), t,
                           torch.ones(1, dtype=torch.int32), 1, 1, t.clone())
