"""Host-side checks of the C-ABI library that need no GPU: it builds, loads, exports every
symbol the header declares, sizes the workspace as documented and rejects bad arguments
before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2411_15785_b200 import binding as B
from paper_2411_15785_b200 import build as bld

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    bld.build()
    return B.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "bct.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bct_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_version_and_error_string(lib):
    assert lib.bct_version() >= 100
    assert isinstance(B.last_error(), str)


def test_params_struct_matches_header_layout():
    assert ctypes.sizeof(B.BctParams) == 12 * 4


def test_cache_bytes_accounts_for_planes_and_staging(lib):
    import torch
    p = B.make_params(64, 32, 32, 128, 2048, torch.bfloat16, init_len=2048)
    nbytes, align = B.cache_bytes(p)
    plane = 64 * 32 * 2048 * 128 * 2
    assert align == 256
    step = 64 * 32 * 128 * 2                                          # q, k, v or out of one token
    progress = 64 * 32 * 8                                            # one 64-bit progress word per (sequence, kv-head) unit
    assert 3 * plane + 2 * 4 * step + progress <= nbytes <= 3 * plane + 2 * 4 * step + progress + 32 * 256   # two staging sets
    p32 = B.make_params(1, 1, 1, 64, 128, torch.float32)
    n32, _ = B.cache_bytes(p32)
    assert 2 * 128 * 64 * 4 <= n32 < 2 * 128 * 64 * 4 + 8192       # no residual plane in float
    big = B.make_params(1, 1, 1, 64, 128, torch.float32, max_stream=100)
    assert B.cache_bytes(big)[0] > n32                               # staging grows with max_stream only


@pytest.mark.parametrize("kw,status", [
    (dict(batch=0), B.BCT_ERR_INVALID_ARG),
    (dict(n_q_heads=5, n_kv_heads=2), B.BCT_ERR_INVALID_ARG),
    (dict(capacity=0), B.BCT_ERR_INVALID_ARG),
    (dict(init_len=9, capacity=8), B.BCT_ERR_INVALID_ARG),
    (dict(flags=1 << 9), B.BCT_ERR_INVALID_ARG),
    (dict(head_dim=96), B.BCT_ERR_UNSUPPORTED),
    (dict(n_q_heads=16, n_kv_heads=1), B.BCT_ERR_UNSUPPORTED),
])
def test_bad_params_rejected_on_host(lib, kw, status):
    import torch
    base = dict(batch=2, n_q_heads=4, n_kv_heads=2, head_dim=64, capacity=8, dtype=torch.bfloat16)
    base.update(kw)
    p = B.make_params(**base)
    n = ctypes.c_size_t(0)
    assert lib.bct_cache_bytes(ctypes.byref(p), ctypes.byref(n), None) == status
    assert B.last_error() != ""


def test_null_arguments_rejected(lib):
    n = ctypes.c_size_t(0)
    assert lib.bct_cache_bytes(None, ctypes.byref(n), None) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_decode_step(None, None, None, None, None, None) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_prefill_stream(None, None, None, None, None, 4, None) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_cache_status(None, None) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_cache_destroy(None) == B.BCT_OK
    h = ctypes.c_void_p(None)
    import torch
    p = B.make_params(1, 1, 1, 64, 8, torch.float32)
    assert lib.bct_cache_create(ctypes.byref(p), None, 1 << 20, None, None, None, ctypes.byref(h)) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_cache_create(ctypes.byref(p), 256, 16, None, None, None, ctypes.byref(h)) == B.BCT_ERR_INVALID_ARG
    assert lib.bct_cache_create(ctypes.byref(p), 264, 1 << 20, None, None, None, ctypes.byref(h)) == B.BCT_ERR_INVALID_ARG
    assert not h.value


def test_a_pointer_that_is_no_live_handle_is_refused_without_being_read(lib):
    # the library looks a handle up in its list of live handles before touching it: an address that was never a
    # handle (here: not even mapped) is answered with BCT_ERR_STATE
    bogus = ctypes.c_void_p(0x1000)
    n = ctypes.c_int32(0)
    assert lib.bct_cache_len(bogus, ctypes.byref(n)) == B.BCT_ERR_STATE
    assert lib.bct_cache_destroy(bogus) == B.BCT_ERR_STATE
    assert lib.bct_decode_step(bogus, 256, 256, 256, 256, None) == B.BCT_ERR_STATE
    assert lib.bct_prefill_stream_host_static(bogus, 256, 256, 256, 256, 1, None) == B.BCT_ERR_STATE
    assert lib.bct_selftest_timeout(bogus, None) == B.BCT_ERR_STATE
    r = ctypes.c_uint64(0)
    assert lib.bct_cache_rows_rewritten(bogus, None, ctypes.byref(r)) == B.BCT_ERR_STATE
    assert "destroyed" in B.last_error()


def test_no_environment_variable_is_read():
    # the library and its binding take every setting through arguments
    assert "environ" not in open(os.path.join(ROOT, "paper_2411_15785_b200", "binding.py")).read()
    csrc = os.path.join(ROOT, "paper_2411_15785_b200", "csrc")
    for name in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, name)).read(), name
