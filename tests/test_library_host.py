"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, sizes its workspace, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2504_09936_b200 import binding as kb
from paper_2504_09936_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kbuild.build()
    return kb.lib()


def test_exports_match_header(lib):
    hdr = open(os.path.join(ROOT, "include", "keepkv.h")).read()
    declared = set(re.findall(r"\b(keepkv_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(kb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layout_matches_header():
    assert C.sizeof(kb.keepkv_params) == 16 * 4
    assert C.sizeof(kb.keepkv_cache) == 5 * 8


def test_workspace_bytes_and_validation(lib):
    p = kb.make_params(B=8, H_q=32, H_kv=8, d=128, N_cap=8320)
    n = kb.keepkv_workspace_bytes(p)
    assert n > 0 and n % 256 == 0
    for bad, code in ((dict(d=96), -2), (dict(H_q=24), -2), (dict(N_cap=100), -2), (dict(B=0), -1),
                      (dict(ema_alpha=1.0), -1), (dict(N_cap=65536), -2)):
        args = dict(B=8, H_q=32, H_kv=8, d=128, N_cap=8320)
        args.update(bad)
        q = kb.make_params(**args)
        sz = C.c_size_t()
        assert lib.keepkv_workspace_bytes(C.byref(q), C.byref(sz)) == code, bad
    assert lib.keepkv_workspace_bytes(None, None) == -1
    assert lib.keepkv_status_string(-3) == b"KEEPKV_ERR_CAPACITY"


def test_calls_reject_null_and_capacity_before_any_launch(lib):
    p = kb.make_params(B=1, H_q=8, H_kv=2, d=64, N_cap=576, period=32)
    c = kb.keepkv_cache(None, None, None, None, None)
    assert lib.keepkv_append(C.byref(p), C.byref(c), None, None, None, None) == -1
    assert lib.keepkv_decode_attention(C.byref(p), C.byref(c), None, None, None, 0, None, 0, None, None) == -1
    fake = kb.keepkv_cache(256, 512, 768, 1024, 1280)      # non-null, aligned, never dereferenced
    fake2 = kb.keepkv_cache(2560, 5120, 7680, 10240, 12800)
    # budget + period beyond N_cap
    assert lib.keepkv_compress(C.byref(p), C.byref(fake), C.byref(fake2), None, 560, None, None, None, None, 256, 1 << 40,
                               256, None) == -3
    # src and dst must differ
    assert lib.keepkv_compress(C.byref(p), C.byref(fake), C.byref(fake), None, 51, None, None, None, None, 256, 1 << 40,
                               256, None) == -1
    # workspace too small
    assert lib.keepkv_compress(C.byref(p), C.byref(fake), C.byref(fake2), None, 51, None, None, None, None, 256, 16,
                               256, None) == -4
    assert lib.keepkv_decode_attention(C.byref(p), C.byref(fake), 256, 256, None, 0, 256, 16, 256, None) == -4


def test_flags_and_decode_step_arguments_are_checked_before_any_launch(lib):
    fake = kb.keepkv_cache(256, 512, 768, 1024, 1280)      # non-null, aligned, never dereferenced
    fake2 = kb.keepkv_cache(2560, 5120, 7680, 10240, 12800)
    sz = C.c_size_t()
    # unknown flag bits are rejected by every call that takes the parameters
    bad = kb.make_params(B=1, H_q=8, H_kv=2, d=64, N_cap=576, period=32, flags=4)
    assert lib.keepkv_workspace_bytes(C.byref(bad), C.byref(sz)) == -1
    idle = kb.make_params(B=1, H_q=8, H_kv=2, d=64, N_cap=576, period=32, flags=kb.FLAG_CACHE_IDLE)
    assert lib.keepkv_workspace_bytes(C.byref(idle), C.byref(sz)) == 0
    # the steady-state promise needs something to keep
    st = kb.make_params(B=1, H_q=8, H_kv=2, d=64, N_cap=576, period=32, flags=kb.FLAG_COMPRESS_STEADY)
    assert lib.keepkv_workspace_bytes(C.byref(st), C.byref(sz)) == 0
    assert lib.keepkv_compress(C.byref(st), C.byref(fake), C.byref(fake2), None, 0, None, None, None, None, 256, 1 << 40,
                               256, None) == -1
    # keepkv_decode_step: null or misaligned token rows, short workspace
    p = kb.make_params(B=1, H_q=8, H_kv=2, d=64, N_cap=576, period=32)
    assert lib.keepkv_decode_step(C.byref(p), C.byref(fake), 256, None, 256, 256, None, 0, 256, 1 << 40, 256, None) == -1
    assert lib.keepkv_decode_step(C.byref(p), C.byref(fake), 256, 264, 256, 256, None, 0, 256, 1 << 40, 256, None) == -1
    assert lib.keepkv_decode_step(C.byref(p), C.byref(fake), 256, 256, 256, 256, None, 0, 256, 16, 256, None) == -4
