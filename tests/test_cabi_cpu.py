"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments on the host before anything is launched (no GPU needed, no compute calls)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def V():
    from paper_2406_12335_b200 import build
    build.build()
    from paper_2406_12335_b200 import vatp
    return vatp


def test_exports_every_declared_symbol(V):
    header = open(os.path.join(ROOT, "include", "vatp.h")).read()
    declared = set(re.findall(r"\b(vatp_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(V.lib, name), f"{name} not exported"
    assert set(V.EXPORTS) == declared, "binding and header disagree"


def test_struct_layout_matches_header(V):
    assert C.sizeof(V.Params) == 72       # 7 int32 + float + 3 int32 + pad + 3 int64
    assert V.Params.stride_b.offset == 48
    assert C.sizeof(V.CacheStruct) == 88


def test_status_strings(V):
    assert V.lib.vatp_status_string(0) == b"ok"
    assert b"workspace" in V.lib.vatp_status_string(3)


def test_host_side_validation(V):
    ok = dict(batch=1, heads=2, seq_len=64, head_dim=64, dtype="f32", budget=16, n_sink=2, n_recent=4)
    assert V.vatp_workspace_bytes(V.make_params(**ok)) == 2048 + 256   # 2 units x one padded 256-token chunk x 4 bytes, then the work-item counters
    assert V.vatp_workspace_bytes(V.make_params(**{**ok, "head_dim": 96})) == 0
    assert V.vatp_workspace_bytes(V.make_params(**{**ok, "n_recent": 15})) == 0     # F + R > B
    p = V.make_params(**ok)
    null = None
    # null data pointers
    assert V.lib.vatp_prefill_scores(C.byref(p), null, null, null, null, null, null, null, null, null, 0, null, null) == 1
    assert V.lib.vatp_select(C.byref(p), null, null, null, 0, null, null) == 1
    bad = V.make_params(**{**ok, "n_sink": 20})
    assert V.lib.vatp_select(C.byref(bad), 16, 16, null, 0, null, null) == 1
    unsup = V.make_params(**{**ok, "head_dim": 80})
    assert V.lib.vatp_select(C.byref(unsup), 16, 16, null, 0, null, null) == 2
    # misaligned q pointer, workspace missing when lse_out is null
    assert V.lib.vatp_prefill_scores(C.byref(p), 8, 16, 16, null, 16, 16, 16, null, null, 0, null, null) == 1
    assert V.lib.vatp_prefill_scores(C.byref(p), 16, 16, 16, null, 16, 16, 16, null, null, 0, null, null) == 3
    assert V.lib.vatp_prefill_scores(C.byref(p), 16, 16, 16, null, 16, 16, 16, null, 256, 8, null, null) == 3
    wp = V.make_params(**{**ok, "indicator": "window", "window": 0})
    assert V.lib.vatp_select(C.byref(wp), 16, 16, null, 0, null, null) == 1
    wp = V.make_params(**{**ok, "indicator": "window", "window": 8})
    assert V.lib.vatp_prefill_scores(C.byref(wp), 16, 16, 16, 16, 16, 16, 16, null, null, 0, null, null) == 1  # win_rows
    # strides that are not multiples of 16 bytes
    sp = V.make_params(**{**ok, "strides": (0, 0, 65)})
    assert V.lib.vatp_prefill_scores(C.byref(sp), 16, 16, 16, 16, 16, 16, 16, null, null, 0, null, null) == 1
    # decode: null cache
    assert V.lib.vatp_decode_step(C.byref(p), null, 16, 16, 16, 16, null, null, null) == 1
