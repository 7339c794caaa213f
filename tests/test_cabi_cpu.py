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
    assert C.sizeof(V.Params) == 80       # 7 int32 + float + 6 int32 + 3 int64
    assert V.Params.norm_kind.offset == 44 and V.Params.flags.offset == 48 and V.Params.kv_heads.offset == 52
    assert V.Params.stride_b.offset == 56
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
    # given-normaliser variant: lse_in is required and 16-byte aligned; then the usual checks apply
    assert V.lib.vatp_prefill_scores_from_lse(C.byref(p), 16, 16, 16, null, null, 16, 16, 16, null, 256, 4096, null, null) == 1
    assert V.lib.vatp_prefill_scores_from_lse(C.byref(p), 16, 16, 16, 8, null, 16, 16, 16, null, 256, 4096, null, null) == 1
    assert V.lib.vatp_prefill_scores_from_lse(C.byref(p), 16, 16, 16, 16, null, 16, 16, 16, null, null, 0, null, null) == 3
    wp = V.make_params(**{**ok, "indicator": "window", "window": 0})
    assert V.lib.vatp_select(C.byref(wp), 16, 16, null, 0, null, null) == 1
    wp = V.make_params(**{**ok, "indicator": "window", "window": 8})
    # the [w, T] probability rows are optional (vatp_compact_window needs none): the call gets as far as the workspace check
    assert V.lib.vatp_prefill_scores(C.byref(wp), 16, 16, 16, 16, 16, 16, 16, null, null, 0, null, null) == 3
    # vatp_compact needs them with a history window; vatp_compact_window needs the window, q and the row normalisers
    cs = V.CacheStruct(*([16] * 11))
    assert V.lib.vatp_compact(C.byref(wp), 16, 16, 16, 16, null, 16, C.byref(cs), null, null) == 1
    assert V.lib.vatp_compact_window(C.byref(p), 16, 16, 16, 16, 16, 16, 16, C.byref(cs), null, null) == 1     # H2O parameters
    assert V.lib.vatp_compact_window(C.byref(wp), 16, 16, 16, null, 16, 16, 16, C.byref(cs), null, null) == 1   # no lse
    assert V.lib.vatp_compact_window(C.byref(wp), null, 16, 16, 16, 16, 16, 16, C.byref(cs), null, null) == 1   # no q
    # strides that are not multiples of 16 bytes
    sp = V.make_params(**{**ok, "strides": (0, 0, 65)})
    assert V.lib.vatp_prefill_scores(C.byref(sp), 16, 16, 16, 16, 16, 16, 16, null, null, 0, null, null) == 1
    # decode: null cache
    assert V.lib.vatp_decode_step(C.byref(p), null, 16, 16, 16, 16, null, null, null) == 1
    # value norm kinds: l1 / l2 / linf are accepted, anything else is unsupported
    for kind in ("l1", "l2", "linf"):
        assert V.vatp_workspace_bytes(V.make_params(**ok, norm=kind)) == 2048 + 256
    odd = V.make_params(**ok)
    odd.norm_kind = 3
    assert V.vatp_workspace_bytes(odd) == 0
    assert V.lib.vatp_select(C.byref(odd), 16, 16, null, 0, null, null) == 2
    # grouped-query attention: kv_heads divides heads, contiguous layouts only; the workspace also holds the G partial indicators
    gq = dict(ok, heads=4)
    assert V.vatp_workspace_bytes(V.make_params(**gq, kv_heads=4)) == V.vatp_workspace_bytes(V.make_params(**gq))
    # (normalisers of the 4 query heads, padded to 256 tokens, the counters, then 2 partial indicators of 2 KV units)
    assert V.vatp_workspace_bytes(V.make_params(**gq, kv_heads=2)) == (4 * 256 * 4 + 256) + 2 * 2 * 64 * 4
    assert V.vatp_workspace_bytes(V.make_params(**gq, kv_heads=3)) == 0
    assert V.vatp_workspace_bytes(V.make_params(**gq, kv_heads=8)) == 0
    assert V.vatp_workspace_bytes(V.make_params(**gq, kv_heads=2, strides=(0, 0, 128))) == 0
    gw = V.make_params(**gq, kv_heads=2, indicator="window", window=8)
    assert V.lib.vatp_prefill_scores(C.byref(gw), 16, 16, 16, 16, 16, 16, 16, 16, 256, 1 << 20, null, null) == 2   # no win_rows with grouped queries
    assert V.lib.vatp_compact(C.byref(gw), 16, 16, 16, 16, 16, 16, C.byref(cs), null, null) == 2                   # nor the gather from them
    # attention forward fused with the scoring: the output array is required and 16-byte aligned, the usual checks follow
    fa = V.lib.vatp_prefill_attention_scores
    assert fa(C.byref(p), 16, 16, 16, null, null, 16, 16, 16, null, 256, 4096, null, null) == 1
    assert fa(C.byref(p), 16, 16, 16, 8, null, 16, 16, 16, null, 256, 4096, null, null) == 1
    assert fa(C.byref(p), 16, 16, 16, 16, null, 16, 16, 16, null, null, 0, null, null) == 3
    assert fa(C.byref(V.make_params(**gq, kv_heads=2)), 16, 16, 16, 16, null, 16, 16, 16, null, null, 0, null, null) == 3   # grouped queries: as far as the workspace check
    # flags: the decode-overlap bit is the only one defined
    assert V.make_params(**ok, decode_overlap=True).flags == V.FLAG_DECODE_OVERLAP == 1
    assert V.vatp_workspace_bytes(V.make_params(**ok, decode_overlap=True)) == 2048 + 256
    odd = V.make_params(**ok)
    odd.flags = 6
    assert V.vatp_workspace_bytes(odd) == 0
    assert V.lib.vatp_decode_step(C.byref(odd), null, 16, 16, 16, 16, null, null, null) == 1


def _probe(V, stream, caches, share):
    """One pretend decode launch touching the given (begin, bytes) ranges."""
    n = len(caches)
    begin = (C.c_uint64 * n)(*[c[0] for c in caches])
    size = (C.c_uint64 * n)(*[c[1] for c in caches])
    return V.lib.vatp_selftest_overlap_policy(C.c_void_p(stream), begin, size, n, share)


def test_decode_overlap_policy(V):
    """Host logic that decides whether a decode launch may run beside its predecessors: it must share no
    buffer with any recorded launch that can still be resident (every launch stays resident until the one
    before it has completed, so the shares of the launches in between bound how far back to look)."""
    MB = 1 << 20
    cache = lambda i: [(0x10_0000_0000 + i * 64 * MB, 32 * MB), (0x90_0000_0000 + i * MB, 4096)]
    # four caches in rotation, each launch holding 43% of the machine: the same cache comes back after
    # three others, whose shares add up to more than the machine -> its previous step has retired
    s = 0xA001
    assert _probe(V, s, cache(0), 0.43) == 0            # nothing known about what ran before the first launch
    assert [_probe(V, s, cache(i), 0.43) for i in (1, 2, 3)] == [1, 1, 1]
    assert [_probe(V, s, cache(i % 4), 0.43) for i in range(4, 12)] == [1] * 8
    # three caches in rotation: only two launches (86%) lie between a cache's steps -> it must wait
    s = 0xA002
    assert _probe(V, s, cache(0), 0.43) == 0
    assert [_probe(V, s, cache(i % 3), 0.43) for i in range(1, 9)] == [1, 1, 0, 0, 0, 0, 0, 0]
    # the same cache twice in a row always waits; a partial overlap of one buffer is enough
    s = 0xA003
    _probe(V, s, cache(0), 0.9)
    assert _probe(V, s, cache(0), 0.9) == 0
    assert _probe(V, s, [(0x10_0000_0000 + 31 * MB, 2 * MB)], 0.9) == 0
    assert _probe(V, s, cache(5), 0.9) == 1
    # tiny launches: more than the recorded history could still be resident -> never assume independence
    s = 0xA004
    got = [_probe(V, s, cache(i), 0.01) for i in range(12)]
    assert got[0] == 0 and got[1:8] == [1] * 7 and got[8:] == [0] * 4
    # streams do not see each other's launches
    assert _probe(V, 0xA005, cache(0), 0.43) == 0 and _probe(V, 0xA005, cache(1), 0.43) == 1
    assert _probe(V, 0xA005, [], 0.5) == -1
    # other work of the library on the stream (prefill, selection, compaction) ends the record: the next
    # launch waits whatever it touches, the ones after it are judged against it alone
    s = 0xA006
    assert [_probe(V, s, cache(i), 0.43) for i in range(4)] == [0, 1, 1, 1]
    assert _probe(V, s, cache(0), -1.0) == 0
    assert [_probe(V, s, cache(i), 0.43) for i in (7, 8, 7)] == [0, 1, 0]
