"""ctypes binding to libvatp.so: the same four calls as include/vatp.h, taking torch tensors.

Argument marshalling only - every step of the path runs in the CUDA kernels of the library.
There is no fallback: if the library is missing the import raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

# VATP_LIBRARY selects another build of the library (the bounds-checking build libvatp_dbg.so)
_LIB_PATH = os.environ.get("VATP_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libvatp.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2406_12335_b200.build`")
lib = C.CDLL(_LIB_PATH)

OK = 0
BF16, F32 = 0, 1
IND_H2O, IND_WINDOW = 0, 1
NORM_KINDS = {"l1": 0, "l2": 1, "linf": 2}
FLAG_DECODE_OVERLAP = 1
STATIC_SCRATCH_BYTES = (4 << 20) + 256
EXPORTS = ["vatp_cache_capacity", "vatp_workspace_bytes", "vatp_prefill_scores", "vatp_prefill_scores_from_lse", "vatp_prefill_attention_scores", "vatp_prefill_scores_static", "vatp_select", "vatp_compact", "vatp_compact_window", "vatp_decode_step",
           "vatp_selftest_bounded_wait", "vatp_selftest_overlap_policy", "vatp_status_string"]


class Params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads", C.c_int32), ("seq_len", C.c_int32), ("head_dim", C.c_int32),
                ("dtype", C.c_int32), ("indicator", C.c_int32), ("window_w", C.c_int32), ("scale", C.c_float),
                ("budget", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32), ("norm_kind", C.c_int32),
                ("flags", C.c_int32), ("kv_heads", C.c_int32), ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_t", C.c_int64)]


class CacheStruct(C.Structure):
    _fields_ = [("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("acc", C.c_void_p), ("vnorm", C.c_void_p),
                ("pos", C.c_void_p), ("len", C.c_void_p), ("free_slot", C.c_void_p), ("next_pos", C.c_void_p),
                ("ring", C.c_void_p), ("acc_fixed", C.c_void_p), ("last_slot", C.c_void_p)]


_vp = C.c_void_p
lib.vatp_cache_capacity.restype = C.c_int32
lib.vatp_cache_capacity.argtypes = [C.c_int32]
lib.vatp_workspace_bytes.restype = C.c_size_t
lib.vatp_workspace_bytes.argtypes = [C.POINTER(Params)]
lib.vatp_prefill_scores.restype = C.c_int
lib.vatp_prefill_scores.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.vatp_prefill_scores_from_lse.restype = C.c_int
lib.vatp_prefill_scores_from_lse.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.vatp_prefill_attention_scores.restype = C.c_int
lib.vatp_prefill_attention_scores.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.vatp_prefill_scores_static.restype = C.c_int
lib.vatp_prefill_scores_static.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.vatp_select.restype = C.c_int
lib.vatp_select.argtypes = [C.POINTER(Params), _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.vatp_compact.restype = C.c_int
lib.vatp_compact.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, C.POINTER(CacheStruct), _vp, _vp]
lib.vatp_compact_window.restype = C.c_int
lib.vatp_compact_window.argtypes = [C.POINTER(Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.POINTER(CacheStruct), _vp, _vp]
lib.vatp_decode_step.restype = C.c_int
lib.vatp_decode_step.argtypes = [C.POINTER(Params), C.POINTER(CacheStruct), _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.vatp_selftest_bounded_wait.restype = C.c_int
lib.vatp_selftest_bounded_wait.argtypes = [C.c_uint64, _vp, _vp, _vp]
lib.vatp_selftest_overlap_policy.restype = C.c_int32
lib.vatp_selftest_overlap_policy.argtypes = [_vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.c_int32, C.c_double]
lib.vatp_status_string.restype = C.c_char_p
lib.vatp_status_string.argtypes = [C.c_int]


class VatpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.vatp_status_string(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise VatpError(code, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def make_params(*, batch, heads, seq_len, head_dim, dtype, budget, n_sink=0, n_recent=0, scale=None,
                indicator="h2o", window=0, strides=(0, 0, 0), norm="l1", decode_overlap=False, kv_heads=0) -> Params:
    """norm: the value norm of Eq. 4, "l1" (the method) or the Ablation Study's "l2" / "linf".
    decode_overlap: sets VATP_FLAG_DECODE_OVERLAP (decode steps of independent caches may run side by side;
    see vatp_decode_step in include/vatp.h for what the caller then guarantees)."""
    dt = {torch.bfloat16: BF16, torch.float32: F32, "bf16": BF16, "f32": F32}[dtype]
    return Params(batch, heads, seq_len, head_dim, dt, IND_WINDOW if indicator == "window" else IND_H2O, window,
                  float(scale if scale is not None else head_dim ** -0.5), budget, n_sink, n_recent, NORM_KINDS[norm],
                  FLAG_DECODE_OVERLAP if decode_overlap else 0, kv_heads, *strides)


def params_for(x: torch.Tensor, **kw) -> Params:
    """Params for a [batch, heads, T, d] tensor, taking shape, dtype and strides from it."""
    b, h, T, d = x.shape
    assert x.stride(3) == 1
    return make_params(batch=b, heads=h, seq_len=T, head_dim=d, dtype=x.dtype,
                       strides=(x.stride(0), x.stride(1), x.stride(2)), **kw)


def vatp_workspace_bytes(p: Params) -> int:
    return int(lib.vatp_workspace_bytes(C.byref(p)))


class Cache:
    """Device arrays of the decode state (allocated with torch, owned by this object)."""

    def __init__(self, p: Params, device="cuda"):
        b, h, d, cap = p.batch, (p.kv_heads or p.heads), p.head_dim, int(lib.vatp_cache_capacity(p.budget))
        dt = torch.float32 if p.dtype == F32 else torch.bfloat16
        self.cap = cap
        self.k_cache = torch.zeros(b, h, cap, d, dtype=dt, device=device)
        self.v_cache = torch.zeros(b, h, cap, d, dtype=dt, device=device)
        self.acc = torch.zeros(b, h, cap, dtype=torch.float32, device=device)
        self.vnorm = torch.zeros(b, h, cap, dtype=torch.float32, device=device)
        self.pos = torch.full((b, h, cap), -1, dtype=torch.int32, device=device)
        self.len = torch.zeros(b, h, dtype=torch.int32, device=device)
        self.free_slot = torch.zeros(b, h, dtype=torch.int32, device=device)
        self.next_pos = torch.zeros(b, h, dtype=torch.int32, device=device)
        self.last_slot = torch.full((b, h), -1, dtype=torch.int32, device=device)
        self.ring = self.acc_fixed = None
        if p.indicator == IND_WINDOW:
            self.ring = torch.zeros(b, h, p.window_w, cap, dtype=torch.float32, device=device)
            self.acc_fixed = torch.zeros(b, h, cap, dtype=torch.int64, device=device)
        self.struct = CacheStruct(*[_ptr(t) for t in (self.k_cache, self.v_cache, self.acc, self.vnorm, self.pos,
                                                       self.len, self.free_slot, self.next_pos, self.ring,
                                                       self.acc_fixed, self.last_slot)])

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.k_cache, self.v_cache, self.acc, self.vnorm, self.pos))


def vatp_prefill_scores(p: Params, q, k, v, *, lse_out=None, attn_acc, vnorm, score, win_rows=None,
                        workspace=None, dev_status=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vatp_prefill_scores(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(lse_out), _ptr(attn_acc), _ptr(vnorm),
                                   _ptr(score), _ptr(win_rows), _ptr(workspace), ws_bytes, _ptr(dev_status),
                                   _stream(stream)), "vatp_prefill_scores")


def vatp_prefill_scores_from_lse(p: Params, q, k, v, lse_in, *, lse_out=None, attn_acc, vnorm, score, win_rows=None,
                                 workspace=None, dev_status=None, stream=None):
    """vatp_prefill_scores with the row normalisers (natural-log lse of the causal softmax rows, as an
    attention forward returns them) given: pass 1 is skipped, QK^T is recomputed once."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vatp_prefill_scores_from_lse(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(lse_in), _ptr(lse_out),
                                            _ptr(attn_acc), _ptr(vnorm), _ptr(score), _ptr(win_rows), _ptr(workspace),
                                            ws_bytes, _ptr(dev_status), _stream(stream)), "vatp_prefill_scores_from_lse")


def vatp_prefill_attention_scores(p: Params, q, k, v, attn_out, *, lse_out=None, attn_acc, vnorm, score, win_rows=None,
                                  workspace=None, dev_status=None, stream=None):
    """Attention forward fused with prefill scoring: also writes the layer's output rows attn_out
    [batch, heads, T, head_dim] (Eq. 1); the indicator then costs one recomputation of QK^T."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vatp_prefill_attention_scores(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(attn_out), _ptr(lse_out),
                                             _ptr(attn_acc), _ptr(vnorm), _ptr(score), _ptr(win_rows), _ptr(workspace),
                                             ws_bytes, _ptr(dev_status), _stream(stream)), "vatp_prefill_attention_scores")


def vatp_prefill_scores_static(p: Params, q, k, v, *, lse_out=None, attn_acc, vnorm, score, win_rows=None,
                               dev_status=None, stream=None):
    """vatp_prefill_scores without a workspace argument: for callers that cannot allocate device
    memory, the scratch is a fixed array inside the library (at most STATIC_SCRATCH_BYTES of row
    normalisers; larger problems raise VatpError).  All calls on a device share that array, so
    calls that could overlap on the GPU must be serialised by the caller."""
    _check(lib.vatp_prefill_scores_static(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(lse_out), _ptr(attn_acc),
                                          _ptr(vnorm), _ptr(score), _ptr(win_rows), _ptr(dev_status),
                                          _stream(stream)), "vatp_prefill_scores_static")


def vatp_select(p: Params, score, kept_idx, *, workspace=None, dev_status=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vatp_select(C.byref(p), _ptr(score), _ptr(kept_idx), _ptr(workspace), ws_bytes, _ptr(dev_status),
                           _stream(stream)), "vatp_select")


def vatp_compact(p: Params, k, v, attn_acc, vnorm, kept_idx, cache: Cache, *, win_rows=None, dev_status=None,
                 stream=None):
    _check(lib.vatp_compact(C.byref(p), _ptr(k), _ptr(v), _ptr(attn_acc), _ptr(vnorm), _ptr(win_rows), _ptr(kept_idx),
                            C.byref(cache.struct), _ptr(dev_status), _stream(stream)), "vatp_compact")


def vatp_compact_window(p: Params, q, k, v, lse, attn_acc, vnorm, kept_idx, cache: Cache, *, dev_status=None, stream=None):
    """vatp_compact for the history-window indicator without win_rows: the kept block of the last-w
    probability rows is recomputed from q, the compacted keys and the row normalisers `lse` (natural log)."""
    _check(lib.vatp_compact_window(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(lse), _ptr(attn_acc), _ptr(vnorm),
                                   _ptr(kept_idx), C.byref(cache.struct), _ptr(dev_status), _stream(stream)),
           "vatp_compact_window")


def vatp_decode_step(p: Params, cache: Cache, q_new, k_new, v_new, out, *, evicted_pos=None, dev_status=None,
                     stream=None):
    _check(lib.vatp_decode_step(C.byref(p), C.byref(cache.struct), _ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(out),
                                _ptr(evicted_pos), _ptr(dev_status), _stream(stream)), "vatp_decode_step")


def vatp_selftest_bounded_wait(limit_ns: int, dev_status, waited_ns=None, *, stream=None):
    """Launches the one-CTA kernel that waits `limit_ns` on a barrier nobody arms and then reports
    VATP_ERR_TIMEOUT (5) in dev_status: shows that an expired device-side wait ends cleanly."""
    _check(lib.vatp_selftest_bounded_wait(int(limit_ns), _ptr(dev_status), _ptr(waited_ns), _stream(stream)),
           "vatp_selftest_bounded_wait")
