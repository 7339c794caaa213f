"""The allocation-free prefill entry point against the ordinary one.

vatp_prefill_scores_static exists for callers that cannot obtain device scratch (plugins inside
an application that owns the allocator, loops where an allocation's device-wide synchronisation
is not acceptable): its scratch is a fixed array inside the library.  It must give, bit for
bit, what vatp_prefill_scores gives with a caller-supplied workspace - here on several calls in a row
with different inputs, because the built-in array is shared and keeps the previous call's contents -
and it must allocate nothing: the device's free memory is the same after the call as before it.

Collected last on purpose (file name), so that a failure here cannot hide another test's result
in a run that stops at the first failure.  Passes alone in a fresh process and after the others.
"""
import pytest
import torch

from paper_2406_12335_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


_static_calls = [0]      # static-scratch calls made so far in this process


def _both(wl, layer, oracle_unit=None):
    """The workspace variant and the static-scratch variant on the same inputs: their outputs must be
    equal bit for bit (both are deterministic and run the same kernels), the static call must leave the
    device's memory as it found it, and one unit may also be checked against the oracle."""
    V = P.vatp()
    q, k, v = synth.prefill_inputs(wl, layer, "cuda")
    p = V.params_for(q, budget=wl.budget, n_sink=wl.n_sink, n_recent=wl.n_recent, scale=wl.scale,
                     indicator=wl.indicator, window=wl.window)
    b, h, T = wl.batch, wl.heads, wl.seq_len
    windowed = wl.indicator == "window"
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def outputs():
        o = {n: torch.empty(b, h, T, dtype=torch.float32, device="cuda") for n in ("lse", "attn_acc", "vnorm", "score")}
        o["win_rows"] = torch.empty(b, h, wl.window, T, dtype=torch.float32, device="cuda") if windowed else None
        return o

    ref, got = outputs(), outputs()
    ws = torch.empty(V.vatp_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    V.vatp_prefill_scores(p, q, k, v, lse_out=ref["lse"], attn_acc=ref["attn_acc"], vnorm=ref["vnorm"],
                          score=ref["score"], win_rows=ref["win_rows"], workspace=ws, dev_status=status)
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    V.vatp_prefill_scores_static(p, q, k, v, lse_out=got["lse"], attn_acc=got["attn_acc"], vnorm=got["vnorm"],
                                 score=got["score"], win_rows=got["win_rows"], dev_status=status)
    torch.cuda.synchronize()
    # (the first call of a process looks up the built-in array, which is when the driver places the
    # library's device image: from the second call on nothing may change)
    if _static_calls[0] > 0:
        assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0, \
            "the static-scratch call changed the device's free memory"
    _static_calls[0] += 1
    assert int(status.item()) == 0
    first = max(T - wl.window, 0) if windowed else 0          # Eq. 3: normalisers exist for the window's rows only
    assert torch.equal(got["lse"][..., first:], ref["lse"][..., first:])
    for name in ("attn_acc", "vnorm", "score") + (("win_rows",) if windowed else ()):
        assert torch.equal(got[name], ref[name]), f"{name}: static-scratch variant differs from the workspace variant"
    rows = min(wl.window, T) if windowed else T
    assert float((got["attn_acc"].double().sum(-1) - rows).abs().max()) <= 2e-3 * rows
    if oracle_unit is not None:
        from oracle import vatp_oracle as O
        bb, hh = oracle_unit
        want = O.prefill(P.to_np64(q[bb, hh]), P.to_np64(k[bb, hh]), P.to_np64(v[bb, hh]), wl.scale,
                         window=wl.window if windowed else None)
        tol = P.TOL[wl.dtype]
        for name, key in (("attn_acc", "S"), ("vnorm", "n1"), ("score", "I")):
            e = P.rel_err(P.to_np64(got[name][bb, hh]), want[key])
            assert e <= tol, f"{name}: static-scratch variant differs from the oracle by {e:.3g}"


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # tensor-core path (bf16, d 128), a ragged length first and a longer prompt second, so the second
    # call finds the first call's normalisers in the shared array
    _both(synth.Workload(95, "noalloc_a", "bf16", 2, 3, 1, 128, 1000, 300, 2, 20, "h2o", 0, 0), 0, oracle_unit=(1, 2))
    _both(synth.Workload(96, "noalloc_b", "bf16", 1, 4, 1, 128, 2304, 512, 0, 64, "h2o", 0, 0), 1)
    # a history window (Eq. 3) after the accumulated indicator: pass 1 now writes the normalisers of the
    # window's tiles only, and the array below them still holds the previous call's
    _both(synth.Workload(98, "noalloc_w", "bf16", 1, 4, 1, 128, 2000, 500, 2, 10, "window", 300, 0), 0, oracle_unit=(0, 3))
    # fp32 FMA path through the same entry point
    _both(synth.Workload(97, "noalloc_c", "f32", 1, 2, 1, 64, 333, 100, 3, 17, "h2o", 0, 0), 0)


def test_static_scratch_rejects_oversized_problem():
    V = P.vatp()
    p = V.make_params(batch=8, heads=32, seq_len=8192, head_dim=128, dtype="bf16", budget=1638, n_recent=256)
    assert V.vatp_workspace_bytes(p) > V.STATIC_SCRATCH_BYTES
    x = torch.empty(16, device="cuda")
    with pytest.raises(V.VatpError) as ei:
        V.vatp_prefill_scores_static(p, x, x, x, attn_acc=x, vnorm=x, score=x)
    assert ei.value.code == 6 and "built-in scratch" in str(ei.value)
