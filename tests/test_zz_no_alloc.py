"""The allocation-free prefill entry point against the ordinary one.

vatp_prefill_scores_static exists for callers that cannot obtain device scratch (plugins inside
an application that owns the allocator, loops where an allocation's device-wide synchronisation
is not acceptable): its scratch is a fixed array inside the library.  It must give what
vatp_prefill_scores gives with a caller-supplied workspace - here on two calls in a row with
different inputs, because the built-in array is shared and keeps the previous call's contents.

Collected last on purpose (file name), so that a failure here cannot hide another test's result
in a run that stops at the first failure.  Passes alone in a fresh process and after the others.
"""
import pytest
import torch

from paper_2406_12335_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


def _both(wl, layer):
    V = P.vatp()
    q, k, v = synth.prefill_inputs(wl, layer, "cuda")
    p = V.params_for(q, budget=wl.budget, n_sink=wl.n_sink, n_recent=wl.n_recent, scale=wl.scale,
                     indicator=wl.indicator, window=wl.window)
    b, h, T = wl.batch, wl.heads, wl.seq_len
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def outputs():
        return {n: torch.empty(b, h, T, dtype=torch.float32, device="cuda") for n in ("lse", "attn_acc", "vnorm", "score")}

    ref, got = outputs(), outputs()
    ws = torch.empty(V.vatp_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    V.vatp_prefill_scores(p, q, k, v, lse_out=ref["lse"], attn_acc=ref["attn_acc"], vnorm=ref["vnorm"],
                          score=ref["score"], workspace=ws, dev_status=status)
    V.vatp_prefill_scores_static(p, q, k, v, lse_out=got["lse"], attn_acc=got["attn_acc"], vnorm=got["vnorm"],
                                 score=got["score"], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tol = P.TOL[wl.dtype]
    for name in ("attn_acc", "vnorm", "score"):
        e = P.rel_err(P.to_np64(got[name]), P.to_np64(ref[name]))
        assert e <= tol, f"{name}: static-scratch variant differs from the workspace variant by {e:.3g}"
    assert float((got["lse"] - ref["lse"]).abs().max()) <= 10 * tol
    assert float((got["attn_acc"].double().sum(-1) - T).abs().max()) <= 2e-3 * T


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # tensor-core path (bf16, d 128), a ragged length first and a longer prompt second, so the second
    # call finds the first call's normalisers in the shared array
    _both(synth.Workload(95, "noalloc_a", "bf16", 2, 3, 1, 128, 1000, 300, 2, 20, "h2o", 0, 0), 0)
    _both(synth.Workload(96, "noalloc_b", "bf16", 1, 4, 1, 128, 2304, 512, 0, 64, "h2o", 0, 0), 1)
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
