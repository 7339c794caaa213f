"""Shared machinery of the GPU parity tests: runs the CUDA path through the C-ABI binding, runs
the float64 oracle on the same bits, and compares.  Not collected by pytest itself."""
from __future__ import annotations

import math

import numpy as np
import torch

from oracle import vatp_oracle as O
from paper_2406_12335_b200 import synth

TOL = {"f32": 1e-5, "bf16": 1e-3}          # relative tolerance on scores, per input dtype
ABS_FLOOR = 1e-30                          # below fp32's normal range relative error is meaningless


def vatp():
    from paper_2406_12335_b200 import vatp as _v
    return _v


def to_np64(x: torch.Tensor) -> np.ndarray:
    return x.detach().to("cpu", torch.float64).numpy()


def attention_forward_lse(q: torch.Tensor, k: torch.Tensor, scale: float) -> torch.Tensor:
    """Stand-in for the log-sum-exp output of an attention forward: plain torch, float64 on the
    inputs' device, one unit at a time; [batch, heads, T] fp32."""
    b, h, T, _ = q.shape
    out = torch.empty(b, h, T, dtype=torch.float32, device=q.device)
    mask = torch.ones(T, T, dtype=torch.bool, device=q.device).triu(1)
    for i in range(b):
        for j in range(h):
            s = (q[i, j].double() @ k[i, j].double().T) * scale
            out[i, j] = torch.logsumexp(s.masked_fill(mask, float("-inf")), dim=-1).float()
    return out


class GpuPrefill:
    """Device buffers and the three prefill-side calls for one layer of a workload."""

    def __init__(self, wl: synth.Workload, q, k, v, *, n_sink=None, lse_given=False, decode_overlap=False,
                 recompute_window=False, fused_forward=False):
        """decode_overlap: decode steps through this object carry VATP_FLAG_DECODE_OVERLAP (steps of
        caches that share no buffer may run side by side on the GPU).  recompute_window (Eq. 3 only): the
        scoring call writes no win_rows and vatp_compact_window rebuilds the kept block of the history.
        fused_forward: scoring through vatp_prefill_attention_scores, which also writes the attention output."""
        V = vatp()
        self.wl = wl
        self.lse_given = lse_given
        self.fused_forward = fused_forward
        self.attn_out = torch.empty_like(q) if fused_forward else None
        self.F = wl.n_sink if n_sink is None else n_sink
        dev = q.device
        b, h, T = wl.batch, wl.heads, wl.seq_len
        self.q, self.k, self.v = q, k, v
        self.p = V.params_for(q, budget=wl.budget, n_sink=self.F, n_recent=wl.n_recent, scale=wl.scale,
                              indicator=wl.indicator, window=wl.window, norm=wl.norm, decode_overlap=decode_overlap)
        f32 = dict(dtype=torch.float32, device=dev)
        self.lse = torch.empty(b, h, T, **f32)
        self.attn_acc = torch.empty(b, h, T, **f32)
        self.vnorm = torch.empty(b, h, T, **f32)
        self.score = torch.empty(b, h, T, **f32)
        self.recompute_window = recompute_window and wl.indicator == "window"
        self.win_rows = torch.empty(b, h, wl.window, T, **f32) if wl.indicator == "window" and not self.recompute_window else None
        self.ws = torch.empty(max(V.vatp_workspace_bytes(self.p), 256), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.kept = torch.empty(b, h, wl.budget, dtype=torch.int32, device=dev)
        self.cache = V.Cache(self.p, device=dev)

    def run(self):
        V = vatp()
        if self.fused_forward:
            V.vatp_prefill_attention_scores(self.p, self.q, self.k, self.v, self.attn_out, lse_out=self.lse,
                                            attn_acc=self.attn_acc, vnorm=self.vnorm, score=self.score,
                                            win_rows=self.win_rows, workspace=self.ws, dev_status=self.status)
        elif self.lse_given:
            # the row normalisers arrive from outside, as from an attention forward that ran before
            self.lse_in = attention_forward_lse(self.q, self.k, self.wl.scale)
            V.vatp_prefill_scores_from_lse(self.p, self.q, self.k, self.v, self.lse_in, lse_out=self.lse,
                                           attn_acc=self.attn_acc, vnorm=self.vnorm, score=self.score,
                                           win_rows=self.win_rows, workspace=self.ws, dev_status=self.status)
        else:
            V.vatp_prefill_scores(self.p, self.q, self.k, self.v, lse_out=self.lse, attn_acc=self.attn_acc,
                                  vnorm=self.vnorm, score=self.score, win_rows=self.win_rows, workspace=self.ws,
                                  dev_status=self.status)
        V.vatp_select(self.p, self.score, self.kept, workspace=self.ws, dev_status=self.status)
        if self.recompute_window:
            V.vatp_compact_window(self.p, self.q, self.k, self.v, self.lse, self.attn_acc, self.vnorm, self.kept,
                                  self.cache, dev_status=self.status)
        else:
            V.vatp_compact(self.p, self.k, self.v, self.attn_acc, self.vnorm, self.kept, self.cache,
                           win_rows=self.win_rows, dev_status=self.status)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0, "device status word set"
        return self


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), ABS_FLOOR))) if ref.size else 0.0


def check_attention_output(got: np.ndarray, ref: np.ndarray, v: np.ndarray, dtype: str):
    """Rows of the attention output against the oracle's (Eq. 1).  fp32: 1e-5 of the largest value.  bf16: the
    probabilities are rounded to bf16 (relative 2^-9) before they meet V and the result is rounded to bf16
    again, so every element is within 2^-9 * sum_i a_i |v_i| + 2^-9 * |out| <= 2^-8 * max|v|; the typical error
    is an order of magnitude below that (independent roundings), and the mean error is held to a tenth of the bound."""
    vmax = float(np.abs(v).max())
    err = np.abs(got - ref)
    if dtype == "f32":
        assert err.max() <= 1e-5 * vmax, f"attention output: max err {err.max():.3g}"
    else:
        assert err.max() <= 2.0 ** -8 * vmax, f"attention output: max err {err.max():.3g} vs bound {2.0 ** -8 * vmax:.3g}"
        assert err.mean() <= 0.1 * 2.0 ** -8 * vmax, f"attention output: mean err {err.mean():.3g}"


def check_prefill_unit(g: GpuPrefill, b: int, h: int, tol: float):
    """Scores, kept set and compacted cache of one unit against the oracle.  Returns the oracle's
    prefill dict and the (validated) kept indices the GPU chose."""
    wl = g.wl
    T, B, F, R = wl.seq_len, wl.budget, g.F, wl.n_recent
    qn, kn, vn = (to_np64(x[b, h]) for x in (g.q, g.k, g.v))
    window = wl.window if wl.indicator == "window" else None
    ref = O.prefill(qn, kn, vn, wl.scale, window=window, norm=wl.norm)

    first = max(T - wl.window, 0) if window else 0
    lse = to_np64(g.lse[b, h])
    if g.fused_forward:
        first = 0                       # the forward normalises every row, inside the history window or not
        check_attention_output(to_np64(g.attn_out[b, h]), ref["out"], vn, wl.dtype)
    assert np.max(np.abs(lse[first:] - ref["lse"][first:])) <= tol * 10, "lse"
    for name, key in (("attn_acc", "S"), ("vnorm", "n1"), ("score", "I")):
        got = to_np64(getattr(g, name)[b, h])
        e = rel_err(got, ref[key])
        assert e <= tol, f"{name} rel err {e:.3g} > {tol} (unit {b},{h})"
    if window and g.win_rows is not None:
        rows = to_np64(g.win_rows[b, h])
        want = np.zeros_like(rows)
        n = ref["window_rows"].shape[0]
        want[wl.window - n:] = ref["window_rows"]
        assert np.max(np.abs(rows - want) - tol * np.abs(want)) <= 1e-30, "window rows"

    # kept set: exact except for scores within tol of the boundary score
    kept_gpu = g.kept[b, h].cpu().numpy().astype(np.int64)
    n_live = min(T, B)
    assert np.all(kept_gpu[n_live:] == -1)
    kept_gpu = kept_gpu[:n_live]
    assert np.all(np.diff(kept_gpu) > 0), "kept indices not strictly ascending"
    kept_ref = O.select_keep(ref["I"], B, F, R)
    assert len(kept_gpu) == len(kept_ref)
    sg, sr = set(kept_gpu.tolist()), set(kept_ref.tolist())
    assert set(range(min(F, T))) <= sg and set(range(max(T - R, 0), T)) <= sg
    n_boundary = 0
    if sg != sr:
        mid_kept = [i for i in kept_ref if F <= i < T - R]
        tau = ref["I"][mid_kept].min()
        for i in sg ^ sr:
            assert abs(ref["I"][i] - tau) <= tol * tau, f"index {i} differs and is not a boundary tie"
            n_boundary += 1

    # compaction: bit-exact gather at the GPU's indices, decode state initialised
    cache = g.cache
    idx = torch.from_numpy(kept_gpu).to(g.k.device)
    assert torch.equal(cache.k_cache[b, h, :n_live], g.k[b, h][idx]), "compacted K not bit-exact"
    assert torch.equal(cache.v_cache[b, h, :n_live], g.v[b, h][idx]), "compacted V not bit-exact"
    assert torch.equal(cache.pos[b, h, :n_live].cpu(), torch.from_numpy(kept_gpu).to(torch.int32))
    assert torch.all(cache.pos[b, h, n_live:] == -1)
    assert torch.equal(cache.vnorm[b, h, :n_live], g.vnorm[b, h][idx])
    if not window:
        assert torch.equal(cache.acc[b, h, :n_live], g.attn_acc[b, h][idx])
    else:
        # history ring: row (j mod w) holds the probabilities of query j on the kept tokens; exact window sums
        w = wl.window
        ring = to_np64(cache.ring[b, h])                      # [w, cap]
        want = np.zeros((w, n_live))
        rows_ref = ref["window_rows"]                         # rows of queries max(T - w, 0) .. T - 1
        j0 = T - rows_ref.shape[0]
        for r in range(rows_ref.shape[0]):
            want[(j0 + r) % w] = rows_ref[r][kept_gpu]
        assert np.max(np.abs(ring[:, :n_live] - want) - tol * np.abs(want)) <= 1e-30, "history ring"
        assert np.all(ring[:, n_live:] == 0)
        fixed = cache.acc_fixed[b, h, :n_live].cpu().numpy().astype(np.float64) / 2.0 ** 52
        assert rel_err(fixed, ref["S"][kept_gpu]) <= tol, "fixed-point window sums"
        assert rel_err(to_np64(cache.acc[b, h, :n_live]), ref["S"][kept_gpu]) <= tol
    assert int(cache.len[b, h]) == n_live and int(cache.next_pos[b, h]) == T and int(cache.free_slot[b, h]) == n_live
    if sg == sr:
        assert cache.k_cache[b, h, :n_live].cpu().view(torch.uint8).numpy().tobytes() == \
            O.compact_rows(g.k[b, h].cpu().view(torch.uint8).numpy().reshape(T, -1), kept_ref).tobytes()
    return ref, kept_gpu, n_boundary


def gpu_invariants(g: GpuPrefill):
    """Checks that need no oracle, on every unit."""
    wl = g.wl
    T, B, F, R = wl.seq_len, wl.budget, g.F, wl.n_recent
    rows = min(wl.window, T) if wl.indicator == "window" else T
    tot = g.attn_acc.double().sum(-1)
    assert torch.all((tot - rows).abs() <= 2e-3 * rows), f"sum of indicators != query rows: {tot.flatten()[:4]}"
    kept = g.kept.long()
    n_live = min(T, B)
    k = kept[..., :n_live]
    assert torch.all(k[..., 1:] > k[..., :-1])
    assert torch.all(k[..., : min(F, T)] == torch.arange(min(F, T), device=k.device))
    if R and T > B:
        assert torch.all(k[..., n_live - R:] == torch.arange(T - R, T, device=k.device))
    assert torch.all((k >= 0) & (k < T))


def run_decode_and_check(g: GpuPrefill, ref_by_unit: dict, dq, dk, dv, steps: int, tol: float,
                         check_state_every: int = 0):
    """Runs `steps` decode steps for all units on the GPU and the oracle on the listed units.
    ref_by_unit: {(b, h): (oracle prefill dict, kept indices)}.  Returns number of adopted ties."""
    V = vatp()
    wl = g.wl
    B, F, R = wl.budget, g.F, wl.n_recent
    window = wl.window if wl.indicator == "window" else None
    dev = g.q.device
    states = {}
    for (b, h), (ref, kept) in ref_by_unit.items():
        states[(b, h)] = O.DecodeState(to_np64(g.k[b, h]), to_np64(g.v[b, h]), ref["S"], ref["n1"], kept, wl.seq_len,
                                       window=window, window_rows=ref["window_rows"], norm=wl.norm)
    out = torch.empty(wl.batch, wl.heads, wl.head_dim, dtype=g.q.dtype, device=dev)
    evicted = torch.empty(wl.batch, wl.heads, dtype=torch.int32, device=dev)
    adopted = 0
    out_eps = 2.0 ** -8 if wl.dtype == "bf16" else 0.0     # round-to-nearest of `out` to bf16 (8 significant bits)
    for s in range(steps):
        V.vatp_decode_step(g.p, g.cache, dq[s], dk[s], dv[s], out, evicted_pos=evicted, dev_status=g.status)
        torch.cuda.synchronize()
        ev = evicted.cpu().numpy()
        out_c = to_np64(out)
        for (b, h), st in states.items():
            res = O.decode_step(st, to_np64(dq[s, b, h]), to_np64(dk[s, b, h]), to_np64(dv[s, b, h]), wl.scale, B, F, R,
                                force_evict=None if ev[b, h] < 0 else int(ev[b, h]), tie_tol=2 * tol, tie_abs=1e-30)
            assert res["evicted"] == ev[b, h], f"step {s} unit {(b, h)}: evicted {ev[b, h]} vs oracle {res['evicted']}"
            adopted += int(res["adopted"])
            ref_out = res["out"]
            bound = tol * np.max(np.abs(ref_out)) + out_eps * np.abs(ref_out) + 1e-30
            err = np.abs(out_c[b, h] - ref_out)
            assert np.all(err <= bound), f"step {s} unit {(b, h)}: out mismatch, worst err/bound {np.max(err / bound):.3g}"
        if check_state_every and ((s + 1) % check_state_every == 0 or s == steps - 1):
            check_decode_state(g, states, tol)
    assert int(g.status.item()) == 0
    return adopted


def check_decode_state(g: GpuPrefill, states: dict, tol: float):
    wl = g.wl
    for (b, h), st in states.items():
        pos = g.cache.pos[b, h].cpu().numpy()
        acc = to_np64(g.cache.acc[b, h])
        vn = to_np64(g.cache.vnorm[b, h])
        live = pos >= 0
        assert int(g.cache.len[b, h]) == live.sum() == len(st.pos)
        assert int(g.cache.next_pos[b, h]) == st.t
        order = np.argsort(pos[live])
        assert pos[live][order].tolist() == st.pos, "live positions differ"
        S_ref = st.indicator()
        # accumulated fp32 additions: one rounding per step on top of the prefill tolerance
        e = rel_err(acc[live][order], S_ref)
        assert e <= 2 * tol, f"indicator state rel err {e:.3g}"
        assert rel_err(vn[live][order], np.array(st.n1)) <= tol
        # cached rows are the original bits
        slot_of = {int(p): int(i) for i, p in enumerate(pos) if p >= 0}
        for p_chk in (st.pos[0], st.pos[len(st.pos) // 2], st.pos[-1]):
            row = to_np64(g.cache.k_cache[b, h, slot_of[p_chk]])
            assert np.array_equal(row, st.K[st.pos.index(p_chk)])
