#!/usr/bin/env python
"""Benchmark of the VATP hot path on B200: prefill score+prune tokens/s and decode us/layer-step.

One "step" = one pass of the whole path over one batch of synthetic input:
  for each layer: vatp_prefill_scores -> vatp_select -> vatp_compact      (score + prune)
  then `decode_steps` generation steps, each visiting every layer with vatp_decode_step.
The workload is config 1 (LLaMA2-7B layer shape: bf16, 32 heads, d 128, prompt 4096, budget 2048,
recent 128, 256 decode steps) held as LAYERS independently seeded layers, so that the decode
working set (LAYERS x 34.6 MB) does not sit in the 126 MB L2 between visits - as in a real model,
where the layers are visited in turn.

Prints ONE JSON line (rank 0).  `--impl reference` times the float64 CPU oracle on a bounded
sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "prefill_score_prune_tokens_per_s"
UNIT = "tokens/s"
LAYERS = 8


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------ reference arm
def oracle_sample(wl, units: int, decode_steps: int):
    """Times the oracle, as it stands, on `units` heads of layer 0 of the workload (prefill, select,
    compact and `decode_steps` generation steps).  Returns (seconds prefill+prune, seconds decode)."""
    import numpy as np
    from oracle import vatp_oracle as O
    from paper_2406_12335_b200 import synth
    sub = wl.with_(heads=units)
    q, k, v = (x.double().numpy() for x in synth.prefill_inputs(sub, 0, "cpu"))
    dq, dk, dv = (x.double().numpy() for x in synth.decode_inputs(sub, 0, decode_steps, "cpu"))
    t_pre = t_dec = 0.0
    window = wl.window if wl.indicator == "window" else None      # Eq. 3 instead of Eq. 2
    for h in range(units):
        t0 = time.perf_counter()
        r = O.prefill(q[0, h], k[0, h], v[0, h], wl.scale, window=window, norm=wl.norm)
        kept = O.select_keep(r["I"], wl.budget, wl.n_sink, wl.n_recent)
        O.compact_rows(k[0, h], kept); O.compact_rows(v[0, h], kept)
        st = O.DecodeState(k[0, h], v[0, h], r["S"], r["n1"], kept, wl.seq_len, window=window,
                           window_rows=r["window_rows"], norm=wl.norm)
        t1 = time.perf_counter()
        for s in range(decode_steps):
            O.decode_step(st, dq[s, 0, h], dk[s, 0, h], dv[s, 0, h], wl.scale, wl.budget, wl.n_sink, wl.n_recent)
        t2 = time.perf_counter()
        t_pre += t1 - t0
        t_dec += t2 - t1
        del r
    return t_pre, t_dec


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    units, dsteps = 2, 16
    for _ in range(args.warmup and 1):
        oracle_sample(wl, 1, 2)
    pre, dec = [], []
    for _ in range(args.steps):
        a, b = oracle_sample(wl, units, dsteps)
        pre.append(a); dec.append(b)
    t_unit = statistics.mean(pre) / units                       # seconds per (layer, head) unit
    all_units = wl.batch * wl.heads
    value = wl.batch * wl.seq_len / (t_unit * all_units)        # tokens/s of one layer, extrapolated from the sample
    dec_us = statistics.mean(dec) / (units * dsteps) * all_units * 1e6
    sample = (f"{units} of {all_units} heads of one layer, full prompt {wl.seq_len}, {dsteps} decode steps each; "
              f"per-layer figure extrapolated x{all_units // units}")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": (statistics.mean(pre) + statistics.mean(dec)) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config{wl.cid} {wl.name} (oracle on a sample)", "sample": sample},
            "decode_us_per_layer_step": dec_us,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(),
                             "kind": "oracle", "form": "float64 numpy, Python lists for the decode state", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ CUDA arm
def max_over_ranks(values, device, world: int):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return t.tolist()


def replica_throughput(units_per_rank: float, ms: float, world: int) -> float:
    """Whole-job units per second when every rank processes `units_per_rank` in `ms` (max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)


class LayerState:
    def __init__(self, V, wl, layer, dev, win_rows=False, kv_heads=0):
        from paper_2406_12335_b200 import synth
        if kv_heads:
            # grouped queries: K and V of kv_heads heads; the queries of a group lean towards their KV head's sinks
            wl_q, wl = wl, wl.with_(heads=kv_heads)
            _, self.k, self.v = synth.prefill_inputs(wl, layer, dev)
            G = wl_q.heads // kv_heads
            u = synth.sink_direction(wl, layer, dev).repeat_interleave(G, dim=1)
            gq = torch.Generator(device=dev).manual_seed(977 + layer)
            shape = (wl_q.batch, wl_q.heads, wl_q.seq_len, wl_q.head_dim)
            self.q = (torch.randn(shape, generator=gq, device=dev) + synth.sink_alpha(wl) * u).to(self.k.dtype)
            self.p = V.make_params(batch=wl_q.batch, heads=wl_q.heads, kv_heads=kv_heads, seq_len=wl.seq_len,
                                   head_dim=wl.head_dim, dtype=wl.dtype, budget=wl.budget, n_sink=wl.n_sink,
                                   n_recent=wl.n_recent, scale=wl.scale, indicator=wl.indicator, window=wl.window,
                                   norm=wl.norm, decode_overlap=True)
        else:
            self.q, self.k, self.v = synth.prefill_inputs(wl, layer, dev)
            self.p = V.params_for(self.q, budget=wl.budget, n_sink=wl.n_sink, n_recent=wl.n_recent, scale=wl.scale,
                                  indicator=wl.indicator, window=wl.window, norm=wl.norm, decode_overlap=True)
        # the same parameters without the opt-in: every decode step then waits for all earlier work in the stream
        self.p_wait = type(self.p).from_buffer_copy(self.p)
        self.p_wait.flags = 0
        b, h, T = wl.batch, wl.heads, wl.seq_len
        f32 = dict(dtype=torch.float32, device=dev)
        self.attn_acc = torch.empty(b, h, T, **f32)
        self.vnorm = torch.empty(b, h, T, **f32)
        self.score = torch.empty(b, h, T, **f32)
        self.lse = torch.empty(b, self.q.shape[1], T, **f32)      # one normaliser row per query head
        # Eq. 3: by default the history of the kept tokens is rebuilt by vatp_compact_window; --win-rows times the
        # variant in which the scoring call writes all w x T probabilities and vatp_compact gathers from them
        self.win_rows = torch.empty(b, h, wl.window, T, **f32) if wl.indicator == "window" and win_rows else None
        self.kept = torch.empty(b, h, wl.budget, dtype=torch.int32, device=dev)
        self.ws = torch.empty(max(V.vatp_workspace_bytes(self.p), 256), dtype=torch.uint8, device=dev)
        self.cache = V.Cache(self.p, device=dev)
        self.dq, self.dk, self.dv = synth.decode_inputs(wl, layer, device=dev)
        if kv_heads:
            self.dq = (torch.randn((wl.decode_steps,) + shape[:2] + shape[3:], generator=gq, device=dev)
                       + synth.sink_alpha(wl) * u.squeeze(2)).to(self.k.dtype)
        self.out = torch.empty(wl.decode_steps, b, self.q.shape[1], wl.head_dim, dtype=self.q.dtype, device=dev)
        self.evicted = torch.empty(wl.decode_steps, b, h, dtype=torch.int32, device=dev)


def prune_launches(wl, args):
    """Kernels of this library that one layer's scoring + selection + compaction launches (memsets not counted)."""
    windowed = wl.indicator == "window"
    tensor_core = wl.dtype == "bf16" and wl.head_dim == 128
    if tensor_core:
        # Eq. 2 with the l1 norm: counter reset, pass 1 (value norms on its side warp), pass 2;
        # otherwise: norm kernel, pass 1 unless the normalisers are given, pass 2
        scoring = 2 if args.lse_given else 3
    else:
        scoring = 1 if args.lse_given else 2       # row statistics, column sums
    compaction = 2 if windowed else 1              # gather, then the window history (rebuilt or gathered)
    if args.kv_heads and args.kv_heads < wl.heads:
        # tensor cores: one launch over all query heads; general kernels: once per query head of the groups; then the group mean
        scoring = (scoring if tensor_core else scoring * (wl.heads // args.kv_heads)) + 1
    return scoring + 1 + compaction


def run_cuda(args, wl):
    from paper_2406_12335_b200 import build as _b
    _b.build()
    from paper_2406_12335_b200 import vatp as V      # raises if libvatp.so is missing: no fallback

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    L, steps_dec = args.layers, wl.decode_steps
    layers = [LayerState(V, wl, l, dev, win_rows=args.win_rows, kv_heads=args.kv_heads) for l in range(L)]
    windowed = wl.indicator == "window"

    def compact(ls):
        if windowed and ls.win_rows is None:
            V.vatp_compact_window(ls.p, ls.q, ls.k, ls.v, ls.lse, ls.attn_acc, ls.vnorm, ls.kept, ls.cache, dev_status=status)
        else:
            V.vatp_compact(ls.p, ls.k, ls.v, ls.attn_acc, ls.vnorm, ls.kept, ls.cache, win_rows=ls.win_rows, dev_status=status)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    lse_given, fill_lse = [False], [True]   # the first call below fills every layer's lse; --lse-given then times pass 2 alone
    # the fused call (attention output + scoring) is timed in a region of its own; one output buffer serves every layer
    fused = [False]
    attn_out = torch.empty_like(layers[0].q)

    def prefill_all(ev=None, parts=(True, True, True)):
        """parts: which of (scoring, selection, compaction) to issue for every layer."""
        for i, ls in enumerate(layers):
            if not parts[0]:
                if parts[1]: V.vatp_select(ls.p, ls.score, ls.kept, dev_status=status)
                if parts[2]: compact(ls)
                continue
            if ev: ev[i][0].record()
            if fused[0]:
                V.vatp_prefill_attention_scores(ls.p, ls.q, ls.k, ls.v, attn_out, lse_out=ls.lse if windowed else None,
                                                attn_acc=ls.attn_acc, vnorm=ls.vnorm, score=ls.score, win_rows=ls.win_rows,
                                                workspace=ls.ws, dev_status=status)
            elif lse_given[0]:
                V.vatp_prefill_scores_from_lse(ls.p, ls.q, ls.k, ls.v, ls.lse, attn_acc=ls.attn_acc, vnorm=ls.vnorm,
                                               score=ls.score, win_rows=ls.win_rows, workspace=ls.ws, dev_status=status)
            else:
                V.vatp_prefill_scores(ls.p, ls.q, ls.k, ls.v, lse_out=ls.lse if (fill_lse[0] or windowed) else None,
                                      attn_acc=ls.attn_acc, vnorm=ls.vnorm, score=ls.score, win_rows=ls.win_rows,
                                      workspace=ls.ws, dev_status=status)
            if ev: ev[i][1].record()
            if not parts[1]: continue
            V.vatp_select(ls.p, ls.score, ls.kept, dev_status=status)
            if ev: ev[i][2].record()
            if not parts[2]: continue
            compact(ls)
            if ev: ev[i][3].record()

    def decode_all(overlap=True):
        for s in range(steps_dec):
            for ls in layers:
                V.vatp_decode_step(ls.p if overlap else ls.p_wait, ls.cache, ls.dq[s], ls.dk[s], ls.dv[s], ls.out[s],
                                   evicted_pos=ls.evicted[s], dev_status=status)

    # warm up once outside any capture (first calls set kernel attributes), then capture the
    # launch-bound decode loop in a CUDA graph
    prefill_all(); decode_all(); torch.cuda.synchronize()
    lse_given[0], fill_lse[0] = args.lse_given, False
    graph = graph_wait = None
    if not args.no_graph:
        prefill_all(); torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            decode_all()
        torch.cuda.synchronize()
        graph_wait = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_wait):
            decode_all(overlap=False)
        torch.cuda.synchronize()

    def run_decode():
        if graph is not None:
            graph.replay()
        else:
            decode_all()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    E = lambda: torch.cuda.Event(enable_timing=True)

    def one_step(per_kernel_events):
        """One step.  The timed steps record three events only: an event between two kernels would break
        the programmatic dependency that lets a launch set up while its predecessor drains."""
        flush.fill_(rank + 1)                       # evict L2 between iterations
        ev = [[E() for _ in range(4)] for _ in range(L)] if per_kernel_events else None
        e0, e1, e2 = E(), E(), E()
        e0.record()
        prefill_all(ev)
        e1.record()
        run_decode()
        e2.record()
        return e0, e1, e2, ev

    for _ in range(args.warmup):
        one_step(False)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    recs = [one_step(False) for _ in range(args.steps)]
    barrier()
    clocks = sampler.stop()
    # per-kernel breakdown of the prefill side: a few extra steps with an event after every call
    brk = [one_step(True) for _ in range(max(2, min(args.steps, 5)))]
    barrier()

    # The same breakdown without events between the calls.  Selection and compaction are programmatic dependents of
    # the launch before them (they set up while it drains); an event between two calls breaks that and adds a full
    # launch latency to each.  Here CUDA events bracket a region of back-to-back calls over all layers: scoring calls
    # only; selection calls only; selection + compaction.  Compaction's cost is the last minus the one before.
    def chain_ms(parts):
        flush.fill_(rank + 1)
        a, b = E(), E()
        a.record(); prefill_all(parts=parts); b.record()
        return a, b

    chain = {}
    for key, parts in (("score", (True, False, False)), ("select", (False, True, False)), ("select+compact", (False, True, True))):
        chain_ms(parts)
        recs_c = [chain_ms(parts) for _ in range(max(3, min(args.steps, 6)))]
        barrier()
        chain[key] = statistics.median(a.elapsed_time(b) for a, b in recs_c) / L       # ms per layer
    # the fused call in the scoring call's place: attention output rows, normalisers, indicator, norms, scores
    fused[0] = True
    chain_ms((True, False, False)); barrier()
    recs_c = [chain_ms((True, False, False)) for _ in range(max(3, min(args.steps, 6)))]
    barrier()
    chain["score_fused"] = statistics.median(a.elapsed_time(b) for a, b in recs_c) / L
    fused[0] = False
    prefill_all(); barrier()     # leave complete caches behind

    # the same decode steps with every launch waiting for all earlier work in the stream (no opt-in to
    # overlapping launches): what a chain of dependent steps costs - in a model, layer l + 1's q/k/v come
    # from layer l's output
    def wait_step():
        flush.fill_(rank + 1)
        prefill_all()
        e1, e2 = E(), E()
        e1.record()
        if graph_wait is not None:
            graph_wait.replay()
        else:
            decode_all(overlap=False)
        e2.record()
        return e1, e2

    wait_step()
    wrecs = [wait_step() for _ in range(max(2, min(args.steps, 5)))]
    barrier()
    dec_wait_ms = max_over_ranks([statistics.mean(a.elapsed_time(b) for a, b in wrecs)], dev, world)[0]
    assert int(status.item()) == 0, "device status word set"

    t_pre = [a.elapsed_time(b) for a, b, _, _ in recs]               # ms, all layers
    t_dec = [b.elapsed_time(c) for _, b, c, _ in recs]
    t_all = [a.elapsed_time(c) for a, _, c, _ in recs]
    t_score = [sum(e[0].elapsed_time(e[1]) for e in r[3]) / L for r in brk]     # ms per layer
    t_select = [sum(e[1].elapsed_time(e[2]) for e in r[3]) / L for r in brk]
    t_compact = [sum(e[2].elapsed_time(e[3]) for e in r[3]) / L for r in brk]
    pre_ms, dec_ms, all_ms = (x / args.steps for x in max_over_ranks([sum(t_pre), sum(t_dec), sum(t_all)], dev, world))

    # ---- end to end through the public API with host buffers (pinned), copies inside the timed region
    host = None if args.no_e2e else [[x.cpu().pin_memory() for x in (ls.q, ls.k, ls.v, ls.dq, ls.dk, ls.dv)] for ls in layers]
    host_kept = [torch.empty_like(ls.kept, device="cpu").pin_memory() for ls in layers]
    host_out = [torch.empty_like(ls.out, device="cpu").pin_memory() for ls in layers]
    h2d = sum(x.numel() * x.element_size() for hl in (host or []) for x in hl)
    d2h = sum(x.numel() * x.element_size() for x in host_kept + host_out)

    def e2e_step():
        flush.fill_(3)
        e0, e1, e2 = E(), E(), E()
        e0.record()
        for ls, hl in zip(layers, host):
            for dst, src in zip((ls.q, ls.k, ls.v, ls.dq, ls.dk, ls.dv), hl):
                dst.copy_(src, non_blocking=True)
        prefill_all()
        for ls, hk in zip(layers, host_kept):
            hk.copy_(ls.kept, non_blocking=True)
        e1.record()
        run_decode()
        for ls, ho in zip(layers, host_out):
            ho.copy_(ls.out, non_blocking=True)
        e2.record()
        return e0, e1, e2

    if host is not None:
        e2e_step(); barrier()
        e2e_recs = [e2e_step() for _ in range(max(2, min(args.steps, 5)))]
        barrier()
        e2e_pre_ms = max_over_ranks([statistics.mean(a.elapsed_time(b) for a, b, _ in e2e_recs)], dev, world)[0]
        e2e_dec_ms = statistics.mean(b.elapsed_time(c) for _, b, c in e2e_recs)

    if rank != 0:
        return
    q_units = wl.batch * wl.heads                              # scoring sweeps run once per query head
    units = wl.batch * (args.kv_heads or wl.heads)             # kept sets, caches and decode states: one per KV head
    T, d, B = wl.seq_len, wl.head_dim, wl.budget
    tokens = wl.batch * T * L                                  # layer-tokens scored and pruned per step
    value = replica_throughput(tokens, pre_ms, world)
    dec_us = dec_ms * 1e3 / (steps_dec * L)
    dec_wait_us = dec_wait_ms * 1e3 / (steps_dec * L)

    # ---- rooflines (algorithmic work only) ----
    if wl.indicator == "window":                               # only the last w query rows (Eq. 3)
        w = min(wl.window, T)
        pairs = w * T - w * (w - 1) / 2
    else:
        pairs = T * (T + 1) / 2
    passes = 1 if args.lse_given else 2
    flops_score = passes * (2.0 * d) * pairs * q_units         # each pass recomputes the causal part of QK^T
    # fused call: the forward's two contractions over every causal pair, then pass 2's one
    flops_fused = (2 * (2.0 * d) * (T * (T + 1) / 2) + (2.0 * d) * pairs) * q_units
    bytes_compact = units * (2 * 2 * B * d * 2 + 12 * B)       # K,V rows read + written, 12 B of state per slot
    if wl.indicator == "window":
        # history ring written; with --win-rows the kept columns of the last-w rows are read too
        bytes_compact += units * (2 if args.win_rows else 1) * 4 * B * min(wl.window, T)
    bytes_decode = units * (B + 1) * (2 * d * 2 + 16 + (8 if wl.indicator == "window" else 0))  # K,V rows once, acc r+w, vnorm, pos (+ ring row r+w)
    bytes_select = units * (4 * T + 4 * B)
    ms = statistics.mean
    t_score_c, t_select_c = chain["score"], chain["select"]                       # ms per layer, back-to-back calls
    t_compact_c = chain["select+compact"] - chain["select"]
    kernels = {
        "prefill_scores": {"bound": "tensor", "achieved": flops_score / (t_score_c * 1e-3) / 1e12,
                           "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "ms_per_launch_pair": t_score_c,
                           "ms_isolated": ms(t_score), "achieved_isolated": flops_score / (ms(t_score) * 1e-3) / 1e12},
        # vatp_prefill_attention_scores in the scoring call's place (not part of the timed step): three contraction sweeps
        "attention_forward_scores": {"bound": "tensor", "achieved": flops_fused / (chain["score_fused"] * 1e-3) / 1e12,
                                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "ms_per_call": chain["score_fused"]},
        "select": {"bound": "hbm", "achieved": bytes_select / (t_select_c * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                   "unit": "GB/s", "us_per_launch": t_select_c * 1e3,
                   "us_isolated": ms(t_select) * 1e3, "achieved_isolated": bytes_select / (ms(t_select) * 1e-3) / 1e9},
        "compact": {"bound": "hbm", "achieved": bytes_compact / (t_compact_c * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "us_per_launch": t_compact_c * 1e3,
                    "us_isolated": ms(t_compact) * 1e3, "achieved_isolated": bytes_compact / (ms(t_compact) * 1e-3) / 1e9},
        "decode_step": {"bound": "hbm", "achieved": bytes_decode / (dec_us * 1e-6) / 1e9, "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "us_per_launch": dec_us,
                        "launches": f"steps of {L} independent layer caches in rotation, overlap flag set: consecutive launches run side by side"},
        # same steps, every launch waiting for all earlier work in the stream (the default of vatp_decode_step)
        "decode_step_dependent": {"bound": "hbm", "achieved": bytes_decode / (dec_wait_us * 1e-6) / 1e9,
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s", "us_per_launch": dec_wait_us},
    }
    for kd in kernels.values():
        kd["frac"] = kd["achieved"] / kd["peak"]
        if "achieved_isolated" in kd:
            kd["frac_isolated"] = kd["achieved_isolated"] / kd["peak"]
        kd["peak_source"] = peaks["source"]
    timing_note = ("prefill-side calls: CUDA events over a region of back-to-back calls over all layers, per layer "
                   "(scoring calls only; selection calls only; compaction = the region of selection + compaction calls "
                   "minus the region of selection calls: both are programmatic dependents of the launch before them and "
                   "set up while it drains).  *_isolated: CUDA events around every single call of a whole prefill chain "
                   "instead; an event between two calls breaks that overlap and costs each call a full launch latency")
    share = {"prefill_scores": t_score_c * L, "select": t_select_c * L, "compact": t_compact_c * L,
             "decode_step": dec_ms}          # (decode_step_dependent is an extra measurement, not part of the timed step)
    dominant = max(share, key=share.get)
    roof = dict(kernels[dominant])
    roof["kernel"] = dominant
    # dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu capture of this kernel at
    # this shape (profiles/); other kernels / shapes: not captured
    roof["traffic"] = 34.54e6 if (dominant == "decode_step" and wl.cid == 1) else None
    roof["traffic_source"] = ("ncu capture of this kernel at this shape, summarised in profiles/decode_mma_config1.md "
                              "(not measured in this run)") if roof["traffic"] else None
    roof["algorithmic_bytes_per_launch"] = bytes_decode if dominant == "decode_step" else None
    roof["time_share"] = share[dominant] / sum(share.values())

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": all_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": f"config{wl.cid} {wl.name}: b{wl.batch} h{wl.heads} d{d} T{T} budget{B} recent{wl.n_recent} "
                               f"sinkF{wl.n_sink} {wl.indicator}, {steps_dec} decode steps, x{L} independently seeded layers",
                   "layers": L,
                   **({"kv_heads": args.kv_heads, "grouped_queries": f"{wl.heads // args.kv_heads} query heads share each KV "
                       "head (group-mean indicator): scoring runs per query head, selection / compaction / decode per KV head"}
                      if args.kv_heads else {}),
                   "l2": f"256 MB flush write between steps; layer rotation over {L} decode states ({L * bytes_decode / 1e6:.0f} MB per visit of all layers)",
                   "replicas": "each GPU runs the whole workload (path does not shard within a call)",
                   "decode_graph": graph is not None},
        "prefill_ms_per_layer": pre_ms / L, "decode_us_per_layer_step": dec_us,
        "decode_us_per_layer_step_dependent": dec_wait_us,
        "roofline": roof, "roofline_all": kernels, "roofline_all_timing": timing_note,
        "e2e": None if host is None else
               {"value": replica_throughput(tokens, e2e_pre_ms, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "decode_us_per_layer_step": e2e_dec_ms * 1e3 / (steps_dec * L)},
        "gpu_launches": args.steps * L * (prune_launches(wl, args) + steps_dec),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        cu, cs = 24, 64      # about 10-20 s of CPU work
        a, b = oracle_sample(wl, cu, cs)
        v = wl.batch * T / (a / cu * units)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "form": "float64 numpy, Python lists for the decode state",
                                "sample": f"{cu} of {units} heads of one layer (full prompt {T}, {cs} decode steps), "
                                          f"{a + b:.1f} s of CPU work, per-layer figure extrapolated x{units / cu:.2f}",
                                "decode_us_per_layer_step": b / (cu * cs) * units * 1e6}
    print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch decode steps directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--win-rows", action="store_true",
                    help="history-window workloads: let the scoring call write all w x T probabilities and gather the "
                         "kept columns from them (vatp_compact) instead of rebuilding them (vatp_compact_window)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--layers", type=int, default=LAYERS, help="independently seeded layers held on the device")
    ap.add_argument("--config", type=int, default=1, choices=sorted([0, 1, 2, 3, 4, 5]),
                    help="workload to time; 1 is the benchmark, the others are for the per-config roofline tables "
                         "(choose --layers so that the inputs fit: config 2 and 4 hold 1.6 GB per layer, config 5 "
                         "6.3 GB); 5 is the shape of the paper's throughput table (batch 12, prompt 4096, 128 steps)")
    ap.add_argument("--budget-ratio", type=float, default=None,
                    help="KV budget as a fraction of the prompt (the throughput table's 1.0 / 0.5 / 0.25), split as "
                         "Appendix A states for --method")
    ap.add_argument("--method", default=None, choices=["h2o", "scissorhands"],
                    help="host method whose Appendix A split --budget-ratio applies (default: the workload's indicator)")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workload's decode steps (profiling runs)")
    ap.add_argument("--lse-given", action="store_true",
                    help="time vatp_prefill_scores_from_lse: the row normalisers come from an earlier attention forward "
                         "(here: from the warm-up's two-pass call), so scoring is one recomputation of QK^T")
    ap.add_argument("--kv-heads", type=int, default=0,
                    help="grouped-query attention: the workload's heads become query heads that share this many KV heads "
                         "(the Limitations section's open case, read as a group-mean indicator); CUDA arm only")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size")
    ap.add_argument("--norm", default="l1", choices=["l1", "l2", "linf"],
                    help="value norm of Eq. 4: l1 is the method (and the benchmark), l2 / linf the Ablation Study's variants")
    args = ap.parse_args()
    from paper_2406_12335_b200 import synth
    wl = synth.CONFIGS[args.config]
    if args.decode_steps is not None:
        wl = wl.with_(decode_steps=args.decode_steps)
    if args.budget_ratio is not None:
        from paper_2406_12335_b200 import presets
        method = args.method or ("scissorhands" if wl.indicator == "window" else "h2o")
        pr = presets.appendix_a(method, wl.seq_len, args.budget_ratio)
        wl = wl.with_(budget=pr["budget"], n_sink=pr["n_sink"], n_recent=pr["n_recent"], indicator=pr["indicator"],
                      window=pr["window"], name=f"{wl.name} {method} budget {args.budget_ratio:g}")
    if args.batch is not None:
        wl = wl.with_(batch=args.batch, name=f"{wl.name} batch {args.batch}")
    if args.kv_heads:
        if wl.heads % args.kv_heads or args.impl == "reference":
            ap.error("--kv-heads must divide the workload's heads and applies to the CUDA arm only")
        wl = wl.with_(name=f"{wl.name} {args.kv_heads} kv heads")
        args.no_cpu_baseline = True          # the sampled oracle baseline is defined for the multi-head workloads
    if args.norm != "l1":
        wl = wl.with_(norm=args.norm, name=f"{wl.name} norm={args.norm}")
    if args.lse_given:
        wl = wl.with_(name=f"{wl.name} lse given")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
