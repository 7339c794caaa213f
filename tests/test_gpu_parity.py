"""GPU parity: the CUDA path through the C ABI against the float64 oracle, element by element,
on the same seeded inputs.  Tolerances: scores 1e-5 relative for fp32 inputs, 1e-3 for bf16;
kept sets exact except for scores within that tolerance of the boundary score; compacted K/V
bit-exact."""
import numpy as np
import pytest
import torch

from paper_2406_12335_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


def _small(dtype, d, T, B, F, R, b=1, h=2, indicator="h2o", window=0, steps=0, cid=90):
    return synth.Workload(cid, f"case_T{T}", dtype, b, h, 1, d, T, B, F, R, indicator, window, steps)


# What the comparison is allowed to forgive, per oracle unit: kept indices that differ from the oracle's only
# because their score lies within the tolerance of the boundary score, and decode steps where the GPU evicted the
# oracle's runner-up because the two importances lie within twice the tolerance of each other (the oracle then
# follows the GPU).  Both are counted, printed and bounded: a handful per unit is arithmetic, more would be a bug.
MAX_BOUNDARY_PER_UNIT = 6


def _max_adopted(steps, n_units):
    return n_units * (2 + steps // 32)


def _run_case(wl, n_sink=None, decode=True, units=None, check_state_every=4, layer=0, lse_given=False,
              decode_units=None, recompute_window=False, fused_forward=False):
    """units: the units the oracle checks at prefill (default: all); decode_units: those of them whose decode
    trajectory it follows (default: all of `units`)."""
    q, k, v = synth.prefill_inputs(wl, layer, "cuda")
    g = P.GpuPrefill(wl, q, k, v, n_sink=n_sink, lse_given=lse_given, recompute_window=recompute_window,
                     fused_forward=fused_forward).run()
    P.gpu_invariants(g)
    tol = P.TOL[wl.dtype]
    units = units or [(b, h) for b in range(wl.batch) for h in range(wl.heads)]
    decode_units = units if decode_units is None else decode_units
    refs, nb = {}, 0
    for (b, h) in units:
        ref, kept, n_boundary = P.check_prefill_unit(g, b, h, tol)
        ref.pop("a")                     # the T x T matrix (8.6 GB at T = 32768) is not needed beyond this point
        if (b, h) in decode_units:
            refs[(b, h)] = (ref, kept)
        assert n_boundary <= MAX_BOUNDARY_PER_UNIT, f"unit {(b, h)}: {n_boundary} kept indices differ from the oracle's"
        nb += n_boundary
        del ref
    adopted = 0
    if decode and wl.decode_steps and refs:
        dq, dk, dv = synth.decode_inputs(wl, layer, device="cuda")
        adopted = P.run_decode_and_check(g, refs, dq, dk, dv, wl.decode_steps, tol, check_state_every)
        assert adopted <= _max_adopted(wl.decode_steps, len(refs)), f"{adopted} near-tie evictions adopted"
    print(f"[parity] {wl.name} layer {layer}: {len(units)} oracle units, {nb} boundary indices tolerated, "
          f"{len(refs)} decode units x {wl.decode_steps if decode else 0} steps, {adopted} near-tie evictions adopted")
    return g, nb, adopted


def test_config0_fp32_tiny():
    """Config 0: fp32, 2 heads, d 64, T 512, budget 256, recent 32, 16 decode steps."""
    _run_case(synth.CONFIGS[0])


@pytest.mark.parametrize("F", [2, 20])
def test_config0_with_sink_retention(F):
    g, _, _ = _run_case(synth.CONFIGS[0], n_sink=F)
    assert torch.all(g.kept[..., :F].cpu() == torch.arange(F))


@pytest.mark.parametrize("dtype,d,T,B,F,R", [
    ("f32", 64, 333, 100, 3, 17),      # ragged tail, several 64-tiles
    ("f32", 128, 200, 64, 0, 8),
    ("bf16", 64, 257, 128, 2, 16),
    ("bf16", 128, 1000, 300, 4, 50),   # ragged against 64- and 128-tiles
    ("bf16", 128, 130, 65, 1, 1),
    ("f32", 64, 40, 20, 2, 3),         # shorter than one tile
])
def test_ragged_shapes(dtype, d, T, B, F, R):
    _run_case(_small(dtype, d, T, B, F, R, steps=6))


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("bf16", 128)])
def test_degenerate_budgets(dtype, d):
    # budget = F + R: sinks and window only, whatever the scores
    wl = _small(dtype, d, 300, 24, 8, 16, steps=5)
    g, _, _ = _run_case(wl)
    assert g.kept[0, 0].cpu().tolist() == list(range(8)) + list(range(284, 300))
    # budget >= T: every token kept, cache grows before evictions start
    wl = _small(dtype, d, 100, 103, 2, 5, steps=8)
    g, _, _ = _run_case(wl)
    assert int(g.cache.len[0, 0]) == 103
    # T == B exactly
    _run_case(_small(dtype, d, 96, 96, 0, 0, steps=3))
    # no recent window and no sinks
    _run_case(_small(dtype, d, 150, 50, 0, 0, steps=4))


@pytest.mark.parametrize("T,B,heads", [
    (5000, 1200, 3),        # one CTA per unit
    (20000, 5000, 3),       # long prompt, 6 units: the range of a unit split over a cluster of four CTAs
    (9000, 4000, 25),       # 50 units: clusters of two
    (8300, 8250, 3),        # all but a handful survive
])
def test_exact_ties_prefer_lower_index(T, B, heads):
    """select on hand-made scores with many exact ties (integer work: bit-exact)."""
    V = P.vatp()
    F, R = 3, 100
    rng = np.random.default_rng(0)
    score = torch.from_numpy(rng.integers(0, 7, size=(2, heads, T)).astype(np.float32)).cuda()
    p = V.make_params(batch=2, heads=heads, seq_len=T, head_dim=64, dtype="f32", budget=B, n_sink=F, n_recent=R)
    kept = torch.empty(2, heads, B, dtype=torch.int32, device="cuda")
    V.vatp_select(p, score, kept)
    torch.cuda.synchronize()
    from oracle import vatp_oracle as O
    for b in range(2):
        for h in (0, 1, heads - 1):
            want = O.select_keep(score[b, h].cpu().numpy(), B, F, R)
            assert kept[b, h].cpu().numpy().tolist() == want.tolist()


def test_select_large_T_unstaged_path():
    """T beyond what one CTA can stage in shared memory."""
    V = P.vatp()
    T, B, F, R = 70000, 7000, 20, 512
    g = torch.Generator(device="cuda").manual_seed(5)
    for heads in (80, 2):                  # many units: one CTA each, keys read from global memory; two units: clusters of four
        score = torch.rand(1, heads, T, generator=g, device="cuda")
        score[0, 0, 1000:1100] = 0.5          # a run of ties
        p = V.make_params(batch=1, heads=heads, seq_len=T, head_dim=128, dtype="bf16", budget=B, n_sink=F, n_recent=R)
        kept = torch.empty(1, heads, B, dtype=torch.int32, device="cuda")
        V.vatp_select(p, score, kept)
        torch.cuda.synchronize()
        from oracle import vatp_oracle as O
        for h in (0, heads - 1):
            want = O.select_keep(score[0, h].cpu().numpy(), B, F, R)
            assert kept[0, h].cpu().numpy().tolist() == want.tolist()


def test_strided_inputs():
    """q/k/v as [b, T, h, d] storage viewed as [b, h, T, d] (non-contiguous token stride)."""
    wl = _small("bf16", 128, 300, 100, 2, 10, b=2, h=3)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    qs, ks, vs = (x.transpose(1, 2).contiguous().transpose(1, 2) for x in (q, k, v))
    assert not qs.is_contiguous()
    g1 = P.GpuPrefill(wl, q, k, v).run()
    g2 = P.GpuPrefill(wl, qs, ks, vs).run()
    assert torch.equal(g1.score, g2.score) and torch.equal(g1.kept, g2.kept)
    assert torch.equal(g1.cache.k_cache, g2.cache.k_cache) and torch.equal(g1.cache.v_cache, g2.cache.v_cache)


def test_run_to_run_determinism():
    # enough (unit, tile) items that the CTAs draw them in a different order every run
    wl = _small("bf16", 128, 700, 200, 2, 20, b=2, h=100)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    a = P.GpuPrefill(wl, q, k, v).run()
    b = P.GpuPrefill(wl, q, k, v).run()
    assert torch.equal(a.score, b.score) and torch.equal(a.kept, b.kept)


def test_config1_llama_layer():
    """Config 1: bf16, 32 heads, d 128, T 4096, budget 2048, recent 128; 256 decode steps on a
    sample of heads (the oracle's python loop is the limit), invariants on all heads."""
    wl = synth.CONFIGS[1]
    _run_case(wl, units=[(0, 0), (0, 13), (0, 31)], check_state_every=64)


@pytest.mark.parametrize("F", [0, 2, 20])
def test_config1_prefill_all_heads(F):
    """Config 1 at its full size, every head against the oracle, without kept leading tokens (the config as
    written) and with F = 2 and F = 20 (the paper's value for LLaMA2-7B-chat)."""
    wl = synth.CONFIGS[1].with_(decode_steps=0)
    g, _, _ = _run_case(wl, decode=False, n_sink=F)
    assert torch.all(g.kept[..., :F].cpu() == torch.arange(F))


def test_config1_decode_with_sink_retention():
    """Config 1 with the first 20 tokens kept: decode trajectories of sampled heads (the low-norm sink tokens
    must never be released)."""
    wl = synth.CONFIGS[1].with_(decode_steps=96)
    g, _, _ = _run_case(wl, n_sink=20, units=[(0, 3), (0, 28)], check_state_every=32)
    assert torch.all(g.cache.pos[0, :, :20].cpu() == torch.arange(20))


@pytest.mark.parametrize("layer,units", [(0, [(0, 0), (7, 31), (4, 9)]), (15, [(1, 30), (6, 4), (2, 16)]),
                                         (31, [(3, 17), (5, 2), (0, 22)])])
def test_config2_stack_layer(layer, units):
    """Config 2 at its full per-layer size (batch 8, 32 heads, T 8192, budget 1638, recent 256; the
    value-norm spread grows with the layer: sigma 0.5, 0.98 and 1.5 here): first, middle and last layer,
    the oracle on nine sampled units in all (prefill; 128 decode steps on two of each layer's three),
    oracle-free invariants on all 256 units of each layer."""
    _run_case(synth.CONFIGS[2], units=units, decode_units=units[:2], check_state_every=64, layer=layer)


@pytest.mark.parametrize("recompute", [True, False])
def test_config3_windowed(recompute):
    """Config 3 at full size: last-256-queries indicator (Eq. 3), batch 16, 32 heads, T 2048, budget
    1024, 512 decode steps with the cache held at budget; oracle on sampled units.  Once with the history
    rebuilt from Q and the kept keys (no win_rows), once through win_rows."""
    _run_case(synth.CONFIGS[3], units=[(0, 0), (9, 14), (15, 31)], check_state_every=128, recompute_window=recompute)


@pytest.mark.parametrize("layer,units", [(0, [(0, 0), (0, 19)]), (31, [(0, 5), (0, 30)])])
def test_config4_long_context_layer(layer, units):
    """Config 4 at full size: T 32768, budget 3277, recent 512, 64 boosted-norm tokens per layer.  The
    oracle materialises the 32768 x 32768 matrix (8.6 GB in float64), one unit at a time: two units of
    the first and two of the last layer (64 decode steps on one of each pair); every other unit of those
    layers is covered by the invariants."""
    _run_case(synth.CONFIGS[4], units=units, decode_units=units[:1], check_state_every=32, layer=layer)


@pytest.mark.parametrize("cid,layer", [(4, 16), (2, 23)])
def test_stack_middle_layers_invariants(cid, layer):
    """Oracle-free checks on every unit of further layers of the 32-layer configs: indicators sum to the
    number of query rows, kept counts, kept leading and recent tokens, ascending order."""
    wl = synth.CONFIGS[cid]
    q, k, v = synth.prefill_inputs(wl, layer, "cuda")
    P.gpu_invariants(P.GpuPrefill(wl, q, k, v).run())


def _interleaved_equals_alone(wls, steps, overlap=True):
    """Steps the caches of `wls` (a) one after the other, each alone with a synchronisation after every
    step, and (b) round robin with no synchronisation (with `overlap`, carrying the flag that lets steps
    of independent caches run side by side); outputs, evictions and final state must be equal bit for
    bit.  Returns a function that prefills fresh caches and the decode inputs."""
    V = P.vatp()

    def prefilled(decode_overlap=False):
        gs = []
        for wl in wls:
            q, k, v = synth.prefill_inputs(wl, 0, "cuda")
            gs.append(P.GpuPrefill(wl, q, k, v, decode_overlap=decode_overlap).run())
        return gs

    ins = [synth.decode_inputs(wl, 0, device="cuda") for wl in wls]
    alone = prefilled()
    outs_a = [torch.empty(steps, wl.batch, wl.heads, wl.head_dim, dtype=torch.bfloat16, device="cuda") for wl in wls]
    evs_a = [torch.empty(steps, wl.batch, wl.heads, dtype=torch.int32, device="cuda") for wl in wls]
    for g, (dq, dk, dv), o, e in zip(alone, ins, outs_a, evs_a):
        for s in range(steps):
            V.vatp_decode_step(g.p, g.cache, dq[s], dk[s], dv[s], o[s], evicted_pos=e[s], dev_status=g.status)
            torch.cuda.synchronize()
    inter = prefilled(decode_overlap=overlap)
    outs_b = [torch.empty_like(o) for o in outs_a]
    evs_b = [torch.empty_like(e) for e in evs_a]
    for s in range(steps):
        for g, (dq, dk, dv), o, e in zip(inter, ins, outs_b, evs_b):
            V.vatp_decode_step(g.p, g.cache, dq[s], dk[s], dv[s], o[s], evicted_pos=e[s], dev_status=g.status)
    torch.cuda.synchronize()
    for ga, gb, oa, ob, ea, eb in zip(alone, inter, outs_a, outs_b, evs_a, evs_b):
        assert int(ga.status.item()) == 0 and int(gb.status.item()) == 0
        assert torch.equal(oa, ob) and torch.equal(ea, eb)
        for name in ("k_cache", "v_cache", "acc", "vnorm", "pos", "len", "free_slot", "next_pos"):
            assert torch.equal(getattr(ga.cache, name), getattr(gb.cache, name)), name
    return prefilled, ins


@pytest.mark.parametrize("overlap", [True, False])
@pytest.mark.parametrize("b,h", [(1, 3), (5, 32)])
def test_interleaved_caches_match_separate_runs(b, h, overlap):
    """Decode steps of three independent caches issued back to back on one stream (launches that share
    no buffer may overlap on the GPU) give bit for bit what each cache gives when stepped alone, and
    the result agrees with the oracle.  With 3 units per cache every launch could still be in flight
    when the same cache comes round again, so the steps wait for one another; with 160 units a launch
    fills half the machine and the steps of different caches run side by side."""
    steps = 12
    wls = [_small("bf16", 128, 900, 300, 2, 30, b=b, h=h, steps=steps, cid=70 + i) for i in range(3)]
    prefilled, ins = _interleaved_equals_alone(wls, steps, overlap)
    # (c) and the trajectory of some units of one cache against the oracle
    g = prefilled()[1]
    units = [(0, 0), (b - 1, h - 1), (b // 2, h // 2)]
    refs = {u: P.check_prefill_unit(g, u[0], u[1], P.TOL["bf16"])[:2] for u in units}
    P.run_decode_and_check(g, refs, *ins[1], steps, P.TOL["bf16"], check_state_every=4)


@pytest.mark.parametrize("T,w,B,F,R", [
    (1000, 300, 400, 2, 10),     # window start inside a tile, ragged prompt
    (200, 256, 80, 0, 10),       # prompt shorter than the window: Eq. 3 is Eq. 2, leading rows of the history are empty
    (768, 128, 300, 4, 10),      # window = exactly the last tile
    (513, 1, 200, 0, 0),         # a window of one query
    (640, 640, 256, 2, 16),      # window = whole prompt
])
@pytest.mark.parametrize("recompute", [True, False])
def test_windowed_indicator_shapes(T, w, B, F, R, recompute):
    """Eq. 3 on the tensor-core path (bf16, d 128) for windows that start anywhere, with decode steps that
    roll the history ring; the history either gathered from win_rows or rebuilt by vatp_compact_window."""
    _run_case(_small("bf16", 128, T, B, F, R, b=1, h=2, indicator="window", window=w, steps=8, cid=60),
              recompute_window=recompute)


@pytest.mark.parametrize("recompute", [True, False])
@pytest.mark.parametrize("dtype,d", [("f32", 64), ("bf16", 64), ("f32", 128)])
def test_windowed_indicator_general_kernels(dtype, d, recompute):
    _run_case(_small(dtype, d, 300, 120, 2, 10, b=1, h=2, indicator="window", window=77, steps=6, cid=61),
              recompute_window=recompute)


def test_window_history_rebuilt_equals_gathered():
    """The two ways to the windowed decode state on the same inputs: probabilities gathered from win_rows and
    probabilities recomputed from Q and the kept keys agree to the accuracy of the scoring pass's exponential
    (one pair in eight takes a polynomial with 7.5e-5 relative error there; the rebuild uses ex2 throughout),
    ring entries and exact window sums alike, and everything else in the state is identical."""
    wl = _small("bf16", 128, 1500, 600, 4, 10, b=2, h=5, indicator="window", window=400, steps=0, cid=69)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    a = P.GpuPrefill(wl, q, k, v).run()
    b = P.GpuPrefill(wl, q, k, v, recompute_window=True).run()
    assert torch.equal(a.score, b.score) and torch.equal(a.kept, b.kept)
    for name in ("k_cache", "v_cache", "vnorm", "pos", "len", "free_slot", "next_pos"):
        assert torch.equal(getattr(a.cache, name), getattr(b.cache, name)), name
    ra, rb = a.cache.ring.double(), b.cache.ring.double()
    assert torch.all((ra - rb).abs() <= 1e-4 * ra.abs() + 1e-30), "ring entries"
    fa, fb = a.cache.acc_fixed.double(), b.cache.acc_fixed.double()
    assert torch.all((fa - fb).abs() <= 1e-4 * fa.abs() + 1.0), "fixed-point sums"


@pytest.mark.parametrize("norm", ["l2", "linf"])
@pytest.mark.parametrize("dtype,d,T,B,indicator,window", [
    ("bf16", 128, 700, 300, "h2o", 0),        # tensor-core prefill (side warp) + tensor-core decode
    ("bf16", 128, 600, 250, "window", 200),   # windowed: the norm kernel of its own
    ("f32", 64, 333, 100, "h2o", 0),          # general kernels
])
def test_value_norm_kinds(norm, dtype, d, T, B, indicator, window):
    """The Ablation Study's l2 and l-infinity norms in place of Eq. 4's l1: prefill norms, scores,
    kept sets, and the norms of tokens appended by decode steps (which decide later evictions)."""
    wl = _small(dtype, d, T, B, 2, 10, b=1, h=3, indicator=indicator, window=window, steps=12, cid=66).with_(norm=norm)
    g, _, _ = _run_case(wl)
    v0 = g.v[0, 0].double()
    ref = v0.pow(2).sum(-1).sqrt() if norm == "l2" else v0.abs().amax(-1)
    assert torch.allclose(g.vnorm[0, 0].double(), ref, rtol=1e-5, atol=0)
    l1 = v0.abs().sum(-1)
    assert torch.all(g.vnorm[0, 0].double() < l1)     # a different norm really was taken


@pytest.mark.parametrize("method,ratio", [("scissorhands", 1.0), ("scissorhands", 0.5), ("scissorhands", 0.25),
                                           ("h2o", 0.5), ("h2o", 0.25)])
def test_appendix_a_presets(method, ratio):
    """Appendix A's hyper-parameters through the product's preset table: H2O (half the budget chosen by
    importance, half local window) and Scissorhands (10 local tokens, history window 400) with the first
    20 tokens kept, at the throughput table's budgets.  At 100% nothing is pruned at prefill and the first
    decode step already evicts.  The oracle takes its split from its own Appendix A function."""
    from oracle import vatp_oracle as O
    from paper_2406_12335_b200 import presets
    T = 900
    pr = presets.appendix_a(method, T, ratio)
    sp = O.appendix_a_split(method, T, ratio)
    assert (pr["budget"], pr["n_sink"], pr["n_recent"], pr["window"]) == (sp["B"], sp["F"], sp["R"], sp["w"] or 0)
    wl = synth.Workload(67, f"preset_{method}_{ratio}", "bf16", 1, 3, 1, 128, T, sp["B"], sp["F"], sp["R"],
                        "window" if sp["w"] else "h2o", sp["w"] or 0, 10)
    g, _, _ = _run_case(wl, check_state_every=5)
    assert int(g.cache.len[0, 0]) == sp["B"]                    # held at budget: 10 appended, 10 evicted
    assert torch.all(g.cache.pos[0, 0, : sp["F"]].cpu() == torch.arange(sp["F"]))


def test_config5_throughput_table_shape():
    """The shape of the paper's throughput measurements (batch 12, prompt 4096, Scissorhands split with
    w = 400, F = 20) at the 50% budget, full per-layer size: oracle on sampled units with decode steps,
    oracle-free invariants on all 384 units."""
    wl = synth.CONFIGS[5].with_(decode_steps=24)
    _run_case(wl, units=[(0, 0), (11, 31)], check_state_every=12, recompute_window=True)


@pytest.mark.parametrize("dtype,d,T,B,indicator,window,norm", [
    ("bf16", 128, 1000, 300, "h2o", 0, "l1"),       # tensor-core pass 2 alone, ragged against 128 and 256
    ("bf16", 128, 640, 200, "h2o", 0, "linf"),      # odd tile count (half a chunk of padding)
    ("bf16", 128, 900, 450, "window", 400, "l1"),   # Eq. 3: only the last 400 normalisers are read
    ("f32", 64, 333, 100, "h2o", 0, "l1"),          # general kernel
    ("f32", 64, 300, 120, "window", 77, "l2"),
    ("bf16", 64, 257, 128, "h2o", 0, "l1"),
])
def test_prefill_from_given_row_normalisers(dtype, d, T, B, indicator, window, norm):
    """vatp_prefill_scores_from_lse: the normalisers of Eq. 1 come from outside (a float64 torch
    computation standing in for an attention forward), pass 1 is skipped; indicator, norms, scores, kept
    sets, compaction and decode steps are checked against the oracle as for the two-pass call, and the
    outputs agree with the two-pass call within the score tolerance."""
    wl = _small(dtype, d, T, B, 2, 10, b=2, h=2, indicator=indicator, window=window, steps=4, cid=68).with_(norm=norm)
    g, _, _ = _run_case(wl, lse_given=True)
    assert torch.equal(g.lse, g.lse_in)                      # lse_out receives a copy
    two = P.GpuPrefill(wl, g.q, g.k, g.v).run()
    tol = P.TOL[dtype]
    for name in ("attn_acc", "vnorm", "score"):
        a, b_ = getattr(g, name).double(), getattr(two, name).double()
        assert torch.all((a - b_).abs() <= 2 * tol * b_.abs() + 1e-30), name


def test_prefill_from_given_row_normalisers_config1():
    """Config 1's shape (32 heads, prompt 4096) with given normalisers: oracle on sampled heads."""
    wl = synth.CONFIGS[1].with_(decode_steps=0)
    _run_case(wl, decode=False, units=[(0, 0), (0, 17)], lse_given=True)


@pytest.mark.parametrize("dtype,d,T,B,indicator,window", [
    ("bf16", 128, 1000, 300, "h2o", 0),       # tensor-core forward: 8 query tiles, ragged last tile
    ("bf16", 128, 130, 65, "h2o", 0),         # two tiles, the second almost empty
    ("bf16", 128, 100, 40, "h2o", 0),         # shorter than one tile
    ("bf16", 128, 700, 200, "window", 150),   # Eq. 3: normalisers of every row, indicator over the last w
    ("f32", 64, 333, 100, "h2o", 0),          # general forward
    ("f32", 64, 200, 64, "window", 50),
    ("bf16", 64, 257, 128, "h2o", 0),
])
@pytest.mark.parametrize("norm", ["l1", "linf"])
def test_fused_attention_forward(dtype, d, T, B, indicator, window, norm):
    """vatp_prefill_attention_scores: the attention output rows (Eq. 1) against the oracle, and everything the
    two-pass call produces - normalisers, indicator, norms, scores, kept sets, compaction, decode steps - checked
    the same way; its scores agree with the two-pass call's within the score tolerance."""
    wl = _small(dtype, d, T, B, 2, 10, b=2, h=3, indicator=indicator, window=window, steps=4, cid=75).with_(norm=norm)
    g, _, _ = _run_case(wl, fused_forward=True)
    two = P.GpuPrefill(wl, g.q, g.k, g.v).run()
    tol = P.TOL[dtype]
    for name in ("attn_acc", "vnorm", "score"):
        a, b_ = getattr(g, name).double(), getattr(two, name).double()
        assert torch.all((a - b_).abs() <= 2 * tol * b_.abs() + 1e-30), name


def test_fused_attention_forward_config1():
    """Config 1's shape through the fused forward: oracle on two sampled heads (output rows, scores, kept set)."""
    wl = synth.CONFIGS[1].with_(decode_steps=0)
    _run_case(wl, decode=False, units=[(0, 3), (0, 30)], fused_forward=True)


def test_fused_attention_forward_strided_inputs_and_determinism():
    """[b, T, h, d] storage viewed as [b, h, T, d]: same bits as the contiguous call (the output is always
    contiguous); and two runs over enough work items that the CTAs draw them in a different order give the same bits."""
    wl = _small("bf16", 128, 300, 100, 2, 10, b=2, h=3, cid=78)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    qs, ks, vs = (x.transpose(1, 2).contiguous().transpose(1, 2) for x in (q, k, v))
    g1 = P.GpuPrefill(wl, q, k, v, fused_forward=True).run()
    g2 = P.GpuPrefill(wl, qs, ks, vs, fused_forward=True)
    g2.attn_out = torch.empty_like(q)
    g2.run()
    assert torch.equal(g1.attn_out, g2.attn_out) and torch.equal(g1.score, g2.score) and torch.equal(g1.lse, g2.lse)
    wl = _small("bf16", 128, 700, 200, 2, 20, b=2, h=100, cid=79)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    a = P.GpuPrefill(wl, q, k, v, fused_forward=True).run()
    b = P.GpuPrefill(wl, q, k, v, fused_forward=True).run()
    assert torch.equal(a.attn_out, b.attn_out) and torch.equal(a.score, b.score) and torch.equal(a.kept, b.kept)


def test_fused_attention_forward_config2_shape():
    """Config 2's per-layer shape (256 units, prompt 8192, the L2-grouped item order) through the fused call: oracle on
    two units of a late layer (wide logits), invariants on all."""
    wl = synth.CONFIGS[2].with_(decode_steps=0)
    _run_case(wl, decode=False, units=[(0, 5), (7, 31)], layer=31, fused_forward=True)


def test_fused_attention_forward_config4_sampled_rows():
    """Config 4's per-layer shape (prompt 32768: the T x T matrix of a head is 8.6 GB) through the fused call: output rows and
    normalisers of sampled (head, query) pairs, each computed on its own by the oracle; scores of every head satisfy the
    oracle-free invariants, and equal the two-pass call's within the score tolerance."""
    from oracle import vatp_oracle as O
    wl = synth.CONFIGS[4].with_(decode_steps=0)
    q, k, v = synth.prefill_inputs(wl, 31, "cuda")
    g = P.GpuPrefill(wl, q, k, v, fused_forward=True).run()
    P.gpu_invariants(g)
    rng = np.random.default_rng(4)
    rows = [0, 1, 127, 128, 255, 256, 16383, 16384, 32639, 32640, 32767] + rng.integers(0, wl.seq_len, 13).tolist()
    for h in (0, 9, 31):
        kn, vn = P.to_np64(k[0, h]), P.to_np64(v[0, h])
        for j in rows:
            o, lse = O.attention_row(P.to_np64(q[0, h, j]), kn[: j + 1], vn[: j + 1], wl.scale)
            P.check_attention_output(P.to_np64(g.attn_out[0, h, j])[None], o[None], vn[: j + 1], "bf16")
            assert abs(float(g.lse[0, h, j]) - lse) <= 1e-2, (h, j)
    two = P.GpuPrefill(wl, q, k, v).run()
    for name in ("attn_acc", "vnorm", "score"):
        a, b_ = getattr(g, name).double(), getattr(two, name).double()
        assert torch.all((a - b_).abs() <= 2e-3 * b_.abs() + 1e-30), name
    assert torch.equal(g.kept, two.kept) or (g.kept != two.kept).sum().item() <= 2 * MAX_BOUNDARY_PER_UNIT * wl.heads


def test_fused_attention_forward_rescales_when_the_maximum_grows():
    """Keys whose logits keep growing along the prompt force the forward to move its reference maximum (and
    rescale the running output) in every chunk; keys whose logits fall never do.  Both against the oracle."""
    wl = _small("bf16", 128, 640, 200, 2, 10, b=1, h=2, steps=0, cid=76)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    ramp = torch.linspace(0.0, 6.0, wl.seq_len, device="cuda")
    for sign in (1.0, -1.0):
        # every query has a positive component along one direction; the keys' component along it ramps up or down
        q2, k2 = q.clone(), k.clone()
        q2[..., 0] = 8.0
        k2[..., 0] = (sign * ramp * 8.0).to(k.dtype)[None, None, :]
        g = P.GpuPrefill(wl, q2, k2, v, fused_forward=True).run()
        for h in range(wl.heads):
            P.check_prefill_unit(g, 0, h, P.TOL["bf16"])


def test_decode_large_cache_state_paths():
    """Caches too large for the per-slot state to sit beside the streaming stages.  Stepped alone, a
    launch waits for its predecessor and takes a whole SM, state included (checked against the
    oracle).  Five such caches of 40 units stepped round robin run side by side, two CTAs per SM: there
    the state is copied into the stage memory after the streaming (budget 3000) or read from global
    memory (budget 6000), and the results must equal those of stepping alone."""
    for T, B in ((3400, 3000), (6500, 6000)):
        _run_case(_small("bf16", 128, T, B, 2, 64, b=1, h=2, steps=5, cid=62), check_state_every=5)
        wls = [_small("bf16", 128, T, B, 2, 64, b=1, h=40, steps=4, cid=64 + i) for i in range(5)]
        _interleaved_equals_alone(wls, 4)


def test_expired_device_wait_reports_timeout_and_context_survives():
    """Failure detection without a fault: a wait that nothing satisfies runs out after its limit, the
    kernel writes VATP_ERR_TIMEOUT to the status word and returns; the next launch works as usual."""
    V = P.vatp()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    V.vatp_selftest_bounded_wait(2_000_000, status, waited)          # 2 ms
    torch.cuda.synchronize()
    assert int(status.item()) == 5
    assert 2_000_000 <= int(waited.item()) < 50_000_000
    with pytest.raises(V.VatpError):
        V.vatp_selftest_bounded_wait(10**9, status)                   # limits above 0.1 s are refused on the host
    _run_case(_small("bf16", 128, 300, 100, 2, 10, steps=3, cid=63))  # the context is intact


def _graphs_equal_stepping_alone(wls, plan, *, overlap, eager_first=0, replays=1, oracle_unit=None, layers=None):
    """Decode steps recorded into a CUDA graph against the same steps issued one by one with a
    synchronisation after each.  plan: list of (cache index, step index) in issue order; the first
    `eager_first` entries are issued directly (not captured), the rest are captured once and the graph is
    replayed `replays` times back to back (every replay repeats the same steps on the advancing caches and
    overwrites the same output rows, which the reference arm does too).  Outputs, evictions and the final state must be equal bit for bit.  With oracle_unit =
    (cache, b, h) that unit's trajectory of the reference arm is also checked against the oracle."""
    V = P.vatp()
    layers = layers or [0] * len(wls)

    def prefilled(decode_overlap):
        gs = []
        for wl, layer in zip(wls, layers):
            q, k, v = synth.prefill_inputs(wl, layer, "cuda")
            gs.append(P.GpuPrefill(wl, q, k, v, decode_overlap=decode_overlap).run())
        return gs

    ins = [synth.decode_inputs(wl, layer, device="cuda") for wl, layer in zip(wls, layers)]
    nsteps = max(s for _, s in plan) + 1
    mk = lambda dt, tail: [torch.zeros((2, nsteps, wl.batch, wl.heads) + tail(wl), dtype=dt, device="cuda") for wl in wls]
    outs_a, outs_b = mk(torch.bfloat16, lambda wl: (wl.head_dim,)), mk(torch.bfloat16, lambda wl: (wl.head_dim,))
    evs_a, evs_b = mk(torch.int32, lambda wl: ()), mk(torch.int32, lambda wl: ())

    def issue(gs, outs, evs, entries, rep):
        for ci, s in entries:
            g, (dq, dk, dv) = gs[ci], ins[ci]
            V.vatp_decode_step(g.p, g.cache, dq[s], dk[s], dv[s], outs[ci][rep, s], evicted_pos=evs[ci][rep, s], dev_status=g.status)

    # reference arm: one by one, no flag
    alone = prefilled(False)
    for rep, entries in enumerate([plan[:eager_first]] + [plan[eager_first:]] * replays):
        for e in entries:
            issue(alone, outs_a, evs_a, [e], min(rep, 1))
            torch.cuda.synchronize()
    # graph arm
    inter = prefilled(overlap)
    issue(inter, outs_b, evs_b, plan[:eager_first], 0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        issue(inter, outs_b, evs_b, plan[eager_first:], 1)
    for _ in range(replays):
        graph.replay()
    torch.cuda.synchronize()
    for ga, gb, oa, ob, ea, eb in zip(alone, inter, outs_a, outs_b, evs_a, evs_b):
        assert int(ga.status.item()) == 0 and int(gb.status.item()) == 0
        assert torch.equal(oa, ob) and torch.equal(ea, eb)
        for name in ("k_cache", "v_cache", "acc", "vnorm", "pos", "len", "free_slot", "next_pos"):
            assert torch.equal(getattr(ga.cache, name), getattr(gb.cache, name)), name
    if oracle_unit is not None:
        ci, b, h = oracle_unit
        g = prefilled(False)[ci]
        ref, kept, _ = P.check_prefill_unit(g, b, h, P.TOL["bf16"])
        order = [s for c, s in plan[:eager_first] if c == ci] + [s for c, s in plan[eager_first:] if c == ci] * replays
        dq, dk, dv = (x[order] for x in ins[ci])
        P.run_decode_and_check(g, {(b, h): (ref, kept)}, dq, dk, dv, len(order), P.TOL["bf16"], check_state_every=4)


@pytest.mark.parametrize("overlap", [True, False])
@pytest.mark.parametrize("h", [3, 8])
def test_same_cache_steps_in_a_graph_with_few_units(h, overlap):
    """One small cache (3 or 8 units: grids of a few dozen CTAs, so that many launches fit on the machine
    together) stepped 24 times from a graph: every step depends on the one before it, and a step may only
    ever run ahead of ONE unfinished predecessor, whose appended row it re-reads."""
    wl = _small("bf16", 128, 900, 300, 2, 30, b=1, h=h, steps=24, cid=71)
    plan = [(0, s) for s in range(24)]
    _graphs_equal_stepping_alone([wl], plan, overlap=overlap, eager_first=2, oracle_unit=(0, 0, h - 1))


@pytest.mark.parametrize("eager_first", [0, 7])
@pytest.mark.parametrize("ncaches", [2, 5])
def test_graph_of_independent_caches_replayed_back_to_back(ncaches, eager_first):
    """Graphs [A, B] and [A .. E] of steps of independent caches (overlap flag set), captured cold
    (eager_first = 0) or after unrelated steps issued directly, replayed three times back to back.
    Whatever preceded a replay - the previous replay's tail included - the result must be that of
    stepping one by one."""
    wls = [_small("bf16", 128, 900, 300, 2, 30, b=2, h=32, steps=8, cid=72 + i) for i in range(ncaches)]
    pre = [(c, 0) for c in range(ncaches)] * 4
    plan = pre[:eager_first] + [(c, 1) for c in range(ncaches)]
    _graphs_equal_stepping_alone(wls, plan, overlap=True, eager_first=eager_first, replays=3, oracle_unit=(1, 1, 31))


def test_config1_layers_interleaved_in_a_graph_match_stepping_alone():
    """The launch configuration the benchmark times: eight independently seeded config-1 layers, their
    decode steps interleaved with the overlap flag set and replayed from a CUDA graph (consecutive
    launches run side by side on the GPU).  Outputs, evictions and final state must equal, bit for bit,
    each layer stepped alone with a synchronisation after every step."""
    wl = synth.CONFIGS[1].with_(decode_steps=6)
    L = 8
    plan = [(l, s) for s in range(wl.decode_steps) for l in range(L)]
    _graphs_equal_stepping_alone([wl] * L, plan, overlap=True, eager_first=2 * L, layers=list(range(L)))


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_optional_outputs_may_be_null(dtype, d):
    """lse_out and evicted_pos are nullable: leaving them out changes nothing else."""
    V = P.vatp()
    wl = _small(dtype, d, 400, 150, 2, 12, b=1, h=3, steps=4, cid=64)
    q, k, v = synth.prefill_inputs(wl, 0, "cuda")
    full = P.GpuPrefill(wl, q, k, v).run()
    bare = P.GpuPrefill(wl, q, k, v)
    V.vatp_prefill_scores(bare.p, q, k, v, attn_acc=bare.attn_acc, vnorm=bare.vnorm, score=bare.score,
                          workspace=bare.ws, dev_status=bare.status)                      # no lse_out
    V.vatp_select(bare.p, bare.score, bare.kept)
    V.vatp_compact(bare.p, k, v, bare.attn_acc, bare.vnorm, bare.kept, bare.cache)
    torch.cuda.synchronize()
    assert torch.equal(full.score, bare.score) and torch.equal(full.kept, bare.kept)
    dq, dk, dv = synth.decode_inputs(wl, 0, device="cuda")
    o1 = torch.empty(1, 3, d, dtype=q.dtype, device="cuda")
    o2 = torch.empty_like(o1)
    ev = torch.empty(1, 3, dtype=torch.int32, device="cuda")
    for s in range(wl.decode_steps):
        V.vatp_decode_step(full.p, full.cache, dq[s], dk[s], dv[s], o1, evicted_pos=ev, dev_status=full.status)
        V.vatp_decode_step(bare.p, bare.cache, dq[s], dk[s], dv[s], o2)                     # no evicted_pos, no status word
        torch.cuda.synchronize()
        assert torch.equal(o1, o2)
    assert torch.equal(full.cache.pos, bare.cache.pos) and torch.equal(full.cache.acc, bare.cache.acc)


def test_bounds_checking_build_reports_no_violation():
    """The library built with -DVATP_DEBUG_BOUNDS range-checks every row, slot, window-row and scratch index its
    kernels compute (an index outside its array is skipped and reported as VATP_ERR_BOUNDS in the status word,
    which every test here asserts to be zero).  Ragged, windowed, large-cache and graph cases run once more on
    that build, in a process of their own; it stands in for a memory checker, which cannot be run here."""
    import os
    import subprocess
    import sys
    from paper_2406_12335_b200 import build
    lib = build.build(debug_bounds=True)
    env = dict(os.environ, VATP_LIBRARY=lib)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sel = ("ragged or degenerate or windowed_indicator_shapes or general_kernels or large_cache or few_units "
           "or exact_ties or unstaged or strided or static_scratch_matches or rebuilt or (fused_attention and not config1) "
           "or grouped_query_caches")
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_zz_no_alloc.py", "-x", "-q",
                        "-m", "gpu", "-k", sel, "-p", "no:cacheprovider"], cwd=root, env=env, capture_output=True, text=True)
    tail = (r.stdout + r.stderr)[-2000:]
    assert r.returncode == 0, tail
    assert " passed" in tail and "libvatp_dbg" in subprocess.run(
        [sys.executable, "-c", "from paper_2406_12335_b200 import vatp; print(vatp._LIB_PATH)"], cwd=root, env=env,
        capture_output=True, text=True).stdout


@pytest.mark.parametrize("dtype,d,heads,kv_heads,T,B,F,R", [
    ("bf16", 128, 8, 2, 700, 250, 2, 20),      # tensor-core scoring, four query heads per KV head
    ("bf16", 128, 6, 3, 1000, 1100, 0, 8),     # budget beyond the prompt: the cache grows before evictions start
    ("f32", 64, 4, 2, 333, 100, 3, 17),        # general kernels
    ("bf16", 64, 8, 1, 257, 128, 2, 16),       # multi-query attention: one KV head
    ("f32", 128, 16, 1, 200, 80, 1, 8),        # sixteen heads per group, 32 pieces per row
    ("bf16", 128, 16, 2, 900, 300, 2, 20),     # eight heads per group: every row of the decode step's MMA tiles is a head
    ("bf16", 128, 32, 2, 300, 120, 1, 8),      # sixteen heads per group: beyond the tensor-core step, general decode kernel
    ("bf16", 128, 10, 2, 500, 200, 1, 12),     # five heads per group: three rows of the MMA tiles repeat the last head
])
@pytest.mark.parametrize("fused", [False, True])
def test_grouped_query_attention(dtype, d, heads, kv_heads, T, B, F, R, fused):
    """Grouped-query attention (the Limitations section's open case, read as a group-mean indicator): the G query
    heads of a KV group share one kept set and one cache.  Scoring, selection, compaction and decode steps of
    every KV unit against the oracle; the row normalisers of every query head as well.  fused: through
    vatp_prefill_attention_scores, the attention output rows of every query head too."""
    from oracle import vatp_oracle as O
    V = P.vatp()
    b, G, steps = 2, heads // kv_heads, 10
    tol = P.TOL[dtype]
    wl_kv = _small(dtype, d, T, B, F, R, b=b, h=kv_heads, steps=steps, cid=77)
    _, k, v = synth.prefill_inputs(wl_kv, 0, "cuda")
    # queries of all heads: Gaussian plus the sink direction of their KV head (the keys of tokens 0 and 1 carry it)
    u = synth.sink_direction(wl_kv, 0, "cuda").repeat_interleave(G, dim=1)
    gq = torch.Generator(device="cuda").manual_seed(4077)
    q = (torch.randn(b, heads, T, d, generator=gq, device="cuda") + synth.sink_alpha(wl_kv) * u).to(k.dtype)
    dq = (torch.randn(steps, b, heads, d, generator=gq, device="cuda") + synth.sink_alpha(wl_kv) * u.squeeze(2)).to(k.dtype)
    _, dk, dv = synth.decode_inputs(wl_kv, 0, device="cuda")

    p = V.make_params(batch=b, heads=heads, kv_heads=kv_heads, seq_len=T, head_dim=d, dtype=dtype, budget=B, n_sink=F,
                      n_recent=R, scale=wl_kv.scale)
    f32 = dict(dtype=torch.float32, device="cuda")
    lse = torch.empty(b, heads, T, **f32)
    attn_acc, vnorm, score = (torch.empty(b, kv_heads, T, **f32) for _ in range(3))
    ws = torch.empty(V.vatp_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kept = torch.empty(b, kv_heads, B, dtype=torch.int32, device="cuda")
    cache = V.Cache(p)
    attn_out = torch.full_like(q, float("nan")) if fused else None
    if fused:
        V.vatp_prefill_attention_scores(p, q, k, v, attn_out, lse_out=lse, attn_acc=attn_acc, vnorm=vnorm, score=score,
                                        workspace=ws, dev_status=status)
    else:
        V.vatp_prefill_scores(p, q, k, v, lse_out=lse, attn_acc=attn_acc, vnorm=vnorm, score=score, workspace=ws, dev_status=status)
    V.vatp_select(p, score, kept, dev_status=status)
    V.vatp_compact(p, k, v, attn_acc, vnorm, kept, cache, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.all((attn_acc.double().sum(-1) - T).abs() <= 2e-3 * T)

    n_live = min(T, B)
    states = {}
    for bi in range(b):
        for g in range(kv_heads):
            ref = O.prefill_gqa(P.to_np64(q[bi, g * G:(g + 1) * G]), P.to_np64(k[bi, g]), P.to_np64(v[bi, g]), wl_kv.scale)
            assert np.max(np.abs(P.to_np64(lse[bi, g * G:(g + 1) * G]) - ref["lse"])) <= 10 * tol
            if fused:
                for hq in range(g * G, (g + 1) * G):
                    want_out = O.attention_output(O.attention_probs(P.to_np64(q[bi, hq]), P.to_np64(k[bi, g]), wl_kv.scale),
                                                  P.to_np64(v[bi, g]))
                    P.check_attention_output(P.to_np64(attn_out[bi, hq]), want_out, P.to_np64(v[bi, g]), dtype)
            for name, key in (("attn_acc", "S"), ("vnorm", "n1"), ("score", "I")):
                e = P.rel_err(P.to_np64(locals()[name][bi, g]), ref[key])
                assert e <= tol, f"{name} rel err {e:.3g} (unit {bi},{g})"
            want = O.select_keep(ref["I"], B, F, R)
            got = kept[bi, g, :n_live].cpu().numpy().astype(np.int64)
            assert np.array_equal(got, want), "kept set"
            assert torch.equal(cache.k_cache[bi, g, :n_live], k[bi, g][torch.from_numpy(got).cuda()])
            states[(bi, g)] = O.DecodeState(P.to_np64(k[bi, g]), P.to_np64(v[bi, g]), ref["S"], ref["n1"], got, T)

    out = torch.empty(b, heads, d, dtype=k.dtype, device="cuda")
    evicted = torch.empty(b, kv_heads, dtype=torch.int32, device="cuda")
    out_eps = 2.0 ** -8 if dtype == "bf16" else 0.0
    for s in range(steps):
        V.vatp_decode_step(p, cache, dq[s], dk[s], dv[s], out, evicted_pos=evicted, dev_status=status)
        torch.cuda.synchronize()
        for (bi, g), st in states.items():
            ev = int(evicted[bi, g])
            res = O.decode_step(st, P.to_np64(dq[s, bi, g * G:(g + 1) * G]), P.to_np64(dk[s, bi, g]), P.to_np64(dv[s, bi, g]),
                                wl_kv.scale, B, F, R, force_evict=None if ev < 0 else ev, tie_tol=2 * tol, tie_abs=1e-30)
            assert res["evicted"] == ev and not res["adopted"]
            ref_out = res["out"]
            bound = tol * np.max(np.abs(ref_out)) + out_eps * np.abs(ref_out) + 1e-30
            assert np.all(np.abs(P.to_np64(out[bi, g * G:(g + 1) * G]) - ref_out) <= bound), f"step {s} unit {(bi, g)}: out"
    assert int(status.item()) == 0
    for (bi, g), st in states.items():
        pos = cache.pos[bi, g].cpu().numpy()
        live = pos >= 0
        order = np.argsort(pos[live])
        assert pos[live][order].tolist() == st.pos and int(cache.len[bi, g]) == len(st.pos)
        assert P.rel_err(P.to_np64(cache.acc[bi, g])[live][order], st.indicator()) <= 2 * tol


@pytest.mark.parametrize("dtype,d,heads,kv_heads,T,B,F,R,w", [
    ("bf16", 128, 8, 2, 700, 250, 2, 10, 150),     # tensor-core scoring per query head, window starts inside a tile
    ("f32", 64, 4, 2, 333, 100, 3, 10, 50),        # general kernels
    ("bf16", 128, 4, 1, 300, 120, 0, 8, 400),      # window longer than the prompt, one KV head
])
def test_grouped_query_attention_with_history_window(dtype, d, heads, kv_heads, T, B, F, R, w):
    """Grouped queries with the windowed indicator (Eq. 3 under the group-mean reading): the indicator over the last w
    queries, the history ring rebuilt by vatp_compact_window as the mean of the heads' probabilities, and decode steps
    through evictions and through the window sliding, every KV unit against the oracle."""
    from oracle import vatp_oracle as O
    V = P.vatp()
    b, G, steps = 2, heads // kv_heads, 12
    tol = P.TOL[dtype]
    wl_kv = _small(dtype, d, T, B, F, R, b=b, h=kv_heads, indicator="window", window=w, steps=steps, cid=81)
    _, k, v = synth.prefill_inputs(wl_kv, 0, "cuda")
    u = synth.sink_direction(wl_kv, 0, "cuda").repeat_interleave(G, dim=1)
    gq = torch.Generator(device="cuda").manual_seed(4081)
    q = (torch.randn(b, heads, T, d, generator=gq, device="cuda") + synth.sink_alpha(wl_kv) * u).to(k.dtype)
    dq = (torch.randn(steps, b, heads, d, generator=gq, device="cuda") + synth.sink_alpha(wl_kv) * u.squeeze(2)).to(k.dtype)
    _, dk, dv = synth.decode_inputs(wl_kv, 0, device="cuda")

    p = V.make_params(batch=b, heads=heads, kv_heads=kv_heads, seq_len=T, head_dim=d, dtype=dtype, budget=B, n_sink=F,
                      n_recent=R, scale=wl_kv.scale, indicator="window", window=w)
    f32 = dict(dtype=torch.float32, device="cuda")
    lse = torch.empty(b, heads, T, **f32)
    attn_acc, vnorm, score = (torch.empty(b, kv_heads, T, **f32) for _ in range(3))
    ws = torch.empty(V.vatp_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kept = torch.empty(b, kv_heads, B, dtype=torch.int32, device="cuda")
    cache = V.Cache(p)
    V.vatp_prefill_scores(p, q, k, v, lse_out=lse, attn_acc=attn_acc, vnorm=vnorm, score=score, workspace=ws, dev_status=status)
    V.vatp_select(p, score, kept, dev_status=status)
    V.vatp_compact_window(p, q, k, v, lse, attn_acc, vnorm, kept, cache, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.all((attn_acc.double().sum(-1) - min(w, T)).abs() <= 2e-3 * min(w, T))

    n_live = min(T, B)
    states = {}
    for bi in range(b):
        for g in range(kv_heads):
            ref = O.prefill_gqa(P.to_np64(q[bi, g * G:(g + 1) * G]), P.to_np64(k[bi, g]), P.to_np64(v[bi, g]), wl_kv.scale, window=w)
            first = max(T - w, 0)
            assert np.max(np.abs(P.to_np64(lse[bi, g * G:(g + 1) * G, first:]) - ref["lse"][:, first:])) <= 10 * tol
            for name, key in (("attn_acc", "S"), ("vnorm", "n1"), ("score", "I")):
                e = P.rel_err(P.to_np64(locals()[name][bi, g]), ref[key])
                assert e <= tol, f"{name} rel err {e:.3g} (unit {bi},{g})"
            got = kept[bi, g, :n_live].cpu().numpy().astype(np.int64)
            want = O.select_keep(ref["I"], B, F, R)
            if not np.array_equal(got, want):        # only indices whose score ties the boundary within the tolerance may differ
                mid = [i for i in want if F <= i < T - R]
                tau = ref["I"][mid].min()
                for i in set(got.tolist()) ^ set(want.tolist()):
                    assert abs(ref["I"][i] - tau) <= tol * tau
            # the ring: row (j mod w) = group-mean probabilities of query j on the kept tokens; exact window sums
            ring = P.to_np64(cache.ring[bi, g])
            rows_ref = ref["window_rows"]
            j0 = T - rows_ref.shape[0]
            want_ring = np.zeros((w, n_live))
            for r in range(rows_ref.shape[0]):
                want_ring[(j0 + r) % w] = rows_ref[r][got]
            assert np.max(np.abs(ring[:, :n_live] - want_ring) - tol * np.abs(want_ring)) <= 1e-30, "history ring"
            fixed = cache.acc_fixed[bi, g, :n_live].cpu().numpy().astype(np.float64) / 2.0 ** 52
            assert P.rel_err(fixed, ref["S"][got]) <= tol
            states[(bi, g)] = O.DecodeState(P.to_np64(k[bi, g]), P.to_np64(v[bi, g]), ref["S"], ref["n1"], got, T, window=w,
                                            window_rows=ref["window_rows"])

    out = torch.empty(b, heads, d, dtype=k.dtype, device="cuda")
    evicted = torch.empty(b, kv_heads, dtype=torch.int32, device="cuda")
    out_eps = 2.0 ** -8 if dtype == "bf16" else 0.0
    for s_ in range(steps):
        V.vatp_decode_step(p, cache, dq[s_], dk[s_], dv[s_], out, evicted_pos=evicted, dev_status=status)
        torch.cuda.synchronize()
        for (bi, g), st in states.items():
            ev = int(evicted[bi, g])
            res = O.decode_step(st, P.to_np64(dq[s_, bi, g * G:(g + 1) * G]), P.to_np64(dk[s_, bi, g]), P.to_np64(dv[s_, bi, g]),
                                wl_kv.scale, B, F, R, force_evict=None if ev < 0 else ev, tie_tol=2 * tol, tie_abs=1e-30)
            assert res["evicted"] == ev
            ref_out = res["out"]
            bound = tol * np.max(np.abs(ref_out)) + out_eps * np.abs(ref_out) + 1e-30
            assert np.all(np.abs(P.to_np64(out[bi, g * G:(g + 1) * G]) - ref_out) <= bound), f"step {s_} unit {(bi, g)}: out"
    assert int(status.item()) == 0
    for (bi, g), st in states.items():
        pos = cache.pos[bi, g].cpu().numpy()
        live = pos >= 0
        order = np.argsort(pos[live])
        assert pos[live][order].tolist() == st.pos and int(cache.len[bi, g]) == len(st.pos)
        assert P.rel_err(P.to_np64(cache.acc[bi, g])[live][order], st.indicator()) <= 2 * tol


@pytest.mark.parametrize("overlap", [True, False])
@pytest.mark.parametrize("b,heads,kv_heads", [(1, 8, 2), (6, 32, 8)])
def test_grouped_query_caches_interleaved_match_separate_runs(b, heads, kv_heads, overlap):
    """The tensor-core decode step with grouped queries (bf16, head_dim 128): steps of three independent caches issued
    round robin on one stream - with the opt-in flag they may run side by side - give bit for bit what each cache
    gives when stepped alone with a synchronisation after every step.  (Each step against the oracle:
    test_grouped_query_attention.)"""
    V = P.vatp()
    d, T, B, F, R, steps = 128, 600, 260, 2, 16, 10
    G = heads // kv_heads

    def prefilled(i, decode_overlap):
        wl_kv = _small("bf16", d, T, B, F, R, b=b, h=kv_heads, steps=steps, cid=80 + i)
        _, k, v = synth.prefill_inputs(wl_kv, 0, "cuda")
        gq = torch.Generator(device="cuda").manual_seed(5000 + i)
        q = torch.randn(b, heads, T, d, generator=gq, device="cuda").to(k.dtype)
        dq = torch.randn(steps, b, heads, d, generator=gq, device="cuda").to(k.dtype)
        _, dk, dv = synth.decode_inputs(wl_kv, 0, device="cuda")
        p = V.make_params(batch=b, heads=heads, kv_heads=kv_heads, seq_len=T, head_dim=d, dtype="bf16", budget=B, n_sink=F,
                          n_recent=R, scale=wl_kv.scale, decode_overlap=decode_overlap)
        f32 = dict(dtype=torch.float32, device="cuda")
        attn_acc, vnorm, score = (torch.empty(b, kv_heads, T, **f32) for _ in range(3))
        ws = torch.empty(V.vatp_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        kept = torch.empty(b, kv_heads, B, dtype=torch.int32, device="cuda")
        cache = V.Cache(p)
        V.vatp_prefill_scores(p, q, k, v, attn_acc=attn_acc, vnorm=vnorm, score=score, workspace=ws, dev_status=status)
        V.vatp_select(p, score, kept, dev_status=status)
        V.vatp_compact(p, k, v, attn_acc, vnorm, kept, cache, dev_status=status)
        torch.cuda.synchronize()
        return dict(p=p, cache=cache, status=status, dq=dq, dk=dk, dv=dv,
                    out=torch.empty(steps, b, heads, d, dtype=k.dtype, device="cuda"),
                    ev=torch.empty(steps, b, kv_heads, dtype=torch.int32, device="cuda"))

    def step(c, s):
        V.vatp_decode_step(c["p"], c["cache"], c["dq"][s], c["dk"][s], c["dv"][s], c["out"][s], evicted_pos=c["ev"][s],
                           dev_status=c["status"])

    alone = [prefilled(i, False) for i in range(3)]
    for c in alone:
        for s in range(steps):
            step(c, s)
            torch.cuda.synchronize()
    inter = [prefilled(i, overlap) for i in range(3)]
    for s in range(steps):
        for c in inter:
            step(c, s)
    torch.cuda.synchronize()
    for ca, cb in zip(alone, inter):
        assert int(ca["status"].item()) == 0 and int(cb["status"].item()) == 0
        assert torch.all(ca["ev"][-1] >= 0), "the last step evicts in every unit"
        assert torch.equal(ca["out"], cb["out"]) and torch.equal(ca["ev"], cb["ev"])
        for name in ("k_cache", "v_cache", "acc", "vnorm", "pos", "len", "free_slot", "next_pos"):
            assert torch.equal(getattr(ca["cache"], name), getattr(cb["cache"], name)), name
