"""Pins for the float64 oracle: closed forms, invariants, special cases and
brute force.  None of these call the CUDA library; none re-type the oracle's
own formulae with the same library calls (brute force is pure-Python loops
with math.exp; closed forms are exact rationals)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import vatp_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- brute force
def brute_attention(q, k, scale):
    """Eq. 1's a_i^t by explicit loops (no numpy arithmetic)."""
    T, d = len(q), len(q[0])
    a = [[0.0] * T for _ in range(T)]
    for t in range(T):
        logits = []
        for i in range(t + 1):
            acc = 0.0
            for c in range(d):
                acc += q[t][c] * k[i][c]
            logits.append(scale * acc)
        mx = max(logits)
        den = sum(math.exp(x - mx) for x in logits)
        for i in range(t + 1):
            a[t][i] = math.exp(logits[i] - mx) / den
    return a


def brute_h2o(a):
    T = len(a)
    return [sum(a[j][k] for j in range(k, T)) for k in range(T)]        # Eq. 2


def brute_window(a, w):
    T = len(a)
    return [sum(a[j][k] for j in range(max(T - w, k), T)) for k in range(T)]   # Eq. 3, last w rows


def brute_select(I, B, F, R):
    T = len(I)
    if T <= B:
        return list(range(T))
    mid = list(range(F, T - R))
    # repeatedly take the best remaining: highest importance, lowest index on ties
    chosen = []
    for _ in range(B - F - R):
        best = None
        for i in mid:
            if i in chosen:
                continue
            if best is None or I[i] > I[best]:
                best = i
        chosen.append(best)
    return sorted(list(range(F)) + chosen + list(range(T - R, T)))


@pytest.mark.parametrize("T,d,seed", [(1, 1, 0), (2, 3, 1), (5, 4, 2), (8, 4, 3), (7, 2, 4)])
def test_attention_and_indicators_match_brute_force(T, d, seed):
    rng = np.random.default_rng(seed)
    q = rng.normal(size=(T, d))
    k = rng.normal(size=(T, d))
    scale = 0.7
    a = O.attention_probs(q, k, scale)
    ab = brute_attention(q.tolist(), k.tolist(), scale)
    np.testing.assert_allclose(a, np.array(ab), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(O.indicator_h2o(a), brute_h2o(ab), rtol=1e-13)
    for w in (1, 2, 3, T, T + 5):
        np.testing.assert_allclose(O.indicator_window(a, w), brute_window(ab, w), rtol=1e-13, atol=1e-300)
    lse = O.row_logsumexp(q, k, scale)
    for t in range(T):
        ref = math.log(sum(math.exp(scale * float(q[t] @ k[i])) for i in range(t + 1)))
        assert abs(lse[t] - ref) < 1e-12


def test_transposed_operands_would_fail():
    """q and k are not interchangeable: a[j,i] uses q_j and k_i."""
    rng = np.random.default_rng(7)
    q = rng.normal(size=(6, 3))
    k = rng.normal(size=(6, 3))
    a = O.attention_probs(q, k, 1.0)
    ab = np.array(brute_attention(k.tolist(), q.tolist(), 1.0))
    assert np.abs(a - ab).max() > 1e-3


# ------------------------------------------------------------------ closed forms
def _harmonic(n):
    return sum(Fraction(1, i) for i in range(1, n + 1))


def test_two_token_example():
    """Uniform attention on T = 2: rows (1), (1/2, 1/2) -> S = (3/2, 1/2)."""
    q = np.zeros((2, 4))
    k = np.ones((2, 4))
    a = O.attention_probs(q, k, 0.5)
    np.testing.assert_allclose(a, [[1.0, 0.0], [0.5, 0.5]], atol=0)
    np.testing.assert_allclose(O.indicator_h2o(a), [1.5, 0.5], atol=1e-15)


@pytest.mark.parametrize("T", [3, 8, 33])
def test_uniform_attention_harmonic_closed_form(T):
    """Q = 0 gives a_i^j = 1/(j+1); Eq. 2 then equals H_T - H_k exactly."""
    rng = np.random.default_rng(T)
    k = rng.normal(size=(T, 5))
    a = O.attention_probs(np.zeros((T, 5)), k, 1.0)
    S = O.indicator_h2o(a)
    exact = [float(_harmonic(T) - _harmonic(kk)) for kk in range(T)]
    np.testing.assert_allclose(S, exact, rtol=1e-13)
    # identical key rows give the same matrix whatever q is
    a2 = O.attention_probs(rng.normal(size=(T, 5)), np.tile(k[:1], (T, 1)), 1.0)
    np.testing.assert_allclose(O.indicator_h2o(a2), exact, rtol=1e-12)


def test_uniform_attention_golden_file():
    """tests/golden/uniform_T8.txt: exact rationals written by make_golden.py."""
    rows = [l.split() for l in open(os.path.join(GOLD, "uniform_T8.txt")) if not l.startswith("#")]
    T = 8
    a = O.attention_probs(np.zeros((T, 2)), np.ones((T, 2)), 1.0)
    S = O.indicator_h2o(a)
    Sw = O.indicator_window(a, 3)
    for r in rows:
        kk = int(r[0])
        assert abs(S[kk] - float(Fraction(r[1]))) < 1e-14
        assert abs(Sw[kk] - float(Fraction(r[2]))) < 1e-14


@pytest.mark.parametrize("T,w", [(8, 3), (16, 16), (9, 1), (5, 12)])
def test_window_uniform_closed_form(T, w):
    a = O.attention_probs(np.zeros((T, 2)), np.ones((T, 2)), 1.0)
    S = O.indicator_window(a, w)
    exact = [float(sum(Fraction(1, j + 1) for j in range(max(T - w, kk), T))) for kk in range(T)]
    np.testing.assert_allclose(S, exact, rtol=1e-13)


def test_window_literal_bounds_is_one_more_row():
    T, w = 10, 4
    rng = np.random.default_rng(0)
    a = O.attention_probs(rng.normal(size=(T, 3)), rng.normal(size=(T, 3)), 1.0)
    np.testing.assert_allclose(O.indicator_window(a, w, inclusive_extra=1), O.indicator_window(a, w + 1))
    assert abs(O.indicator_window(a, w, inclusive_extra=1).sum() - (w + 1)) < 1e-12


# -------------------------------------------------------------------- invariants
@pytest.mark.parametrize("T,d", [(17, 8), (64, 16), (200, 64)])
def test_rows_sum_to_one_and_mass_conservation(T, d):
    rng = np.random.default_rng(T * 31 + d)
    q = rng.normal(size=(T, d)) * 2
    k = rng.normal(size=(T, d)) * 2
    a = O.attention_probs(q, k, 1 / math.sqrt(d))
    assert np.abs(a.sum(axis=1) - 1).max() < 1e-12
    assert np.all(np.triu(a, 1) == 0)
    assert abs(O.indicator_h2o(a).sum() - T) < 1e-9
    for w in (1, 5, T, 3 * T):
        assert abs(O.indicator_window(a, w).sum() - min(w, T)) < 1e-9


def test_window_at_least_T_is_h2o():
    rng = np.random.default_rng(5)
    a = O.attention_probs(rng.normal(size=(40, 8)), rng.normal(size=(40, 8)), 0.3)
    np.testing.assert_array_equal(O.indicator_window(a, 40), O.indicator_h2o(a))
    np.testing.assert_array_equal(O.indicator_window(a, 400), O.indicator_h2o(a))


def test_one_hot_limit():
    """A huge logit on key 0 sends every row's mass there: S_0 -> T."""
    T, d = 12, 4
    q = np.ones((T, d))
    k = np.zeros((T, d))
    k[0] = 100.0
    a = O.attention_probs(q, k, 1.0)
    S = O.indicator_h2o(a)
    assert abs(S[0] - T) < 1e-9 and S[1:].max() < 1e-9


def test_shift_invariance_of_softmax():
    rng = np.random.default_rng(11)
    q = rng.normal(size=(9, 4))
    k = rng.normal(size=(9, 4))
    a = O.attention_probs(q, k, 1.0)
    # adding the same vector to every key shifts each row's logits by a constant
    a2 = O.attention_probs(q, k, 1.0)
    shift = rng.normal(size=4)
    a2 = O.attention_probs(q, k + shift, 1.0)
    np.testing.assert_allclose(a, a2, rtol=1e-10, atol=1e-14)


# ------------------------------------------------------------------------ norms
def test_l1_norm_closed_forms():
    d = 128
    rng = np.random.default_rng(0)
    v = rng.choice([-1.0, 1.0], size=(10, d))
    np.testing.assert_array_equal(O.value_l1_norm(v), np.full(10, float(d)))
    np.testing.assert_allclose(O.value_l1_norm(np.full((3, d), -0.25)), 0.25 * d)
    big = rng.normal(size=(20000, d))
    assert abs(O.value_l1_norm(big).mean() - d * math.sqrt(2 / math.pi)) < 0.2   # E|N(0,1)| = sqrt(2/pi)
    # l1, not l2 or l-infinity
    assert O.value_l1_norm(np.array([[3.0, -4.0]]))[0] == 7.0


def test_norm_kinds_closed_forms_and_orderings():
    """The Ablation Study's three norms: closed forms on sign vectors and a 3-4-12 row, the textbook
    chain linf <= l2 <= l1 <= sqrt(d) l2 <= d linf, brute force by loops, homogeneity, and the fact
    that "l1" is the norm Eq. 4 uses."""
    d = 128
    rng = np.random.default_rng(5)
    sign = rng.choice([-1.0, 1.0], size=(6, d))
    np.testing.assert_array_equal(O.value_norm(sign, "l1"), np.full(6, float(d)))
    np.testing.assert_allclose(O.value_norm(sign, "l2"), math.sqrt(d), rtol=1e-15)
    np.testing.assert_array_equal(O.value_norm(sign, "linf"), np.ones(6))
    row = np.array([[3.0, -4.0, 12.0]])
    assert O.value_norm(row, "l1")[0] == 19.0 and O.value_norm(row, "l2")[0] == 13.0 and O.value_norm(row, "linf")[0] == 12.0
    v = rng.normal(size=(50, d)) * np.exp(rng.normal(size=(50, 1)))
    l1, l2, li = (O.value_norm(v, kd) for kd in ("l1", "l2", "linf"))
    eps = 1e-12
    assert np.all(li <= l2 * (1 + eps)) and np.all(l2 <= l1 * (1 + eps))
    assert np.all(l1 <= math.sqrt(d) * l2 * (1 + eps)) and np.all(l2 <= math.sqrt(d) * li * (1 + eps))
    for r in range(5):   # brute force
        assert abs(math.fsum(abs(x) for x in v[r]) - l1[r]) <= 1e-12 * l1[r]
        assert abs(math.sqrt(math.fsum(x * x for x in v[r])) - l2[r]) <= 1e-12 * l2[r]
        assert max(abs(x) for x in v[r]) == li[r]
    for kd in ("l1", "l2", "linf"):   # |c| comes out; a one-hot row has all three norms equal
        np.testing.assert_allclose(O.value_norm(-2.5 * v, kd), 2.5 * O.value_norm(v, kd), rtol=1e-14)
        onehot = np.zeros((1, d)); onehot[0, 17] = -0.75
        assert O.value_norm(onehot, kd)[0] == 0.75
    np.testing.assert_array_equal(O.value_norm(v, "l1"), O.value_l1_norm(v))
    with pytest.raises(ValueError):
        O.value_norm(v, "l3")


def test_norm_kind_reaches_prefill_and_decode():
    """prefill(norm=...) multiplies Eq. 4 by the chosen norm and decode steps take the same norm of
    the tokens they append; a value row with one large channel ranks differently under l1 and linf."""
    rng = np.random.default_rng(9)
    T, d = 12, 8
    q, k, v = rng.normal(size=(T, d)), rng.normal(size=(T, d)), rng.normal(size=(T, d))
    for kd in ("l1", "l2", "linf"):
        r = O.prefill(q, k, v, 0.3, norm=kd)
        np.testing.assert_array_equal(r["n1"], O.value_norm(v, kd))
        np.testing.assert_array_equal(r["I"], r["S"] * O.value_norm(v, kd))
        st = O.DecodeState(k, v, r["S"], r["n1"], np.arange(T), T, norm=kd)
        vn = rng.normal(size=d)
        O.decode_step(st, rng.normal(size=d), rng.normal(size=d), vn, 0.3, B=T + 1, F=0, R=1)
        assert st.n1[-1] == O.value_norm(vn, kd)[0]
    spike = np.zeros(d); spike[0] = 3.0           # l1 3, linf 3
    flat = np.full(d, 1.0)                        # l1 8, linf 1
    both = np.stack([spike, flat])
    assert O.value_norm(both, "l1")[0] < O.value_norm(both, "l1")[1]
    assert O.value_norm(both, "linf")[0] > O.value_norm(both, "linf")[1]


def test_importance_is_product():
    S = np.array([0.5, 2.0, 0.0])
    n = np.array([4.0, 0.25, 9.0])
    np.testing.assert_array_equal(O.importance(S, n), [2.0, 0.5, 0.0])


# -------------------------------------------------------------------- selection
@pytest.mark.parametrize("seed", range(6))
def test_select_matches_brute_force_with_ties(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(6, 14))
    I = rng.integers(0, 4, size=T).astype(float)      # many exact ties
    F = int(rng.integers(0, 3))
    R = int(rng.integers(0, 3))
    B = int(rng.integers(F + R, T + 2))
    got = O.select_keep(I, B, F, R)
    assert list(got) == brute_select(I.tolist(), B, F, R)


def test_select_properties():
    rng = np.random.default_rng(3)
    T, B, F, R = 100, 40, 4, 10
    I = rng.random(T)
    kept = O.select_keep(I, B, F, R)
    assert len(kept) == B and np.all(np.diff(kept) > 0)
    assert set(range(F)) <= set(kept) and set(range(T - R, T)) <= set(kept)
    mid_kept = [i for i in kept if F <= i < T - R]
    mid_drop = [i for i in range(F, T - R) if i not in set(kept)]
    assert min(I[mid_kept]) >= max(I[mid_drop])
    # sink + window only (the StreamingLLM policy) when the budget is F + R
    np.testing.assert_array_equal(O.select_keep(I, F + R, F, R), list(range(F)) + list(range(T - R, T)))
    # budget >= T keeps everything
    np.testing.assert_array_equal(O.select_keep(I, T, F, R), np.arange(T))
    np.testing.assert_array_equal(O.select_keep(I, T + 7, F, R), np.arange(T))
    with pytest.raises(ValueError):
        O.select_keep(I, 5, 4, 10)


def test_tie_goes_to_lower_index():
    I = np.array([9, 1, 1, 1, 1, 9], dtype=float)
    np.testing.assert_array_equal(O.select_keep(I, 4, 1, 1), [0, 1, 2, 5])


def test_equal_norms_reduce_to_attention_only():
    """With all value norms equal Eq. 4 ranks like Eq. 2 / Eq. 3 alone."""
    rng = np.random.default_rng(9)
    T, d = 64, 8
    q, k = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    v = rng.choice([-1.0, 1.0], size=(T, d)) * 0.37          # every row has l1 norm 0.37 d
    for window in (None, 16):
        r = O.prefill(q, k, v, 0.35, window=window)
        np.testing.assert_array_equal(O.select_keep(r["I"], 30, 2, 8), O.select_keep(r["S"], 30, 2, 8))


def test_value_scaling_and_single_token_boost():
    rng = np.random.default_rng(10)
    T, d = 48, 8
    q, k, v = (rng.normal(size=(T, d)) for _ in range(3))
    base = O.prefill(q, k, v, 0.35)
    kept = O.select_keep(base["I"], 20, 2, 4)
    np.testing.assert_array_equal(O.select_keep(O.prefill(q, k, 3.5 * v, 0.35)["I"], 20, 2, 4), kept)
    dropped = [i for i in range(2, T - 4) if i not in set(kept)][0]
    v2 = v.copy()
    v2[dropped] *= 1e6
    assert dropped in set(O.select_keep(O.prefill(q, k, v2, 0.35)["I"], 20, 2, 4))
    held = [i for i in kept if 2 <= i < T - 4][0]
    v3 = v.copy()
    v3[held] *= 1e-9
    assert held not in set(O.select_keep(O.prefill(q, k, v3, 0.35)["I"], 20, 2, 4))


def test_low_norm_sinks_are_evicted_without_F_and_kept_with_F():
    """The sink argument of the method: huge attention, near-zero value norm."""
    rng = np.random.default_rng(12)
    T, d = 64, 16
    q, k, v = (rng.normal(size=(T, d)) for _ in range(3))
    u = np.ones(d) / math.sqrt(d)
    q += 4 * u
    k[:2] += 4 * u
    v[:2] *= 1e-4
    r = O.prefill(q, k, v, 1 / math.sqrt(d))
    assert r["S"][:2].min() > np.sort(r["S"])[-3] * 0.99          # sinks dominate attention
    assert not {0, 1} & set(O.select_keep(r["I"], 32, 0, 8))      # value-aware score drops them
    assert {0, 1} <= set(O.select_keep(r["S"], 32, 0, 8))         # attention-only keeps them
    assert {0, 1} <= set(O.select_keep(r["I"], 32, 2, 8))         # sink retention keeps them


def test_compact_is_bitwise_gather():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(20, 6)).astype(np.float32)
    kept = np.array([0, 3, 4, 19])
    out = O.compact_rows(x, kept)
    assert out.tobytes() == b"".join(x[i].tobytes() for i in kept)
    assert O.compact_rows(x, np.arange(20)).tobytes() == x.tobytes()


# ----------------------------------------------------------------------- decode
def _state(q, k, v, scale, B, F, R, window=None):
    T = q.shape[0]
    r = O.prefill(q, k, v, scale, window=window)
    kept = O.select_keep(r["I"], B, F, R)
    return O.DecodeState(k, v, r["S"], r["n1"], kept, T, window=window, window_rows=r["window_rows"]), r


@pytest.mark.parametrize("window", [None, 5, 1000])
def test_prefill_decode_consistency(window):
    """No eviction (budget > T+steps): prefill on T tokens + decode steps must
    equal prefill on the longer prompt, and out must equal row T of A V."""
    rng = np.random.default_rng(21)
    T, d, steps = 12, 4, 3
    q, k, v = (rng.normal(size=(T + steps, d)) for _ in range(3))
    scale = 0.5
    st, _ = _state(q[:T], k[:T], v[:T], scale, T + steps + 1, 2, 3, window)
    for s in range(steps):
        res = O.decode_step(st, q[T + s], k[T + s], v[T + s], scale, T + steps + 1, 2, 3)
        full = O.prefill(q[: T + s + 1], k[: T + s + 1], v[: T + s + 1], scale, window=window)
        np.testing.assert_allclose(res["out"], full["a"][-1] @ v[: T + s + 1], rtol=1e-12)
        np.testing.assert_allclose(st.indicator(), full["S"], rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(st.importance(), full["I"], rtol=1e-12, atol=1e-15)
        assert res["evicted"] == -1 and abs(res["p"].sum() - 1) < 1e-14


def test_decode_eviction_invariants():
    rng = np.random.default_rng(22)
    T, d, B, F, R, steps = 40, 8, 16, 2, 4, 12
    q, k, v = (rng.normal(size=(T + steps, d)) for _ in range(3))
    st, _ = _state(q[:T], k[:T], v[:T], 0.35, B, F, R)
    for s in range(steps):
        t = T + s
        before = sum(st.S)
        res = O.decode_step(st, q[t], k[t], v[t], 0.35, B, F, R)
        assert len(st.pos) == B and st.pos == sorted(st.pos)
        assert set(range(F)) <= set(st.pos) and set(range(t - R + 1, t + 1)) <= set(st.pos)
        e = res["evicted"]
        assert F <= e <= t - R
        I, pos = res["I"], res["pos"]
        elig = [I[i] for i, p in enumerate(pos) if F <= p <= t - R]
        assert res["I_evicted"] == min(elig)
        # Eq. 2 adds exactly one unit of probability mass per step before the eviction
        assert abs(sum(I / np.array([st_n for st_n in _norms(res, st, v, k)])) - (before + 1)) < 1e-9


def _norms(res, st, v, k):
    # value norms of the entries listed in res["pos"], recomputed from the inputs
    return [np.abs(v[p]).sum() for p in res["pos"]]


def test_decode_tie_evicts_highest_position():
    """Equal importances among eligible entries: the largest position goes."""
    T, d, B = 6, 2, 6
    q = np.zeros((T + 1, d))
    k = np.ones((T + 1, d))
    v = np.ones((T + 1, d))
    r = O.prefill(q[:T], k[:T], v[:T], 1.0)
    st = O.DecodeState(k[:T], v[:T], np.ones(T), r["n1"], np.arange(T), T)   # flat indicator by hand
    res = O.decode_step(st, q[T], k[T], v[T], 1.0, B, 1, 2)
    # all eligible (positions 1..4) have S = 1 + 1/7: tie -> position 4 evicted
    assert res["evicted"] == 4 and res["runner_up"] == 3


def test_decode_equal_norms_is_attention_only_argmin():
    rng = np.random.default_rng(23)
    T, d, B, F, R = 30, 4, 12, 1, 3
    q, k = rng.normal(size=(T + 1, d)), rng.normal(size=(T + 1, d))
    v = rng.choice([-1.0, 1.0], size=(T + 1, d))
    st, _ = _state(q[:T], k[:T], v[:T], 0.5, B, F, R)
    res = O.decode_step(st, q[T], k[T], v[T], 0.5, B, F, R)
    S = res["I"] / d
    elig = [(S[i], -p) for i, p in enumerate(res["pos"]) if F <= p <= T - R]
    assert res["evicted"] == -min(elig)[1]


def test_window_decode_drops_old_rows_and_long_window_is_h2o():
    rng = np.random.default_rng(24)
    T, d, B, F, R, steps, w = 24, 4, 10, 1, 2, 8, 4
    q, k, v = (rng.normal(size=(T + steps, d)) for _ in range(3))
    st_w, _ = _state(q[:T], k[:T], v[:T], 0.5, B, F, R, window=w)
    st_big, _ = _state(q[:T], k[:T], v[:T], 0.5, B, F, R, window=10_000)
    st_h, _ = _state(q[:T], k[:T], v[:T], 0.5, B, F, R)
    for s in range(steps):
        t = T + s
        rw = O.decode_step(st_w, q[t], k[t], v[t], 0.5, B, F, R)
        rb = O.decode_step(st_big, q[t], k[t], v[t], 0.5, B, F, R)
        rh = O.decode_step(st_h, q[t], k[t], v[t], 0.5, B, F, R)
        assert rb["evicted"] == rh["evicted"]
        np.testing.assert_allclose(rb["I"], rh["I"], rtol=1e-12)
        # windowed mass before eviction: the last w rows each summed to 1, minus what evicted tokens held
        assert rw["I"].shape[0] == B + 1
        assert st_w.hist.shape == (w, B)
    # after more than w steps no prefill row is left in the history
    assert steps > w


def test_forced_eviction_only_within_tolerance():
    rng = np.random.default_rng(25)
    T, d, B, F, R = 20, 4, 8, 1, 2
    q, k, v = (rng.normal(size=(T + 1, d)) for _ in range(3))
    st, _ = _state(q[:T], k[:T], v[:T], 0.5, B, F, R)
    import copy
    st2 = copy.deepcopy(st)
    res = O.decode_step(st, q[T], k[T], v[T], 0.5, B, F, R)
    with pytest.raises(ValueError):
        O.decode_step(st2, q[T], k[T], v[T], 0.5, B, F, R, force_evict=res["runner_up"], tie_tol=1e-12)


# ------------------------------------------------------------------ Appendix A hyper-parameters
def _appendix_a_rows():
    rows = []
    with open(os.path.join(GOLD, "appendix_a_presets.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            left, right = line.split("|")
            method, model, vatp, T, ratio = left.split()
            rows.append((method, model, bool(int(vatp)), int(T), float(ratio), [int(x) for x in right.split()]))
    return rows


def test_appendix_a_split_matches_the_papers_values():
    """tests/golden/appendix_a_presets.txt holds what Appendix A states (k/2 + k/2 for H2O; k-10, 10 and
    w = 400 for Scissorhands; F = 20 / 40), written out by hand for the budgets of the throughput table."""
    rows = _appendix_a_rows()
    assert len(rows) >= 9
    for method, model, vatp, T, ratio, (k, F, R, w, chosen) in rows:
        s = O.appendix_a_split(method, T, ratio, model, vatp=vatp)
        assert (s["B"], s["F"], s["R"], s["w"] or 0) == (k, F, R, w), (method, model, ratio)
        assert s["n_scored"] + s["F"] == chosen and s["n_scored"] + s["F"] + s["R"] == k


def test_appendix_a_split_invariants_and_the_product_presets():
    """Every split is a valid argument of select_keep (F + R <= B, kept count = B), tiny budgets
    included; the product's own preset table (written separately) gives the same numbers."""
    from paper_2406_12335_b200 import presets
    rng = np.random.default_rng(5)
    for method in ("h2o", "scissorhands"):
        for model in ("llama2-7b-chat", "vicuna-v1.5-7b-16k"):
            for T in (7, 33, 100, 1001, 4096, 18409):
                for ratio in (0.1, 0.25, 0.5, 1.0):
                    for vatp in (True, False):
                        s = O.appendix_a_split(method, T, ratio, model, vatp=vatp)
                        assert 0 <= s["F"] and 0 <= s["R"] and s["F"] + s["R"] <= s["B"] <= T
                        assert s["n_scored"] == s["B"] - s["F"] - s["R"] >= 0
                        kept = O.select_keep(rng.random(T), s["B"], s["F"], s["R"])
                        assert len(kept) == s["B"]
                        assert set(range(s["F"])) <= set(kept.tolist())
                        assert set(range(T - s["R"], T)) <= set(kept.tolist()) or s["B"] >= T
                        p = presets.appendix_a(method, T, ratio, model, sinks=vatp)
                        assert (p["budget"], p["n_sink"], p["n_recent"], p["window"]) == \
                            (s["B"], s["F"], s["R"], s["w"] or 0)
                        assert p["indicator"] == ("window" if s["w"] else "h2o")
    with pytest.raises(ValueError):
        O.appendix_a_split("fastgen", 100)


def test_workload5_is_the_scissorhands_split_at_half_budget():
    """The added timing workload (prompt 4096, batch 12, 128 steps: the paper's throughput measurements) carries
    Appendix A's Scissorhands split at 50%, as both the oracle's and the product's tables give it."""
    from paper_2406_12335_b200 import presets, synth
    wl = synth.CONFIGS[5]
    s = O.appendix_a_split("scissorhands", wl.seq_len, 0.5, "llama2-7b-chat")
    assert (wl.budget, wl.n_sink, wl.n_recent, wl.window, wl.indicator) == (s["B"], s["F"], s["R"], s["w"], "window")
    assert (wl.batch, wl.heads, wl.head_dim, wl.seq_len, wl.decode_steps) == (12, 32, 128, 4096, 128)
    p = presets.appendix_a("scissorhands", wl.seq_len, 0.5)
    assert (p["budget"], p["n_sink"], p["n_recent"], p["window"]) == (wl.budget, wl.n_sink, wl.n_recent, wl.window)


# ------------------------------------------------------------------ grouped-query attention (Limitations)
def _loop_group_indicator(qg, k, scale):
    """Mean over the group's heads of the accumulated attention, by explicit loops with math.exp."""
    G, T, d = qg.shape
    S = [0.0] * T
    for g in range(G):
        for j in range(T):
            logits = [scale * sum(float(qg[g, j, c]) * float(k[i, c]) for c in range(d)) for i in range(j + 1)]
            m = max(logits)
            e = [math.exp(x - m) for x in logits]
            z = math.fsum(e)
            for i in range(j + 1):
                S[i] += e[i] / z / G
    return np.array(S)


def test_gqa_prefill_matches_loops_and_reductions():
    rng = np.random.default_rng(11)
    G, T, d = 3, 7, 4
    qg, k, v = rng.normal(size=(G, T, d)), rng.normal(size=(T, d)), rng.normal(size=(T, d))
    r = O.prefill_gqa(qg, k, v, 0.5)
    assert np.allclose(r["S"], _loop_group_indicator(qg, k, 0.5), rtol=1e-12, atol=1e-14)
    assert np.allclose(r["I"], r["S"] * np.abs(v).sum(1), rtol=1e-14)
    assert abs(r["S"].sum() - T) < 1e-12                       # a mean of G indicators that each sum to T
    # one head per group is plain multi-head attention
    one = O.prefill_gqa(qg[:1], k, v, 0.5)
    mha = O.prefill(qg[0], k, v, 0.5)
    assert np.array_equal(one["S"], mha["S"]) and np.array_equal(one["I"], mha["I"]) and np.array_equal(one["lse"][0], mha["lse"])
    # identical query heads change nothing either
    same = O.prefill_gqa(np.stack([qg[0]] * 4), k, v, 0.5)
    assert np.allclose(same["S"], mha["S"], rtol=1e-13)
    # the group mean really mixes the heads: it differs from every single head's indicator and is their average
    assert all(not np.allclose(r["S"], r["S_heads"][g]) for g in range(G))
    assert np.allclose(r["S"], r["S_heads"].mean(axis=0), rtol=1e-14)
    # a head that puts all its mass on key 0 lifts S_0 by exactly T / G over the other heads' share
    hot = qg.copy(); kk = k.copy()
    kk[0] = 0; kk[0, 0] = 200.0
    hot[1] = 0; hot[1, :, 0] = 1.0                             # head 1: logit 100 on key 0, 0 elsewhere
    rh = O.prefill_gqa(hot, kk, v, 0.5)
    assert abs(rh["S_heads"][1][0] - T) < 1e-9 and np.all(rh["S_heads"][1][1:] < 1e-9)
    # windowed indicator (Eq. 3) under the same group mean; w >= T is the accumulated one
    rw = O.prefill_gqa(qg, k, v, 0.5, window=3)
    assert abs(rw["S"].sum() - 3) < 1e-12
    assert np.allclose(O.prefill_gqa(qg, k, v, 0.5, window=T)["S"], r["S"], rtol=1e-14)


def test_gqa_decode_step_matches_prefill_on_the_longer_prompt():
    """Prefill on T tokens + one grouped decode step with nothing evicted = prefill on T + 1 tokens: the
    indicator (group mean) and every head's output row."""
    rng = np.random.default_rng(12)
    G, T, d = 4, 9, 6
    qg, k, v = rng.normal(size=(G, T + 1, d)), rng.normal(size=(T + 1, d)), rng.normal(size=(T + 1, d))
    scale = 0.4
    short = O.prefill_gqa(qg[:, :T], k[:T], v[:T], scale)
    full = O.prefill_gqa(qg, k, v, scale)
    st = O.DecodeState(k[:T], v[:T], short["S"], short["n1"], np.arange(T), T)
    res = O.decode_step(st, qg[:, T], k[T], v[T], scale, B=T + 5, F=0, R=0)
    assert res["evicted"] == -1 and res["out"].shape == (G, d)
    assert np.allclose(st.indicator(), full["S"], rtol=1e-12)
    for g in range(G):
        a = O.attention_probs(qg[g], k, scale)
        assert np.allclose(res["out"][g], a[T] @ v, rtol=1e-12)
    # one head per group is the ordinary step
    st1 = O.DecodeState(k[:T], v[:T], short["S"], short["n1"], np.arange(T), T)
    st2 = O.DecodeState(k[:T], v[:T], short["S"], short["n1"], np.arange(T), T)
    r1 = O.decode_step(st1, qg[:1, T], k[T], v[T], scale, B=4, F=1, R=2)
    r2 = O.decode_step(st2, qg[0, T], k[T], v[T], scale, B=4, F=1, R=2)
    assert r1["evicted"] == r2["evicted"] and np.allclose(r1["out"][0], r2["out"]) and np.allclose(st1.S, st2.S)
    # the step evicts on the group-mean indicator: with equal norms the victim is the arg-min of the mean
    st3 = O.DecodeState(k[:T], np.ones((T, d)), short["S"], np.full(T, float(d)), np.arange(T), T)
    r3 = O.decode_step(st3, qg[:, T], k[T], np.ones(d), scale, B=T, F=0, R=1)
    mean_after = short["S"] + r3["p"][:T]
    assert r3["evicted"] == int(np.argmin(mean_after))
    # history window (Eq. 3) with grouped queries: the group-mean row enters the history; prefill + steps = longer prefill
    for w in (4, 1, 50):
        shortw = O.prefill_gqa(qg[:, :T - 2], k[:T - 2], v[:T - 2], scale, window=w)
        # the window rows are the mean over heads of each head's last rows, written out with loops
        for r in range(shortw["window_rows"].shape[0]):
            j = (T - 2) - shortw["window_rows"].shape[0] + r
            for i in range(T - 2):
                want = sum(O.attention_probs(qg[g, :T - 2], k[:T - 2], scale)[j, i] for g in range(G)) / G
                assert abs(shortw["window_rows"][r, i] - want) < 1e-14
        stw = O.DecodeState(k[:T - 2], v[:T - 2], shortw["S"], shortw["n1"], np.arange(T - 2), T - 2, window=w,
                            window_rows=shortw["window_rows"])
        for step in range(3):
            tt = T - 2 + step
            O.decode_step(stw, qg[:, tt], k[tt], v[tt], scale, B=T + 5, F=0, R=0)
            fullw = O.prefill_gqa(qg[:, :tt + 1], k[:tt + 1], v[:tt + 1], scale, window=w)
            assert np.allclose(stw.indicator(), fullw["S"], rtol=1e-12, atol=1e-15)
            assert abs(stw.indicator().sum() - min(w, tt + 1)) < 1e-12


# ----------------------------------------------------------------- attention output (Section 3.1)
def test_attention_output_matches_loops_and_closed_forms():
    rng = np.random.default_rng(5)
    T, d = 9, 4
    q, k, v = rng.standard_normal((T, d)), rng.standard_normal((T, d)), rng.standard_normal((T, d))
    scale = 0.5
    a = brute_attention(q.tolist(), k.tolist(), scale)
    out = O.attention_output(O.attention_probs(q, k, scale), v)
    for j in range(T):
        for c in range(d):
            acc = 0.0
            for i in range(j + 1):
                acc += a[j][i] * float(v[i][c])
            assert abs(out[j, c] - acc) < 1e-12
    # a transposed probability matrix would put future values into early rows
    assert np.abs(O.attention_probs(q, k, scale).T @ v - out).max() > 1e-3
    # the first query sees only the first token
    np.testing.assert_allclose(out[0], v[0], rtol=0, atol=1e-15)
    # constant values come back unchanged (rows of a sum to one)
    ones = np.full((T, d), 3.25)
    np.testing.assert_allclose(O.attention_output(O.attention_probs(q, k, scale), ones), ones, rtol=0, atol=1e-13)
    # uniform attention (all keys equal): row j is the mean of the first j + 1 values
    ku = np.tile(k[:1], (T, 1))
    outu = O.prefill(q, ku, v, scale)["out"]
    for j in range(T):
        np.testing.assert_allclose(outu[j], v[: j + 1].mean(axis=0), rtol=0, atol=1e-13)


def test_attention_output_last_row_is_the_decode_steps_output():
    """Row T of the prompt's output equals what the decode step returns for token T (no eviction yet)."""
    rng = np.random.default_rng(6)
    T, d = 12, 8
    q, k, v = rng.standard_normal((T + 1, d)), rng.standard_normal((T + 1, d)), rng.standard_normal((T + 1, d))
    scale = d ** -0.5
    st, _ = _state(q[:T], k[:T], v[:T], scale, B=T + 4, F=1, R=2)
    res = O.decode_step(st, q[T], k[T], v[T], scale, T + 4, 1, 2)
    np.testing.assert_allclose(res["out"], O.prefill(q, k, v, scale)["out"][T], rtol=0, atol=1e-12)


def test_attention_row_is_a_row_of_the_matrix_form():
    rng = np.random.default_rng(8)
    T, d = 11, 5
    q, k, v = rng.standard_normal((T, d)), rng.standard_normal((T, d)), rng.standard_normal((T, d))
    full = O.prefill(q, k, v, 0.4)
    a = brute_attention(q.tolist(), k.tolist(), 0.4)
    for j in (0, 3, T - 1):
        o, lse = O.attention_row(q[j], k[: j + 1], v[: j + 1], 0.4)
        np.testing.assert_allclose(o, full["out"][j], rtol=0, atol=1e-14)
        assert abs(lse - full["lse"][j]) < 1e-13
        # against the loops: probabilities of row j times the values
        want = [sum(a[j][i] * float(v[i][c]) for i in range(j + 1)) for c in range(d)]
        np.testing.assert_allclose(o, want, rtol=0, atol=1e-13)
