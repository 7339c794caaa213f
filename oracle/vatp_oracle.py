"""Float64 CPU oracle for Value-Aware Token Pruning (VATP).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what
the pruning path computes.  It is imported by the tests, by the smoke check
and by the CPU-baseline leg of the benchmark, and by nothing else.  It shares
no code with the CUDA library and never imports it.

Everything is float64 numpy, one (layer, batch, head) unit at a time.  The
full T x T causal attention matrix is materialised on purpose: the method's
quantities are *defined* on that matrix, and the oracle is the definition.

Notation follows the paper: a_i^t attention probability of query t on key i
(Eq. 1), S_k^t the indicator (Eq. 2 accumulated / Eq. 3 windowed), I_k^t the
importance S_k^t * ||v_k||_1 (Eq. 4), F the number of always-kept leading
tokens ("Attention Sink Tokens" paragraph), B the KV budget and R the local
(recent) window (Appendix A, implementation details).

Readings of points the paper leaves open are marked "reading:" below.

Pins (tests/test_oracle_*.py): harmonic-number closed forms for uniform
attention, row sums, sum of indicators = number of query rows, brute-force
triple loops on tiny inputs, w >= T reduction of Eq. 3 to Eq. 2, equal-norm
reduction of Eq. 4 to attention-only selection, sink+window special case,
prefill/decode consistency.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "attention_probs",
    "attention_output",
    "attention_row",
    "indicator_h2o",
    "indicator_window",
    "value_l1_norm",
    "value_norm",
    "importance",
    "select_keep",
    "appendix_a_split",
    "compact_rows",
    "prefill",
    "prefill_gqa",
    "DecodeState",
    "decode_step",
]


def _f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


def attention_probs(q, k, scale: float) -> np.ndarray:
    """Causal softmax attention matrix a[j, i] = a_i^j of Eq. 1.

    q, k: [T, d].  Logit s[j, i] = scale * <q_j, k_i>; query j sees keys
    i <= j only (Eq. 1 sums over i <= t).  Entries with i > j are exactly 0.
    reading: the paper never writes the softmax; scale is passed explicitly
    (1/sqrt(d) in all workloads).
    """
    q = _f64(q)
    k = _f64(k)
    T = q.shape[0]
    s = scale * (q @ k.T)
    causal = np.tril(np.ones((T, T), dtype=bool))
    s = np.where(causal, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)          # exp(-inf) = 0 above the diagonal
    return e / e.sum(axis=1, keepdims=True)


def row_logsumexp(q, k, scale: float) -> np.ndarray:
    """lse_j = log sum_{i<=j} exp(s[j, i]); the row normaliser of Eq. 1."""
    q = _f64(q)
    k = _f64(k)
    T = q.shape[0]
    s = scale * (q @ k.T)
    causal = np.tril(np.ones((T, T), dtype=bool))
    s = np.where(causal, s, -np.inf)
    m = s.max(axis=1)
    return m + np.log(np.exp(s - m[:, None]).sum(axis=1))


def attention_output(a: np.ndarray, v) -> np.ndarray:
    """The attention layer's output rows o_j = sum_{i<=j} a_i^j v_i (Section 3.1: the
    output is the probability-weighted sum of the value vectors, which is why
    Eq. 4 looks at their norms).  a: [T, T] from attention_probs, v: [T, d]."""
    return a @ _f64(v)


def attention_row(q_j, k, v, scale: float):
    """One query row of Eq. 1 on its own: query j = len(k) - 1 against the keys 0..j it may see.
    Returns (o_j, lse_j).  For prompts whose T x T matrix is too large to materialise; the same arithmetic
    as attention_probs / attention_output / row_logsumexp restricted to one row."""
    q_j, k, v = _f64(q_j), _f64(k), _f64(v)
    s = scale * (k @ q_j)
    m = s.max()
    e = np.exp(s - m)
    den = e.sum()
    return (e / den) @ v, m + np.log(den)


def indicator_h2o(a: np.ndarray) -> np.ndarray:
    """Eq. 2 at t = T-1: S_k = sum_{k <= j <= T-1} a_k^j (column sums)."""
    return a.sum(axis=0)


def indicator_window(a: np.ndarray, w: int, inclusive_extra: int = 0) -> np.ndarray:
    """Eq. 3 at t = T-1: column sums over the history window only.

    reading: the window holds the last w queries, j in [max(T-w, k), T-1]
    (the prose speaks of "the last w tokens").  Eq. 3 as printed has bounds
    max(t-w, k) <= j <= t, which is w+1 queries; inclusive_extra=1 gives that
    literal form.  When the window covers every row this is Eq. 2.
    """
    T = a.shape[0]
    first = max(T - (w + inclusive_extra), 0)
    return a[first:, :].sum(axis=0)


def value_l1_norm(v) -> np.ndarray:
    """||v_k||_1 over the head's d channels (the norm in Eq. 4)."""
    return np.abs(_f64(v)).sum(axis=1)


def value_norm(v, kind: str = "l1") -> np.ndarray:
    """Norm of every value row over the head's d channels, for the three kinds
    the Ablation Study compares (its table of norms): "l1" = sum of |v_c| (the
    one Eq. 4 uses), "l2" = square root of the sum of v_c^2, "linf" = the
    largest |v_c|."""
    x = np.abs(_f64(v))
    if x.ndim == 1:
        x = x[None, :]
    if kind == "l1":
        return x.sum(axis=1)
    if kind == "l2":
        return np.sqrt((x * x).sum(axis=1))
    if kind == "linf":
        return x.max(axis=1)
    raise ValueError("norm kind must be 'l1', 'l2' or 'linf'")


def importance(S: np.ndarray, n1: np.ndarray) -> np.ndarray:
    """Eq. 4: I_k = S_k * ||v_k||_1."""
    return _f64(S) * _f64(n1)


def select_keep(I, B: int, F: int, R: int) -> np.ndarray:
    """Indices kept after the one-shot prune of a T-token prompt, ascending.

    Kept set = first F tokens (sink retention) + last R tokens (local window)
    + the B-F-R highest-importance tokens of the middle range [F, T-R), so
    that exactly B survive (Appendix A: budget split into score-selected
    tokens and a local window; "Attention Sink Tokens": first F always kept).
    reading: F counts inside the budget.  Ties: the lower index outranks the
    higher (stable sort by descending importance).  T <= B keeps everything.
    """
    I = _f64(I)
    T = I.shape[0]
    if F < 0 or R < 0 or F + R > B:
        raise ValueError("need 0 <= F, 0 <= R, F + R <= B")
    if T <= B:
        return np.arange(T, dtype=np.int64)
    mid = np.arange(F, T - R, dtype=np.int64)
    order = mid[np.argsort(-I[mid], kind="stable")]
    top = order[: B - F - R]
    kept = np.concatenate([np.arange(0, F), top, np.arange(T - R, T)]).astype(np.int64)
    kept.sort()
    return kept


def appendix_a_split(method: str, prompt_len: int, ratio: float = 0.5, model: str = "llama2-7b-chat",
                     vatp: bool = True) -> dict:
    """Hyper-parameters of Appendix A ("Implementation Details") for one prompt.

    The KV budget k is a fraction of the prompt length (50% in the accuracy
    tables; 100/50/25% in the throughput table of "Inference Efficiency"),
    the same for every head and layer.  With H2O, k/2 tokens are chosen by
    importance and k/2 form the local window.  With Scissorhands, k-10 tokens
    are chosen by importance, the local window is 10 tokens and the history
    window is w = 400 queries.  VATP additionally keeps the first F tokens,
    F = 20 for LLaMA2-7B-chat and 40 for Vicuna-v1.5-7B-16k; the plain
    baselines (vatp=False) keep none.
    reading: k is rounded half up; for odd k the local window takes the
    floor; the F kept tokens count inside the importance-chosen share, so
    exactly k tokens survive; when the shares do not fit, the window is cut
    first to k and F to what is left.
    Returns B (= k), F, R, w (None for H2O) and n_scored = B - F - R.
    """
    k = int(np.floor(ratio * prompt_len + 0.5))
    if method == "h2o":
        R, w = k // 2, None
    elif method == "scissorhands":
        R, w = 10, 400
    else:
        raise ValueError("method must be 'h2o' or 'scissorhands'")
    F = {"llama2-7b-chat": 20, "vicuna-v1.5-7b-16k": 40}[model] if vatp else 0
    R = min(R, k)
    F = min(F, k - R)
    return {"B": k, "F": F, "R": R, "w": w, "n_scored": k - F - R}


def compact_rows(x: np.ndarray, kept: np.ndarray) -> np.ndarray:
    """Rows of x at the kept indices, in ascending index order, bit for bit."""
    return np.ascontiguousarray(np.asarray(x)[np.asarray(kept, dtype=np.int64)])


def prefill(q, k, v, scale: float, *, window: int | None = None, inclusive_extra: int = 0, norm: str = "l1"):
    """One unit's prefill quantities: dict with a, out, lse, S, n1, I (and the
    window rows a[T-w:, :] when the indicator is Eq. 3).  norm: which value
    norm Eq. 4 multiplies by ("l1" is the method; "l2" / "linf" are the
    ablation's variants); the key stays "n1" for all kinds."""
    a = attention_probs(q, k, scale)
    if window is None:
        S = indicator_h2o(a)
        rows = None
    else:
        S = indicator_window(a, window, inclusive_extra)
        first = max(a.shape[0] - (window + inclusive_extra), 0)
        rows = a[first:, :].copy()
    n1 = value_l1_norm(v) if norm == "l1" else value_norm(v, norm)
    return {
        "a": a,
        "out": attention_output(a, v),
        "lse": row_logsumexp(q, k, scale),
        "S": S,
        "n1": n1,
        "I": importance(S, n1),
        "window_rows": rows,
    }


def prefill_gqa(q_group, k, v, scale: float, *, window: int | None = None, norm: str = "l1"):
    """Grouped-query attention: the G query heads q_group[g] ([G, T, d]) of one KV group share the keys and
    values k, v ([T, d]), hence one cache and one kept set.  The Limitations section ("Compatibility with
    grouped-query attention") leaves this to future work and points at a group-wise score:
    reading: the indicator of a cached token is the MEAN over the group's query heads of its Eq. 2 (or Eq. 3)
    indicator, S_k = (1/G) sum_g S_k^(g); Eq. 4 multiplies it by the norm of the shared value row.  With G = 1
    this is `prefill`.  Returns dict with lse [G, T], S, n1, I, S_heads [G, T], and with a history window the
    group mean of the heads' last-w probability rows (window_rows: what the decode state keeps); no attention
    matrices."""
    q_group = _f64(q_group)
    if q_group.ndim != 3:
        raise ValueError("q_group must be [G, T, d]")
    per_head = []
    lse = []
    rows = None
    for g in range(q_group.shape[0]):
        a = attention_probs(q_group[g], k, scale)
        per_head.append(indicator_h2o(a) if window is None else indicator_window(a, window))
        lse.append(row_logsumexp(q_group[g], k, scale))
        if window is not None:
            r = a[max(a.shape[0] - window, 0):, :]
            rows = r.copy() if rows is None else rows + r
        del a
    S_heads = np.stack(per_head)
    S = S_heads.sum(axis=0) / q_group.shape[0]
    n1 = value_l1_norm(v) if norm == "l1" else value_norm(v, norm)
    return {"lse": np.stack(lse), "S": S, "n1": n1, "I": importance(S, n1), "S_heads": S_heads,
            "window_rows": None if rows is None else rows / q_group.shape[0]}


class DecodeState:
    """Pruned cache of one unit, as lists ordered by original position.

    pos[i]   original token position of cache entry i (ascending)
    K, V     rows of the cached keys / values (float64 copies of input bits)
    n1       value norm per entry (||v||_1 unless norm says otherwise)
    norm     kind of the value norm taken of tokens appended by decode steps
    S        H2O indicator per entry (Eq. 2), maintained incrementally
    hist     windowed mode only: the last <= w probability rows as a matrix
             [rows, entries] whose columns follow pos; Eq. 3 is re-summed from
             it every step (no subtraction).  A token that was not cached when
             an old row was produced has a 0 in that row; an evicted token's
             column is deleted.
    t        position of the next token to be generated
    """

    def __init__(self, k, v, S, n1, kept, T: int, *, window: int | None = None,
                 window_rows: np.ndarray | None = None, inclusive_extra: int = 0, norm: str = "l1"):
        kept = np.asarray(kept, dtype=np.int64)
        self.norm = norm
        self.pos = [int(p) for p in kept]
        self.K = [_f64(k)[p].copy() for p in kept]
        self.V = [_f64(v)[p].copy() for p in kept]
        self.n1 = [float(_f64(n1)[p]) for p in kept]
        self.S = [float(_f64(S)[p]) for p in kept]
        self.t = int(T)
        self.window = None if window is None else int(window) + int(inclusive_extra)
        self.hist = None
        if self.window is not None:
            rows = np.asarray(window_rows, dtype=np.float64)
            self.hist = rows[-self.window:][:, kept].copy()

    def indicator(self) -> np.ndarray:
        if self.window is None:
            return np.array(self.S, dtype=np.float64)
        return self.hist[-self.window:].sum(axis=0)

    def importance(self) -> np.ndarray:
        return self.indicator() * np.array(self.n1, dtype=np.float64)


def decode_step(state: DecodeState, q, k, v, scale: float, B: int, F: int, R: int,
                *, force_evict: int | None = None, tie_tol: float = 0.0,
                tie_abs: float = 0.0):
    """One generation step on the pruned cache (Eq. 1-4 at step t).

    Order of operations (reading: the new query also attends to the token that
    this step evicts, because S^t of Eq. 2/3 includes the j = t term):
      1. append the new token's (k, v) at position t;
      2. p = softmax(scale * <q, k_i>) over every cached entry, out = sum p_i v_i;
      3. indicator update: Eq. 2 adds p_i (the new token starts at its own
         probability, the j = k term); Eq. 3 appends the row to the history;
      4. I_i = S_i * ||v_i||_1;
      5. if more than B entries are cached, remove the lowest-importance entry
         among those that are neither one of the first F positions nor one of
         the R most recent positions (pos > t - R).  Ties: among equal
         importances the highest position goes (the lower index outranks it).

    force_evict: a position the caller wants evicted instead (used to keep a
    trajectory aligned after a tolerated near-tie); accepted only when its
    importance is within tie_tol (relative) + tie_abs (absolute) of the
    oracle's own minimum, otherwise ValueError.

    Grouped-query attention (see prefill_gqa): q may be [G, d], the new token's query under each head of the
    KV group.  Every head attends over the shared cache, out is [G, d], p is [G, entries], and the indicator
    advances by the mean of the heads' probabilities (Eq. 2), or that mean row enters the history (Eq. 3).

    Returns dict(out, p, evicted (position or -1), runner_up, I_evicted,
    I_runner_up, adopted (a forced near-tie was taken), I (importances before eviction), pos (positions before
    eviction)).
    """
    t = state.t
    state.pos.append(t)
    state.K.append(_f64(k).copy())
    state.V.append(_f64(v).copy())
    state.n1.append(float(value_norm(v, state.norm)[0]))
    state.S.append(0.0)
    if state.window is not None:
        state.hist = np.concatenate([state.hist, np.zeros((state.hist.shape[0], 1))], axis=1)

    Kmat = np.stack(state.K)
    Vmat = np.stack(state.V)
    qv = _f64(q)
    if qv.ndim == 2:                         # grouped-query attention: one softmax per query head of the group
        s = scale * (qv @ Kmat.T)
        e = np.exp(s - s.max(axis=1, keepdims=True))
        p_heads = e / e.sum(axis=1, keepdims=True)
        out = p_heads @ Vmat
        p = p_heads.sum(axis=0) / qv.shape[0]     # what the indicator advances by
    else:
        s = scale * (Kmat @ qv)
        e = np.exp(s - s.max())
        p = e / e.sum()
        out = p @ Vmat

    for i in range(len(state.pos)):
        state.S[i] += float(p[i])
    if state.window is not None:
        state.hist = np.concatenate([state.hist, p[None, :]], axis=0)[-state.window:]

    I = state.importance()
    pos_before = list(state.pos)
    res = {"out": out, "p": p, "evicted": -1, "runner_up": -1,
           "I_evicted": None, "I_runner_up": None, "I": I, "pos": pos_before, "adopted": False}

    if len(state.pos) > B:
        elig = [i for i, pp in enumerate(state.pos) if pp >= F and pp <= t - R]
        # rank: descending importance, ties by ascending position; the last goes
        elig.sort(key=lambda i: (-I[i], state.pos[i]))
        victim = elig[-1]
        runner = elig[-2] if len(elig) > 1 else -1
        if force_evict is not None and force_evict != state.pos[victim]:
            cand = state.pos.index(force_evict)
            if cand not in elig:
                raise ValueError("forced eviction of a protected position")
            gap = abs(I[cand] - I[victim])
            if gap > tie_tol * max(abs(I[victim]), abs(I[cand])) + tie_abs:
                raise ValueError("forced eviction is not a near-tie")
            victim = cand
            res["adopted"] = True
        res["evicted"] = state.pos[victim]
        res["I_evicted"] = float(I[victim])
        if runner >= 0:
            res["runner_up"] = state.pos[runner]
            res["I_runner_up"] = float(I[runner])
        for lst in (state.pos, state.K, state.V, state.n1, state.S):
            del lst[victim]
        if state.window is not None:
            state.hist = np.delete(state.hist, victim, axis=1)
    state.t = t + 1
    return res
