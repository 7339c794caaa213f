"""Hyper-parameter presets of the paper's Appendix A ("Implementation Details") as keyword
arguments for `vatp.make_params` / `vatp.params_for`.

Host-side bookkeeping only: how a KV budget, given as a fraction of the prompt length, is divided
between always-kept leading tokens, importance-selected tokens and the local window, and which
indicator (Eq. 2 or Eq. 3) the host method uses.
"""
from __future__ import annotations

import math

SINK_TOKENS = {"llama2-7b-chat": 20, "vicuna-v1.5-7b-16k": 40}   # first F tokens VATP always keeps
SCISSORHANDS_LOCAL = 10                                          # local window of Scissorhands
SCISSORHANDS_HISTORY = 400                                       # its history window w (queries)


def appendix_a(method: str, prompt_len: int, ratio: float = 0.5, model: str = "llama2-7b-chat",
               sinks: bool = True) -> dict:
    """Keyword arguments (budget, n_sink, n_recent, indicator, window) for one prompt.

    method "h2o": accumulated attention (Eq. 2); half of the budget is the local window, the
    other half is chosen by importance.  method "scissorhands": attention of the last 400 queries
    (Eq. 3); 10 local tokens, the rest chosen by importance.  With `sinks` the first 20 (LLaMA2) or
    40 (Vicuna) tokens are kept as VATP does, counted inside the importance share so that exactly
    `budget` tokens survive; without, none (the unmodified host method).  The budget is
    round-half-up(ratio * prompt_len); shares that do not fit a tiny budget are cut, window first.
    """
    budget = int(math.floor(ratio * prompt_len + 0.5))
    if method == "h2o":
        recent, indicator, window = budget // 2, "h2o", 0
    elif method == "scissorhands":
        recent, indicator, window = SCISSORHANDS_LOCAL, "window", SCISSORHANDS_HISTORY
    else:
        raise ValueError(f"unknown method {method!r}")
    recent = min(recent, budget)
    n_sink = min(SINK_TOKENS[model], budget - recent) if sinks else 0
    return {"budget": budget, "n_sink": n_sink, "n_recent": recent, "indicator": indicator, "window": window}
