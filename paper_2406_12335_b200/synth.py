"""Seeded synthetic workloads shaped like LLaMA2-7B attention inputs.

This module only draws random tensors (torch's generators); it contains none
of the pruning method's arithmetic and imports neither the CUDA binding nor
the CPU oracle, so both sides of a parity test can be fed from it.

Structure of the data (what the paper reports about real activations):
value-vector l1 norms are far from uniform across tokens, the first two
tokens are attention sinks with massive attention but near-zero value norm,
and an occasional token has a much larger norm than its neighbours.

Recipe, per layer (generator seeded by (seed, config id, layer)):
  * Q, K entries ~ N(0, 1); the softmax scale is 1/sqrt(d), so logits ~ N(0, 1).
  * sinks: one random unit direction u per (batch, head); every query gets
    q += alpha*u and keys 0 and 1 get k += alpha*u with alpha^2/sqrt(d) = ln T,
    which lifts each sink logit by about ln T.
  * V rows = g * exp(sigma*z), g ~ N(0, I_d), z ~ N(0, 1) per token; rows 0 and
    1 are scaled by 1e-3; `boost` random positions per layer (config 4) by 10.
  * decode-step q, k, v: same distributions (queries carry the sink bias).
Values are rounded once to the workload dtype.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

SEED = 240612335


@dataclass(frozen=True)
class Workload:
    cid: int
    name: str
    dtype: str            # "f32" | "bf16"
    batch: int
    heads: int
    layers: int
    head_dim: int
    seq_len: int
    budget: int
    n_sink: int
    n_recent: int
    indicator: str        # "h2o" | "window"
    window: int
    decode_steps: int
    sigma_lo: float = 1.0
    sigma_hi: float = 1.0
    boost: int = 0
    norm: str = "l1"      # value norm of Eq. 4: "l1" (the method) | "l2" | "linf" (the Ablation Study's variants)

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def sigma(self, layer: int) -> float:
        if self.layers == 1:
            return self.sigma_lo
        return self.sigma_lo + (self.sigma_hi - self.sigma_lo) * layer / (self.layers - 1)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _round_half_up(x: float) -> int:
    return int(math.floor(x + 0.5))


CONFIGS = {
    0: Workload(0, "tiny_f32", "f32", 1, 2, 1, 64, 512, 256, 0, 32, "h2o", 0, 16),
    1: Workload(1, "llama2_7b_layer_4k", "bf16", 1, 32, 1, 128, 4096, 2048, 0, 128, "h2o", 0, 256),
    2: Workload(2, "llama2_7b_stack_8k_b8", "bf16", 8, 32, 32, 128, 8192, _round_half_up(0.2 * 8192), 0, 256,
                "h2o", 0, 128, sigma_lo=0.5, sigma_hi=1.5),
    3: Workload(3, "windowed_2k_b16", "bf16", 16, 32, 1, 128, 2048, 1024, 0, 10, "window", 256, 512),
    4: Workload(4, "long_32k", "bf16", 1, 32, 32, 128, 32768, _round_half_up(0.1 * 32768), 0, 512, "h2o", 0, 64,
                boost=64),
    # the shape of the paper's throughput measurements ("Inference Efficiency": prompt 4096, 128 generated tokens,
    # batch 12) with Appendix A's Scissorhands split at a 50% budget (10 local tokens, history window 400) and
    # F = 20 kept leading tokens; other budgets of that table: see presets.appendix_a
    5: Workload(5, "throughput_table_b12_4k", "bf16", 12, 32, 1, 128, 4096, 2048, 20, 10, "window", 400, 128),
}


def _gen(wl: Workload, layer: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(SEED + 1_000_003 * wl.cid + 7919 * layer + 104_729 * stream)
    return g


def sink_direction(wl: Workload, layer: int, device="cpu") -> torch.Tensor:
    g = _gen(wl, layer, 0, device)
    u = torch.randn(wl.batch, wl.heads, 1, wl.head_dim, generator=g, device=device, dtype=torch.float32)
    return u / u.norm(dim=-1, keepdim=True)


def sink_alpha(wl: Workload) -> float:
    return math.sqrt(math.log(wl.seq_len) * math.sqrt(wl.head_dim))


def prefill_inputs(wl: Workload, layer: int = 0, device="cpu"):
    """(q, k, v), each [batch, heads, seq_len, head_dim] in the workload dtype."""
    b, h, T, d = wl.batch, wl.heads, wl.seq_len, wl.head_dim
    u = sink_direction(wl, layer, device)
    alpha = sink_alpha(wl)
    out = []
    for stream in (1, 2):
        g = _gen(wl, layer, stream, device)
        x = torch.randn(b, h, T, d, generator=g, device=device, dtype=torch.float32)
        if stream == 1:
            x += alpha * u
        else:
            x[:, :, : min(2, T)] += alpha * u
        out.append(x.to(wl.torch_dtype))
        del x
    g = _gen(wl, layer, 3, device)
    v = torch.randn(b, h, T, d, generator=g, device=device, dtype=torch.float32)
    z = torch.randn(b, h, T, 1, generator=g, device=device, dtype=torch.float32)
    v *= torch.exp(wl.sigma(layer) * z)
    v[:, :, : min(2, T)] *= 1e-3
    if wl.boost:
        gp = torch.Generator(device="cpu")
        gp.manual_seed(SEED + 31 * wl.cid + layer)
        where = (torch.randperm(T - 2, generator=gp)[: wl.boost] + 2).to(device)
        v[:, :, where] *= 10.0
    out.append(v.to(wl.torch_dtype))
    return tuple(out)


def decode_inputs(wl: Workload, layer: int = 0, steps: int | None = None, device="cpu"):
    """(q, k, v), each [steps, batch, heads, head_dim] in the workload dtype."""
    steps = wl.decode_steps if steps is None else steps
    b, h, d = wl.batch, wl.heads, wl.head_dim
    u = sink_direction(wl, layer, device).squeeze(2)
    g = _gen(wl, layer, 4, device)
    q = torch.randn(steps, b, h, d, generator=g, device=device, dtype=torch.float32) + sink_alpha(wl) * u
    k = torch.randn(steps, b, h, d, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(steps, b, h, d, generator=g, device=device, dtype=torch.float32)
    z = torch.randn(steps, b, h, 1, generator=g, device=device, dtype=torch.float32)
    v *= torch.exp(wl.sigma(layer) * z)
    return q.to(wl.torch_dtype), k.to(wl.torch_dtype), v.to(wl.torch_dtype)
