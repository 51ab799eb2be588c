"""Seeded synthetic inputs for the DASC hot path.

This module only draws inputs (decay parameters, states, token streams, slot
lists).  It holds none of the method's arithmetic and is the one module that
both the CUDA tests/benchmark and the CPU oracle's callers share.

Recipe (the benchmark configurations' own wording):
  * per-unit decay rate log-uniform in [lo, hi]; the plan sees it as
    ``A_log = ln(rate)`` with ``dt_bias = 0``;
  * q, k ~ N(0,1), L2-normalised over d_k per (token, head) in fp32, then cast;
  * v ~ N(0,1);  beta = sigmoid(N(0,1));  log alpha = -softplus(N(0,1)) * rate;
  * dense states ~ N(0,1) fp32.
All draws come from one ``torch.Generator`` seeded by the caller, in a fixed
order, so a (seed, shape, device) triple names one input set.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

KDA, GDN = 0, 1


def generator(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def decay_rates(gen, n_layers, n_heads, units_per_head, lo, hi, device="cpu") -> torch.Tensor:
    """Log-uniform rates in [lo, hi], fp32, shape [L, H, units_per_head]."""
    u = torch.rand((n_layers, n_heads, units_per_head), generator=gen, device=device, dtype=torch.float32)
    return torch.exp(u * (math.log(hi) - math.log(lo)) + math.log(lo))


def skew_layers(rates: torch.Tensor, skew: float) -> torch.Tensor:
    """Imbalanced per-layer decay profile: layer l's rates are multiplied by exp(skew * (l/(L-1) - 1/2)), so the
    first layers decay slowly (long horizons) and the last ones fast.  skew = 0 leaves the rates as drawn."""
    L = rates.shape[0]
    if skew == 0.0 or L < 2:
        return rates
    pos = torch.arange(L, dtype=torch.float32, device=rates.device) / (L - 1) - 0.5
    return rates * torch.exp(skew * pos).view(L, *([1] * (rates.dim() - 1)))


def decay_params(rates: torch.Tensor):
    """(A_log, dt_bias) such that exp(A_log) = rate and dt_bias = 0."""
    return torch.log(rates).to(torch.float32), torch.zeros_like(rates)


def states(gen, shape, device="cpu") -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def special_values_(state: torch.Tensor, gen) -> torch.Tensor:
    """Sprinkle -0.0, denormals, infinities and NaN payloads over a CPU state tensor."""
    flat = state.view(-1)
    bits = flat.view(torch.int32)
    n = flat.numel()
    idx = torch.randperm(n, generator=gen)[: min(n, 64)]
    specials = [-0x80000000, 0x00000001, 0x007FFFFF, 0x7F800000, -0x00800000, 0x7FC00001, 0x7F800123, -0x00400000 + 0x00012345]
    for j, i in enumerate(idx.tolist()):
        bits[i] = specials[j % len(specials)]
    return state


@dataclass
class TokenStreams:
    q: torch.Tensor      # [L, T, H_k, d_k]
    k: torch.Tensor      # [L, T, H_k, d_k]
    v: torch.Tensor      # [L, T, H_v, d_v]
    g: torch.Tensor      # [L, T, H_v, d_k] (KDA) or [L, T, H_v] (GDN), fp32
    beta: torch.Tensor   # [L, T, H_v] fp32


def token_streams(gen, kind, n_layers, T, H_v, H_k, d_k, d_v, rates, io_dtype=torch.bfloat16,
                  device="cpu") -> TokenStreams:
    """Token streams of one call.  ``rates`` is [L, H_v, d_k] (KDA) or [L, H_v, 1] (GDN)."""
    def normal(*shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)

    q = normal(n_layers, T, H_k, d_k)
    q = q / q.norm(dim=-1, keepdim=True)
    k = normal(n_layers, T, H_k, d_k)
    k = k / k.norm(dim=-1, keepdim=True)
    v = normal(n_layers, T, H_v, d_v)
    beta = torch.sigmoid(normal(n_layers, T, H_v))
    rates = rates.to(device)
    if kind == KDA:
        g = -torch.nn.functional.softplus(normal(n_layers, T, H_v, d_k)) * rates.view(n_layers, 1, H_v, d_k)
    else:
        g = -torch.nn.functional.softplus(normal(n_layers, T, H_v)) * rates.view(n_layers, 1, H_v)
    return TokenStreams(q.to(io_dtype).contiguous(), k.to(io_dtype).contiguous(),
                        v.to(io_dtype).contiguous(), g.contiguous(), beta.contiguous())


def uniform_cu_seqlens(n_req: int, suffix: int) -> torch.Tensor:
    return (torch.arange(n_req + 1, dtype=torch.int64) * suffix).to(torch.int32)


def ragged_cu_seqlens(gen, n_req: int, lo: int, hi: int) -> torch.Tensor:
    """Suffix lengths uniform in [lo, hi] (inclusive), as int32 prefix sums."""
    lens = torch.randint(lo, hi + 1, (n_req,), generator=gen, dtype=torch.int64)
    cu = torch.zeros(n_req + 1, dtype=torch.int64)
    cu[1:] = torch.cumsum(lens, 0)
    return cu.to(torch.int32)


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (CPU)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
