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


@dataclass
class TraceRound:
    """One round of the mixed serving trace: the checkpoints stored and the cache hits served while both run."""
    store_slots: list      # pool slot of each new checkpoint
    hit_slots: list        # pool slot of each cache hit
    suffix: list           # tokens since the hit checkpoint, per hit


def serving_trace(seed: int, n_requests: int = 512, prefix_lo: int = 1024, prefix_hi: int = 131072,
                  interval: int = 1024, n_slots: int = 2048, batch: int = 64, concurrency: int = 96,
                  followups: int = 4, suffix_hi: int = 1024):
    """Event list of the mixed serving trace, generated on the host from one seed.

    `n_requests` requests with prefix lengths log-uniform in [prefix_lo, prefix_hi] are prefilled `concurrency` at a
    time; a request that is picked (uniformly among the active ones) advances by `interval` tokens and stores one
    checkpoint.  A finished request is followed up `followups` times, each after a random delay: the follow-up shares
    a prefix of random length with it, hits the newest checkpoint at or below that length if it is still resident,
    and replays the tokens since that checkpoint (uniform in [1, suffix_hi]).  Checkpoints live in a bounded pool of
    `n_slots` slots recycled least-recently-used first (a store or a hit makes a slot recent); slot 0 is reserved,
    as in the paper's allocator.  Events are cut into rounds of at most `batch` stores and `batch` hits such that no
    hit reads a slot written in its own round and no store recycles a slot read in its own round, so the two sides
    of a round may run concurrently.  Returns (rounds, stats)."""
    import numpy as np
    from collections import OrderedDict

    rng = np.random.default_rng(seed)
    prefix = np.exp(rng.uniform(math.log(prefix_lo), math.log(prefix_hi), size=n_requests)).astype(np.int64)
    n_ckpt = prefix // interval
    lru = OrderedDict()                      # slot -> (request, checkpoint index), least recently used first
    where = {}                               # (request, checkpoint index) -> slot
    free = list(range(n_slots - 1, 0, -1))   # slot 0 reserved
    rounds, cur = [], TraceRound([], [], [])
    written, read = set(), set()
    stats = dict(stores=0, hits=0, misses=0, evictions=0, tokens_replayed=0, checkpoints_total=int(n_ckpt.sum()),
                 prefix_tokens_total=int(prefix.sum()))

    def close():
        nonlocal cur, written, read
        if cur.store_slots or cur.hit_slots:
            rounds.append(cur)
        cur, written, read = TraceRound([], [], []), set(), set()

    def store(req, j):
        if free:
            slot = free.pop()
        else:
            slot, old = next(iter(lru.items()))
            if slot in read or slot in written:
                close()
            del lru[slot]
            del where[old]
            stats["evictions"] += 1
        if len(cur.store_slots) == batch:
            close()
        lru[slot] = (req, j)
        where[(req, j)] = slot
        cur.store_slots.append(slot)
        written.add(slot)
        stats["stores"] += 1

    def hit(req):
        shared = int(rng.integers(interval, prefix[req] + 1))          # length of the shared prefix
        j = min(shared // interval, int(n_ckpt[req]))
        while j >= 1 and (req, j) not in where:                        # newest resident checkpoint at or below it
            j -= 1
        if j < 1:
            stats["misses"] += 1
            return
        slot = where[(req, j)]
        if slot in written or len(cur.hit_slots) == batch:
            close()
        lru.move_to_end(slot)
        n = int(rng.integers(1, suffix_hi + 1))
        cur.hit_slots.append(slot)
        cur.suffix.append(n)
        read.add(slot)
        stats["hits"] += 1
        stats["tokens_replayed"] += n

    nxt, active, due, clock = 0, [], [], 0       # due: (time, request) follow-ups
    progress = {}
    while nxt < n_requests or active or due:
        while nxt < n_requests and len(active) < concurrency:
            progress[nxt] = 0
            active.append(nxt)
            nxt += 1
        clock += 1
        ready = [d for d in due if d[0] <= clock]
        if ready:
            due = [d for d in due if d[0] > clock]
            for _, req in ready:
                hit(req)
        if not active:
            if due:
                clock = min(d[0] for d in due) - 1
            continue
        req = active[int(rng.integers(0, len(active)))]
        progress[req] += 1
        if progress[req] <= n_ckpt[req]:
            store(req, progress[req])
        if progress[req] >= n_ckpt[req]:
            active.remove(req)
            for _ in range(followups):
                due.append((clock + 1 + int(rng.exponential(4.0 * concurrency)), req))
    close()
    stats["rounds"] = len(rounds)
    return rounds, stats
