"""Helpers for parity checks at benchmark size: the fp64 oracle cannot replay 10^7-10^8
token-heads, so a deterministic sample of (request, layer, head) units is copied back and each
is replayed by the oracle as a one-unit problem on exactly the bits the GPU saw."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2608_30386_b200 as dasc
from helpers import _current_test, error_report, flush_error_log, log_errors, rel_err, stream_np


def sample_units(seed: int, n_req: int, n_layers: int, n_heads: int, count: int):
    """`count` distinct (request, layer, head) triples, spread by a fixed multiplicative hash."""
    total = n_req * n_layers * n_heads
    out, i = [], 0
    seen = set()
    while len(out) < min(count, total):
        u = ((seed + 1) * 2654435761 + i * 40503) % total
        i += 1
        if u in seen:
            continue
        seen.add(u)
        out.append((u // (n_layers * n_heads), (u // n_heads) % n_layers, u % n_heads))
    return out


def oracle_one_unit(kind, H_v, H_k, state0_unit, q, k, v, g, beta, cu, r, l, h, *, mode, keep_rows, q_scale=1.0):
    """Replay one unit on the oracle.  Streams are the device tensors of the call ([Lc][T][H][d]);
    `state0_unit` is the unit's [d_k, d_v] fp32 start state (numpy).  Returns (state64, o64)."""
    t0, t1 = int(cu[r]), int(cu[r + 1])
    hk = h // (H_v // H_k)
    d_k, d_v = state0_unit.shape
    qs = stream_np(q[l, t0:t1, hk].contiguous()).reshape(1, t1 - t0, 1, d_k)
    ks = stream_np(k[l, t0:t1, hk].contiguous()).reshape(1, t1 - t0, 1, d_k)
    vs = stream_np(v[l, t0:t1, h].contiguous()).reshape(1, t1 - t0, 1, d_v)
    if kind == dasc.KDA:
        gs = g[l, t0:t1, h].contiguous().cpu().numpy().reshape(1, t1 - t0, 1, d_k)
    else:
        gs = g[l, t0:t1, h].contiguous().cpu().numpy().reshape(1, t1 - t0, 1)
    bs = beta[l, t0:t1, h].contiguous().cpu().numpy().reshape(1, t1 - t0, 1)
    st = np.ascontiguousarray(state0_unit, np.float32).copy()
    if kind == dasc.KDA:
        mask = np.ascontiguousarray(keep_rows, np.uint8).reshape(1, d_k)     # this head's rows as a 1-head layer
    else:
        mask = np.array([[1 if keep_rows[0] else 0]], np.uint8)
    o, s64 = oracle.refresh(kind, 1, 1, 1, d_k, d_v, st, d_k * d_v, d_k * d_v, [0], qs, ks, vs,
                            np.ascontiguousarray(gs, np.float32), np.ascontiguousarray(bs, np.float32), [0, t1 - t0],
                            q_scale=q_scale, mode=mode, mask=mask, want_state64=True)
    return s64[0, 0, 0], o[0, :, 0]


def check_sampled_refresh(kind, plan, oplan, state_before, state_after, layer_stride, req_stride, q, k, v, g, beta, o,
                          cu, units, tol, *, mode=oracle.MODE_CONTINUE, layer_begin=0):
    """state_before / state_after: device fp32 tensors (flat) addressed by the strides; `o` may be None."""
    H_v, H_k, d_k, d_v = plan.n_v_heads, plan.n_k_heads, plan.d_k, plan.d_v
    worst = 0.0
    n_l = oplan.mask.shape[1]
    for (r, l, h) in units:
        off = r * req_stride + (layer_begin + l) * layer_stride + h * d_k * d_v
        s0 = state_before.view(-1)[off: off + d_k * d_v].cpu().numpy().reshape(d_k, d_v)
        s1 = state_after.view(-1)[off: off + d_k * d_v].cpu().numpy().reshape(d_k, d_v)
        if kind == dasc.KDA:
            keep = oplan.mask[layer_begin + l].reshape(H_v, d_k)[h]
        else:
            keep = np.full(d_k, oplan.mask[layer_begin + l][h], np.uint8)
        ref_s, ref_o = oracle_one_unit(kind, H_v, H_k, s0, q, k, v, g, beta, cu, r, l, h, mode=mode, keep_rows=keep)
        e = rel_err(s1, ref_s)
        worst = max(worst, e)
        log_errors(_current_test(), kind, "state", error_report(s1, ref_s))
        assert e <= tol, f"state of unit {(r, l, h)}: {e:.3e} > {tol}"
        if o is not None:
            t0, t1 = int(cu[r]), int(cu[r + 1])
            got_o = o[l, t0:t1, h].float().cpu().numpy()
            e = rel_err(got_o, ref_o)
            worst = max(worst, e)
            log_errors(_current_test(), kind, "output", error_report(got_o, ref_o))
            assert e <= tol, f"output of unit {(r, l, h)}: {e:.3e} > {tol}"
    flush_error_log()
    return worst
