"""Shared helpers of the GPU parity tests: build a seeded workload, run the CUDA
path through the binding and the oracle on the same bits, and compare."""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth


def rel_err(x, ref):
    """max|x - ref| / max|ref| over one tensor (0 when both are all zero)."""
    x = np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.abs(ref).max() if ref.size else 0.0
    num = np.abs(x - ref).max() if ref.size else 0.0
    if den == 0.0:
        return 0.0 if num == 0.0 else math.inf
    return num / den


def error_report(x, ref):
    """The per-tensor metric beside two finer ones, for the log (only the first is asserted on):
    tensor  max|x - ref| / max|ref| over the whole tensor;
    row     the worst row of a [rows, cols] tensor taken on its own, max|x_r - ref_r| / max|ref_r| (a KDA selection
            unit is one key-channel row of the state); rows whose reference is all zero are left out;
    elem    max over elements of |x - ref| / max(|ref|, 1e-6 * max|ref|)."""
    x = np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    top = np.abs(ref).max() if ref.size else 0.0
    if top == 0.0:
        return {"tensor": rel_err(x, ref), "row": 0.0, "elem": 0.0}
    err = np.abs(x - ref)
    row_top = np.abs(ref.reshape(ref.shape[0], -1)).max(1)
    row_err = err.reshape(ref.shape[0], -1).max(1)
    live = row_top > 0
    return {"tensor": float(err.max() / top), "row": float((row_err[live] / row_top[live]).max()) if live.any() else 0.0,
            "elem": float((err / np.maximum(np.abs(ref), 1e-6 * top)).max())}


_ERROR_LOG = {}


def log_errors(name, kind, what, rep):
    """Keep the worst figures per (test, kind, tensor kind); written out as JSON lines when DASC_ERROR_LOG names a file."""
    key = (name, kind, what)
    cur = _ERROR_LOG.setdefault(key, {"tensor": 0.0, "row": 0.0, "elem": 0.0, "units": 0})
    for k in ("tensor", "row", "elem"):
        cur[k] = max(cur[k], rep[k])
    cur["units"] += 1


def flush_error_log():
    import json
    import os
    path = os.environ.get("DASC_ERROR_LOG")
    if not path or not _ERROR_LOG:
        return
    with open(path, "a") as f:
        for (name, kind, what), v in sorted(_ERROR_LOG.items()):
            f.write(json.dumps({"test": name, "kind": "KDA" if kind == dasc.KDA else "GDN", "what": what, **v}) + "\n")
    _ERROR_LOG.clear()


def make_plans(kind, L, H_v, H_k, d_k, d_v, rates, *, sel, scope=dasc.SCOPE_LAYER, keep_ratio=1.0, w_max=0.0,
               device=0):
    """The library plan and the oracle plan for the same decay parameters."""
    A_log, dt = synth.decay_params(rates)
    A = A_log.cpu().numpy()
    B = dt.cpu().numpy()
    uph = d_k if kind == dasc.KDA else 1
    p = dasc.dasc_plan(kind, L, H_v, H_k, d_k, d_v, A, B, sel=sel, scope=scope, keep_ratio=keep_ratio, w_max=w_max,
                       device=device)
    o = oracle.plan(kind, L, H_v, uph, A, B, sel=sel, scope=scope, keep_ratio=keep_ratio, w_max=w_max,
                    unit_bytes=int(p.unit_floats) * 4)
    np.testing.assert_array_equal(p.mask(), o.mask)
    return p, o


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int32).numpy().view(np.uint32)


def stream_np(t: torch.Tensor) -> np.ndarray:
    """Token stream as the oracle wants it: uint16 bit patterns for bf16, float32 otherwise."""
    if t.dtype == torch.bfloat16:
        return synth.bf16_bits(t)
    return t.detach().cpu().contiguous().numpy()


@dataclass
class RefreshCase:
    kind: int
    L: int
    H_v: int
    H_k: int
    d_k: int
    d_v: int
    cu: torch.Tensor           # int32 [n_req+1], CPU
    streams: synth.TokenStreams  # on the device
    state0: torch.Tensor       # [n_req, L, H_v, d_k, d_v] fp32, device
    plan: object
    oplan: object


def run_refresh_gpu(case: RefreshCase, *, mode=dasc.REFRESH_CONTINUE, algo=dasc.ALGO_AUTO, o_dtype=torch.float32,
                    want_o=True, q_scale=1.0, layer_begin=0, layer_end=None):
    """Returns (final state [n_req, L, H_v, d_k, d_v] numpy fp32, o numpy or None)."""
    dev = case.state0.device
    n_req = case.cu.numel() - 1
    T = int(case.cu[-1])
    layer_end = case.L if layer_end is None else layer_end
    Lc = layer_end - layer_begin
    state = case.state0.clone()
    s = case.streams
    sl = slice(layer_begin, layer_end)
    q, k, v, g, beta = (x[sl].contiguous() for x in (s.q, s.k, s.v, s.g, s.beta))
    o = torch.full((Lc, T, case.H_v, case.d_v), float("nan"), device=dev, dtype=o_dtype) if want_o else None
    ws_bytes = dasc.dasc_refresh_workspace_bytes(case.plan, n_req, Lc, algo)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device=dev) if ws_bytes else None
    lens = (case.cu[1:] - case.cu[:-1])
    dasc.dasc_refresh(case.plan, state, case.H_v * case.d_k * case.d_v, case.L * case.H_v * case.d_k * case.d_v,
                      torch.arange(n_req, dtype=torch.int32, device=dev), q, k, v, g, beta, case.cu.to(dev), T,
                      int(lens.max()) if n_req else 0, layer_begin=layer_begin, layer_end=layer_end, q_scale=q_scale,
                      o=o, mode=mode, algo=algo, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    return state.cpu().numpy(), (o.float().cpu().numpy() if want_o else None)


def run_refresh_oracle(case: RefreshCase, *, mode=oracle.MODE_CONTINUE, want_o=True, q_scale=1.0):
    """Oracle on the same bits: (state64 [n_req, L, H_v, d_k, d_v], o fp64 [L, T, H_v, d_v] or None)."""
    n_req = case.cu.numel() - 1
    state = case.state0.cpu().numpy().copy()
    s = case.streams
    o, s64 = oracle.refresh(case.kind, case.L, case.H_v, case.H_k, case.d_k, case.d_v, state,
                            case.H_v * case.d_k * case.d_v, case.L * case.H_v * case.d_k * case.d_v,
                            np.arange(n_req, dtype=np.int32), stream_np(s.q), stream_np(s.k), stream_np(s.v),
                            stream_np(s.g), stream_np(s.beta), case.cu.numpy(), q_scale=q_scale, want_o=want_o,
                            mode=mode, mask=case.oplan.mask, want_state64=True)
    return s64, o


def assert_refresh_close(case: RefreshCase, got_state, got_o, ref_state, ref_o, tol):
    """Per unit: final state and output block each within `tol` (max abs err / max |ref|)."""
    n_req = case.cu.numel() - 1
    worst = 0.0
    for r in range(n_req):
        t0, t1 = int(case.cu[r]), int(case.cu[r + 1])
        for l in range(case.L):
            for h in range(case.H_v):
                e = rel_err(got_state[r, l, h], ref_state[r, l, h])
                worst = max(worst, e)
                log_errors(_current_test(), case.kind, "state", error_report(got_state[r, l, h], ref_state[r, l, h]))
                assert e <= tol, f"state r={r} l={l} h={h}: {e:.3e} > {tol}"
                if got_o is not None and t1 > t0:
                    e = rel_err(got_o[l, t0:t1, h], ref_o[l, t0:t1, h])
                    worst = max(worst, e)
                    log_errors(_current_test(), case.kind, "output", error_report(got_o[l, t0:t1, h], ref_o[l, t0:t1, h]))
                    assert e <= tol, f"o r={r} l={l} h={h}: {e:.3e} > {tol}"
    flush_error_log()
    return worst


def _current_test():
    import os
    return os.environ.get("PYTEST_CURRENT_TEST", "smoke").split(" ")[0].split("::")[-1]


def make_refresh_case(seed, kind, L, H_v, H_k, d_k, d_v, lens, *, io_dtype=torch.bfloat16, keep_ratio=0.4,
                      scope=dasc.SCOPE_HEAD, rate_lo=1e-3, rate_hi=1.0, device="cuda") -> RefreshCase:
    gen = synth.generator(seed)
    uph = d_k if kind == dasc.KDA else 1
    rates = synth.decay_rates(gen, L, H_v, uph, rate_lo, rate_hi)
    plan, oplan = make_plans(kind, L, H_v, H_k, d_k, d_v, rates, sel=dasc.SEL_TOP_RATIO, scope=scope,
                             keep_ratio=keep_ratio)
    cu = torch.zeros(len(lens) + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(torch.tensor(lens, dtype=torch.int64), 0).to(torch.int32)
    T = int(cu[-1])
    streams = synth.token_streams(gen, kind, L, T, H_v, H_k, d_k, d_v, rates, io_dtype=io_dtype)
    state0 = synth.states(gen, (len(lens), L, H_v, d_k, d_v))
    for f in ("q", "k", "v", "g", "beta"):
        setattr(streams, f, getattr(streams, f).to(device))
    return RefreshCase(kind, L, H_v, H_k, d_k, d_v, cu, streams, state0.to(device), plan, oplan)
