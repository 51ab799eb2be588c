"""GPU parity: dasc_refresh_window, the suffix-refresh load policy of Section 4.2 with the window of Eq. 7
(replay the last W prefix tokens from a zero scratch state, merge only omitted units), against the oracle
run on the token slices the definition names."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth
from helpers import RefreshCase, make_plans, make_refresh_case, rel_err, stream_np

pytestmark = pytest.mark.gpu


def _oracle_window(case: RefreshCase, W: int, want_o: bool):
    """Slices each request's last min(W, prefix) tokens out of the streams and runs the oracle's
    SCRATCH_MERGE_LOCAL mode on them.  Returns (state64, o or None, begins, new cu)."""
    cu = case.cu.numpy().astype(np.int64)
    n_req = cu.size - 1
    begins = np.maximum(cu[:-1], cu[1:] - W)
    idx = np.concatenate([np.arange(b, e) for b, e in zip(begins, cu[1:])]).astype(np.int64) if n_req else np.zeros(0, np.int64)
    new_cu = np.zeros(n_req + 1, np.int32)
    new_cu[1:] = np.cumsum(cu[1:] - begins)
    s = case.streams
    sl = [np.ascontiguousarray(stream_np(x)[:, idx]) for x in (s.q, s.k, s.v, s.g, s.beta)]
    state = case.state0.cpu().numpy().copy()
    dense = case.H_v * case.d_k * case.d_v
    o, s64 = oracle.refresh(case.kind, case.L, case.H_v, case.H_k, case.d_k, case.d_v, state, dense, case.L * dense,
                            np.arange(n_req, dtype=np.int32), *sl, new_cu, want_o=want_o,
                            mode=oracle.MODE_SCRATCH_MERGE_LOCAL, mask=case.oplan.mask, want_state64=True)
    return s64, o, begins, new_cu, idx


def _run(case: RefreshCase, W: int, *, with_o: bool, algo=dasc.ALGO_AUTO, tol=1e-3, window_arg=None):
    dev = case.state0.device
    n_req = case.cu.numel() - 1
    T = int(case.cu[-1])
    dense = case.H_v * case.d_k * case.d_v
    state = case.state0.clone()
    s = case.streams
    o = torch.full((case.L, T, case.H_v, case.d_v), float("nan"), device=dev) if with_o else None
    wb = torch.full((n_req,), -7, dtype=torch.int32, device=dev)
    ws_bytes = dasc.dasc_refresh_workspace_bytes(case.plan, n_req, case.L, algo)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device=dev) if ws_bytes else None
    dasc.dasc_refresh_window(case.plan, state, dense, case.L * dense, torch.arange(n_req, dtype=torch.int32, device=dev),
                             s.q if with_o else None, s.k, s.v, s.g, s.beta, case.cu.to(dev), T, wb,
                             window=W if window_arg is None else window_arg, o=o, algo=algo, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    ref_state, ref_o, begins, new_cu, idx = _oracle_window(case, W, with_o)
    np.testing.assert_array_equal(wb.cpu().numpy(), begins.astype(np.int32))
    got = state.cpu().numpy()
    before = case.state0.cpu().numpy()
    keep = case.oplan.mask.astype(bool)                                   # [L, n_l]
    worst = 0.0
    for r in range(n_req):
        for l in range(case.L):
            rows = keep[l].reshape(case.H_v, -1)                          # KDA: [H, d_k]; GDN: [H, 1]
            for h in range(case.H_v):
                # retained units keep their stored bits; omitted units take the scratch state
                kept = rows[h] if case.kind == dasc.KDA else np.full(case.d_k, rows[h][0])
                np.testing.assert_array_equal(got[r, l, h][kept].view(np.uint32), before[r, l, h][kept].view(np.uint32))
                e = rel_err(got[r, l, h], ref_state[r, l, h])
                worst = max(worst, e)
                assert e <= tol, f"state r={r} l={l} h={h}: {e:.3e}"
                if with_o and new_cu[r + 1] > new_cu[r]:
                    a = o[l, int(begins[r]): int(case.cu[r + 1]), h].cpu().numpy()
                    e = rel_err(a, ref_o[l, new_cu[r]:new_cu[r + 1], h])
                    worst = max(worst, e)
                    assert e <= tol, f"o r={r} l={l} h={h}: {e:.3e}"
    if with_o:                                                            # tokens before a window are not written
        untouched = np.ones(T, bool)
        untouched[idx] = False
        assert torch.isnan(o[:, torch.from_numpy(untouched)]).all()
    return worst


@pytest.mark.parametrize("with_o", [False, True])
def test_kda_chunked_windows_clipped_by_the_prefix(with_o):
    # prefixes longer than, equal to, shorter than the window, and empty; ragged chunk tails
    case = make_refresh_case(21, dasc.KDA, 2, 4, 4, 128, 128, [200, 37, 0, 64, 131], keep_ratio=0.4)
    w = _run(case, 64, with_o=with_o, algo=dasc.ALGO_CHUNKED)
    print(f"worst relative error {w:.2e}")


def test_gdn_chunked_state_only():
    case = make_refresh_case(22, dasc.GDN, 2, 8, 4, 128, 128, [96, 10, 150], keep_ratio=0.5, scope=dasc.SCOPE_LAYER)
    _run(case, 128, with_o=False, algo=dasc.ALGO_CHUNKED)
    _run(case, 128, with_o=True, algo=dasc.ALGO_CHUNKED)


def test_sequential_fp32_small_shapes():
    case = make_refresh_case(23, dasc.KDA, 2, 3, 3, 64, 64, [50, 5, 0, 33], io_dtype=torch.float32, keep_ratio=0.4)
    _run(case, 16, with_o=False, tol=1e-5)
    _run(case, 16, with_o=True, tol=1e-5)


def test_window_defaults_to_the_plans_w_replay():
    # threshold rule with W_max = 64: Eq. 7 gives W_replay = 64 (some omitted horizon exceeds 32)
    gen = synth.generator(24)
    L, H, d = 1, 2, 128
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_THRESHOLD, w_max=64.0)
    assert plan.w_replay == 64
    lens = [100, 20]
    cu = torch.tensor([0, 100, 120], dtype=torch.int32)
    streams = synth.token_streams(gen, dasc.KDA, L, 120, H, H, d, d, rates)
    for f in ("q", "k", "v", "g", "beta"):
        setattr(streams, f, getattr(streams, f).to("cuda"))
    state0 = synth.states(gen, (len(lens), L, H, d, d)).to("cuda")
    case = RefreshCase(dasc.KDA, L, H, H, d, d, cu, streams, state0, plan, oplan)
    _run(case, 64, with_o=False, window_arg=0)


def test_argument_errors():
    case = make_refresh_case(25, dasc.KDA, 1, 2, 2, 64, 64, [8], io_dtype=torch.float32)
    dev = "cuda"
    s = case.streams
    state = case.state0.clone()
    wb = torch.zeros(1, dtype=torch.int32, device=dev)
    o = torch.zeros((1, 8, 2, 64), device=dev)
    with pytest.raises(dasc.DascError) as e:                              # outputs wanted but no queries
        dasc.dasc_refresh_window(case.plan, state, 2 * 64 * 64, 2 * 64 * 64, torch.zeros(1, dtype=torch.int32, device=dev),
                                 None, s.k, s.v, s.g, s.beta, case.cu.to(dev), 8, wb, window=4, o=o)
    assert e.value.status == 1
    torch.cuda.synchronize()
    assert torch.equal(state, case.state0)
