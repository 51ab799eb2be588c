"""What the refresh call does outside the comfortable middle: log-decays beyond the tensor-core kernel's range,
requests of a handful of tokens, and a device-side wait that runs out.  In every case the stored states stay
recoverable, the status says what happened, and DASC_ALGO_AUTO returns results within the stated tolerance of the
fp64 oracle on the unchanged metric (max abs error / max |reference| per unit)."""
import numpy as np
import pytest
import torch

import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding
from helpers import (assert_refresh_close, make_refresh_case, rel_err, run_refresh_gpu, run_refresh_oracle)

pytestmark = pytest.mark.gpu

TOL = 1e-3


def _strong_decay_case(seed=41):
    # (request 0, layer 0, head 1): one key channel decays by e^-7 per token from token 40 on, i.e. 112 over half a
    # chunk -- beyond the 80 the midpoint factors can carry in fp32.  Every other unit is ordinary.
    case = make_refresh_case(seed, dasc.KDA, 2, 4, 4, 128, 128, [96, 70], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    case.streams.g[0, 40:96, 1, 5] = -7.0
    return case


def _call(case, algo, mode=dasc.REFRESH_CONTINUE):
    dev = case.state0.device
    n_req, T = case.cu.numel() - 1, int(case.cu[-1])
    s = case.streams
    state = case.state0.clone()
    o = torch.full((case.L, T, case.H_v, case.d_v), float("nan"), device=dev)
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(case.plan, n_req, case.L, algo), dtype=torch.uint8, device=dev)
    dasc.dasc_refresh(case.plan, state, case.H_v * 128 * 128, case.L * case.H_v * 128 * 128,
                      torch.arange(n_req, dtype=torch.int32, device=dev), s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), T,
                      int((case.cu[1:] - case.cu[:-1]).max()), o=o, mode=mode, algo=algo, workspace=ws)
    torch.cuda.synchronize()
    return state, o, ws


def test_chunked_alone_leaves_an_out_of_range_unit_untouched_and_reports_it():
    case = _strong_decay_case()
    ref_s, ref_o = run_refresh_oracle(case)
    state, o, ws = _call(case, dasc.ALGO_CHUNKED)
    assert dasc.dasc_refresh_status(ws) == binding.ERR_DOMAIN
    handed, replayed = dasc.dasc_refresh_counters(ws)
    assert (handed, replayed) == (1, 0)
    unit = int(ws[256:260].view(torch.int32).item())
    assert unit == (0 * case.L + 0) * case.H_v + 1                       # (request 0, layer 0, head 1)
    got = state.cpu().numpy()
    # the flagged unit still holds the bits it had before the call ...
    np.testing.assert_array_equal(got[0, 0, 1].view(np.uint32), case.state0[0, 0, 1].cpu().numpy().view(np.uint32))
    # ... every other unit is complete and within tolerance
    o_np = o.cpu().numpy()
    for r in range(2):
        t0, t1 = int(case.cu[r]), int(case.cu[r + 1])
        for l in range(case.L):
            for h in range(case.H_v):
                if (r, l, h) == (0, 0, 1):
                    continue
                assert rel_err(got[r, l, h], ref_s[r, l, h]) <= TOL
                assert rel_err(o_np[l, t0:t1, h], ref_o[l, t0:t1, h]) <= TOL
    # the exact kernel replays the flagged unit from that untouched state
    seq_s, seq_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL)
    assert rel_err(seq_s[0, 0, 1], ref_s[0, 0, 1]) <= TOL
    assert rel_err(seq_o[0, 0:96, 1], ref_o[0, 0:96, 1]) <= TOL


@pytest.mark.parametrize("mode", [dasc.REFRESH_CONTINUE, dasc.REFRESH_SCRATCH_MERGE_LOCAL])
def test_auto_replays_out_of_range_units_with_the_exact_kernel(mode):
    import oracle
    case = _strong_decay_case(seed=42)
    omode = oracle.MODE_CONTINUE if mode == dasc.REFRESH_CONTINUE else oracle.MODE_SCRATCH_MERGE_LOCAL
    ref_s, ref_o = run_refresh_oracle(case, mode=omode)
    state, o, ws = _call(case, dasc.ALGO_AUTO, mode)
    assert dasc.dasc_refresh_status(ws) == binding.OK
    assert dasc.dasc_refresh_counters(ws) == (1, 1)
    assert_refresh_close(case, state.cpu().numpy(), o.cpu().numpy(), ref_s, ref_o, TOL)


def test_auto_sends_requests_of_a_few_tokens_to_the_exact_kernel():
    # Requests of 1, 2, 8 tokens (and an empty one) beside a long one, replayed from a zero scratch state: with so few
    # tokens every output is a sum of a few q.k products, the case in which one tf32-rounded product can exceed the
    # output tolerance.  AUTO hands those requests to the exact kernel; the bar is the unchanged one.
    import oracle
    case = make_refresh_case(43, dasc.KDA, 1, 4, 4, 128, 128, [1, 2, 0, 8, 9, 70], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    for mode, omode in ((dasc.REFRESH_SCRATCH_MERGE_LOCAL, oracle.MODE_SCRATCH_MERGE_LOCAL),
                        (dasc.REFRESH_CONTINUE, oracle.MODE_CONTINUE)):
        ref_s, ref_o = run_refresh_oracle(case, mode=omode)
        state, o, ws = _call(case, dasc.ALGO_AUTO, mode)
        assert dasc.dasc_refresh_status(ws) == binding.OK
        handed, replayed = dasc.dasc_refresh_counters(ws)
        # requests of 1, 2, 8 tokens, 4 heads each; the empty request is handed over only where it has work to do
        # (the scratch mode replaces its omitted units by zeros)
        want = 3 * 4 + (4 if mode == dasc.REFRESH_SCRATCH_MERGE_LOCAL else 0)
        assert (handed, replayed) == (want, want)
        got_s, got_o = state.cpu().numpy(), o.cpu().numpy()
        assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
        # and the exact kernel is exact: its units agree with the oracle to fp32 rounding
        for r in (0, 1, 3):
            for h in range(4):
                assert rel_err(got_s[r, 0, h], ref_s[r, 0, h]) <= 1e-5
    # GDN goes the same way
    case = make_refresh_case(44, dasc.GDN, 1, 4, 2, 128, 128, [3, 40], scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    ref_s, ref_o = run_refresh_oracle(case)
    state, o, ws = _call(case, dasc.ALGO_AUTO)
    assert dasc.dasc_refresh_counters(ws) == (4, 4)
    assert_refresh_close(case, state.cpu().numpy(), o.cpu().numpy(), ref_s, ref_o, TOL)


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    # The issuing warp's first wait (for the first chunk's operand tiles, which take thousands of cycles to build) is
    # given a single poll through the test hook: it gives up, the CTA skips the rest of its waits, lets its
    # tensor-core work drain, frees its tensor memory and returns without writing its unit back.
    case = make_refresh_case(45, dasc.KDA, 1, 1, 1, 128, 128, [32], scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    try:
        dasc.dasc_debug_set_refresh_poll_limit(1)
        state, o, ws = _call(case, dasc.ALGO_CHUNKED)
    finally:
        dasc.dasc_debug_set_refresh_poll_limit(0)
    assert dasc.dasc_refresh_status(ws) == binding.ERR_TIMEOUT
    assert torch.equal(state, case.state0)                                # nothing was written back
    # the next call on the same context, same workspace, is clean and correct
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED)
    assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
    s = case.streams
    dev = state.device
    dasc.dasc_refresh(case.plan, state, 128 * 128, 128 * 128, torch.zeros(1, dtype=torch.int32, device=dev), s.q, s.k,
                      s.v, s.g, s.beta, case.cu.to(dev), 32, 32, o=o, algo=dasc.ALGO_CHUNKED, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == binding.OK
    assert rel_err(state.cpu().numpy()[0, 0, 0], ref_s[0, 0, 0]) <= TOL


def test_refresh_window_checks_every_argument_before_it_writes_window_begin():
    case = make_refresh_case(46, dasc.KDA, 1, 2, 2, 128, 128, [40], scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    dev = case.state0.device
    s = case.streams
    wb = torch.full((1,), -7, dtype=torch.int32, device=dev)
    state = case.state0.clone()
    with pytest.raises(dasc.DascError) as e:                               # no workspace for the chunked kernel
        dasc.dasc_refresh_window(case.plan, state, 2 * 128 * 128, 2 * 128 * 128, torch.zeros(1, dtype=torch.int32, device=dev),
                                 None, s.k, s.v, s.g, s.beta, case.cu.to(dev), 40, wb, window=16, workspace=None)
    assert e.value.status == binding.ERR_WORKSPACE
    with pytest.raises(dasc.DascError) as e:                               # layer range outside the plan
        dasc.dasc_refresh_window(case.plan, state, 2 * 128 * 128, 2 * 128 * 128, torch.zeros(1, dtype=torch.int32, device=dev),
                                 None, s.k, s.v, s.g, s.beta, case.cu.to(dev), 40, wb, window=16, layer_end=3,
                                 algo=dasc.ALGO_SEQUENTIAL)
    assert e.value.status == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(wb.item()) == -7 and torch.equal(state, case.state0)
