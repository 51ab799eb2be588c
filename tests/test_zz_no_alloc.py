"""The workspace-free refresh entry point (dasc_refresh_static) against dasc_refresh and the oracle.

Some callers cannot pass a workspace because they cannot allocate device memory where they call
from (a serving engine that has already handed every byte of HBM to its pools).  For them the
library keeps the kernel's scratch in a fixed array of its own.  This file is collected last so
that a run stopping at the first failure has already run every other test; the tests also pass
when run alone in a fresh process."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding
from helpers import assert_refresh_close, make_refresh_case, run_refresh_oracle

pytestmark = pytest.mark.gpu

TOL = 1e-3   # the refresh tolerance of the other GPU tests (max abs error / max |reference| per unit)


def _run(case, state0, use_static, *, mode=dasc.REFRESH_CONTINUE, want_o=True, o_dtype=torch.bfloat16):
    dev = state0.device
    n_req = case.cu.numel() - 1
    T = int(case.cu[-1])
    s = case.streams
    state = state0.clone()
    o = torch.full((case.L, T, case.H_v, case.d_v), float("nan"), device=dev, dtype=o_dtype) if want_o else None
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    ls, rs = case.H_v * case.d_k * case.d_v, case.L * case.H_v * case.d_k * case.d_v
    lens = case.cu[1:] - case.cu[:-1]
    if use_static:
        free_before = torch.cuda.mem_get_info()[0]
        scratch = dasc.dasc_refresh_static(case.plan, state, ls, rs, ids, s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), T,
                                           int(lens.max()), o=o, mode=mode)
        torch.cuda.synchronize()
        assert scratch != 0
        assert dasc.dasc_refresh_status(scratch) == binding.OK           # both flag words (8 bytes) are read
        assert torch.cuda.mem_get_info()[0] >= free_before                # the call took no device memory
    else:
        ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(case.plan, n_req, case.L, dasc.ALGO_CHUNKED),
                         dtype=torch.uint8, device=dev)
        dasc.dasc_refresh(case.plan, state, ls, rs, ids, s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), T,
                          int(lens.max()), o=o, mode=mode, algo=dasc.ALGO_CHUNKED, workspace=ws)
        torch.cuda.synchronize()
        assert dasc.dasc_refresh_status(ws) == binding.OK
    return state, o


def _same(got, want):
    # the two entry points run the same kernel, which is deterministic: the results are the same bits, and the
    # tolerance of the other tests (TOL) is met with nothing to spare being needed
    assert torch.equal(got[0], want[0])
    if want[1] is not None:
        assert torch.equal(got[1].view(torch.int16), want[1].view(torch.int16))
        rel = (got[1].float() - want[1].float()).abs().max() / want[1].float().abs().max()
        assert float(rel) <= TOL


def test_static_scratch_refresh_matches_workspace_refresh_twice_in_a_row():
    case = make_refresh_case(31, dasc.KDA, 2, 4, 4, 128, 128, [70, 5, 128], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    # first call
    want1 = _run(case, case.state0, use_static=False)
    got1 = _run(case, case.state0, use_static=True)
    _same(got1, want1)
    # second call, straight after, continuing from the first call's state: the shared scratch
    # still holds the first call's contents and must not disturb it
    want2 = _run(case, want1[0], use_static=False)
    got2 = _run(case, got1[0], use_static=True)
    _same(got2, want2)
    assert not np.array_equal(got2[0].cpu().numpy(), got1[0].cpu().numpy())


def test_static_scratch_refresh_against_the_oracle_in_both_modes():
    case = make_refresh_case(33, dasc.KDA, 1, 4, 4, 128, 128, [40, 97], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    ref_s, ref_o = run_refresh_oracle(case)
    got = _run(case, case.state0, use_static=True, o_dtype=torch.float32)
    assert_refresh_close(case, got[0].cpu().numpy(), got[1].cpu().numpy(), ref_s, ref_o, TOL)
    # the paper's load policy (zero scratch state, only omitted units merged), without outputs
    ref_s, _ = run_refresh_oracle(case, mode=oracle.MODE_SCRATCH_MERGE_LOCAL, want_o=False)
    got = _run(case, case.state0, use_static=True, mode=dasc.REFRESH_SCRATCH_MERGE_LOCAL, want_o=False)
    assert_refresh_close(case, got[0].cpu().numpy(), None, ref_s, None, TOL)
    want = _run(case, case.state0, use_static=False, mode=dasc.REFRESH_SCRATCH_MERGE_LOCAL, want_o=False)
    _same(got, want)


def test_static_scratch_refresh_replays_units_outside_the_chunked_range_exactly():
    # one channel of (request 0, head 1) decays by e^-7 per token: outside what the tensor-core kernel's midpoint
    # factors can carry.  That unit is listed in the static array, left unwritten by the tensor-core kernel and
    # replayed by the exact kernel on the same stream; the status stays OK and the result matches the oracle.
    case = make_refresh_case(34, dasc.KDA, 1, 2, 2, 128, 128, [64, 33], scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    case.streams.g[0, 0:64, 1, 5] = -7.0
    ref_s, ref_o = run_refresh_oracle(case)
    got = _run(case, case.state0, use_static=True, o_dtype=torch.float32)
    assert_refresh_close(case, got[0].cpu().numpy(), got[1].cpu().numpy(), ref_s, ref_o, TOL)
    dev = case.state0.device
    s = case.streams
    scratch = dasc.dasc_refresh_static(case.plan, case.state0.clone(), 2 * 128 * 128, 2 * 128 * 128,
                                       torch.arange(2, dtype=torch.int32, device=dev), s.q, s.k, s.v, s.g, s.beta,
                                       case.cu.to(dev), 97, 64)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_counters(scratch) == (1, 1)


def test_static_scratch_refresh_refuses_what_the_chunked_kernel_cannot_take():
    case = make_refresh_case(32, dasc.KDA, 1, 2, 2, 64, 64, [8])        # d = 64: not the chunked kernel's shape
    dev = case.state0.device
    s = case.streams
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    state = case.state0.clone()
    with pytest.raises(dasc.DascError) as e:
        dasc.dasc_refresh_static(case.plan, state, 2 * 64 * 64, 2 * 64 * 64, ids, s.q, s.k, s.v, s.g, s.beta,
                                 case.cu.to(dev), 8, 8)
    assert e.value.status == binding.ERR_SHAPE
    torch.cuda.synchronize()
    assert torch.equal(state, case.state0)
