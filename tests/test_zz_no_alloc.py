"""The workspace-free refresh entry point (dasc_refresh_static) against dasc_refresh.

Some callers cannot pass a workspace because they cannot allocate device memory where they call
from (a serving engine that has already handed every byte of HBM to its pools).  For them the
library keeps the kernel's scratch in a fixed array of its own.  This file is collected last so
that a run stopping at the first failure has already run every other test; the test also passes
when run alone in a fresh process."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding
from helpers import make_refresh_case, rel_err

pytestmark = pytest.mark.gpu

TOL = 1e-3   # the refresh tolerance of the other GPU tests (max abs error / max |reference| per unit)


def _run(case, state0, use_static):
    dev = state0.device
    n_req = case.cu.numel() - 1
    T = int(case.cu[-1])
    s = case.streams
    state = state0.clone()
    o = torch.full((case.L, T, case.H_v, case.d_v), float("nan"), device=dev, dtype=torch.bfloat16)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    ls, rs = case.H_v * case.d_k * case.d_v, case.L * case.H_v * case.d_k * case.d_v
    lens = case.cu[1:] - case.cu[:-1]
    if use_static:
        free_before = torch.cuda.mem_get_info()[0]
        scratch = dasc.dasc_refresh_static(case.plan, state, ls, rs, ids, s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), T,
                                           int(lens.max()), o=o)
        torch.cuda.synchronize()
        assert scratch != 0
        assert dasc.lib().dasc_refresh_status(ctypes.c_void_p(scratch), 4) == binding.OK
        assert torch.cuda.mem_get_info()[0] >= free_before          # the call took no device memory
    else:
        ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(case.plan, n_req, case.L, dasc.ALGO_CHUNKED),
                         dtype=torch.uint8, device=dev)
        dasc.dasc_refresh(case.plan, state, ls, rs, ids, s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), T,
                          int(lens.max()), o=o, algo=dasc.ALGO_CHUNKED, workspace=ws)
        torch.cuda.synchronize()
        assert dasc.dasc_refresh_status(ws) == binding.OK
    return state, o


def _close(case, got, want):
    gs, go = got[0].cpu().numpy(), got[1].float().cpu().numpy()
    ws_, wo = want[0].cpu().numpy(), want[1].float().cpu().numpy()
    n_req = case.cu.numel() - 1
    for r in range(n_req):
        t0, t1 = int(case.cu[r]), int(case.cu[r + 1])
        for l in range(case.L):
            for h in range(case.H_v):
                assert rel_err(gs[r, l, h], ws_[r, l, h]) <= TOL
                if t1 > t0:
                    assert rel_err(go[l, t0:t1, h], wo[l, t0:t1, h]) <= TOL


def test_static_scratch_refresh_matches_workspace_refresh_twice_in_a_row():
    case = make_refresh_case(31, dasc.KDA, 2, 4, 4, 128, 128, [70, 5, 128], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    # first call
    want1 = _run(case, case.state0, use_static=False)
    got1 = _run(case, case.state0, use_static=True)
    _close(case, got1, want1)
    # second call, straight after, continuing from the first call's state: the shared scratch
    # still holds the first call's contents and must not disturb it
    want2 = _run(case, want1[0], use_static=False)
    got2 = _run(case, got1[0], use_static=True)
    _close(case, got2, want2)
    assert not np.array_equal(got2[0].cpu().numpy(), got1[0].cpu().numpy())


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
