"""GPU parity of the chunked tensor-core refresh kernel (DASC_ALGO_CHUNKED) against the
token-by-token fp64 oracle: bf16 q/k/v, fp32 state, tolerance 1e-3 (max abs error over
max |reference| per unit tensor)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from helpers import assert_refresh_close, make_refresh_case, rel_err, run_refresh_gpu, run_refresh_oracle

pytestmark = pytest.mark.gpu

TOL = 1e-3


@pytest.mark.parametrize("kind,H_k", [(dasc.KDA, 4), (dasc.GDN, 2)])
def test_chunked_ragged_suffixes_both_modes(kind, H_k):
    # one token, a ragged tail, an empty request, exactly one chunk, several chunks with a tail
    case = make_refresh_case(21, kind, 2, 4, H_k, 128, 128, [1, 37, 0, 64, 200], scope=dasc.SCOPE_LAYER,
                             keep_ratio=0.5)
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED)
    worst = assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
    print("worst rel err", worst)
    np.testing.assert_array_equal(got_s[2], case.state0.cpu().numpy()[2])       # empty suffix: untouched
    ref_s, _ = run_refresh_oracle(case, mode=oracle.MODE_SCRATCH_MERGE_LOCAL, want_o=False)
    got_s, _ = run_refresh_gpu(case, mode=dasc.REFRESH_SCRATCH_MERGE_LOCAL, algo=dasc.ALGO_CHUNKED, want_o=False)
    assert_refresh_close(case, got_s, None, ref_s, None, TOL)
    keep = case.oplan.mask.astype(bool)
    s0 = case.state0.cpu().numpy()
    if kind == dasc.KDA:
        keep = keep.reshape(2, 4, 128)
        np.testing.assert_array_equal(got_s[:, keep], s0[:, keep])              # retained rows untouched
    else:
        np.testing.assert_array_equal(got_s[:, keep], s0[:, keep])


@pytest.mark.parametrize("with_o", [True, False])
def test_chunk_boundaries_of_the_producer_pipeline(with_o):
    # one chunk minus / exactly / plus one token, two and three chunks around their boundaries, two tokens: the
    # producer warps run a chunk ahead of the chain, so every count of chunks from 1 to 4 and every tail is a case
    case = make_refresh_case(27, dasc.KDA, 1, 2, 2, 128, 128, [31, 32, 33, 63, 64, 65, 96, 97, 2], scope=dasc.SCOPE_LAYER,
                             keep_ratio=0.38)
    ref_s, ref_o = run_refresh_oracle(case, want_o=with_o)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED, want_o=with_o)
    worst = assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
    print("worst rel err", worst)


def test_chunked_long_suffix_from_partially_restored_state():
    # aggressive KDA: keep 20 % of the channels, zero-fill the rest, then a 1024-token suffix
    case = make_refresh_case(3, dasc.KDA, 1, 2, 2, 128, 128, [1024], scope=dasc.SCOPE_LAYER, keep_ratio=0.2)
    keep = torch.from_numpy(case.oplan.mask.reshape(1, 2, 128, 1).astype(bool)).to(case.state0.device)
    case.state0 = torch.where(keep, case.state0, torch.zeros((), device=case.state0.device))
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED)
    worst = assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
    print("worst rel err", worst)


def test_chunked_matches_sequential_and_auto_picks_it():
    case = make_refresh_case(22, dasc.KDA, 1, 4, 4, 128, 128, [130, 64], scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    seq_s, seq_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL)
    chk_s, chk_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED, q_scale=1.0)
    auto_s, auto_o = run_refresh_gpu(case, algo=dasc.ALGO_AUTO)
    np.testing.assert_array_equal(auto_s, chk_s)            # AUTO = chunked for d = 128, bf16
    np.testing.assert_array_equal(auto_o, chk_o)
    for r in range(2):
        for h in range(4):
            assert rel_err(chk_s[r, 0, h], seq_s[r, 0, h]) <= TOL
    # bf16 output and a query scale
    ref_s, ref_o = run_refresh_oracle(case, q_scale=0.5)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_CHUNKED, q_scale=0.5, o_dtype=torch.bfloat16)
    for r in range(2):
        t0, t1 = int(case.cu[r]), int(case.cu[r + 1])
        for h in range(4):
            ref = ref_o[0, t0:t1, h]
            bound = TOL * np.abs(ref).max() + np.abs(ref) * 2.0 ** -8
            assert np.all(np.abs(got_o[0, t0:t1, h] - ref) <= bound)


def test_log_decay_outside_the_chunked_range_is_reported():
    # one channel of one head decays by e^-7 per token: 112 over half a chunk, beyond the 80 the midpoint
    # reference can hold in fp32.  The call must say so (DASC_ERR_DOMAIN from the status query); the same streams
    # go through the sequential kernel without complaint and match the oracle.
    import paper_2608_30386_b200.binding as binding
    case = make_refresh_case(31, dasc.KDA, 1, 2, 2, 128, 128, [64], scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    case.streams.g[0, :, 1, 5] = -7.0
    dev = case.state0.device
    s = case.streams
    state = case.state0.clone()
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(case.plan, 1, 1, dasc.ALGO_CHUNKED), dtype=torch.uint8, device=dev)
    dasc.dasc_refresh(case.plan, state, 2 * 128 * 128, 2 * 128 * 128, torch.arange(1, dtype=torch.int32, device=dev),
                      s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), 64, 64, o=None, algo=dasc.ALGO_CHUNKED, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == binding.ERR_DOMAIN
    assert dasc.status_string(binding.ERR_DOMAIN) == "log-decay outside the chunked kernel's range"
    # a call inside the range clears the flag again
    case.streams.g[0, :, 1, 5] = -1.0
    dasc.dasc_refresh(case.plan, state, 2 * 128 * 128, 2 * 128 * 128, torch.arange(1, dtype=torch.int32, device=dev),
                      s.q, s.k, s.v, s.g, s.beta, case.cu.to(dev), 64, 64, o=None, algo=dasc.ALGO_CHUNKED, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == binding.OK
    case.streams.g[0, :, 1, 5] = -7.0
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL)
    assert_refresh_close(case, got_s, got_o, ref_s, ref_o, TOL)
