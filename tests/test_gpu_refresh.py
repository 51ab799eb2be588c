"""GPU parity: dasc_refresh through the C ABI against the token-by-token fp64 oracle.

Tolerances (max abs error / max |reference| per unit tensor): 1e-3 with bf16 q/k/v and fp32
state, 1e-5 with all-fp32 inputs.  Outputs are compared in fp32; a bf16 output tensor is
checked separately to be the rounding of a value within tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from helpers import (assert_refresh_close, make_refresh_case, rel_err, run_refresh_gpu, run_refresh_oracle)

pytestmark = pytest.mark.gpu

TOL_BF16 = 1e-3
TOL_FP32 = 1e-5


@pytest.mark.parametrize("io_dtype,tol", [(torch.bfloat16, TOL_BF16), (torch.float32, TOL_FP32)])
def test_tiny_kda_config_both_modes(io_dtype, tol):
    # 1 layer, 4 heads, d = 64, keep 40 % per head, suffix 64 tokens
    case = make_refresh_case(0, dasc.KDA, 1, 4, 4, 64, 64, [64], io_dtype=io_dtype)
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL)
    assert_refresh_close(case, got_s, got_o, ref_s, ref_o, tol)
    ref_s, _ = run_refresh_oracle(case, mode=oracle.MODE_SCRATCH_MERGE_LOCAL, want_o=False)
    got_s, _ = run_refresh_gpu(case, mode=dasc.REFRESH_SCRATCH_MERGE_LOCAL, algo=dasc.ALGO_SEQUENTIAL, want_o=False)
    assert_refresh_close(case, got_s, None, ref_s, None, tol)
    # retained rows are untouched bit for bit in the merge mode
    keep = case.oplan.mask.reshape(1, 4, 64).astype(bool)
    s0 = case.state0.cpu().numpy()
    np.testing.assert_array_equal(got_s[0][keep], s0[0][keep])


def test_tiny_kda_checkpoint_every_64_tokens():
    # prefix 256 with a checkpoint every 64 tokens: pack -> restore -> refresh per segment,
    # everything retained, equals the uninterrupted replay of the whole prefix
    case = make_refresh_case(0, dasc.KDA, 1, 4, 4, 64, 64, [256], io_dtype=torch.float32, keep_ratio=1.0)
    case.state0.zero_()
    ref_s, ref_o = run_refresh_oracle(case)
    dev = case.state0.device
    state = case.state0.clone()
    pool = torch.zeros((1, int(case.plan.slot_floats)), device=dev)
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    dense = 4 * 64 * 64
    s = case.streams
    o_all = torch.zeros((1, 256, 4, 64), device=dev)
    for seg in range(4):
        sl = slice(seg * 64, (seg + 1) * 64)
        cu = torch.tensor([0, 64], dtype=torch.int32, device=dev)
        o = torch.zeros((1, 64, 4, 64), device=dev)
        dasc.dasc_refresh(case.plan, state, dense, dense, ids, s.q[:, sl].contiguous(), s.k[:, sl].contiguous(),
                          s.v[:, sl].contiguous(), s.g[:, sl].contiguous(), s.beta[:, sl].contiguous(), cu, 64, 64,
                          o=o, algo=dasc.ALGO_SEQUENTIAL)
        o_all[:, sl] = o
        dasc.dasc_pack(case.plan, state, dense, dense, ids, pool, ids)
        state.fill_(float("nan"))
        dasc.dasc_restore(case.plan, pool, ids, state, dense, dense, ids)
    torch.cuda.synchronize()
    assert_refresh_close(case, state.cpu().numpy().reshape(1, 1, 4, 64, 64), o_all.cpu().numpy(), ref_s, ref_o, TOL_FP32)


@pytest.mark.parametrize("kind,H_k", [(dasc.KDA, 4), (dasc.GDN, 2)])
@pytest.mark.parametrize("io_dtype,tol", [(torch.bfloat16, TOL_BF16), (torch.float32, TOL_FP32)])
def test_sequential_d128_ragged_suffixes(kind, H_k, io_dtype, tol):
    # d = 128; suffixes of 1, 37, 0, 100 tokens span token groups with ragged tails and an empty request
    case = make_refresh_case(11, kind, 2, 4, H_k, 128, 128, [1, 37, 0, 100], io_dtype=io_dtype,
                             scope=dasc.SCOPE_LAYER, keep_ratio=0.5)
    ref_s, ref_o = run_refresh_oracle(case)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL)
    assert_refresh_close(case, got_s, got_o, ref_s, ref_o, tol)
    # the empty request's state is untouched
    np.testing.assert_array_equal(got_s[2], case.state0.cpu().numpy()[2])
    ref_s, _ = run_refresh_oracle(case, mode=oracle.MODE_SCRATCH_MERGE_LOCAL, want_o=False)
    got_s, _ = run_refresh_gpu(case, mode=dasc.REFRESH_SCRATCH_MERGE_LOCAL, algo=dasc.ALGO_SEQUENTIAL, want_o=False)
    assert_refresh_close(case, got_s, None, ref_s, None, tol)


def test_sequential_layer_range_q_scale_and_bf16_output():
    case = make_refresh_case(12, dasc.KDA, 3, 2, 2, 128, 128, [50, 20], io_dtype=torch.bfloat16)
    ref_s, ref_o = run_refresh_oracle(case, q_scale=0.125)
    got_s, got_o = run_refresh_gpu(case, algo=dasc.ALGO_SEQUENTIAL, q_scale=0.125, layer_begin=1, layer_end=3,
                                   o_dtype=torch.bfloat16)
    s0 = case.state0.cpu().numpy()
    np.testing.assert_array_equal(got_s[:, 0], s0[:, 0])             # layer 0 not in the call
    for r in range(2):
        t0, t1 = int(case.cu[r]), int(case.cu[r + 1])
        for l in (1, 2):
            for h in range(2):
                assert rel_err(got_s[r, l, h], ref_s[r, l, h]) <= TOL_BF16
                ref = ref_o[l, t0:t1, h]
                got = got_o[l - 1, t0:t1, h]
                # bf16 output: within tolerance plus half a bf16 ulp of each element
                bound = TOL_BF16 * np.abs(ref).max() + np.abs(ref) * 2.0 ** -8
                assert np.all(np.abs(got - ref) <= bound)


def test_refresh_argument_errors():
    case = make_refresh_case(13, dasc.KDA, 1, 2, 2, 64, 64, [8], io_dtype=torch.float32)
    dev = case.state0.device
    s = case.streams
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    state = case.state0.clone()
    with pytest.raises(dasc.DascError):          # layer range outside the plan
        dasc.dasc_refresh(case.plan, state, 2 * 64 * 64, 2 * 64 * 64, ids, s.q, s.k, s.v, s.g, s.beta,
                          case.cu.to(dev), 8, 8, layer_begin=0, layer_end=2)
    with pytest.raises(dasc.DascError):          # the chunked kernel needs d = 128
        dasc.dasc_refresh(case.plan, state, 2 * 64 * 64, 2 * 64 * 64, ids, s.q, s.k, s.v, s.g, s.beta,
                          case.cu.to(dev), 8, 8, algo=dasc.ALGO_CHUNKED)
    torch.cuda.synchronize()
    assert torch.equal(state, case.state0)
