"""Host logic of the library (no GPU): the C-ABI loads and exports every declared
symbol, and the plan builder agrees with the oracle's plan on seeded inputs."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dasc.h")).read()
    declared = set(re.findall(r"\b(dasc_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    L = dasc.lib()
    for name in declared:
        assert isinstance(getattr(L, name), ctypes._CFuncPtr)
    assert re.fullmatch(r"\d+\.\d+\.\d+", dasc.version())
    assert dasc.status_string(binding.ERR_TIMEOUT) == "device-side wait timed out"


def _rates(rng, shape, lo=1e-3, hi=1.0):
    return np.exp(rng.uniform(math.log(lo), math.log(hi), size=shape)).astype(np.float32)


def _compare(p: dasc.Plan, o: oracle.Plan, unit_floats):
    np.testing.assert_array_equal(p.mask(), o.mask)
    np.testing.assert_allclose(p.horizon(), o.Hs, rtol=1e-14)
    np.testing.assert_array_equal(p.layer_counts(), o.r_l)
    np.testing.assert_array_equal(p.layer_offsets(), o.o_l)
    np.testing.assert_array_equal(p.window().astype(np.float64), o.W_u)
    assert p.units_total == o.sum_n and p.units_retained == o.sum_r and p.r_max == o.R_max
    assert p.slot_floats == o.sum_r * unit_floats
    assert p.w_replay == o.W_replay and p.w_max_used == o.w_max_used
    for a, b in ((p.c_temp_rag, o.C_temp_rag), (p.c_temp_pad, o.C_temp_pad), (p.c_ckpt_rag, o.C_ckpt_rag)):
        assert a == b or a == pytest.approx(b, rel=1e-14)


@pytest.mark.parametrize("w_max", [4.0, 16.0, 64.0, 512.0, 1e6])
def test_threshold_plan_matches_oracle(w_max):
    rng = np.random.default_rng(int(w_max))
    L, H, d = 5, 6, 32
    A_log = np.log(_rates(rng, (L, H, d)))
    dt = rng.normal(scale=0.5, size=(L, H, d)).astype(np.float32)
    p = dasc.dasc_plan(dasc.KDA, L, H, H, d, 64, A_log, dt, w_max=w_max, conv_bytes_per_ckpt=12345, device=-1)
    o = oracle.plan(oracle.KDA, L, H, d, A_log, dt, w_max=w_max, unit_bytes=64 * 4, conv_bytes=12345)
    _compare(p, o, 64)
    assert p.device == -1 and p.unit_floats == 64 and p.units_per_layer == H * d


@pytest.mark.parametrize("kind,scope,ratio", [
    (dasc.KDA, dasc.SCOPE_HEAD, 0.4), (dasc.KDA, dasc.SCOPE_LAYER, 0.38), (dasc.KDA, dasc.SCOPE_LAYER, 0.2),
    (dasc.KDA, dasc.SCOPE_MODEL, 0.25), (dasc.KDA, dasc.SCOPE_LAYER, 1.0), (dasc.KDA, dasc.SCOPE_LAYER, 0.0),
    (dasc.GDN, dasc.SCOPE_LAYER, 0.5), (dasc.GDN, dasc.SCOPE_MODEL, 0.3),
])
def test_top_ratio_plan_matches_oracle(kind, scope, ratio):
    rng = np.random.default_rng(7)
    L, H, d = 4, 8, 16
    uph = d if kind == dasc.KDA else 1
    rates = _rates(rng, (L, H, uph), 1e-4, 1.0)
    rates[0, 1, 0] = rates[0, 2, 0] = rates[0, 5, 0]          # ties
    A_log = np.log(rates)
    dt = np.zeros_like(A_log)
    p = dasc.dasc_plan(kind, L, H, H // 2, d, d, A_log, dt, sel=dasc.SEL_TOP_RATIO, scope=scope, keep_ratio=ratio,
                       device=-1)
    o = oracle.plan(kind, L, H, uph, A_log, dt, sel=oracle.SEL_TOP_RATIO, keep_ratio=ratio, scope=scope,
                    unit_bytes=(d if kind == dasc.KDA else d * d) * 4)
    _compare(p, o, d if kind == dasc.KDA else d * d)


def test_random_and_explicit_plans_match_oracle():
    rng = np.random.default_rng(8)
    L, H, d = 3, 4, 16
    A_log = np.log(_rates(rng, (L, H, d)))
    dt = np.zeros_like(A_log)
    for seed in (1234, 2027, 3407, 4519, 5683):
        p = dasc.dasc_plan(dasc.KDA, L, H, H, d, d, A_log, dt, w_max=64.0, randomize=True, seed=seed, device=-1)
        o = oracle.plan(oracle.KDA, L, H, d, A_log, dt, w_max=64.0, randomize=True, seed=seed, unit_bytes=d * 4)
        _compare(p, o, d)
    em = (rng.random((L, H * d)) < 0.3).astype(np.uint8)
    p = dasc.dasc_plan(dasc.KDA, L, H, H, d, d, A_log, dt, sel=dasc.SEL_EXPLICIT, explicit_mask=em, device=-1)
    o = oracle.plan(oracle.KDA, L, H, d, A_log, dt, sel=oracle.SEL_EXPLICIT, explicit_mask=em, unit_bytes=d * 4)
    _compare(p, o, d)
    np.testing.assert_array_equal(p.mask(), em)


def test_benchmark_scale_plan_matches_oracle():
    # 24 layers x 32 heads x 128 channels, keep 38 % per layer: the serving-scale KDA shape
    rng = np.random.default_rng(1)
    L, H, d = 24, 32, 128
    A_log = np.log(_rates(rng, (L, H, d)))
    dt = np.zeros_like(A_log)
    p = dasc.dasc_plan(dasc.KDA, L, H, H, d, d, A_log, dt, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_LAYER,
                       keep_ratio=0.38, device=-1)
    o = oracle.plan(oracle.KDA, L, H, d, A_log, dt, sel=oracle.SEL_TOP_RATIO, keep_ratio=0.38,
                    scope=oracle.SCOPE_LAYER, unit_bytes=d * 4)
    _compare(p, o, d)
    assert np.all(p.layer_counts() == math.ceil(0.38 * 4096))
    assert p.slot_floats * 4 == 24 * 1557 * 512


def test_plan_argument_errors():
    A = np.zeros((1, 2, 8), np.float32)
    with pytest.raises(dasc.DascError) as e:
        dasc.dasc_plan(dasc.KDA, 1, 2, 2, 8, 6, A, A, device=-1)             # d_v not a multiple of 4
    assert e.value.status == binding.ERR_SHAPE
    with pytest.raises(dasc.DascError) as e:
        dasc.dasc_plan(dasc.KDA, 1, 2, 2, 8, 8, A, A, eps=2.0, device=-1)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(dasc.DascError):
        dasc.dasc_plan(dasc.KDA, 1, 2, 2, 8, 8, A, A, sel=dasc.SEL_TOP_RATIO, keep_ratio=1.5, device=-1)
    with pytest.raises(dasc.DascError):
        dasc.dasc_plan(dasc.GDN, 1, 3, 2, 8, 8, np.zeros((1, 3, 1), np.float32), np.zeros((1, 3, 1), np.float32), device=-1)
    with pytest.raises(ValueError):
        dasc.dasc_plan(dasc.KDA, 1, 2, 2, 8, 8, A[:, :1], A[:, :1], device=-1)
    # device calls on a host-only plan are refused before any CUDA work
    p = dasc.dasc_plan(dasc.KDA, 1, 2, 2, 8, 8, A, A, device=-1)
    st = dasc.lib().dasc_pack(p.handle, None, 0, 0, None, None, 0, None, 1, None)
    assert st == binding.ERR_INVALID_ARG


def test_checkpoint_accounting_and_slot_budget_match_oracle_and_paper():
    """Host arithmetic of Eq. 6 / Appendix B / Appendix C.1 against the oracle's plan and the paper's byte budgets."""
    rng = np.random.default_rng(11)
    L, H, d = 6, 4, 32
    A_log = np.log(_rates(rng, (L, H, d)))
    dt = np.zeros_like(A_log)
    conv = 4096
    p = dasc.dasc_plan(dasc.KDA, L, H, H, d, 64, A_log, dt, w_max=64.0, conv_bytes_per_ckpt=conv, device=-1)
    o = oracle.plan(oracle.KDA, L, H, d, A_log, dt, w_max=64.0, unit_bytes=64 * 4, conv_bytes=conv)
    rag = dasc.dasc_checkpoint_bytes(p, dasc.LAYOUT_RAGGED, conv)
    pad = dasc.dasc_checkpoint_bytes(p, dasc.LAYOUT_PADDED, conv)
    dense = dasc.dasc_checkpoint_bytes(p, dasc.LAYOUT_DENSE, conv)
    assert rag == o.sum_r * 256 + conv and pad == L * o.R_max * 256 + conv and dense == o.sum_n * 256 + conv
    assert dense / rag == pytest.approx(o.C_ckpt_rag, rel=1e-14)
    # temporal-only ratios: the layout gain is R_max / mean(r_l)
    t = [dasc.dasc_checkpoint_bytes(p, lay, 0) for lay in (dasc.LAYOUT_RAGGED, dasc.LAYOUT_PADDED, dasc.LAYOUT_DENSE)]
    assert t[2] / t[0] == pytest.approx(o.C_temp_rag) and t[2] / t[1] == pytest.approx(o.C_temp_pad)
    assert t[1] / t[0] == pytest.approx(o.R_max / o.r_l.mean())
    assert dasc.dasc_padded_pool_floats(p, 7) == L * 7 * o.R_max * 64
    # slot budget: the oracle's function on the same inputs, and the paper's dense budgets (128 slots -> 127)
    for budget, per_rank, cv in ((1000, [90, 240, 10], 10), (694681600, [5242880] * 8, 184320),
                                 (1236271104, [9437184] * 8, 221184)):
        assert dasc.dasc_slot_budget(budget, per_rank, cv) == oracle.slot_budget(budget, per_rank, cv)
    assert dasc.dasc_slot_budget(694681600, [20 * 32 * 128 * 128 * 4 // 8] * 8, 20 * 3 * (3 * 32 * 128) // 8 * 2) == 127
    with pytest.raises(dasc.DascError):
        dasc.dasc_checkpoint_bytes(p, 9, 0)
    with pytest.raises(dasc.DascError):
        dasc.dasc_slot_budget(100, [0, 0], 0)


@pytest.mark.parametrize("kind,H,hpb,T", [(dasc.KDA, 8, 1, 2), (dasc.KDA, 32, 1, 8), (dasc.GDN, 32, 2, 8), (dasc.GDN, 8, 2, 4)])
def test_head_bundle_placement_matches_oracle(kind, H, hpb, T):
    # Section 4.3, first stage: the library's placement (sort-based) against the oracle's (scan-based) on the bundle
    # weights of a seeded plan, and the payloads it reports against a recount from the mask
    rng = np.random.default_rng(H * 10 + T)
    L, d = 4, 16
    uph = d if kind == dasc.KDA else 1
    A_log = np.log(_rates(rng, (L, H, uph)))
    p = dasc.dasc_plan(kind, L, H, H // hpb, d, d, A_log, np.zeros_like(A_log), sel=dasc.SEL_TOP_RATIO,
                       scope=dasc.SCOPE_MODEL, keep_ratio=0.37, device=-1)
    perm, U = dasc.dasc_tp_head_permutation(p, T, hpb)
    weight = p.mask().reshape(L, H // hpb, hpb * uph).sum(-1)
    o_perm, o_U = oracle.tp_head_permutation(weight, T)
    np.testing.assert_array_equal(perm, o_perm)
    np.testing.assert_array_equal(U, o_U)
    assert U.sum() == p.units_retained
    # the placement never leaves the heaviest rank above the contiguous split's heaviest rank on these profiles
    per = (H // hpb) // T
    contiguous = weight.reshape(L, T, per).sum((0, 2))
    assert U.max() <= contiguous.max()
    with pytest.raises(dasc.DascError):
        dasc.dasc_tp_head_permutation(p, 3, hpb)             # bundles do not divide among 3 ranks


def test_plan_save_and_load_round_trip_and_reject_damaged_blobs():
    rng = np.random.default_rng(77)
    for kind, H, Hk, d in ((dasc.KDA, 4, 4, 16), (dasc.GDN, 8, 4, 8)):
        L = 3
        uph = d if kind == dasc.KDA else 1
        A_log = np.log(_rates(rng, (L, H, uph)))
        p = dasc.dasc_plan(kind, L, H, Hk, d, d, A_log, np.zeros_like(A_log), sel=dasc.SEL_TOP_RATIO,
                           scope=dasc.SCOPE_MODEL, keep_ratio=0.37, conv_bytes_per_ckpt=4096, device=-1)
        blob = dasc.dasc_plan_save(p)
        q = dasc.dasc_plan_load(blob, device=-1)
        for f, _ in binding.PlanInfo._fields_:
            assert getattr(q.info, f) == getattr(p.info, f), f
        np.testing.assert_array_equal(q.mask(), p.mask())
        np.testing.assert_array_equal(q.horizon(), p.horizon())
        np.testing.assert_array_equal(q.window(), p.window())
        np.testing.assert_array_equal(q.layer_counts(), p.layer_counts())
        np.testing.assert_array_equal(q.layer_offsets(), p.layer_offsets())
        assert dasc.dasc_plan_save(q) == blob
        # damaged blobs are refused: truncated, wrong magic, a mask that no longer matches the counts, a bad shape field
        bad = [blob[:-1], b"X" + blob[1:], blob[:-1] + bytes([blob[-1] ^ 1])]
        shape = bytearray(blob)
        shape[24 + 4] ^= 0x7F                                   # n_layers inside the info struct
        bad.append(bytes(shape))
        for b in bad:
            with pytest.raises(dasc.DascError) as e:
                dasc.dasc_plan_load(b, device=-1)
            assert e.value.status == binding.ERR_INVALID_ARG
