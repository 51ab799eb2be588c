"""GPU parity: dasc_pack_padded / dasc_restore_padded (Appendix B, Scheme 1 pool [L][slots][R_max][unit])
through the C ABI against the oracle, bit for bit, padding included."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth
from helpers import bits, make_plans

pytestmark = pytest.mark.gpu


def _case(seed, kind, L, H, d_k, d_v, n_req, n_slots, *, sel, scope=dasc.SCOPE_LAYER, keep_ratio=1.0, w_max=0.0,
          layer_pad=0, req_pad=0):
    dev = "cuda"
    gen = synth.generator(seed)
    uph = d_k if kind == dasc.KDA else 1
    rates = synth.decay_rates(gen, L, H, uph, 1e-3, 1.0)
    plan, oplan = make_plans(kind, L, H, H, d_k, d_v, rates, sel=sel, scope=scope, keep_ratio=keep_ratio, w_max=w_max)
    dense = H * d_k * d_v
    layer_stride = dense + layer_pad
    req_stride = L * layer_stride + req_pad
    state = synth.states(gen, (n_req * req_stride,))
    synth.special_values_(state, gen)
    n_pairs = min(n_req, n_slots)
    src_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)
    dst_slot = torch.randperm(n_slots, generator=gen)[:n_pairs].to(torch.int32)
    dst_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)
    uw, R_max = int(plan.unit_floats), int(plan.r_max)
    floats = dasc.dasc_padded_pool_floats(plan, n_slots)
    assert floats == L * n_slots * R_max * uw

    d_state = state.to(dev)
    d_pool = torch.full((max(floats, 4) + 4,), 7.0, device=dev)
    dasc.dasc_pack_padded(plan, d_state, layer_stride, req_stride, src_req.to(dev), d_pool, n_slots, dst_slot.to(dev))
    d_out = torch.full_like(d_state, -3.0)
    dasc.dasc_restore_padded(plan, d_pool, n_slots, dst_slot.to(dev), d_out, layer_stride, req_stride, dst_req.to(dev))
    torch.cuda.synchronize()

    o_pool = np.full((max(floats, 4) + 4,), np.float32(7.0))
    oracle.pack_padded(oplan.mask, uw, state.numpy(), layer_stride, req_stride, src_req.numpy(), o_pool, n_slots, R_max,
                       dst_slot.numpy())
    o_out = np.full(state.shape, np.float32(-3.0))
    oracle.restore_padded(oplan.mask, uw, o_pool, n_slots, R_max, dst_slot.numpy(), o_out, layer_stride, req_stride,
                          dst_req.numpy())
    np.testing.assert_array_equal(bits(d_pool), o_pool.view(np.uint32))       # padding keeps its 7.0 on both sides
    np.testing.assert_array_equal(bits(d_out), o_out.view(np.uint32))
    return plan


def test_tiny_kda_config():
    _case(0, dasc.KDA, 1, 4, 64, 64, n_req=4, n_slots=4, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_HEAD, keep_ratio=0.4)


@pytest.mark.parametrize("ratio", [0.0, 0.25, 1.0])
def test_kda_model_scope_makes_layers_ragged(ratio):
    # model-wide top ratio: r_l differs from layer to layer, so most layers have padding
    plan = _case(1, dasc.KDA, 5, 6, 128, 128, n_req=7, n_slots=9, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_MODEL,
                 keep_ratio=ratio, layer_pad=64, req_pad=32)
    if 0 < ratio < 1:
        assert plan.r_max * 5 > plan.units_retained


def test_threshold_rule_and_odd_widths():
    _case(2, dasc.KDA, 3, 5, 48, 96, n_req=5, n_slots=5, sel=dasc.SEL_THRESHOLD, w_max=64.0)
    _case(3, dasc.KDA, 2, 3, 20, 12, n_req=3, n_slots=4, sel=dasc.SEL_THRESHOLD, w_max=128.0, layer_pad=4)


def test_gdn_head_units():
    _case(4, dasc.GDN, 6, 8, 128, 128, n_req=5, n_slots=6, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_MODEL, keep_ratio=0.4)
    _case(5, dasc.GDN, 2, 4, 64, 32, n_req=3, n_slots=3, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.3)


def test_both_layouts_restore_the_same_state():
    dev = "cuda"
    gen = synth.generator(6)
    L, H, d = 4, 4, 128
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, _ = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_THRESHOLD, w_max=64.0)
    dense = H * d * d
    state = synth.states(gen, (3, L, dense)).to(dev)
    ids = torch.arange(3, dtype=torch.int32, device=dev)
    ragged = torch.empty((3, int(plan.slot_floats)), device=dev)
    padded = torch.empty(dasc.dasc_padded_pool_floats(plan, 3), device=dev)
    dasc.dasc_pack(plan, state, dense, L * dense, ids, ragged, ids)
    dasc.dasc_pack_padded(plan, state, dense, L * dense, ids, padded, 3, ids)
    a, b = torch.full_like(state, 1.0), torch.full_like(state, 2.0)
    dasc.dasc_restore(plan, ragged, ids, a, dense, L * dense, ids)
    dasc.dasc_restore_padded(plan, padded, 3, ids, b, dense, L * dense, ids)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
