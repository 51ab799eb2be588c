"""GPU parity: dasc_pack / dasc_restore through the C ABI against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding, synth
from helpers import bits, make_plans

pytestmark = pytest.mark.gpu


def _roundtrip_case(seed, kind, L, H, d_k, d_v, n_req, n_slots, *, sel, scope=dasc.SCOPE_LAYER, keep_ratio=1.0,
                    w_max=0.0, layer_pad=0, req_pad=0, slot_pad=0, specials=True):
    dev = "cuda"
    gen = synth.generator(seed)
    uph = d_k if kind == dasc.KDA else 1
    rates = synth.decay_rates(gen, L, H, uph, 1e-3, 1.0)
    plan, oplan = make_plans(kind, L, H, H, d_k, d_v, rates, sel=sel, scope=scope, keep_ratio=keep_ratio, w_max=w_max)
    dense = H * d_k * d_v
    layer_stride = dense + layer_pad
    req_stride = L * layer_stride + req_pad
    slot_stride = int(plan.slot_floats) + slot_pad
    state = synth.states(gen, (n_req * req_stride,))
    if specials:
        synth.special_values_(state, gen)
    n_pairs = min(n_req, n_slots)
    src_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)
    dst_slot = torch.randperm(n_slots, generator=gen)[:n_pairs].to(torch.int32)
    dst_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)

    # --- CUDA path
    d_state = state.to(dev)
    d_pool = torch.full((n_slots * slot_stride + 4,), 7.0, device=dev)
    dasc.dasc_pack(plan, d_state, layer_stride, req_stride, src_req.to(dev), d_pool, dst_slot.to(dev),
                   slot_stride=slot_stride)
    d_out = torch.full_like(d_state, -3.0)
    dasc.dasc_restore(plan, d_pool, dst_slot.to(dev), d_out, layer_stride, req_stride, dst_req.to(dev),
                      slot_stride=slot_stride)
    torch.cuda.synchronize()

    # --- oracle on the same bits
    uw = int(plan.unit_floats)
    o_pool = np.full((n_slots * slot_stride + 4,), np.float32(7.0))
    oracle.pack(oplan.mask, uw, state.numpy(), layer_stride, req_stride, src_req.numpy(), o_pool, slot_stride,
                dst_slot.numpy())
    o_out = np.full(state.shape, np.float32(-3.0))
    oracle.restore(oplan.mask, uw, o_pool, slot_stride, dst_slot.numpy(), o_out, layer_stride, req_stride,
                   dst_req.numpy())
    np.testing.assert_array_equal(bits(d_pool), o_pool.view(np.uint32))
    np.testing.assert_array_equal(bits(d_out), o_out.view(np.uint32))
    return plan


def test_tiny_kda_config():
    # 1 layer, 4 heads, d = 64, keep 40 % of the channels of every head (26 of 64)
    plan = _roundtrip_case(0, dasc.KDA, 1, 4, 64, 64, n_req=4, n_slots=4, sel=dasc.SEL_TOP_RATIO,
                           scope=dasc.SCOPE_HEAD, keep_ratio=0.4)
    assert plan.units_retained == 4 * 26


@pytest.mark.parametrize("ratio", [0.0, 0.25, 0.38, 0.5, 1.0])
def test_kda_ragged_layer_scope(ratio):
    # several CTAs per (pair, layer), a ragged tail, padded strides
    _roundtrip_case(1, dasc.KDA, 5, 6, 128, 128, n_req=7, n_slots=9, sel=dasc.SEL_TOP_RATIO, keep_ratio=ratio,
                    layer_pad=64, req_pad=32, slot_pad=16)


def test_kda_threshold_and_odd_widths():
    _roundtrip_case(2, dasc.KDA, 3, 5, 48, 96, n_req=5, n_slots=5, sel=dasc.SEL_THRESHOLD, w_max=64.0)
    _roundtrip_case(3, dasc.KDA, 2, 3, 20, 12, n_req=3, n_slots=4, sel=dasc.SEL_THRESHOLD, w_max=128.0, layer_pad=4)


def test_gdn_head_units():
    _roundtrip_case(4, dasc.GDN, 6, 8, 128, 128, n_req=5, n_slots=6, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    _roundtrip_case(5, dasc.GDN, 2, 4, 64, 32, n_req=3, n_slots=3, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.3,
                    slot_pad=8)


def test_all_retained_roundtrip_is_identity_on_device():
    dev = "cuda"
    gen = synth.generator(6)
    L, H, d = 3, 4, 128
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, _ = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=1.0)
    state = synth.special_values_(synth.states(gen, (5, L, H, d, d)), gen).to(dev)
    pool = torch.zeros((5, int(plan.slot_floats)), device=dev)
    ids = torch.arange(5, dtype=torch.int32, device=dev)
    dasc.dasc_pack(plan, state, H * d * d, L * H * d * d, ids, pool, ids.flip(0).contiguous())
    out = torch.full_like(state, 1.0)
    dasc.dasc_restore(plan, pool, ids.flip(0).contiguous(), out, H * d * d, L * H * d * d, ids)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int32), state.view(torch.int32))


def test_empty_and_invalid_calls():
    dev = "cuda"
    gen = synth.generator(7)
    rates = synth.decay_rates(gen, 2, 2, 32, 1e-3, 1.0)
    plan, _ = make_plans(dasc.KDA, 2, 2, 2, 32, 32, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    state = torch.zeros(2 * 2 * 2 * 32 * 32, device=dev)
    pool = torch.full((2 * int(plan.slot_floats),), 5.0, device=dev)
    empty = torch.zeros(0, dtype=torch.int32, device=dev)
    dasc.dasc_pack(plan, state, 2 * 32 * 32, 2 * 2 * 32 * 32, empty, pool, empty)       # n_pairs = 0: no-op
    dasc.dasc_restore(plan, pool, empty, state, 2 * 32 * 32, 2 * 2 * 32 * 32, empty)
    torch.cuda.synchronize()
    assert torch.all(pool == 5.0)
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(dasc.DascError) as e:                                             # misaligned base
        dasc.dasc_pack(plan, state[1:], 2 * 32 * 32, 2 * 2 * 32 * 32, ids, pool, ids)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(dasc.DascError):                                                  # stride not 16-byte
        dasc.dasc_pack(plan, state, 2 * 32 * 32 + 2, 2 * 2 * 32 * 32, ids, pool, ids)
    with pytest.raises(dasc.DascError):                                                  # slot stride too small
        dasc.dasc_restore(plan, pool, ids, state, 2 * 32 * 32, 2 * 2 * 32 * 32, ids, slot_stride=4)
    torch.cuda.synchronize()
    assert torch.all(pool == 5.0) and torch.all(state == 0.0)


@pytest.mark.parametrize("ratio", [0.25, 0.38, 0.5, 1.0])
def test_serving_scale_kda_sampled_against_oracle(ratio):
    """24 layers x 32 heads x 128x128 fp32, 64 requests (3 GiB dense), the launch the benchmark
    times.  All requests are checked on the device by the masking property; three sampled
    requests and their slots are compared with the oracle bit for bit."""
    dev = "cuda"
    L, H, d, n_req = 24, 32, 128, 64
    gen = synth.generator(1)
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=ratio)
    dgen = synth.generator(1, dev)
    state = synth.states(dgen, (L, n_req, H * d, d), dev)           # layer-major active pool
    layer_stride, req_stride = n_req * H * d * d, H * d * d
    pool = torch.empty((n_req, int(plan.slot_floats)), device=dev)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    slots = torch.randperm(n_req, generator=gen).to(torch.int32).to(dev)
    dasc.dasc_pack(plan, state, layer_stride, req_stride, ids, pool, slots)
    out = torch.full_like(state, float("nan"))
    dasc.dasc_restore(plan, pool, slots, out, layer_stride, req_stride, ids)
    torch.cuda.synchronize()
    keep = torch.from_numpy(oplan.mask.astype(bool)).to(dev).view(L, 1, H * d, 1)
    want = torch.where(keep, state, torch.zeros((), device=dev))
    assert torch.equal(out.view(torch.int32), want.view(torch.int32))
    del want
    for r in (0, 17, 63):
        one = state[:, r].contiguous().cpu().numpy()                # [L, H*d, d]
        o_pool = np.zeros((1, int(plan.slot_floats)), np.float32)
        oracle.pack(oplan.mask, d, one, H * d * d, 0, [0], o_pool, int(plan.slot_floats), [0])
        np.testing.assert_array_equal(bits(pool[int(slots[r])]), o_pool[0].view(np.uint32))
        o_out = np.full_like(one, np.float32(-1.0))
        oracle.restore(oplan.mask, d, o_pool, int(plan.slot_floats), [0], o_out, H * d * d, 0, [0])
        np.testing.assert_array_equal(bits(out[:, r]), o_out.view(np.uint32))


def test_mixed_per_head_ratios_explicit_mask():
    """Every head keeps its own fraction of channels (ragged per-head counts): the mask is assembled from head-scope
    plans of the library and fed back as an explicit mask; pack / restore against the oracle on that mask."""
    dev = "cuda"
    gen = synth.generator(9)
    L, H, d = 3, 8, 128
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    A, B = synth.decay_params(rates)
    ratios = (0.25, 0.38, 0.5, 1.0)
    masks = [dasc.dasc_plan(dasc.KDA, L, H, H, d, d, A.numpy(), B.numpy(), sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_HEAD,
                            keep_ratio=r, device=-1).mask().reshape(L, H, d) for r in ratios]
    pick = torch.randint(0, 4, (L, H), generator=gen).numpy()
    mask = np.choose(pick[:, :, None], masks).reshape(L, H * d).astype(np.uint8)
    counts = mask.reshape(L, H, d).sum(-1)
    assert len(set(counts.ravel().tolist())) > 1                    # ragged per-head channel counts
    plan = dasc.dasc_plan(dasc.KDA, L, H, H, d, d, A.numpy(), B.numpy(), sel=dasc.SEL_EXPLICIT, explicit_mask=mask)
    oplan = oracle.plan(oracle.KDA, L, H, d, A.numpy(), B.numpy(), sel=oracle.SEL_EXPLICIT, explicit_mask=mask,
                        unit_bytes=d * 4)
    np.testing.assert_array_equal(plan.mask(), oplan.mask)
    np.testing.assert_array_equal(plan.mask(), mask)
    dense, n_req = H * d * d, 5
    state = synth.states(gen, (n_req, L, dense))
    synth.special_values_(state, gen)
    ids = torch.arange(n_req, dtype=torch.int32)
    slots = torch.flip(ids, [0]).contiguous()
    slot = int(plan.slot_floats)
    d_pool = torch.full((n_req, slot), 7.0, device=dev)
    dasc.dasc_pack(plan, state.to(dev), dense, L * dense, ids.to(dev), d_pool, slots.to(dev))
    d_out = torch.full((n_req, L, dense), -3.0, device=dev)
    dasc.dasc_restore(plan, d_pool, slots.to(dev), d_out, dense, L * dense, ids.to(dev))
    torch.cuda.synchronize()
    o_pool = np.full((n_req, slot), np.float32(7.0))
    oracle.pack(oplan.mask, d, state.numpy(), dense, L * dense, ids.numpy(), o_pool, slot, slots.numpy())
    o_out = np.full((n_req, L, dense), np.float32(-3.0))
    oracle.restore(oplan.mask, d, o_pool, slot, slots.numpy(), o_out, dense, L * dense, ids.numpy())
    np.testing.assert_array_equal(bits(d_pool), o_pool.view(np.uint32))
    np.testing.assert_array_equal(bits(d_out), o_out.view(np.uint32))


@pytest.mark.gpu
def test_a_saved_and_reloaded_plan_packs_and_restores_the_same_bits():
    import torch
    import paper_2608_30386_b200 as dasc
    from paper_2608_30386_b200 import synth
    from helpers import bits, make_plans
    gen = synth.generator(91)
    L, H, d = 3, 4, 32
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_LAYER, keep_ratio=0.38)
    again = dasc.dasc_plan_load(dasc.dasc_plan_save(plan), device=0)
    assert again.device == 0 and again.units_retained == plan.units_retained
    dense = H * d * d
    state = synth.states(gen, (2, L, dense)).cuda()
    ids = torch.arange(2, dtype=torch.int32, device="cuda")
    pools, outs = [], []
    for p in (plan, again):
        pool = torch.zeros((2, int(p.slot_floats)), device="cuda")
        out = torch.full_like(state, float("nan"))
        dasc.dasc_pack(p, state, dense, L * dense, ids, pool, ids)
        dasc.dasc_restore(p, pool, ids, out, dense, L * dense, ids)
        pools.append(bits(pool))
        outs.append(bits(out))
    np.testing.assert_array_equal(pools[0], pools[1])
    np.testing.assert_array_equal(outs[0], outs[1])
