"""GPU parity at the sizes of the benchmark configurations, in the launch configuration
bench.py times: the whole batch runs through the C ABI; all requests are checked on the device
by properties, sampled requests / units are compared with the oracle on the same bits."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth
from helpers import bits, make_plans
from helpers_fullsize import check_sampled_refresh, sample_units

pytestmark = pytest.mark.gpu
TOL = 1e-3


def _streams(dgen, kind, L, T, H_v, H_k, d, rates, dev):
    """Token streams drawn layer by layer on the device (bounds the generator's temporaries)."""
    parts = [synth.token_streams(dgen, kind, 1, T, H_v, H_k, d, d, rates[l:l + 1], device=dev) for l in range(L)]
    cat = lambda f: torch.cat([getattr(p, f) for p in parts])
    return cat("q"), cat("k"), cat("v"), cat("g"), cat("beta")


def test_gdn_headwise_config_pack_restore_refresh():
    """36 layers, 32 value heads / 16 key heads, d = 128, keep the 16 longest-horizon heads of every
    layer, 128 requests (9 GiB of dense state), refresh over a 256-token bf16 suffix."""
    dev = "cuda"
    L, H_v, H_k, d, n_req, suffix = 36, 32, 16, 128, 128, 256
    gen = synth.generator(2)
    rates = synth.decay_rates(gen, L, H_v, 1, 1e-4, 1.0)
    plan, oplan = make_plans(dasc.GDN, L, H_v, H_k, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    assert np.all(plan.layer_counts() == 16) and plan.unit_floats == d * d
    dgen = synth.generator(2, dev)
    dense = H_v * d * d
    state = synth.states(dgen, (L, n_req, dense), dev)
    ls, rs = n_req * dense, dense
    pool = torch.empty((n_req, int(plan.slot_floats)), device=dev)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    slots = torch.randperm(n_req, generator=gen).to(torch.int32).to(dev)
    dasc.dasc_pack(plan, state, ls, rs, ids, pool, slots)
    active = torch.full_like(state, float("nan"))
    dasc.dasc_restore(plan, pool, slots, active, ls, rs, ids)
    torch.cuda.synchronize()
    keep = torch.from_numpy(oplan.mask.astype(bool)).to(dev).view(L, 1, H_v, 1).expand(L, 1, H_v, d * d).reshape(L, 1, dense)
    want = torch.where(keep, state, torch.zeros((), device=dev))
    assert torch.equal(active.view(torch.int32), want.view(torch.int32))
    del want, keep
    for r in (5, 127):                                                  # sampled requests against the oracle
        one = state[:, r].contiguous().cpu().numpy()
        o_pool = np.zeros((1, int(plan.slot_floats)), np.float32)
        oracle.pack(oplan.mask, d * d, one, dense, 0, [0], o_pool, int(plan.slot_floats), [0])
        np.testing.assert_array_equal(bits(pool[int(slots[r])]), o_pool[0].view(np.uint32))
        o_out = np.full_like(one, np.float32(-1.0))
        oracle.restore(oplan.mask, d * d, o_pool, int(plan.slot_floats), [0], o_out, dense, 0, [0])
        np.testing.assert_array_equal(bits(active[:, r]), o_out.view(np.uint32))
    del state, pool
    # refresh (CONTINUE) of the restored states
    T = n_req * suffix
    q, k, v, g, beta = _streams(dgen, synth.GDN, L, T, H_v, H_k, d, rates, dev)
    o = torch.empty((L, T, H_v, d), dtype=torch.float32, device=dev)
    cu = synth.uniform_cu_seqlens(n_req, suffix)
    before = active.clone()
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, n_req, L), dtype=torch.uint8, device=dev)
    dasc.dasc_refresh(plan, active, ls, rs, ids, q, k, v, g, beta, cu.to(dev), T, suffix, o=o, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    units = sample_units(2, n_req, L, H_v, 96)
    worst = check_sampled_refresh(dasc.GDN, plan, oplan, before, active, ls, rs, q, k, v, g, beta, o, cu, units, TOL)
    print("GDN config: worst sampled rel err", worst)


@pytest.mark.parametrize("suffix", [256, 1024, 4096])
def test_aggressive_kda_refresh_config(suffix):
    """24 layers x 32 heads x d = 128, keep 20 % of the channels per layer, batch 32, suffix 256 / 1024 / 4096
    bf16 tokens.  Token streams of all 24 layers do not fit beside each other at 4096 tokens, so the
    layers run in groups through layer_begin / layer_end, as the benchmark does; two groups are run here."""
    dev = "cuda"
    L, H, d, n_req = 24, 32, 128, 32
    gen = synth.generator(3)
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.2)
    dgen = synth.generator(3, dev)
    dense = H * d * d
    full = synth.states(dgen, (L, n_req, dense), dev)
    ls, rs = n_req * dense, dense
    pool = torch.empty((n_req, int(plan.slot_floats)), device=dev)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    dasc.dasc_pack(plan, full, ls, rs, ids, pool, ids)
    active = torch.empty_like(full)
    dasc.dasc_restore(plan, pool, ids, active, ls, rs, ids)      # partially restored state: 80 % of the rows are zero
    torch.cuda.synchronize()
    del full, pool
    T = n_req * suffix
    cu = synth.uniform_cu_seqlens(n_req, suffix)
    group = 2 if suffix == 4096 else 3
    worst = 0.0
    for lb in (0, L - group):                                      # first and last layer group
        q, k, v, g, beta = _streams(dgen, synth.KDA, group, T, H, H, d, rates[lb:lb + group], dev)
        o = torch.empty((group, T, H, d), dtype=torch.float32, device=dev)
        before = active.clone()
        ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, n_req, group), dtype=torch.uint8, device=dev)
        dasc.dasc_refresh(plan, active, ls, rs, ids, q, k, v, g, beta, cu.to(dev), T, suffix, layer_begin=lb,
                          layer_end=lb + group, o=o, workspace=ws)
        torch.cuda.synchronize()
        assert dasc.dasc_refresh_status(ws) == 0
        units = sample_units(suffix + lb, n_req, group, H, 8 if suffix == 4096 else 32)
        worst = max(worst, check_sampled_refresh(dasc.KDA, plan, oplan, before, active, ls, rs, q, k, v, g, beta, o,
                                                 cu, units, TOL, layer_begin=lb))
        # layers outside the group are untouched
        other = 5 if lb == 0 else 1
        assert torch.equal(active[other], before[other])
        del q, k, v, g, beta, o, before
    print(f"KDA 20 % config, suffix {suffix}: worst sampled rel err", worst)


def test_mixed_trace_two_streams():
    """A reduced mixed serving trace: KDA 24x32x128x128, keep 0.38, one bounded contiguous slot pool recycled least
    recently used first, event list from `synth.serving_trace` (seed 4, fewer and shorter requests than the benchmark's
    512 x [1 Ki, 128 Ki]).  In every round new checkpoints are packed on one stream while cached ones are restored and
    refreshed (suffix lengths uniform in [1, 1024], ragged) on another.  Every round is checked: stored slots bit for
    bit on the device, restored states against the masked checkpoint that the slot holds (evictions included), sampled
    refreshed units against the oracle."""
    dev = "cuda"
    L, H, d = 24, 32, 128
    n_slots, batch = 24, 8
    rounds, st = synth.serving_trace(4, n_requests=12, prefix_hi=16384, n_slots=n_slots, batch=batch, concurrency=6)
    assert st["evictions"] > 0 and st["hits"] > 0
    gen = synth.generator(4)
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.38)
    dgen = synth.generator(4, dev)
    dense = H * d * d
    ls, rs = batch * dense, dense
    pool = torch.zeros((n_slots, int(plan.slot_floats)), device=dev)
    keep_rows = torch.from_numpy(oplan.mask.astype(bool)).to(dev)             # [L, H*d]
    s_pack, s_load = torch.cuda.Stream(priority=-1), torch.cuda.Stream()
    ids = torch.arange(batch, dtype=torch.int32, device=dev)
    content = {}                           # slot -> seed of the checkpoint state it holds

    def ckpt_state(seed):                  # [L, dense] state of one checkpoint, regenerated on demand
        return synth.states(synth.generator(seed, dev), (L, dense), dev)

    checked_hits = 0
    for ri, r in enumerate(rounds):
        if checked_hits >= 3 and ri >= 6:
            break
        n_s, n_h = len(r.store_slots), len(r.hit_slots)
        seeds = [1000 * ri + j for j in range(n_s)]
        new_states = torch.zeros((L, batch, dense), device=dev)
        for j, sd in enumerate(seeds):
            new_states[:, j] = ckpt_state(sd)
        new_slots = torch.tensor(r.store_slots, dtype=torch.int32, device=dev)
        hit_slots = torch.tensor(r.hit_slots, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        if n_s:
            dasc.dasc_pack(plan, new_states, ls, rs, ids[:n_s], pool, new_slots, stream=s_pack)
        if n_h:
            cu = torch.zeros(n_h + 1, dtype=torch.int32)
            cu[1:] = torch.cumsum(torch.tensor(r.suffix, dtype=torch.int64), 0).to(torch.int32)
            T = int(cu[-1])
            q, k, v, g, beta = _streams(dgen, synth.KDA, L, T, H, H, d, rates, dev)
            o = torch.empty((L, T, H, d), dtype=torch.float32, device=dev)   # fp32 outputs: parity at 1e-3 (bf16 adds 2^-8)
            active = torch.empty((L, batch, dense), device=dev)
            ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, n_h, L), dtype=torch.uint8, device=dev)
            torch.cuda.synchronize()
            with torch.cuda.stream(s_load):
                dasc.dasc_restore(plan, pool, hit_slots, active, ls, rs, ids[:n_h], stream=s_load)
                restored = active.clone()
                dasc.dasc_refresh(plan, active, ls, rs, ids[:n_h], q, k, v, g, beta, cu.to(dev), T, max(r.suffix),
                                  o=o, workspace=ws, stream=s_load)
        torch.cuda.synchronize()
        # new checkpoints landed bit for bit
        if n_s:
            packed = new_states.view(L, batch, H * d, d)[:, :n_s][keep_rows.view(L, 1, H * d).expand(L, n_s, H * d)]
            packed = packed.view(L, n_s, -1, d).permute(1, 0, 2, 3).reshape(n_s, -1)
            assert torch.equal(pool[new_slots.long()].view(torch.int32), packed.view(torch.int32))
        if n_h:
            assert dasc.dasc_refresh_status(ws) == 0
            # restored = the checkpoint the slot held before this round, masked
            for j, slot in enumerate(r.hit_slots):
                src = ckpt_state(content[slot]).view(L, H * d, d)
                want = torch.where(keep_rows.view(L, H * d, 1), src, torch.zeros((), device=dev)).view(L, dense)
                assert torch.equal(restored[:, j].view(torch.int32), want.view(torch.int32))
            units = sample_units(40 + ri, n_h, L, H, 6)
            worst = check_sampled_refresh(dasc.KDA, plan, oplan, restored, active, ls, rs, q, k, v, g, beta, o, cu, units, TOL)
            print(f"mixed trace round {ri}: {n_s} stores, {n_h} hits, {T} tokens, worst sampled rel err {worst:.2e}")
            checked_hits += 1
            del q, k, v, g, beta, o, active, restored
        for slot, sd in zip(r.store_slots, seeds):
            content[slot] = sd
    assert checked_hits >= 3


def test_kda_serving_config_refresh_in_the_benchmarks_launch():
    """The benchmark line's own refresh launch: 64 requests x 24 layers x 32 heads in ONE call (49,152 CTAs), keep 0.38
    per layer, 256-token bf16 suffix, bf16 outputs, plus the state-only window refresh of the same tokens.  Sampled
    (request, layer, head) units against the oracle on the same bits."""
    dev = "cuda"
    L, H, d, n_req, suffix = 24, 32, 128, 64, 256
    gen = synth.generator(1)
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.38)
    dgen = synth.generator(1, dev)
    dense = H * d * d
    ls, rs = n_req * dense, dense
    active = synth.states(dgen, (L, n_req, dense), dev)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    T = n_req * suffix
    cu = synth.uniform_cu_seqlens(n_req, suffix)
    q, k, v, g, beta = _streams(dgen, synth.KDA, L, T, H, H, d, rates, dev)
    o = torch.empty((L, T, H, d), dtype=torch.bfloat16, device=dev)
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, n_req, L), dtype=torch.uint8, device=dev)
    before = active.clone()
    dasc.dasc_refresh(plan, active, ls, rs, ids, q, k, v, g, beta, cu.to(dev), T, suffix, o=o, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    units = sample_units(11, n_req, L, H, 128)
    # bf16 outputs carry their own rounding (half an ulp is up to 2^-8 of the value): states at 1e-3, outputs at 1e-3 + 2^-8
    worst = check_sampled_refresh(dasc.KDA, plan, oplan, before, active, ls, rs, q, k, v, g, beta, None, cu, units, TOL)
    worst_o = check_sampled_refresh(dasc.KDA, plan, oplan, before, active, ls, rs, q, k, v, g, beta, o, cu, units,
                                    TOL + 2.0 ** -8)
    print(f"KDA serving config, one launch: worst sampled state err {worst:.2e}, with bf16 outputs {worst_o:.2e}")
    # the same launch once more: every one of the 49,152 states and all outputs must come out with the same bits
    again, o2 = before.clone(), torch.empty_like(o)
    dasc.dasc_refresh(plan, again, ls, rs, ids, q, k, v, g, beta, cu.to(dev), T, suffix, o=o2, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    assert torch.equal(again.view(torch.int32), active.view(torch.int32))
    assert torch.equal(o2.view(torch.int16), o.view(torch.int16))
    del again, o2
    # the paper's load policy on the same launch shape: scratch replay of the same 256 tokens, no outputs
    merged = before.clone()
    wb = torch.empty(n_req, dtype=torch.int32, device=dev)
    dasc.dasc_refresh_window(plan, merged, ls, rs, ids, None, k, v, g, beta, cu.to(dev), T, wb, window=suffix, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0
    assert torch.equal(wb.cpu(), cu[:-1])
    worst_w = check_sampled_refresh(dasc.KDA, plan, oplan, before, merged, ls, rs, q, k, v, g, beta, None, cu, units, TOL,
                                    mode=oracle.MODE_SCRATCH_MERGE_LOCAL)
    print(f"window refresh, state only: worst sampled err {worst_w:.2e}")
