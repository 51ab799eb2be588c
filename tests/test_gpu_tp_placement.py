"""TP-balanced placement on the device (Section 4.3, second stage): every virtual rank packs its own retained units
straight into the pools of the ranks that own them, and gathers them back.  The ranks are virtual -- T plans, T
states and T pool buffers on one GPU, one call per rank -- which is exactly what a rank does with peer mappings of
the other GPUs' pools.  Expected pools are the oracle's: oracle.pack of every rank, placed by oracle.tp_place."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import binding, synth
from helpers import bits, make_plans

pytestmark = pytest.mark.gpu


def _ranks(kind, T, L, H, d, keeps, seed, n_req):
    gen = synth.generator(seed)
    out = []
    for r in range(T):
        uph = d if kind == dasc.KDA else 1
        rates = synth.decay_rates(gen, L, H, uph, 1e-3, 1.0)
        plan, oplan = make_plans(kind, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_LAYER,
                                 keep_ratio=keeps[r % len(keeps)])
        state = synth.states(gen, (n_req, L, H * d * d))
        state.view(-1)[::97] = -0.0
        state.view(torch.int32).view(-1)[5::193] = 0x7FC12345          # NaN payloads travel as bits
        out.append((plan, oplan, state))
    return out


@pytest.mark.parametrize("kind,T,keeps", [
    (dasc.KDA, 2, (0.38, 0.1)), (dasc.KDA, 3, (0.5, 0.0, 0.2)), (dasc.KDA, 8, (0.9, 0.05, 0.38, 0.0, 0.6, 0.2, 0.45, 0.3)),
    (dasc.GDN, 2, (0.5, 0.25)), (dasc.GDN, 3, (0.75, 0.0, 0.25)),
])
def test_pack_tp_and_restore_tp_match_the_oracle_bit_for_bit(kind, T, keeps):
    dev = "cuda"
    L, H, d, n_req, n_slots = 3, 4, 32 if kind == dasc.KDA else 16, 3, 5
    ranks = _ranks(kind, T, L, H, d, keeps, 70 + T, n_req)
    U = np.array([int(p.units_retained) for p, _, _ in ranks], np.int64)
    assert (U == 0).any() == (0.0 in keeps)                              # the empty rank is really empty
    unit = int(ranks[0][0].unit_floats)
    width, send = dasc.dasc_tp_balance(U)
    assert width == -(-int(U.sum()) // T)
    dense = H * d * d
    slot_stride = width * unit + 8                                       # padded slots: the stride is honoured
    guard = 123.25
    pools = [torch.full((n_slots, slot_stride), guard, device=dev) for _ in range(T)]
    src = torch.tensor([2, 0, 1], dtype=torch.int32, device=dev)
    dst = torch.tensor([4, 1, 3], dtype=torch.int32, device=dev)
    d_states = [st.to(dev) for _, _, st in ranks]
    for r, (plan, _, _) in enumerate(ranks):
        dasc.dasc_pack_tp(plan, d_states[r], dense, L * dense, src, pools, U, r, dst, slot_stride=slot_stride)
    torch.cuda.synchronize()

    # oracle: every rank packs its slot, then its units are placed one by one
    want = [np.full((n_slots, slot_stride), guard, np.float32) for _ in range(T)]
    for r, (plan, oplan, st) in enumerate(ranks):
        packed = np.zeros((n_slots, max(1, int(U[r])) * unit), np.float32)
        oracle.pack(oplan.mask, unit, st.numpy(), dense, L * dense, src.cpu().numpy(), packed, packed.shape[1], dst.cpu().numpy())
        for slot in dst.cpu().numpy():
            oracle.tp_place(packed[slot], U, r, unit, [w[slot] for w in want])
    for r in range(T):
        np.testing.assert_array_equal(bits(pools[r]), want[r].view(np.uint32), err_msg=f"pool of rank {r}")
        # what rank r received from each rank is what the split sizes say
    assert send.sum() == U.sum() and (send.sum(0) <= width).all()

    # Load: the inverse gather + zero-fill gives every rank its masked state back
    for r, (plan, oplan, st) in enumerate(ranks):
        out = torch.full((n_req, L, dense), float("nan"), device=dev)
        dasc.dasc_restore_tp(plan, pools, U, r, dst, out, dense, L * dense, src, slot_stride=slot_stride)
        torch.cuda.synchronize()
        n_l = oplan.mask.shape[1]
        keep = np.repeat(oplan.mask.astype(bool), dense // n_l, axis=1)          # [L, dense]
        want_state = np.where(keep[None], st.numpy().view(np.uint32), np.uint32(0))
        np.testing.assert_array_equal(bits(out), want_state)


def test_tp_argument_errors_are_caught_before_any_launch():
    dev = "cuda"
    (plan, _, st), = _ranks(dasc.KDA, 1, 1, 2, 32, (0.5,), 9, 1)
    U = np.array([int(plan.units_retained), 7], np.int64)
    pools = [torch.zeros(64 * 32, device=dev) for _ in range(2)]
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(dasc.DascError) as e:                               # U[rank] is not this plan's payload
        dasc.dasc_pack_tp(plan, st.to(dev), 2 * 32 * 32, 2 * 32 * 32, ids, pools, U, 1, ids)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(dasc.DascError) as e:                               # slot stride below C units
        dasc.dasc_pack_tp(plan, st.to(dev), 2 * 32 * 32, 2 * 32 * 32, ids, pools, U, 0, ids, slot_stride=32)
    assert e.value.status == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert all(float(p.abs().max()) == 0.0 for p in pools)


def test_conv_state_blobs_travel_with_the_checkpoint():
    # Section 4.1: the bf16 convolution state is stored uncompressed beside the temporal state
    dev = "cuda"
    conv_bytes, n_req, n_slots = 3 * 9216 // 16 * 16, 5, 7
    g = torch.Generator().manual_seed(5)
    conv = torch.randint(0, 256, (n_req, conv_bytes + 32), dtype=torch.uint8, generator=g)
    pool = torch.full((n_slots, conv_bytes + 64), 0xAB, dtype=torch.uint8)
    src, dst = np.array([4, 0, 2], np.int32), np.array([1, 6, 3], np.int32)
    d_conv, d_pool = conv.to(dev), pool.to(dev)
    dasc.dasc_conv_store(d_conv, conv.shape[1], torch.from_numpy(src).to(dev), d_pool, pool.shape[1],
                         torch.from_numpy(dst).to(dev), conv_bytes)
    want = pool.numpy().copy()
    oracle.copy_blobs(conv.numpy(), conv.shape[1], src, want, pool.shape[1], dst, conv_bytes)
    np.testing.assert_array_equal(d_pool.cpu().numpy(), want)
    back = torch.full_like(d_conv, 0x11)
    dasc.dasc_conv_load(d_pool, pool.shape[1], torch.from_numpy(dst).to(dev), back, conv.shape[1],
                        torch.from_numpy(src).to(dev), conv_bytes)
    want_back = np.full_like(conv.numpy(), 0x11)
    oracle.copy_blobs(want, pool.shape[1], dst, want_back, conv.shape[1], src, conv_bytes)
    np.testing.assert_array_equal(back.cpu().numpy(), want_back)
    np.testing.assert_array_equal(want_back[src][:, :conv_bytes], conv.numpy()[src][:, :conv_bytes])
