"""GPU parity: dasc_pack_int8 / dasc_restore_int8 (Appendix D, Eq. 10 fused into the copies) through the
C ABI against the oracle, bit for bit: codes, scales and the dequantised, zero-filled states.
The oracle side composes its own pack / quantise / dequantise / restore."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth
from helpers import bits, make_plans

pytestmark = pytest.mark.gpu


def _finite_specials_(state: torch.Tensor, gen: torch.Generator, d_v: int):
    """Finite edge values: all-zero rows (scale floor), -0.0, denormals, huge and tiny magnitudes, exact ties."""
    rows = state.view(-1)[: state.numel() // d_v * d_v].view(-1, d_v)
    n = rows.shape[0]
    pick = torch.randperm(n, generator=gen)[: max(8, n // 50)]
    for j, r in enumerate(pick.tolist()):
        kind = j % 8
        if kind == 0:
            rows[r] = 0.0
        elif kind == 1:
            rows[r] = -0.0
        elif kind == 2:
            rows[r] = torch.full((d_v,), 1e-42)                  # denormals: below the 1e-8 floor
        elif kind == 3:
            rows[r] *= 1e30
        elif kind == 4:
            rows[r] *= 1e-30
        elif kind == 5:                                          # exact halves: ties go to even
            rows[r] = (torch.arange(d_v, dtype=torch.float32) % 127) + 0.5
            rows[r, 0] = 127.0
        elif kind == 6:
            rows[r] = 0.0
            rows[r, d_v - 1] = -3.5                              # single non-zero value maps to -127
        else:
            rows[r, ::2] = -rows[r, ::2].abs().max()             # many elements at the abs-max


def _oracle_int8(oplan, uw, d_v, state_np, layer_stride, req_stride, src_req, dst_req, fill):
    """Expected codes [pairs][rows][d_v], scales [pairs][rows] and restored states, from oracle calls only."""
    n_pairs = len(src_req)
    slot = int(oplan.mask.sum()) * uw
    ids = np.arange(n_pairs, dtype=np.int32)
    pool = np.zeros((n_pairs, max(slot, 1)), np.float32)
    oracle.pack(oplan.mask, uw, state_np, layer_stride, req_stride, src_req, pool, max(slot, 1), ids)
    rows = pool[:, :slot].reshape(-1, d_v)
    q, s = oracle.int8_quantize(rows) if rows.size else (np.zeros((0, d_v), np.int8), np.zeros(0, np.float32))
    deq = oracle.int8_dequantize(q, s) if rows.size else rows
    pool2 = np.zeros_like(pool)
    pool2[:, :slot] = deq.reshape(n_pairs, slot)
    out = np.full(state_np.shape, np.float32(fill))
    oracle.restore(oplan.mask, uw, pool2, max(slot, 1), ids, out, layer_stride, req_stride, dst_req)
    return q.reshape(n_pairs, slot // d_v, d_v), s.reshape(n_pairs, slot // d_v), out


def _case(seed, kind, L, H, d_k, d_v, n_req, n_slots, *, sel, scope=dasc.SCOPE_LAYER, keep_ratio=1.0, w_max=0.0,
          layer_pad=0, req_pad=0, slot_pad=0):
    dev = "cuda"
    gen = synth.generator(seed)
    uph = d_k if kind == dasc.KDA else 1
    rates = synth.decay_rates(gen, L, H, uph, 1e-3, 1.0)
    plan, oplan = make_plans(kind, L, H, H, d_k, d_v, rates, sel=sel, scope=scope, keep_ratio=keep_ratio, w_max=w_max)
    dense = H * d_k * d_v
    layer_stride = dense + layer_pad
    req_stride = L * layer_stride + req_pad
    state = synth.states(gen, (n_req * req_stride,))
    _finite_specials_(state, gen, d_v)
    n_pairs = min(n_req, n_slots)
    src_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)
    dst_slot = torch.randperm(n_slots, generator=gen)[:n_pairs].to(torch.int32)
    dst_req = torch.randperm(n_req, generator=gen)[:n_pairs].to(torch.int32)

    slot_bytes = dasc.dasc_int8_slot_bytes(plan)
    packed_rows = int(plan.slot_floats) // d_v
    assert slot_bytes == (packed_rows * (d_v + 4) + 15) // 16 * 16
    stride = slot_bytes + slot_pad
    d_state = state.to(dev)
    d_pool = torch.full((n_slots * stride + 16,), 0x5A, dtype=torch.uint8, device=dev)
    dasc.dasc_pack_int8(plan, d_state, layer_stride, req_stride, src_req.to(dev), d_pool, dst_slot.to(dev),
                        slot_stride_bytes=stride)
    d_out = torch.full_like(d_state, -3.0)
    dasc.dasc_restore_int8(plan, d_pool, dst_slot.to(dev), d_out, layer_stride, req_stride, dst_req.to(dev),
                           slot_stride_bytes=stride)
    torch.cuda.synchronize()

    q, s, out = _oracle_int8(oplan, int(plan.unit_floats), d_v, state.numpy(), layer_stride, req_stride,
                             src_req.numpy(), dst_req.numpy(), -3.0)
    pool = d_pool.cpu().numpy()
    used = np.zeros(pool.size, bool)
    for i, slot in enumerate(dst_slot.tolist()):
        b = slot * stride
        codes = pool[b: b + packed_rows * d_v].view(np.int8).reshape(packed_rows, d_v)
        scales = pool[b + packed_rows * d_v: b + packed_rows * (d_v + 4)].view(np.float32)
        np.testing.assert_array_equal(codes, q[i])
        np.testing.assert_array_equal(scales.view(np.uint32), s[i].view(np.uint32))
        used[b: b + packed_rows * (d_v + 4)] = True
    assert np.all(pool[~used] == 0x5A)                          # nothing outside codes and scales is written
    np.testing.assert_array_equal(bits(d_out), out.view(np.uint32))
    return plan


def test_tiny_kda_config():
    plan = _case(0, dasc.KDA, 1, 4, 64, 64, n_req=4, n_slots=4, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_HEAD,
                 keep_ratio=0.4)
    assert plan.units_retained == 4 * 26


@pytest.mark.parametrize("ratio", [0.0, 0.25, 0.38, 1.0])
def test_kda_ragged_layer_scope(ratio):
    # several CTAs per (pair, layer), a ragged tail, padded strides
    _case(1, dasc.KDA, 5, 6, 128, 128, n_req=7, n_slots=9, sel=dasc.SEL_TOP_RATIO, keep_ratio=ratio, layer_pad=64,
          req_pad=32, slot_pad=32)


def test_narrow_rows_and_threshold_rule():
    _case(2, dasc.KDA, 3, 5, 48, 32, n_req=5, n_slots=5, sel=dasc.SEL_THRESHOLD, w_max=64.0)
    _case(3, dasc.KDA, 2, 3, 20, 8, n_req=3, n_slots=4, sel=dasc.SEL_THRESHOLD, w_max=128.0, layer_pad=4)
    _case(4, dasc.KDA, 2, 3, 10, 4, n_req=3, n_slots=3, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)


def test_gdn_head_units():
    _case(5, dasc.GDN, 6, 8, 128, 128, n_req=5, n_slots=6, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    _case(6, dasc.GDN, 2, 4, 64, 32, n_req=3, n_slots=3, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.3, slot_pad=16)


def test_capacity():
    # Appendix D: d_v + 4 = 132 bytes per retained row instead of 512 (3.88x)
    plan = _case(7, dasc.KDA, 2, 4, 128, 128, n_req=2, n_slots=2, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    rows = int(plan.slot_floats) // 128
    assert dasc.dasc_int8_slot_bytes(plan) == rows * 132 and rows * 512 / (rows * 132) == pytest.approx(3.88, abs=5e-3)


def test_argument_errors_launch_nothing():
    gen = synth.generator(8)
    rates = synth.decay_rates(gen, 1, 2, 8, 1e-3, 1.0)
    plan96, _ = make_plans(dasc.KDA, 1, 2, 2, 8, 96, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    plan, _ = make_plans(dasc.KDA, 1, 2, 2, 8, 64, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.5)
    dev = "cuda"
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    state = torch.zeros(2 * 8 * 96, device=dev)
    pool = torch.full((4096,), 0x11, dtype=torch.uint8, device=dev)
    with pytest.raises(dasc.DascError) as e:                     # d_v = 96 is not a power of two
        dasc.dasc_pack_int8(plan96, state, 2 * 8 * 96, 2 * 8 * 96, ids, pool, ids)
    assert e.value.status == 2
    need = dasc.dasc_int8_slot_bytes(plan)
    with pytest.raises(dasc.DascError) as e:                     # stride smaller than a slot
        dasc.dasc_pack_int8(plan, state, 2 * 8 * 64, 2 * 8 * 64, ids, pool, ids, slot_stride_bytes=need - 16)
    assert e.value.status == 1
    with pytest.raises(dasc.DascError) as e:                     # stride not a multiple of 16
        dasc.dasc_restore_int8(plan, pool, ids, state, 2 * 8 * 64, 2 * 8 * 64, ids, slot_stride_bytes=need + 4)
    assert e.value.status == 1
    with pytest.raises(dasc.DascError) as e:                     # misaligned pool
        dasc.dasc_pack_int8(plan, state, 2 * 8 * 64, 2 * 8 * 64, ids, pool[4:], ids)
    assert e.value.status == 1
    torch.cuda.synchronize()
    assert bool((pool == 0x11).all())


def test_kda_serving_size_sampled_requests():
    """The benchmark's launch shape (24 x 32 x 128 x 128, 64 requests, keep 0.38 per layer); four requests are
    copied back and checked whole against the oracle."""
    dev = "cuda"
    L, H, d, n_req = 24, 32, 128, 64
    gen = synth.generator(1)
    rates = synth.decay_rates(gen, L, H, d, 1e-3, 1.0)
    plan, oplan = make_plans(dasc.KDA, L, H, H, d, d, rates, sel=dasc.SEL_TOP_RATIO, keep_ratio=0.38)
    dense = H * d * d
    layer_stride, req_stride = n_req * dense, dense               # layer-major, as the benchmark lays it out
    dgen = synth.generator(1, dev)
    state = synth.states(dgen, (L * n_req * dense,), dev)
    stride = dasc.dasc_int8_slot_bytes(plan)
    pool = torch.empty((n_req * stride,), dtype=torch.uint8, device=dev)
    ids = torch.arange(n_req, dtype=torch.int32, device=dev)
    slots = torch.flip(ids, [0]).contiguous()
    dasc.dasc_pack_int8(plan, state, layer_stride, req_stride, ids, pool, slots)
    out = torch.full_like(state, -3.0)
    dasc.dasc_restore_int8(plan, pool, slots, out, layer_stride, req_stride, ids)
    torch.cuda.synchronize()
    packed_rows = int(plan.slot_floats) // d
    for r in (0, 17, 40, 63):
        host = state.view(L, n_req, dense)[:, r].contiguous().cpu().numpy().reshape(-1)       # [L][dense]
        q, s, want = _oracle_int8(oplan, d, d, host, dense, 0, np.zeros(1, np.int32), np.zeros(1, np.int32), -3.0)
        b = int(slots[r]) * stride
        got = pool[b: b + stride].cpu().numpy()
        np.testing.assert_array_equal(got[: packed_rows * d].view(np.int8).reshape(packed_rows, d), q[0])
        np.testing.assert_array_equal(got[packed_rows * d: packed_rows * (d + 4)].view(np.uint32), s[0].view(np.uint32))
        np.testing.assert_array_equal(bits(out.view(L, n_req, dense)[:, r].contiguous()).reshape(-1),
                                      want.view(np.uint32))
