"""Seeded random sweep of the refresh call as a user makes it (DASC_ALGO_AUTO: the tensor-core kernel, with the exact
kernel taking requests of a handful of tokens): kinds, head groupings, ragged lengths (empty requests included),
both modes, with and without outputs, layer sub-ranges, a permuted request-to-state map and state strides with
padding between requests and layers.  Every (request, layer, head) unit of every case is replayed by the fp64 oracle
on the bits the GPU saw; guard values around each state show that nothing outside a unit is written."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_30386_b200 as dasc
from paper_2608_30386_b200 import synth
from helpers import make_plans, rel_err
from helpers_fullsize import oracle_one_unit

pytestmark = pytest.mark.gpu

TOL = 1e-3
GUARD = -123.0


@pytest.mark.parametrize("seed", range(16))
def test_random_chunked_refresh_calls(seed):
    rng = np.random.default_rng(1000 + seed)
    dev = "cuda"
    d = 128
    kind = dasc.KDA if rng.random() < 0.6 else dasc.GDN
    H_v = int(rng.choice([2, 4, 8]))
    H_k = H_v if kind == dasc.KDA else int(rng.choice([h for h in (1, 2, 4, 8) if H_v % h == 0]))
    L = int(rng.integers(1, 4))
    n_req = int(rng.integers(1, 6))
    lens = [int(x) for x in rng.choice([0, 1, 5, 31, 32, 33, 64, 70, 97, 130], size=n_req)]
    mode = dasc.REFRESH_CONTINUE if rng.random() < 0.5 else dasc.REFRESH_SCRATCH_MERGE_LOCAL
    with_o = bool(rng.random() < 0.7)
    o_dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    q_scale = float(rng.choice([1.0, 0.5, d ** -0.5]))
    layer_begin = int(rng.integers(0, L))
    layer_end = int(rng.integers(layer_begin + 1, L + 1))
    Lc = layer_end - layer_begin
    n_slots = n_req + 2
    req_idx = rng.permutation(n_slots)[:n_req].astype(np.int32)          # request i lives in state slot req_idx[i]
    dense = H_v * d * d
    layer_stride = dense + 4 * int(rng.integers(0, 3)) * 64               # padding between layers (16-byte multiples)
    req_stride = L * layer_stride + 4 * int(rng.integers(0, 3)) * 32      # and between requests

    gen = synth.generator(seed)
    rates = synth.decay_rates(gen, L, H_v, d if kind == dasc.KDA else 1, 1e-3, 1.0)
    plan, oplan = make_plans(kind, L, H_v, H_k, d, d, rates, sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_LAYER,
                             keep_ratio=float(rng.choice([0.2, 0.38, 0.5, 1.0])))
    cu = torch.zeros(n_req + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(torch.tensor(lens, dtype=torch.int64), 0).to(torch.int32)
    T = int(cu[-1])
    s = synth.token_streams(gen, kind, L, max(T, 1), H_v, H_k, d, d, rates, io_dtype=torch.bfloat16)
    q, k, v, g, beta = (getattr(s, f)[layer_begin:layer_end, :T].contiguous().to(dev) for f in ("q", "k", "v", "g", "beta"))
    state = torch.full((n_slots * req_stride,), GUARD, dtype=torch.float32, device=dev)
    init = synth.states(gen, (n_slots, L, dense))
    sv = state.view(n_slots, req_stride)
    for l in range(L):
        sv[:, l * layer_stride: l * layer_stride + dense] = init[:, l].to(dev)
    before = state.clone()
    o = torch.full((Lc, max(T, 1), H_v, d), float("nan"), dtype=o_dtype, device=dev) if with_o else None
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, n_req, Lc, dasc.ALGO_AUTO), dtype=torch.uint8, device=dev)
    dasc.dasc_refresh(plan, state, layer_stride, req_stride, torch.from_numpy(req_idx).to(dev), q, k, v, g, beta,
                      cu.to(dev), T, max(lens), layer_begin=layer_begin, layer_end=layer_end, q_scale=q_scale, o=o,
                      mode=mode, algo=dasc.ALGO_AUTO, workspace=ws)
    torch.cuda.synchronize()
    assert dasc.dasc_refresh_status(ws) == 0

    after = state.cpu().numpy().reshape(n_slots, req_stride)
    b4 = before.cpu().numpy().reshape(n_slots, req_stride)
    touched = np.zeros_like(after, dtype=bool)
    o_np = o.float().cpu().numpy() if with_o else None
    omode = oracle.MODE_CONTINUE if mode == dasc.REFRESH_CONTINUE else oracle.MODE_SCRATCH_MERGE_LOCAL
    out_tol = TOL + (2.0 ** -8 if o_dtype == torch.bfloat16 else 0.0)
    worst, worst_strict = 0.0, 0.0
    for r in range(n_req):
        t0, t1 = int(cu[r]), int(cu[r + 1])
        for l in range(Lc):
            for h in range(H_v):
                off = (layer_begin + l) * layer_stride + h * d * d
                s0 = b4[req_idx[r], off: off + d * d].reshape(d, d)
                s1 = after[req_idx[r], off: off + d * d].reshape(d, d)
                touched[req_idx[r], off: off + d * d] = True
                if t1 == t0 and mode == dasc.REFRESH_CONTINUE:
                    np.testing.assert_array_equal(s1, s0)                 # an empty suffix leaves the state as it was
                    continue
                if kind == dasc.KDA:
                    keep = oplan.mask[layer_begin + l].reshape(H_v, d)[h]
                else:
                    keep = np.full(d, oplan.mask[layer_begin + l][h], np.uint8)
                ref_s, ref_o = oracle_one_unit(kind, H_v, H_k, s0, q, k, v, g, beta, cu, r, l, h, mode=omode,
                                               keep_rows=keep, q_scale=q_scale)
                e = rel_err(s1, ref_s)
                worst = max(worst, e)
                assert e <= TOL, (seed, r, l, h, e)
                if mode == dasc.REFRESH_SCRATCH_MERGE_LOCAL:
                    kept = keep.astype(bool)
                    np.testing.assert_array_equal(s1[kept], s0[kept])     # retained rows keep their stored bits
                if with_o and t1 > t0:
                    ref = ref_o
                    got = o_np[l, t0:t1, h]
                    # the stated metric, unchanged: max abs error over max |reference| of the unit's output block
                    # (a bf16 output adds its own final rounding of up to 2^-8 of each value)
                    strict = float(np.abs(got - ref).max() / np.abs(ref).max())
                    worst_strict = max(worst_strict, strict if o_dtype == torch.float32 else 0.0)
                    bound = TOL * np.abs(ref).max() + (np.abs(ref) * 2.0 ** -8 if o_dtype == torch.bfloat16 else 0.0)
                    bad = np.abs(got - ref) > bound
                    assert not bad.any(), (seed, r, l, h, lens, strict, np.argwhere(bad)[:4].tolist())
    # nothing outside the addressed units changed: padding, other layers, unused slots
    np.testing.assert_array_equal(after[~touched], b4[~touched])
    print(f"seed {seed}: kind {kind} H_v {H_v} H_k {H_k} L {L} layers [{layer_begin},{layer_end}) lens {lens} mode {mode} "
          f"o {with_o} worst state err {worst:.2e}, worst fp32 output err relative to its own max {worst_strict:.2e}")
