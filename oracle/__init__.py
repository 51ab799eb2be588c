"""DASC oracle -- TEST INFRASTRUCTURE ONLY.

ctypes front end of ``dasc_oracle.c``: a plain fp64 CPU statement of the DASC
hot path (plan, pack, restore with zero-fill, token-by-token suffix refresh),
written from the paper.  Nothing in the product package imports this module;
only the tests, the smoke check and the benchmark's CPU-baseline leg do.

Arrays are numpy; bf16 streams travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dasc_oracle.c")
_LIB = os.path.join(_HERE, "libdasc_oracle.so")

KDA, GDN = 0, 1
SEL_THRESHOLD, SEL_TOP_RATIO, SEL_EXPLICIT = 0, 1, 2
SCOPE_HEAD, SCOPE_LAYER, SCOPE_MODEL = 0, 1, 2
MODE_CONTINUE, MODE_SCRATCH_MERGE_LOCAL = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, OpenMP over independent units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_replay_window_unit.restype = C.c_double
        _lib.oracle_replay_window_unit.argtypes = [C.c_double, C.c_double]
        _lib.oracle_slot_budget.restype = C.c_int64
        _lib.oracle_max_threads.restype = C.c_int32
        _lib.oracle_splitmix64.restype = C.c_uint64
        _lib.oracle_splitmix64.argtypes = [C.c_uint64]
    return _lib


def _p(a, ty=C.c_void_p):
    return None if a is None else a.ctypes.data_as(ty)


def horizon(A_log, dt_bias, a=-0.3, eps=1e-3):
    """Eq. 2 / Eq. 3: (g, H_s) per unit, fp64."""
    A_log = np.ascontiguousarray(A_log, np.float32).ravel()
    dt_bias = np.ascontiguousarray(dt_bias, np.float32).ravel()
    g = np.empty(A_log.size, np.float64)
    Hs = np.empty(A_log.size, np.float64)
    lib().oracle_horizon(C.c_int64(A_log.size), _p(A_log), _p(dt_bias), C.c_double(a),
                         C.c_double(eps), _p(g), _p(Hs))
    return g, Hs


def splitmix64(x: int) -> int:
    """The key function of the count-matched random selector (Appendix C.3 control)."""
    return int(lib().oracle_splitmix64(C.c_uint64(x & 0xFFFFFFFFFFFFFFFF)))


def replay_window_unit(Hs: float, w_max: float) -> float:
    """Eq. 7, one unit: clamp(next_pow2(H_s), 4, w_max)."""
    return lib().oracle_replay_window_unit(Hs, w_max)


@dataclass
class Plan:
    kind: int
    n_layers: int
    n_heads: int
    units_per_head: int
    Hs: np.ndarray        # [L, n_l] fp64
    mask: np.ndarray      # [L, n_l] uint8, 1 = retained
    r_l: np.ndarray       # [L] int64
    o_l: np.ndarray       # [L+1] int64
    W_u: np.ndarray       # [L, n_l] fp64
    sum_n: int
    sum_r: int
    R_max: int
    C_temp_rag: float
    C_temp_pad: float
    C_ckpt_rag: float
    W_replay: float
    w_max_used: float

    @property
    def n_l(self) -> int:
        return self.n_heads * self.units_per_head


def plan(kind, n_layers, n_heads, units_per_head, A_log, dt_bias, *, a=-0.3, eps=1e-3,
         sel=SEL_THRESHOLD, w_max=0.0, keep_ratio=1.0, scope=SCOPE_LAYER, randomize=False,
         seed=0, explicit_mask=None, unit_bytes=0, conv_bytes=0) -> Plan:
    """Selection plan of Section 4.1 with Eq. 6 / Eq. 7 / Appendix B outputs."""
    n_l = n_heads * units_per_head
    n_all = n_l * n_layers
    A_log = np.ascontiguousarray(A_log, np.float32).ravel()
    dt_bias = np.ascontiguousarray(dt_bias, np.float32).ravel()
    assert A_log.size == n_all and dt_bias.size == n_all
    em = None
    if explicit_mask is not None:
        em = np.ascontiguousarray(explicit_mask, np.uint8).ravel()
        assert em.size == n_all
    Hs = np.empty(n_all, np.float64)
    mask = np.empty(n_all, np.uint8)
    r_l = np.zeros(n_layers, np.int64)
    o_l = np.zeros(n_layers + 1, np.int64)
    W_u = np.empty(n_all, np.float64)
    stats = np.zeros(8, np.float64)
    rc = lib().oracle_plan(C.c_int(kind), C.c_int32(n_layers), C.c_int32(n_heads),
                           C.c_int32(units_per_head), _p(A_log), _p(dt_bias), C.c_double(a),
                           C.c_double(eps), C.c_int(sel), C.c_double(w_max), C.c_double(keep_ratio),
                           C.c_int(scope), C.c_int(1 if randomize else 0), C.c_uint64(seed), _p(em),
                           C.c_int64(unit_bytes), C.c_int64(conv_bytes), _p(Hs), _p(mask), _p(r_l),
                           _p(o_l), _p(W_u), _p(stats))
    if rc != 0:
        raise RuntimeError(f"oracle_plan failed: {rc}")
    return Plan(kind, n_layers, n_heads, units_per_head, Hs.reshape(n_layers, n_l),
                mask.reshape(n_layers, n_l), r_l, o_l, W_u.reshape(n_layers, n_l),
                int(stats[0]), int(stats[1]), int(stats[2]), float(stats[3]), float(stats[4]),
                float(stats[5]), float(stats[6]), float(stats[7]))


def slot_budget(budget_bytes, temporal_bytes_per_rank, conv_bytes) -> int:
    """Appendix C.1: N = floor(B / max_r[b_r + b_conv]) - 1."""
    t = np.ascontiguousarray(temporal_bytes_per_rank, np.int64)
    return int(lib().oracle_slot_budget(C.c_int64(budget_bytes), _p(t), C.c_int32(t.size),
                                        C.c_int64(conv_bytes)))


def tp_balance(units_per_rank):
    """Section 4.3: (C, send[T][T]) for the store-time redistribution of packed units over the TP group."""
    U = np.ascontiguousarray(units_per_rank, np.int64)
    send = np.zeros((U.size, U.size), np.int64)
    lib().oracle_tp_balance.restype = C.c_int64
    c = lib().oracle_tp_balance(_p(U), C.c_int32(U.size), _p(send))
    return int(c), send


def tp_place(packed, units_per_rank, rank, unit_words, pools):
    """Section 4.3: put rank ``rank``'s packed slot (``U[rank]`` units) where the balanced placement wants it;
    ``pools[s]`` is rank s's slot (numpy, 4-byte dtype, at least C units), written in place."""
    U = np.ascontiguousarray(units_per_rank, np.int64)
    ptrs = (C.c_void_p * U.size)(*[_words(p).ctypes.data for p in pools])
    lib().oracle_tp_place(_p(_words(np.ascontiguousarray(packed))), _p(U), C.c_int32(U.size), C.c_int32(rank),
                          C.c_int64(unit_words), ptrs)


def tp_head_permutation(weight, n_ranks):
    """Section 4.3, first stage: (perm[L][n_bundles], load[T]) for per-layer bundle weights ``weight[L][n_bundles]``."""
    w = np.ascontiguousarray(weight, np.int64)
    L, B = w.shape
    assert B % n_ranks == 0
    perm = np.full((L, B), -1, np.int32)
    load = np.zeros(n_ranks, np.int64)
    lib().oracle_tp_head_permutation(_p(w), C.c_int32(L), C.c_int32(B), C.c_int32(n_ranks), _p(perm), _p(load))
    return perm, load


def copy_blobs(src, src_stride, src_idx, dst, dst_stride, dst_idx, blob_bytes):
    """dst[dst_idx[i]] = src[src_idx[i]] for opaque blobs (uint8 arrays, strides in bytes), in place on ``dst``."""
    src_idx = np.ascontiguousarray(src_idx, np.int32)
    dst_idx = np.ascontiguousarray(dst_idx, np.int32)
    assert src.dtype == np.uint8 and dst.dtype == np.uint8
    lib().oracle_copy_blobs(_p(src), C.c_int64(src_stride), _p(src_idx), _p(dst), C.c_int64(dst_stride), _p(dst_idx),
                            C.c_int64(blob_bytes), C.c_int32(src_idx.size))


def _words(a):
    assert a.dtype.itemsize == 4 and a.flags.c_contiguous
    return a.view(np.uint32)


def pack(mask, unit_words, state, layer_stride, req_stride, src_req, pool, slot_stride, dst_slot):
    """Gather retained units into the ragged pool (in place on ``pool``)."""
    mask = np.ascontiguousarray(mask, np.uint8)
    L, n_l = mask.shape
    src_req = np.ascontiguousarray(src_req, np.int32)
    dst_slot = np.ascontiguousarray(dst_slot, np.int32)
    lib().oracle_pack(_p(mask), C.c_int32(L), C.c_int64(n_l), C.c_int64(unit_words),
                      _p(_words(state)), C.c_int64(layer_stride), C.c_int64(req_stride), _p(src_req),
                      _p(_words(pool)), C.c_int64(slot_stride), _p(dst_slot), C.c_int32(src_req.size))


def restore(mask, unit_words, pool, slot_stride, src_slot, state, layer_stride, req_stride, dst_req):
    """Scatter retained units back, omitted units become +0.0 (in place on ``state``)."""
    mask = np.ascontiguousarray(mask, np.uint8)
    L, n_l = mask.shape
    src_slot = np.ascontiguousarray(src_slot, np.int32)
    dst_req = np.ascontiguousarray(dst_req, np.int32)
    lib().oracle_restore(_p(mask), C.c_int32(L), C.c_int64(n_l), C.c_int64(unit_words),
                         _p(_words(pool)), C.c_int64(slot_stride), _p(src_slot), _p(_words(state)),
                         C.c_int64(layer_stride), C.c_int64(req_stride), _p(dst_req),
                         C.c_int32(src_slot.size))


def pack_padded(mask, unit_words, state, layer_stride, req_stride, src_req, pool, n_slots, R_max, dst_slot):
    """Appendix B padded layout: ``pool`` is [L][n_slots][R_max][unit_words]; padding is not written."""
    mask = np.ascontiguousarray(mask, np.uint8)
    L, n_l = mask.shape
    src_req = np.ascontiguousarray(src_req, np.int32)
    dst_slot = np.ascontiguousarray(dst_slot, np.int32)
    assert pool.size >= L * n_slots * R_max * unit_words
    lib().oracle_pack_padded(_p(mask), C.c_int32(L), C.c_int64(n_l), C.c_int64(unit_words), _p(_words(state)),
                             C.c_int64(layer_stride), C.c_int64(req_stride), _p(src_req), _p(_words(pool)),
                             C.c_int64(n_slots), C.c_int64(R_max), _p(dst_slot), C.c_int32(src_req.size))


def restore_padded(mask, unit_words, pool, n_slots, R_max, src_slot, state, layer_stride, req_stride, dst_req):
    """Zero-fill load from the padded pool (in place on ``state``)."""
    mask = np.ascontiguousarray(mask, np.uint8)
    L, n_l = mask.shape
    src_slot = np.ascontiguousarray(src_slot, np.int32)
    dst_req = np.ascontiguousarray(dst_req, np.int32)
    lib().oracle_restore_padded(_p(mask), C.c_int32(L), C.c_int64(n_l), C.c_int64(unit_words), _p(_words(pool)),
                                C.c_int64(n_slots), C.c_int64(R_max), _p(src_slot), _p(_words(state)),
                                C.c_int64(layer_stride), C.c_int64(req_stride), _p(dst_req),
                                C.c_int32(src_slot.size))


def refresh(kind, n_layers, H_v, H_k, d_k, d_v, state, layer_stride, req_stride, req_idx,
            q, k, v, g, beta, cu_seqlens, *, q_scale=1.0, want_o=True, mode=MODE_CONTINUE,
            mask=None, want_state64=False, n_threads=0):
    """Token-by-token replay of Eq. 1 over each request's suffix.

    ``state`` (fp32 numpy) is updated in place.  ``q/k/v`` are uint16 (bf16 bits)
    or float32, shaped as documented in ``dasc_oracle.c``.  Returns
    ``(o, state64)``: fp64 outputs ``[L][T][H_v][d_v]`` (or None) and the fp64
    final states ``[n_req][L][H_v][d_k][d_v]`` (or None).
    """
    io_bf16 = q.dtype == np.uint16
    assert k.dtype == q.dtype and v.dtype == q.dtype and (io_bf16 or q.dtype == np.float32)
    for a in (q, k, v, g, beta, state):
        assert a.flags.c_contiguous
    assert g.dtype == np.float32 and beta.dtype == np.float32 and state.dtype == np.float32
    cu = np.ascontiguousarray(cu_seqlens, np.int32)
    n_req = cu.size - 1
    T = int(cu[-1])
    req_idx = np.ascontiguousarray(req_idx, np.int32)
    assert req_idx.size == n_req
    assert q.size == n_layers * T * H_k * d_k and v.size == n_layers * T * H_v * d_v
    assert g.size == n_layers * T * H_v * (d_k if kind == KDA else 1)
    assert beta.size == n_layers * T * H_v
    o = np.zeros((n_layers, T, H_v, d_v), np.float64) if want_o else None
    s64 = np.zeros((n_req, n_layers, H_v, d_k, d_v), np.float64) if want_state64 else None
    m = None
    if mode == MODE_SCRATCH_MERGE_LOCAL:
        assert mask is not None
        m = np.ascontiguousarray(mask, np.uint8)
    rc = lib().oracle_refresh(C.c_int(kind), C.c_int32(n_layers), C.c_int32(H_v), C.c_int32(H_k),
                              C.c_int32(d_k), C.c_int32(d_v), _p(state), C.c_int64(layer_stride),
                              C.c_int64(req_stride), _p(req_idx), _p(q), _p(k), _p(v),
                              C.c_int(1 if io_bf16 else 0), _p(g), _p(beta), _p(cu), C.c_int32(n_req),
                              C.c_double(q_scale), _p(o), C.c_int(mode), _p(m), _p(s64),
                              C.c_int32(n_threads))
    if rc != 0:
        raise RuntimeError(f"oracle_refresh failed: {rc}")
    return o, s64


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def int8_quantize(rows):
    """Appendix D quantiser: returns (q int8 [n, w], scale fp32 [n])."""
    rows = np.ascontiguousarray(rows, np.float32)
    n, w = rows.shape
    q = np.empty((n, w), np.int8)
    s = np.empty(n, np.float32)
    lib().oracle_int8_quantize(_p(rows), C.c_int64(n), C.c_int64(w), _p(q), _p(s))
    return q, s


def int8_dequantize(q, scale):
    q = np.ascontiguousarray(q, np.int8)
    scale = np.ascontiguousarray(scale, np.float32)
    n, w = q.shape
    rows = np.empty((n, w), np.float32)
    lib().oracle_int8_dequantize(_p(q), _p(scale), C.c_int64(n), C.c_int64(w), _p(rows))
    return rows
