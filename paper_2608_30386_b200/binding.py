"""Thin ctypes binding of libdasc: the same four calls as the C ABI
(``dasc_plan``, ``dasc_pack``, ``dasc_restore``, ``dasc_refresh``), taking torch
tensors for device memory.  Argument marshalling only: every step runs in the
library.  There is no fallback: if the shared library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdasc.so")

KDA, GDN = 0, 1
SEL_THRESHOLD, SEL_TOP_RATIO, SEL_EXPLICIT = 0, 1, 2
SCOPE_HEAD, SCOPE_LAYER, SCOPE_MODEL = 0, 1, 2
IO_BF16, IO_FP32 = 0, 1
REFRESH_CONTINUE, REFRESH_SCRATCH_MERGE_LOCAL = 0, 1
ALGO_AUTO, ALGO_SEQUENTIAL, ALGO_CHUNKED = 0, 1, 2

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT, ERR_DOMAIN = range(9)

# Every symbol include/dasc.h declares.
EXPORTS = (
    "dasc_plan", "dasc_plan_destroy", "dasc_plan_info", "dasc_plan_horizon", "dasc_plan_mask",
    "dasc_plan_window", "dasc_plan_layer_counts", "dasc_plan_layer_offsets", "dasc_plan_save_bytes", "dasc_plan_save",
    "dasc_plan_load", "dasc_pack", "dasc_restore",
    "dasc_int8_slot_bytes", "dasc_pack_int8", "dasc_restore_int8",
    "dasc_padded_pool_floats", "dasc_pack_padded", "dasc_restore_padded", "dasc_checkpoint_bytes", "dasc_slot_budget",
    "dasc_tp_balance", "dasc_pack_tp", "dasc_restore_tp", "dasc_tp_head_permutation", "dasc_conv_store", "dasc_conv_load",
    "dasc_refresh_counters", "dasc_debug_set_refresh_poll_limit",
    "dasc_refresh_workspace_bytes", "dasc_refresh", "dasc_refresh_status", "dasc_refresh_window", "dasc_refresh_static",
    "dasc_status_string", "dasc_version",
)


class DascError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class PlanDesc(C.Structure):
    _fields_ = [
        ("kind", C.c_int32), ("n_layers", C.c_int32), ("n_v_heads", C.c_int32), ("n_k_heads", C.c_int32),
        ("d_k", C.c_int32), ("d_v", C.c_int32),
        ("A_log", C.c_void_p), ("dt_bias", C.c_void_p),
        ("a", C.c_double), ("eps", C.c_double),
        ("sel", C.c_int32), ("scope", C.c_int32),
        ("w_max", C.c_double), ("keep_ratio", C.c_double),
        ("randomize", C.c_int32), ("seed", C.c_uint64),
        ("explicit_mask", C.c_void_p),
        ("conv_bytes_per_ckpt", C.c_int64),
    ]


class PlanInfo(C.Structure):
    _fields_ = [
        ("kind", C.c_int32), ("n_layers", C.c_int32), ("n_v_heads", C.c_int32), ("n_k_heads", C.c_int32),
        ("d_k", C.c_int32), ("d_v", C.c_int32),
        ("units_per_layer", C.c_int64), ("unit_floats", C.c_int64), ("units_total", C.c_int64),
        ("units_retained", C.c_int64), ("r_max", C.c_int64), ("slot_floats", C.c_int64),
        ("dense_floats_per_layer", C.c_int64),
        ("c_temp_rag", C.c_double), ("c_temp_pad", C.c_double), ("c_ckpt_rag", C.c_double),
        ("w_max_used", C.c_double), ("w_replay", C.c_int64), ("device", C.c_int32),
    ]


_lib = None


def lib() -> C.CDLL:
    """Load libdasc.so (built in-tree by ``build.py``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2608_30386_b200.build` "
                              "(there is no non-CUDA fallback)")
        L = C.CDLL(LIB_PATH)
        L.dasc_plan.restype = C.c_int
        L.dasc_plan.argtypes = [C.POINTER(PlanDesc), C.c_int32, C.POINTER(C.c_void_p)]
        L.dasc_plan_destroy.restype = None
        L.dasc_plan_destroy.argtypes = [C.c_void_p]
        L.dasc_plan_info.argtypes = [C.c_void_p, C.POINTER(PlanInfo)]
        for name in ("dasc_plan_horizon", "dasc_plan_mask", "dasc_plan_window", "dasc_plan_layer_counts",
                     "dasc_plan_layer_offsets"):
            getattr(L, name).argtypes = [C.c_void_p, C.c_void_p]
        L.dasc_plan_save_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        L.dasc_plan_save.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        L.dasc_plan_load.argtypes = [C.c_void_p, C.c_size_t, C.c_int32, C.POINTER(C.c_void_p)]
        L.dasc_pack.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                C.c_void_p, C.c_int32, C.c_void_p]
        L.dasc_restore.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                   C.c_void_p, C.c_int32, C.c_void_p]
        L.dasc_padded_pool_floats.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int64)]
        L.dasc_pack_padded.argtypes = L.dasc_pack.argtypes
        L.dasc_restore_padded.argtypes = L.dasc_restore.argtypes
        L.dasc_checkpoint_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.POINTER(C.c_int64)]
        L.dasc_slot_budget.argtypes = [C.c_int64, C.c_void_p, C.c_int32, C.c_int64, C.POINTER(C.c_int64)]
        L.dasc_tp_balance.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.c_void_p]
        L.dasc_pack_tp.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_int32, C.c_void_p]
        L.dasc_restore_tp.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                      C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int32, C.c_void_p]
        L.dasc_tp_head_permutation.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.dasc_conv_store.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                      C.c_int32, C.c_void_p]
        L.dasc_conv_load.argtypes = L.dasc_conv_store.argtypes
        L.dasc_refresh_counters.argtypes = [C.c_void_p, C.c_size_t, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.dasc_debug_set_refresh_poll_limit.restype = None
        L.dasc_debug_set_refresh_poll_limit.argtypes = [C.c_uint32]
        L.dasc_int8_slot_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        L.dasc_pack_int8.argtypes = L.dasc_pack.argtypes
        L.dasc_restore_int8.argtypes = L.dasc_restore.argtypes
        L.dasc_refresh_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
        L.dasc_refresh.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int64,
                                   C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
        L.dasc_refresh_status.argtypes = [C.c_void_p, C.c_size_t]
        L.dasc_refresh_window.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                          C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.dasc_refresh_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                          C.c_int32, C.c_int32, C.POINTER(C.c_void_p), C.c_void_p]
        L.dasc_status_string.restype = C.c_char_p
        L.dasc_status_string.argtypes = [C.c_int]
        L.dasc_version.restype = C.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().dasc_status_string(int(status)).decode()


def version() -> str:
    return lib().dasc_version().decode()


def _check(status: int, where: str):
    if status != OK:
        raise DascError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return C.c_void_p(t.data_ptr())
    if isinstance(t, np.ndarray):
        return C.c_void_p(t.ctypes.data)
    return C.c_void_p(int(t))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


@dataclass
class Plan:
    """Owns a ``dasc_plan_t``; attributes mirror ``dasc_plan_info_t``."""
    handle: int
    info: PlanInfo

    def __getattr__(self, name):
        info = object.__getattribute__(self, "info")
        if name in {f[0] for f in PlanInfo._fields_}:
            return getattr(info, name)
        raise AttributeError(name)

    def _array(self, fn, dtype, shape):
        out = np.empty(shape, dtype)
        _check(getattr(lib(), fn)(self.handle, out.ctypes.data_as(C.c_void_p)), fn)
        return out

    def horizon(self):
        return self._array("dasc_plan_horizon", np.float64, (self.info.n_layers, self.info.units_per_layer))

    def mask(self):
        return self._array("dasc_plan_mask", np.uint8, (self.info.n_layers, self.info.units_per_layer))

    def window(self):
        return self._array("dasc_plan_window", np.int64, (self.info.n_layers, self.info.units_per_layer))

    def layer_counts(self):
        return self._array("dasc_plan_layer_counts", np.int64, (self.info.n_layers,))

    def layer_offsets(self):
        return self._array("dasc_plan_layer_offsets", np.int64, (self.info.n_layers + 1,))

    def destroy(self):
        if self.handle:
            lib().dasc_plan_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def dasc_plan(kind, n_layers, n_v_heads, n_k_heads, d_k, d_v, A_log, dt_bias, *, a=-0.3, eps=1e-3,
              sel=SEL_THRESHOLD, scope=SCOPE_LAYER, w_max=0.0, keep_ratio=1.0, randomize=False, seed=0,
              explicit_mask=None, conv_bytes_per_ckpt=0, device=0) -> Plan:
    """Build the selection plan.  ``A_log``/``dt_bias``: host arrays, one entry per unit.
    ``device=-1`` builds a host-only plan (no CUDA needed)."""
    A = np.ascontiguousarray(torch.as_tensor(A_log).detach().cpu().numpy() if isinstance(A_log, torch.Tensor) else A_log, np.float32)
    B = np.ascontiguousarray(torch.as_tensor(dt_bias).detach().cpu().numpy() if isinstance(dt_bias, torch.Tensor) else dt_bias, np.float32)
    uph = d_k if kind == KDA else 1
    if A.size != n_layers * n_v_heads * uph or B.size != A.size:
        raise ValueError("A_log / dt_bias need one entry per selection unit")
    em = None
    if explicit_mask is not None:
        em = np.ascontiguousarray(explicit_mask, np.uint8)
        if em.size != A.size:
            raise ValueError("explicit_mask needs one entry per selection unit")
    desc = PlanDesc(kind, n_layers, n_v_heads, n_k_heads, d_k, d_v, A.ctypes.data, B.ctypes.data, a, eps, sel, scope,
                    w_max, keep_ratio, 1 if randomize else 0, seed, em.ctypes.data if em is not None else None,
                    conv_bytes_per_ckpt)
    handle = C.c_void_p()
    _check(lib().dasc_plan(C.byref(desc), int(device), C.byref(handle)), "dasc_plan")
    info = PlanInfo()
    _check(lib().dasc_plan_info(handle, C.byref(info)), "dasc_plan_info")
    return Plan(handle.value, info)


def dasc_plan_save(plan: Plan) -> bytes:
    """The plan as a self-contained blob (build it once where the weights are, load it in the serving processes)."""
    n = C.c_size_t()
    _check(lib().dasc_plan_save_bytes(plan.handle, C.byref(n)), "dasc_plan_save_bytes")
    buf = C.create_string_buffer(n.value)
    _check(lib().dasc_plan_save(plan.handle, buf, n.value), "dasc_plan_save")
    return buf.raw


def dasc_plan_load(blob: bytes, device: int = 0) -> Plan:
    """Rebuild a plan from ``dasc_plan_save``'s blob; ``device=-1`` gives a host-only plan."""
    handle = C.c_void_p()
    _check(lib().dasc_plan_load(blob, len(blob), int(device), C.byref(handle)), "dasc_plan_load")
    info = PlanInfo()
    _check(lib().dasc_plan_info(handle, C.byref(info)), "dasc_plan_info")
    return Plan(handle.value, info)


def dasc_pack(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, src_req: torch.Tensor,
              pool: torch.Tensor, dst_slot: torch.Tensor, slot_stride: int = 0, stream=None):
    """Gather the retained units of ``state`` (requests ``src_req``) into pool slots ``dst_slot``."""
    _check(lib().dasc_pack(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(src_req), _ptr(pool), slot_stride,
                           _ptr(dst_slot), int(src_req.numel()), _stream_ptr(stream)), "dasc_pack")


def dasc_restore(plan: Plan, pool: torch.Tensor, src_slot: torch.Tensor, state: torch.Tensor, layer_stride: int,
                 req_stride: int, dst_req: torch.Tensor, slot_stride: int = 0, stream=None):
    """Scatter pool slots ``src_slot`` into the dense states ``dst_req``; omitted units become +0.0."""
    _check(lib().dasc_restore(plan.handle, _ptr(pool), slot_stride, _ptr(src_slot), _ptr(state), layer_stride,
                              req_stride, _ptr(dst_req), int(src_slot.numel()), _stream_ptr(stream)), "dasc_restore")


LAYOUT_RAGGED, LAYOUT_PADDED, LAYOUT_DENSE = 0, 1, 2


def dasc_padded_pool_floats(plan: Plan, n_slots: int) -> int:
    """Floats of a padded pool [L][n_slots][R_max][unit_floats] (Appendix B, Scheme 1)."""
    out = C.c_int64()
    _check(lib().dasc_padded_pool_floats(plan.handle, int(n_slots), C.byref(out)), "dasc_padded_pool_floats")
    return int(out.value)


def dasc_pack_padded(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, src_req: torch.Tensor,
                     pool: torch.Tensor, n_slots: int, dst_slot: torch.Tensor, stream=None):
    """``dasc_pack`` into the padded pool; padding entries are not written."""
    _check(lib().dasc_pack_padded(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(src_req), _ptr(pool),
                                  int(n_slots), _ptr(dst_slot), int(src_req.numel()), _stream_ptr(stream)),
           "dasc_pack_padded")


def dasc_restore_padded(plan: Plan, pool: torch.Tensor, n_slots: int, src_slot: torch.Tensor, state: torch.Tensor,
                        layer_stride: int, req_stride: int, dst_req: torch.Tensor, stream=None):
    """``dasc_restore`` from the padded pool."""
    _check(lib().dasc_restore_padded(plan.handle, _ptr(pool), int(n_slots), _ptr(src_slot), _ptr(state), layer_stride,
                                     req_stride, _ptr(dst_req), int(src_slot.numel()), _stream_ptr(stream)),
           "dasc_restore_padded")


def dasc_checkpoint_bytes(plan: Plan, layout: int, conv_bytes: int = 0) -> int:
    """Bytes of one checkpoint (temporal state under ``layout`` + convolution state), Eq. 6 / Appendix B."""
    out = C.c_int64()
    _check(lib().dasc_checkpoint_bytes(plan.handle, int(layout), int(conv_bytes), C.byref(out)), "dasc_checkpoint_bytes")
    return int(out.value)


def dasc_slot_budget(budget_bytes: int, temporal_bytes_per_rank, conv_bytes: int = 0) -> int:
    """Appendix C.1: N = floor(B / max_r(b_r + b_conv)) - 1."""
    arr = np.ascontiguousarray(temporal_bytes_per_rank, np.int64)
    out = C.c_int64()
    _check(lib().dasc_slot_budget(int(budget_bytes), arr.ctypes.data_as(C.c_void_p), int(arr.size), int(conv_bytes),
                                  C.byref(out)), "dasc_slot_budget")
    return int(out.value)


def dasc_tp_balance(units_per_rank):
    """Section 4.3: (C, send[T][T]) — slot width and the split sizes of the store-time all-to-all."""
    U = np.ascontiguousarray(units_per_rank, np.int64)
    send = np.zeros((U.size, U.size), np.int64)
    width = C.c_int64()
    _check(lib().dasc_tp_balance(U.ctypes.data_as(C.c_void_p), int(U.size), C.byref(width),
                                 send.ctypes.data_as(C.c_void_p)), "dasc_tp_balance")
    return int(width.value), send


def _tp_args(pools, units_per_rank):
    bases = (C.c_void_p * len(pools))(*[p.data_ptr() for p in pools])
    U = np.ascontiguousarray(units_per_rank, np.int64)
    if U.size != len(pools):
        raise ValueError("one pool and one unit count per rank")
    return bases, U


def dasc_pack_tp(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, src_req: torch.Tensor, pools,
                 units_per_rank, rank: int, dst_slot: torch.Tensor, slot_stride: int = 0, stream=None):
    """Section 4.3 Store: ``dasc_pack`` with every packed unit stored straight into the pool of the rank that owns
    its global position.  ``pools``: one device tensor per rank (this GPU's view of that rank's pool)."""
    bases, U = _tp_args(pools, units_per_rank)
    _check(lib().dasc_pack_tp(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(src_req), bases,
                              U.ctypes.data_as(C.c_void_p), int(U.size), int(rank), int(slot_stride), _ptr(dst_slot),
                              int(src_req.numel()), _stream_ptr(stream)), "dasc_pack_tp")


def dasc_restore_tp(plan: Plan, pools, units_per_rank, rank: int, src_slot: torch.Tensor, state: torch.Tensor,
                    layer_stride: int, req_stride: int, dst_req: torch.Tensor, slot_stride: int = 0, stream=None):
    """Section 4.3 Load: the inverse gather of ``dasc_pack_tp``, omitted units zero-filled."""
    bases, U = _tp_args(pools, units_per_rank)
    _check(lib().dasc_restore_tp(plan.handle, bases, U.ctypes.data_as(C.c_void_p), int(U.size), int(rank),
                                 int(slot_stride), _ptr(src_slot), _ptr(state), layer_stride, req_stride, _ptr(dst_req),
                                 int(src_slot.numel()), _stream_ptr(stream)), "dasc_restore_tp")


def dasc_tp_head_permutation(plan: Plan, n_ranks: int, heads_per_bundle: int = 1):
    """Section 4.3, first stage: (perm[L][n_bundles], units_per_rank[T]) of the load-time head-bundle placement."""
    n_bundles = plan.info.n_v_heads // max(1, heads_per_bundle)
    perm = np.full((plan.info.n_layers, n_bundles), -1, np.int32)
    U = np.zeros(n_ranks, np.int64)
    _check(lib().dasc_tp_head_permutation(plan.handle, int(n_ranks), int(heads_per_bundle),
                                          perm.ctypes.data_as(C.c_void_p), U.ctypes.data_as(C.c_void_p)),
           "dasc_tp_head_permutation")
    return perm, U


def dasc_conv_store(conv: torch.Tensor, req_stride_bytes: int, src_req: torch.Tensor, pool: torch.Tensor,
                    slot_stride_bytes: int, dst_slot: torch.Tensor, conv_bytes: int, stream=None):
    """Copy the convolution-state blob of each request into its checkpoint slot (Section 4.1, B_conv)."""
    _check(lib().dasc_conv_store(_ptr(conv), int(req_stride_bytes), _ptr(src_req), _ptr(pool), int(slot_stride_bytes),
                                 _ptr(dst_slot), int(conv_bytes), int(src_req.numel()), _stream_ptr(stream)),
           "dasc_conv_store")


def dasc_conv_load(pool: torch.Tensor, slot_stride_bytes: int, src_slot: torch.Tensor, conv: torch.Tensor,
                   req_stride_bytes: int, dst_req: torch.Tensor, conv_bytes: int, stream=None):
    """The inverse of ``dasc_conv_store``."""
    _check(lib().dasc_conv_load(_ptr(pool), int(slot_stride_bytes), _ptr(src_slot), _ptr(conv), int(req_stride_bytes),
                                _ptr(dst_req), int(conv_bytes), int(src_slot.numel()), _stream_ptr(stream)),
           "dasc_conv_load")


def dasc_int8_slot_bytes(plan: Plan) -> int:
    """Bytes of one INT8 slot: codes [packed_rows][d_v] then fp32 scales [packed_rows], rounded up to 16."""
    out = C.c_size_t()
    _check(lib().dasc_int8_slot_bytes(plan.handle, C.byref(out)), "dasc_int8_slot_bytes")
    return int(out.value)


def dasc_pack_int8(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, src_req: torch.Tensor,
                   pool: torch.Tensor, dst_slot: torch.Tensor, slot_stride_bytes: int = 0, stream=None):
    """Like ``dasc_pack`` with the Appendix D quantiser fused in; ``pool`` is a byte (uint8) tensor."""
    _check(lib().dasc_pack_int8(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(src_req), _ptr(pool),
                                slot_stride_bytes, _ptr(dst_slot), int(src_req.numel()), _stream_ptr(stream)),
           "dasc_pack_int8")


def dasc_restore_int8(plan: Plan, pool: torch.Tensor, src_slot: torch.Tensor, state: torch.Tensor, layer_stride: int,
                      req_stride: int, dst_req: torch.Tensor, slot_stride_bytes: int = 0, stream=None):
    """Like ``dasc_restore`` with the dequantisation fused in; ``pool`` is a byte (uint8) tensor."""
    _check(lib().dasc_restore_int8(plan.handle, _ptr(pool), slot_stride_bytes, _ptr(src_slot), _ptr(state),
                                   layer_stride, req_stride, _ptr(dst_req), int(src_slot.numel()),
                                   _stream_ptr(stream)), "dasc_restore_int8")


def dasc_refresh_workspace_bytes(plan: Plan, n_req: int, n_layers_in_call: int, algo: int = ALGO_AUTO) -> int:
    out = C.c_size_t()
    _check(lib().dasc_refresh_workspace_bytes(plan.handle, n_req, n_layers_in_call, algo, C.byref(out)),
           "dasc_refresh_workspace_bytes")
    return int(out.value)


def dasc_refresh(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, req_idx: torch.Tensor,
                 q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, g: torch.Tensor, beta: torch.Tensor,
                 cu_seqlens: torch.Tensor, total_tokens: int, max_seqlen: int, *, layer_begin: int = 0,
                 layer_end: int | None = None, q_scale: float = 1.0, o: torch.Tensor | None = None,
                 mode: int = REFRESH_CONTINUE, algo: int = ALGO_AUTO, workspace: torch.Tensor | None = None,
                 stream=None):
    """Replay the gated delta rule over each request's suffix, in place on ``state``."""
    io = IO_BF16 if q.dtype == torch.bfloat16 else IO_FP32
    o_io = IO_BF16 if (o is not None and o.dtype == torch.bfloat16) else IO_FP32
    if layer_end is None:
        layer_end = plan.info.n_layers
    ws_bytes = int(workspace.numel() * workspace.element_size()) if workspace is not None else 0
    _check(lib().dasc_refresh(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(req_idx), _ptr(q), _ptr(k),
                              _ptr(v), io, _ptr(g), _ptr(beta), _ptr(cu_seqlens), int(cu_seqlens.numel() - 1),
                              int(total_tokens), int(max_seqlen), layer_begin, layer_end, float(q_scale), _ptr(o),
                              o_io, mode, algo, _ptr(workspace), ws_bytes, _stream_ptr(stream)), "dasc_refresh")


def dasc_refresh_window(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, req_idx: torch.Tensor,
                        q: torch.Tensor | None, k: torch.Tensor, v: torch.Tensor, g: torch.Tensor, beta: torch.Tensor,
                        cu_seqlens: torch.Tensor, total_tokens: int, window_begin: torch.Tensor, *, window: int = 0,
                        layer_begin: int = 0, layer_end: int | None = None, q_scale: float = 1.0,
                        o: torch.Tensor | None = None, algo: int = ALGO_AUTO, workspace: torch.Tensor | None = None,
                        stream=None):
    """The paper's suffix-refresh load policy: replay each request's last ``window`` prefix tokens (0 = the
    plan's W_replay) from a zero scratch state and merge only the omitted units.  ``window_begin`` (int32
    [n_req], device) receives the first replayed token of each request.  ``q`` may be None when ``o`` is."""
    io = IO_BF16 if k.dtype == torch.bfloat16 else IO_FP32
    o_io = IO_BF16 if (o is not None and o.dtype == torch.bfloat16) else IO_FP32
    if layer_end is None:
        layer_end = plan.info.n_layers
    ws_bytes = int(workspace.numel() * workspace.element_size()) if workspace is not None else 0
    _check(lib().dasc_refresh_window(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(req_idx), _ptr(q),
                                     _ptr(k), _ptr(v), io, _ptr(g), _ptr(beta), _ptr(cu_seqlens),
                                     int(cu_seqlens.numel() - 1), int(total_tokens), int(window), layer_begin,
                                     layer_end, float(q_scale), _ptr(o), o_io, algo, _ptr(window_begin),
                                     _ptr(workspace), ws_bytes, _stream_ptr(stream)), "dasc_refresh_window")


def dasc_refresh_status(workspace) -> int:
    """Status of the last refresh that used ``workspace`` (a tensor, or the device address ``dasc_refresh_static``
    returned); call after synchronising the stream.  Reads both flag words (8 bytes)."""
    if workspace is None:
        return OK
    if isinstance(workspace, torch.Tensor):
        return int(lib().dasc_refresh_status(_ptr(workspace), int(workspace.numel() * workspace.element_size())))
    return int(lib().dasc_refresh_status(C.c_void_p(int(workspace)), 8))


def dasc_refresh_counters(workspace):
    """(units the chunked kernel handed over, units the exact kernel replayed) of the last call that used ``workspace``."""
    a, b = C.c_int32(), C.c_int32()
    if isinstance(workspace, torch.Tensor):
        ptr, n = _ptr(workspace), int(workspace.numel() * workspace.element_size())
    else:
        ptr, n = C.c_void_p(int(workspace)), 16
    _check(lib().dasc_refresh_counters(ptr, n, C.byref(a), C.byref(b)), "dasc_refresh_counters")
    return int(a.value), int(b.value)


def dasc_debug_set_refresh_poll_limit(polls: int):
    """Test hook: poll limit of the chunked kernel's first wait (0 = normal)."""
    lib().dasc_debug_set_refresh_poll_limit(int(polls))


def dasc_refresh_static(plan: Plan, state: torch.Tensor, layer_stride: int, req_stride: int, req_idx: torch.Tensor,
                        q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, g: torch.Tensor, beta: torch.Tensor,
                        cu_seqlens: torch.Tensor, total_tokens: int, max_seqlen: int, *, layer_begin: int = 0,
                        layer_end: int | None = None, q_scale: float = 1.0, o: torch.Tensor | None = None,
                        mode: int = REFRESH_CONTINUE, stream=None) -> int:
    """``dasc_refresh`` for callers that cannot allocate: no workspace argument, the kernel's scratch
    is a fixed array inside the library.  bf16 streams and d_k = d_v = 128 only.  Returns the device
    address of that array: pass it to ``dasc_refresh_status`` after a synchronise (both flag words are
    read: a wait that ran out, a log-decay outside the kernel's range).  Calls that overlap on the GPU
    share the array and race on it."""
    if q.dtype != torch.bfloat16:
        raise ValueError("dasc_refresh_static takes bf16 token streams")
    o_io = IO_BF16 if (o is not None and o.dtype == torch.bfloat16) else IO_FP32
    if layer_end is None:
        layer_end = plan.info.n_layers
    scratch = C.c_void_p()
    _check(lib().dasc_refresh_static(plan.handle, _ptr(state), layer_stride, req_stride, _ptr(req_idx), _ptr(q),
                                     _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu_seqlens),
                                     int(cu_seqlens.numel() - 1), int(total_tokens), int(max_seqlen), layer_begin,
                                     layer_end, float(q_scale), _ptr(o), o_io, mode, C.byref(scratch),
                                     _stream_ptr(stream)), "dasc_refresh_static")
    return int(scratch.value or 0)
