"""ctypes binding of liblibra.so: same names as the C ABI (include/libra.h), argument marshalling only.

Importing this module loads the shared library and raises if it has not been built
(``python -m paper_2606_03077_b200.build``); there is no fallback path of any kind.
Tensors are passed as raw device pointers (``tensor.data_ptr()``) and streams as
``torch.cuda.current_stream().cuda_stream``; this module itself never imports torch.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblibra.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2606_03077_b200.build`")
lib = C.CDLL(_LIB_PATH)
LIB_PATH = _LIB_PATH

STATIC_SCRATCH_BYTES = 8 << 20
OK, INVALID_ARGUMENT, UNSUPPORTED_SHAPE, WORKSPACE_TOO_SMALL, NOT_PLANNED, CUDA_ERROR, DEVICE_FLAGGED = range(7)
KV_BF16, KV_E4M3 = 0, 1
RING_F32, RING_BF16 = 0, 1
ERR_WAIT_TIMEOUT, ERR_BAD_PAGE_ID, ERR_SEQ_LEN_MISMATCH, ERR_PLAN_OVERFLOW = 1, 2, 4, 8


class PlanParams(C.Structure):
    _fields_ = [("n_sm", C.c_int32), ("ctas_per_sm", C.c_int32), ("items_per_slot", C.c_int32),
                ("chunk_align", C.c_int32), ("min_chunk", C.c_int32), ("max_splits", C.c_int32),
                ("refine", C.c_int32)]


class Config(C.Structure):
    _fields_ = [("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("num_pages", C.c_int64), ("max_batch", C.c_int32),
                ("block_table_ld", C.c_int32), ("kv_stride_page", C.c_int64), ("kv_stride_head", C.c_int64),
                ("kv_stride_token", C.c_int64), ("sm_scale", C.c_float), ("device", C.c_int32),
                ("plan", PlanParams)]


class PlanView(C.Structure):
    _fields_ = [("batch", C.c_int32), ("chunk_target", C.c_int32), ("num_items", C.c_int32),
                ("num_combine", C.c_int32), ("num_empty", C.c_int32),
                ("bucket", C.POINTER(C.c_int32)), ("num_splits", C.POINTER(C.c_int32)),
                ("chunk_len", C.POINTER(C.c_int32)), ("item_offset", C.POINTER(C.c_int32)),
                ("items", C.POINTER(C.c_int32)), ("combine", C.POINTER(C.c_int32)),
                ("empty", C.POINTER(C.c_int32))]


RING_MAX_MEMBERS = 64
RING_OP_SEND, RING_OP_RECV_REDUCE, RING_OP_RECV_COPY = 0, 1, 2


class Ring(C.Structure):
    """libra_ring_t: the live replicas in ring order (host metadata)."""
    _fields_ = [("n_members", C.c_int32), ("members", C.c_int32 * RING_MAX_MEMBERS), ("epoch", C.c_uint32)]


class RingOp(C.Structure):
    _fields_ = [("kind", C.c_int32), ("phase", C.c_int32), ("step", C.c_int32), ("segment", C.c_int32),
                ("piece", C.c_int32), ("peer", C.c_int32), ("offset", C.c_int64), ("bytes", C.c_int64)]


_i32p = C.POINTER(C.c_int32)
_vp = C.c_void_p

# every symbol include/libra.h declares, with its signature
SIGNATURES = {
    "libra_version": (C.c_int, []),
    "libra_status_string": (C.c_char_p, [C.c_int]),
    "libra_create": (C.c_int, [C.POINTER(_vp), C.POINTER(Config)]),
    "libra_destroy": (C.c_int, [_vp]),
    "libra_workspace_size": (C.c_int, [_vp, C.POINTER(C.c_size_t)]),
    "libra_get_plan_params": (C.c_int, [_vp, C.POINTER(PlanParams)]),
    "libra_set_variant": (C.c_int, [_vp, C.c_int32, C.c_int32]),
    "libra_set_dependent_launch": (C.c_int, [_vp, C.c_int32]),
    "libra_set_max_query_tokens": (C.c_int, [_vp, C.c_int32]),
    "libra_set_early_prefetch": (C.c_int, [_vp, C.c_int32]),
    "libra_set_cache_warmup": (C.c_int, [_vp, C.c_int32]),
    "libra_set_lse_output": (C.c_int, [_vp, _vp]),
    "libra_set_kv_dtype": (C.c_int, [_vp, C.c_int32, C.c_float, C.c_float]),
    "libra_decode_attn_multi": (C.c_int, [_vp, _vp, C.c_int32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_decode_attn_multi_append": (C.c_int, [_vp, _vp, C.c_int32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_ring_step": (C.c_int, [C.c_int32, _vp, _vp, _vp, C.c_size_t, C.c_int32, _vp, C.c_uint32, C.c_uint32, _vp, C.c_int32,
                                  _vp]),
    "libra_ring_init": (C.c_int, [C.POINTER(Ring), _i32p, C.c_int32]),
    "libra_ring_remove": (C.c_int, [C.POINTER(Ring), C.c_int32]),
    "libra_ring_insert": (C.c_int, [C.POINTER(Ring), C.c_int32, C.c_int32]),
    "libra_ring_neighbors": (C.c_int, [C.POINTER(Ring), C.c_int32, _i32p, _i32p]),
    "libra_ring_schedule": (C.c_int, [C.POINTER(Ring), C.c_int32, C.c_int64, C.c_int64, C.POINTER(RingOp), C.c_int32,
                                      _i32p]),
    "libra_ring_all_reduce_local": (C.c_int, [C.c_int32, C.POINTER(_vp), C.c_int32, C.c_size_t, C.c_int32, C.c_size_t,
                                              _vp, C.c_uint32, C.c_uint32, _vp, C.c_int32, _vp]),
    "libra_merge_parts": (C.c_int, [C.c_int32, _vp, _vp, C.c_int32, C.c_int64, C.c_int32, _vp, _vp, _vp]),
    "libra_debug_stream_read": (C.c_int, [_vp, _vp, C.c_size_t, _vp]),
    "libra_debug_gather_read": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_set_combine_mode": (C.c_int, [_vp, C.c_int32]),
    "libra_set_length_hint": (C.c_int, [_vp, C.c_int32]),
    "libra_plan_host": (C.c_int, [C.POINTER(PlanParams), C.c_int32, _i32p, C.c_int32, _i32p, _i32p, _i32p, _i32p,
                                  _i32p, _i32p, C.c_int32, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "libra_workspace_invalidate": (C.c_int, [_vp]),
    "libra_plan": (C.c_int, [_vp, _i32p, C.c_int32, _vp, C.c_size_t, _vp]),
    "libra_plan_device": (C.c_int, [_vp, _vp, C.c_int32, _vp, C.c_size_t, _vp]),
    "libra_plan_export": (C.c_int, [_vp, C.POINTER(PlanView)]),
    "libra_decode_attn": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_decode_attn_append": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_decode_attn_host": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, _vp, _vp, C.c_size_t, _vp,
                                         C.c_size_t, _vp]),
    "libra_decode_attn_static": (C.c_int, [_vp, _i32p, C.c_int32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "libra_host_staging_size": (C.c_int, [_vp, C.c_int32, C.POINTER(C.c_size_t)]),
    "libra_decode_attn_host_io": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, _vp, _vp, C.c_size_t, _vp,
                                            C.c_size_t, _vp]),
    "libra_host_io_staging_size": (C.c_int, [_vp, C.c_int32, C.POINTER(C.c_size_t)]),
    "libra_last_cuda_error": (C.c_int, [_vp]),
    "libra_debug_error_word": (C.c_int, [_vp, C.POINTER(C.c_uint32)]),
    "libra_kv_gather": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp,
                                  _vp, _vp]),
    "libra_kv_scatter": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp,
                                   _vp, _vp]),
    "libra_rollout_dp": (C.c_int, [C.c_int32, _i32p, C.c_int32, _i32p, C.c_int32, C.POINTER(C.c_double),
                                   C.POINTER(C.c_double), _i32p, _i32p, _i32p, C.c_int32, _i32p]),
    "libra_trie_create": (C.c_int, [C.POINTER(_vp), _i32p, C.c_int32]),
    "libra_trie_destroy": (C.c_int, [_vp]),
    "libra_trie_insert": (C.c_int, [_vp, C.c_int64, _i32p, C.c_int32, _i32p]),
    "libra_trie_lookup": (C.c_int, [_vp, C.c_int64, _i32p, C.c_int32, C.POINTER(C.c_double), _i32p,
                                    C.POINTER(C.c_int64)]),
    "libra_trie_route": (C.c_int, [_vp, C.c_int64, _i32p, C.c_int32, C.c_int32, C.POINTER(C.c_double),
                                   C.POINTER(C.c_double), _i32p, C.POINTER(C.c_double)]),
    "libra_debug_wait_selftest": (C.c_int, [_vp, _vp]),
    "libra_profile_begin": (C.c_int, [_vp]),
    "libra_profile_end": (C.c_int, [_vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int32)]),
    "libra_launch_count": (C.c_int, [_vp, C.POINTER(C.c_int64)]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class LibraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {libra_status_string(status)} (status {status})")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise LibraError(status, where)


def libra_version() -> int:
    return lib.libra_version()


def libra_status_string(status: int) -> str:
    return lib.libra_status_string(status).decode()


def _as_i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def libra_plan_host(seq_lens, num_kv_heads: int, params: PlanParams, items_capacity: int | None = None) -> dict:
    """Pure host planner; returns the plan as a dict of NumPy arrays / ints."""
    lens = _as_i32(seq_lens)
    B = int(lens.shape[0])
    cap = (B * 64 + 1) if items_capacity is None else items_capacity
    out = {k: np.zeros(max(B, 1), dtype=np.int32) for k in ("bucket", "num_splits", "chunk_len", "item_offset",
                                                            "combine", "empty")}
    items = np.zeros((max(cap, 1), 4), dtype=np.int32)
    scal = {k: C.c_int32(0) for k in ("chunk_target", "num_items", "num_combine", "num_empty")}
    p = lambda a: a.ctypes.data_as(_i32p)
    st = lib.libra_plan_host(C.byref(params), num_kv_heads, p(lens), B, C.byref(scal["chunk_target"]),
                             p(out["bucket"]), p(out["num_splits"]), p(out["chunk_len"]), p(out["item_offset"]),
                             p(items), cap, C.byref(scal["num_items"]), p(out["combine"]),
                             C.byref(scal["num_combine"]), p(out["empty"]), C.byref(scal["num_empty"]))
    _check(st, "libra_plan_host")
    n = scal["num_items"].value
    return {"chunk_target": scal["chunk_target"].value, "bucket": out["bucket"][:B].copy(),
            "num_splits": out["num_splits"][:B].copy(), "chunk_len": out["chunk_len"][:B].copy(),
            "item_offset": out["item_offset"][:B].copy(), "items": items[:n].copy(),
            "combine": out["combine"][:scal["num_combine"].value].copy(),
            "empty": out["empty"][:scal["num_empty"].value].copy()}


def libra_ring_step(device: int, dst_ptr: int, own_ptr: int, received_ptr: int, nbytes: int, dtype: int,
                    ready_flag_ptr: int, expected: int, timeout_us: int, status_ptr: int, num_blocks: int,
                    stream: int) -> None:
    """One copy / reduce step of the ring all-reduce's data plane (own_ptr = 0 for a copy step)."""
    _check(lib.libra_ring_step(device, dst_ptr, own_ptr or None, received_ptr, nbytes, dtype, ready_flag_ptr, expected,
                               timeout_us, status_ptr, num_blocks, stream), "libra_ring_step")


def libra_ring_init(ids) -> Ring:
    ring = Ring()
    a = _as_i32(ids)
    _check(lib.libra_ring_init(C.byref(ring), a.ctypes.data_as(_i32p), len(a)), "libra_ring_init")
    return ring


def libra_ring_remove(ring: Ring, member_id: int) -> None:
    _check(lib.libra_ring_remove(C.byref(ring), member_id), "libra_ring_remove")


def libra_ring_insert(ring: Ring, member_id: int, position: int) -> None:
    _check(lib.libra_ring_insert(C.byref(ring), member_id, position), "libra_ring_insert")


def libra_ring_neighbors(ring: Ring, member_id: int):
    pred, succ = C.c_int32(0), C.c_int32(0)
    _check(lib.libra_ring_neighbors(C.byref(ring), member_id, C.byref(pred), C.byref(succ)), "libra_ring_neighbors")
    return pred.value, succ.value


def libra_ring_schedule(ring: Ring, member_id: int, nbytes: int, piece_bytes: int):
    """The member's records, in issue order, as dicts."""
    n = C.c_int32(0)
    st = lib.libra_ring_schedule(C.byref(ring), member_id, nbytes, piece_bytes, None, 0, C.byref(n))
    if st not in (OK, WORKSPACE_TOO_SMALL):
        _check(st, "libra_ring_schedule")
    ops = (RingOp * max(1, n.value))()
    _check(lib.libra_ring_schedule(C.byref(ring), member_id, nbytes, piece_bytes, ops, n.value, C.byref(n)),
           "libra_ring_schedule")
    return [{f: getattr(ops[i], f) for f, _ in RingOp._fields_} for i in range(n.value)]


def libra_ring_all_reduce_local(device: int, buf_ptrs, nbytes: int, dtype: int, piece_bytes: int, ready_flag_ptr: int,
                                expected: int, timeout_us: int, status_ptr: int, num_blocks: int, stream: int) -> None:
    """ReduceScatter + AllGather over vectors on one device (buf_ptrs[i] = the member at ring position i)."""
    arr = (_vp * len(buf_ptrs))(*buf_ptrs)
    _check(lib.libra_ring_all_reduce_local(device, arr, len(buf_ptrs), nbytes, dtype, piece_bytes, ready_flag_ptr,
                                           expected, timeout_us, status_ptr, num_blocks, stream),
           "libra_ring_all_reduce_local")


def libra_merge_parts(device: int, parts_out_ptr: int, parts_lse_ptr: int, n_parts: int, rows: int, head_dim: int,
                      out_ptr: int, lse_out_ptr: int, stream: int) -> None:
    """Log-sum-exp merge of (out, lse) pairs computed over disjoint parts of the same sequences."""
    _check(lib.libra_merge_parts(device, parts_out_ptr, parts_lse_ptr, n_parts, rows, head_dim, out_ptr,
                                 lse_out_ptr or None, stream), "libra_merge_parts")


def libra_rollout_dp(n_gpus: int, lengths, tp_set, cost_coef):
    """RolloutDP: returns (makespan, [(tp, first_sorted_index, count), ...])."""
    lens = _as_i32(lengths)
    tps = _as_i32(tp_set)
    coef = np.ascontiguousarray(cost_coef, dtype=np.float64).reshape(len(tps), 4)
    cap = max(1, n_gpus)
    itp, ifirst, icount = (np.zeros(cap, np.int32) for _ in range(3))
    mk, n = C.c_double(0), C.c_int32(0)
    p = lambda a: a.ctypes.data_as(_i32p)
    st = lib.libra_rollout_dp(n_gpus, p(lens), len(lens), p(tps), len(tps), coef.ctypes.data_as(C.POINTER(C.c_double)),
            C.byref(mk), p(itp), p(ifirst), p(icount), cap, C.byref(n))
    _check(st, "libra_rollout_dp")
    return mk.value, [(int(itp[k]), int(ifirst[k]), int(icount[k])) for k in range(n.value)]


class Trie:
    """Owns one libra_trie_t (the causality-aware prefix tree)."""

    def __init__(self, bin_upper):
        self.bins = _as_i32(bin_upper)
        self._t = _vp()
        _check(lib.libra_trie_create(C.byref(self._t), self.bins.ctypes.data_as(_i32p), len(self.bins)), "libra_trie_create")

    def close(self):
        if self._t:
            lib.libra_trie_destroy(self._t)
            self._t = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def insert(self, prompt_id: int, states, residual_lengths) -> None:
        s, r = _as_i32(states), _as_i32(residual_lengths)
        assert len(r) == len(s) + 1
        _check(lib.libra_trie_insert(self._t, prompt_id, s.ctypes.data_as(_i32p), len(s), r.ctypes.data_as(_i32p)),
               "libra_trie_insert")

    def lookup(self, prompt_id: int, states):
        s = _as_i32(states)
        hist = np.zeros(len(self.bins) + 1, np.float64)
        depth, n = C.c_int32(0), C.c_int64(0)
        _check(lib.libra_trie_lookup(self._t, prompt_id, s.ctypes.data_as(_i32p), len(s),
                                     hist.ctypes.data_as(C.POINTER(C.c_double)), C.byref(depth), C.byref(n)),
               "libra_trie_lookup")
        return hist, depth.value, n.value

    def route(self, prompt_id: int, states, decode_cost, migration_cost):
        s = _as_i32(states)
        dc = np.ascontiguousarray(decode_cost, dtype=np.float64)
        mc = np.ascontiguousarray(migration_cost, dtype=np.float64)
        best, cost = C.c_int32(0), C.c_double(0)
        _check(lib.libra_trie_route(self._t, prompt_id, s.ctypes.data_as(_i32p), len(s), len(mc),
                                    dc.ctypes.data_as(C.POINTER(C.c_double)), mc.ctypes.data_as(C.POINTER(C.c_double)),
                                    C.byref(best), C.byref(cost)), "libra_trie_route")
        return best.value, cost.value


class Handle:
    """Owns one libra_handle_t."""

    def __init__(self, num_q_heads: int, num_kv_heads: int, head_dim: int, num_pages: int, max_batch: int,
                 block_table_ld: int, page_size: int = 16, kv_strides=(0, 0, 0), sm_scale: float = 0.0,
                 device: int = 0, plan: PlanParams | None = None):
        self.cfg = Config(num_q_heads, num_kv_heads, head_dim, page_size, num_pages, max_batch, block_table_ld,
                          kv_strides[0], kv_strides[1], kv_strides[2], sm_scale, device, plan or PlanParams())
        self._h = _vp()
        _check(lib.libra_create(C.byref(self._h), C.byref(self.cfg)), "libra_create")

    def close(self) -> None:
        if self._h:
            lib.libra_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- thin wrappers, one per entry point
    def workspace_size(self) -> int:
        n = C.c_size_t(0)
        _check(lib.libra_workspace_size(self._h, C.byref(n)), "libra_workspace_size")
        return n.value

    def plan_params(self) -> PlanParams:
        p = PlanParams()
        _check(lib.libra_get_plan_params(self._h, C.byref(p)), "libra_get_plan_params")
        return p

    def set_variant(self, warps: int, stages: int) -> None:
        _check(lib.libra_set_variant(self._h, warps, stages), "libra_set_variant")

    def set_dependent_launch(self, on: bool) -> None:
        _check(lib.libra_set_dependent_launch(self._h, 1 if on else 0), "libra_set_dependent_launch")

    def set_combine_mode(self, mode: int) -> None:
        """0: separate combine kernel, 1: inside the decode kernel (default)."""
        _check(lib.libra_set_combine_mode(self._h, int(mode)), "libra_set_combine_mode")

    def plan(self, seq_lens_host: np.ndarray, workspace_ptr: int, workspace_bytes: int, stream: int) -> None:
        lens = _as_i32(seq_lens_host)
        _check(lib.libra_plan(self._h, lens.ctypes.data_as(_i32p), int(lens.shape[0]), workspace_ptr,
                              workspace_bytes, stream), "libra_plan")

    def plan_device(self, seq_lens_dev_ptr: int, batch: int, workspace_ptr: int, workspace_bytes: int,
                    stream: int) -> None:
        _check(lib.libra_plan_device(self._h, seq_lens_dev_ptr, batch, workspace_ptr, workspace_bytes, stream),
               "libra_plan_device")

    def plan_export(self) -> dict:
        v = PlanView()
        _check(lib.libra_plan_export(self._h, C.byref(v)), "libra_plan_export")
        arr = lambda ptr, n: np.ctypeslib.as_array(ptr, shape=(n,)).copy() if n > 0 else np.zeros(0, np.int32)
        return {"chunk_target": v.chunk_target, "bucket": arr(v.bucket, v.batch),
                "num_splits": arr(v.num_splits, v.batch), "chunk_len": arr(v.chunk_len, v.batch),
                "item_offset": arr(v.item_offset, v.batch), "items": arr(v.items, v.num_items * 4).reshape(-1, 4),
                "combine": arr(v.combine, v.num_combine), "empty": arr(v.empty, v.num_empty)}

    def decode_attn(self, q_ptr: int, k_ptr: int, v_ptr: int, block_table_ptr: int, seq_lens_ptr: int,
                    out_ptr: int, stream: int) -> None:
        _check(lib.libra_decode_attn(self._h, q_ptr, k_ptr, v_ptr, block_table_ptr, seq_lens_ptr, out_ptr, stream),
               "libra_decode_attn")

    def debug_stream_read(self, buf_ptr: int, nbytes: int, stream: int) -> None:
        _check(lib.libra_debug_stream_read(self._h, buf_ptr, nbytes, stream), "libra_debug_stream_read")

    def debug_gather_read(self, q_ptr: int, k_ptr: int, v_ptr: int, block_table_ptr: int, seq_lens_ptr: int,
                          out_ptr: int, stream: int) -> None:
        _check(lib.libra_debug_gather_read(self._h, q_ptr, k_ptr, v_ptr, block_table_ptr, seq_lens_ptr, out_ptr, stream),
               "libra_debug_gather_read")

    def set_kv_dtype(self, dtype: int, k_scale: float = 1.0, v_scale: float = 1.0) -> None:
        _check(lib.libra_set_kv_dtype(self._h, dtype, k_scale, v_scale), "libra_set_kv_dtype")

    def set_lse_output(self, lse_ptr: int) -> None:
        _check(lib.libra_set_lse_output(self._h, lse_ptr or None), "libra_set_lse_output")

    def set_cache_warmup(self, on: bool) -> None:
        _check(lib.libra_set_cache_warmup(self._h, 1 if on else 0), "libra_set_cache_warmup")

    def set_length_hint(self, max_seq_len: int) -> None:
        """The caller's bound on the lengths of device-planned batches (0 = none): picks the block shape."""
        _check(lib.libra_set_length_hint(self._h, int(max_seq_len)), "libra_set_length_hint")

    def set_early_prefetch(self, on: bool) -> None:
        _check(lib.libra_set_early_prefetch(self._h, 1 if on else 0), "libra_set_early_prefetch")

    def set_max_query_tokens(self, max_q_len: int) -> None:
        _check(lib.libra_set_max_query_tokens(self._h, max_q_len), "libra_set_max_query_tokens")

    def decode_attn_multi(self, q_ptr: int, q_len: int, k_ptr: int, v_ptr: int, block_table_ptr: int,
                          seq_lens_ptr: int, out_ptr: int, stream: int) -> None:
        _check(lib.libra_decode_attn_multi(self._h, q_ptr, q_len, k_ptr, v_ptr, block_table_ptr, seq_lens_ptr,
                                           out_ptr, stream), "libra_decode_attn_multi")

    def decode_attn_multi_append(self, q_ptr: int, q_len: int, k_new_ptr: int, v_new_ptr: int, k_ptr: int, v_ptr: int,
                                 block_table_ptr: int, seq_lens_ptr: int, out_ptr: int, stream: int) -> None:
        _check(lib.libra_decode_attn_multi_append(self._h, q_ptr, q_len, k_new_ptr, v_new_ptr, k_ptr, v_ptr,
                                                  block_table_ptr, seq_lens_ptr, out_ptr, stream),
               "libra_decode_attn_multi_append")

    def decode_attn_append(self, q_ptr: int, k_new_ptr: int, v_new_ptr: int, k_ptr: int, v_ptr: int,
                           block_table_ptr: int, seq_lens_ptr: int, out_ptr: int, stream: int) -> None:
        _check(lib.libra_decode_attn_append(self._h, q_ptr, k_new_ptr, v_new_ptr, k_ptr, v_ptr, block_table_ptr,
                                            seq_lens_ptr, out_ptr, stream), "libra_decode_attn_append")

    def decode_attn_static(self, seq_lens_host: np.ndarray, q_ptr: int, k_ptr: int, v_ptr: int,
                           block_table_ptr: int, seq_lens_ptr: int, out_ptr: int, stream: int) -> None:
        """Plan + decode + combine on the scratch region built into the library: no workspace argument
        and no allocation.  Calls on one device share that region, so they must not overlap on the GPU."""
        lens = _as_i32(seq_lens_host)
        _check(lib.libra_decode_attn_static(self._h, lens.ctypes.data_as(_i32p), int(lens.shape[0]), q_ptr, k_ptr,
                                            v_ptr, block_table_ptr, seq_lens_ptr, out_ptr, stream),
               "libra_decode_attn_static")

    def workspace_invalidate(self) -> None:
        _check(lib.libra_workspace_invalidate(self._h), "libra_workspace_invalidate")

    def host_staging_size(self, batch: int) -> int:
        n = C.c_size_t(0)
        _check(lib.libra_host_staging_size(self._h, batch, C.byref(n)), "libra_host_staging_size")
        return n.value

    def decode_attn_host(self, q_host_ptr: int, k_host_ptr: int, v_host_ptr: int, block_table_host_ptr: int,
                         seq_lens_host_ptr: int, batch: int, out_host_ptr: int, staging_ptr: int,
                         staging_bytes: int, workspace_ptr: int, workspace_bytes: int, stream: int) -> None:
        _check(lib.libra_decode_attn_host(self._h, q_host_ptr, k_host_ptr, v_host_ptr, block_table_host_ptr,
                                          seq_lens_host_ptr, batch, out_host_ptr, staging_ptr, staging_bytes,
                                          workspace_ptr, workspace_bytes, stream), "libra_decode_attn_host")

    def host_io_staging_size(self, batch: int) -> int:
        n = C.c_size_t(0)
        _check(lib.libra_host_io_staging_size(self._h, batch, C.byref(n)), "libra_host_io_staging_size")
        return n.value

    def decode_attn_host_io(self, q_host_ptr: int, k_ptr: int, v_ptr: int, block_table_host_ptr: int,
                            seq_lens_host_ptr: int, batch: int, out_host_ptr: int, staging_ptr: int,
                            staging_bytes: int, workspace_ptr: int, workspace_bytes: int, stream: int) -> None:
        _check(lib.libra_decode_attn_host_io(self._h, q_host_ptr, k_ptr, v_ptr, block_table_host_ptr,
                                             seq_lens_host_ptr, batch, out_host_ptr, staging_ptr, staging_bytes,
                                             workspace_ptr, workspace_bytes, stream), "libra_decode_attn_host_io")

    def last_cuda_error(self) -> int:
        return lib.libra_last_cuda_error(self._h)

    def debug_error_word(self) -> int:
        w = C.c_uint32(0)
        _check(lib.libra_debug_error_word(self._h, C.byref(w)), "libra_debug_error_word")
        return w.value

    def kv_gather(self, k_ptr: int, v_ptr: int, block_table_ptr: int, seq_lens_ptr: int, token_offsets_ptr: int,
                  batch: int, max_seq_len: int, head_begin: int, head_count: int, k_dense_ptr: int, v_dense_ptr: int,
                  error_word_ptr: int, stream: int) -> None:
        _check(lib.libra_kv_gather(self._h, k_ptr, v_ptr, block_table_ptr, seq_lens_ptr, token_offsets_ptr, batch,
                                   max_seq_len, head_begin, head_count, k_dense_ptr, v_dense_ptr, error_word_ptr,
                                   stream), "libra_kv_gather")

    def kv_scatter(self, k_dense_ptr: int, v_dense_ptr: int, block_table_ptr: int, seq_lens_ptr: int,
                   token_offsets_ptr: int, batch: int, max_seq_len: int, head_begin: int, head_count: int, k_ptr: int,
                   v_ptr: int, error_word_ptr: int, stream: int) -> None:
        _check(lib.libra_kv_scatter(self._h, k_dense_ptr, v_dense_ptr, block_table_ptr, seq_lens_ptr,
                                    token_offsets_ptr, batch, max_seq_len, head_begin, head_count, k_ptr, v_ptr,
                                    error_word_ptr, stream), "libra_kv_scatter")

    def debug_wait_selftest(self, stream: int) -> None:
        _check(lib.libra_debug_wait_selftest(self._h, stream), "libra_debug_wait_selftest")

    def profile_begin(self) -> None:
        _check(lib.libra_profile_begin(self._h), "libra_profile_begin")

    def profile_end(self):
        d, c, n = C.c_double(0), C.c_double(0), C.c_int32(0)
        _check(lib.libra_profile_end(self._h, C.byref(d), C.byref(c), C.byref(n)), "libra_profile_end")
        return d.value, c.value, n.value

    def launch_count(self) -> int:
        n = C.c_int64(0)
        _check(lib.libra_launch_count(self._h, C.byref(n)), "libra_launch_count")
        return n.value
