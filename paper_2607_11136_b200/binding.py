"""ctypes binding of libxema.so: the same names as the C ABI, argument marshalling only.

Every step of the hot path runs inside the CUDA library.  There is no CPU fallback: if the
library is missing, loading raises, and nothing here imports the test oracle.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("XEMA_LIB") or os.path.join(_HERE, "libxema.so")

XEMA_OK, XEMA_EINVAL, XEMA_ENOSPC, XEMA_EBUDGET = 0, -1, -2, -3
XEMA_EALIGN, XEMA_ECUDA, XEMA_ETIMEOUT, XEMA_ESTATE = -4, -5, -6, -7
EPI_BIAS, EPI_BIAS_GELU, EPI_GATE_RES_F32, EPI_GATE_RES_BF16, EPI_BIAS_NORM_ROPE = 0, 1, 2, 3, 4

EXPORTS = (
    "xema_trace", "xema_trace_phases", "xema_plan_arena", "xema_chunks_for_budget",
    "xema_phase_chunks_for_budget", "xema_pressure_ranges", "xema_trace_mitigated", "xema_mitigation_for_budget", "xema_rope_table",
    "xema_plan_create", "xema_plan_create_phases", "xema_plan_create_mitigated", "xema_plan_destroy",
    "xema_plan_info", "xema_plan_phase_chunks", "xema_plan_mitigation", "xema_plan_tensor",
    "xema_plan_tensor_at", "xema_plan_bind", "xema_block_forward", "xema_step_forward",
    "xema_block_forward_static",
    "xema_shard_rows", "xema_trace_sharded", "xema_plan_create_sharded", "xema_plan_shard", "xema_plan_gather_point", "xema_plan_create_guarded", "xema_plan_guard_bytes",
    "xema_plan_launch_count", "xema_forward_host", "xema_forward_prefix", "xema_forward_range", "xema_plan_op", "xema_op_mod", "xema_op_ln_modulate",
    "xema_op_rmsnorm_rope", "xema_op_gemm", "xema_op_attention", "xema_strerror",
    "xema_last_cuda_error", "xema_version", "xema_selftest_wait_timeout",
    "xema_pluggable_malloc", "xema_pluggable_free", "xema_pluggable_mode", "xema_pluggable_recorded",
    "xema_pluggable_set_plan", "xema_pluggable_step_begin", "xema_pluggable_stats",
)
ALLOC_PASSTHROUGH, ALLOC_RECORD, ALLOC_REPLAY = 0, 1, 2
SPLIT_ROWS, SPLIT_BATCH = 0, 1


class xema_mitigation(C.Structure):
    _fields_ = [("chunks", C.c_int32 * 3), ("axis", C.c_int32 * 3)]


class XemaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = "%s: %s (status %d" % (where, strerror(status), status)
        if status == XEMA_ECUDA:
            msg += ", cuda error %d" % last_cuda_error()
        super().__init__(msg + ")")


class xema_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "s_text", "grid_t", "grid_h", "grid_w", "hidden", "heads",
                                         "head_dim", "ffn", "temb_dim", "rope_dim_t", "rope_dim_h", "rope_dim_w")]
    _fields_ += [("rope_base", C.c_float), ("ln_eps", C.c_float), ("rms_eps", C.c_float), ("n_blocks", C.c_int32)]


class xema_tensor(C.Structure):
    _fields_ = [("name", C.c_char * 24), ("kind", C.c_uint32), ("dtype", C.c_uint32), ("block", C.c_int32),
                ("chunk", C.c_int32), ("bytes", C.c_uint64), ("birth", C.c_uint32), ("death", C.c_uint32)]


_WEIGHT_FIELDS = ("w_mod", "b_mod", "w_qkv", "b_qkv", "g_q", "g_k", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2")


class xema_block_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WEIGHT_FIELDS]


class xema_gemm_args(C.Structure):
    _fields_ = [("a", C.c_void_p), ("lda", C.c_int64), ("a_batch_rows", C.c_int64),
                ("w", C.c_void_p), ("ldw", C.c_int64), ("bias", C.c_void_p),
                ("out", C.c_void_p), ("ldo", C.c_int64), ("out_batch_rows", C.c_int64),
                ("resid", C.c_void_p), ("ldr", C.c_int64), ("resid_batch_rows", C.c_int64),
                ("gate", C.c_void_p), ("gate_stride", C.c_int64),
                ("batch", C.c_int32), ("rows", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
                ("epilogue", C.c_int32), ("head_dim", C.c_int32), ("norm_cols", C.c_int32),
                ("rope_pos0", C.c_int32), ("rms_eps", C.c_float), ("norm_out_scale", C.c_float),
                ("norm_gain", C.c_void_p),
                ("rope", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Loads libxema.so (built in-tree by paper_2607_11136_b200.build).  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libxema.so is not built: run `python -m paper_2607_11136_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64, u32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_uint32, C.c_size_t
        P = C.POINTER
        sig = {
            "xema_trace": [P(xema_config), i32, P(xema_tensor), sz, P(sz), P(u32)],
            "xema_trace_phases": [P(xema_config), P(i32), P(xema_tensor), sz, P(sz), P(u32)],
            "xema_phase_chunks_for_budget": [P(xema_config), u64, i32, P(i32), P(u64)],
            "xema_plan_create_phases": [P(xema_config), P(i32), P(vp)],
            "xema_trace_mitigated": [P(xema_config), P(xema_mitigation), P(xema_tensor), sz, P(sz), P(u32)],
            "xema_mitigation_for_budget": [P(xema_config), u64, i32, P(xema_mitigation), P(u64)],
            "xema_plan_create_mitigated": [P(xema_config), P(xema_mitigation), P(vp)],
            "xema_plan_create_sharded": [P(xema_config), P(xema_mitigation), i32, i32, P(vp)],
            "xema_trace_sharded": [P(xema_config), P(xema_mitigation), i32, i32, P(xema_tensor), sz, P(sz), P(u32)],
            "xema_shard_rows": [P(xema_config), i32, i32, P(i64), P(i64)],
            "xema_plan_shard": [vp, P(i32), P(i32), P(i64), P(i64)],
            "xema_plan_create_guarded": [P(xema_config), P(xema_mitigation), i32, i32, u64, P(vp)],
            "xema_plan_guard_bytes": [vp],
            "xema_plan_gather_point": [vp, i32, P(u32), P(u64)],
            "xema_plan_mitigation": [vp, P(xema_mitigation)],
            "xema_plan_phase_chunks": [vp, P(i32)],
            "xema_plan_arena": [P(xema_tensor), sz, P(u64), P(u64), P(u64)],
            "xema_pressure_ranges": [P(xema_tensor), sz, u32, u64, P(u32), sz, P(sz)],
            "xema_pluggable_mode": [C.c_int],
            "xema_pluggable_recorded": [P(xema_tensor), sz, P(sz), P(u32)],
            "xema_pluggable_set_plan": [vp, u64, P(u64), sz],
            "xema_pluggable_step_begin": [],
            "xema_pluggable_stats": [P(u64), P(u64), P(u64)],
            "xema_chunks_for_budget": [P(xema_config), u64, i32, P(i32), P(u64)],
            "xema_rope_table": [P(xema_config), vp],
            "xema_plan_create": [P(xema_config), i32, P(vp)],
            "xema_plan_info": [vp, P(u64), P(u64), P(sz), P(u32), P(i32)],
            "xema_plan_tensor": [vp, C.c_char_p, P(u64), P(u64)],
            "xema_plan_tensor_at": [vp, sz, P(xema_tensor), P(u64)],
            "xema_plan_bind": [vp, vp, u64, P(xema_block_weights), vp, vp],
            "xema_block_forward": [vp, vp],
            "xema_step_forward": [vp, vp],
            "xema_forward_host": [vp, vp, vp, vp, vp],
            "xema_block_forward_static": [P(xema_config), i32, P(xema_block_weights), vp, vp, vp, vp, vp, vp],
            "xema_plan_launch_count": [vp],
            "xema_forward_prefix": [vp, u32, vp],
            "xema_forward_range": [vp, u32, u32, vp],
            "xema_plan_op": [vp, u32, C.c_char_p, P(i32), P(i32), P(C.c_double), P(C.c_double)],
            "xema_op_mod": [vp, vp, vp, vp, i32, i32, i32, vp],
            "xema_op_ln_modulate": [vp, i32, i64, vp, vp, vp, i64, i32, i32, i32, C.c_float, vp],
            "xema_op_rmsnorm_rope": [vp, i64, i64, vp, vp, i32, i32, i32, i32, i32, C.c_float, vp],
            "xema_op_gemm": [P(xema_gemm_args), vp, vp],
            "xema_op_attention": [vp, i64, i64, vp, vp, i64, i64, vp, vp, i32, i32, i32, i32, i32, C.c_float, vp, vp],
            "xema_last_cuda_error": [],
            "xema_selftest_wait_timeout": [vp, i64, vp, vp],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.xema_plan_destroy.argtypes = [vp]
        L.xema_plan_destroy.restype = None
        L.xema_strerror.argtypes = [C.c_int]
        L.xema_strerror.restype = C.c_char_p
        L.xema_plan_guard_bytes.restype = C.c_uint64
        L.xema_version.argtypes = []
        L.xema_version.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != XEMA_OK:
        raise XemaError(status, where)


def strerror(status: int) -> str:
    return lib().xema_strerror(status).decode()


def last_cuda_error() -> int:
    return lib().xema_last_cuda_error()


def version() -> str:
    return lib().xema_version().decode()


def make_config(t) -> xema_config:
    """xema_config from any object with the template's attribute names."""
    c = xema_config()
    for name, _ in xema_config._fields_:
        setattr(c, name, getattr(t, name))
    return c


def _tensor_dict(t: xema_tensor) -> dict:
    return {"name": t.name.decode(), "kind": t.kind, "dtype": t.dtype, "block": t.block, "chunk": t.chunk,
            "bytes": t.bytes, "birth": t.birth, "death": t.death}


def xema_trace(cfg: xema_config, chunks: int):
    """-> (list of tensor dicts in id order, n_ops)"""
    n, ops = C.c_size_t(0), C.c_uint32(0)
    rc = lib().xema_trace(C.byref(cfg), chunks, None, 0, C.byref(n), C.byref(ops))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_trace")
    arr = (xema_tensor * n.value)()
    _check(lib().xema_trace(C.byref(cfg), chunks, arr, n.value, C.byref(n), C.byref(ops)), "xema_trace")
    return [_tensor_dict(t) for t in arr], ops.value


def _triple(chunks):
    ca, cb, cc = (int(v) for v in chunks)
    return (C.c_int32 * 3)(ca, cb, cc)


def xema_trace_phases(cfg: xema_config, chunks):
    """chunks = (C_A, C_B, C_C) -> (list of tensor dicts in id order, n_ops)"""
    c3 = _triple(chunks)
    n, ops = C.c_size_t(0), C.c_uint32(0)
    rc = lib().xema_trace_phases(C.byref(cfg), c3, None, 0, C.byref(n), C.byref(ops))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_trace_phases")
    arr = (xema_tensor * n.value)()
    _check(lib().xema_trace_phases(C.byref(cfg), c3, arr, n.value, C.byref(n), C.byref(ops)), "xema_trace_phases")
    return [_tensor_dict(t) for t in arr], ops.value


def xema_phase_chunks_for_budget(cfg: xema_config, budget_bytes: int, max_chunks: int):
    """-> ((C_A, C_B, C_C), peak_bytes); the triple is None when nothing fits."""
    c3, peak = (C.c_int32 * 3)(), C.c_uint64(0)
    rc = lib().xema_phase_chunks_for_budget(C.byref(cfg), budget_bytes, max_chunks, c3, C.byref(peak))
    if rc == XEMA_EBUDGET:
        return None, peak.value
    _check(rc, "xema_phase_chunks_for_budget")
    return tuple(c3), peak.value


def _mitigation(chunks, axes):
    m = xema_mitigation()
    for i in range(3):
        m.chunks[i], m.axis[i] = int(chunks[i]), int(axes[i])
    return m


def xema_trace_mitigated(cfg: xema_config, chunks, axes):
    """chunks = (C_A, C_B, C_C), axes = per-phase SPLIT_ROWS / SPLIT_BATCH -> (tensor dicts, n_ops)"""
    m = _mitigation(chunks, axes)
    n, ops = C.c_size_t(0), C.c_uint32(0)
    rc = lib().xema_trace_mitigated(C.byref(cfg), C.byref(m), None, 0, C.byref(n), C.byref(ops))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_trace_mitigated")
    arr = (xema_tensor * n.value)()
    _check(lib().xema_trace_mitigated(C.byref(cfg), C.byref(m), arr, n.value, C.byref(n), C.byref(ops)),
           "xema_trace_mitigated")
    return [_tensor_dict(t) for t in arr], ops.value


def xema_trace_sharded(cfg: xema_config, chunks, axes, shard: int, shards: int):
    """The trace of sequence-parallel shard `shard` of `shards` -> (tensor dicts, n_ops)"""
    c3 = (chunks,) * 3 if isinstance(chunks, int) else chunks
    m = _mitigation(c3, axes or (SPLIT_ROWS,) * 3)
    n, ops = C.c_size_t(0), C.c_uint32(0)
    rc = lib().xema_trace_sharded(C.byref(cfg), C.byref(m), shard, shards, None, 0, C.byref(n), C.byref(ops))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_trace_sharded")
    arr = (xema_tensor * n.value)()
    _check(lib().xema_trace_sharded(C.byref(cfg), C.byref(m), shard, shards, arr, n.value, C.byref(n), C.byref(ops)),
           "xema_trace_sharded")
    return [_tensor_dict(t) for t in arr], ops.value


def xema_shard_rows(cfg: xema_config, shard: int, shards: int):
    """-> (first row, rows) owned by the shard"""
    r0, n = C.c_int64(0), C.c_int64(0)
    _check(lib().xema_shard_rows(C.byref(cfg), shard, shards, C.byref(r0), C.byref(n)), "xema_shard_rows")
    return r0.value, n.value


def xema_mitigation_for_budget(cfg: xema_config, budget_bytes: int, max_chunks: int):
    """-> ((C_A, C_B, C_C), axes, peak_bytes); counts and axes are None when nothing fits."""
    m, peak = xema_mitigation(), C.c_uint64(0)
    rc = lib().xema_mitigation_for_budget(C.byref(cfg), budget_bytes, max_chunks, C.byref(m), C.byref(peak))
    if rc == XEMA_EBUDGET:
        return None, None, peak.value
    _check(rc, "xema_mitigation_for_budget")
    return tuple(m.chunks), tuple(m.axis), peak.value


def xema_pressure_ranges(tensors: Sequence[dict], n_ops: int, budget_bytes: int):
    """-> list of half-open op ranges (first, end) where the live bytes exceed the budget"""
    n = len(tensors)
    arr = (xema_tensor * max(n, 1))()
    for i, d in enumerate(tensors):
        arr[i].bytes, arr[i].birth, arr[i].death = d["bytes"], d["birth"], d["death"]
    cnt = C.c_size_t(0)
    rc = lib().xema_pressure_ranges(arr, n, n_ops, budget_bytes, None, 0, C.byref(cnt))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_pressure_ranges")
    if cnt.value == 0:
        return []
    out = (C.c_uint32 * (2 * cnt.value))()
    _check(lib().xema_pressure_ranges(arr, n, n_ops, budget_bytes, out, cnt.value, C.byref(cnt)), "xema_pressure_ranges")
    return [(out[2 * i], out[2 * i + 1]) for i in range(cnt.value)]


def xema_plan_arena(tensors: Sequence[dict]):
    """tensors: dicts with bytes, birth, death -> (offsets, peak_bytes, max_live_bytes)"""
    n = len(tensors)
    arr = (xema_tensor * max(n, 1))()
    for i, d in enumerate(tensors):
        arr[i].bytes, arr[i].birth, arr[i].death = d["bytes"], d["birth"], d["death"]
    offs = (C.c_uint64 * max(n, 1))()
    peak, live = C.c_uint64(0), C.c_uint64(0)
    _check(lib().xema_plan_arena(arr, n, offs, C.byref(peak), C.byref(live)), "xema_plan_arena")
    return list(offs[:n]), peak.value, live.value


def xema_chunks_for_budget(cfg: xema_config, budget_bytes: int, max_chunks: int):
    """-> (chunks, peak_bytes); chunks is None when nothing fits (peak = smallest seen)."""
    ch, peak = C.c_int32(0), C.c_uint64(0)
    rc = lib().xema_chunks_for_budget(C.byref(cfg), budget_bytes, max_chunks, C.byref(ch), C.byref(peak))
    if rc == XEMA_EBUDGET:
        return None, peak.value
    _check(rc, "xema_chunks_for_budget")
    return ch.value, peak.value


def xema_pluggable_mode(mode: int):
    _check(lib().xema_pluggable_mode(mode), "xema_pluggable_mode")


def xema_pluggable_recorded():
    """-> (list of tensor dicts in request order, n_events)"""
    n, ev = C.c_size_t(0), C.c_uint32(0)
    rc = lib().xema_pluggable_recorded(None, 0, C.byref(n), C.byref(ev))
    if rc != XEMA_ENOSPC:
        _check(rc, "xema_pluggable_recorded")
    if n.value == 0:
        return [], ev.value
    arr = (xema_tensor * n.value)()
    _check(lib().xema_pluggable_recorded(arr, n.value, C.byref(n), C.byref(ev)), "xema_pluggable_recorded")
    return [_tensor_dict(t) for t in arr], ev.value


def xema_pluggable_set_plan(arena_ptr: int, arena_bytes: int, offsets: Sequence[int]):
    offs = (C.c_uint64 * max(len(offsets), 1))(*offsets)
    _check(lib().xema_pluggable_set_plan(arena_ptr, arena_bytes, offs, len(offsets)), "xema_pluggable_set_plan")


def xema_pluggable_step_begin():
    _check(lib().xema_pluggable_step_begin(), "xema_pluggable_step_begin")


def xema_pluggable_stats():
    """-> (served from the arena, fell back to cudaMalloc, index of the next request)"""
    a, b, c = C.c_uint64(0), C.c_uint64(0), C.c_uint64(0)
    _check(lib().xema_pluggable_stats(C.byref(a), C.byref(b), C.byref(c)), "xema_pluggable_stats")
    return a.value, b.value, c.value


def xema_rope_table(cfg: xema_config) -> np.ndarray:
    S = cfg.s_text + cfg.grid_t * cfg.grid_h * cfg.grid_w
    out = np.empty((S, cfg.head_dim // 2, 2), dtype=np.float32)
    _check(lib().xema_rope_table(C.byref(cfg), out.ctypes.data_as(C.c_void_p)), "xema_rope_table")
    return out


class Plan:
    """Owner of an xema_plan handle."""

    def __init__(self, cfg: xema_config, chunks, axes=None, shard=None, guard_bytes: int = 0):
        """chunks: one count (xema_plan_create) or a per-phase triple (xema_plan_create_phases);
        with `axes` (per-phase SPLIT_ROWS / SPLIT_BATCH) xema_plan_create_mitigated; with
        `shard` = (p, P) xema_plan_create_sharded (the plan of one sequence-parallel shard); with
        `guard_bytes` xema_plan_create_guarded (debug layout with a guard band after every tensor)."""
        self.cfg = cfg
        self._h = C.c_void_p()
        self.guard_bytes = int(guard_bytes)
        if guard_bytes:
            c3 = (chunks,) * 3 if isinstance(chunks, int) else chunks
            m = _mitigation(c3, axes or (SPLIT_ROWS,) * 3)
            sh = shard or (0, 1)
            _check(lib().xema_plan_create_guarded(C.byref(cfg), C.byref(m), sh[0], sh[1], guard_bytes, C.byref(self._h)),
                   "xema_plan_create_guarded")
        elif shard is not None:
            c3 = (chunks,) * 3 if isinstance(chunks, int) else chunks
            m = _mitigation(c3, axes or (SPLIT_ROWS,) * 3)
            _check(lib().xema_plan_create_sharded(C.byref(cfg), C.byref(m), shard[0], shard[1], C.byref(self._h)),
                   "xema_plan_create_sharded")
        elif axes is not None:
            c3 = (chunks,) * 3 if isinstance(chunks, int) else chunks
            _check(lib().xema_plan_create_mitigated(C.byref(cfg), C.byref(_mitigation(c3, axes)), C.byref(self._h)),
                   "xema_plan_create_mitigated")
        elif isinstance(chunks, int):
            _check(lib().xema_plan_create(C.byref(cfg), chunks, C.byref(self._h)), "xema_plan_create")
        else:
            _check(lib().xema_plan_create_phases(C.byref(cfg), _triple(chunks), C.byref(self._h)),
                   "xema_plan_create_phases")
        peak, live, n, ops, ch = C.c_uint64(), C.c_uint64(), C.c_size_t(), C.c_uint32(), C.c_int32()
        _check(lib().xema_plan_info(self._h, C.byref(peak), C.byref(live), C.byref(n), C.byref(ops), C.byref(ch)),
               "xema_plan_info")
        self.peak_bytes, self.max_live_bytes = peak.value, live.value
        self.n_tensors, self.n_ops, self.chunks = n.value, ops.value, ch.value
        c3 = (C.c_int32 * 3)()
        _check(lib().xema_plan_phase_chunks(self._h, c3), "xema_plan_phase_chunks")
        self.phase_chunks = tuple(c3)
        m = xema_mitigation()
        _check(lib().xema_plan_mitigation(self._h, C.byref(m)), "xema_plan_mitigation")
        self.axes = tuple(m.axis)
        p_, P_, r0, n = C.c_int32(), C.c_int32(), C.c_int64(), C.c_int64()
        _check(lib().xema_plan_shard(self._h, C.byref(p_), C.byref(P_), C.byref(r0), C.byref(n)), "xema_plan_shard")
        self.shard, self.row0, self.rows = (p_.value, P_.value), r0.value, n.value
        self._keep = None

    def gather_point(self, block: int):
        """-> (index of the first op that needs every shard's keys and values of `block`,
        arena offset of its kv tensor [B, S, 2D])"""
        op, off = C.c_uint32(), C.c_uint64()
        _check(lib().xema_plan_gather_point(self._h, block, C.byref(op), C.byref(off)), "xema_plan_gather_point")
        return op.value, off.value

    def close(self):
        if self._h:
            lib().xema_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def tensor(self, name: str):
        off, nbytes = C.c_uint64(), C.c_uint64()
        _check(lib().xema_plan_tensor(self._h, name.encode(), C.byref(off), C.byref(nbytes)), "xema_plan_tensor")
        return off.value, nbytes.value

    def tensors(self):
        out = []
        for i in range(self.n_tensors):
            t, off = xema_tensor(), C.c_uint64()
            _check(lib().xema_plan_tensor_at(self._h, i, C.byref(t), C.byref(off)), "xema_plan_tensor_at")
            d = _tensor_dict(t)
            d["offset"] = off.value
            out.append(d)
        return out

    def bind(self, arena_ptr: int, arena_bytes: int, weights: Sequence[dict], rope_ptr: int,
             status_ptr: Optional[int] = None):
        """weights: one dict per block mapping the twelve parameter names to device pointers."""
        arr = (xema_block_weights * len(weights))()
        for i, w in enumerate(weights):
            for f in _WEIGHT_FIELDS:
                setattr(arr[i], f, w[f])
        _check(lib().xema_plan_bind(self._h, arena_ptr, arena_bytes, arr, rope_ptr, status_ptr), "xema_plan_bind")
        self._keep = arr

    def launch_count(self) -> int:
        return lib().xema_plan_launch_count(self._h)

    def block_forward(self, stream: int = 0):
        _check(lib().xema_block_forward(self._h, stream), "xema_block_forward")

    def step_forward(self, stream: int = 0):
        _check(lib().xema_step_forward(self._h, stream), "xema_step_forward")

    def forward_host(self, hid_in_host: int, temb_host: int, hid_out_host: int, stream: int = 0):
        """Host pointers in and out; both copies and the forward are enqueued on `stream`."""
        _check(lib().xema_forward_host(self._h, hid_in_host, temb_host, hid_out_host, stream), "xema_forward_host")

    def forward_range(self, first_op: int, end_op: int, stream: int = 0):
        _check(lib().xema_forward_range(self._h, first_op, end_op, stream), "xema_forward_range")

    def op(self, i: int) -> dict:
        name = C.create_string_buffer(8)
        blk, ch, fl, by = C.c_int32(), C.c_int32(), C.c_double(), C.c_double()
        _check(lib().xema_plan_op(self._h, i, name, C.byref(blk), C.byref(ch), C.byref(fl), C.byref(by)),
               "xema_plan_op")
        return {"name": name.value.decode(), "block": blk.value, "chunk": ch.value, "flops": fl.value,
                "bytes": by.value}

    def forward_prefix(self, n_logical_ops: int, stream: int = 0):
        _check(lib().xema_forward_prefix(self._h, n_logical_ops, stream), "xema_forward_prefix")


DEVICE_STATUS_TIMEOUT = 0x54310001


def xema_selftest_wait_timeout(status: int, limit_cycles: int, waited_cycles: Optional[int] = None, stream: int = 0):
    _check(lib().xema_selftest_wait_timeout(status, limit_cycles, waited_cycles, stream),
           "xema_selftest_wait_timeout")


STATIC_ARENA_BYTES = 4 << 20


def xema_block_forward_static(cfg: xema_config, chunks: int, weights: dict, rope_ptr: int, hid_in: int, temb: int,
                              hid_out: int, status: Optional[int] = None, stream: int = 0):
    """One block whose intermediates live in the library's fixed scratch array; for callers
    that may not allocate device memory.  weights maps the twelve parameter names to device
    pointers; the other arguments are device pointers.  Raises XemaError(XEMA_ENOSPC) when the
    template needs more than STATIC_ARENA_BYTES."""
    w = xema_block_weights()
    for f in _WEIGHT_FIELDS:
        setattr(w, f, weights[f])
    _check(lib().xema_block_forward_static(C.byref(cfg), chunks, C.byref(w), rope_ptr, hid_in, temb, hid_out,
                                           status, stream), "xema_block_forward_static")


def xema_op_mod(temb, w_mod, b_mod, mod, batch, temb_dim, n_out, stream=0):
    _check(lib().xema_op_mod(temb, w_mod, b_mod, mod, batch, temb_dim, n_out, stream), "xema_op_mod")


def xema_op_ln_modulate(inp, in_is_f32, in_batch_rows, out, shift, scale, mod_stride, batch, rows, D, eps, stream=0):
    _check(lib().xema_op_ln_modulate(inp, in_is_f32, in_batch_rows, out, shift, scale, mod_stride, batch, rows, D,
                                     eps, stream), "xema_op_ln_modulate")


def xema_op_rmsnorm_rope(x, ld, batch_rows, g, rope, pos0, batch, rows, heads, head_dim, eps, stream=0):
    _check(lib().xema_op_rmsnorm_rope(x, ld, batch_rows, g, rope, pos0, batch, rows, heads, head_dim, eps, stream),
           "xema_op_rmsnorm_rope")


def xema_op_gemm(status=None, stream=0, **kw):
    a = xema_gemm_args()
    for k, v in kw.items():
        setattr(a, k, v)
    _check(lib().xema_op_gemm(C.byref(a), status, stream), "xema_op_gemm")


def exponent_scale(head_dim: int) -> float:
    """log2(e) / sqrt(head_dim) as the float32 the library uses: q k^T times this = exponents to base 2."""
    import numpy as np
    return float(np.float32(1.4426950408889634) / np.sqrt(np.float32(head_dim)))


def xema_op_attention(q, ldq, q_batch_rows, k, v, ldkv, kv_batch_rows, o, lse, batch, rows, keys, heads, head_dim,
                      status=None, stream=0, q_scale=None):
    """q_scale: None for a plain q (log2(e) / sqrt(head_dim) is passed), 1.0 for a q that was
    already multiplied by exponent_scale(head_dim)."""
    if q_scale is None:
        q_scale = exponent_scale(head_dim)
    _check(lib().xema_op_attention(q, ldq, q_batch_rows, k, v, ldkv, kv_batch_rows, o, lse, batch, rows, keys, heads,
                                   head_dim, q_scale, status, stream), "xema_op_attention")
