"""Thin ctypes binding over the C-ABI library (include/emo.h): argument marshalling only.

Function names and argument order follow the header.  Device buffers are torch tensors (or raw
integer addresses); torch is used for device memory and streams, never for the computation.
Loading fails loudly when the CUDA library has not been built: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libemo_b200.so")

EMO_OK = 0
EMO_E_INVALID_ARG, EMO_E_NOT_TOPOLOGICAL, EMO_E_RANGE, EMO_E_OVERFLOW = -1, -2, -3, -4
EMO_E_NONFINITE, EMO_E_OOM, EMO_E_CUDA, EMO_E_TIMEOUT, EMO_E_UNSUPPORTED = -5, -6, -7, -8, -9
EMO_F_HOST_ONLY = 0x1
EMO_F_VALIDATE = 0x1
EMO_F_NO_STAGING = 0x2
EMO_F_PAIR_KERNEL = 0x4
EMO_F_LANE_KERNEL = 0x8
EMO_F_FLOW_KERNEL = 0x10
EMO_F_SPINE_KERNEL = 0x20
EMO_F_GENERIC = 0x4        # load flag (shares its value with the call flag EMO_F_PAIR_KERNEL)
EMO_F_INTERVALS = 0x2      # load flag (shares its value with the call flag EMO_F_NO_STAGING)
EMO_F_TEST_STALL = 0x100

EXPORTS = [
    "emo_strerror", "emo_graph_load", "emo_graph_free", "emo_graph_info", "emo_workspace_bytes",
    "emo_eval_policies", "emo_slack_batch", "emo_slack", "emo_baseline", "emo_target_from_delta",
    "emo_select", "emo_transpose_policies", "emo_slack_batch_host", "emo_graph_program",
    "emo_set_pass_events", "emo_select_static", "emo_graph_flow", "emo_graph_spine", "emo_graph_spine_view", "emo_set_wait_limit", "emo_call_path", "emo_set_flow_counters", "emo_workspace_bytes_for", "emo_measure_int_issue", "emo_measure_warp_costs", "emo_eval_intervals", "emo_workspace_bytes_intervals", "emo_search_dp", "emo_workspace_bytes_search", "emo_pack_greedy", "emo_pack_tables", "emo_pack_model", "emo_pack_classes", "emo_pack_levels", "emo_unpack_levels", "emo_slack_batch_host_packed", "emo_levels_prefetch", "emo_slack_batch_prefetched",
]


def EMO_F_LANES(c: int) -> int:
    return (c & 0xFF) << 8


def EMO_F_LOOKAHEAD(d: int) -> int:
    return (d & 0xFF) << 16


def EMO_F_FLOW_SYNC(s: int) -> int:
    return ((s // 8) & 0xF) << 4


def EMO_F_SPINE_STAGE(k: int) -> int:
    return (1 if k == 8 else (3 if k == 32 else 2)) << 30


def EMO_F_FLOW_STAGE(k: int) -> int:
    return (k & 0x3F) << 24


class EmoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class emo_info(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("m", ctypes.c_int64), ("L", ctypes.c_int32), ("rows", ctypes.c_int32),
                ("depth", ctypes.c_int32), ("max_span", ctypes.c_int32), ("T_worst", ctypes.c_int64),
                ("T_best", ctypes.c_int64), ("lanes", ctypes.c_int32),
                ("steps_fwd", ctypes.c_int32), ("slots_fwd", ctypes.c_int32), ("aux_fwd", ctypes.c_int32),
                ("steps_bwd", ctypes.c_int32), ("slots_bwd", ctypes.c_int32), ("aux_bwd", ctypes.c_int32),
                ("lanes_bwd", ctypes.c_int32), ("sync_fwd", ctypes.c_int32), ("sync_bwd", ctypes.c_int32)]


class emo_flow_view(ctypes.Structure):
    _fields_ = ([(k, ctypes.c_int32) for k in ("ok32", "lanes", "K", "sync", "stages", "steps", "Lp", "slots_tag_fwd",
                                                "slots_set_fwd", "pool_stride_fwd", "slots_tag_bwd", "slots_set_bwd",
                                                "pool_stride_bwd")] +
                [(k, ctypes.c_int64) for k in ("pushes", "pruned_fwd", "pruned_bwd")] +
                [(k, ctypes.c_void_p) for k in ("hdr", "rows", "node", "step", "tab_fwd", "tab_bwd", "rec_fwd", "pool_fwd",
                                                "rec_bwd", "pool_bwd", "seg_fwd", "seg_bwd", "lbes", "push_base")])


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_12324_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        p, i32, i64, u32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_size_t
        L.emo_strerror.argtypes = [ctypes.c_int]
        L.emo_strerror.restype = ctypes.c_char_p
        L.emo_graph_load.argtypes = [i32, p, p, p, i32, i32, p, p, p, u32, ctypes.POINTER(p)]
        L.emo_graph_free.argtypes = [p]
        L.emo_graph_info.argtypes = [p, ctypes.POINTER(emo_info)]
        L.emo_workspace_bytes.argtypes = [p, i64, ctypes.c_int, ctypes.POINTER(sz)]
        L.emo_workspace_bytes_for.argtypes = [p, i64, ctypes.c_int, u32, ctypes.c_int, ctypes.POINTER(sz)]
        L.emo_eval_policies.argtypes = [p, i64, p, i64, p, p, p, p, p, sz, p, u32, p]
        L.emo_slack_batch.argtypes = [p, i64, p, i64, p, p, p, i64, p, p, p, p, p, p, p, sz, p, u32, p]
        L.emo_slack.argtypes = [p, p, p, p, p, p, p, p, sz, p, p]
        L.emo_baseline.argtypes = [p, p, p, p, sz, p, p]
        L.emo_target_from_delta.argtypes = [i64, i64]
        L.emo_target_from_delta.restype = i64
        L.emo_select.argtypes = [i64, p, p, i64, p, i64, p, p, p, p, sz, p]
        L.emo_transpose_policies.argtypes = [i64, i64, p, i64, p, i64, p]
        L.emo_slack_batch_host.argtypes = [p, i64, p, i64, p, p, i64, i64, p, p, p, p, p, p, sz, u32, p]
        L.emo_graph_program.argtypes = [p, ctypes.c_int, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                        ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(p),
                                        ctypes.POINTER(p), ctypes.POINTER(p)]
        L.emo_set_pass_events.argtypes = [p, p, p, p]
        L.emo_graph_flow.argtypes = [p, ctypes.POINTER(emo_flow_view)]
        L.emo_graph_spine.argtypes = [p, ctypes.POINTER(ctypes.c_int64)]
        L.emo_graph_spine_view.argtypes = [p, ctypes.POINTER(emo_spine_view)]
        L.emo_set_wait_limit.argtypes = [i64]
        L.emo_set_flow_counters.argtypes = [p]
        L.emo_measure_int_issue.argtypes = [p, p, p]
        L.emo_measure_warp_costs.argtypes = [p, p, p]
        L.emo_eval_intervals.argtypes = [p, i64, p, i64, i32, p, p, p, p, p, p, ctypes.c_size_t, p, u32, p]
        L.emo_workspace_bytes_intervals.argtypes = [p, i64, i32, ctypes.c_int, p]
        L.emo_search_dp.argtypes = [p, i32, p, p, i64, i64, i64, p, p, p, p, p, p, ctypes.c_size_t, p]
        L.emo_workspace_bytes_search.argtypes = [p, i32, i64, ctypes.c_int, p]
        L.emo_pack_greedy.argtypes = [i32, p, p, p, p, p, i64, p, p, p]
        L.emo_pack_tables.argtypes = [i32, i32, p, p, p, i32, p, p]
        L.emo_pack_model.argtypes = [i32, i32, i32, i32, p, p, p, p, p, p, p, p, p]
        L.emo_pack_classes.argtypes = [i32, p, p, i32, p, p]
        L.emo_pack_levels.argtypes = [ctypes.c_int, i64, i64, p, i64, p, i64, p]
        L.emo_unpack_levels.argtypes = [ctypes.c_int, i64, i64, p, i64, p, i64, p]
        L.emo_slack_batch_host_packed.argtypes = [p, i64, ctypes.c_int, p, i64, p, p, i64, p, i64, i64, p, p, p, p, p, p, sz, u32, p]
        L.emo_levels_prefetch.argtypes = [p, p, i64, p, p, p]
        L.emo_slack_batch_prefetched.argtypes = [p, i64, ctypes.c_int, p, i64, p, p, i64, p, i64, i64, p, p, p, p, p, p, sz, u32, p]
        L.emo_call_path.argtypes = [p, i64, p, i64, i64, ctypes.c_int, u32]
        L.emo_select_static.argtypes = [i64, p, p, i64, p, i64, p, p, p, p]
        for name in EXPORTS:
            if name not in ("emo_strerror", "emo_target_from_delta"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().emo_strerror(int(code)).decode()


def _addr(x) -> Optional[int]:
    """Address of a torch tensor, numpy array, int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return int(x.data_ptr())


def _check(rc: int, where: str):
    if rc != EMO_OK:
        raise EmoError(rc, where)


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream) or None
    if isinstance(stream, int):
        return stream or None
    return int(stream.cuda_stream) or None


class Graph:
    """Owner of an emo_graph handle."""

    def __init__(self, handle: int):
        self.handle = handle

    def free(self):
        if self.handle:
            lib().emo_graph_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    @property
    def info(self) -> emo_info:
        return emo_graph_info(self)


def emo_graph_load(n, row_ptr, col, level_ptr, L, lat, energy, group_of=None, flags: int = 0) -> Graph:
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int64)
    col = np.ascontiguousarray(col, dtype=np.int32)
    lat = np.ascontiguousarray(lat, dtype=np.int64)
    energy = np.ascontiguousarray(energy, dtype=np.float64)
    lp = None if level_ptr is None else np.ascontiguousarray(level_ptr, dtype=np.int32)
    go = None if group_of is None else np.ascontiguousarray(group_of, dtype=np.int32)
    out = ctypes.c_void_p()
    rc = lib().emo_graph_load(int(n), _addr(row_ptr), _addr(col), _addr(lp), 0 if lp is None else len(lp) - 1,
                              int(L), _addr(lat), _addr(energy), _addr(go), int(flags), ctypes.byref(out))
    _check(rc, "emo_graph_load")
    return Graph(out.value)


def load_workload(g, flags: int = 0, group_of=None, with_levels: bool = True) -> Graph:
    """emo_graph_load on a workloads.Graph."""
    return emo_graph_load(g.n, g.row_ptr, g.col, g.level_ptr if with_levels and len(g.level_ptr) > 2 else None,
                          g.L, g.lat, g.energy, group_of, flags)


def emo_graph_info(g: Graph) -> emo_info:
    info = emo_info()
    _check(lib().emo_graph_info(g.handle, ctypes.byref(info)), "emo_graph_info")
    return info


def emo_workspace_bytes(g: Graph, B: int, need_slack: int = 0, flags: int = 0, aligned: bool = True) -> int:
    """Workspace a call on B policies needs; flags / aligned as in emo_workspace_bytes_for."""
    out = ctypes.c_size_t()
    _check(lib().emo_workspace_bytes_for(g.handle, int(B), int(need_slack), int(flags), int(bool(aligned)),
                                         ctypes.byref(out)), "emo_workspace_bytes_for")
    return int(out.value)


def _nbytes(ws) -> int:
    return 0 if ws is None else int(ws.numel() * ws.element_size())


def emo_eval_policies(g: Graph, B, lvl, ldb, makespan, energy, ws=None, status=None, flags=0, stream=None,
                      T0=None, E0=None):
    _check(lib().emo_eval_policies(g.handle, int(B), _addr(lvl), int(ldb), _addr(makespan), _addr(energy),
                                   _addr(T0), _addr(E0), _addr(ws), _nbytes(ws), _addr(status), int(flags),
                                   _stream(stream)),
           "emo_eval_policies")


def emo_slack_batch(g: Graph, B, lvl, ldb, ES, LS, slack, ldo, makespan, energy, slack_sum=None,
                    n_critical=None, ws=None, status=None, flags=0, stream=None, T0=None, E0=None):
    _check(lib().emo_slack_batch(g.handle, int(B), _addr(lvl), int(ldb), _addr(ES), _addr(LS), _addr(slack),
                                 int(ldo), _addr(makespan), _addr(energy), _addr(slack_sum), _addr(n_critical),
                                 _addr(T0), _addr(E0), _addr(ws), _nbytes(ws), _addr(status), int(flags),
                                 _stream(stream)),
           "emo_slack_batch")


def emo_slack(g: Graph, lvl_one, ES, LS, slack, makespan, energy=None, ws=None, status=None, stream=None):
    _check(lib().emo_slack(g.handle, _addr(lvl_one), _addr(ES), _addr(LS), _addr(slack), _addr(makespan),
                           _addr(energy), _addr(ws), _nbytes(ws), _addr(status), _stream(stream)), "emo_slack")


def emo_baseline(g: Graph, T0, E0, ws, status=None, stream=None):
    _check(lib().emo_baseline(g.handle, _addr(T0), _addr(E0), _addr(ws), _nbytes(ws), _addr(status),
                              _stream(stream)), "emo_baseline")


def emo_target_from_delta(T0: int, delta_ppm: int) -> int:
    return int(lib().emo_target_from_delta(int(T0), int(delta_ppm)))


def emo_select(B, makespan, energy, target, out_index, out_T=None, out_E=None, ws=None, target_dev=None,
               delta_ppm: int = 0, stream=None):
    _check(lib().emo_select(int(B), _addr(makespan), _addr(energy), int(target), _addr(target_dev),
                            int(delta_ppm), _addr(out_index), _addr(out_T), _addr(out_E), _addr(ws),
                            _nbytes(ws), _stream(stream)), "emo_select")


EMO_SELECT_STATIC_MAX_B = 1048576


def emo_select_static(B, makespan, energy, target, out_index, out_T=None, out_E=None, target_dev=None,
                      delta_ppm: int = 0, stream=None):
    """emo_select without a workspace: the per-block candidates live in a fixed array inside the
    library, for callers that may not allocate device memory.  At most EMO_SELECT_STATIC_MAX_B
    policies; calls on one device must not overlap."""
    _check(lib().emo_select_static(int(B), _addr(makespan), _addr(energy), int(target), _addr(target_dev),
                                   int(delta_ppm), _addr(out_index), _addr(out_T), _addr(out_E), _stream(stream)),
           "emo_select_static")


def emo_transpose_policies(B, rows, src, lds, dst, ldb, stream=None):
    _check(lib().emo_transpose_policies(int(B), int(rows), _addr(src), int(lds), _addr(dst), int(ldb),
                                        _stream(stream)), "emo_transpose_policies")


def emo_slack_batch_host(g: Graph, B, lvl_host, ldb, dev_lvl, slack_dev, ldo, delta_ppm, makespan_host,
                         energy_host, slack_sum_host, n_critical_host, sel_host, ws, flags=0, stream=None):
    _check(lib().emo_slack_batch_host(g.handle, int(B), _addr(lvl_host), int(ldb), _addr(dev_lvl),
                                      _addr(slack_dev), int(ldo), int(delta_ppm), _addr(makespan_host),
                                      _addr(energy_host), _addr(slack_sum_host), _addr(n_critical_host),
                                      _addr(sel_host), _addr(ws), _nbytes(ws), int(flags), _stream(stream)),
           "emo_slack_batch_host")


def emo_set_pass_events(fwd_start=None, fwd_stop=None, bwd_start=None, bwd_stop=None):
    """Events are torch.cuda.Event objects created with enable_timing=True (or None)."""
    def h(ev):
        if ev is None:
            return None
        if not ev.cuda_event:          # torch creates the handle lazily, on the first record
            ev.record()
        return int(ev.cuda_event)
    _check(lib().emo_set_pass_events(h(fwd_start), h(fwd_stop), h(bwd_start), h(bwd_stop)), "emo_set_pass_events")


def emo_graph_program(g: Graph, direction: int):
    """(lanes, steps, slots, Lp, entries[steps][lanes][8], rows[steps][lanes], lat[steps*lanes][Lp]), all
    uint32 numpy copies of the compiled program (host-side inspection)."""
    lanes, steps, slots, Lp = (ctypes.c_int32() for _ in range(4))
    pe, pr, pl = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
    _check(lib().emo_graph_program(g.handle, int(direction), ctypes.byref(lanes), ctypes.byref(steps),
                                   ctypes.byref(slots), ctypes.byref(Lp), ctypes.byref(pe), ctypes.byref(pr),
                                   ctypes.byref(pl)), "emo_graph_program")
    q = steps.value * lanes.value
    if q == 0:
        return lanes.value, 0, slots.value, Lp.value, np.zeros((0, max(lanes.value, 1), 8), np.uint32), \
            np.zeros((0, max(lanes.value, 1)), np.uint32), np.zeros((0, Lp.value), np.uint32)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    ent = np.ctypeslib.as_array(ctypes.cast(pe, u32p), shape=(q * 8,)).copy()
    rows = np.ctypeslib.as_array(ctypes.cast(pr, u32p), shape=(q,)).copy()
    lat = np.ctypeslib.as_array(ctypes.cast(pl, u32p), shape=(q * Lp.value,)).copy()
    return lanes.value, steps.value, slots.value, Lp.value, ent.reshape(steps.value, lanes.value, 8), \
        rows.reshape(steps.value, lanes.value), lat.reshape(q, Lp.value)


def emo_graph_spine(g: Graph) -> dict:
    """Sizes of the spine program (see emo.h)."""
    out = (ctypes.c_int64 * 12)()
    _check(lib().emo_graph_spine(g.handle, out), "emo_graph_spine")
    keys = ("ok", "lanes", "K", "stages", "segments", "ops_fwd", "ops_bwd", "slots_fwd", "slots_bwd", "max_segs", "acc_words", "pushes")
    return dict(zip(keys, [int(x) for x in out]))


class emo_spine_view(ctypes.Structure):
    _fields_ = ([(k, ctypes.c_int32) for k in ("ok", "lanes", "K", "stages", "Lp", "max_ops_fwd", "max_ops_bwd", "max_pool",
                                               "acc_words", "slots_fwd", "slots_bwd")]
                + [("pushes", ctypes.c_int64)]
                + [(k, ctypes.c_void_p) for k in ("n_ops_fwd", "ops_fwd", "n_ops_bwd", "ops_bwd", "mem", "pos", "rows", "tab_fwd",
                                                  "tab_bwd", "pool", "push_base")])


def emo_graph_spine_view(g: Graph) -> dict:
    """The spine program as numpy copies (host-side inspection; see emo.h for the layouts)."""
    v = emo_spine_view()
    _check(lib().emo_graph_spine_view(g.handle, ctypes.byref(v)), "emo_graph_spine_view")
    out = {k: getattr(v, k) for k, _ in emo_spine_view._fields_[:12]}
    if not v.ok:
        return out

    def arr(ptr, count, ctype, dtype):
        if count == 0:
            return np.zeros(0, dtype)
        return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ctype)), shape=(count,)).astype(dtype, copy=True)

    u32 = ctypes.c_uint32
    q = v.stages * v.lanes * v.K
    out["n_ops_fwd"] = arr(v.n_ops_fwd, v.stages, u32, np.uint32)
    out["n_ops_bwd"] = arr(v.n_ops_bwd, v.stages, u32, np.uint32)
    out["ops_fwd"] = arr(v.ops_fwd, v.stages * v.max_ops_fwd * 8, u32, np.uint32).reshape(v.stages, v.max_ops_fwd, 8)
    out["ops_bwd"] = arr(v.ops_bwd, v.stages * v.max_ops_bwd * 12, u32, np.uint32).reshape(v.stages, v.max_ops_bwd, 12)
    out["mem"] = arr(v.mem, q * 8, u32, np.uint32).reshape(v.stages, v.lanes * v.K, 8)
    out["pos"] = arr(v.pos, q, u32, np.uint32).reshape(v.stages, v.lanes * v.K)
    out["rows"] = arr(v.rows, q, u32, np.uint32).reshape(v.stages, v.lanes * v.K)
    out["tab_fwd"] = arr(v.tab_fwd, q * v.Lp * 3, u32, np.uint32).reshape(v.stages, v.lanes * v.K, v.Lp, 3)
    out["tab_bwd"] = arr(v.tab_bwd, q * v.Lp, u32, np.uint32).reshape(v.stages, v.lanes * v.K, v.Lp)
    out["pool"] = arr(v.pool, v.stages * v.max_pool, ctypes.c_uint64, np.uint64).reshape(v.stages, v.max_pool)
    out["push_base"] = arr(v.push_base, v.stages + 1, ctypes.c_int64, np.int64)
    return out


def emo_graph_flow(g: Graph, arrays: bool = True) -> dict:
    """The lane-stream program of the 32-bit pass kernels as numpy copies (host-side inspection);
    arrays=False gives the sizes only."""
    v = emo_flow_view()
    _check(lib().emo_graph_flow(g.handle, ctypes.byref(v)), "emo_graph_flow")
    out = {k: getattr(v, k) for k, _ in emo_flow_view._fields_[:16]}
    if not v.ok32 or not arrays:
        return out
    q = v.stages * v.lanes * v.K

    def arr(ptr, count, ctype, dtype):
        if count == 0:
            return np.zeros(0, dtype)
        return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ctype)), shape=(count,)).astype(dtype, copy=True)

    u32, i64 = ctypes.c_uint32, ctypes.c_int64
    out["hdr"] = arr(v.hdr, v.stages * v.lanes * 8, u32, np.uint32).reshape(v.stages, v.lanes, 8)
    for k in ("rows", "node", "step"):
        out[k] = arr(getattr(v, k), q, u32, np.uint32).reshape(v.stages, v.lanes, v.K)
    out["tab_fwd"] = arr(v.tab_fwd, q * v.Lp * 3, u32, np.uint32).reshape(v.stages, v.lanes, v.K, v.Lp, 3)
    out["tab_bwd"] = arr(v.tab_bwd, q * v.Lp, u32, np.uint32).reshape(v.stages, v.lanes, v.K, v.Lp)
    out["rec_fwd"] = arr(v.rec_fwd, q * 8, u32, np.uint32).reshape(v.stages, v.lanes, v.K, 8)
    out["rec_bwd"] = arr(v.rec_bwd, q * 16, u32, np.uint32).reshape(v.stages, v.lanes, v.K, 16)
    out["pool_fwd"] = arr(v.pool_fwd, v.stages * v.pool_stride_fwd, u32, np.uint32).reshape(v.stages, v.pool_stride_fwd)
    out["pool_bwd"] = arr(v.pool_bwd, v.stages * v.pool_stride_bwd, u32, np.uint32).reshape(v.stages, v.pool_stride_bwd)
    out["seg_fwd"] = arr(v.seg_fwd, v.stages * v.lanes * 40, ctypes.c_uint8, np.uint8).reshape(v.stages, v.lanes, 40)
    out["seg_bwd"] = arr(v.seg_bwd, v.stages * v.lanes * 40, ctypes.c_uint8, np.uint8).reshape(v.stages, v.lanes, 40)
    out["lbes"] = arr(v.lbes, q, i64, np.int64).reshape(v.stages, v.lanes, v.K)
    out["push_base"] = arr(v.push_base, v.stages + 1, i64, np.int64)
    return out


def emo_set_wait_limit(cycles: int):
    _check(lib().emo_set_wait_limit(int(cycles)), "emo_set_wait_limit")


def emo_call_path(g: Graph, B, lvl, ldb, ldo, need_slack: bool, flags: int = 0) -> int:
    """2 = 32-bit lane-stream kernels, 1 = staged 64-bit kernels, 0 = plain-load kernels."""
    rc = lib().emo_call_path(g.handle, int(B), _addr(lvl), int(ldb), int(ldo), int(bool(need_slack)), int(flags))
    if rc < 0:
        raise EmoError(rc, "emo_call_path")
    return rc


def emo_set_flow_counters(dev):
    _check(lib().emo_set_flow_counters(_addr(dev)), "emo_set_flow_counters")


def emo_measure_int_issue(scratch_dev, stream=None) -> dict:
    """Warp-level integer operations per second of this GPU: 32/64-bit add and max (see include/emo.h)."""
    out = (ctypes.c_double * 4)()
    _check(lib().emo_measure_int_issue(ctypes.cast(out, ctypes.c_void_p), _addr(scratch_dev), _stream(stream)),
           "emo_measure_int_issue")
    return {"add32": out[0], "max32": out[1], "add64": out[2], "max64": out[3]}


def emo_measure_warp_costs(scratch_dev, stream=None) -> dict:
    """Cycles one warp alone pays for the steps of the pass kernels (see include/emo.h)."""
    out = (ctypes.c_double * 8)()
    _check(lib().emo_measure_warp_costs(ctypes.cast(out, ctypes.c_void_p), _addr(scratch_dev), _stream(stream)),
           "emo_measure_warp_costs")
    names = ("add_dependent", "max_sub_dependent", "shared_load_dependent", "add_independent", "body_with_untaken_branch",
             "body_without_branch", "redux_add_dependent", "barrier_5_warps")
    return {k: out[i] for i, k in enumerate(names)}


def emo_workspace_bytes_intervals(g, B, I, with_idle=True) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().emo_workspace_bytes_intervals(g.handle, int(B), int(I), int(bool(with_idle)), ctypes.byref(out)),
           "emo_workspace_bytes_intervals")
    return int(out.value)


def emo_eval_intervals(g, B, F, ldb, I, breaks, p_idle, makespan, energy, energy_idle, ws, status=None, flags=0, stream=None):
    """breaks: host int64 numpy array [I]; everything else device tensors (see include/emo.h)."""
    brk = np.ascontiguousarray(breaks, dtype=np.int64)
    if brk.shape != (int(I),):
        raise ValueError("breaks must hold I change points")
    return _check(lib().emo_eval_intervals(g.handle, int(B), _addr(F), int(ldb), int(I), brk.ctypes.data_as(ctypes.c_void_p),
                                           _addr(p_idle), _addr(makespan), _addr(energy), _addr(energy_idle), _addr(ws),
                                           _nbytes(ws), _addr(status), int(flags), _stream(stream)), "emo_eval_intervals")


def emo_workspace_bytes_search(g, I, max_batch=0, with_idle=True) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().emo_workspace_bytes_search(g.handle, int(I), int(max_batch), int(bool(with_idle)), ctypes.byref(out)),
           "emo_workspace_bytes_search")
    return int(out.value)


def emo_search_dp(g, breaks, p_idle, T_max, bin_ns, ws, max_batch=0, stream=None) -> dict:
    """Alg. 2 on the GPU evaluator (see include/emo.h).  breaks: host int64 [I]; p_idle: device tensor or None."""
    brk = np.ascontiguousarray(breaks, dtype=np.int64)
    I = int(brk.shape[0])
    F = np.zeros(I, np.uint8)
    T, E, calls, found = ctypes.c_int64(0), ctypes.c_double(0.0), ctypes.c_int64(0), ctypes.c_int32(0)
    _check(lib().emo_search_dp(g.handle, I, brk.ctypes.data_as(ctypes.c_void_p), _addr(p_idle), int(T_max), int(bin_ns), int(max_batch),
                               F.ctypes.data_as(ctypes.c_void_p), ctypes.byref(T), ctypes.byref(E), ctypes.byref(calls),
                               ctypes.byref(found), _addr(ws), _nbytes(ws), _stream(stream)), "emo_search_dp")
    return {"found": bool(found.value), "F": F, "T": int(T.value), "E": float(E.value), "n_pred": int(calls.value)}


def emo_pack_greedy(n, row_ptr, col, is_kernel, stream_of, t_default, delta_max):
    """Host arrays in, (crit, pack_of, n_packs) out (see include/emo.h)."""
    rp = np.ascontiguousarray(row_ptr, np.int64)
    cl = np.ascontiguousarray(col, np.int32)
    isk = np.ascontiguousarray(is_kernel, np.uint8)
    so = np.ascontiguousarray(stream_of, np.int32)
    td = np.ascontiguousarray(t_default, np.int64)
    crit = np.zeros(int(n), np.int32)
    pack_of = np.zeros(int(n), np.int32)
    cnt = ctypes.c_int32(0)
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().emo_pack_greedy(int(n), vp(rp), vp(cl), vp(isk), vp(so), vp(td), int(delta_max), vp(crit), vp(pack_of),
                                 ctypes.byref(cnt)), "emo_pack_greedy")
    return crit, pack_of, int(cnt.value)


def emo_pack_tables(lat, energy, pack_of, n_packs):
    lt = np.ascontiguousarray(lat, np.int64)
    en = np.ascontiguousarray(energy, np.float64)
    po = np.ascontiguousarray(pack_of, np.int32)
    n, L = lt.shape
    pl = np.zeros((int(n_packs), L), np.int64)
    pe = np.zeros((int(n_packs), L), np.float64)
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().emo_pack_tables(int(n), int(L), vp(lt), vp(en), vp(po), int(n_packs), vp(pl), vp(pe)), "emo_pack_tables")
    return pl, pe


def emo_pack_classes(pack_of, name_id, n_packs):
    po = np.ascontiguousarray(pack_of, np.int32)
    nm = np.ascontiguousarray(name_id, np.int32)
    cls = np.zeros(int(n_packs), np.int32)
    cnt = ctypes.c_int32(0)
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().emo_pack_classes(int(po.shape[0]), vp(po), vp(nm), int(n_packs), vp(cls), ctypes.byref(cnt)), "emo_pack_classes")
    return cls, int(cnt.value)


def emo_pack_model(n_packs, n_metrics, m, L, Bmat, feat, Tb, Eb, x, T_out, E_out, status=None, stream=None):
    """Device tensors in and out (see include/emo.h)."""
    return _check(lib().emo_pack_model(int(n_packs), int(n_metrics), int(m), int(L), _addr(Bmat), _addr(feat), _addr(Tb), _addr(Eb),
                                       _addr(x), _addr(T_out), _addr(E_out), _addr(status), _stream(stream)), "emo_pack_model")


def emo_pack_levels(bits, rows, B, lvl, ldb, packed, ldp, stream=None):
    _check(lib().emo_pack_levels(int(bits), int(rows), int(B), _addr(lvl), int(ldb), _addr(packed), int(ldp), _stream(stream)),
           "emo_pack_levels")


def emo_unpack_levels(bits, rows, B, packed, ldp, lvl, ldb, stream=None):
    _check(lib().emo_unpack_levels(int(bits), int(rows), int(B), _addr(packed), int(ldp), _addr(lvl), int(ldb), _stream(stream)),
           "emo_unpack_levels")


def _event(ev) -> Optional[int]:
    if ev is None:
        return None
    if not ev.cuda_event:          # torch creates the handle lazily, on the first record
        ev.record()
    return int(ev.cuda_event)


def emo_levels_prefetch(g: Graph, lvl_host, ld_host, dev_packed, copy_stream, ready):
    """Enqueues the copy of packed levels on copy_stream and records the torch event `ready` behind it."""
    _check(lib().emo_levels_prefetch(g.handle, _addr(lvl_host), int(ld_host), _addr(dev_packed), _stream(copy_stream),
                                     _event(ready)), "emo_levels_prefetch")


def emo_slack_batch_prefetched(g: Graph, B, bits, dev_packed, ld_packed, ready, dev_lvl, ldb, slack_dev, ldo, delta_ppm,
                               makespan_host, energy_host, slack_sum_host, n_critical_host, sel_host, ws, flags=0, stream=None):
    _check(lib().emo_slack_batch_prefetched(g.handle, int(B), int(bits), _addr(dev_packed), int(ld_packed), _event(ready),
                                            _addr(dev_lvl), int(ldb), _addr(slack_dev), int(ldo), int(delta_ppm),
                                            _addr(makespan_host), _addr(energy_host), _addr(slack_sum_host),
                                            _addr(n_critical_host), _addr(sel_host), _addr(ws), _nbytes(ws), int(flags),
                                            _stream(stream)), "emo_slack_batch_prefetched")


def emo_slack_batch_host_packed(g: Graph, B, bits, lvl_host, ld_host, dev_packed, dev_lvl, ldb, slack_dev, ldo, delta_ppm,
                                makespan_host, energy_host, slack_sum_host, n_critical_host, sel_host, ws, flags=0, stream=None):
    _check(lib().emo_slack_batch_host_packed(g.handle, int(B), int(bits), _addr(lvl_host), int(ld_host), _addr(dev_packed),
                                             _addr(dev_lvl), int(ldb), _addr(slack_dev), int(ldo), int(delta_ppm),
                                             _addr(makespan_host), _addr(energy_host), _addr(slack_sum_host),
                                             _addr(n_critical_host), _addr(sel_host), _addr(ws), _nbytes(ws), int(flags),
                                             _stream(stream)), "emo_slack_batch_host_packed")
