"""Python face of the CPU oracle (oracle/emo_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the bench's
CPU-baseline leg.  It imports nothing from the CUDA package and the CUDA package imports nothing
from here.  The arithmetic lives in the C file; this module only builds it with gcc, loads it
with ctypes and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "emo_oracle.c")
_LIB = os.path.join(_HERE, "libemo_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                                   "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        p = ctypes.c_void_p
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        L.emo_oracle_topo.argtypes = [i32, p, p, p]
        L.emo_oracle_topo.restype = ctypes.c_int
        L.emo_oracle_durations.argtypes = [i32, i32, p, p, p, p, i64, p, p]
        L.emo_oracle_durations.restype = ctypes.c_int
        L.emo_oracle_forward.argtypes = [i32, p, p, p, p, p, p]
        L.emo_oracle_forward.restype = i64
        L.emo_oracle_backward.argtypes = [i32, p, p, p, p, i64, p]
        L.emo_oracle_backward.restype = ctypes.c_int
        L.emo_oracle_energy.argtypes = [i32, p]
        L.emo_oracle_energy.restype = ctypes.c_double
        L.emo_oracle_batch.argtypes = [i32, p, p, i32, p, p, p, p, i64, i64, i64, p, p, p, p, p, i64, i64, p, p]
        L.emo_oracle_batch.restype = ctypes.c_int
        L.emo_oracle_target.argtypes = [i64, i64]
        L.emo_oracle_target.restype = i64
        L.emo_oracle_select.argtypes = [i64, p, p, i64]
        L.emo_oracle_select.restype = i64
        L.emo_oracle_intervals.argtypes = [i32, p, p, i32, p, p, p, i32, i32, p, p, i64, i64, i64, p, p, p, p, p, i64]
        L.emo_oracle_intervals.restype = ctypes.c_int
        L.emo_oracle_search_dp.argtypes = [i32, p, p, i32, p, p, p, i32, i32, p, p, i64, i64, p, p, p, p, p]
        L.emo_oracle_search_dp.restype = ctypes.c_int
        L.emo_oracle_nnls.argtypes = [i32, i32, p, p, p, p]
        L.emo_oracle_nnls.restype = ctypes.c_int
        L.emo_oracle_pack_model.argtypes = [i32, i32, i32, i32, p, p, p, p, p, p, p]
        L.emo_oracle_pack_model.restype = ctypes.c_int
        L.emo_oracle_crit_pred.argtypes = [i32, p, p, p, p, p]
        L.emo_oracle_crit_pred.restype = ctypes.c_int
        L.emo_oracle_pack_greedy.argtypes = [i32, p, p, p, p, p, p, i64, p, p]
        L.emo_oracle_pack_greedy.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


class OracleError(RuntimeError):
    pass


def topo_order(n, row_ptr, col) -> np.ndarray:
    row_ptr = _c(row_ptr, np.int64)
    col = _c(col, np.int32)
    order = np.empty(max(n, 1), dtype=np.int32)
    rc = lib().emo_oracle_topo(n, _ptr(row_ptr), _ptr(col), _ptr(order))
    if rc:
        raise OracleError(f"emo_oracle_topo rc={rc}")
    return order[:n]


def forward(n, row_ptr, col, dur, order=None):
    """One policy given its durations: returns (T, ES, C)."""
    row_ptr = _c(row_ptr, np.int64)
    col = _c(col, np.int32)
    dur = _c(dur, np.int64)
    order = topo_order(n, row_ptr, col) if order is None else _c(order, np.int32)
    ES = np.empty(max(n, 1), dtype=np.int64)
    C = np.empty(max(n, 1), dtype=np.int64)
    T = lib().emo_oracle_forward(n, _ptr(row_ptr), _ptr(col), _ptr(order), _ptr(dur), _ptr(ES), _ptr(C))
    return int(T), ES[:n], C[:n]


def backward(n, row_ptr, col, dur, T, order=None):
    row_ptr = _c(row_ptr, np.int64)
    col = _c(col, np.int32)
    dur = _c(dur, np.int64)
    order = topo_order(n, row_ptr, col) if order is None else _c(order, np.int32)
    LS = np.empty(max(n, 1), dtype=np.int64)
    rc = lib().emo_oracle_backward(n, _ptr(row_ptr), _ptr(col), _ptr(order), _ptr(dur), int(T), _ptr(LS))
    if rc:
        raise OracleError(f"emo_oracle_backward rc={rc}")
    return LS[:n]


def energy_sum(e) -> float:
    e = _c(e, np.float64)
    return float(lib().emo_oracle_energy(e.shape[0], _ptr(e)))


def batch(g, lvl, B=None, b0=0, b1=None, want_slack=False, want_arrays=False, group_of=None,
          threads: int = 1):
    """Evaluate policies b0..b1 of the uint8 level matrix lvl[rows][ldb] on graph g (any object with
    n, row_ptr, col, L, lat, energy).  Returns a dict of numpy arrays: makespan, energy and, when
    asked, slack_sum / n_critical and ES / LS / slack as [n][b1-b0].

    threads > 1 only splits the policy range over Python threads; every thread runs the same plain
    single-policy C routine on its own columns."""
    lvl = np.ascontiguousarray(lvl, dtype=np.uint8)
    if lvl.ndim == 1:
        lvl = lvl.reshape(-1, 1)
    ldb = lvl.shape[1]
    B = int(B if B is not None else ldb)
    b1 = int(B if b1 is None else b1)
    nb = b1 - b0
    row_ptr = _c(g.row_ptr, np.int64)
    col = _c(g.col, np.int32)
    lat = _c(g.lat, np.int64)
    en = _c(g.energy, np.float64)
    go = None if group_of is None else _c(group_of, np.int32)
    out = {"makespan": np.zeros(B, dtype=np.int64), "energy": np.zeros(B, dtype=np.float64)}
    if want_slack or want_arrays:
        out["slack_sum"] = np.zeros(B, dtype=np.int64)
        out["n_critical"] = np.zeros(B, dtype=np.int32)
    if want_arrays:
        for k in ("ES", "LS", "slack"):
            out[k] = np.zeros((g.n, max(nb, 1)), dtype=np.int64)

    def run(lo, hi):
        rc = lib().emo_oracle_batch(
            g.n, _ptr(row_ptr), _ptr(col), g.L, _ptr(lat), _ptr(en), _ptr(go), _ptr(lvl), ldb, lo, hi,
            _ptr(out["makespan"]), _ptr(out["energy"]),
            _ptr(out.get("ES")), _ptr(out.get("LS")), _ptr(out.get("slack")), max(nb, 1), b0,
            _ptr(out.get("slack_sum")), _ptr(out.get("n_critical")))
        if rc:
            raise OracleError(f"emo_oracle_batch rc={rc}")

    threads = max(1, min(int(threads), max(nb, 1)))
    if threads == 1 or nb <= 1:
        run(b0, b1)
    else:
        cuts = np.linspace(b0, b1, threads + 1).astype(np.int64)
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda i: run(int(cuts[i]), int(cuts[i + 1])), range(threads)))
    out["makespan"] = out["makespan"][b0:b1]
    out["energy"] = out["energy"][b0:b1]
    if "slack_sum" in out:
        out["slack_sum"] = out["slack_sum"][b0:b1]
        out["n_critical"] = out["n_critical"][b0:b1]
    return out


def target_from_delta(T0: int, delta_ppm: int) -> int:
    return int(lib().emo_oracle_target(int(T0), int(delta_ppm)))


def select(makespan, energy, target: int) -> int:
    makespan = _c(makespan, np.int64)
    energy = _c(energy, np.float64)
    return int(lib().emo_oracle_select(makespan.shape[0], _ptr(makespan), _ptr(energy), int(target)))


def intervals(g, dev_of, breaks, F, p_idle=None, b0: int = 0, b1: Optional[int] = None, want_levels: bool = False):
    """Alg. 1 with time-interval policies.  F: uint8 [D][I][B]; breaks: int64 [I] change points (breaks[0] = 0).
    Returns a dict with makespan, e_active, e_idle, energy (their sum) and, if asked, levels [n][b1 - b0]."""
    F = _c(F, np.uint8)
    D, I, B = F.shape
    b1 = B if b1 is None else b1
    dev_of = _c(dev_of, np.int32)
    breaks = _c(breaks, np.int64)
    row_ptr, col = _c(g.row_ptr, np.int64), _c(g.col, np.int32)
    lat, energy = _c(g.lat, np.int64), _c(g.energy, np.float64)
    pi = None if p_idle is None else _c(p_idle, np.float64)
    T = np.zeros(B, np.int64)
    ea = np.zeros(B, np.float64)
    ei = np.zeros(B, np.float64)
    lv = np.zeros((g.n, max(b1 - b0, 1)), np.uint8) if want_levels else None
    rc = lib().emo_oracle_intervals(g.n, _ptr(row_ptr), _ptr(col), g.L, _ptr(lat), _ptr(energy), _ptr(dev_of), D, I,
                                    _ptr(breaks), _ptr(F), B, b0, b1, _ptr(pi), _ptr(T), _ptr(ea), _ptr(ei),
                                    _ptr(lv), lv.shape[1] if lv is not None else 0)
    if rc:
        raise OracleError(f"emo_oracle_intervals failed with {rc}")
    out = {"makespan": T[b0:b1], "e_active": ea[b0:b1], "e_idle": ei[b0:b1], "energy": (ea + ei)[b0:b1]}
    if want_levels:
        out["levels"] = lv
    return out


def search_dp(g, dev_of, breaks, p_idle, T_max: int, bin_ns: int = 1):
    """Alg. 2 over the intervals given by `breaks`.  Returns a dict: found, F (uint8 [I]), T, E, n_pred."""
    dev_of = _c(dev_of, np.int32)
    D = int(dev_of.max()) + 1 if dev_of.size and dev_of.max() >= 0 else 1
    breaks = _c(breaks, np.int64)
    I = int(breaks.shape[0])
    row_ptr, col = _c(g.row_ptr, np.int64), _c(g.col, np.int32)
    lat, energy = _c(g.lat, np.int64), _c(g.energy, np.float64)
    pi = None if p_idle is None else _c(p_idle, np.float64)
    F = np.zeros(I, np.uint8)
    T = ctypes.c_int64(0)
    E = ctypes.c_double(0.0)
    calls = ctypes.c_int64(0)
    found = ctypes.c_int32(0)
    rc = lib().emo_oracle_search_dp(g.n, _ptr(row_ptr), _ptr(col), g.L, _ptr(lat), _ptr(energy), _ptr(dev_of), D, I,
                                    _ptr(breaks), _ptr(pi), int(T_max), int(bin_ns), _ptr(F), ctypes.byref(T),
                                    ctypes.byref(E), ctypes.byref(calls), ctypes.byref(found))
    if rc:
        raise OracleError(f"emo_oracle_search_dp failed with {rc}")
    return {"found": bool(found.value), "F": F, "T": int(T.value), "E": float(E.value), "n_pred": int(calls.value)}


def crit_pred(g, dur):
    """Eq. 5 with Alg. 1's tie rule.  dur: int64 [n].  Returns (C int64 [n], crit int32 [n])."""
    row_ptr, col = _c(g.row_ptr, np.int64), _c(g.col, np.int32)
    dur = _c(dur, np.int64)
    C = np.zeros(g.n, np.int64)
    crit = np.zeros(g.n, np.int32)
    rc = lib().emo_oracle_crit_pred(g.n, _ptr(row_ptr), _ptr(col), _ptr(dur), _ptr(C), _ptr(crit))
    if rc:
        raise OracleError(f"emo_oracle_crit_pred failed with {rc}")
    return C, crit


def pack_greedy(g, is_kernel, stream_of, t_default, crit, delta_max: int):
    """Dependency-aware greedy packing.  Returns (pack_of int32 [n], number of packs)."""
    row_ptr, col = _c(g.row_ptr, np.int64), _c(g.col, np.int32)
    isk, so = _c(is_kernel, np.uint8), _c(stream_of, np.int32)
    td, cr = _c(t_default, np.int64), _c(crit, np.int32)
    pack_of = np.zeros(g.n, np.int32)
    cnt = ctypes.c_int32(0)
    rc = lib().emo_oracle_pack_greedy(g.n, _ptr(row_ptr), _ptr(col), _ptr(isk), _ptr(so), _ptr(td), _ptr(cr), int(delta_max),
                                      _ptr(pack_of), ctypes.byref(cnt))
    if rc:
        raise OracleError(f"emo_oracle_pack_greedy failed with {rc}")
    return pack_of, int(cnt.value)


def nnls(B, b):
    """Eq. 6 for one pack: argmin ||B x - b||^2, x >= 0.  Returns (x, squared residual)."""
    B = _c(B, np.float64)
    b = _c(b, np.float64)
    n, m = B.shape
    x = np.zeros(m, np.float64)
    r2 = ctypes.c_double(0.0)
    rc = lib().emo_oracle_nnls(n, m, _ptr(B), _ptr(b), _ptr(x), ctypes.byref(r2))
    if rc:
        raise OracleError(f"emo_oracle_nnls failed with {rc}")
    return x, float(r2.value)


def pack_model(B, feat, Tb, Eb):
    """Eq. 6 and Eq. 7 for every pack.  feat [packs][n], Tb / Eb [m][L].  Returns (x, T, E)."""
    B, feat, Tb, Eb = _c(B, np.float64), _c(feat, np.float64), _c(Tb, np.float64), _c(Eb, np.float64)
    n, m = B.shape
    P, L = feat.shape[0], Tb.shape[1]
    x = np.zeros((P, m)); T = np.zeros((P, L)); E = np.zeros((P, L))
    rc = lib().emo_oracle_pack_model(P, n, m, L, _ptr(B), _ptr(feat), _ptr(Tb), _ptr(Eb), _ptr(x), _ptr(T), _ptr(E))
    if rc:
        raise OracleError(f"emo_oracle_pack_model failed with {rc}")
    return x, T, E
