"""Seeded synthetic inputs: execution graphs, latency/energy tables and policy batches.

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/bench. It holds none of the method's arithmetic (no longest path, no slack, no
selection): it only draws graphs shaped like the execution graphs of Sec. 4.2/4.3 (a CPU
launch chain of runtime-API intervals, GPU streams in program order, event waits between
streams, host syncs, collectives joining device timelines), the frequency-indexed
per-node tables of Eq. 3, and frequency-level policies.

Everything is a pure function of (seed, index): a counter-based generator built on the
splitmix64 finaliser, so host and device can draw the same policy entries without
sharing state.  Graphs are numpy; policies are torch tensors so the same code fills a
host buffer or a device buffer.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

F_MIN_MHZ = 990.0
F_MAX_MHZ = 1965.0
P_STATIC_W = 100.0
P_DYN_W_AT_FMAX = 900.0
CPU_NODE_NS = 5_000
COLLECTIVE_NS = 50_000

KIND_CPU = 0
KIND_KERNEL = 1
KIND_COLLECTIVE = 2


# --------------------------------------------------------------------------------------
# counter-based random numbers (numpy, uint64 wrap-around arithmetic on arrays)
# --------------------------------------------------------------------------------------
def _mix64(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * _C1
        x = (x ^ (x >> np.uint64(27))) * _C2
        x = x ^ (x >> np.uint64(31))
    return x


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        a = _mix64(np.array([np.uint64(seed) * _GOLD + np.uint64(0x1234567)], dtype=np.uint64))[0]
        b = _mix64(np.array([a ^ (np.uint64(stream) * _C2 + _GOLD)], dtype=np.uint64))[0]
    return b


def rand_u64(seed: int, stream: int, counters) -> np.ndarray:
    """64 random bits per counter value; pure function of (seed, stream, counter)."""
    c = np.asarray(counters, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix64(_key(seed, stream) + c * _GOLD)


def rand_uniform(seed: int, stream: int, counters) -> np.ndarray:
    """Uniform doubles in [0, 1) from the top 53 bits."""
    return (rand_u64(seed, stream, counters) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def rand_normal(seed: int, stream: int, counters) -> np.ndarray:
    """Standard normals by Box-Muller from two uniform streams."""
    c = np.asarray(counters, dtype=np.uint64)
    u1 = rand_uniform(seed, stream, c * np.uint64(2))
    u2 = rand_uniform(seed, stream, c * np.uint64(2) + np.uint64(1))
    u1 = np.maximum(u1, 2.0 ** -53)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def rand_beta22(seed: int, stream: int, counters) -> np.ndarray:
    """Beta(2,2) as the median of three independent uniforms."""
    c = np.asarray(counters, dtype=np.uint64)
    u = np.stack([rand_uniform(seed, stream, c * np.uint64(3) + np.uint64(k)) for k in range(3)])
    return np.sort(u, axis=0)[1]


# --------------------------------------------------------------------------------------
# graph container
# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class Graph:
    """Predecessor-CSR DAG with per-node tables, nodes numbered level by level."""

    n: int
    row_ptr: np.ndarray      # int64 [n+1]
    col: np.ndarray          # int32 [m]  predecessors of node v: col[row_ptr[v]:row_ptr[v+1]]
    level_ptr: np.ndarray    # int32 [n_levels+1] node ranges of the hop-count levels
    L: int
    lat: np.ndarray          # int64 [n][L] nanoseconds
    energy: np.ndarray       # float64 [n][L] joules
    kind: np.ndarray         # uint8 [n]
    name: str = ""
    meta: Dict = dataclasses.field(default_factory=dict)

    @property
    def m(self) -> int:
        return int(self.col.shape[0])

    @property
    def n_levels(self) -> int:
        return int(self.level_ptr.shape[0] - 1)

    def preds(self, v: int) -> np.ndarray:
        return self.col[self.row_ptr[v]:self.row_ptr[v + 1]]

    def edges(self) -> List[Tuple[int, int]]:
        out = []
        for v in range(self.n):
            for k in self.preds(v):
                out.append((int(k), v))
        return out


def frequencies_mhz(L: int) -> np.ndarray:
    if L == 1:
        return np.array([F_MAX_MHZ])
    return F_MIN_MHZ + (F_MAX_MHZ - F_MIN_MHZ) * np.arange(L, dtype=np.float64) / (L - 1)


def kernel_tables(t_mem_ns: np.ndarray, t_comp_ns: np.ndarray, L: int) -> Tuple[np.ndarray, np.ndarray]:
    """lat[v][l] = rint(t_mem + t_comp * fmax / f_l); energy = lat * (P_static + k f^3)."""
    f = frequencies_mhz(L)
    lat = np.rint(t_mem_ns[:, None] + t_comp_ns[:, None] * (F_MAX_MHZ / f[None, :])).astype(np.int64)
    k = P_DYN_W_AT_FMAX / F_MAX_MHZ ** 3
    power = P_STATIC_W + k * f ** 3
    energy = lat.astype(np.float64) * 1e-9 * power[None, :]
    return lat, energy


def from_edges(n: int, edges: np.ndarray, lat: np.ndarray, energy: np.ndarray, kind: np.ndarray,
               name: str = "", meta: Optional[Dict] = None, keep_order: bool = False) -> Graph:
    """Renumber nodes level by level (hop-count level, ties by original id) and emit pred-CSR.

    `edges` is an int array [m][2] of (pred, succ) pairs in any numbering that is
    topological (pred < succ).  With keep_order the numbering is left as it is (the levels
    are then not contiguous ranges and level_ptr has a single range)."""
    edges = np.asarray(edges, dtype=np.int64).reshape(-1, 2)
    L = lat.shape[1]
    if edges.shape[0]:
        assert (edges[:, 0] < edges[:, 1]).all(), "generator edges must go forward"
    order = np.lexsort((edges[:, 0], edges[:, 1])) if edges.shape[0] else np.zeros(0, dtype=np.int64)
    e = edges[order]
    deg = np.bincount(e[:, 1], minlength=n) if e.shape[0] else np.zeros(n, dtype=np.int64)
    rp = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg, out=rp[1:])
    pc = e[:, 0].copy() if e.shape[0] else np.zeros(0, dtype=np.int64)
    hop = np.zeros(n, dtype=np.int64)
    rpl = rp.tolist()
    pcl = pc.tolist()
    hl = [0] * n
    for v in range(n):
        a, b = rpl[v], rpl[v + 1]
        if b > a:
            hl[v] = 1 + max(hl[k] for k in pcl[a:b])
    hop = np.asarray(hl, dtype=np.int64)
    if keep_order:
        new_of_old = np.arange(n, dtype=np.int64)
        level_ptr = np.array([0, n], dtype=np.int32)
    else:
        perm = np.lexsort((np.arange(n), hop))         # old ids in new order
        new_of_old = np.empty(n, dtype=np.int64)
        new_of_old[perm] = np.arange(n)
        nl = int(hop.max()) + 1 if n else 0
        cnt = np.bincount(hop, minlength=nl)
        level_ptr = np.zeros(nl + 1, dtype=np.int32)
        np.cumsum(cnt, out=level_ptr[1:])
    ne = np.stack([new_of_old[e[:, 0]], new_of_old[e[:, 1]]], axis=1) if e.shape[0] else e
    order2 = np.lexsort((ne[:, 0], ne[:, 1])) if ne.shape[0] else order
    ne = ne[order2]
    deg2 = np.bincount(ne[:, 1], minlength=n) if ne.shape[0] else np.zeros(n, dtype=np.int64)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg2, out=row_ptr[1:])
    col = ne[:, 0].astype(np.int32) if ne.shape[0] else np.zeros(0, dtype=np.int32)
    inv = np.empty(n, dtype=np.int64)
    inv[new_of_old] = np.arange(n)
    m = dict(meta or {})
    m["orig_of_new"] = inv
    return Graph(n=n, row_ptr=row_ptr, col=col, level_ptr=level_ptr, L=L,
                 lat=np.ascontiguousarray(lat[inv]), energy=np.ascontiguousarray(energy[inv]),
                 kind=np.ascontiguousarray(kind[inv]).astype(np.uint8), name=name, meta=m)


# --------------------------------------------------------------------------------------
# one device timeline: CPU launch chain + streams
# --------------------------------------------------------------------------------------
def _timeline(seed: int, tl: int, K: int, weights, r: int, p_ev: float, W: int, p_hs: float):
    """Nodes of one timeline in a topological 'trace order' numbering and its edge list.

    Local ids: CPU node j -> j ... interleaved so that every edge goes forward:
    id(cpu_j) = j*(r+1), id(kernel i) = (i//r)*(r+1) + 1 + i%r.  Returns
    (n_local, edges[m][2], kind[n_local], stream_of_kernel[K], id_of_kernel[K], id_of_cpu[ncpu])."""
    ncpu = (K + r - 1) // r
    kid = (np.arange(K) // r) * (r + 1) + 1 + (np.arange(K) % r)
    cid = np.arange(ncpu) * (r + 1)
    n_local = int(max(kid[-1], cid[-1])) + 1
    kind = np.full(n_local, 255, dtype=np.uint8)
    kind[cid] = KIND_CPU
    kind[kid] = KIND_KERNEL
    base = 16 * tl
    cw = np.cumsum(np.asarray(weights, dtype=np.float64))
    cw /= cw[-1]
    u = rand_uniform(seed, base + 1, np.arange(K))
    stream = np.searchsorted(cw, u, side="right").astype(np.int64)
    stream = np.minimum(stream, len(weights) - 1)
    u_ev = rand_uniform(seed, base + 2, np.arange(K))
    u_pick = rand_uniform(seed, base + 3, np.arange(K))
    u_hs = rand_uniform(seed, base + 4, np.arange(K))
    edges = []
    for j in range(1, ncpu):
        edges.append((cid[j - 1], cid[j]))
    last_on = [-1] * len(weights)
    st = stream.tolist()
    for i in range(K):
        edges.append((cid[i // r], kid[i]))                       # launch
        s = st[i]
        if last_on[s] >= 0:
            edges.append((kid[last_on[s]], kid[i]))               # stream program order
        if u_ev[i] < p_ev:                                        # event wait on another stream
            lo = max(0, i - W)
            cand = [q for q in range(lo, i) if st[q] != s]
            if cand:
                q = cand[min(int(u_pick[i] * len(cand)), len(cand) - 1)]
                edges.append((kid[q], kid[i]))
        if p_hs > 0.0 and u_hs[i] < p_hs and (i // r) + 1 < ncpu:  # host sync back to the CPU chain
            edges.append((kid[i], cid[i // r + 1]))
        last_on[s] = i
    keep = kind != 255
    assert keep.all()
    return n_local, np.asarray(edges, dtype=np.int64), kind, stream, kid, cid


def _durations(seed: int, stream_id: int, K: int, mode: str, median_ns: float, sigma: float,
               heavy_frac: float = 0.0) -> Tuple[np.ndarray, np.ndarray]:
    idx = np.arange(K)
    if mode == "independent":       # t_mem and t_comp each lognormal
        t_mem = np.exp(math.log(median_ns) + sigma * rand_normal(seed, stream_id, idx))
        t_comp = np.exp(math.log(median_ns) + sigma * rand_normal(seed, stream_id + 1, idx))
        return t_mem, t_comp
    total = np.exp(math.log(median_ns) + sigma * rand_normal(seed, stream_id, idx))
    if heavy_frac > 0.0:
        uh = rand_uniform(seed, stream_id + 2, idx)
        uv = rand_uniform(seed, stream_id + 3, idx)
        total = np.where(uh < heavy_frac, 1.0e6 + 4.0e6 * uv, total)
    x = rand_beta22(seed, stream_id + 1, idx)
    return total * (1.0 - x), total * x


def _assemble(seed: int, name: str, L: int, timelines: int, K: int, weights, r: int, p_ev: float,
              W: int, p_hs: float, dur_mode: str, median_ns: float, sigma: float,
              heavy_frac: float = 0.0, collective_every: int = 0) -> Graph:
    parts = []
    off = 0
    all_edges = []
    kinds = []
    lat_rows = []
    en_rows = []
    kid_global = []
    n_stream, n_launch, n_cpu = [], [], []
    for tl in range(timelines):
        n_local, edges, kind, stream, kid, cid = _timeline(seed, tl, K, weights, r, p_ev, W, p_hs)
        t_mem, t_comp = _durations(seed, 1000 + 16 * tl, K, dur_mode, median_ns, sigma, heavy_frac)
        klat, ken = kernel_tables(t_mem, t_comp, L)
        lat = np.full((n_local, L), CPU_NODE_NS, dtype=np.int64)
        en = np.zeros((n_local, L), dtype=np.float64)
        lat[kid] = klat
        en[kid] = ken
        all_edges.append(edges + off)
        kinds.append(kind)
        lat_rows.append(lat)
        en_rows.append(en)
        kid_global.append(kid + off)
        ns = np.full(n_local, -1, dtype=np.int64)
        nl_ = np.full(n_local, -1, dtype=np.int64)
        nc = np.full(n_local, -1, dtype=np.int64)
        ns[kid] = stream
        nl_[kid] = np.arange(K)
        nc[cid] = np.arange(len(cid))
        n_stream.append(ns)
        n_launch.append(nl_)
        n_cpu.append(nc)
        parts.append((off, n_local, stream))
        off += n_local
    n = off
    edges = np.concatenate(all_edges) if all_edges else np.zeros((0, 2), dtype=np.int64)
    kind = np.concatenate(kinds)
    lat = np.concatenate(lat_rows)
    en = np.concatenate(en_rows)
    meta = {"K": K, "timelines": timelines, "r": r, "n_streams": len(weights)}
    node_stream = np.concatenate(n_stream)
    node_launch = np.concatenate(n_launch)
    node_cpu = np.concatenate(n_cpu)
    node_tl = np.concatenate([np.full(p[1], t, dtype=np.int64) for t, p in enumerate(parts)])
    if collective_every and timelines > 1:
        # Nodes of several timelines must stay in a topological numbering: interleave by
        # giving every node the sort key (position within its timeline, timeline) and putting
        # the j-th collective right after position of the (j*every)-th kernel.
        pos = np.concatenate([np.arange(p[1]) for p in parts]).astype(np.float64)
        ncoll = (K - 1) // collective_every
        coll_edges = []
        coll_pos = []
        for j in range(1, ncoll + 1):
            cnode = n + (j - 1)
            src_local = (((j * collective_every - 1) // r) * (r + 1) + 1 + ((j * collective_every - 1) % r))
            dst_local = (((j * collective_every) // r) * (r + 1) + 1 + ((j * collective_every) % r))
            for tl in range(timelines):
                coll_edges.append((parts[tl][0] + src_local, cnode))
                coll_edges.append((cnode, parts[tl][0] + dst_local))
            coll_pos.append(src_local + 0.5)
        n_all = n + ncoll
        pos = np.concatenate([pos, np.asarray(coll_pos)])
        tl_of = np.concatenate([np.full(p[1], t) for t, p in enumerate(parts)] + [np.full(ncoll, timelines)])
        order = np.lexsort((tl_of, pos))
        new_of_old = np.empty(n_all, dtype=np.int64)
        new_of_old[order] = np.arange(n_all)
        edges = np.concatenate([edges, np.asarray(coll_edges, dtype=np.int64)])
        edges = new_of_old[edges]
        kind = np.concatenate([kind, np.full(ncoll, KIND_COLLECTIVE, dtype=np.uint8)])[order]
        lat = np.concatenate([lat, np.full((ncoll, L), COLLECTIVE_NS, dtype=np.int64)])[order]
        en = np.concatenate([en, np.zeros((ncoll, L))])[order]
        pad = np.full(ncoll, -1, dtype=np.int64)
        node_stream = np.concatenate([node_stream, pad])[order]
        node_launch = np.concatenate([node_launch, pad])[order]
        node_cpu = np.concatenate([node_cpu, pad])[order]
        node_tl = np.concatenate([node_tl, pad])[order]
        n = n_all
        meta["collectives"] = ncoll
    g = from_edges(n, edges, lat, en, kind, name=name, meta=meta)
    inv = g.meta["orig_of_new"]
    g.meta["node_stream"] = node_stream[inv]
    g.meta["node_launch"] = node_launch[inv]
    g.meta["node_cpu"] = node_cpu[inv]
    g.meta["node_timeline"] = node_tl[inv]
    return g


# --------------------------------------------------------------------------------------
# the five workload configurations
# --------------------------------------------------------------------------------------
CONFIGS = {
    "cfg0-tiny": dict(index=0, L=8, B=64, delta_ppm=[], policy_mode="uniform"),
    "cfg1-train": dict(index=1, L=16, B=4096, delta_ppm=[30_000], policy_mode="mixed", q_max=0.5),
    "cfg2-packed": dict(index=2, L=16, B=65536, delta_ppm=[20_000, 50_000], policy_mode="mixed", q_max=0.1),
    "cfg3-8dev": dict(index=3, L=24, B=8192, delta_ppm=[50_000], policy_mode="mixed", q_max=0.5),
    "cfg4-llm": dict(index=4, L=32, B=16384, delta_ppm=[50_000], policy_mode="mixed", q_max=0.5),
}


def make_graph(name: str, scale: float = 1.0) -> Graph:
    """Build the graph of a named configuration.  `scale` < 1 shrinks the kernel count
    (same structure, for fast tests); 1.0 gives the full size."""
    cfg = CONFIGS[name]
    seed = cfg["index"]

    def sc(k: int) -> int:
        return max(8, int(round(k * scale)))

    if name == "cfg0-tiny":
        g = _assemble(seed, name, 8, 1, sc(200), [0.5, 0.5], 1, 0.1, 16, 0.0, "independent", 20_000.0, 1.0)
    elif name == "cfg1-train":
        g = _assemble(seed, name, 16, 1, sc(5000), [0.70, 0.15, 0.15], 1, 0.05, 64, 0.002, "split", 40_000.0, 1.0)
    elif name == "cfg2-packed":
        base = _assemble(1, "cfg1-train", 16, 1, sc(5000), [0.70, 0.15, 0.15], 1, 0.05, 64, 0.002, "split",
                         40_000.0, 1.0)
        g = pack_graph(base, min_packs=max(4, int(round(500 * scale))), name=name)
    elif name == "cfg3-8dev":
        g = _assemble(seed, name, 24, 8, sc(8000), [0.75, 0.25], 1, 0.05, 64, 0.0, "split", 40_000.0, 1.0,
                      collective_every=max(4, int(round(200 * min(1.0, max(scale, 0.05))))))
    elif name == "cfg4-llm":
        g = _assemble(seed, name, 32, 1, sc(200_000), [0.25, 0.25, 0.25, 0.25], 4, 0.1, 32, 0.0, "split",
                      8_000.0, 1.0, heavy_frac=0.01)
    else:
        raise KeyError(name)
    g.meta.update(config=name, scale=scale, policy_seed=1000 + cfg["index"], B=cfg["B"],
                  delta_ppm=list(cfg["delta_ppm"]), policy_mode=cfg["policy_mode"],
                  q_max=cfg.get("q_max", 0.5))
    return g


# --------------------------------------------------------------------------------------
# packing stand-in (contiguous same-stream runs; inner dependencies dropped, Sec. 4.4)
# --------------------------------------------------------------------------------------
def pack_graph(g: Graph, min_packs: int, name: str = "packed") -> Graph:
    """Collapse kernels into packs: a pack is a run of consecutive kernels of one stream.

    A run is cut before a kernel that has an incoming event edge and after a kernel that has an
    outgoing event or host-sync edge, so every kept cross-stream edge starts at a pack's last
    kernel and ends at a pack's first kernel; the longest runs are then split until there are at
    least `min_packs`.  Launch edges into non-first members are dropped (only the first
    kernel's incoming and the last kernel's outgoing dependencies survive).  The pack table is
    the per-level sum of its members' tables.  CPU nodes are merged into segments that end at a
    kept launch source and start at a host-sync target."""
    n = g.n
    kind = g.kind
    preds = [g.preds(v).tolist() for v in range(n)]
    succs: List[List[int]] = [[] for _ in range(n)]
    for v in range(n):
        for k in preds[v]:
            succs[k].append(v)
    is_k = kind == KIND_KERNEL
    K = g.meta["K"]
    r = g.meta["r"]
    assert g.meta["timelines"] == 1
    launch_idx = g.meta["node_launch"]
    cpu_idx = g.meta["node_cpu"]
    node_of_kernel = np.empty(K, dtype=np.int64)
    node_of_kernel[launch_idx[is_k]] = np.nonzero(is_k)[0]
    ncpu = int(cpu_idx.max()) + 1
    node_of_cpu = np.empty(ncpu, dtype=np.int64)
    node_of_cpu[cpu_idx[cpu_idx >= 0]] = np.nonzero(cpu_idx >= 0)[0]
    n_streams = g.meta["n_streams"]
    stream = g.meta["node_stream"][node_of_kernel]
    stream_prev = np.full(K, -1, dtype=np.int64)
    event_in: List[List[int]] = [[] for _ in range(K)]
    launch_src = np.full(K, -1, dtype=np.int64)
    hs_out: List[List[int]] = [[] for _ in range(K)]
    last_on = [-1] * n_streams
    for i in range(K):
        s = int(stream[i])
        stream_prev[i] = last_on[s]
        last_on[s] = i
    for i in range(K):
        v = int(node_of_kernel[i])
        for k in preds[v]:
            if kind[k] == KIND_CPU:
                launch_src[i] = cpu_idx[k]
            else:
                q = int(launch_idx[k])
                if q != stream_prev[i]:
                    event_in[i].append(q)
        for w in succs[v]:
            if kind[w] == KIND_CPU:
                hs_out[i].append(int(cpu_idx[w]))
    has_event_out = np.zeros(K, dtype=bool)
    for i in range(K):
        for q in event_in[i]:
            has_event_out[q] = True
    # runs per stream
    cut_before = np.zeros(K, dtype=bool)
    for i in range(K):
        if stream_prev[i] < 0 or event_in[i]:
            cut_before[i] = True
        p = stream_prev[i]
        if p >= 0 and (has_event_out[p] or hs_out[p]):
            cut_before[i] = True
    chains: List[List[int]] = [[] for _ in range(n_streams)]
    for i in range(K):
        chains[int(stream[i])].append(i)
    packs: List[List[int]] = []
    for ch in chains:
        cur: List[int] = []
        for i in ch:
            if cut_before[i] and cur:
                packs.append(cur)
                cur = []
            cur.append(i)
        if cur:
            packs.append(cur)
    while len(packs) < min_packs:
        j = max(range(len(packs)), key=lambda t: (len(packs[t]), -packs[t][0]))
        p = packs[j]
        if len(p) < 2:
            break
        h = len(p) // 2
        packs[j:j + 1] = [p[:h], p[h:]]
    packs.sort(key=lambda p: p[0])
    pack_of = np.empty(K, dtype=np.int64)
    for j, p in enumerate(packs):
        for i in p:
            pack_of[i] = j
    # CPU segments: end after a kept launch source, start before a host-sync target
    end_after = np.zeros(ncpu, dtype=bool)
    start_before = np.zeros(ncpu, dtype=bool)
    for p in packs:
        end_after[launch_src[p[0]]] = True
    for i in range(K):
        for c in hs_out[i]:
            start_before[c] = True
    seg_of = np.empty(ncpu, dtype=np.int64)
    seg = 0
    for j in range(ncpu):
        if j > 0 and (start_before[j] or end_after[j - 1]):
            seg += 1
        seg_of[j] = seg
    nseg = seg + 1
    # node ids in a forward order: sort key = (launch position, is-pack)
    first_cpu = np.full(nseg, ncpu, dtype=np.int64)
    count_cpu = np.zeros(nseg, dtype=np.int64)
    for j in range(ncpu):
        first_cpu[seg_of[j]] = min(first_cpu[seg_of[j]], j)
        count_cpu[seg_of[j]] += 1
    L = g.L
    npk = len(packs)
    nn = nseg + npk
    # trace position: CPU node j sits at j*(r+1); kernel i at (i//r)*(r+1)+1+i%r
    seg_last = first_cpu + count_cpu - 1
    keys = [(int(seg_last[s]) * (r + 1), 0, s) for s in range(nseg)]
    keys += [(((p[0] // r) * (r + 1) + 1 + p[0] % r), 1, nseg + j) for j, p in enumerate(packs)]
    # a pack must come after every predecessor: its first kernel's launch source segment (ends at or
    # before its own cpu), its stream-prev pack (earlier first kernel... but a later *last* kernel is
    # possible only on other streams); event sources are pack-last kernels launched earlier.
    order = sorted(range(nn), key=lambda t: keys[t])
    new_of = np.empty(nn, dtype=np.int64)
    for pos, t in enumerate(order):
        new_of[keys[t][2]] = pos
    lat = np.zeros((nn, L), dtype=np.int64)
    en = np.zeros((nn, L), dtype=np.float64)
    kd = np.zeros(nn, dtype=np.uint8)
    for s in range(nseg):
        lat[new_of[s], :] = CPU_NODE_NS * count_cpu[s]
        kd[new_of[s]] = KIND_CPU
    for j, p in enumerate(packs):
        rows = node_of_kernel[np.asarray(p)]
        lat[new_of[nseg + j]] = g.lat[rows].sum(axis=0)
        en[new_of[nseg + j]] = g.energy[rows].sum(axis=0)
        kd[new_of[nseg + j]] = KIND_KERNEL
    edges = set()
    for s in range(1, nseg):
        edges.add((int(new_of[s - 1]), int(new_of[s])))
    for j, p in enumerate(packs):
        me = int(new_of[nseg + j])
        f = p[0]
        edges.add((int(new_of[seg_of[launch_src[f]]]), me))
        if stream_prev[f] >= 0:
            edges.add((int(new_of[nseg + pack_of[stream_prev[f]]]), me))
        for q in event_in[f]:
            edges.add((int(new_of[nseg + pack_of[q]]), me))
        la = p[-1]
        for c in hs_out[la]:
            edges.add((me, int(new_of[seg_of[c]])))
    ed = np.asarray(sorted(edges), dtype=np.int64)
    # the sort key above is a heuristic order; make it topological by a stable Kahn pass
    ed, lat, en, kd, perm = _topo_relabel(nn, ed, lat, en, kd)
    meta = {"K": K, "r": r, "packs": npk, "cpu_segments": nseg,
            "pack_members": [node_of_kernel[np.asarray(p)].tolist() for p in packs],
            "pack_new_id": [int(perm[new_of[nseg + j]]) for j in range(npk)],
            "seg_new_id": [int(perm[new_of[s]]) for s in range(nseg)],
            "seg_members": [node_of_cpu[first_cpu[s]:first_cpu[s] + count_cpu[s]].tolist() for s in range(nseg)]}
    return from_edges(nn, ed, lat, en, kd, name=name, meta=meta)


def _topo_relabel(n, edges, lat, en, kd):
    indeg = np.zeros(n, dtype=np.int64)
    succ: List[List[int]] = [[] for _ in range(n)]
    for a, b in edges.tolist():
        succ[a].append(b)
        indeg[b] += 1
    import heapq
    heap = [v for v in range(n) if indeg[v] == 0]
    heapq.heapify(heap)
    new = np.full(n, -1, dtype=np.int64)
    t = 0
    while heap:
        v = heapq.heappop(heap)
        new[v] = t
        t += 1
        for w in succ[v]:
            indeg[w] -= 1
            if indeg[w] == 0:
                heapq.heappush(heap, w)
    assert t == n, "packed graph has a cycle"
    inv = np.empty(n, dtype=np.int64)
    inv[new] = np.arange(n)
    e2 = new[edges] if edges.shape[0] else edges
    return e2, lat[inv], en[inv], kd[inv], new


# --------------------------------------------------------------------------------------
# small hand-made and random DAGs for exhaustive tests
# --------------------------------------------------------------------------------------
def tiny_graph(n: int, edges, lat, energy=None, name: str = "tiny", keep_order: bool = True) -> Graph:
    lat = np.asarray(lat, dtype=np.int64).reshape(n, -1)
    if energy is None:
        energy = lat.astype(np.float64) * 0.5 + 1.0
    energy = np.asarray(energy, dtype=np.float64).reshape(n, -1)
    ed = np.asarray(list(edges), dtype=np.int64).reshape(-1, 2)
    return from_edges(n, ed, lat, energy, np.full(n, KIND_KERNEL, dtype=np.uint8), name=name,
                      keep_order=keep_order)


def random_dag(seed: int, n: int, p_edge: float, L: int = 3, max_dur: int = 20,
               monotone: bool = True, keep_order: bool = True) -> Graph:
    """Random DAG on n nodes: each ordered pair i<j is an edge with probability p_edge;
    small integer durations so ties are frequent."""
    pairs = [(i, j) for i in range(n) for j in range(i + 1, n)]
    u = rand_uniform(seed, 50, np.arange(len(pairs))) if pairs else np.zeros(0)
    edges = [pq for pq, x in zip(pairs, u) if x < p_edge]
    d = (rand_u64(seed, 51, np.arange(n * L)) % np.uint64(max_dur + 1)).astype(np.int64).reshape(n, L)
    if monotone:
        d = -np.sort(-d, axis=1)            # non-increasing in the level (higher level = faster)
    e = rand_uniform(seed, 52, np.arange(n * L)).reshape(n, L) * 10.0
    return tiny_graph(n, edges, d, e, name=f"rand{seed}", keep_order=keep_order)


# --------------------------------------------------------------------------------------
# policies (torch, device-agnostic)
# --------------------------------------------------------------------------------------
def _t_const(x: int) -> int:
    x &= 0xFFFFFFFFFFFFFFFF
    return x - (1 << 64) if x >= (1 << 63) else x


def _t_lsr(x, k: int):
    return (x >> k) & ((1 << (64 - k)) - 1)


def _t_mix64(x):
    x = (x ^ _t_lsr(x, 30)) * _t_const(0xBF58476D1CE4E5B9)
    x = (x ^ _t_lsr(x, 27)) * _t_const(0x94D049BB133111EB)
    return x ^ _t_lsr(x, 31)


def policy_q(policy_seed: int, B: int, n_rows: int, q_max: float) -> np.ndarray:
    """Per-policy perturbation probability: log-uniform in [1/n_rows, q_max] (numpy, host)."""
    u = rand_uniform(policy_seed, 7, np.arange(B))
    lo = math.log(1.0 / max(n_rows, 2))
    hi = math.log(q_max)
    return np.exp(lo + (hi - lo) * u)


def policy_levels(policy_seed: int, n_rows: int, L: int, B: int, mode: str = "mixed", q_max: float = 0.5,
                  rows: Optional[Tuple[int, int]] = None, cols: Optional[Tuple[int, int]] = None,
                  device="cpu", out=None):
    """uint8 tensor [r1-r0][c1-c0] of frequency levels, entry (v, b) a pure function of
    (policy_seed, v, b).

    mode "uniform": every entry uniform in [0, L).
    mode "mixed":   policy 0 is all L-1 (the default, maximum frequency); policies 1..B/2-1 keep
                    L-1 except that each node is re-drawn uniformly with probability q_b;
                    policies B/2..B-1 are uniform."""
    import torch
    r0, r1 = rows if rows is not None else (0, n_rows)
    c0, c1 = cols if cols is not None else (0, B)
    dev = torch.device(device)
    v = torch.arange(r0, r1, dtype=torch.int64, device=dev)[:, None]
    b = torch.arange(c0, c1, dtype=torch.int64, device=dev)[None, :]
    key = int(_key(policy_seed, 3))
    ctr = v * int(B) + b
    h = _t_mix64(ctr * _t_const(0x9E3779B97F4A7C15) + _t_const(key))
    lvl = (_t_lsr(h, 40) * L) >> 24                       # 24 random bits -> [0, L)
    if mode == "mixed":
        q = torch.from_numpy(policy_q(policy_seed, B, n_rows, q_max)[c0:c1]).to(dev)
        thr = (q * float(1 << 24)).to(torch.int64)[None, :]
        draw = h & ((1 << 24) - 1)                        # low 24 bits, independent of the level bits
        half = B // 2
        sparse = (b >= 1) & (b < half)
        keep = sparse & (draw >= thr)
        lvl = torch.where(keep | (b == 0), torch.full_like(lvl, L - 1), lvl)
    elif mode != "uniform":
        raise ValueError(mode)
    res = lvl.to(torch.uint8)
    if out is not None:
        out.copy_(res)
        return out
    return res


def policies_for(g: Graph, B: Optional[int] = None, device="cpu", ldb: Optional[int] = None):
    """Full [n][ldb] level matrix of a configuration graph (padding columns hold 0xFF so that a
    read of padding is caught by validation)."""
    import torch
    B = int(B if B is not None else g.meta["B"])
    ldb = int(ldb if ldb is not None else (B + 15) // 16 * 16)
    out = torch.full((g.n, ldb), 0xFF, dtype=torch.uint8, device=device)
    step = max(1, (1 << 24) // max(B, 1))
    for r0 in range(0, g.n, step):
        r1 = min(g.n, r0 + step)
        out[r0:r1, :B] = policy_levels(g.meta["policy_seed"], g.n, g.L, B, g.meta["policy_mode"],
                                       g.meta["q_max"], rows=(r0, r1), device=device)
    return out


# --------------------------------------------------------------------------------------
# time-interval policies (inputs of Alg. 1 in its own form: change points and one level per interval)
# --------------------------------------------------------------------------------------
def device_of(g: Graph) -> np.ndarray:
    """int32 [n]: the device timeline whose policy governs a kernel node, -1 for CPU and collective nodes
    (their duration does not depend on the GPU frequency)."""
    tl = np.asarray(g.meta.get("node_timeline", np.zeros(g.n, np.int64)), dtype=np.int64)
    return np.where(g.kind == KIND_KERNEL, tl, -1).astype(np.int32)


def interval_breaks(T_ref_ns: int, I: int) -> np.ndarray:
    """int64 [I]: I change points on a uniform grid over [0, 1.05 * T_ref) (the paper re-assigns the frequency
    every 20 ms; here the grid follows the workload's length)."""
    delta = max(1, int(T_ref_ns * 1.05) // int(I))
    return (np.arange(I, dtype=np.int64) * delta).astype(np.int64)


def interval_policies(policy_seed: int, n_dev: int, I: int, L: int, B: int, device="cpu", ldb: Optional[int] = None):
    """uint8 tensor [n_dev][I][ldb]: the 'mixed' recipe of policy_levels with one row per (device, interval):
    policy 0 holds the maximum frequency everywhere, the first half lowers a few intervals, the second half is
    uniform random.  Padding columns hold 0xFF."""
    import torch
    ldb = int(ldb if ldb is not None else (B + 15) // 16 * 16)
    out = torch.full((n_dev * I, ldb), 0xFF, dtype=torch.uint8, device=device)
    out[:, :B] = policy_levels(policy_seed + 7, n_dev * I, L, B, "mixed", 0.5, device=device)
    return out.reshape(n_dev, I, ldb)


def idle_power(L: int) -> np.ndarray:
    """fp64 [L] watts: idle power at each level, rising with the frequency (synthetic: 60 W + 40 W * f / f_max)."""
    f = 990.0 + 975.0 * np.arange(L) / max(L - 1, 1)
    return 60.0 + 40.0 * f / 1965.0


# --------------------------------------------------------------------------------------
# pack modelling inputs (Sec. 4.5; synthetic: the paper's micro-benchmark measurements are not available)
# --------------------------------------------------------------------------------------
def microbench_model(seed: int, n_metrics: int = 16, m: int = 12, L: int = 16):
    """(B [n_metrics][m] metric matrix, Tb [m][L] ns, Eb [m][L] J): every micro-benchmark stresses a few metrics,
    its time falls with the frequency, its energy follows 100 W + k f^3 as in the workload tables."""
    u = rand_uniform(seed, 70, np.arange(n_metrics * m)).reshape(n_metrics, m)
    hot = rand_uniform(seed, 71, np.arange(n_metrics * m)).reshape(n_metrics, m) < 0.3
    B = 0.05 * u + np.where(hot, 1.0 + 4.0 * rand_uniform(seed, 72, np.arange(n_metrics * m)).reshape(n_metrics, m), 0.0)
    B[np.arange(m) % n_metrics, np.arange(m)] += 3.0          # every benchmark has a metric of its own
    f = 990.0 + 975.0 * np.arange(L) / max(L - 1, 1)
    t_mem = 1000.0 + 9000.0 * rand_uniform(seed, 73, np.arange(m))
    t_comp = 1000.0 + 9000.0 * rand_uniform(seed, 74, np.arange(m))
    Tb = t_mem[:, None] + t_comp[:, None] * 1965.0 / f[None, :]
    Eb = Tb * 1e-9 * (100.0 + 900.0 * (f[None, :] / 1965.0) ** 3)
    return B, Tb, Eb


def pack_features(seed: int, B: np.ndarray, n_packs: int, noise: float = 0.02):
    """feat [n_packs][n_metrics]: sparse non-negative mixtures of the micro-benchmarks plus noise, so that the
    constraint x >= 0 is active for some of them."""
    n, m = B.shape
    w = rand_uniform(seed, 75, np.arange(n_packs * m)).reshape(n_packs, m)
    on = rand_uniform(seed, 76, np.arange(n_packs * m)).reshape(n_packs, m) < 0.3
    x = np.where(on, 10.0 * w, 0.0)
    z = rand_uniform(seed, 77, np.arange(n_packs * n)).reshape(n_packs, n) - 0.5
    return x @ B.T + noise * z * (1.0 + np.abs(x @ B.T))


def kernel_names(g: Graph, period: int = 48) -> np.ndarray:
    """int32 [n]: a name number for every kernel (-1 for other nodes).  The synthetic traces have no kernel names;
    an iteration of a model launches the same kernels layer after layer, so the name is the kernel's position in its
    stream's launch order modulo `period`, offset by the stream."""
    st = np.asarray(g.meta["node_stream"], np.int64)
    out = np.full(g.n, -1, np.int64)
    key = np.asarray(g.meta.get("node_timeline", np.zeros(g.n, np.int64)), np.int64) * 64 + st
    for s in np.unique(key[g.kind == KIND_KERNEL]):
        idx = np.flatnonzero((g.kind == KIND_KERNEL) & (key == s))
        out[idx] = (np.arange(idx.shape[0]) % period) + 1000 * (int(s) % 64)
    return out.astype(np.int32)
