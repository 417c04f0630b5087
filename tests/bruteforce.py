"""Brute-force reference for tiny DAGs: enumerate every source-to-sink path.

Independent of the oracle: no topological order, no recurrence.  For one vector of node
durations it returns
    T        = the longest source-to-sink path (sum of node durations on it),
    ES[v]    = the longest sum of durations of the nodes strictly before v over all paths that
               reach v from a source (0 for a source),
    through  = the longest source-to-sink path that contains v,
    slack[v] = T - through[v]   (total float of the critical-path method).
"""
from __future__ import annotations

import numpy as np


def all_paths(n, preds):
    succs = [[] for _ in range(n)]
    for v in range(n):
        for k in preds[v]:
            if v not in succs[k]:
                succs[k].append(v)
    sources = [v for v in range(n) if len(preds[v]) == 0]
    paths = []

    def walk(path):
        v = path[-1]
        if not succs[v]:
            paths.append(tuple(path))
            return
        for u in succs[v]:
            walk(path + [u])

    for s in sources:
        walk([s])
    return paths


def evaluate(n, preds, dur_matrix):
    """dur_matrix: [P][n] durations of P policies.  Returns T[P], ES[P][n], slack[P][n]."""
    dur = np.asarray(dur_matrix, dtype=np.int64)
    P = dur.shape[0]
    paths = all_paths(n, preds)
    T = np.zeros(P, dtype=np.int64)
    ES = np.zeros((P, n), dtype=np.int64)
    through = np.full((P, n), -1, dtype=np.int64)
    for p in paths:
        idx = np.asarray(p)
        d = dur[:, idx]
        total = d.sum(axis=1)
        T = np.maximum(T, total)
        before = np.cumsum(d, axis=1) - d
        for pos, v in enumerate(p):
            ES[:, v] = np.maximum(ES[:, v], before[:, pos])
            through[:, v] = np.maximum(through[:, v], total)
    slack = T[:, None] - through
    return T, ES, slack
