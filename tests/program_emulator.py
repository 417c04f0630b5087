"""Host-side interpreter of the compiled step programs, used only to test the scheduler and slot
allocation without a GPU.  It follows the kernels' rules: in a step every lane reads its operands
(its own register and slots written in earlier steps), then writes; a slot read and written in
the same step is reported as a hazard."""
from __future__ import annotations

import numpy as np

NONE = 0xFFFFFFFF
VALID, REGPRED, WRITE, TERMINAL, AUX = 1, 2, 4, 8, 0x80


def run(entries, lat, Lp, L, slots, lvl, n, backward, ES_in=None, T_in=None):
    """entries [steps][lanes][4], lat [steps*lanes][Lp], lvl uint8 [rows][B].
    Forward: returns dict(T[B], ES[n][B], seen[n]).  Backward: dict(LS, slack)."""
    steps, lanes, _ = entries.shape
    B = lvl.shape[1]
    h = np.zeros((lanes, B), dtype=np.int64)
    slot = np.zeros((max(slots, 1), B), dtype=np.int64)
    slot_valid = np.zeros(max(slots, 1), dtype=bool)
    seen = np.zeros(n, dtype=np.int64)
    out = {}
    if not backward:
        ES = np.zeros((n, B), dtype=np.int64)
        T = np.zeros(B, dtype=np.int64)
    else:
        LS = np.zeros((n, B), dtype=np.int64)
        SL = np.zeros((n, B), dtype=np.int64)
    for t in range(steps):
        writes = []
        read_ids = set()
        for w in range(lanes):
            row, node, flags, ops = (int(x) for x in entries[t, w])
            if not flags & VALID:
                continue
            lv = lvl[row] if row != NONE else np.zeros(B, dtype=np.uint8)
            assert (lv < L).all()
            q = t * lanes + w
            dur = lat[q][lv.astype(np.int64) & (Lp - 1)].astype(np.int64)
            start = h[w].copy() if flags & REGPRED else np.zeros(B, dtype=np.int64)
            ops |= (flags >> 16) << 32
            for k in range((flags >> 4) & 7):
                s = (ops >> (8 * k)) & 255
                assert slot_valid[s], f"step {t} lane {w} reads slot {s} before any write"
                read_ids.add(s)
                start = np.maximum(start, slot[s])
            val = start + dur
            if node != NONE:
                seen[node] += 1
                assert not flags & AUX
                if not backward:
                    ES[node] = start
                    if flags & TERMINAL:
                        T = np.maximum(T, val)
                else:
                    LS[node] = T_in - val
                    SL[node] = LS[node] - ES_in[node]
            else:
                assert flags & AUX
                assert (dur == 0).all()
            writes.append((w, val, (flags >> 8) & 255 if flags & WRITE else None))
        for w, val, s in writes:
            h[w] = val
            if s is not None:
                assert s not in read_ids, f"step {t}: slot {s} read and written in the same step"
                slot[s] = val
                slot_valid[s] = True
    out["seen"] = seen
    if not backward:
        out["T"], out["ES"] = T, ES
    else:
        out["LS"], out["slack"] = LS, SL
    return out
