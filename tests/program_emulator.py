"""Host-side interpreter of the compiled step programs, used only to test the scheduler and slot
allocation without a GPU.  It follows the kernels' rules: in a step every lane reads its operands
(its own register and slots written in earlier steps), then writes; a slot read and written in
the same step is reported as a hazard."""
from __future__ import annotations

import numpy as np

NONE = 0xFFFFFFFF
VALID, REGPRED, WRITE, TERMINAL, AUX = 1, 2, 4, 8, 0x80
SYNC_STEPS = 8      # default distance between two barriers of a group's warps (a program names its own)


def run(entries, rows, lat, Lp, L, slots, lvl, n, backward, ES_in=None, T_in=None, sync=SYNC_STEPS):
    """entries [steps][lanes][8], lat [steps*lanes][Lp], lvl uint8 [rows][B].
    Forward: returns dict(T[B], ES[n][B], seen[n]).  Backward: dict(LS, slack)."""
    steps, lanes, _ = entries.shape
    main_rows = []
    B = lvl.shape[1]
    h = np.zeros((lanes, B), dtype=np.int64)
    slot = np.zeros((max(slots, 1), B), dtype=np.int64)
    slot_valid = np.zeros(max(slots, 1), dtype=bool)
    n_written = np.zeros(max(slots, 1), dtype=np.int64)      # values written to a slot so far
    last_read = np.full(max(slots, 1), -1, dtype=np.int64)
    write_step = np.full(max(slots, 1), -1, dtype=np.int64)
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
            main_row, flags, ops, ops_hi, node = (int(x) for x in entries[t, w][:5])
            row = int(rows[t, w])
            if not flags & VALID:
                continue
            lv = lvl[row] if row != NONE else np.zeros(B, dtype=np.uint8)
            assert (lv < L).all()
            mask = (flags >> 8) & 255
            assert mask == (Lp - 1 if row != NONE else 0)
            if row == NONE and node != NONE:
                assert (lat[t * lanes + w][:L] == lat[t * lanes + w][0]).all(), "row skipped for a level-dependent node"
            if node != NONE:
                main_rows.append((node, main_row))
            q = t * lanes + w
            dur = lat[q][lv.astype(np.int64) & mask].astype(np.int64)
            start = h[w].copy() if flags & REGPRED else np.zeros(B, dtype=np.int64)
            ops |= ops_hi << 32
            settled = ((flags >> 4) & 7) > 0
            for k in range((flags >> 4) & 7):
                s = (ops >> (8 * k)) & 255
                settled = settled and write_step[s] // sync < t // sync
                assert slot_valid[s], f"step {t} lane {w} reads slot {s} before any write"
                # the parity in the entry names the value that is in the slot now
                assert ((flags >> (25 + k)) & 1) == (n_written[s] - 1) % 2, f"step {t} lane {w}: operand parity"
                last_read[s] = t
                read_ids.add(s)
                start = np.maximum(start, slot[s])
            # word 6: every slot operand was written before the group's last barrier
            assert (int(entries[t, w][6]) & 1) == int(settled), f"step {t} lane {w}: settled flag"
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
            writes.append((w, val, (flags >> 16) & 255 if flags & WRITE else None))
        for w, val, s in writes:
            h[w] = val
            if s is not None:
                assert s not in read_ids, f"step {t}: slot {s} read and written in the same step"
                # between barriers the warps drift: the last read must lie in an earlier block
                assert last_read[s] < 0 or last_read[s] // sync < t // sync, \
                    f"step {t}: slot {s} rewritten in the block of its last read"
                assert ((int(entries[t, w, 1]) >> 24) & 1) == n_written[s] % 2, f"step {t} lane {w}: write parity"
                n_written[s] += 1
                slot[s] = val
                slot_valid[s] = True
                write_step[s] = t
    out["seen"] = seen
    out["main_rows"] = main_rows
    if not backward:
        out["T"], out["ES"] = T, ES
    else:
        out["LS"], out["slack"] = LS, SL
    return out
