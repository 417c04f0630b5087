"""Host-side interpreter of the spine program (the form of the schedule that the spine kernels walk), in numpy,
vectorised over the policies.  It follows the kernels' division of work: per stage the sums per segment (one
stream of positions per lane), then the spine's operations in order, then - backward - the stores per position
(slack, ES, LS, folds).  `late_stores=True` delays a stage's stores until just before the spine starts the
stage two further on, the latest the kernels allow; the results must not depend on it."""
from __future__ import annotations

import numpy as np

NONE = 0xFFFFFFFF
M32 = np.uint64(0xFFFFFFFF)


def _fs(x, d):
    """floor_sub: max(x, d) - d on unsigned 32-bit values held in uint64."""
    d = np.uint64(d)
    return np.maximum(x, d) - d


def run(view: dict, lv: np.ndarray, L: int, late_stores: bool = False) -> dict:
    """lv: [rows][B] levels.  Returns makespan, energy, slack / ES / LS [n][B] (n = largest node id + 1)."""
    st_n, lanes, K, Lp = view["stages"], view["lanes"], view["K"], view["Lp"]
    B = lv.shape[1]
    lmask = Lp - 1
    n = int(view["mem"][:, :, 0][view["mem"][:, :, 0] != NONE].max()) + 1 if (view["mem"][:, :, 0] != NONE).any() else 0
    cols = np.arange(B)

    def levels(st, q):
        row = int(view["rows"][st, q])
        if row == NONE:
            return np.zeros(B, dtype=np.int64)
        return (lv[row].astype(np.int64) & lmask)

    # ---- forward ----------------------------------------------------------------------------------------
    slots = np.zeros((view["slots_fwd"], B), dtype=np.uint64)
    restore = np.zeros((int(view["pushes"]) + lanes, B), dtype=np.uint64)
    T = np.zeros(B, dtype=np.int64)
    E = np.zeros(B, dtype=np.float64)
    acc = np.zeros((view["acc_words"], B), dtype=np.uint64)
    for st in range(st_n):
        for ln in range(lanes):
            runsum = np.zeros(B, dtype=np.uint64)
            for pos in range(K):
                q = ln * K + pos
                pw = int(view["pos"][st, q])
                l = levels(st, q)
                tab = view["tab_fwd"][st, q]
                d = tab[l, 0].astype(np.uint64)
                bits = (tab[l, 1].astype(np.uint64) << np.uint64(32)) | tab[l, 2].astype(np.uint64)
                E += bits.view(np.float64)
                runsum = d if (pw & 1) else (runsum + d) & M32
                if pw & 2:
                    acc[pw >> 16] = runsum
        tcount = 0
        for i in range(int(view["n_ops_fwd"][st])):
            a0, d0, a1, d1, o_lane, o_pub, ao, fl = (int(x) for x in view["ops_fwd"][st, i])
            x0, x1 = slots[a0 // 128], slots[a1 // 128]
            S = np.zeros(B, dtype=np.uint64) if (fl & 1) else acc[ao // 128]
            y = (np.maximum(_fs(x0, d0), _fs(x1, d1)) + S) & M32
            if fl & 2:
                restore[int(view["push_base"][st]) + ((fl >> 8) & 0xFFF)] = x0
            if fl & 4:
                T = np.maximum(T, np.int64(view["pool"][st, tcount]) + y.astype(np.int64))
                tcount += 1
            slots[o_lane // 128] = y
            slots[o_pub // 128] = y
    for ln in range(lanes):
        restore[int(view["pushes"]) + ln] = slots[ln]

    # ---- backward ---------------------------------------------------------------------------------------
    slots = np.zeros((view["slots_bwd"], B), dtype=np.uint64)
    for ln in range(lanes):
        slots[lanes + 2 + ln] = restore[int(view["pushes"]) + ln]
    slack = np.full((n, B), -1, dtype=np.int64)
    ES = np.full((n, B), -1, dtype=np.int64)
    LS = np.full((n, B), -1, dtype=np.int64)
    accs = {}

    def stores(st):
        a = accs.pop(st)
        for ln in range(lanes):
            qv = np.zeros(B, dtype=np.uint64)
            for pos in range(K):
                q = ln * K + pos
                node, fold_a, fold_d, pw, A_lo, A_hi, lb_lo, lb_hi = (int(x) for x in view["mem"][st, q])
                X, qh = a[pw >> 16], a[view["acc_words"] + ((pw >> 4) & 0xFFF)]      # the region where every head's tail is kept
                if pw & 1:
                    qv = qh.copy()
                if node != NONE:
                    A = np.int64(A_lo | (A_hi << 32))
                    sl = (T - A) - X.astype(np.int64)
                    es = np.int64(lb_lo | (lb_hi << 32)) + ((X - qv) & M32).astype(np.int64)
                    slack[node], ES[node], LS[node] = sl, es, es + sl
                slots[fold_a // 128] = np.maximum(slots[fold_a // 128], _fs(qv, fold_d))
                d = view["tab_bwd"][st, q][levels(st, q)].astype(np.uint64)
                qv = (qv - d) & M32

    order = list(range(st_n - 1, -1, -1))
    for k, st in enumerate(order):
        a = np.zeros((view["acc_words"] + 4096, B), dtype=np.uint64)
        for ln in range(lanes):
            runsum = np.zeros(B, dtype=np.uint64)
            for pos in range(K):
                q = ln * K + pos
                pw = int(view["mem"][st, q, 3])
                d = view["tab_bwd"][st, q][levels(st, q)].astype(np.uint64)
                runsum = d if (pw & 1) else (runsum + d) & M32
                if pw & 2:
                    a[pw >> 16] = runsum
        if late_stores and k >= 2:
            stores(order[k - 2])          # the spine waits for the stores of the stage two back, no earlier
        for i in range(int(view["n_ops_bwd"][st])):
            a0, d0, a1, d1, o_lane, o_pub, ao, fl, a_clear, c_slot, qo_narrow, qo_off = (int(x) for x in view["ops_bwd"][st, i])
            x0, x1 = slots[a0 // 128], slots[a1 // 128]
            S = np.zeros(B, dtype=np.uint64) if (fl & 1) else a[ao // 128].copy()
            c = slots[c_slot // 128].copy()
            qin = np.maximum(_fs(x0, d0), _fs(x1, d1))
            qo = (qin + S) & M32
            cprev = (c - S) & M32
            if fl & 2:
                rrow = int(view["push_base"][st]) + ((fl >> 8) & 0xFFF)
                cprev = restore[rrow]
            a[ao // 128] = (c + qin) & M32
            a[qo_off // 128] = qo
            a[qo_narrow // 128] = qo      # the place beside X (segments with folded members), else a scratch word
            slots[a_clear // 128] = 0
            slots[o_lane // 128] = qo
            slots[o_pub // 128] = qo
            slots[c_slot // 128] = cprev
        accs[st] = a
        if not late_stores:
            stores(st)
    for st in list(accs):
        stores(st)
    _ = cols
    return {"makespan": T, "energy": E, "slack": slack, "ES": ES, "LS": LS}
