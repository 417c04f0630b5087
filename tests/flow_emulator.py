"""Host-side interpreter of the lane-stream program (emo_graph_flow), for tests of the compiler.

It follows the rules of the 32-bit pass kernels literally - unsigned 32-bit offsets, corrections
floored at zero, tagged and settled exchange slots, the restore list, recovery of completion offsets
by subtraction in the backward walk - but runs the entries of a period in step order on the host,
vectorised over policies with numpy.  It checks what the kernels rely on: a tagged slot read finds
the tag it expects, a settled slot was written in an earlier period, a slot is not overwritten while
a reader of the old value is still to come in the same period.
"""
from __future__ import annotations

import numpy as np

NONE = 0xFFFFFFFF
SEG_SPECIAL, SEG_BARRIER, SEG_IN, SEG_OUT = 16, 32, 64, 128
B_SIMPLE = 64
F_HASREG, F_REGDELTA, F_OUTTAG, F_OUTSET, F_TERMINAL, F_PUSH, F_OUTACC = 1 << 8, 1 << 9, 1 << 10, 1 << 11, 1 << 12, 1 << 13, 1 << 14
B_HASREG, B_REGDELTA, B_OUTTAG, B_OUTSET, B_POP, B_OUTACC = 1, 2, 4, 8, 16, 32
OP_NOPOLL, OP_WORD, OP_CLEAR, OP_OFF = 1 << 31, 1 << 30, 1 << 29, (1 << 29) - 1


def _floor_sub(x, d):
    return np.maximum(x, np.uint32(d)) - np.uint32(d)


class _Slots:
    def __init__(self, B):
        self.val, self.tag, self.period = {}, {}, {}
        self.B = B

    def read(self, w, tag, period_now):
        off = int(w & OP_OFF)
        assert off in self.val, "slot read before any write"
        if not (w & OP_CLEAR):
            assert self.tag[off] == tag, f"slot {off}: found tag {self.tag[off]}, expected {tag}"
        if w & OP_NOPOLL:
            assert self.period[off] < period_now, "a read without polling needs a barrier after the write"
        x = self.val[off].copy()
        if w & OP_CLEAR:
            self.val[off] = np.zeros(self.B, np.uint32)
        return x

    def write(self, off, x, tag, period_now, acc):
        off = int(off)
        if acc:
            # folded in with a maximum, whatever the slot holds (the kernels zero all slots at the start)
            assert self.tag.get(off, "acc") == "acc", "a shared slot must only ever hold running maxima"
            self.val[off] = np.maximum(self.val.get(off, np.zeros(self.B, np.uint32)), x)
        else:
            assert self.tag.get(off) != "acc", "a plain value must not land in a shared slot"
            self.val[off] = x.copy()
        self.tag[off] = "acc" if acc else tag
        self.period[off] = period_now


def _period_entries(f, st, p, reverse):
    """(step, lane, pos) of the entries of period p of stage st, in processing order."""
    out = []
    for ln in range(f["lanes"]):
        for pos in range(f["K"]):
            if int(f["node"][st, ln, pos]) == NONE:
                break
            step = int(f["step"][st, ln, pos])
            if (step % f["K"]) // f["sync"] == p:
                out.append((step, ln, pos))
    out.sort(reverse=reverse)
    return out


def segments(f, st, ln, backward):
    """The segments of one lane of one stage as (barrier, special position or None, run positions, kind bits)."""
    seg = f["seg_bwd" if backward else "seg_fwd"][st, ln]
    h0 = int(f["hdr"][st, ln, 0])
    nseg, total = (h0 >> 8) & 255 if backward else h0 & 255, (h0 >> 16) & 255
    pos = total if backward else 0
    out = []
    for i in range(nseg):
        b = int(seg[i])
        special = None
        if b & SEG_SPECIAL:
            if backward:
                pos -= 1
                special = pos
            else:
                special = pos
                pos += 1
        r = b & 15
        if backward:
            run = list(range(pos - 1, pos - 1 - r, -1))
            pos -= r
        else:
            run = list(range(pos, pos + r))
            pos += r
        out.append((bool(b & SEG_BARRIER), special, run, b & (SEG_IN | SEG_OUT)))
    assert pos == (0 if backward else total)
    return out


def run_forward(f, lvl, L):
    """lvl: uint8 [rows][B].  Returns makespan int64 [B], energy float64 [B], restore uint32 [pushes+lanes][B]."""
    B = lvl.shape[1]
    lanes, K, nper = f["lanes"], f["K"], f["K"] // f["sync"]
    h = np.zeros((lanes, B), np.uint32)
    ea = np.zeros((lanes, B), np.float64)
    acc = np.zeros((lanes, B), np.int64)
    restore = np.zeros((int(f["pushes"]) + lanes, B), np.uint32)
    slots = _Slots(B)
    cols = np.arange(B)
    for st in range(f["stages"]):
        npushed = [0] * lanes
        for p in range(nper):
            period = st * nper + p
            for _, ln, pos in _period_entries(f, st, p, False):
                rec = f["rec_fwd"][st, ln, pos]
                fl = int(rec[0])
                row = int(f["rows"][st, ln, pos])
                l = lvl[row] if row != NONE else np.zeros(B, np.uint8)
                assert row == NONE or int(l.max()) < L
                tab = f["tab_fwd"][st, ln, pos]
                doff = tab[l, 0]
                e = ((tab[l, 1].astype(np.uint64) << np.uint64(32)) | tab[l, 2].astype(np.uint64)).view(np.float64)
                pool = f["pool_fwd"][st]
                pp = int(rec[3])
                hin = h[ln].copy()
                v = hin.copy() if fl & F_HASREG else np.zeros(B, np.uint32)
                assert bool(fl & F_REGDELTA) == (int(rec[7]) != 0)
                v = _floor_sub(v, rec[7])
                for k in range(fl >> 16):
                    if k == 0:      # the first operand sits in the record
                        w, tag, delta = int(rec[4]), int(rec[5]), int(rec[6])
                    else:
                        w, tag, delta = int(pool[pp]), int(pool[pp + 1]), int(pool[pp + 2])
                        pp += 3
                    v = np.maximum(v, _floor_sub(slots.read(w, tag, period), delta))
                if fl & F_PUSH:
                    restore[int(f["push_base"][st]) + int(f["hdr"][st, ln, 5]) + npushed[ln]] = hin
                    npushed[ln] += 1
                else:
                    assert (fl & F_HASREG) and not (fl & F_REGDELTA) and (fl >> 16) == 0
                ea[ln] += e
                v = v + doff
                if fl & F_OUTTAG:
                    slots.write(rec[1], v, int(rec[2]), period, False)
                if fl & F_OUTSET:
                    slots.write(rec[1], _floor_sub(v, rec[2]), int(st * lanes * K + ln * K + pos + 1), period, bool(fl & F_OUTACC))
                if fl & F_TERMINAL:
                    lbc = int(pool[pp]) | (int(pool[pp + 1]) << 32)
                    acc[ln] = np.maximum(acc[ln], lbc + v.astype(np.int64))
                h[ln] = v
        for ln in range(lanes):
            assert npushed[ln] == int(f["hdr"][st, ln, 4])
    for ln in range(lanes):
        restore[int(f["pushes"]) + ln] = h[ln]
    del cols
    return acc.max(axis=0), ea.sum(axis=0) if lanes else np.zeros(B), restore


def run_backward(f, lvl, L, T, restore, n):
    """Returns ES, LS, slack int64 [n][B]."""
    B = lvl.shape[1]
    lanes, K, nper = f["lanes"], f["K"], f["K"] // f["sync"]
    q = np.zeros((lanes, B), np.uint32)
    c = np.stack([restore[int(f["pushes"]) + ln] for ln in range(lanes)]) if lanes else np.zeros((0, B), np.uint32)
    ES = np.zeros((n, B), np.int64)
    LS = np.zeros((n, B), np.int64)
    SL = np.zeros((n, B), np.int64)
    slots = _Slots(B)
    T = T.astype(np.int64)
    for st in range(f["stages"] - 1, -1, -1):
        npop = [int(f["hdr"][st, ln, 4]) for ln in range(lanes)]
        for p in range(nper - 1, -1, -1):
            period = (f["stages"] * nper - 1) - (st * nper + p)
            for _, ln, pos in _period_entries(f, st, p, True):
                rec = f["rec_bwd"][st, ln, pos]
                fl = int(rec[0])
                row = int(f["rows"][st, ln, pos])
                l = lvl[row] if row != NONE else np.zeros(B, np.uint8)
                doff = f["tab_bwd"][st, ln, pos][l]
                pool = f["pool_bwd"][st]
                pp = int(rec[3])
                qin = q[ln].copy() if fl & B_HASREG else np.zeros(B, np.uint32)
                assert bool(fl & B_REGDELTA) == (int(rec[7]) != 0)
                qin = _floor_sub(qin, rec[7])
                if fl & B_SIMPLE:
                    # a simple entry: at most one operand, a settled single-reader slot named in word 3
                    assert (fl & B_HASREG) and not (fl & B_OUTTAG) and (fl >> 16) <= 1
                    if fl >> 16:
                        qin = np.maximum(qin, slots.read(OP_WORD | OP_NOPOLL | OP_CLEAR | int(rec[3]), None, period))
                else:
                    for k in range(fl >> 16):
                        if k < 2:      # the first two operands sit in the record
                            w, tag, delta = int(rec[8 + 4 * k]), int(rec[9 + 4 * k]), int(rec[10 + 4 * k])
                        else:
                            w, tag, delta = int(pool[pp]), int(pool[pp + 1]), int(pool[pp + 2])
                            pp += 3
                        qin = np.maximum(qin, _floor_sub(slots.read(w, tag, period), delta))
                A = int(rec[4]) | (int(rec[5]) << 32)
                v = int(rec[6])
                sl = T - A - (qin.astype(np.int64) + c[ln].astype(np.int64))
                qn = qin + doff
                if fl & B_OUTTAG:
                    slots.write(rec[1], qn, int(rec[2]), period, False)
                if fl & B_OUTSET:
                    slots.write(rec[1], _floor_sub(qn, rec[2]), int(st * lanes * K + ln * K + pos + 1), period, bool(fl & B_OUTACC))
                eo = c[ln] - doff
                es = int(f["lbes"][st, ln, pos]) + eo.astype(np.int64)
                SL[v], ES[v], LS[v] = sl, es, sl + es
                if fl & B_POP:
                    npop[ln] -= 1
                    c[ln] = restore[int(f["push_base"][st]) + int(f["hdr"][st, ln, 5]) + npop[ln]]
                else:
                    c[ln] = eo
                q[ln] = qn
        assert all(x == 0 for x in npop)
    return ES, LS, SL
