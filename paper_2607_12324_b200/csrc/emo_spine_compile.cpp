// Back-end for spine programs (see emo_flow.h): segments, the spine's operations per direction with
// their value slots, the segment and member lists of the storing warps.
#include <algorithm>
#include <cstring>

#include "../../include/emo.h"
#include "emo_flow.h"

namespace emo {

namespace {

struct Seg {
    int32_t stage = 0, lane = 0, first = 0, count = 0, head = -1, tail = -1;
    uint32_t flags = 0;
    uint32_t acc = 0;         // word offset of the segment's sum inside the stage's sums
    int32_t idx = 0;          // index inside its stage (forward order)
    int32_t push = -1;        // restore row inside the stage, -1: the head's start follows from the lane's value
    int32_t pubF = -1, pubB = -1, readersF = 0, readersB = 0;
};

// Free list of slot numbers; slots [0, fixed) are never handed out.
struct SlotPool {
    std::vector<int32_t> free_ids;
    int32_t next = 0;
    int32_t take()
    {
        if (!free_ids.empty()) {
            const int32_t id = free_ids.back();
            free_ids.pop_back();
            return id;
        }
        return next++;
    }
    void give(int32_t id) { free_ids.push_back(id); }
};

struct Operand {
    uint32_t slot, delta;
    bool clear;
};

}  // namespace

int build_spine(const SpineIn &in, Spine &out, std::string &err)
{
    out = Spine();
    const int32_t n = in.n;
    const int lanes = in.lanes, K = in.K, stages = in.stages, L = in.L;
    const auto &pp = *in.pp, &sp = *in.sp;
    const auto &pc = *in.pc, &sc = *in.sc;
    const auto &liveF = *in.liveF, &liveB = *in.liveB, &constant = *in.constant;
    const auto &lbES = *in.lbES, &lbC = *in.lbC, &lbQin = *in.lbQin, &lbQ = *in.lbQ;
    const auto &step_of = *in.step_of, &lane_of = *in.lane_of, &prev = *in.prev_on_lane, &next = *in.next_on_lane, &pos_of = *in.pos_of;
    if (n == 0 || stages == 0) return EMO_OK;
    if (lanes > 255 || K > 255) return EMO_OK;
    auto stage_of = [&](int32_t v) { return step_of[v] / K; };

    // ---- what every node's live edges ask of it ---------------------------------------------------
    std::vector<int32_t> nFin((size_t)n, 0), nBout((size_t)n, 0), fold_reader((size_t)n, -1);
    std::vector<char> linkF((size_t)n, 0), linkB((size_t)n, 0), fpub((size_t)n, 0), bpub((size_t)n, 0);
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
            const int32_t k = pc[e];
            const bool lane_link = prev[v] == k;
            if (liveF[e]) {
                nFin[v]++;
                if (lane_link) linkF[v] = 1;
                else fpub[k] = 1;                    // k's completion is read off its lane: k ends a segment
            }
            if (liveB[e]) {
                nBout[k]++;
                if (lane_link) {
                    linkB[v] = 1;
                } else if (fold_reader[v] < 0 && stage_of(v) >= stage_of(k) + 2) {
                    fold_reader[v] = k;              // v's tail is folded into a slot of k by the storing warps
                } else {
                    bpub[v] = 1;                     // v's tail is read off its lane: v begins a segment
                }
            }
        }
    auto invertible = [&](int32_t v) { return linkF[v] && nFin[v] == 1 && lbES[v] == lbC[prev[v]]; };
    auto pure_link = [&](int32_t v) {
        const int32_t p = prev[v];
        return p >= 0 && stage_of(p) == stage_of(v) && linkF[v] && linkB[v] && nFin[v] == 1 && nBout[p] == 1 && !fpub[p] && !bpub[v] &&
               lbES[v] == lbC[p] && lbQin[p] == lbQ[v];
    };

    // ---- segments -----------------------------------------------------------------------------------
    std::vector<int32_t> by_step((size_t)n);
    for (int32_t v = 0; v < n; ++v) by_step[v] = v;
    std::sort(by_step.begin(), by_step.end(), [&](int32_t a, int32_t b) {
        return step_of[a] != step_of[b] ? step_of[a] < step_of[b] : lane_of[a] < lane_of[b];
    });
    std::vector<Seg> segs;
    std::vector<int32_t> seg_of((size_t)n, -1);
    {
        std::vector<int32_t> open((size_t)lanes, -1);      // the lane's current segment
        for (int32_t v : by_step) {
            const int ln = lane_of[v];
            if (open[ln] >= 0 && pure_link(v) && segs[open[ln]].tail == prev[v]) {
                Seg &s = segs[open[ln]];
                s.count++;
                s.tail = v;
            } else {
                Seg s;
                s.stage = stage_of(v);
                s.lane = ln;
                s.first = pos_of[v];
                s.count = 1;
                s.head = s.tail = v;
                open[ln] = (int32_t)segs.size();
                segs.push_back(s);
            }
            seg_of[v] = open[ln];
            Seg &s = segs[open[ln]];
            bool has_energy = false;
            for (int l = 0; l < L; ++l) has_energy = has_energy || in.energy[(size_t)v * L + l] != 0.0;
            if (!constant[v]) s.flags |= kSpSeg_PreF | kSpSeg_PreB;
            else if (has_energy) s.flags |= kSpSeg_PreF;
            if (fold_reader[v] >= 0) s.flags |= kSpSeg_Fold;
        }
    }
    out.segments = (int64_t)segs.size();
    // per stage, in forward order (by the head's step, then lane): index and sum offset
    std::vector<std::vector<int32_t>> stage_segs((size_t)stages);
    for (size_t i = 0; i < segs.size(); ++i) stage_segs[segs[i].stage].push_back((int32_t)i);
    int max_segs = 0, acc_words = 0;
    for (int st = 0; st < stages; ++st) {
        auto &ss = stage_segs[st];
        std::sort(ss.begin(), ss.end(), [&](int32_t a, int32_t b) {
            const int32_t ha = segs[a].head, hb = segs[b].head;
            return step_of[ha] != step_of[hb] ? step_of[ha] < step_of[hb] : segs[a].lane < segs[b].lane;
        });
        uint32_t off = 0;
        for (size_t i = 0; i < ss.size(); ++i) {
            Seg &s = segs[ss[i]];
            s.idx = (int32_t)i;
            s.acc = off;
            off += (s.flags & kSpSeg_Fold) ? 2u : 1u;      // the sum, then X; beside it the head's tail where members are folded
        }
        max_segs = std::max(max_segs, (int)ss.size());
        acc_words = std::max(acc_words, (int)off);
    }
    out.max_segs = max_segs;
    out.acc_words = acc_words + 2;      // two scratch words behind the stage's sums (merge operations write there)
    out.acc_words_all = out.acc_words + max_segs;      // with the heads' tails of all segments behind them (calls that want ES / LS / sums)
    const uint32_t scratch_acc = (uint32_t)acc_words;

    // ---- segment and member lists ---------------------------------------------------------------------
    out.n_segs.assign((size_t)stages, 0);
    out.seg.assign((size_t)stages * std::max(max_segs, 1) * kSpSegWords, 0);
    out.mem.assign((size_t)stages * lanes * K * kSpMemWords, 0);
    out.posw.assign((size_t)stages * lanes * K, 0);
    const uint32_t zero_slot = (uint32_t)lanes, dummy_slot = (uint32_t)lanes + 1u;
    auto slot_addr = [](uint32_t id) { return id * 128u; };
    if (max_segs >= 4096 || acc_words + 2 >= 65536) return EMO_OK;      // the position word has no room: no spine program
    // unused positions: no node, folds go to the slot nobody reads
    for (size_t q = 0; q < (size_t)stages * lanes * K; ++q) {
        out.mem[q * kSpMemWords + 0] = kNone;
        out.mem[q * kSpMemWords + 1] = slot_addr(dummy_slot);
        out.posw[q] = (uint32_t)(acc_words) << 16;      // sums of unused positions go to the scratch word
        out.mem[q * kSpMemWords + 3] = out.posw[q];
    }
    for (int st = 0; st < stages; ++st) {
        out.n_segs[st] = (uint32_t)stage_segs[st].size();
        for (int32_t si : stage_segs[st]) {
            const Seg &s = segs[si];
            uint32_t *w = &out.seg[((size_t)st * max_segs + s.idx) * kSpSegWords];
            const int64_t A = lbQ[s.head] + lbES[s.head];
            w[0] = (uint32_t)s.lane | ((uint32_t)s.first << 8) | ((uint32_t)s.count << 16) | (s.flags << 24);
            w[1] = s.acc * 128u;
            w[2] = (uint32_t)(uint64_t)A;
            w[3] = (uint32_t)((uint64_t)A >> 32);
            for (int32_t j = 0; j < s.count; ++j) {
                const size_t q = ((size_t)st * lanes + s.lane) * K + s.first + j;
                const uint32_t pw = (j == 0 ? kSpPos_First : 0u) | (j == s.count - 1 ? kSpPos_Last : 0u) | ((uint32_t)s.idx << 4) | (s.acc << 16);
                out.posw[q] = pw;
                out.mem[q * kSpMemWords + 3] = pw;
                out.mem[q * kSpMemWords + 4] = w[2];
                out.mem[q * kSpMemWords + 5] = w[3];
            }
        }
    }

    // ---- forward operations -----------------------------------------------------------------------------
    // fixed slots: the lanes' values, a slot that stays zero, a slot nobody reads; published values behind them
    // restore rows in the numbering of the lane-stream program to pair with: nodes whose start does not follow from the
    // lane's value, per stage of pair_K steps the lanes in order, a lane's nodes by step
    std::vector<int64_t> pair_row((size_t)n, -1);
    out.pair_K = in.pair_K;
    out.pair_ok = in.pair_K > 0;
    out.pair_base.assign((size_t)stages, 0);
    if (in.pair_K > 0) {
        std::vector<int32_t> pushing;
        for (int32_t v = 0; v < n; ++v)
            if (!invertible(v)) pushing.push_back(v);
        std::sort(pushing.begin(), pushing.end(), [&](int32_t a, int32_t b) {
            const int sa = step_of[a] / in.pair_K, sb = step_of[b] / in.pair_K;
            if (sa != sb) return sa < sb;
            if (lane_of[a] != lane_of[b]) return lane_of[a] < lane_of[b];
            return step_of[a] < step_of[b];
        });
        for (size_t i = 0; i < pushing.size(); ++i) pair_row[pushing[i]] = (int64_t)i;
        std::vector<int64_t> lo((size_t)stages, -1);
        for (int32_t v : pushing) {
            const int st = stage_of(v);
            if (lo[st] < 0 || pair_row[v] < lo[st]) lo[st] = pair_row[v];
        }
        for (int st = 0; st < stages; ++st) out.pair_base[st] = lo[st] < 0 ? 0 : lo[st];
    }
    std::vector<std::vector<uint32_t>> opsF((size_t)stages), opsB((size_t)stages);
    std::vector<std::vector<uint64_t>> pools((size_t)stages);
    out.push_base.assign((size_t)stages + 1, 0);
    {
        SlotPool pool;
        pool.next = lanes + 2;
        // readers of every published completion
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e)
                if (liveF[e] && prev[v] != pc[e]) segs[seg_of[pc[e]]].readersF++;
        for (int st = 0; st < stages; ++st) {
            int32_t npush = 0;
            for (int32_t si : stage_segs[st]) {
                Seg &s = segs[si];
                const int32_t h = s.head, t = s.tail;
                const bool terminal = sp[t + 1] == sp[t];
                const bool inv = invertible(h);
                if (!inv) s.push = npush++;
                if (inv && !(s.flags & kSpSeg_PreB) && !fpub[t] && !terminal) continue;      // the lane's value passes through unchanged
                std::vector<Operand> ops;
                std::vector<int32_t> done;       // published slots whose last reader this is
                // the lane's slot is always the first operand of the segment's own operation (the kernel takes the value
                // that goes to the restore list from there); a correction of 2^32 - 1 floors it to zero when the head
                // does not continue from the lane
                Operand lane_op{(uint32_t)s.lane, 0xFFFFFFFFu, false};
                for (int64_t e = pp[h]; e < pp[h + 1]; ++e) {
                    if (!liveF[e]) continue;
                    const int32_t k = pc[e];
                    const uint32_t delta = (uint32_t)(lbES[h] - lbC[k]);
                    if (prev[h] == k) {
                        lane_op.delta = delta;
                    } else {
                        Seg &w = segs[seg_of[k]];
                        if (w.tail != k || w.pubF < 0) { err = "internal: spine operand is not published"; return EMO_E_UNSUPPORTED; }
                        ops.push_back(Operand{(uint32_t)w.pubF, delta, false});
                        if (--w.readersF == 0) done.push_back(w.pubF);
                    }
                }
                std::vector<int32_t> temps;
                while (ops.size() > 1) {
                    const int32_t tmp = pool.take();
                    temps.push_back(tmp);
                    const uint32_t w8[kSpOpWordsF] = {slot_addr(ops[0].slot), ops[0].delta, slot_addr(ops[1].slot), ops[1].delta,
                                                      slot_addr(dummy_slot), slot_addr((uint32_t)tmp), scratch_acc * 128u, kSp_NoSum};
                    opsF[st].insert(opsF[st].end(), w8, w8 + kSpOpWordsF);
                    ops.erase(ops.begin(), ops.begin() + 2);
                    ops.insert(ops.begin(), Operand{(uint32_t)tmp, 0u, false});
                }
                if (ops.empty()) ops.push_back(Operand{zero_slot, 0u, false});
                ops.insert(ops.begin(), lane_op);
                if (fpub[t] && s.readersF > 0) s.pubF = pool.take();
                uint32_t fl = (s.flags & kSpSeg_PreB) ? 0u : kSp_NoSum;
                if (!inv) {
                    fl |= kSp_Push | ((uint32_t)s.push << 8);
                    if (in.pair_K > 0) {
                        const int64_t rel = pair_row[h] - out.pair_base[st];
                        if (rel < 0 || rel >= 4096) out.pair_ok = false;
                        else fl |= (uint32_t)rel << 20;
                    }
                }
                if (terminal) {
                    fl |= kSp_Terminal;      // the kernel takes the stage's bounds in order
                    pools[st].push_back((uint64_t)lbC[t]);
                }
                if (s.push >= 4096 || pools[st].size() >= 4096) { err = "internal: spine stage too large"; return EMO_E_UNSUPPORTED; }
                const uint32_t w8[kSpOpWordsF] = {slot_addr(ops[0].slot), ops[0].delta, slot_addr(ops[1].slot), ops[1].delta,
                                                  slot_addr((uint32_t)s.lane), slot_addr(s.pubF >= 0 ? (uint32_t)s.pubF : dummy_slot), s.acc * 128u, fl};
                opsF[st].insert(opsF[st].end(), w8, w8 + kSpOpWordsF);
                for (int32_t id : temps) pool.give(id);
                for (int32_t id : done) pool.give(id);
            }
            out.push_base[st + 1] = out.push_base[st] + npush;
        }
        out.f.slots = pool.next;
    }
    out.pushes = out.push_base[stages];

    // ---- backward operations ----------------------------------------------------------------------------
    // fixed slots: the lanes' tails, zero, unread, the lanes' completion offsets, an unread one of those
    {
        // Fold slots are numbered apart from the others (tagged with the top bit until the count of the others
        // is known): a free one always holds zero, because its reader clears it.
        SlotPool pool, fpool;
        const uint32_t c_slot0 = (uint32_t)lanes + 2u, dummy_c = 2u * (uint32_t)lanes + 2u;
        const uint32_t kFoldTag = 0x80000000u;
        pool.next = 2 * lanes + 3;
        std::vector<int32_t> fold_slot((size_t)n, -1);
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e)
                if (liveB[e] && prev[v] != pc[e] && fold_reader[v] != pc[e]) segs[seg_of[v]].readersB++;
        for (int st = stages - 1; st >= 0; --st) {
            std::vector<int32_t> order(stage_segs[st]);
            std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
                const int32_t ta = segs[a].tail, tb = segs[b].tail;
                return step_of[ta] != step_of[tb] ? step_of[ta] > step_of[tb] : segs[a].lane < segs[b].lane;
            });
            for (int32_t si : order) {
                Seg &s = segs[si];
                const int32_t h = s.head, t = s.tail;
                // the members' records; a fold slot is taken when its first writer comes by
                {
                    int32_t u = h;
                    for (int32_t j = 0; j < s.count; ++j, u = next[u]) {
                        uint32_t *w = &out.mem[(((size_t)st * lanes + s.lane) * K + s.first + j) * kSpMemWords];
                        w[0] = (uint32_t)u;
                        w[1] = slot_addr(dummy_slot);
                        w[6] = (uint32_t)(uint64_t)lbES[u];
                        w[7] = (uint32_t)((uint64_t)lbES[u] >> 32);
                        const int32_t r = fold_reader[u];
                        if (r >= 0) {
                            if (fold_slot[r] < 0) fold_slot[r] = fpool.take();
                            w[1] = kFoldTag | slot_addr((uint32_t)fold_slot[r]);
                            w[2] = (uint32_t)(lbQin[r] - lbQ[u]);
                        }
                    }
                }
                std::vector<Operand> ops;
                std::vector<int32_t> done;
                bool fold_seen = false;
                for (int64_t e = sp[t]; e < sp[t + 1]; ++e) {
                    const int32_t u = sc[e];
                    const int64_t ee = std::lower_bound(pc.begin() + pp[u], pc.begin() + pp[u + 1], t) - pc.begin();
                    if (!liveB[ee]) continue;
                    const uint32_t delta = (uint32_t)(lbQin[t] - lbQ[u]);
                    if (next[t] == u) {
                        ops.insert(ops.begin(), Operand{(uint32_t)s.lane, delta, false});
                    } else if (fold_reader[u] == t) {
                        if (fold_seen) continue;
                        fold_seen = true;
                        if (fold_slot[t] < 0) { err = "internal: spine fold slot missing"; return EMO_E_UNSUPPORTED; }
                        ops.push_back(Operand{kFoldTag | slot_addr((uint32_t)fold_slot[t]), 0u, true});
                    } else {
                        Seg &w = segs[seg_of[u]];
                        if (w.head != u || w.pubB < 0) { err = "internal: spine tail is not published"; return EMO_E_UNSUPPORTED; }
                        ops.push_back(Operand{(uint32_t)w.pubB, delta, false});
                        if (--w.readersB == 0) done.push_back(w.pubB);
                    }
                }
                std::vector<int32_t> temps;
                auto addr_of = [&](const Operand &a) { return a.clear ? a.slot : slot_addr(a.slot); };      // fold operands carry their tagged address
                auto clear_of = [&](const Operand &a, const Operand &b) { return a.clear ? a.slot : (b.clear ? b.slot : slot_addr(dummy_slot)); };
                while (ops.size() > 2) {
                    const int32_t tmp = pool.take();
                    temps.push_back(tmp);
                    const uint32_t w12[kSpOpWordsB] = {addr_of(ops[0]), ops[0].delta, addr_of(ops[1]), ops[1].delta,
                                                       slot_addr(dummy_slot), slot_addr((uint32_t)tmp), scratch_acc * 128u, kSp_NoSum,
                                                       clear_of(ops[0], ops[1]), slot_addr(dummy_c), (scratch_acc + 1u) * 128u, (scratch_acc + 1u) * 128u};
                    opsB[st].insert(opsB[st].end(), w12, w12 + kSpOpWordsB);
                    ops.erase(ops.begin(), ops.begin() + 2);
                    ops.insert(ops.begin(), Operand{(uint32_t)tmp, 0u, false});
                }
                while (ops.size() < 2) ops.push_back(Operand{zero_slot, 0u, false});
                if (bpub[h] && s.readersB > 0) s.pubB = pool.take();
                uint32_t fl = (s.flags & kSpSeg_PreB) ? 0u : kSp_NoSum;
                if (s.push >= 0) fl |= kSp_Push | ((uint32_t)s.push << 8);
                const bool wide = (s.flags & kSpSeg_Fold) != 0;
                const uint32_t w12[kSpOpWordsB] = {addr_of(ops[0]), ops[0].delta, addr_of(ops[1]), ops[1].delta,
                                                   slot_addr((uint32_t)s.lane), slot_addr(s.pubB >= 0 ? (uint32_t)s.pubB : dummy_slot), s.acc * 128u, fl,
                                                   clear_of(ops[0], ops[1]), slot_addr(c_slot0 + (uint32_t)s.lane),
                                                   (wide ? s.acc + 1u : scratch_acc + 1u) * 128u,
                                                   ((uint32_t)out.acc_words + (uint32_t)s.idx) * 128u};
                opsB[st].insert(opsB[st].end(), w12, w12 + kSpOpWordsB);
                for (int32_t id : temps) pool.give(id);
                for (int32_t id : done) pool.give(id);
                if (fold_seen) fpool.give(fold_slot[t]);
            }
        }
        // fold slots follow the others
        const uint32_t base = (uint32_t)pool.next * 128u;
        auto fix = [&](uint32_t &w) {
            if (w & kFoldTag) w = (w & ~kFoldTag) + base;
        };
        for (auto &o : opsB)
            for (size_t i = 0; i + kSpOpWordsB <= o.size(); i += kSpOpWordsB) {
                fix(o[i + 0]);
                fix(o[i + 2]);
                fix(o[i + 8]);
            }
        for (size_t i = 0; i + kSpMemWords <= out.mem.size(); i += kSpMemWords) fix(out.mem[i + 1]);
        out.b.slots = pool.next + fpool.next;
    }

    // ---- pack --------------------------------------------------------------------------------------------
    auto pack = [&](std::vector<std::vector<uint32_t>> &src, SpineDir &d, int words) {
        size_t mx = 1;
        for (auto &o : src) mx = std::max(mx, o.size() / words);
        d.max_ops = (int)mx;
        d.n_ops.assign((size_t)stages, 0);
        d.ops.assign((size_t)stages * mx * words, 0);
        for (int st = 0; st < stages; ++st) {
            d.n_ops[st] = (uint32_t)(src[st].size() / words);
            std::copy(src[st].begin(), src[st].end(), d.ops.begin() + (size_t)st * mx * words);
        }
    };
    pack(opsF, out.f, kSpOpWordsF);
    pack(opsB, out.b, kSpOpWordsB);
    size_t mp = 1;
    for (auto &p : pools) mp = std::max(mp, p.size());
    out.max_pool = (int)mp;
    out.pool.assign((size_t)stages * mp, 0);
    for (int st = 0; st < stages; ++st) std::copy(pools[st].begin(), pools[st].end(), out.pool.begin() + (size_t)st * mp);
    out.ok = true;
    return EMO_OK;
}

}  // namespace emo
