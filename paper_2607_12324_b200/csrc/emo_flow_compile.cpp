// Compiler for lane-stream programs (see emo_flow.h): static bounds, pruning, one schedule for both
// passes, slots per direction, records, operand pools and schedule-ordered tables.
#include <algorithm>
#include <climits>
#include <cstring>
#include <queue>

#include "../../include/emo.h"
#include "emo_flow.h"

namespace emo {

namespace {

struct SlotUse {
    int32_t obj = -1;       // slot object holding the value (-1: the value is read from registers only)
    bool settled = false;   // every slot reader sits behind a barrier: value only, no tag
    bool pre = false;       // settled with one reader: the writer applies the reader's correction
    bool acc = false;       // same as pre: the slot collects a maximum (shared with the reader's other such operands)
    uint32_t pre_delta = 0;
};

// A slot object: one value, or the running maximum of several values that one reader consumes.
struct SlotObj {
    int32_t first = 0, last = 0;   // periods (processing order of the direction) of the first write / last read
    bool settled = false;
    bool acc = false;              // single-reader settled values (slots of their own kind: the reader resets them to 0)
    int32_t id = -1;               // slot number within its kind
};

// Assigns slot numbers.  A slot is free again in the first period after its last read.
void assign_slots(std::vector<SlotObj> &objs, int &n_tag, int &n_set)   // n_set counts both settled kinds
{
    using Key = std::pair<int32_t, int32_t>;
    std::vector<int32_t> order(objs.size());
    for (size_t i = 0; i < objs.size(); ++i) order[i] = (int32_t)i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return objs[a].first < objs[b].first; });
    std::priority_queue<int32_t, std::vector<int32_t>, std::greater<int32_t>> free_ids[3];
    std::priority_queue<Key, std::vector<Key>, std::greater<Key>> busy[3];
    int next_id[3] = {0, 0, 0};
    for (int32_t i : order) {
        const int kind = objs[i].acc ? 2 : (objs[i].settled ? 1 : 0);
        while (!busy[kind].empty() && busy[kind].top().first < objs[i].first) {
            free_ids[kind].push(busy[kind].top().second);
            busy[kind].pop();
        }
        int32_t id;
        if (!free_ids[kind].empty()) {
            id = free_ids[kind].top();
            free_ids[kind].pop();
        } else {
            id = next_id[kind]++;
        }
        objs[i].id = id;
        busy[kind].push({objs[i].last, id});
    }
    n_tag = next_id[0];
    n_set = next_id[1] + next_id[2];
    // shared slots are numbered behind the plain settled ones
    for (SlotObj &o : objs)
        if (o.acc) o.id += next_id[1];
}

}  // namespace

int compile_flow(const HostGraph &g, const int64_t *lat, const double *energy, int lanes, int lookahead, int K, int sync,
                 Flow &out, std::string &err, bool spine, int pair_K)
{
    out = Flow();
    const int32_t n = g.n;
    const int L = g.L;
    int Lp = 4;
    while (Lp < L) Lp <<= 1;
    if (K <= 0) K = 32;
    if (sync <= 0 || sync > K) sync = K;
    if (K > kFlowMaxStage || sync < 1 || K % sync != 0 || K / sync > 4) return EMO_E_INVALID_ARG;
    out.Lp = Lp;
    out.K = K;
    out.sync = sync;
    if (n == 0) return EMO_OK;

    // ---- deduplicated predecessor and successor lists -------------------------------------------
    std::vector<int64_t> pp((size_t)n + 1, 0);
    std::vector<int32_t> pc;
    pc.reserve((size_t)g.m);
    for (int32_t v = 0; v < n; ++v) {
        std::vector<int32_t> p(g.col.begin() + g.row_ptr[v], g.col.begin() + g.row_ptr[v + 1]);
        std::sort(p.begin(), p.end());
        p.erase(std::unique(p.begin(), p.end()), p.end());
        pc.insert(pc.end(), p.begin(), p.end());
        pp[v + 1] = (int64_t)pc.size();
    }
    const int64_t m = (int64_t)pc.size();
    std::vector<int64_t> sp((size_t)n + 1, 0);
    for (int64_t e = 0; e < m; ++e) sp[pc[e] + 1]++;
    for (int32_t v = 0; v < n; ++v) sp[v + 1] += sp[v];
    std::vector<int32_t> sc((size_t)std::max<int64_t>(m, 1));
    {
        std::vector<int64_t> fill(sp.begin(), sp.end() - 1);
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e) sc[fill[pc[e]]++] = v;
    }

    // ---- static bounds --------------------------------------------------------------------------
    std::vector<int64_t> dmin((size_t)n), dmax((size_t)n);
    std::vector<char> constant((size_t)n, 1);
    for (int32_t v = 0; v < n; ++v) {
        int64_t lo = lat[(size_t)v * L], hi = lo;
        if (g.group[v] >= 0) {
            for (int l = 1; l < L; ++l) {
                lo = std::min(lo, lat[(size_t)v * L + l]);
                hi = std::max(hi, lat[(size_t)v * L + l]);
                if (lat[(size_t)v * L + l] != lat[(size_t)v * L] || energy[(size_t)v * L + l] != energy[(size_t)v * L]) constant[v] = 0;
            }
        }
        dmin[v] = lo;
        dmax[v] = hi;
    }
    std::vector<int64_t> lbES((size_t)n, 0), ubES((size_t)n, 0), lbC((size_t)n), ubC((size_t)n);
    std::vector<int32_t> bestF((size_t)n, -1), bestB((size_t)n, -1);
    for (int32_t v = 0; v < n; ++v) {
        for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
            const int32_t k = pc[e];
            ubES[v] = std::max(ubES[v], ubC[k]);
            if (bestF[v] < 0 || lbC[k] > lbC[bestF[v]]) bestF[v] = k;
        }
        if (bestF[v] >= 0) lbES[v] = lbC[bestF[v]];
        lbC[v] = lbES[v] + dmin[v];
        ubC[v] = ubES[v] + dmax[v];
    }
    std::vector<int64_t> lbQin((size_t)n, 0), ubQin((size_t)n, 0), lbQ((size_t)n), ubQ((size_t)n);
    for (int32_t v = n - 1; v >= 0; --v) {
        for (int64_t e = sp[v]; e < sp[v + 1]; ++e) {
            const int32_t u = sc[e];
            ubQin[v] = std::max(ubQin[v], ubQ[u]);
            if (bestB[v] < 0 || lbQ[u] > lbQ[bestB[v]]) bestB[v] = u;
        }
        if (bestB[v] >= 0) lbQin[v] = lbQ[bestB[v]];
        lbQ[v] = lbQin[v] + dmin[v];
        ubQ[v] = ubQin[v] + dmax[v];
    }
    const int64_t kMax32 = 0xFFFFFFFFLL;
    for (int32_t v = 0; v < n; ++v)
        if (ubC[v] - lbC[v] > kMax32 || ubQ[v] - lbQ[v] > kMax32) return EMO_OK;   // ok32 stays false

    // ---- live edges and the schedule ------------------------------------------------------------
    // edge e (k = pc[e] -> v): live forward unless C_k can never exceed the start every policy gives v
    // through its strongest predecessor; live backward under the mirrored test on the tails
    std::vector<char> liveF((size_t)std::max<int64_t>(m, 1), 0), liveB((size_t)std::max<int64_t>(m, 1), 0);
    // An edge that is live in one direction only keeps its two nodes a period apart in the schedule:
    // its reader (in that direction) then finds the value settled behind a barrier instead of polling
    // for it, and nothing waits for the reader in the other direction.  (Typical: a launch node and
    // the kernels it launches - forward the launch never decides a kernel's start, backward the launch
    // node collects its kernels' tails.)  Kept only if it does not stretch the schedule.
    std::vector<std::vector<int32_t>> preds((size_t)n), gaps((size_t)n);
    bool any_gap = false;
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
            const int32_t k = pc[e];
            liveF[e] = (k == bestF[v]) || ubC[k] > lbES[v];
            liveB[e] = (v == bestB[k]) || ubQ[v] > lbQin[k];
            if (!liveF[e]) out.f.pruned++;
            if (!liveB[e]) out.b.pruned++;
            if (liveF[e] || liveB[e]) {
                preds[v].push_back(k);
                gaps[v].push_back(liveF[e] != liveB[e] ? (spine ? 2 * K : sync) : 1);      // spine programs fold such values two stages back
                any_gap = any_gap || liveF[e] != liveB[e];
            }
        }
    std::vector<int32_t> step_of, lane_of, prev_on_lane;
    int32_t S = 0;
    const int lanes_req = lanes;
    int rc = schedule_ops(preds, lanes_req, lookahead, step_of, lane_of, prev_on_lane, S, lanes, err, any_gap ? &gaps : nullptr, false);
    if (rc != EMO_OK) return rc;
    if (any_gap) {
        std::vector<int32_t> s2, l2, p2;
        int32_t S2 = 0;
        int lanes2 = 0;
        rc = schedule_ops(preds, lanes_req, lookahead, s2, l2, p2, S2, lanes2, err, nullptr);
        if (rc != EMO_OK) return rc;
        if ((int64_t)S * 100 > (int64_t)S2 * 105 + 3200) {      // more than 5 % (and 32 steps) longer: not worth it
            step_of.swap(s2);
            lane_of.swap(l2);
            prev_on_lane.swap(p2);
            S = S2;
            lanes = lanes2;
        }
    }
    if (lanes > kFlowMaxLanes) return EMO_OK;
    std::vector<int32_t> next_on_lane((size_t)n, -1);
    for (int32_t v = 0; v < n; ++v)
        if (prev_on_lane[v] >= 0) next_on_lane[prev_on_lane[v]] = v;
    const int stages = (S + K - 1) / K;
    out.lanes = lanes;
    out.steps = S;
    out.stages = stages;
    out.entries = n;

    // ---- positions --------------------------------------------------------------------------------
    // entry of node v: (stage, lane, pos); pos counts the lane's entries inside the stage in step order
    std::vector<int32_t> pos_of((size_t)n, 0);
    std::vector<int32_t> by_step((size_t)n);
    for (int32_t v = 0; v < n; ++v) by_step[v] = v;
    std::sort(by_step.begin(), by_step.end(), [&](int32_t a, int32_t b) {
        return step_of[a] != step_of[b] ? step_of[a] < step_of[b] : lane_of[a] < lane_of[b];
    });
    const size_t Q = (size_t)stages * lanes * K;
    out.hdr.assign((size_t)stages * lanes * kHdrWords, 0);
    out.rows.assign(Q, kNone);
    out.node.assign(Q, kNone);
    out.step.assign(Q, kNone);
    out.lbes.assign(Q, 0);
    out.dmin.assign(Q, 0);
    out.grp.assign(Q, kNone);
    out.tabF.assign(Q * Lp * 3, 0);
    out.tabB.assign(Q * Lp, 0);
    {
        std::vector<int32_t> cnt((size_t)stages * lanes, 0);
        for (int32_t v : by_step) {
            const int st = step_of[v] / K, ln = lane_of[v];
            pos_of[v] = cnt[(size_t)st * lanes + ln]++;
        }
    }
    auto slot_index = [&](int32_t v) { return ((size_t)(step_of[v] / K) * lanes + lane_of[v]) * K + pos_of[v]; };
    auto tag_of = [&](int32_t v) { return (uint32_t)slot_index(v) + 1u; };

    // ---- operands and slots, per direction --------------------------------------------------------
    // forward: value of k is read by v (edge live forward) from the lane's register when k is the
    // entry just before v on v's lane, else from k's slot; backward: value of u is read by v (edge
    // v -> u live backward) from the register when u is the entry just after v on v's lane.
    const int nper = K / sync;
    auto fper = [&](int32_t v) { return step_of[v] / sync; };                      // forward period number
    auto bper = [&](int32_t v) { return (stages * nper - 1) - step_of[v] / sync; };   // backward: later = larger
    std::vector<SlotUse> useF((size_t)n), useB((size_t)n);
    std::vector<SlotObj> objF, objB;
    {
        std::vector<int32_t> lastF((size_t)n, -1), lastB((size_t)n, -1), readersF((size_t)n, 0), readersB((size_t)n, 0);
        std::vector<int32_t> readerF((size_t)n, -1), readerB((size_t)n, -1);     // the (last seen) slot reader of a value
        std::vector<char> allsetF((size_t)n, 1), allsetB((size_t)n, 1);
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
                const int32_t k = pc[e];
                if (liveF[e] && prev_on_lane[v] != k) {
                    lastF[k] = std::max(lastF[k], fper(v));
                    readersF[k]++;
                    readerF[k] = v;
                    if (fper(v) <= fper(k)) allsetF[k] = 0;
                }
                if (liveB[e] && next_on_lane[k] != v) {
                    lastB[v] = std::max(lastB[v], bper(k));
                    readersB[v]++;
                    readerB[v] = k;
                    if (bper(k) <= bper(v)) allsetB[v] = 0;
                }
            }
        // a settled value with one reader is written already corrected for that reader; several such
        // operands of one reader share a slot that holds their running maximum
        std::vector<int32_t> npreF((size_t)n, 0), npreB((size_t)n, 0), accobjF((size_t)n, -1), accobjB((size_t)n, -1);
        for (int32_t v = 0; v < n; ++v) {
            useF[v].settled = lastF[v] >= 0 && allsetF[v];
            useB[v].settled = lastB[v] >= 0 && allsetB[v];
            useF[v].pre = useF[v].settled && readersF[v] == 1;
            useB[v].pre = useB[v].settled && readersB[v] == 1;
            if (useF[v].pre) {
                npreF[readerF[v]]++;
                useF[v].pre_delta = (uint32_t)(lbES[readerF[v]] - lbC[v]);
            }
            if (useB[v].pre) {
                npreB[readerB[v]]++;
                useB[v].pre_delta = (uint32_t)(lbQin[readerB[v]] - lbQ[v]);
            }
        }
        auto build = [&](std::vector<SlotUse> &use, std::vector<SlotObj> &objs, const std::vector<int32_t> &last,
                         const std::vector<int32_t> &reader, const std::vector<int32_t> &npre, std::vector<int32_t> &accobj,
                         bool backward) {
            for (int32_t v = 0; v < n; ++v) {
                if (last[v] < 0) continue;
                const int32_t per = backward ? bper(v) : fper(v);
                if (use[v].pre) {
                    // single-reader settled values live in slots of their own kind, which their reader
                    // resets: the operands of one reader share a slot that collects their maximum
                    const int32_t r = reader[v];
                    use[v].acc = true;
                    if (accobj[r] < 0) {
                        SlotObj o;
                        o.first = per;
                        o.last = backward ? bper(r) : fper(r);
                        o.settled = true;
                        o.acc = true;
                        accobj[r] = (int32_t)objs.size();
                        objs.push_back(o);
                    }
                    objs[accobj[r]].first = std::min(objs[accobj[r]].first, per);
                    use[v].obj = accobj[r];
                } else {
                    SlotObj o;
                    o.first = per;
                    o.last = last[v];
                    o.settled = use[v].settled;
                    use[v].obj = (int32_t)objs.size();
                    objs.push_back(o);
                }
            }
        };
        build(useF, objF, lastF, readerF, npreF, accobjF, false);
        build(useB, objB, lastB, readerB, npreB, accobjB, true);
        assign_slots(objF, out.f.slots_tag, out.f.slots_set);
        assign_slots(objB, out.b.slots_tag, out.b.slots_set);
    }
    // slot byte offsets inside a group's slot area: tagged slots first (256 bytes each), then settled (128)
    auto slot_off = [&](const SlotUse &u, const std::vector<SlotObj> &objs, const FlowDir &d) {
        const SlotObj &o = objs[u.obj];
        return o.settled ? (uint32_t)d.slots_tag * 256u + (uint32_t)o.id * 128u : (uint32_t)o.id * 256u;
    };

    // ---- records, pools, tables ---------------------------------------------------------------------
    out.f.rec.assign(Q * kFRecWords, 0);
    out.b.rec.assign(Q * kBRecWords, 0);
    std::vector<std::vector<uint32_t>> poolF((size_t)stages), poolB((size_t)stages);
    std::vector<uint32_t> npush((size_t)stages * lanes, 0);
    std::vector<char> push_flag((size_t)n, 0);
    for (int32_t v : by_step) {
        const size_t q = slot_index(v);
        const int st = step_of[v] / K, ln = lane_of[v];
        out.node[q] = (uint32_t)v;
        out.step[q] = (uint32_t)step_of[v];
        out.lbes[q] = lbES[v];
        out.dmin[q] = (uint32_t)dmin[v];
        if (g.group[v] >= 0) out.grp[q] = (uint32_t)g.group[v];
        if (g.group[v] >= 0 && !constant[v]) out.rows[q] = (uint32_t)g.group[v];
        for (int l = 0; l < Lp; ++l) {
            const int ll = (g.group[v] < 0 || constant[v]) ? 0 : (l < L ? l : L - 1);
            const uint32_t doff = (uint32_t)(lat[(size_t)v * L + ll] - dmin[v]);
            uint64_t bits;
            std::memcpy(&bits, &energy[(size_t)v * L + ll], 8);
            out.tabF[(q * Lp + l) * 3 + 0] = doff;
            out.tabF[(q * Lp + l) * 3 + 1] = (uint32_t)(bits >> 32);
            out.tabF[(q * Lp + l) * 3 + 2] = (uint32_t)bits;
            out.tabB[q * Lp + l] = doff;
        }
        // forward record
        {
            uint32_t *r = &out.f.rec[q * kFRecWords];
            std::vector<uint32_t> &pool = poolF[st];
            uint32_t fl = 0, nops = 0;
            std::vector<uint32_t> opw;      // operand descriptors, 3 words each
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
                const int32_t k = pc[e];
                if (!liveF[e] || prev_on_lane[v] != k) continue;
                fl |= kF_HasReg;
                r[7] = (uint32_t)(lbES[v] - lbC[k]);
                if (r[7]) fl |= kF_RegDelta;
            }
            bool acc_seen = false;
            for (int64_t e = pp[v]; e < pp[v + 1]; ++e) {
                const int32_t k = pc[e];
                if (!liveF[e] || prev_on_lane[v] == k) continue;
                if (useF[k].acc) {
                    // the members of a shared slot appear as one operand, reset after the read
                    if (acc_seen) continue;
                    acc_seen = true;
                }
                uint32_t w = slot_off(useF[k], objF, out.f);
                if (useF[k].settled) w |= kOpWord;
                if (fper(k) < fper(v)) w |= kOpNoPoll;
                if (useF[k].pre) w |= kOpClear;
                opw.push_back(w);
                opw.push_back(tag_of(k));
                opw.push_back(useF[k].pre ? 0u : (uint32_t)(lbES[v] - lbC[k]));
                ++nops;
            }
            if (useF[v].obj >= 0) {
                fl |= useF[v].settled ? kF_OutSet : kF_OutTag;
                if (useF[v].acc) fl |= kF_OutAcc;
                r[1] = slot_off(useF[v], objF, out.f);
                r[2] = useF[v].settled ? useF[v].pre_delta : tag_of(v);
            }
            // the first operand sits in the record, the others (and a terminal node's bound) in the pool
            r[3] = (uint32_t)pool.size();
            for (size_t k = 0; k < opw.size(); ++k) {
                if (k < 3) r[4 + k] = opw[k];
                else pool.push_back(opw[k]);
            }
            if (sp[v + 1] == sp[v]) {
                fl |= kF_Terminal;
                pool.push_back((uint32_t)(uint64_t)lbC[v]);
                pool.push_back((uint32_t)((uint64_t)lbC[v] >> 32));
            }
            const bool invertible = (fl & kF_HasReg) && !(fl & kF_RegDelta) && nops == 0;
            if (!invertible) {
                fl |= kF_Push;
                push_flag[v] = 1;
                npush[(size_t)st * lanes + ln]++;
            }
            if (nops > 0xFFFFu) { err = "a node has more than 65535 exchanged operands"; return EMO_E_UNSUPPORTED; }
            r[0] = fl | (nops << kF_NopsShift);
        }
        // backward record
        {
            uint32_t *r = &out.b.rec[q * kBRecWords];
            std::vector<uint32_t> &pool = poolB[st];
            uint32_t fl = 0, nops = 0, simple_in_off = kNone;
            std::vector<uint32_t> opw;
            bool acc_seen = false;
            for (int64_t e = sp[v]; e < sp[v + 1]; ++e) {
                const int32_t u = sc[e];
                // the edge v -> u: find its liveness (position of v among u's predecessors)
                const int64_t ee = std::lower_bound(pc.begin() + pp[u], pc.begin() + pp[u + 1], v) - pc.begin();
                if (!liveB[ee]) continue;
                const uint32_t delta = (uint32_t)(lbQin[v] - lbQ[u]);
                if (next_on_lane[v] == u) {
                    fl |= kB_HasReg;
                    if (delta) fl |= kB_RegDelta;
                    r[7] = delta;
                    continue;
                }
                if (useB[u].acc) {
                    if (acc_seen) continue;
                    acc_seen = true;
                }
                uint32_t w = slot_off(useB[u], objB, out.b);
                if (useB[u].settled) w |= kOpWord;
                if (bper(u) < bper(v)) w |= kOpNoPoll;
                if (useB[u].pre) w |= kOpClear;
                simple_in_off = useB[u].pre ? (w & kOpOffMask) : kNone;
                opw.push_back(w);
                opw.push_back(tag_of(u));
                opw.push_back(useB[u].pre ? 0u : delta);
                ++nops;
            }
            if (useB[v].obj >= 0) {
                fl |= useB[v].settled ? kB_OutSet : kB_OutTag;
                if (useB[v].acc) fl |= kB_OutAcc;
                r[1] = slot_off(useB[v], objB, out.b);
                r[2] = useB[v].settled ? useB[v].pre_delta : tag_of(v);
            }
            r[3] = (uint32_t)pool.size();
            for (size_t k = 0; k < opw.size(); ++k) {
                if (k < 3) r[8 + k] = opw[k];
                else if (k < 6) r[12 + (k - 3)] = opw[k];
                else pool.push_back(opw[k]);
            }
            if (push_flag[v]) fl |= kB_Pop;
            if (nops > 0xFFFFu) { err = "a node has more than 65535 exchanged operands"; return EMO_E_UNSUPPORTED; }
            const int64_t A = lbQ[v] + lbES[v];
            r[0] = fl | (nops << kB_NopsShift);
            // a simple entry (see emo_flow.h) names its one operand slot in word 3
            {
                const bool in_ok = nops == 0 || (nops == 1 && simple_in_off != kNone);
                const bool out_ok = !(fl & kB_OutTag) && (!(fl & kB_OutSet) || useB[v].pre);
                if ((fl & kB_HasReg) && in_ok && out_ok) {
                    r[0] |= kB_Simple;
                    if (nops == 1) r[3] = simple_in_off;
                }
            }
            r[4] = (uint32_t)(uint64_t)A;
            r[5] = (uint32_t)((uint64_t)A >> 32);
            r[6] = (uint32_t)v;
        }
    }
    // ---- segments ------------------------------------------------------------------------------------
    // The kernels walk a lane's entries of a stage in segments: an optional entry that needs its
    // record (anything but a simple entry) followed by a run of up to kFlowRun simple entries, whose
    // look-ups are issued together.  A segment stays inside one period; the first segment of a period
    // carries the barrier flag (a lane without entries in a period gets an empty one).
    out.f.seg.assign((size_t)stages * lanes * kSegBytes, 0);
    out.b.seg.assign((size_t)stages * lanes * kSegBytes, 0);
    {
        const int nper_ = K / sync;
        std::vector<std::vector<int32_t>> ents((size_t)stages * lanes);      // nodes per (stage, lane) by position
        for (int32_t v : by_step) ents[(size_t)(step_of[v] / K) * lanes + lane_of[v]].push_back(v);
        for (int st = 0; st < stages; ++st)
            for (int ln = 0; ln < lanes; ++ln) {
                const std::vector<int32_t> &ev = ents[(size_t)st * lanes + ln];
                uint32_t *h = &out.hdr[((size_t)st * lanes + ln) * kHdrWords];
                for (int dir = 0; dir < 2; ++dir) {
                    uint8_t *sg = (dir ? out.b.seg.data() : out.f.seg.data()) + ((size_t)st * lanes + ln) * kSegBytes;
                    int nseg = 0;
                    for (int pi = 0; pi < nper_; ++pi) {
                        const int p = dir ? nper_ - 1 - pi : pi;
                        bool first = true, open = false;
                        uint32_t kind = 0;
                        auto start = [&](uint8_t byte) {
                            sg[nseg++] = (uint8_t)(byte | (first ? kSegBarrier : 0));
                            first = false;
                        };
                        const int ne = (int)ev.size();
                        for (int ii = 0; ii < ne; ++ii) {
                            const int32_t v = ev[dir ? ne - 1 - ii : ii];
                            if ((step_of[v] % K) / sync != p) continue;
                            const size_t q = slot_index(v);
                            bool simple;
                            uint32_t k2 = 0;
                            if (!dir) {
                                simple = out.f.rec[q * kFRecWords] == kF_HasReg;
                            } else {
                                const uint32_t w = out.b.rec[q * kBRecWords];
                                simple = (w & kB_Simple) != 0;
                                k2 = ((w >> kB_NopsShift) ? kSegIn : 0u) | ((w & kB_OutSet) ? kSegOut : 0u);
                            }
                            if (!simple) {
                                start(kSegSpecial);
                                open = true;          // a run may follow the special entry
                                kind = 0xFFu;         // ... of whatever kind comes first
                                continue;
                            }
                            uint8_t &cur = sg[nseg > 0 ? nseg - 1 : 0];
                            if (open && (cur & kSegRunMask) < kFlowRun && (kind == 0xFFu || kind == k2)) {
                                if (kind == 0xFFu) cur = (uint8_t)(cur | k2);
                                cur = (uint8_t)(cur + 1);
                            } else {
                                start((uint8_t)(1u | k2));
                                open = true;
                            }
                            kind = k2;
                        }
                        if (first) start(0);
                    }
                    if (nseg > kSegBytes) { err = "internal: too many segments"; return EMO_E_UNSUPPORTED; }
                    h[0] |= (uint32_t)nseg << (dir ? 8 : 0);
                }
                h[0] |= (uint32_t)ev.size() << 16;
            }
    }
    // restore list: rows per stage and lane
    out.push_base.assign((size_t)stages + 1, 0);
    for (int st = 0; st < stages; ++st) {
        uint32_t off = 0;
        for (int ln = 0; ln < lanes; ++ln) {
            uint32_t *h = &out.hdr[((size_t)st * lanes + ln) * kHdrWords];
            h[4] = npush[(size_t)st * lanes + ln];
            h[5] = off;
            h[6] = (uint32_t)out.push_base[st];
            off += h[4];
        }
        out.push_base[st + 1] = out.push_base[st] + off;
    }
    out.pushes = out.push_base[stages];
    auto pack_pool = [&](std::vector<std::vector<uint32_t>> &pools, FlowDir &d) {
        size_t mx = 4;
        for (auto &p : pools) mx = std::max(mx, p.size());
        mx = (mx + 3) / 4 * 4;
        d.pool_stride = (int)mx;
        d.pool.assign((size_t)stages * mx, 0);
        for (int st = 0; st < stages; ++st) std::copy(pools[st].begin(), pools[st].end(), d.pool.begin() + (size_t)st * mx);
    };
    pack_pool(poolF, out.f);
    pack_pool(poolB, out.b);
    out.ok32 = true;
    if (spine) {
        SpineIn in;
        in.n = n;
        in.lanes = lanes;
        in.K = K;
        in.stages = stages;
        in.L = L;
        in.pp = &pp;
        in.sp = &sp;
        in.pc = &pc;
        in.sc = &sc;
        in.liveF = &liveF;
        in.liveB = &liveB;
        in.constant = &constant;
        in.lbES = &lbES;
        in.lbC = &lbC;
        in.lbQin = &lbQin;
        in.lbQ = &lbQ;
        in.step_of = &step_of;
        in.lane_of = &lane_of;
        in.prev_on_lane = &prev_on_lane;
        in.next_on_lane = &next_on_lane;
        in.pos_of = &pos_of;
        in.energy = energy;
        in.pair_K = pair_K;
        rc = build_spine(in, out.spine, err);
        if (rc != EMO_OK) return rc;
    }
    return EMO_OK;
}

}  // namespace emo
