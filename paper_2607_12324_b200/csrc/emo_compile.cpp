// Step-program compiler: list scheduling of the (forward or reversed) DAG onto `lanes` warps,
// register/slot assignment for the values that flow along edges, and the schedule-ordered copies
// of the duration and energy tables (Eq. 3) the kernels stream through.
#include "emo_compile.h"

#include <algorithm>
#include <climits>
#include <queue>

#include "../../include/emo.h"

namespace emo {

namespace {

struct Op {
    int32_t node;                 // caller's node id, -1 for a helper op that only takes a maximum
    std::vector<int32_t> preds;   // op indices whose values this op needs
};

// A node with more operands than one entry can name is split: helper ops take the maximum of up
// to kMaxSlotPreds operands each (duration 0, no output), and the node reads the helpers.
// A node with more operands than kMaxOperands is split: helper ops take the maximum of a few
// operands each (duration 0, no output) and the node reads the helpers.  The operands that are
// ready earliest (smallest hop level) go into helpers, the latest one stays with the node, so the
// helpers can run on other warps ahead of time and the node's own warp - typically a serial chain
// such as the launch chain in the backward direction, whose every node waits for four kernels -
// is left with a short step.
void add_with_helpers(std::vector<Op> &ops, std::vector<int32_t> &hop, int32_t node, std::vector<int32_t> preds, int &n_aux)
{
    std::sort(preds.begin(), preds.end());
    preds.erase(std::unique(preds.begin(), preds.end()), preds.end());
    auto by_hop = [&](int32_t a, int32_t b) { return hop[a] != hop[b] ? hop[a] < hop[b] : a < b; };
    std::sort(preds.begin(), preds.end(), by_hop);
    while ((int)preds.size() > kMaxOperands) {
        const int take = std::min<int>(kMaxOperands, (int)preds.size() - kMaxOperands + 1);
        Op h;
        h.node = -1;
        h.preds.assign(preds.begin(), preds.begin() + take);
        int32_t lvl = 0;
        for (int32_t q : h.preds) lvl = std::max(lvl, hop[q] + 1);
        preds.erase(preds.begin(), preds.begin() + take);
        const int32_t id = (int32_t)ops.size();
        ops.push_back(std::move(h));
        hop.push_back(lvl);
        preds.insert(std::upper_bound(preds.begin(), preds.end(), id, by_hop), id);
        ++n_aux;
    }
    int32_t lvl = 0;
    for (int32_t q : preds) lvl = std::max(lvl, hop[q] + 1);
    Op o;
    o.node = node;
    o.preds = std::move(preds);
    ops.push_back(std::move(o));
    hop.push_back(lvl);
}

}  // namespace

int pick_lanes(int64_t n_ops, int depth)
{
    if (depth <= 0) return 1;
    // a little spare capacity (10 %) lets the list scheduler catch up after a narrow stretch
    int64_t c = (n_ops * 11 + (int64_t)depth * 10 - 1) / ((int64_t)depth * 10);
    if (c < 1) c = 1;
    if (c > kMaxLanes) c = kMaxLanes;
    return (int)c;
}

// Target steps and list scheduling of ops (given by their operand lists, in a topological order)
// onto `lanes` warps.  On return step_of / warp_of give every op's place, prev_on_warp the op the
// same warp handled just before it (-1: none), S the number of steps.
int schedule_ops(const std::vector<std::vector<int32_t>> &preds, int lanes, int lookahead, std::vector<int32_t> &step_of,
                 std::vector<int32_t> &warp_of, std::vector<int32_t> &prev_on_warp, int32_t &S_out, int &lanes_out,
                 std::string &err, const std::vector<std::vector<int32_t>> *gaps, bool hard_gaps)
{
    const int32_t N = (int32_t)preds.size();
    // distance in steps an op keeps from operand k of its list (1 unless the caller asks for more)
    auto gap = [&](int32_t i, size_t k) { return gaps ? (*gaps)[i][k] : 1; };
    // consumers of each op
    std::vector<int64_t> cp((size_t)N + 1, 0);
    for (int32_t i = 0; i < N; ++i)
        for (int32_t p : preds[i]) cp[p + 1]++;
    for (int32_t i = 0; i < N; ++i) cp[i + 1] += cp[i];
    std::vector<int32_t> cons((size_t)std::max<int64_t>(cp[N], 1)), cgap((size_t)std::max<int64_t>(cp[N], 1), 1);
    {
        std::vector<int64_t> f(cp.begin(), cp.end() - 1);
        for (int32_t i = 0; i < N; ++i)
            for (size_t k = 0; k < preds[i].size(); ++k) {
                const int32_t p = preds[i][k];
                cgap[f[p]] = gap(i, k);
                cons[f[p]++] = i;
            }
    }

    // hop levels: earliest step (asap) and the number of hops to the end (rem; alap = D - rem)
    std::vector<int32_t> asap((size_t)N, 0), rem((size_t)N, 1), tgt((size_t)N, 0);
    int32_t D = 0;
    for (int32_t i = 0; i < N; ++i) {
        int32_t a = 0;
        for (size_t k = 0; k < preds[i].size(); ++k) a = std::max(a, asap[preds[i][k]] + gap(i, k));
        asap[i] = a;
        D = std::max(D, a + 1);
    }
    for (int32_t i = N - 1; i >= 0; --i) {
        int32_t r = 1;
        for (int64_t e = cp[i]; e < cp[i + 1]; ++e) r = std::max(r, rem[cons[e]] + cgap[e]);
        rem[i] = r;
    }
    // Target steps.  A value occupies an exchange slot from the step that produces it to the step
    // of its last consumer, so the targets are moved, within the precedence constraints, to
    // shorten the summed lifetimes: starting from the earliest steps, a backward sweep moves an op
    // later (next to its earliest consumer) when that shortens its own value's life by more than
    // it stretches its operands' lives, and a forward sweep moves an op earlier under the mirrored
    // test.  This puts a chain that has hop slack (a launch chain running ahead of the kernels, or
    // short streams beside a long launch chain) next to the ops it exchanges values with.
    // Two starting points are refined, all ops at their earliest and all at their latest steps,
    // and the one with the smaller summed lifetime is kept.
    auto last_cons_excl = [&](int32_t p, int32_t skip) {
        int32_t m = -1;
        for (int64_t e = cp[p]; e < cp[p + 1]; ++e)
            if (cons[e] != skip) m = std::max(m, tgt[cons[e]]);
        return m;
    };
    auto sweep_later = [&]() {
        for (int32_t i = N - 1; i >= 0; --i) {
            if (cp[i + 1] == cp[i]) continue;
            int32_t hi = INT32_MAX;
            for (int64_t e = cp[i]; e < cp[i + 1]; ++e) hi = std::min(hi, tgt[cons[e]] - cgap[e]);
            if (hi <= tgt[i]) continue;
            int64_t gain = hi - tgt[i], cost = 0;
            for (int32_t p : preds[i]) {
                if (cp[p + 1] - cp[p] == 1) continue;   // its only consumer: it follows later in this sweep
                int32_t other = last_cons_excl(p, i);
                cost += std::max(other, hi) - std::max(other, tgt[i]);
            }
            if (gain > cost) tgt[i] = hi;
        }
    };
    auto sweep_earlier = [&]() {
        for (int32_t i = 0; i < N; ++i) {
            if (preds[i].empty()) continue;
            int32_t lo = 0;
            for (size_t k = 0; k < preds[i].size(); ++k) lo = std::max(lo, tgt[preds[i][k]] + gap(i, k));
            if (lo >= tgt[i]) continue;
            bool held = false;   // a consumer with other operands keeps this op's value alive
            for (int64_t e = cp[i]; e < cp[i + 1]; ++e) held |= preds[cons[e]].size() > 1;
            int64_t cost = held ? tgt[i] - lo : 0, gain = 0;
            for (int32_t p : preds[i]) {
                int32_t other = last_cons_excl(p, i);
                gain += std::max(other, tgt[i]) - std::max(other, lo);
            }
            if (gain > cost) tgt[i] = lo;
        }
    };
    auto total_life = [&]() {
        int64_t sum = 0;
        for (int32_t i = 0; i < N; ++i) {
            int32_t m = last_cons_excl(i, -1);
            if (m >= 0) sum += m - tgt[i];
        }
        return sum;
    };
    tgt = asap;
    for (int round = 0; round < 2; ++round) { sweep_later(); sweep_earlier(); }
    const int64_t life_early = total_life();
    std::vector<int32_t> tgt_early = tgt;
    for (int32_t i = 0; i < N; ++i) tgt[i] = D - rem[i];
    for (int round = 0; round < 2; ++round) { sweep_earlier(); sweep_later(); }
    if (life_early <= total_life()) tgt.swap(tgt_early);
    if (lanes <= 0) lanes = pick_lanes(N, D);
    if (lanes > kMaxLanes) lanes = kMaxLanes;
    if (lookahead <= 0) lookahead = 8;
    lanes_out = lanes;

    // ---- list scheduling ----------------------------------------------------------------------
    // Priority: smallest target step first (ties: the more critical op).  An op is not started more
    // than `lookahead` steps before its target step, which keeps a cheap chain from running far
    // ahead of the ops that consume its values.
    step_of.assign((size_t)N, -1);
    warp_of.assign((size_t)N, -1);
    prev_on_warp.assign((size_t)N, -1);
    std::vector<int32_t> left((size_t)N);
    std::vector<int32_t> unsched_cons((size_t)N);
    using Key = std::pair<int64_t, int32_t>;   // (target step, alap | op)
    std::priority_queue<Key, std::vector<Key>, std::greater<Key>> ready;
    auto prio = [&](int32_t i) { return ((int64_t)tgt[i] << 32) | (uint32_t)(D - rem[i]); };
    for (int32_t i = 0; i < N; ++i) {
        left[i] = (int32_t)preds[i].size();
        unsched_cons[i] = (int32_t)(cp[i + 1] - cp[i]);
        if (left[i] == 0) ready.push({prio(i), i});
    }
    std::vector<int32_t> last((size_t)lanes, -1);
    std::vector<std::vector<int32_t>> sched;   // per step: op per warp (-1 idle)
    std::vector<int32_t> chosen, next_ready;
    std::priority_queue<std::pair<int32_t, int32_t>, std::vector<std::pair<int32_t, int32_t>>, std::greater<std::pair<int32_t, int32_t>>>
        held;      // (earliest step, op): operands done, but the op keeps its distance from one of them
    int32_t done = 0;
    int32_t t = 0;
    while (done < N) {
        while (!held.empty() && held.top().first <= t) {
            ready.push({prio(held.top().second), held.top().second});
            held.pop();
        }
        chosen.clear();
        while (!ready.empty() && (int)chosen.size() < lanes) {
            Key k = ready.top();
            // an op that is not due yet waits, unless the step would otherwise be empty
            if ((k.first >> 32) > t + lookahead && !chosen.empty()) break;
            ready.pop();
            chosen.push_back(k.second);
        }
        std::vector<int32_t> row((size_t)lanes, -1);
        std::vector<char> placed(chosen.size(), 0);
        // first the ops whose operand sits in a free warp's register.  Where several operands do,
        // the op follows the one with the fewest readers: a value with one reader that travels in a
        // register is never written to a slot, and a serial chain (the launch chain, whose nodes
        // each have one chain successor but also read several kernels) stays on one warp instead
        // of hopping from warp to warp with a slot hand-over on its critical path every step.
        for (size_t j = 0; j < chosen.size(); ++j) {
            int32_t i = chosen[j];
            int best_w = -1;
            int64_t best_fan = 0;
            for (int32_t p : preds[i]) {
                int w = warp_of[p];
                if (w >= 0 && last[w] == p && row[w] < 0) {
                    const int64_t fan = cp[p + 1] - cp[p];
                    if (best_w < 0 || fan < best_fan) {
                        best_w = w;
                        best_fan = fan;
                    }
                }
            }
            if (best_w >= 0) {
                row[best_w] = i;
                placed[j] = 1;
            }
        }
        // then the rest: prefer a warp whose register value nobody is waiting for
        for (size_t j = 0; j < chosen.size(); ++j) {
            if (placed[j]) continue;
            int best = -1;
            for (int w = 0; w < lanes; ++w) {
                if (row[w] >= 0) continue;
                bool dead = last[w] < 0 || unsched_cons[last[w]] == 0;
                if (dead) { best = w; break; }
                if (best < 0) best = w;
            }
            row[best] = chosen[j];
        }
        next_ready.clear();
        for (int w = 0; w < lanes; ++w) {
            int32_t i = row[w];
            if (i < 0) continue;
            step_of[i] = t;
            warp_of[i] = w;
            prev_on_warp[i] = last[w];
            ++done;
        }
        for (int w = 0; w < lanes; ++w) {
            int32_t i = row[w];
            if (i < 0) continue;
            last[w] = i;
            for (int32_t p : preds[i]) unsched_cons[p]--;
            for (int64_t e = cp[i]; e < cp[i + 1]; ++e)
                if (--left[cons[e]] == 0) next_ready.push_back(cons[e]);
        }
        for (int32_t i : next_ready) {
            int32_t est = 0;
            for (size_t k = 0; k < preds[i].size(); ++k) est = std::max(est, step_of[preds[i][k]] + (hard_gaps ? gap(i, k) : 1));
            if (est <= t + 1) ready.push({prio(i), i});
            else held.push({est, i});
        }
        sched.push_back(std::move(row));
        ++t;
        if (chosen.empty() && ready.empty() && held.empty() && done < N) {
            err = "scheduler stalled (graph is not acyclic?)";
            return EMO_E_NOT_TOPOLOGICAL;
        }
    }
    S_out = t;
    return EMO_OK;
}

int compile_program(const HostGraph &g, const int64_t *lat, const double *energy, bool backward,
                    int lanes, int lookahead, int sync_steps, const std::vector<uint32_t> *row_in_other,
                    Program &out, std::string &err)
{
    if (sync_steps != 8 && sync_steps != 16 && sync_steps != 32) sync_steps = kSyncSteps;
    const int32_t n = g.n;
    const int L = g.L;
    int Lp = 4;   // at least 4 so that a table row is a multiple of 16 bytes (bulk-copy granularity)
    while (Lp < L) Lp <<= 1;
    out = Program();
    out.Lp = Lp;
    out.sync = sync_steps;

    // ---- ops in a topological order of the direction being compiled --------------------------
    std::vector<Op> ops;
    ops.reserve((size_t)n + 16);
    std::vector<int32_t> op_of_node((size_t)std::max(n, 1), -1);
    std::vector<int32_t> op_hop;      // hop level of every op built so far
    op_hop.reserve((size_t)n + 16);
    int n_aux = 0;
    // Bounds of every node's value over all policies (forward: completion time C_v; backward: the
    // longest tail Q_v), from the smallest and the largest entry of its duration row.  An operand
    // whose upper bound does not exceed the lower bound of another operand of the same node can
    // never decide that node's maximum (Eq. 1), under any policy, so the edge is dropped before
    // scheduling: typically the launch edge of a kernel whose stream predecessor always finishes
    // long after the launch chain has issued it.  Results are unchanged; slots, waits and maximum
    // operations for such edges disappear.
    std::vector<int64_t> lbv((size_t)std::max(n, 1), 0), ubv((size_t)std::max(n, 1), 0);
    int64_t n_pruned = 0;
    auto dur_bounds = [&](int32_t v, int64_t &lo, int64_t &hi) {
        lo = hi = lat[(size_t)v * L];
        if (g.group[v] < 0) return;
        for (int l = 1; l < L; ++l) {
            lo = std::min(lo, lat[(size_t)v * L + l]);
            hi = std::max(hi, lat[(size_t)v * L + l]);
        }
    };
    auto add_node = [&](int32_t v, std::vector<int32_t> &pn) {
        std::sort(pn.begin(), pn.end());
        pn.erase(std::unique(pn.begin(), pn.end()), pn.end());
        int64_t lo_start = 0, hi_start = 0;
        int32_t best = -1;
        for (int32_t k : pn) {
            hi_start = std::max(hi_start, ubv[k]);
            if (best < 0 || lbv[k] > lbv[best]) best = k;
        }
        if (best >= 0) lo_start = lbv[best];
        std::vector<int32_t> p;
        for (int32_t k : pn) {
            if (k != best && ubv[k] <= lbv[best]) { ++n_pruned; continue; }
            p.push_back(op_of_node[k]);
        }
        int64_t dlo, dhi;
        dur_bounds(v, dlo, dhi);
        lbv[v] = lo_start + dlo;
        ubv[v] = hi_start + dhi;
        add_with_helpers(ops, op_hop, v, std::move(p), n_aux);
        op_of_node[v] = (int32_t)ops.size() - 1;
    };
    if (!backward) {
        for (int32_t v = 0; v < n; ++v) {
            std::vector<int32_t> pn(g.col.begin() + g.row_ptr[v], g.col.begin() + g.row_ptr[v + 1]);
            add_node(v, pn);
        }
    } else {
        std::vector<int64_t> sp((size_t)n + 1, 0);
        for (int64_t e = 0; e < g.m; ++e) sp[g.col[e] + 1]++;
        for (int32_t v = 0; v < n; ++v) sp[v + 1] += sp[v];
        std::vector<int32_t> succ((size_t)std::max<int64_t>(g.m, 1));
        std::vector<int64_t> fill(sp.begin(), sp.end() - 1);
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = g.row_ptr[v]; e < g.row_ptr[v + 1]; ++e) succ[fill[g.col[e]]++] = v;
        for (int32_t v = n - 1; v >= 0; --v) {
            std::vector<int32_t> pn(succ.begin() + sp[v], succ.begin() + sp[v + 1]);
            add_node(v, pn);
        }
    }
    out.pruned = n_pruned;
    const int32_t N = (int32_t)ops.size();
    out.aux = n_aux;

    std::vector<std::vector<int32_t>> op_preds((size_t)N);
    for (int32_t i = 0; i < N; ++i) op_preds[i] = ops[i].preds;
    std::vector<int32_t> step_of, warp_of, prev_on_warp;
    int32_t S = 0;
    {
        int rc = schedule_ops(op_preds, lanes, lookahead, step_of, warp_of, prev_on_warp, S, lanes, err);
        if (rc != EMO_OK) return rc;
    }
    out.lanes = lanes;
    out.steps = S;
    std::vector<std::vector<int32_t>> sched((size_t)S, std::vector<int32_t>((size_t)lanes, -1));
    for (int32_t i = 0; i < N; ++i) sched[step_of[i]][warp_of[i]] = i;
    // consumers of each op
    std::vector<int64_t> cp((size_t)N + 1, 0);
    for (int32_t i = 0; i < N; ++i)
        for (int32_t p : ops[i].preds) cp[p + 1]++;
    for (int32_t i = 0; i < N; ++i) cp[i + 1] += cp[i];

    // ---- slots ---------------------------------------------------------------------------------
    // An operand is read from the warp's register when the producing op was the previous op of the
    // same warp; every other operand is read from the producer's slot.  A slot lives from the
    // producer's step to the last step that reads it.  The warps of a group only meet at a barrier
    // every sync_steps steps and otherwise run at their own pace, so a slot is reused no earlier
    // than the first step of the block after its last read: the barrier between the two blocks
    // orders the last read before the next write.  Readers find out that a value has been written
    // from a per-slot phase counter; the entry carries the phase parity of every value it touches.
    std::vector<int32_t> last_use((size_t)N, -1);
    for (int32_t i = 0; i < N; ++i)
        for (int32_t p : ops[i].preds)
            if (!(warp_of[p] == warp_of[i] && prev_on_warp[i] == p)) last_use[p] = std::max(last_use[p], step_of[i]);
    std::vector<int32_t> slot_of((size_t)N, -1);
    std::vector<uint8_t> parity_of((size_t)N, 0);
    {
        using Key = std::pair<int64_t, int32_t>;
        std::vector<uint8_t> phase;   // number of values written to a slot so far, mod 2
        std::priority_queue<int32_t, std::vector<int32_t>, std::greater<int32_t>> free_ids;
        std::priority_queue<Key, std::vector<Key>, std::greater<Key>> busy;   // (last use step, slot)
        int32_t next_id = 0;
        for (int32_t s = 0; s < S; ++s) {
            while (!busy.empty() && busy.top().first / sync_steps < s / sync_steps) {
                free_ids.push(busy.top().second);
                busy.pop();
            }
            for (int w = 0; w < lanes; ++w) {
                int32_t i = sched[s][w];
                if (i < 0 || last_use[i] < 0) continue;
                int32_t id;
                if (!free_ids.empty()) {
                    id = free_ids.top();
                    free_ids.pop();
                } else {
                    id = next_id++;
                    phase.push_back(0);
                }
                slot_of[i] = id;
                parity_of[i] = phase[id];
                phase[id] ^= 1;
                busy.push({last_use[i], id});
            }
        }
        out.slots = next_id;
        if (next_id > kMaxSlots) {
            err = "graph needs " + std::to_string(next_id) + " live exchange values per policy; at most " +
                  std::to_string(kMaxSlots) + " are supported";
            return EMO_E_UNSUPPORTED;
        }
    }

    // ---- entries and schedule-ordered tables -------------------------------------------------
    const size_t Q = (size_t)S * lanes;
    out.entries.assign(Q * kEntryWords, 0);
    out.rows.assign(Q, kNone);
    out.groups.assign(Q, kNone);
    out.pos_of_node.assign((size_t)std::max(n, 1), kNone);
    out.lat.assign(Q * Lp, 0);
    if (!backward) out.energy.assign(Q * Lp, 0.0);
    for (int32_t s = 0; s < S; ++s) {
        for (int w = 0; w < lanes; ++w) {
            int32_t i = sched[s][w];
            size_t q = (size_t)s * lanes + w;
            uint32_t *en = &out.entries[q * kEntryWords];
            en[0] = kNone;
            en[4] = kNone;
            out.rows[q] = kNone;
            out.groups[q] = kNone;
            if (i < 0) continue;
            const Op &o = ops[i];
            uint32_t flags = kValid;
            uint32_t operands = 0, operands_hi = 0;
            int np = 0;
            bool settled = true;      // every slot operand was written before the group's last barrier
            for (int32_t p : o.preds) {
                if (warp_of[p] == w && prev_on_warp[i] == p) {
                    flags |= kRegPred;
                } else {
                    settled = settled && step_of[p] / sync_steps < s / sync_steps;
                    if (np < 4) operands |= (uint32_t)slot_of[p] << (8 * np);
                    else operands_hi |= (uint32_t)slot_of[p] << (8 * (np - 4));
                    flags |= (uint32_t)parity_of[p] << (kOperandParityShift + np);
                    ++np;
                }
            }
            flags |= (uint32_t)np << kNPredShift;
            if (slot_of[i] >= 0)
                flags |= kWriteSlot | ((uint32_t)slot_of[i] << kOutShift) | ((uint32_t)parity_of[i] << kOutParityShift);
            if (o.node < 0) {
                flags |= kAux;
            } else {
                int32_t v = o.node;
                // word 0: the row this entry addresses in the kernel's main per-node array - the
                // node's position in the other direction's program when that is known (the forward
                // pass leaves ES where the backward pass will stream it from), else the node id
                en[0] = row_in_other ? (*row_in_other)[v] : (uint32_t)v;
                en[4] = (uint32_t)v;
                out.pos_of_node[v] = (uint32_t)q;
                // a node whose duration and energy do not depend on the level needs no level
                bool constant = true;
                for (int l = 1; l < L && constant; ++l)
                    constant = lat[(size_t)v * L + l] == lat[(size_t)v * L] && energy[(size_t)v * L + l] == energy[(size_t)v * L];
                if (g.group[v] >= 0) out.groups[q] = (uint32_t)g.group[v];
                if (g.group[v] >= 0 && !constant) {
                    out.rows[q] = (uint32_t)g.group[v];
                    flags |= (uint32_t)(Lp - 1) << kMaskShift;
                }
                if (cp[i + 1] == cp[i]) flags |= kTerminal;
                for (int l = 0; l < Lp; ++l) {
                    int ll = l < L ? l : L - 1;
                    out.lat[q * Lp + l] = (uint32_t)lat[(size_t)v * L + ll];
                    if (!backward) out.energy[q * Lp + l] = energy[(size_t)v * L + ll];
                }
            }
            en[1] = flags;
            en[2] = operands;
            en[3] = operands_hi;
            // word 6: 1 when the entry has slot operands and all of them are settled - the barrier the
            // group passed since has ordered the writes before this read, so no slot needs polling
            en[6] = (np > 0 && settled) ? 1u : 0u;
        }
    }
    // Runs of simple entries.  An entry is simple when its only operand is the warp's register and
    // it neither writes a slot nor ends a path: the kernels handle a run of them in a tight loop
    // without decoding flags.  Every simple entry carries the length of the run that starts at it
    // (in the bits that name slots, unused here); a run stays inside one block of sync_steps steps (and names at most 15 entries)
    // and its entries agree on whether they read a level.
    for (int w = 0; w < lanes; ++w) {
        uint32_t next_run = 0, next_mask = 0;
        for (int32_t s = S - 1; s >= 0; --s) {
            uint32_t &fl = out.entries[((size_t)s * lanes + w) * kEntryWords + 1];
            const bool simple = (fl & kValid) && (fl & kRegPred) && !(fl & (kWriteSlot | kTerminal | kAux)) &&
                                ((fl >> kNPredShift) & 7u) == 0;
            uint32_t run = 0;
            const uint32_t mask = (fl >> kMaskShift) & 255u;
            if (simple) {
                run = 1;
                if ((s + 1) % sync_steps != 0 && next_run > 0 && next_mask == mask) run = std::min<uint32_t>(next_run + 1, 15u);
                fl |= kSimple | (run << kRunShift);
            }
            next_run = run;
            next_mask = mask;
        }
    }
    // Runs of plain entries for the one-policy-per-thread kernel (word 5).  An entry is plain when its
    // only operand is the warp's register and it handles a real node; forward it also writes no
    // slot and ends no path, backward it may write one (there nearly every node hands its value to
    // the node that launched it).  Forward, an idle entry counts as plain too (nothing is stored for
    // it and its duration and energy are 0), so idle steps do not cut a run.
    // Word 5 of a plain entry is the length of the run that starts at
    // it, inside one block of sync_steps steps and 15 at most; 0 for every other entry.
    for (int w = 0; w < lanes; ++w) {
        uint32_t next_run = 0;
        for (int32_t s = S - 1; s >= 0; --s) {
            uint32_t *en = &out.entries[((size_t)s * lanes + w) * kEntryWords];
            const uint32_t fl = en[1];
            bool plain = (fl & kValid) && (fl & kRegPred) && !(fl & kAux) && ((fl >> kNPredShift) & 7u) == 0;
            if (plain && !backward && (fl & (kWriteSlot | kTerminal))) plain = false;
            if (!backward && !(fl & kValid)) plain = true;
            uint32_t run = 0;
            if (plain) run = ((s + 1) % sync_steps != 0) ? std::min<uint32_t>(next_run + 1, 15u) : 1;
            en[5] = run;
            next_run = run;
        }
    }
    return EMO_OK;
}

}  // namespace emo
