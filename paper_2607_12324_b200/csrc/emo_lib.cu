// C-ABI entry points (see include/emo.h) and the CUDA kernels behind them.  sm_100a only.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <map>
#include <cstring>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "../../include/emo.h"
#include "emo_compile.h"
#include "emo_flow.h"
#include "emo_kernels.cuh"
#include "emo_pass_lane.cuh"
#include "emo_pass_staged.cuh"
#include "emo_flow.cuh"
#include "emo_spine.cuh"
#include "emo_intervals.cuh"
#include "emo_model.cuh"
#include "emo_generic.cuh"

using namespace emo;

struct DevProgram {
    unsigned char *rec = nullptr;   // records: entry, duration row, (forward) energy row
    uint32_t *rows = nullptr;
    uint32_t *groups = nullptr;     // the nodes' groups (time-interval policies)
    int rec_bytes = 0;
};

// The same program in the layout of emo_pass_lane (see emo_lane_layout.cuh), padded to whole stages.
struct DevProgramLane {
    unsigned char *ent = nullptr;   // [Qp][32]
    unsigned char *tab = nullptr;   // [Qp][tab_entry]
    uint32_t *rows = nullptr;       // [Qp]
    int steps_pad = 0;
    unsigned tab_entry = 0;
};

// The lane-stream program on the device: one blob per stage and direction (see emo_flow.cuh).
struct DevFlow {
    unsigned char *blobF = nullptr, *blobB = nullptr;
    unsigned char *blobFI = nullptr;      // the forward blob followed by 16 bytes per entry {lbES_v, group, dmin_v}: time-interval policies
    uint32_t *rows = nullptr, *push_base = nullptr;
    unsigned blobF_bytes = 0, blobB_bytes = 0, blobFI_bytes = 0, f_off_meta = 0;
    unsigned off_seg = 0;
    unsigned f_off_rec = 0, f_off_pool = 0, f_off_tab = 0;
    unsigned b_off_rec = 0, b_off_pool = 0, b_off_lbes = 0, b_off_tab = 0;
    int max_push = 0;               // most restore rows of one stage
    bool ready = false;
};

// The spine program on the device (emo_spine.cuh): per direction one blob per stage.
struct DevSpine {
    unsigned char *blobF = nullptr, *blobB = nullptr;
    uint32_t *rows = nullptr, *push_base = nullptr;
    unsigned blobF_bytes = 0, blobB_bytes = 0;
    unsigned f_off_ops = 0, f_front = 0, f_off_tpool = 0, f_off_pos = 0, f_off_tab = 0;      // f_front: bytes that the spine needs
    unsigned b_off_ops = 0, b_off_mem = 0, b_off_tab = 0;
    int max_push = 0;
    bool ready = false;
};

struct emo_graph {
    HostGraph h;
    Program fwd, bwd;
    Flow flow;                       // lane-stream program of the 32-bit pass kernels (flow.ok32: usable)
    DevProgram dfwd, dbwd;
    DevProgramLane lfwd, lbwd;       // only for programs of at most kLaneMaxLanes lanes
    DevFlow dflow;
    Flow sflow;                      // the same graph compiled with short stages and its spine program (sflow.spine.ok: usable)
    DevSpine dspine;
    bool host_only = false;
    // graphs beyond the schedule compilers' limits (or loaded with EMO_F_GENERIC): evaluated by the generic kernels
    bool generic = false;
    int64_t *gen_row_ptr = nullptr, *gen_srow_ptr = nullptr, *gen_lat = nullptr;
    int32_t *gen_col = nullptr, *gen_scol = nullptr, *gen_group = nullptr;
    double *gen_energy = nullptr;
    std::vector<int64_t> host_lat;      // kept only for the generic path's upload
    std::vector<double> host_energy;
    int device = 0;
    int sm_count = 148;
    size_t smem_optin = 0;
};

namespace {

constexpr int kManySlots = 48;       // above this, a program is compiled with the short barrier distance
constexpr size_t kSmallWs = 65536;   // head of the workspace: selection partials and scalars

// Optional timing hook: events recorded around the forward and the backward pass kernel.
cudaEvent_t g_pass_events[4] = {nullptr, nullptr, nullptr, nullptr};

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// workspace area for one policy's levels laid out [rows][16] (row pitch a bulk copy accepts)
size_t lvl_area(const emo_graph *g);

#define EMO_CUDA(call)                                  \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) { (void)cudaGetLastError(); return EMO_E_CUDA; } \
    } while (0)

template <typename T>
int upload(T **dst, const void *src, size_t bytes)
{
    *dst = nullptr;
    if (bytes == 0) bytes = 16;
    if (cudaMalloc((void **)dst, bytes) != cudaSuccess) { (void)cudaGetLastError(); *dst = nullptr; return EMO_E_OOM; }
    if (src && cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice) != cudaSuccess) { (void)cudaGetLastError(); return EMO_E_CUDA; }
    return EMO_OK;
}

int upload_program(const Program &p, DevProgram &d)
{
    const size_t Q = (size_t)p.steps * p.lanes;
    const bool fwd = !p.energy.empty();
    d.rec_bytes = 32 + p.Lp * 4 + (fwd ? p.Lp * 8 : 0);
    std::vector<unsigned char> rec(Q * d.rec_bytes);
    for (size_t q = 0; q < Q; ++q) {
        unsigned char *r = rec.data() + q * d.rec_bytes;
        std::memcpy(r, &p.entries[q * kEntryWords], 32);
        std::memcpy(r + 32, &p.lat[q * p.Lp], (size_t)p.Lp * 4);
        if (fwd) std::memcpy(r + 32 + p.Lp * 4, &p.energy[q * p.Lp], (size_t)p.Lp * 8);
    }
    int rc = upload(&d.rec, rec.data(), rec.size());
    if (rc) return rc;
    rc = upload(&d.rows, p.rows.data(), p.rows.size() * sizeof(uint32_t));
    if (rc) return rc;
    return upload(&d.groups, p.groups.data(), p.groups.size() * sizeof(uint32_t));
}

int upload_program_lane(const Program &p, DevProgramLane &d)
{
    const bool fwd = !p.energy.empty();
    const size_t Q = (size_t)p.steps * p.lanes;
    d.steps_pad = (p.steps + kLaneStepPad - 1) / kLaneStepPad * kLaneStepPad;
    const size_t Qp = (size_t)d.steps_pad * p.lanes;
    d.tab_entry = (unsigned)p.Lp * (fwd ? 12u : 4u);
    std::vector<uint32_t> ent(Qp * 8, 0), rows(Qp, kNone);
    std::vector<unsigned char> tab(Qp * d.tab_entry, 0);
    for (size_t q = 0; q < Qp; ++q) {
        uint32_t *w = &ent[q * 8];
        w[0] = kNone;
        w[1] = kLaneNoSlot | kLaneIdle;
        w[2] = 0xFFFFFFFFu;      // idle: the lane keeps its value
        w[5] = kNone;
        if (q >= Q) continue;
        const uint32_t *en = &p.entries[q * kEntryWords];
        const uint32_t fl = en[1];
        if (!(fl & kValid)) {
            w[1] |= (en[5] & 15u) << kLaneRunShift;      // forward: an idle entry may sit inside a run
            continue;
        }
        const uint32_t np = (fl >> kNPredShift) & 7u;
        const uint32_t out = (fl & kWriteSlot) ? ((fl >> kOutShift) & 255u) : kLaneNoSlot;
        const uint32_t outpar = (fl & kWriteSlot) ? ((fl >> kOutParityShift) & 1u) : 0u;
        const uint32_t oppar = (fl >> kOperandParityShift) & 63u;
        w[0] = en[0];
        w[1] = out | (np << kLaneNpShift) | ((fl & kTerminal) ? kLaneTerminal : 0u) | (outpar << kLaneOutParShift) | (oppar << kLaneOpParShift);
        w[1] |= (en[5] & 15u) << kLaneRunShift;
        if (en[6] & 1u) w[1] |= kLaneSettled;
        w[2] = (fl & kRegPred) ? 0xFFFFFFFFu : 0u;
        w[3] = en[2];
        w[4] = en[3];
        w[5] = en[4];
        rows[q] = p.rows[q];
        // a node that ignores the policy (level mask 0) gets its level-0 value at every index:
        // the kernel indexes the row with whatever byte it finds
        const bool uses_level = ((fl >> kMaskShift) & 255u) != 0;
        for (int l = 0; l < p.Lp; ++l) {
            const size_t src = q * p.Lp + (uses_level ? l : 0);
            unsigned char *t = tab.data() + q * d.tab_entry + (size_t)l * (fwd ? 12 : 4);
            std::memcpy(t, &p.lat[src], 4);
            if (fwd) {
                uint64_t bits;
                std::memcpy(&bits, &p.energy[src], 8);
                const uint32_t hi = (uint32_t)(bits >> 32), lo = (uint32_t)bits;
                std::memcpy(t + 4, &hi, 4);
                std::memcpy(t + 8, &lo, 4);
            }
        }
    }
    int rc = upload(&d.ent, ent.data(), ent.size() * 4);
    if (rc == EMO_OK) rc = upload(&d.tab, tab.data(), tab.size());
    if (rc == EMO_OK) rc = upload(&d.rows, rows.data(), rows.size() * 4);
    return rc;
}

void free_program_lane(DevProgramLane &d)
{
    if (d.ent) cudaFree(d.ent);
    if (d.tab) cudaFree(d.tab);
    if (d.rows) cudaFree(d.rows);
    d = DevProgramLane();
}

void free_program(DevProgram &d)
{
    if (d.rec) cudaFree(d.rec);
    if (d.rows) cudaFree(d.rows);
    if (d.groups) cudaFree(d.groups);
    d = DevProgram();
}

// Longest path with one duration per node (used for the overflow guard and the info block).
template <typename F>
__int128 host_longest(const HostGraph &h, F dur)
{
    std::vector<__int128> C((size_t)std::max(h.n, 1));
    __int128 T = 0;
    for (int32_t v = 0; v < h.n; ++v) {
        __int128 s = 0;
        for (int64_t e = h.row_ptr[v]; e < h.row_ptr[v + 1]; ++e) s = std::max(s, C[h.col[e]]);
        C[v] = s + dur(v);
        T = std::max(T, C[v]);
    }
    return T;
}

size_t lvl_area(const emo_graph *g) { return round_up((size_t)std::max(g->h.rows, 1) * 16, 256); }

struct LaunchShape {
    int groups, grid, threads;
    size_t smem;
};

// Policy groups (32 policies each) per block: enough to give every SM one block, bounded by the
// block size, the named barriers (ids 1..15) and shared memory.
int shape_for(const emo_graph *g, const Program &p, int64_t NB, LaunchShape &s)
{
    int64_t n_groups = (NB + 31) / 32;
    int gmax = std::min(32 / p.lanes, 15);
    if (gmax < 1) return EMO_E_UNSUPPORTED;
    size_t per_group = (size_t)p.slots * 256 + (size_t)p.lanes * 32 * 16;
    size_t budget = g->smem_optin ? g->smem_optin : 48 * 1024;
    while (gmax > 1 && per_group * gmax > budget) --gmax;
    if (per_group * gmax > budget) return EMO_E_UNSUPPORTED;
    int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    s.groups = (int)std::max<int64_t>(1, std::min<int64_t>(gmax, want));
    s.grid = (int)((n_groups + s.groups - 1) / s.groups);
    s.threads = s.groups * p.lanes * 32;
    s.smem = per_group * s.groups;
    return EMO_OK;
}

// Shape of the staged kernel: groups of 64 policies (two per thread), one more warp produces, then
// as many steps per stage as fit beside the slots.  Returns false when it cannot be used.
bool staged_shape(const emo_graph *g, const Program &p, int rec_bytes, bool backward, int64_t NB, LaunchShape &s,
                  StagedParams &sp)
{
    if (p.steps == 0 || !g->smem_optin) return false;
    int64_t n_groups = (NB + 63) / 64;
    int gmax = std::min((32 - kProducerWarps) / p.lanes, 15);
    if (gmax < 1) return false;
    int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    int G = (int)std::max<int64_t>(1, std::min<int64_t>(gmax, want));
    const size_t budget = g->smem_optin;
    static const int kTry[5][2] = {{16, 4}, {16, 3}, {8, 4}, {8, 3}, {8, 2}};   // {steps per stage, stages}
    for (; G >= 1; --G) {
        const size_t P = 64 * (size_t)G;
        const size_t fixed = (size_t)G * p.slots * kSlotStride + (size_t)G * p.lanes * 1024 + 256 + 128;
        for (int t = 0; t < 5; ++t) {
            const int sc = kTry[t][0], stages = kTry[t][1];
            const size_t ne = (size_t)sc * p.lanes;
            if (ne > 32 * (size_t)kRowRegs) continue;
            const size_t stage_bytes = round_up(ne * ((size_t)rec_bytes + P + (backward ? P * 8 : 0)), 128);
            if (fixed + stages * stage_bytes > budget) continue;
            sp.sc = sc;
            sp.stages = stages;
            sp.ptile = (int)P;
            sp.off_lvl = (unsigned)(ne * rec_bytes);
            sp.off_es = sp.off_lvl + (unsigned)(ne * P);
            sp.stage_bytes = (unsigned)stage_bytes;
            sp.off_part = (unsigned)round_up((size_t)G * p.slots * kSlotStride, 16);
            sp.off_bar = sp.off_part + (unsigned)((size_t)G * p.lanes * 1024);
            sp.off_stage0 = (unsigned)round_up(sp.off_bar + 256, 128);
            s.groups = G;
            s.grid = (int)((n_groups + G - 1) / G);
            s.threads = (G * p.lanes + kProducerWarps) * 32;
            s.smem = sp.off_stage0 + (size_t)stages * sp.stage_bytes;
            if (s.smem > budget) continue;
            return true;
        }
    }
    return false;
}

// Shape of the kernel with one warp per schedule lane and one policy per thread: groups of 32
// policies, one more warp produces; slot area, partial results, barriers, then the stage ring.
bool lane_shape(const emo_graph *g, const Program &p, bool backward, int64_t NB, LaunchShape &s, StagedParams &sp)
{
    if (p.steps == 0 || !g->smem_optin || !g->lfwd.ent || !g->lbwd.ent) return false;
    const size_t rec_bytes = 32 + (size_t)p.Lp * (backward ? 4 : 12);     // entry and table row
    const int64_t n_groups = (NB + 31) / 32;
    const int gmax = std::min((32 - kProducerWarps) / p.lanes, 15);
    if (gmax < 1) return false;
    const int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    int G = (int)std::max<int64_t>(1, std::min<int64_t>(gmax, want));
    const size_t budget = g->smem_optin;
    // {steps per stage, stages}: long stages first - a stage boundary costs every warp about a
    // microsecond (measured: 8, 16, 32 steps per stage gave 15.1, 12.3, 11.4 ms on the same forward
    // pass), while two stages hide the refill as well as four
    static const int kTry[10][2] = {{32, 2}, {16, 3}, {16, 2}, {8, 3}, {8, 2}, {4, 6}, {4, 5}, {4, 4}, {4, 3}, {4, 2}};
    for (; G >= 1; --G) {
        const size_t P = 32 * (size_t)G;
        const size_t slot_bytes = round_up((size_t)G * p.slots * kLaneSlotStride, 16);
        const size_t part_bytes = (size_t)G * p.lanes * 32 * 16;
        const size_t head = round_up(slot_bytes + part_bytes + 256, 128);
        for (int t = 0; t < 10; ++t) {
            const int sc = kTry[t][0], stages = kTry[t][1];
            const size_t ne = (size_t)sc * p.lanes;
            if (ne > 32 * (size_t)kRowRegs || stages > kMaxStages || kLaneStepPad % sc != 0) continue;
            const size_t stage_bytes = round_up(ne * (rec_bytes + P + (backward ? P * 8 : 0)), 128);
            // behind the last stage: room for the look-ahead of its last step
            const size_t pad = round_up((size_t)p.lanes * std::max<size_t>(P * 8, rec_bytes), 128);
            const size_t total = head + stages * stage_bytes + pad;
            if (total > budget) continue;
            sp.sc = sc;
            sp.stages = stages;
            sp.ptile = (int)P;
            sp.off_lvl = (unsigned)(ne * rec_bytes);
            sp.off_es = sp.off_lvl + (unsigned)(ne * P);
            sp.stage_bytes = (unsigned)stage_bytes;
            sp.off_part = (unsigned)slot_bytes;
            sp.off_bar = (unsigned)(slot_bytes + part_bytes);
            sp.off_stage0 = (unsigned)head;
            s.groups = G;
            s.grid = (int)((n_groups + G - 1) / G);
            s.threads = (G * p.lanes + kProducerWarps) * 32;
            s.smem = total;
            return true;
        }
    }
    return false;
}

// How the two passes of one call will run: both staged (earliest starts travel through the tiled
// spill) or both with the plain kernels (through an [n][ldes] array).
struct PassPlan {
    bool staged = false;
    bool lane_f = false, lane_b = false;   // staged, one policy per thread (forward / backward pass)
    LaunchShape sf{}, sb{};   // forward / backward launch shapes
    StagedParams pf{}, pb{};
    size_t spill_bytes = 0;   // tiled spill: [tiles][rows of the backward program][backward tile]
};

// rows of one tile of the spill: the entries of the backward program (padded to whole stages for the lane kernel)
size_t spill_rows_of(const emo_graph *g, bool lane)
{
    return (size_t)(lane ? g->lbwd.steps_pad : g->bwd.steps) * g->bwd.lanes;
}

bool aligned16(const void *q) { return ((uintptr_t)q % 16) == 0; }

// Decides the plan for B policies (+ the virtual baseline column in the forward pass).
int make_plan(const emo_graph *g, int64_t B, bool want_base, bool need_bwd, const uint8_t *lvl, int64_t ldb,
              int64_t ldes_plain, int64_t ldo, uint32_t flags, PassPlan &pl)
{
    const int64_t big = (int64_t)1 << 28;
    const int64_t NBf = B + (want_base ? 1 : 0);
    const bool can_stage = !(flags & EMO_F_NO_STAGING) && ldb % 16 == 0 && aligned16(lvl) && ldb < big && ldes_plain < big && ldo < big;
    // One policy per thread gives twice the warps, which the path is short of; once a batch is so
    // large that even two policies per thread give every SM 16 consumer warps, the pair kernel is
    // the cheaper one (measured: 65 536 policies, 3 lanes: 0.96 ms against 1.02 ms for both passes,
    // 0.24 ms against 0.42 ms for the forward pass).
    const int64_t pair_warps = (NBf + 63) / 64 * std::max(g->fwd.lanes, g->bwd.lanes);
    const bool prefer_pair = (flags & EMO_F_PAIR_KERNEL) || (!(flags & EMO_F_LANE_KERNEL) && pair_warps >= 16 * (int64_t)g->sm_count);
    // Each pass picks its kernel (they only share the spill, whose tiling follows the backward pass).
    // A pass whose lane-kernel grid would need a second wave of blocks while the pair kernel's fits
    // the SMs once takes the pair kernel (a wide forward program: 18 lanes leave room for one group
    // of 32 policies per block; measured 2.7 ms against 4.5 ms).
    auto pick = [&](const Program &p, int rec_bytes, bool backward, int64_t NB, LaunchShape &ls, StagedParams &sp, bool &lane) {
        LaunchShape l1, l2;
        StagedParams s1, s2;
        const bool ok_lane = lane_shape(g, p, backward, NB, l1, s1);
        const bool ok_pair = staged_shape(g, p, rec_bytes, backward, NB, l2, s2);
        bool use_lane = ok_lane && !prefer_pair;
        if (use_lane && ok_pair && !(flags & EMO_F_LANE_KERNEL) && !backward && l1.grid > g->sm_count && l2.grid <= g->sm_count) use_lane = false;
        if (!use_lane && !ok_pair) use_lane = ok_lane;
        if (use_lane) { ls = l1; sp = s1; lane = true; return true; }
        if (ok_pair) { ls = l2; sp = s2; lane = false; return true; }
        return false;
    };
    pl.staged = can_stage && pick(g->fwd, g->dfwd.rec_bytes, false, NBf, pl.sf, pl.pf, pl.lane_f) &&
                (!need_bwd || pick(g->bwd, g->dbwd.rec_bytes, true, B, pl.sb, pl.pb, pl.lane_b));
    if (!pl.staged) {
        int rc = shape_for(g, g->fwd, NBf, pl.sf);
        if (rc == EMO_OK && need_bwd) rc = shape_for(g, g->bwd, B, pl.sb);
        return rc;
    }
    if (need_bwd) {
        const size_t tiles = ((size_t)B + pl.pb.ptile - 1) / pl.pb.ptile;
        pl.spill_bytes = tiles * spill_rows_of(g, pl.lane_b) * pl.pb.ptile * sizeof(int64_t);
    }
    return EMO_OK;
}

// One pass under a plan.  Forward: B policies from lvl plus, when base_T/base_E are given, the
// virtual all-max column.
int launch_pass(const emo_graph *g, const PassPlan &pl, bool backward, int64_t B, const uint8_t *lvl, int64_t ldb,
                int64_t *ES, int64_t ldes, int64_t *spill, int64_t *LS, int64_t *slack, int64_t ldo,
                int64_t *makespan, double *energy, int64_t *slack_sum, int32_t *n_critical,
                int64_t *base_T, double *base_E, int32_t *status, cudaStream_t st)
{
    const Program &p = backward ? g->bwd : g->fwd;
    const DevProgram &d = backward ? g->dbwd : g->dfwd;
    const int want_base = (!backward && (base_T || base_E)) ? 1 : 0;
    if (B + want_base == 0) return EMO_OK;
    const LaunchShape &s = backward ? pl.sb : pl.sf;
    PassParams a;
    a.rec = d.rec;
    a.rows = d.rows;
    a.rec_bytes = d.rec_bytes;
    a.steps = p.steps;
    a.lanes = p.lanes;
    a.Lp = p.Lp;
    a.L = g->h.L;
    a.slots = p.slots;
    a.sync = p.sync;
    a.groups = s.groups;
    a.want_base = want_base;
    a.B = B;
    a.lvl = lvl;
    a.ldb = ldb;
    a.ES = ES;
    a.ldes = ldes;
    a.spill = spill;
    a.spill_rows = (int64_t)spill_rows_of(g, pl.lane_b);
    a.spill_ptile = pl.staged ? pl.pb.ptile : 64;
    a.LS = LS;
    a.slack = slack;
    a.ldo = ldo;
    a.makespan = makespan;
    a.energy = energy;
    a.slack_sum = slack_sum;
    a.n_critical = n_critical;
    a.base_T = base_T;
    a.base_E = base_E;
    a.status = status;
    cudaEvent_t ev0 = g_pass_events[backward ? 2 : 0], ev1 = g_pass_events[backward ? 3 : 1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    if (pl.staged) {
        StagedParams sp = backward ? pl.pb : pl.pf;
        sp.p = a;
        sp.vec_es = (ES && ldes % 2 == 0 && aligned16(ES)) ? 1 : 0;
        sp.vec_out = (ldo % 2 == 0 && aligned16(LS) && aligned16(slack)) ? 1 : 0;
        sp.want_sums = (slack_sum || n_critical) ? 1 : 0;
        // two register budgets: blocks of at most 512 threads may use 128 registers per thread
        // lean instantiation when the call asks for nothing beyond the spill (forward) or the slack
        // matrix with 16-byte aligned rows (backward); register budget by block size
        const bool extra = backward ? (LS != nullptr || sp.want_sums || !sp.vec_out) : (ES != nullptr);
        void (*kern)(StagedParams) = nullptr;
        if (backward ? pl.lane_b : pl.lane_f) {
            const DevProgramLane &di = backward ? g->lbwd : g->lfwd;
            LaneParams ip;
            const unsigned ne = (unsigned)sp.sc * (unsigned)p.lanes;
            sp.p.steps = di.steps_pad;
            sp.p.rows = di.rows;
            ip.tab_entry = di.tab_entry;
            ip.st.off_tab = ne * 32u;
            int nb = 0;
            auto bulk = [&](const void *src, unsigned per_entry, unsigned off, unsigned long long per_block) {
                sp.bsrc[nb] = (const unsigned char *)src;
                sp.bentry[nb] = per_entry;
                sp.boff[nb] = off;
                sp.bblock[nb] = per_block;
                ++nb;
            };
            bulk(di.ent, 32, 0, 0);
            bulk(di.tab, di.tab_entry, ip.st.off_tab, 0);
            if (backward) bulk(spill, (unsigned)sp.ptile * 8u, sp.off_es, (unsigned long long)a.spill_rows * sp.ptile * 8ull);
            sp.nbulk = nb;
            void (*kern_lane)(LaneParams) = nullptr;
            const bool extra_l = backward ? (LS != nullptr || sp.want_sums) : (ES != nullptr);
#define EMO_PICK_L(MAXT)                                                                                        \
    kern_lane = backward ? (extra_l ? emo_pass_lane<true, true, MAXT> : emo_pass_lane<true, false, MAXT>)           \
                        : (extra_l ? emo_pass_lane<false, true, MAXT> : emo_pass_lane<false, false, MAXT>)
            if (s.threads <= 512) EMO_PICK_L(512);
            else if (s.threads <= 768) EMO_PICK_L(768);
            else EMO_PICK_L(1024);
#undef EMO_PICK_L
            ip.sp = sp;
            EMO_CUDA(cudaFuncSetAttribute(kern_lane, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin));      // the same value from every call
            kern_lane<<<s.grid, s.threads, s.smem, st>>>(ip);
        } else {
            sp.nbulk = 0;
            sp.bsrc[sp.nbulk] = d.rec; sp.bentry[sp.nbulk] = (unsigned)d.rec_bytes; sp.boff[sp.nbulk] = 0; sp.bblock[sp.nbulk] = 0;
            ++sp.nbulk;
            if (backward) {
                sp.bsrc[sp.nbulk] = (const unsigned char *)spill; sp.bentry[sp.nbulk] = (unsigned)sp.ptile * 8u; sp.boff[sp.nbulk] = sp.off_es;
                sp.bblock[sp.nbulk] = (unsigned long long)a.spill_rows * sp.ptile * 8ull;
                ++sp.nbulk;
            }
#define EMO_PICK(MAXT)                                                                                         \
    kern = backward ? (extra ? emo_pass_pair<true, true, MAXT> : emo_pass_pair<true, false, MAXT>)                 \
                    : (extra ? emo_pass_pair<false, true, MAXT> : emo_pass_pair<false, false, MAXT>)
        if (s.threads <= 512) EMO_PICK(512);
        else if (s.threads <= 768) EMO_PICK(768);
        else EMO_PICK(1024);
#undef EMO_PICK
        EMO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin));
        kern<<<s.grid, s.threads, s.smem, st>>>(sp);
        }
    } else if (backward) {
        if (s.smem > 48 * 1024) EMO_CUDA(cudaFuncSetAttribute(emo_pass_plain<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin));
        emo_pass_plain<true><<<s.grid, s.threads, s.smem, st>>>(a);
    } else {
        if (s.smem > 48 * 1024) EMO_CUDA(cudaFuncSetAttribute(emo_pass_plain<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin));
        emo_pass_plain<false><<<s.grid, s.threads, s.smem, st>>>(a);
    }
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}


// ---- lane-stream program: upload, launch shape, launches -------------------------------------------
long long *g_flow_prof = nullptr;           // optional device array for the kernels' cycle counters (measurement hook)
long long g_wait_cycles = 4000000000LL;    // bound of every device-side wait of the 32-bit kernels (about two seconds)

int upload_flow(const Flow &f, DevFlow &d, bool intervals)
{
    if (!f.ok32 || f.stages == 0) return EMO_OK;
    const size_t per = (size_t)f.lanes * f.K;
    auto r16 = [](size_t x) { return (x + 15) / 16 * 16; };
    d.off_seg = (unsigned)r16((size_t)f.lanes * kHdrWords * 4);
    d.f_off_rec = (unsigned)r16(d.off_seg + (size_t)f.lanes * kSegBytes);
    d.f_off_pool = (unsigned)r16(d.f_off_rec + per * kFRecWords * 4);
    d.f_off_tab = (unsigned)r16(d.f_off_pool + (size_t)f.f.pool_stride * 4);
    d.blobF_bytes = (unsigned)r16(d.f_off_tab + per * f.Lp * 12);
    d.b_off_rec = d.f_off_rec;
    d.b_off_pool = (unsigned)r16(d.b_off_rec + per * kBRecWords * 4);
    d.b_off_lbes = (unsigned)r16(d.b_off_pool + (size_t)f.b.pool_stride * 4);
    d.b_off_tab = (unsigned)r16(d.b_off_lbes + per * 8);
    d.blobB_bytes = (unsigned)r16(d.b_off_tab + per * f.Lp * 4);
    std::vector<unsigned char> bf((size_t)f.stages * d.blobF_bytes, 0), bb((size_t)f.stages * d.blobB_bytes, 0);
    std::vector<uint32_t> pb((size_t)f.stages + 1);
    for (int st = 0; st <= f.stages; ++st) pb[st] = (uint32_t)f.push_base[st];
    for (int st = 0; st < f.stages; ++st) {
        d.max_push = std::max(d.max_push, (int)(pb[st + 1] - pb[st]));
        std::vector<uint32_t> hdr(f.hdr.begin() + (size_t)st * f.lanes * kHdrWords, f.hdr.begin() + (size_t)(st + 1) * f.lanes * kHdrWords);
        unsigned char *F = bf.data() + (size_t)st * d.blobF_bytes, *Bk = bb.data() + (size_t)st * d.blobB_bytes;
        std::memcpy(F, hdr.data(), hdr.size() * 4);
        std::memcpy(Bk, hdr.data(), hdr.size() * 4);
        std::memcpy(F + d.off_seg, &f.f.seg[(size_t)st * f.lanes * kSegBytes], (size_t)f.lanes * kSegBytes);
        std::memcpy(Bk + d.off_seg, &f.b.seg[(size_t)st * f.lanes * kSegBytes], (size_t)f.lanes * kSegBytes);
        std::memcpy(F + d.f_off_rec, &f.f.rec[(size_t)st * per * kFRecWords], per * kFRecWords * 4);
        std::memcpy(F + d.f_off_pool, &f.f.pool[(size_t)st * f.f.pool_stride], (size_t)f.f.pool_stride * 4);
        std::memcpy(F + d.f_off_tab, &f.tabF[(size_t)st * per * f.Lp * 3], per * f.Lp * 12);
        std::memcpy(Bk + d.b_off_rec, &f.b.rec[(size_t)st * per * kBRecWords], per * kBRecWords * 4);
        std::memcpy(Bk + d.b_off_pool, &f.b.pool[(size_t)st * f.b.pool_stride], (size_t)f.b.pool_stride * 4);
        std::memcpy(Bk + d.b_off_lbes, &f.lbes[(size_t)st * per], per * 8);
        std::memcpy(Bk + d.b_off_tab, &f.tabB[(size_t)st * per * f.Lp], per * f.Lp * 4);
    }
    int rc = upload(&d.blobF, bf.data(), bf.size());
    if (rc == EMO_OK) rc = upload(&d.blobB, bb.data(), bb.size());
    if (rc == EMO_OK && intervals) {
        d.f_off_meta = d.blobF_bytes;
        d.blobFI_bytes = (unsigned)r16(d.f_off_meta + per * 16);
        std::vector<unsigned char> bi((size_t)f.stages * d.blobFI_bytes, 0);
        for (int st = 0; st < f.stages; ++st) {
            unsigned char *dst = bi.data() + (size_t)st * d.blobFI_bytes;
            std::memcpy(dst, bf.data() + (size_t)st * d.blobF_bytes, d.blobF_bytes);
            for (size_t e = 0; e < per; ++e) {
                const size_t q = (size_t)st * per + e;
                const int64_t lb = f.lbes[q];
                const uint32_t w[4] = {(uint32_t)(uint64_t)lb, (uint32_t)((uint64_t)lb >> 32), f.grp[q], f.dmin[q]};
                std::memcpy(dst + d.f_off_meta + e * 16, w, 16);
            }
        }
        rc = upload(&d.blobFI, bi.data(), bi.size());
    }
    if (rc == EMO_OK) rc = upload(&d.rows, f.rows.data(), f.rows.size() * 4);
    if (rc == EMO_OK) rc = upload(&d.push_base, pb.data(), pb.size() * 4);
    d.ready = rc == EMO_OK;
    return rc;
}

void free_flow(DevFlow &d)
{
    if (d.blobF) cudaFree(d.blobF);
    if (d.blobB) cudaFree(d.blobB);
    if (d.blobFI) cudaFree(d.blobFI);
    if (d.rows) cudaFree(d.rows);
    if (d.push_base) cudaFree(d.push_base);
    d = DevFlow();
}


int upload_spine(const Flow &f, DevSpine &d)
{
    const Spine &sp = f.spine;
    if (!f.ok32 || !sp.ok || f.stages == 0) return EMO_OK;
    const size_t per = (size_t)f.lanes * f.K;
    auto r16 = [](size_t x) { return (x + 15) / 16 * 16; };
    // forward: header, terminal bounds and operations lie together at the front (what the spine needs: a worker copies
    // it to the group's own ring, so that the stage buffer is free again as soon as the sums are taken)
    d.f_off_tpool = 16;
    d.f_off_ops = (unsigned)r16(d.f_off_tpool + (size_t)sp.max_pool * 8);
    d.f_front = (unsigned)(d.f_off_ops + (size_t)(sp.f.max_ops + 1) * kSpOpWordsF * 4);
    d.f_off_pos = d.f_front;
    d.f_off_tab = (unsigned)r16(d.f_off_pos + per * 4);
    d.blobF_bytes = (unsigned)r16(d.f_off_tab + per * f.Lp * 12);
    d.b_off_ops = 16;
    d.b_off_mem = (unsigned)(d.b_off_ops + (size_t)(sp.b.max_ops + 1) * kSpOpWordsB * 4);
    d.b_off_tab = (unsigned)(d.b_off_mem + per * kSpMemWords * 4);
    d.blobB_bytes = (unsigned)r16(d.b_off_tab + per * f.Lp * 4);
    std::vector<unsigned char> bf((size_t)f.stages * d.blobF_bytes, 0), bb((size_t)f.stages * d.blobB_bytes, 0);
    std::vector<uint32_t> pb((size_t)f.stages + 1);
    for (int st = 0; st <= f.stages; ++st) pb[st] = (uint32_t)sp.push_base[st];
    for (int st = 0; st < f.stages; ++st) {
        d.max_push = std::max(d.max_push, (int)(pb[st + 1] - pb[st]));
        unsigned char *F = bf.data() + (size_t)st * d.blobF_bytes, *Bk = bb.data() + (size_t)st * d.blobB_bytes;
        const uint32_t hf[4] = {sp.f.n_ops[st], sp.n_segs[st], pb[st], (uint32_t)sp.pair_base[st]}, hb[4] = {sp.b.n_ops[st], sp.n_segs[st], pb[st], 0u};
        std::memcpy(F, hf, 16);
        std::memcpy(Bk, hb, 16);
        std::memcpy(F + d.f_off_ops, &sp.f.ops[(size_t)st * sp.f.max_ops * kSpOpWordsF], (size_t)sp.f.max_ops * kSpOpWordsF * 4);
        std::memcpy(Bk + d.b_off_ops, &sp.b.ops[(size_t)st * sp.b.max_ops * kSpOpWordsB], (size_t)sp.b.max_ops * kSpOpWordsB * 4);
        std::memcpy(F + d.f_off_tpool, &sp.pool[(size_t)st * sp.max_pool], (size_t)sp.max_pool * 8);
        std::memcpy(F + d.f_off_pos, &sp.posw[(size_t)st * per], per * 4);
        std::memcpy(Bk + d.b_off_mem, &sp.mem[(size_t)st * per * kSpMemWords], per * kSpMemWords * 4);
        std::memcpy(Bk + d.b_off_tab, &f.tabB[(size_t)st * per * f.Lp], per * f.Lp * 4);
        // forward table rows: {duration, energy high word, low word} per level, 12 bytes apart (3 is coprime with the 32
        // banks: the 32 policies of a warp, whatever their levels, read each of the three words without a bank conflict)
        std::memcpy(F + d.f_off_tab, &f.tabF[(size_t)st * per * f.Lp * 3], per * f.Lp * 12);
    }
    int rc = upload(&d.blobF, bf.data(), bf.size());
    if (rc == EMO_OK) rc = upload(&d.blobB, bb.data(), bb.size());
    if (rc == EMO_OK) rc = upload(&d.rows, f.rows.data(), f.rows.size() * 4);
    if (rc == EMO_OK) rc = upload(&d.push_base, pb.data(), pb.size() * 4);
    d.ready = rc == EMO_OK;
    return rc;
}

void free_spine(DevSpine &d)
{
    if (d.blobF) cudaFree(d.blobF);
    if (d.blobB) cudaFree(d.blobB);
    if (d.rows) cudaFree(d.rows);
    if (d.push_base) cudaFree(d.push_base);
    d = DevSpine();
}

// Launch shape of the 32-bit kernels: both passes use the same policy tile (the restore list is laid
// out by tile), as many groups per block as cover the SMs once, two stage buffers (three when they fit).
struct FlowPlan {
    bool ok = false;
    int groups = 0, grid_f = 0, grid_b = 0, threads = 0;
    FlowParams pf, pb;
    size_t smem_f = 0, smem_b = 0;
    size_t restore_bytes = 0;
};

// intv: the plan of the forward kernel for time-interval policies (no level rows are staged; the blob carries
// 16 more bytes per entry; extra_fixed + G * extra_per_group bytes of the block are set aside for the change
// points and the block's columns of F).
bool flow_plan(const emo_graph *g, int64_t B, bool want_base, bool need_bwd, FlowPlan &pl, bool intv = false,
               size_t extra_fixed = 0, size_t extra_per_group = 0)
{
    const Flow &f = g->flow;
    const DevFlow &d = g->dflow;
    pl.ok = false;
    if (!f.ok32 || !d.ready || !g->smem_optin || f.stages == 0) return false;
    if (intv && !d.blobFI) return false;
    if (f.lanes * f.K > 32 * kFlowRowRegs) return false;
    const int64_t NBf = B + (want_base ? 1 : 0);
    const int64_t n_groups = (NBf + 31) / 32;
    const int gmax = std::min((32 - 2) / f.lanes, 15);
    if (gmax < 1) return false;
    const int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    const size_t budget = g->smem_optin;
    for (int G = (int)std::max<int64_t>(1, std::min<int64_t>(gmax, want)); G >= 1; --G) {
        // four producer warps where the block has room for them (they share the level-row pieces)
        const int nprod = G * f.lanes + 4 <= 24 ? 4 : 2;
        const size_t P = 32 * (size_t)G;
        const size_t lvl_bytes = intv ? 0 : (size_t)G * f.lanes * f.K * 32;
        const size_t extra = intv ? round_up(extra_fixed + extra_per_group * G, 128) : 0;
        auto shape = [&](bool backward, FlowParams &p, size_t &smem) {
            const FlowDir &dir = backward ? f.b : f.f;
            const size_t slot_bytes = (size_t)dir.slots_tag * 256 + (size_t)dir.slots_set * 128;
            const size_t blob = backward ? d.blobB_bytes : (intv ? d.blobFI_bytes : d.blobF_bytes);
            const size_t rst = backward ? (size_t)d.max_push * P * 4 : 0;
            const size_t stage = round_up(blob + lvl_bytes + rst, 128);
            const size_t off_bar = round_up(G * slot_bytes, 16);
            const size_t head = round_up(off_bar + 256, 128) + extra;
            int nbuf = 0;
            for (int nb = 3; nb >= 2; --nb)
                if (head + nb * stage <= budget) { nbuf = nb; break; }
            if (!nbuf || nbuf * stage < (size_t)G * f.lanes * 32 * 16) return false;
            p = FlowParams();
            p.blob = backward ? d.blobB : (intv ? d.blobFI : d.blobF);
            p.rows = d.rows;
            p.push_base = d.push_base;
            p.blob_bytes = (unsigned)blob;
            p.off_seg = d.off_seg;
            p.off_rec = backward ? d.b_off_rec : d.f_off_rec;
            p.off_pool = backward ? d.b_off_pool : d.f_off_pool;
            p.off_tab = backward ? d.b_off_tab : d.f_off_tab;
            p.off_lbes = backward ? d.b_off_lbes : 0;
            p.off_meta = d.f_off_meta;
            p.off_brk = (unsigned)round_up(off_bar + 256, 128);
            p.off_Fs = p.off_brk + (unsigned)round_up(extra_fixed, 16);
            p.tab_row = (unsigned)f.Lp * (backward ? 4u : 12u);
            p.stages = f.stages;
            p.lanes = f.lanes;
            p.K = f.K;
            p.kshift = 0;
            while ((1 << p.kshift) < f.K) ++p.kshift;
            p.Lp = f.Lp;
            p.L = g->h.L;
            p.groups = G;
            p.ptile = (int)P;
            p.nbuf = nbuf;
            p.nprod = nprod;
            p.slot_bytes = (unsigned)slot_bytes;
            p.stage_bytes = (unsigned)stage;
            p.off_lvl = (unsigned)blob;
            p.off_rst = (unsigned)(blob + lvl_bytes);
            p.off_bar = (unsigned)off_bar;
            p.off_stage0 = (unsigned)head;
            p.pushes = f.pushes;
            p.restore_rows = f.pushes + f.lanes;
            p.wait_cycles = g_wait_cycles;
            p.stall_stage = -1;
            p.prof = nullptr;
            smem = head + nbuf * stage;
            return true;
        };
        if (!shape(false, pl.pf, pl.smem_f)) continue;
        if (need_bwd && !shape(true, pl.pb, pl.smem_b)) continue;
        pl.groups = G;
        pl.grid_f = (int)((n_groups + G - 1) / G);
        pl.grid_b = (int)(((B + 31) / 32 + G - 1) / G);
        pl.threads = (G * f.lanes + nprod) * 32;
        pl.restore_bytes = need_bwd ? round_up((size_t)pl.grid_f * (size_t)(f.pushes + f.lanes) * P * 4, 256) : 0;
        pl.ok = true;
        return true;
    }
    return false;
}

// The opt-in shared-memory size is set once per kernel (not per launch: concurrent callers with
// different batch sizes would otherwise race on the attribute).
template <typename K>
int flow_optin(K kern, const emo_graph *g)
{
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin) == cudaSuccess ? EMO_OK : EMO_E_CUDA;
}

int launch_flow_fwd(const emo_graph *g, const FlowPlan &pl, int64_t B, const uint8_t *lvl, int64_t ldb, uint32_t *restore,
                    int64_t *makespan, double *energy, int64_t *base_T, double *base_E, int32_t *status, uint32_t flags,
                    cudaStream_t st)
{
    FlowParams p = pl.pf;
    p.want_base = (base_T || base_E) ? 1 : 0;
    if (B + p.want_base == 0) return EMO_OK;
    p.B = B;
    p.lvl = lvl;
    p.ldb = ldb;
    p.restore = restore;
    p.makespan = makespan;
    p.energy = energy;
    p.base_T = base_T;
    p.base_E = base_E;
    p.status = status;
    p.prof = g_flow_prof;
    if (flags & EMO_F_TEST_STALL) p.stall_stage = p.stages / 2;
    cudaEvent_t ev0 = g_pass_events[0], ev1 = g_pass_events[1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    void (*kern)(FlowParams) = nullptr;
    if (p.prof) kern = pl.threads <= 512 ? emo_flow_fwd<512, false, true> : (pl.threads <= 768 ? emo_flow_fwd<768, false, true> : emo_flow_fwd<1024, false, true>);
    else kern = pl.threads <= 512 ? emo_flow_fwd<512, false, false> : (pl.threads <= 768 ? emo_flow_fwd<768, false, false> : emo_flow_fwd<1024, false, false>);
    if (flow_optin(kern, g) != EMO_OK) { (void)cudaGetLastError(); return EMO_E_CUDA; }
    kern<<<pl.grid_f, pl.threads, pl.smem_f, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

int launch_flow_bwd(const emo_graph *g, const FlowPlan &pl, int64_t B, const uint8_t *lvl, int64_t ldb, uint32_t *restore,
                    int64_t *ES, int64_t *LS, int64_t *slack, int64_t ldo, int64_t *makespan, int64_t *slack_sum,
                    int32_t *n_critical, int32_t *status, uint32_t flags, cudaStream_t st)
{
    if (B == 0) return EMO_OK;
    FlowParams p = pl.pb;
    p.B = B;
    p.lvl = lvl;
    p.ldb = ldb;
    p.restore = restore;
    p.makespan = makespan;
    p.ES = ES;
    p.LS = LS;
    p.slack = slack;
    p.ldo = ldo;
    p.slack_sum = slack_sum;
    p.n_critical = n_critical;
    p.status = status;
    p.prof = g_flow_prof ? g_flow_prof + 131072 : nullptr;
    if (flags & EMO_F_TEST_STALL) p.stall_stage = p.stages / 2;
    cudaEvent_t ev0 = g_pass_events[2], ev1 = g_pass_events[3];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    const bool extra = ES || LS || slack_sum || n_critical;
    void (*kern)(FlowParams) = nullptr;
#define EMO_PICK_F(MAXT)                                                                                   \
    kern = p.prof ? (extra ? emo_flow_bwd<true, MAXT, true> : emo_flow_bwd<false, MAXT, true>)                 \
                  : (extra ? emo_flow_bwd<true, MAXT, false> : emo_flow_bwd<false, MAXT, false>)
    if (pl.threads <= 512) EMO_PICK_F(512);
    else if (pl.threads <= 768) EMO_PICK_F(768);
    else EMO_PICK_F(1024);
#undef EMO_PICK_F
    if (flow_optin(kern, g) != EMO_OK) { (void)cudaGetLastError(); return EMO_E_CUDA; }
    kern<<<pl.grid_b, pl.threads, pl.smem_b, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

// Launch shape of the spine kernels: the policy tile of flow_plan; per group one spine warp and as many worker
// warps as the block has room for (at most 6); three buffers of sums when they fit (workers one stage ahead and
// one behind the spine) and up to six stage buffers.
bool spine_plan(const emo_graph *g, int64_t B, bool want_base, bool need_bwd, FlowPlan &pl, bool extra = false)
{
    const Flow &f = g->sflow;
    const Spine &sp = f.spine;
    const DevSpine &d = g->dspine;
    pl.ok = false;
    if (!f.ok32 || !sp.ok || !d.ready || !g->smem_optin || f.stages == 0) return false;
    if (f.lanes * f.K > 32 * kFlowRowRegs) return false;
    const int64_t NBf = B + (want_base ? 1 : 0);
    const int64_t n_groups = (NBf + 31) / 32;
    const int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    const size_t budget = g->smem_optin;
    for (int G = (int)std::max<int64_t>(1, std::min<int64_t>(7, want)); G >= 1; --G) {
        const int nprod = G <= 4 ? 4 : 2;
        // a worker takes whole lanes: more workers than lanes would only wait
        const int W = std::min(f.lanes, std::min(6, (32 - nprod - G) / G));
        if (W < 1) continue;
        const size_t P = 32 * (size_t)G;
        const size_t lvl_bytes = (size_t)G * f.lanes * f.K * 32;
        auto shape = [&](bool backward, FlowParams &p, size_t &smem) {
            const SpineDir &dir = backward ? sp.b : sp.f;
            const size_t slot_bytes = (size_t)dir.slots * 128;
            const size_t acc_bytes = (size_t)((backward && extra) ? sp.acc_words_all : sp.acc_words) * 128;
            const size_t blob = backward ? d.blobB_bytes : d.blobF_bytes;
            const size_t rst = backward ? (size_t)d.max_push * P * 4 : 0;
            const size_t stage = round_up(blob + lvl_bytes + rst, 128);
            const size_t off_bar = round_up(G * slot_bytes, 16);
            const size_t off_sbar = off_bar + 192;
            const size_t oring = backward ? 0 : d.f_front;      // forward: the spine's part of a stage, per group and buffer of sums
            const size_t off_oring = round_up(off_sbar + (size_t)G * kFlowMaxBuf * 3 * 8, 128);
            int nbuf = 0, nacc = 0;
            size_t head = 0, off_acc = 0;
            // a stage is short (about a microsecond of work): several stages must be on their way at any time
            for (int na = 3; na >= 2 && !nbuf; --na)
                for (int nb = std::min(6, kFlowMaxBuf); nb >= 2 && !nbuf; --nb) {
                    off_acc = round_up(off_oring + (size_t)na * G * oring, 128);
                    head = round_up(off_acc + (size_t)na * G * acc_bytes, 128);
                    if (head + nb * stage <= budget) {
                        nbuf = nb;
                        nacc = na;
                    }
                }
            if (!nbuf || nbuf * stage < (size_t)G * W * 32 * 8) return false;
            p = FlowParams();
            p.blob = backward ? d.blobB : d.blobF;
            p.rows = d.rows;
            p.push_base = d.push_base;
            p.blob_bytes = (unsigned)blob;
            p.off_ops = backward ? d.b_off_ops : d.f_off_ops;
            p.off_mem = d.b_off_mem;
            p.off_tpool = d.f_off_tpool;
            p.off_pos = d.f_off_pos;
            p.off_tab = backward ? d.b_off_tab : d.f_off_tab;
            p.tab_row = (unsigned)f.Lp * (backward ? 4u : 12u);
            p.stages = f.stages;
            p.lanes = f.lanes;
            p.K = f.K;
            p.Lp = f.Lp;
            p.L = g->h.L;
            p.groups = G;
            p.ptile = (int)P;
            p.nbuf = nbuf;
            p.nacc = nacc;
            p.nprod = nprod;
            p.workers = W;
            p.slot_bytes = (unsigned)slot_bytes;
            p.stage_bytes = (unsigned)stage;
            p.off_lvl = (unsigned)blob;
            p.off_rst = (unsigned)(blob + lvl_bytes);
            p.off_bar = (unsigned)off_bar;
            p.off_sbar = (unsigned)off_sbar;
            p.off_acc = (unsigned)off_acc;
            p.off_oring = (unsigned)off_oring;
            p.oring_bytes = (unsigned)oring;
            p.acc_bytes = (unsigned)acc_bytes;
            p.acc_all_off = (unsigned)sp.acc_words * 128u;
            p.off_stage0 = (unsigned)head;
            p.pushes = sp.pushes;
            p.restore_rows = sp.pushes + f.lanes;
            p.wait_cycles = g_wait_cycles;
            p.stall_stage = -1;
            p.prof = nullptr;
            smem = head + nbuf * stage;
            return true;
        };
        if (!shape(false, pl.pf, pl.smem_f)) continue;
        if (need_bwd && !shape(true, pl.pb, pl.smem_b)) continue;
        pl.groups = G;
        pl.grid_f = (int)((n_groups + G - 1) / G);
        pl.grid_b = (int)(((B + 31) / 32 + G - 1) / G);
        pl.threads = (G * (1 + W) + nprod) * 32;
        pl.restore_bytes = need_bwd ? round_up((size_t)pl.grid_f * (size_t)(sp.pushes + f.lanes) * P * 4, 256) : 0;
        pl.ok = true;
        return true;
    }
    return false;
}

int launch_spine_fwd(const emo_graph *g, const FlowPlan &pl, int64_t B, const uint8_t *lvl, int64_t ldb, uint32_t *restore,
                     int64_t *makespan, double *energy, int64_t *base_T, double *base_E, int32_t *status, uint32_t flags,
                     cudaStream_t st, bool pair = false)
{
    FlowParams p = pl.pf;
    p.pair_rows = pair ? 1 : 0;
    p.want_base = (base_T || base_E) ? 1 : 0;
    if (B + p.want_base == 0) return EMO_OK;
    p.B = B;
    p.lvl = lvl;
    p.ldb = ldb;
    p.restore = restore;
    p.makespan = makespan;
    p.energy = energy;
    p.base_T = base_T;
    p.base_E = base_E;
    p.status = status;
    p.prof = g_flow_prof;
    if (flags & EMO_F_TEST_STALL) p.stall_stage = p.stages / 2;
    cudaEvent_t ev0 = g_pass_events[0], ev1 = g_pass_events[1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    void (*kern)(FlowParams) = pl.threads <= 512 ? emo_spine_fwd<512> : emo_spine_fwd<1024>;
    if (flow_optin(kern, g) != EMO_OK) { (void)cudaGetLastError(); return EMO_E_CUDA; }
    kern<<<pl.grid_f, pl.threads, pl.smem_f, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

int launch_spine_bwd(const emo_graph *g, const FlowPlan &pl, int64_t B, const uint8_t *lvl, int64_t ldb, uint32_t *restore,
                     int64_t *ES, int64_t *LS, int64_t *slack, int64_t ldo, int64_t *makespan, int64_t *slack_sum,
                     int32_t *n_critical, int32_t *status, uint32_t flags, cudaStream_t st)
{
    if (B == 0) return EMO_OK;
    FlowParams p = pl.pb;
    p.B = B;
    p.lvl = lvl;
    p.ldb = ldb;
    p.restore = restore;
    p.makespan = makespan;
    p.ES = ES;
    p.LS = LS;
    p.slack = slack;
    p.ldo = ldo;
    p.slack_sum = slack_sum;
    p.n_critical = n_critical;
    p.status = status;
    p.prof = g_flow_prof ? g_flow_prof + 131072 : nullptr;
    if (flags & EMO_F_TEST_STALL) p.stall_stage = p.stages / 2;
    cudaEvent_t ev0 = g_pass_events[2], ev1 = g_pass_events[3];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    const bool extra = ES || LS || slack_sum || n_critical;
    void (*kern)(FlowParams) = pl.threads <= 512 ? (extra ? emo_spine_bwd<512, true> : emo_spine_bwd<512, false>)
                                                 : (extra ? emo_spine_bwd<1024, true> : emo_spine_bwd<1024, false>);
    if (flow_optin(kern, g) != EMO_OK) { (void)cudaGetLastError(); return EMO_E_CUDA; }
    kern<<<pl.grid_b, pl.threads, pl.smem_b, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

// Whether the forward spine kernel can feed the lane-stream backward kernel: both programs come from one schedule (same
// lanes and steps; the lane-stream program's barrier distance is the gap that the spine program's schedule keeps) and
// the restore rows could be numbered the lane-stream way.
bool spine_pairs(const emo_graph *g)
{
    const Flow &f = g->flow, &s = g->sflow;
    return f.ok32 && s.ok32 && s.spine.ok && g->dspine.ready && s.spine.pair_ok && s.spine.pair_K == f.K && f.sync == 2 * s.K &&
           f.steps == s.steps && f.lanes == s.lanes && f.pushes == s.spine.pushes && s.lanes <= 8;
}

// Whether a call takes the spine kernels: the program exists and either the caller asks for them (EMO_F_SPINE_KERNEL) or
// the graph is narrow and the batch leaves at most three policy groups to an SM (or the graph is short).
bool spine_allowed(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t ldo, bool fwd_only, uint32_t flags)
{
    const int64_t big = (int64_t)1 << 28;
    if (!g->sflow.ok32 || !g->sflow.spine.ok || !g->dspine.ready) return false;
    if (flags & (EMO_F_NO_STAGING | EMO_F_PAIR_KERNEL | EMO_F_LANE_KERNEL | EMO_F_FLOW_KERNEL)) return false;
    // Measured: on graphs of up to eight lanes the spine kernels are the fastest pair while a block holds at most three
    // policy groups (75 000 nodes, both passes, spine / lane-stream: 3.6 / 5.5 ms with one group per SM, 4.4 / 6.0 with
    // two, 5.7 / 6.3 with three, 8.9 / 6.8 with four: the workers then take the issue slots and the shared-memory pipe
    // that the spine warp needs) and on short graphs whatever the batch (1 013 nodes x 65 536 policies: 0.61 against
    // 0.90 ms); one warp carries the recurrence of all lanes, so wide graphs (17 lanes: 21.9 against 9.0 ms) stay with
    // the other kernels unless the caller asks.
    if (!(flags & EMO_F_SPINE_KERNEL)) {
        const int64_t per_sm = ((B + 1 + 31) / 32 + g->sm_count - 1) / std::max(g->sm_count, 1);
        // (forward only, the spine kernel still wins with four groups: 250 000 nodes x 16 384 policies 7.5 against 8.2 ms)
        if (g->sflow.lanes > 8 || (per_sm > (fwd_only ? 4 : 3) && g->h.n > 8192)) return false;
    }
    return ldb % 16 == 0 && aligned16(lvl) && ldb < big && ldo < big;
}

// Whether a call takes the 32-bit lane-stream kernels: the program exists, the level matrix can be
// fetched in 16-byte pieces, and either the caller asks for them (EMO_F_FLOW_KERNEL) or the batch is
// large (for the graph or for the SMs).  Measured on the five workloads: on the 250 000-node graph with 16 384 policies they are
// the faster pair (25.8 ms against 30.1 ms for both passes) and need 1.6 GB of workspace instead of
// 37.7 GB; on the smaller workloads, where a block holds one or two policy groups and every step is
// latency, the 64-bit staged kernels with their one-step-ahead fetch are faster (2.3 ms against 3.7 ms on
// 10 000 nodes x 4 096 policies).
bool flow_allowed(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t ldo, uint32_t flags)
{
    const int64_t big = (int64_t)1 << 28;
    if (!g->flow.ok32 || !g->dflow.ready) return false;
    if (flags & (EMO_F_NO_STAGING | EMO_F_PAIR_KERNEL | EMO_F_LANE_KERNEL)) return false;
    if (!(flags & EMO_F_FLOW_KERNEL)) {
        // large batches, and on narrow graphs every batch with more than three policy groups per SM (where the spine
        // kernels stop; 75 000 nodes x 16 384 policies: 6.8 ms against 9.0 ms for the 64-bit staged kernels)
        const int64_t per_sm = ((B + 1 + 31) / 32 + g->sm_count - 1) / std::max(g->sm_count, 1);
        if ((int64_t)g->h.n * B < ((int64_t)1 << 31) && !(g->flow.lanes <= 8 && per_sm > 3)) return false;
    }
    return ldb % 16 == 0 && aligned16(lvl) && ldb < big && ldo < big;
}

int launch_validate(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int32_t *status, cudaStream_t st)
{
    if (!status) return EMO_E_INVALID_ARG;
    int64_t total = (int64_t)g->h.rows * B;
    if (total == 0) return EMO_OK;
    int grid = (int)std::min<int64_t>((total + 255) / 256, (int64_t)g->sm_count * 16);
    emo_validate_levels<<<grid, 256, 0, st>>>(lvl, ldb, g->h.rows, B, g->h.L, status);
    EMO_CUDA(cudaGetLastError());
    return EMO_OK;
}

}  // namespace

extern "C" {

const char *emo_strerror(int code)
{
    switch (code) {
        case EMO_OK: return "ok";
        case EMO_E_INVALID_ARG: return "invalid argument";
        case EMO_E_NOT_TOPOLOGICAL: return "nodes are not numbered topologically";
        case EMO_E_RANGE: return "value out of the supported range";
        case EMO_E_OVERFLOW: return "slowest-level makespan does not fit below 2^62 ns";
        case EMO_E_NONFINITE: return "non-finite energy";
        case EMO_E_OOM: return "out of memory or workspace too small";
        case EMO_E_CUDA: return "CUDA runtime error";
        case EMO_E_TIMEOUT: return "bounded device wait ran out";
        case EMO_E_UNSUPPORTED: return "no path for these arguments (see the call's description)";
        default: return "unknown status";
    }
}

int emo_set_pass_events(void *fwd_start, void *fwd_stop, void *bwd_start, void *bwd_stop)
{
    g_pass_events[0] = (cudaEvent_t)fwd_start;
    g_pass_events[1] = (cudaEvent_t)fwd_stop;
    g_pass_events[2] = (cudaEvent_t)bwd_start;
    g_pass_events[3] = (cudaEvent_t)bwd_stop;
    return EMO_OK;
}

int emo_call_path(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t ldo, int need_slack, uint32_t flags)
{
    if (!g || B < 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (g->generic) return 3;
    if (spine_allowed(g, B, lvl, ldb, need_slack ? ldo : 0, need_slack == 0, flags)) {
        FlowPlan fp;
        if (spine_plan(g, B, true, need_slack != 0, fp)) return 4;
    }
    if (flow_allowed(g, B, lvl, ldb, need_slack ? ldo : 0, flags)) {
        FlowPlan fp, sp;
        if (flow_plan(g, B, true, need_slack != 0, fp)) {
            if (need_slack && !(flags & EMO_F_FLOW_KERNEL) && spine_pairs(g) && spine_plan(g, B, true, false, sp) && sp.groups == fp.groups &&
                sp.grid_f == fp.grid_f)
                return 5;
            return 2;
        }
    }
    PassPlan pl;
    const int64_t ld_ws = (int64_t)round_up((size_t)B, 16);
    int rc = make_plan(g, B, true, need_slack != 0, lvl, ldb, ld_ws, ldo, flags, pl);
    if (rc) return rc;
    return pl.staged ? 1 : 0;
}

int emo_measure_int_issue(double *ops_per_s, void *scratch_dev, void *stream)
{
    if (!ops_per_s || !scratch_dev) return EMO_E_INVALID_ARG;
    int dev = 0, sms = 0;
    EMO_CUDA(cudaGetDevice(&dev));
    EMO_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    EMO_CUDA(cudaEventCreate(&e0));
    EMO_CUDA(cudaEventCreate(&e1));
    const int grid = sms * 8, iters = 2048;                    // 64 warps per SM, 8 chains x 4 x iters operations per thread
    unsigned long long *sink = (unsigned long long *)scratch_dev;
    int rc = EMO_OK;
    for (int op = 0; op < 4 && rc == EMO_OK; ++op) {
        float best = 0.f;
        for (int rep = 0; rep < 4; ++rep) {                    // the first repetition warms up
            cudaEventRecord(e0, st);
            if (op == 0) emo_int_chains<0><<<grid, 256, 0, st>>>(sink, iters, 12345u);
            else if (op == 1) emo_int_chains<1><<<grid, 256, 0, st>>>(sink, iters, 12345u);
            else if (op == 2) emo_int_chains<2><<<grid, 256, 0, st>>>(sink, iters, 12345u);
            else emo_int_chains<3><<<grid, 256, 0, st>>>(sink, iters, 12345u);
            cudaEventRecord(e1, st);
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) { rc = EMO_E_CUDA; break; }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            if (rep > 0 && (best == 0.f || ms < best)) best = ms;
        }
        const double warp_ops = (double)grid * 8.0 /* warps per block */ * 8.0 * 4.0 * iters;
        ops_per_s[op] = best > 0.f ? warp_ops / (best * 1e-3) : 0.0;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return rc;
}

int emo_measure_warp_costs(double *cycles, void *scratch_dev, void *stream)
{
    if (!cycles || !scratch_dev) return EMO_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    long long *out = (long long *)scratch_dev;                 // 9 results, then one zero word the kernel reads
    const int iters = 512;
    if (cudaMemsetAsync(scratch_dev, 0, 128, st) != cudaSuccess) return EMO_E_CUDA;
    long long h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int rep = 0; rep < 2; ++rep) {                        // the first repetition warms up
        emo_warp_costs<<<1, 160, 0, st>>>(out, (const unsigned *)(out + 12), iters, 12345u);
        if (cudaMemcpyAsync(h, out, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return EMO_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return EMO_E_CUDA;
    }
    for (int k = 0; k < 8; ++k) cycles[k] = (double)h[k] / iters;
    return EMO_OK;
}

int emo_set_flow_counters(void *dev)
{
    g_flow_prof = (long long *)dev;
    return EMO_OK;
}

int emo_set_wait_limit(int64_t cycles)
{
    if (cycles <= 0) return EMO_E_INVALID_ARG;
    g_wait_cycles = cycles;
    return EMO_OK;
}

int emo_graph_load(int32_t n, const int64_t *row_ptr, const int32_t *col, const int32_t *level_ptr,
                   int32_t n_levels, int32_t L, const int64_t *lat, const double *energy,
                   const int32_t *group_of, uint32_t flags, emo_graph **out)
{
    if (!out) return EMO_E_INVALID_ARG;
    *out = nullptr;
    if (n < 0 || !row_ptr) return EMO_E_INVALID_ARG;
    if (L < 1 || L > 255) return EMO_E_RANGE;
    if (n > 0 && (!lat || !energy)) return EMO_E_INVALID_ARG;
    if (row_ptr[0] != 0) return EMO_E_INVALID_ARG;
    for (int32_t v = 0; v < n; ++v)
        if (row_ptr[v + 1] < row_ptr[v]) return EMO_E_INVALID_ARG;
    const int64_t m = row_ptr[n];
    if (m > 0 && !col) return EMO_E_INVALID_ARG;
    int32_t max_span = 0;
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            if (col[e] < 0 || col[e] >= n) return EMO_E_INVALID_ARG;
            if (col[e] >= v) return EMO_E_NOT_TOPOLOGICAL;
            max_span = std::max(max_span, v - col[e]);
        }
    if (level_ptr) {
        // the whole array is checked before anything is indexed with it
        if (n_levels < 0 || level_ptr[0] != 0 || level_ptr[n_levels] != n) return EMO_E_INVALID_ARG;
        for (int32_t l = 0; l < n_levels; ++l)
            if (level_ptr[l] < 0 || level_ptr[l + 1] > n || level_ptr[l + 1] < level_ptr[l]) return EMO_E_INVALID_ARG;
        try {
            std::vector<int32_t> lev((size_t)std::max(n, 1));
            for (int32_t l = 0; l < n_levels; ++l)
                for (int32_t v = level_ptr[l]; v < level_ptr[l + 1]; ++v) lev[v] = l;
            for (int32_t v = 0; v < n; ++v)
                for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e)
                    if (lev[col[e]] >= lev[v]) return EMO_E_NOT_TOPOLOGICAL;
        } catch (const std::bad_alloc &) {
            return EMO_E_OOM;
        }
    }
    for (int64_t i = 0; i < (int64_t)n * L; ++i) {
        if (lat[i] < 0 || lat[i] >= ((int64_t)1 << 32)) return EMO_E_RANGE;
        if (!std::isfinite(energy[i])) return EMO_E_NONFINITE;
    }
    int32_t rows = n;
    if (group_of) {
        rows = 0;
        for (int32_t v = 0; v < n; ++v) {
            if (group_of[v] < -1) return EMO_E_INVALID_ARG;
            rows = std::max(rows, group_of[v] + 1);
        }
    }

    emo_graph *g = new (std::nothrow) emo_graph();
    if (!g) return EMO_E_OOM;
    try {
        HostGraph &h = g->h;
        h.n = n;
        h.L = L;
        h.rows = rows;
        h.m = m;
        h.max_span = max_span;
        h.row_ptr.assign(row_ptr, row_ptr + n + 1);
        h.col.assign(col, col + m);
        h.group.resize((size_t)n);
        for (int32_t v = 0; v < n; ++v) h.group[v] = group_of ? group_of[v] : v;
        __int128 tw = host_longest(h, [&](int32_t v) {
            int64_t x = 0;
            for (int l = 0; l < L; ++l) x = std::max(x, lat[(size_t)v * L + l]);
            return (__int128)x;
        });
        __int128 tb = host_longest(h, [&](int32_t v) {
            int64_t x = lat[(size_t)v * L];
            for (int l = 1; l < L; ++l) x = std::min(x, lat[(size_t)v * L + l]);
            return (__int128)x;
        });
        if (tw >= ((__int128)1 << 62)) { delete g; return EMO_E_OVERFLOW; }
        h.T_worst = (int64_t)tw;
        h.T_best = (int64_t)tb;
        int lanes = (int)((flags >> 8) & 0xFF);
        int look = (int)((flags >> 16) & 0xFF);
        std::string err;
        // backward first: the forward entries name the row of the backward program that will read
        // the node's earliest start
        // (each direction picks its own number of lanes from its ops and depth unless one is forced)
        // The distance between the group barriers: the longest of 32, 16, 8 steps that costs few slots
        // (a barrier makes every warp of a group wait for the slowest; slots take shared memory from
        // the stages).  Measured on the 250 000-node workload: forward 18 / 26 / 37 slots and
        // 11.2 / 10.5 / 10.0 ms with 8 / 16 / 32, backward 82 slots and 20.4 ms with 8, 24.5 ms with 16.
        auto compile_dir = [&](bool backward, const std::vector<uint32_t> *row_in_other, Program &out) {
            int rc = EMO_E_UNSUPPORTED;
            for (int sync = 32; sync >= 8; sync /= 2) {
                Program cand;
                rc = compile_program(h, lat, energy, backward, lanes, look, sync, row_in_other, cand, err);
                if (rc != EMO_OK && rc != EMO_E_UNSUPPORTED) return rc;
                if (rc == EMO_OK && (cand.slots <= kManySlots || sync == 8)) {
                    out = std::move(cand);
                    return EMO_OK;
                }
            }
            return rc;
        };
        int rc = (flags & EMO_F_GENERIC) ? EMO_E_UNSUPPORTED : compile_dir(true, nullptr, g->bwd);
        if (rc == EMO_OK) rc = compile_dir(false, &g->bwd.pos_of_node, g->fwd);
        if (rc == EMO_E_UNSUPPORTED) {
            // more live exchanged values than the on-chip schedules can hold: the generic kernels take the graph
            g->generic = true;
            g->fwd = Program();
            g->bwd = Program();
            g->host_lat.assign(lat, lat + (size_t)n * L);
            g->host_energy.assign(energy, energy + (size_t)n * L);
            rc = EMO_OK;
        }
        if (rc != EMO_OK) { delete g; return rc; }
        if (!g->generic) {
            // stage length: the longest of 32, 16, 8 steps whose entries the producers can index
            // (32 * kFlowRowRegs per stage); one barrier per stage unless the caller says otherwise (measured on the
            // 250 000-node workload with 16 384 policies: 8 / 16 / 32 steps between barriers gave 24.8 / 22.3 / 21.3 ms for
            // both passes)
            int fk = (int)((flags >> 24) & 0x3F), fs = (int)((flags >> 4) & 0xF) * 8;
            const int flanes = g->fwd.lanes > 0 ? std::max(g->fwd.lanes, g->bwd.lanes) : 1;
            if (fk == 0) fk = flanes * 32 <= 32 * kFlowRowRegs ? 32 : (flanes * 16 <= 32 * kFlowRowRegs ? 16 : 8);
            if (fs == 0) fs = fk;
            if (fs > fk) fs = fk;
            // the spine program: short stages (its sums per stage live in shared memory), 16 steps unless the caller
            // says otherwise; compiled on a thread of its own beside the lane-stream program (they share nothing but
            // their inputs)
            const bool want_spine = !(flags & EMO_F_INTERVALS);
            int rc_s = EMO_OK;
            std::string err_s;
            std::thread spine_thread;
            if (want_spine) {
                const int code = (int)((flags >> 30) & 3u);
                int sk = code == 1 ? 8 : (code == 3 ? 32 : 16);
                while (sk > 8 && flanes * sk > 32 * kFlowRowRegs) sk /= 2;
                spine_thread = std::thread([&, sk]() {
                    try {
                        rc_s = compile_flow(h, lat, energy, lanes, look, sk, sk, g->sflow, err_s, true, fk);
                    } catch (const std::bad_alloc &) {
                        rc_s = EMO_E_OOM;
                    }
                });
            }
            try {
                rc = compile_flow(h, lat, energy, lanes, look, fk, fs, g->flow, err);
            } catch (const std::bad_alloc &) {
                rc = EMO_E_OOM;
            }
            if (spine_thread.joinable()) spine_thread.join();
            if (rc == EMO_E_UNSUPPORTED) {      // the 64-bit programs exist: they serve
                g->flow = Flow();
                rc = EMO_OK;
            }
            if (rc == EMO_OK && rc_s != EMO_OK && rc_s != EMO_E_UNSUPPORTED) rc = rc_s;
            if (rc != EMO_OK) { delete g; return rc; }
            if (!want_spine || rc_s != EMO_OK || !g->flow.ok32 || !g->sflow.spine.ok) g->sflow = Flow();
            else {
                // only the spine's parts are kept
                g->sflow.f = FlowDir();
                g->sflow.b = FlowDir();
            }
        }
        std::vector<int32_t> hop((size_t)std::max(n, 1), 0);
        int32_t depth = 0;
        for (int32_t v = 0; v < n; ++v) {
            int32_t a = 0;
            for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) a = std::max(a, hop[col[e]] + 1);
            hop[v] = a;
            depth = std::max(depth, a + 1);
        }
        h.depth = depth;
    } catch (const std::bad_alloc &) {
        delete g;
        return EMO_E_OOM;
    }
    g->host_only = (flags & EMO_F_HOST_ONLY) != 0;
    if (!g->host_only) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); delete g; return EMO_E_CUDA; }
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { (void)cudaGetLastError(); delete g; return EMO_E_CUDA; }
        g->device = dev;
        g->sm_count = prop.multiProcessorCount;
        g->smem_optin = prop.sharedMemPerBlockOptin;
        int rc = EMO_OK;
        try {
        if (g->generic) {
            // successor CSR from the predecessor CSR, then everything the generic kernels read
            const HostGraph &hh = g->h;
            std::vector<int64_t> sp((size_t)hh.n + 1, 0);
            std::vector<int32_t> sc((size_t)std::max<int64_t>(hh.m, 1));
            for (int64_t e = 0; e < hh.m; ++e) sp[(size_t)hh.col[e] + 1]++;
            for (int32_t v = 0; v < hh.n; ++v) sp[(size_t)v + 1] += sp[(size_t)v];
            std::vector<int64_t> fill(sp.begin(), sp.end() - 1);
            for (int32_t v = 0; v < hh.n; ++v)
                for (int64_t e = hh.row_ptr[v]; e < hh.row_ptr[v + 1]; ++e) sc[(size_t)fill[(size_t)hh.col[e]]++] = v;
            rc = upload(&g->gen_row_ptr, hh.row_ptr.data(), hh.row_ptr.size() * 8);
            if (rc == EMO_OK) rc = upload(&g->gen_col, hh.col.data(), hh.col.size() * 4);
            if (rc == EMO_OK) rc = upload(&g->gen_srow_ptr, sp.data(), sp.size() * 8);
            if (rc == EMO_OK) rc = upload(&g->gen_scol, sc.data(), (size_t)hh.m * 4);
            if (rc == EMO_OK) rc = upload(&g->gen_group, hh.group.data(), hh.group.size() * 4);
            if (rc == EMO_OK) rc = upload(&g->gen_lat, g->host_lat.data(), g->host_lat.size() * 8);
            if (rc == EMO_OK) rc = upload(&g->gen_energy, g->host_energy.data(), g->host_energy.size() * 8);
            g->host_lat = std::vector<int64_t>();
            g->host_energy = std::vector<double>();
        } else {
        rc = upload_program(g->fwd, g->dfwd);
        if (rc == EMO_OK) rc = upload_program(g->bwd, g->dbwd);
        if (rc == EMO_OK && g->fwd.lanes <= 32 - kProducerWarps && g->bwd.lanes <= 32 - kProducerWarps) {
            rc = upload_program_lane(g->fwd, g->lfwd);
            if (rc == EMO_OK) rc = upload_program_lane(g->bwd, g->lbwd);
        }
        if (rc == EMO_OK) rc = upload_flow(g->flow, g->dflow, (flags & EMO_F_INTERVALS) != 0);
        // One barrier per stage needs more exchange slots than one every 16 steps (on the 250 000-node graph 20.9 KB
        // against 13.8 KB per policy group, at 0.3 scale 29.8 KB against 17.9 KB).  Where four groups then no longer fit a
        // block, the grid doubles and the gain turns into a loss (11.7 ms against 6.8 ms at 0.3 scale): take the shorter
        // distance unless the caller chose one.
        if (rc == EMO_OK && g->flow.ok32 && g->dflow.ready && !(flags & 0xF0u) && g->flow.sync > 16) {
            FlowPlan probe;
            const int gmax = std::min((32 - 2) / std::max(g->flow.lanes, 1), 15);
            const bool fits = flow_plan(g, (int64_t)4 * 32 * g->sm_count - 1, true, true, probe) && probe.groups >= std::min(4, gmax);
            if (!fits) {
                const int fk = g->flow.K, look = (int)((flags >> 16) & 0xFF);
                int lanes = (int)((flags >> 8) & 0xFF);
                std::string err;
                free_flow(g->dflow);
                rc = compile_flow(g->h, lat, energy, lanes, look, fk, 16, g->flow, err);
                if (rc == EMO_E_UNSUPPORTED) {
                    g->flow = Flow();
                    rc = EMO_OK;
                }
                if (rc == EMO_OK) rc = upload_flow(g->flow, g->dflow, (flags & EMO_F_INTERVALS) != 0);
            }
        }
        if (rc == EMO_OK) rc = upload_spine(g->sflow, g->dspine);
        }
        } catch (const std::bad_alloc &) {
            rc = EMO_E_OOM;
        }
        if (rc != EMO_OK) { emo_graph_free(g); return rc; }
    }
    *out = g;
    return EMO_OK;
}

int emo_graph_free(emo_graph *g)
{
    if (!g) return EMO_OK;
    if (!g->host_only) {
        free_program(g->dfwd);
        free_program(g->dbwd);
        free_program_lane(g->lfwd);
        free_program_lane(g->lbwd);
        free_flow(g->dflow);
        free_spine(g->dspine);
        void *gen[] = {g->gen_row_ptr, g->gen_col, g->gen_srow_ptr, g->gen_scol, g->gen_group, g->gen_lat, g->gen_energy};
        for (void *q : gen)
            if (q) cudaFree(q);
    }
    delete g;
    return EMO_OK;
}

int emo_graph_info(const emo_graph *g, emo_info *info)
{
    if (!g || !info) return EMO_E_INVALID_ARG;
    info->n = g->h.n;
    info->m = g->h.m;
    info->L = g->h.L;
    info->rows = g->h.rows;
    info->depth = g->h.depth;
    info->max_span = g->h.max_span;
    info->T_worst = g->h.T_worst;
    info->T_best = g->h.T_best;
    info->lanes = g->fwd.lanes;
    info->lanes_bwd = g->bwd.lanes;
    info->sync_fwd = g->fwd.sync;
    info->sync_bwd = g->bwd.sync;
    info->steps_fwd = g->fwd.steps;
    info->slots_fwd = g->fwd.slots;
    info->aux_fwd = g->fwd.aux;
    info->steps_bwd = g->bwd.steps;
    info->slots_bwd = g->bwd.slots;
    info->aux_bwd = g->bwd.aux;
    return EMO_OK;
}

int emo_graph_flow(const emo_graph *g, emo_flow_view *v)
{
    if (!g || !v) return EMO_E_INVALID_ARG;
    const Flow &f = g->flow;
    std::memset(v, 0, sizeof *v);
    v->ok32 = f.ok32 ? 1 : 0;
    v->lanes = f.lanes;
    v->K = f.K;
    v->sync = f.sync;
    v->stages = f.stages;
    v->steps = f.steps;
    v->Lp = f.Lp;
    v->slots_tag_fwd = f.f.slots_tag;
    v->slots_set_fwd = f.f.slots_set;
    v->pool_stride_fwd = f.f.pool_stride;
    v->slots_tag_bwd = f.b.slots_tag;
    v->slots_set_bwd = f.b.slots_set;
    v->pool_stride_bwd = f.b.pool_stride;
    v->pushes = f.pushes;
    v->pruned_fwd = f.f.pruned;
    v->pruned_bwd = f.b.pruned;
    v->hdr = f.hdr.data();
    v->rows = f.rows.data();
    v->node = f.node.data();
    v->step = f.step.data();
    v->tab_fwd = f.tabF.data();
    v->tab_bwd = f.tabB.data();
    v->rec_fwd = f.f.rec.data();
    v->pool_fwd = f.f.pool.data();
    v->rec_bwd = f.b.rec.data();
    v->pool_bwd = f.b.pool.data();
    v->seg_fwd = f.f.seg.data();
    v->seg_bwd = f.b.seg.data();
    v->lbes = f.lbes.data();
    v->push_base = f.push_base.data();
    return EMO_OK;
}

int emo_graph_spine(const emo_graph *g, int64_t out[12])
{
    if (!g || !out) return EMO_E_INVALID_ARG;
    for (int i = 0; i < 12; ++i) out[i] = 0;
    const Flow &f = g->sflow;
    if (!f.ok32 || !f.spine.ok) return EMO_OK;
    int64_t nf = 0, nb = 0;
    for (uint32_t c : f.spine.f.n_ops) nf += c;
    for (uint32_t c : f.spine.b.n_ops) nb += c;
    const int64_t v[12] = {1, f.lanes, f.K, f.stages, f.spine.segments, nf, nb, f.spine.f.slots, f.spine.b.slots,
                           f.spine.max_segs, f.spine.acc_words, f.spine.pushes};
    for (int i = 0; i < 12; ++i) out[i] = v[i];
    return EMO_OK;
}

int emo_graph_spine_view(const emo_graph *g, emo_spine_view *v)
{
    if (!g || !v) return EMO_E_INVALID_ARG;
    std::memset(v, 0, sizeof *v);
    const Flow &f = g->sflow;
    const Spine &sp = f.spine;
    if (!f.ok32 || !sp.ok) return EMO_OK;
    v->ok = 1;
    v->lanes = f.lanes;
    v->K = f.K;
    v->stages = f.stages;
    v->Lp = f.Lp;
    v->max_ops_fwd = sp.f.max_ops;
    v->max_ops_bwd = sp.b.max_ops;
    v->max_pool = sp.max_pool;
    v->acc_words = sp.acc_words;
    v->slots_fwd = sp.f.slots;
    v->slots_bwd = sp.b.slots;
    v->pushes = sp.pushes;
    v->n_ops_fwd = sp.f.n_ops.data();
    v->ops_fwd = sp.f.ops.data();
    v->n_ops_bwd = sp.b.n_ops.data();
    v->ops_bwd = sp.b.ops.data();
    v->mem = sp.mem.data();
    v->pos = sp.posw.data();
    v->rows = f.rows.data();
    v->tab_fwd = f.tabF.data();
    v->tab_bwd = f.tabB.data();
    v->pool = sp.pool.data();
    v->push_base = sp.push_base.data();
    return EMO_OK;
}

int emo_graph_program(const emo_graph *g, int dir, int32_t *lanes, int32_t *steps, int32_t *slots,
                      int32_t *Lp, const uint32_t **entries, const uint32_t **rows, const uint32_t **lat)
{
    if (!g || (dir != 0 && dir != 1)) return EMO_E_INVALID_ARG;
    const Program &p = dir ? g->bwd : g->fwd;
    if (lanes) *lanes = p.lanes;
    if (steps) *steps = p.steps;
    if (slots) *slots = p.slots;
    if (Lp) *Lp = p.Lp;
    if (entries) *entries = p.entries.data();
    if (rows) *rows = p.rows.data();
    if (lat) *lat = p.lat.data();
    return EMO_OK;
}

}  // extern "C"

namespace {

// Spill area behind the head of the workspace: large enough for either layout.
size_t spill_need(const emo_graph *g, int64_t B)
{
    size_t plain = (size_t)g->h.n * round_up((size_t)B, 16) * sizeof(int64_t);
    size_t tiled = 0;
    if (!g->host_only && B > 0) {
        LaunchShape s;
        StagedParams sp;
        // either staged kernel may run (the call's flags decide): room for the wider tiling
        for (int which = 0; which < 2; ++which) {
            const bool ok = which ? staged_shape(g, g->bwd, g->dbwd.rec_bytes, true, B, s, sp) : lane_shape(g, g->bwd, true, B, s, sp);
            if (!ok) continue;
            const size_t tiles = ((size_t)B + sp.ptile - 1) / sp.ptile;
            tiled = std::max(tiled, tiles * spill_rows_of(g, which == 0) * sp.ptile * sizeof(int64_t));
        }
    }
    return round_up(std::max(plain, tiled), 256);
}

}  // namespace

extern "C" {

// The generic kernels: completion times (and, for the backward pass, tails) of every node in the workspace.
static size_t generic_need(const emo_graph *g, int64_t B, bool need_bwd)
{
    const size_t ldw = round_up((size_t)B + 1, 16);
    return (size_t)std::max(g->h.n, 1) * ldw * 8 * (need_bwd ? 2 : 1);
}

static int launch_generic(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, bool need_bwd, int64_t *ES, int64_t *LS,
                          int64_t *slack, int64_t ldo, int64_t *makespan, double *energy, int64_t *slack_sum, int32_t *n_critical,
                          int64_t *T0, double *E0, void *ws, size_t ws_bytes, cudaStream_t st)
{
    const size_t head = kSmallWs + lvl_area(g);
    if (!ws || ws_bytes < head + generic_need(g, B, need_bwd)) return EMO_E_OOM;
    GenericParams p;
    p.n = g->h.n;
    p.L = g->h.L;
    p.row_ptr = g->gen_row_ptr;
    p.col = g->gen_col;
    p.srow_ptr = g->gen_srow_ptr;
    p.scol = g->gen_scol;
    p.group = g->gen_group;
    p.lat = g->gen_lat;
    p.energy = g->gen_energy;
    p.B = B;
    p.want_base = (T0 || E0) ? 1 : 0;
    p.lvl = lvl;
    p.ldb = ldb;
    p.ldw = (int64_t)round_up((size_t)B + 1, 16);
    p.C = (int64_t *)((char *)ws + head);
    p.Q = p.C + (size_t)std::max(g->h.n, 1) * p.ldw;
    p.ES = ES;
    p.LS = LS;
    p.slack = slack;
    p.ldo = ldo;
    p.makespan = makespan;
    p.energy_out = energy;
    p.slack_sum = slack_sum;
    p.n_critical = n_critical;
    p.base_T = T0;
    p.base_E = E0;
    const int64_t cols = B + p.want_base;
    if (cols == 0) return EMO_OK;
    cudaEvent_t ev0 = g_pass_events[0], ev1 = g_pass_events[1], ev2 = g_pass_events[2], ev3 = g_pass_events[3];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    emo_generic_fwd<<<(unsigned)((cols + 127) / 128), 128, 0, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    if (need_bwd && B > 0) {
        if (ev2) EMO_CUDA(cudaEventRecord(ev2, st));
        emo_generic_bwd<<<(unsigned)((B + 127) / 128), 128, 0, st>>>(p);
        EMO_CUDA(cudaGetLastError());
        if (ev3) EMO_CUDA(cudaEventRecord(ev3, st));
    }
    return EMO_OK;
}

int emo_workspace_bytes_for(const emo_graph *g, int64_t B, int need_slack, uint32_t flags, int aligned, size_t *out)
{
    if (!g || !out || B < 0) return EMO_E_INVALID_ARG;
    size_t bytes = kSmallWs + lvl_area(g);
    if (g->generic) {
        bytes += generic_need(g, B, need_slack != 0);
        if (need_slack == 2) bytes += 4 * round_up((size_t)B * 8, 256) + 256;
        *out = bytes;
        return EMO_OK;
    }
    if (need_slack) {
        // what the call with these flags will run: the 32-bit kernels keep a restore list between the
        // passes, the 64-bit kernels the earliest starts of every node
        size_t need = 0;
        FlowPlan fp;
        const uint8_t *fake = aligned ? (const uint8_t *)16 : (const uint8_t *)1;
        if (!g->host_only && B > 0 && flow_allowed(g, B, fake, aligned ? 16 : 1, 0, flags) && flow_plan(g, B, true, true, fp))
            need = fp.restore_bytes;
        else
            need = spill_need(g, B);
        if (!g->host_only && B > 0 && spine_allowed(g, B, fake, aligned ? 16 : 1, 0, false, flags) && spine_plan(g, B, true, true, fp))
            need = std::max(need, fp.restore_bytes);
        bytes += need;
    }
    if (need_slack == 2) bytes += 4 * round_up((size_t)B * 8, 256) + 256;
    *out = bytes;
    return EMO_OK;
}

int emo_workspace_bytes(const emo_graph *g, int64_t B, int need_slack, size_t *out)
{
    return emo_workspace_bytes_for(g, B, need_slack, 0, 1, out);
}

int emo_eval_policies(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t *makespan,
                      double *energy, int64_t *T0, double *E0, void *ws, size_t ws_bytes, int32_t *status,
                      uint32_t flags, void *stream)
{
    if (!g || B < 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (B == 0 && !T0 && !E0) return EMO_OK;
    if (B > 0 && (!lvl || !makespan || !energy || ldb < B)) return EMO_E_INVALID_ARG;
    (void)ws;
    (void)ws_bytes;
    cudaStream_t st = (cudaStream_t)stream;
    if ((flags & EMO_F_VALIDATE) && B > 0) {
        int rc = launch_validate(g, B, lvl, ldb, status, st);
        if (rc) return rc;
    }
    if (B == 0) { lvl = nullptr; ldb = 0; }
    if (g->generic)
        return launch_generic(g, B, lvl, ldb, false, nullptr, nullptr, nullptr, 0, makespan, energy, nullptr, nullptr, T0, E0, ws,
                              ws_bytes, st);
    if (spine_allowed(g, B, lvl, ldb, 0, true, flags)) {
        FlowPlan fp;
        if (spine_plan(g, B, T0 || E0, false, fp))
            return launch_spine_fwd(g, fp, B, lvl, ldb, nullptr, makespan, energy, T0, E0, status, flags, st);
    }
    if (flow_allowed(g, B, lvl, ldb, 0, flags)) {
        FlowPlan fp;
        if (flow_plan(g, B, T0 || E0, false, fp))
            return launch_flow_fwd(g, fp, B, lvl, ldb, nullptr, makespan, energy, T0, E0, status, flags, st);
    }
    PassPlan pl;
    int rc = make_plan(g, B, T0 || E0, false, lvl, ldb, 0, 0, flags, pl);
    if (rc) return rc;
    return launch_pass(g, pl, false, B, lvl, ldb, nullptr, 0, nullptr, nullptr, nullptr, 0, makespan, energy, nullptr,
                       nullptr, T0, E0, status, st);
}

int emo_workspace_bytes_intervals(const emo_graph *g, int64_t B, int32_t I, int with_idle, size_t *out)
{
    if (!g || !out || B < 0 || I < 1) return EMO_E_INVALID_ARG;
    size_t bytes = round_up((size_t)I * 8, 256);
    if (with_idle) bytes += (size_t)std::max(g->h.rows, 1) * (size_t)I * round_up((size_t)B, 16) * 8;
    *out = bytes;
    return EMO_OK;
}

int emo_eval_intervals(const emo_graph *g, int64_t B, const uint8_t *F, int64_t ldb, int32_t I, const int64_t *breaks,
                       const double *p_idle, int64_t *makespan, double *energy, double *energy_idle, void *ws,
                       size_t ws_bytes, int32_t *status, uint32_t flags, void *stream)
{
    (void)flags;
    (void)status;
    if (!g || B < 0 || I < 1 || I > 4096 || !breaks || breaks[0] != 0) return EMO_E_INVALID_ARG;
    for (int32_t i = 1; i < I; ++i)
        if (breaks[i] <= breaks[i - 1]) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (g->generic) return EMO_E_UNSUPPORTED;      // the time-interval form needs a compiled schedule
    if (B == 0) return EMO_OK;
    if (!F || !makespan || !energy || ldb < B) return EMO_E_INVALID_ARG;
    if (energy_idle && !p_idle) return EMO_E_INVALID_ARG;
    size_t need = 0;
    emo_workspace_bytes_intervals(g, B, I, p_idle != nullptr, &need);
    if (!ws || ws_bytes < need) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    int64_t *d_breaks = (int64_t *)ws;
    unsigned long long *busy = p_idle ? (unsigned long long *)((char *)ws + round_up((size_t)I * 8, 256)) : nullptr;
    const int64_t ldw = (int64_t)round_up((size_t)B, 16);
    const int rows = std::max(g->h.rows, 1);
    EMO_CUDA(cudaMemcpyAsync(d_breaks, breaks, (size_t)I * 8, cudaMemcpyHostToDevice, st));
    if (busy) EMO_CUDA(cudaMemsetAsync(busy, 0, (size_t)rows * (size_t)I * (size_t)ldw * 8, st));
    const float inv_mean = (I > 1) ? (float)((double)(I - 1) / (double)breaks[I - 1]) : 0.0f;
    long long delta = (I > 1) ? breaks[1] : 0;
    for (int32_t i = 1; i < I && delta > 0; ++i)
        if (breaks[i] != (int64_t)i * delta) delta = 0;
    cudaEvent_t ev0 = g_pass_events[0], ev1 = g_pass_events[1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    bool done = false;
    if (!(flags & EMO_F_NO_STAGING) && g->dflow.blobFI && delta > 0) {
        // the lane-stream forward kernel with the look-up inside the chain: uniform grids, F's columns in shared memory
        FlowPlan fp;
        const size_t brk_b = round_up((size_t)I * 8, 16), f_per_group = (size_t)rows * (size_t)I * 32;
        if (flow_plan(g, B, false, false, fp, true, brk_b, f_per_group)) {
            FlowParams q = fp.pf;
            q.B = B;
            q.lvl = nullptr;
            q.ldb = 0;
            q.restore = nullptr;
            q.makespan = makespan;
            q.energy = energy;
            q.status = status;
            q.F = F;
            q.ldF = ldb;
            q.I = I;
            q.rowsF = rows;
            q.delta = delta;
            q.inv_mean = inv_mean;
            q.breaks = (const long long *)d_breaks;
            q.busy = busy;
            q.ldw = ldw;
            void (*kern)(FlowParams) = fp.threads <= 512 ? emo_flow_fwd<512, true, false> : (fp.threads <= 768 ? emo_flow_fwd<768, true, false> : emo_flow_fwd<1024, true, false>);
            if (flow_optin(kern, g) != EMO_OK) { (void)cudaGetLastError(); return EMO_E_CUDA; }
            kern<<<fp.grid_f, fp.threads, fp.smem_f, st>>>(q);
            EMO_CUDA(cudaGetLastError());
            done = true;
        }
    }
    if (!done) {
    const Program &p = g->fwd;
    const DevProgram &d = g->dfwd;
    if (p.steps == 0) return EMO_E_UNSUPPORTED;
    LaunchShape s;
    int rc = shape_for(g, p, B, s);
    if (rc) return rc;
    const size_t brk_bytes = round_up((size_t)I * 8, 16);
    const size_t budget = g->smem_optin ? g->smem_optin : 48 * 1024;
    if (d.rec_bytes % 16) return EMO_E_UNSUPPORTED;      // a warp copies a record 16 bytes per thread
    const size_t rec_pad = round_up((size_t)d.rec_bytes, 16) + 16;      // the record and, in the last 16 bytes, the node's group
    const size_t off_rec = round_up(s.smem + brk_bytes, 16);
    const size_t off_F = off_rec + (size_t)(s.threads / 32) * 4 * rec_pad;
    if (off_F > budget) return EMO_E_UNSUPPORTED;
    const int rows_ = std::max(g->h.rows, 1);
    const size_t f_bytes = (size_t)rows_ * (size_t)I * (size_t)s.groups * 32;
    const bool stage_F = off_F + f_bytes <= budget;
    IntervalParams a;
    a.p = PassParams();
    a.p.rec = d.rec;
    a.p.rows = d.groups;
    a.p.rec_bytes = d.rec_bytes;
    a.p.steps = p.steps;
    a.p.lanes = p.lanes;
    a.p.Lp = p.Lp;
    a.p.L = g->h.L;
    a.p.slots = p.slots;
    a.p.sync = p.sync;
    a.p.groups = s.groups;
    a.p.B = B;
    a.p.makespan = makespan;
    a.p.energy = energy;
    a.F = F;
    a.ldb = ldb;
    a.I = I;
    a.breaks = d_breaks;
    a.inv_mean = inv_mean;
    a.delta = delta;
    a.busy = busy;
    a.ldw = ldw;
    a.slot_bytes = (unsigned)s.smem;
    a.off_rec = (unsigned)off_rec;
    a.rec_pad = (unsigned)rec_pad;
    a.off_F = (unsigned)off_F;
    a.stage_F = stage_F ? 1 : 0;
    a.rows = rows_;
    const size_t smem = off_F + (stage_F ? f_bytes : 0);
    void (*kern)(IntervalParams) = delta > 0 ? (stage_F ? emo_pass_intervals<true, true> : emo_pass_intervals<true, false>)
                                             : (stage_F ? emo_pass_intervals<false, true> : emo_pass_intervals<false, false>);
    if (smem > 48 * 1024) EMO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem_optin));
    kern<<<s.grid, s.threads, smem, st>>>(a);
    EMO_CUDA(cudaGetLastError());
    }
    if (p_idle) {
        emo_idle_energy<<<(unsigned)((B + 255) / 256), 256, 0, st>>>(B, rows, I, d_breaks, F, ldb, busy, ldw, p_idle, g->h.L, makespan,
                                                                       energy, energy_idle);
        EMO_CUDA(cudaGetLastError());
    }
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

// Workspace of emo_search_dp: the candidates' levels, their times and energies, and what the evaluation needs.
static void search_layout(const emo_graph *g, int32_t I, int64_t batch, int with_idle, size_t &off_T, size_t &off_E, size_t &off_ws,
                          size_t &total, int64_t &ldb)
{
    ldb = (int64_t)round_up((size_t)batch, 16);
    const size_t f_bytes = round_up((size_t)std::max(g->h.rows, 1) * (size_t)I * (size_t)ldb, 256);
    off_T = f_bytes;
    off_E = off_T + round_up((size_t)batch * 8, 256);
    off_ws = off_E + round_up((size_t)batch * 8, 256);
    size_t iv = 0;
    emo_workspace_bytes_intervals(g, batch, I, with_idle, &iv);
    total = off_ws + iv;
}

int emo_workspace_bytes_search(const emo_graph *g, int32_t I, int64_t max_batch, int with_idle, size_t *out)
{
    if (!g || !out || I < 1 || max_batch < 0) return EMO_E_INVALID_ARG;
    if (max_batch == 0) max_batch = 16384;
    size_t a, b, c, total;
    int64_t ldb;
    search_layout(g, I, max_batch, with_idle, a, b, c, total, ldb);
    *out = total;
    return EMO_OK;
}

int emo_search_dp(const emo_graph *g, int32_t I, const int64_t *breaks, const double *p_idle, int64_t T_max, int64_t bin_ns,
                  int64_t max_batch, uint8_t *F_best, int64_t *T_best, double *E_best, int64_t *n_pred, int32_t *found,
                  void *ws, size_t ws_bytes, void *stream)
{
    if (!g || I < 1 || I > 4096 || !breaks || bin_ns < 1 || max_batch < 0 || !found) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (max_batch == 0) max_batch = 16384;
    const int L = g->h.L, rows = std::max(g->h.rows, 1);
    size_t off_T, off_E, off_ws, total;
    int64_t ldb;
    search_layout(g, I, max_batch, p_idle != nullptr, off_T, off_E, off_ws, total, ldb);
    if (!ws || ws_bytes < total) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *dF = (uint8_t *)ws;
    int64_t *dT = (int64_t *)((char *)ws + off_T);
    double *dE = (double *)((char *)ws + off_E);
    void *iws = (char *)ws + off_ws;
    const size_t iws_bytes = total - off_ws;
    struct State {
        int64_t t;
        double E;
        std::vector<uint8_t> P;
    };
    int64_t calls = 0;
    *found = 0;
    try {
        std::vector<uint8_t> hF((size_t)rows * I * ldb);
        std::vector<int64_t> hT((size_t)max_batch);
        std::vector<double> hE((size_t)max_batch);
        // Pred of a chunk of candidates (policy c = cand[c], the same levels for every device row)
        auto predict = [&](const std::vector<const uint8_t *> &cand, const std::vector<std::pair<int32_t, uint8_t>> &patch) -> int {
            const int64_t nb = (int64_t)cand.size();
            for (int r = 0; r < rows; ++r)
                for (int32_t i = 0; i < I; ++i) {
                    uint8_t *dst = &hF[((size_t)r * I + i) * ldb];
                    for (int64_t c = 0; c < nb; ++c) dst[c] = (patch[c].first == i) ? patch[c].second : cand[c][i];
                }
            if (cudaMemcpyAsync(dF, hF.data(), hF.size(), cudaMemcpyHostToDevice, st) != cudaSuccess) return EMO_E_CUDA;
            int rc = emo_eval_intervals(g, nb, dF, ldb, I, breaks, p_idle, dT, dE, nullptr, iws, iws_bytes, nullptr, 0, stream);
            if (rc) return rc;
            if (cudaMemcpyAsync(hT.data(), dT, (size_t)nb * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return EMO_E_CUDA;
            if (cudaMemcpyAsync(hE.data(), dE, (size_t)nb * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return EMO_E_CUDA;
            if (cudaStreamSynchronize(st) != cudaSuccess) return EMO_E_CUDA;
            calls += nb;
            return EMO_OK;
        };
        // P_0 = default level in all intervals; dp[0][t_0] = (E_0, P_0)   (Alg. 2 lines 1-3)
        std::map<int64_t, State> cur, nxt;
        {
            std::vector<uint8_t> P0((size_t)I, (uint8_t)(L - 1));
            int rc = predict({P0.data()}, {{-1, 0}});
            if (rc) return rc;
            cur[hT[0] / bin_ns] = State{hT[0], hE[0], P0};
        }
        for (int32_t i = 0; i < I; ++i) {
            nxt.clear();
            // candidates in the order of Alg. 2: states by ascending time, levels ascending; evaluated in chunks
            std::vector<const uint8_t *> cand;
            std::vector<std::pair<int32_t, uint8_t>> patch;
            auto flush = [&]() -> int {
                if (cand.empty()) return EMO_OK;
                int rc = predict(cand, patch);
                if (rc) return rc;
                for (size_t c = 0; c < cand.size(); ++c) {
                    if (hT[c] > T_max) continue;
                    const int64_t key = hT[c] / bin_ns;
                    auto it = nxt.find(key);
                    if (it == nxt.end() || hE[c] < it->second.E) {      // strict: the first of equals stays
                        State s2{hT[c], hE[c], std::vector<uint8_t>(cand[c], cand[c] + I)};
                        s2.P[(size_t)i] = patch[c].second;
                        nxt[key] = std::move(s2);
                    }
                }
                cand.clear();
                patch.clear();
                return EMO_OK;
            };
            for (auto &kv : cur)
                for (int f = 0; f < L; ++f) {
                    cand.push_back(kv.second.P.data());
                    patch.push_back({i, (uint8_t)f});
                    if ((int64_t)cand.size() == max_batch) {
                        int rc = flush();
                        if (rc) return rc;
                    }
                }
            int rc = flush();
            if (rc) return rc;
            cur.swap(nxt);      // dp[i] is no longer needed
        }
        // (E*, P*) = the entry of dp[N] of least energy, the earliest time among equals
        const State *best = nullptr;
        for (auto &kv : cur)
            if (!best || kv.second.E < best->E) best = &kv.second;
        if (best) {
            *found = 1;
            if (F_best) std::memcpy(F_best, best->P.data(), (size_t)I);
            if (T_best) *T_best = best->t;
            if (E_best) *E_best = best->E;
        }
    } catch (const std::bad_alloc &) {
        return EMO_E_OOM;
    }
    if (n_pred) *n_pred = calls;
    return EMO_OK;
}

int emo_pack_model(int32_t n_packs, int32_t n_metrics, int32_t m, int32_t L, const double *Bmat, const double *feat,
                   const double *Tb, const double *Eb, double *x, double *T_out, double *E_out, int32_t *status, void *stream)
{
    if (n_packs < 0 || n_metrics < 1 || m < 1 || m > kModelMaxM || L < 1) return EMO_E_INVALID_ARG;
    if (n_packs == 0) return EMO_OK;
    if (!Bmat || !feat || !Tb || !Eb || !x || !T_out || !E_out) return EMO_E_INVALID_ARG;
    const size_t smem = ((size_t)m * m + (size_t)n_metrics * m + 2 * (size_t)m * L) * sizeof(double);
    if (smem > 48 * 1024) return EMO_E_UNSUPPORTED;
    ModelParams p;
    p.n_packs = n_packs;
    p.n = n_metrics;
    p.m = m;
    p.L = L;
    p.B = Bmat;
    p.feat = feat;
    p.Tb = Tb;
    p.Eb = Eb;
    p.x = x;
    p.T_out = T_out;
    p.E_out = E_out;
    p.status = status;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t ev0 = g_pass_events[0], ev1 = g_pass_events[1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    emo_pack_model_kernel<<<(unsigned)((n_packs + 127) / 128), 128, smem, st>>>(p);
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
}

int emo_slack_batch(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t *ES,
                    int64_t *LS, int64_t *slack, int64_t ldo, int64_t *makespan, double *energy,
                    int64_t *slack_sum, int32_t *n_critical, int64_t *T0, double *E0, void *ws, size_t ws_bytes,
                    int32_t *status, uint32_t flags, void *stream)
{
    if (!g || B < 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (B == 0) return emo_eval_policies(g, 0, nullptr, 0, nullptr, nullptr, T0, E0, ws, ws_bytes, status, flags, stream);
    if (!lvl || !makespan || !energy || ldb < B) return EMO_E_INVALID_ARG;
    if ((ES || LS || slack) && ldo < B) return EMO_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (flags & EMO_F_VALIDATE) {
        int rc = launch_validate(g, B, lvl, ldb, status, st);
        if (rc) return rc;
    }
    if (g->generic)
        return launch_generic(g, B, lvl, ldb, true, ES, LS, slack, ldo, makespan, energy, slack_sum, n_critical, T0, E0, ws, ws_bytes,
                              st);
    if (spine_allowed(g, B, lvl, ldb, ldo, false, flags)) {
        FlowPlan fp;
        if (spine_plan(g, B, T0 || E0, true, fp, ES || LS || slack_sum || n_critical)) {
            const size_t head = kSmallWs + lvl_area(g);
            if (!ws || ws_bytes < head + fp.restore_bytes) return EMO_E_OOM;
            uint32_t *restore = (uint32_t *)((char *)ws + head);
            int rc = launch_spine_fwd(g, fp, B, lvl, ldb, restore, makespan, energy, T0, E0, status, flags, st);
            if (rc) return rc;
            return launch_spine_bwd(g, fp, B, lvl, ldb, restore, ES, LS, slack, ldo, makespan, slack_sum, n_critical, status, flags, st);
        }
    }
    if (flow_allowed(g, B, lvl, ldb, ldo, flags)) {
        FlowPlan fp;
        if (flow_plan(g, B, T0 || E0, true, fp)) {
            const size_t head = kSmallWs + lvl_area(g);
            if (!ws || ws_bytes < head + fp.restore_bytes) return EMO_E_OOM;
            uint32_t *restore = (uint32_t *)((char *)ws + head);
            // The forward spine kernel is the faster forward pass even with four groups per block (7.5 against 8.2 ms on
            // the 250 000-node graph); where its program shares the schedule of the lane-stream program it writes the
            // restore list in that program's numbering and the lane-stream backward kernel follows.
            FlowPlan sp;
            int rc;
            if (!(flags & EMO_F_FLOW_KERNEL) && spine_pairs(g) && spine_plan(g, B, T0 || E0, false, sp) && sp.groups == fp.groups &&
                sp.grid_f == fp.grid_f) {
                sp.pf.pushes = fp.pf.pushes;
                sp.pf.restore_rows = fp.pf.restore_rows;
                rc = launch_spine_fwd(g, sp, B, lvl, ldb, restore, makespan, energy, T0, E0, status, flags, st, true);
            } else
                rc = launch_flow_fwd(g, fp, B, lvl, ldb, restore, makespan, energy, T0, E0, status, flags, st);
            if (rc) return rc;
            return launch_flow_bwd(g, fp, B, lvl, ldb, restore, ES, LS, slack, ldo, makespan, slack_sum, n_critical, status,
                                   flags, st);
        }
    }
    const int64_t ld_ws = (int64_t)round_up((size_t)B, 16);
    PassPlan pl;
    int rc = make_plan(g, B, T0 || E0, true, lvl, ldb, ES ? ldo : ld_ws, ldo, flags, pl);
    if (rc) return rc;
    int64_t *area = (int64_t *)((char *)ws + kSmallWs + lvl_area(g));
    int64_t *spill = nullptr, *es = ES;
    int64_t ldes = ldo;
    if (pl.staged) {
        if (!ws || ws_bytes < kSmallWs + lvl_area(g) + pl.spill_bytes) return EMO_E_OOM;
        spill = area;
    } else if (!es) {
        if (!ws || ws_bytes < kSmallWs + lvl_area(g) + (size_t)g->h.n * ld_ws * sizeof(int64_t)) return EMO_E_OOM;
        es = area;
        ldes = ld_ws;
    }
    rc = launch_pass(g, pl, false, B, lvl, ldb, es, ldes, spill, nullptr, nullptr, 0, makespan, energy, nullptr,
                     nullptr, T0, E0, status, st);
    if (rc) return rc;
    return launch_pass(g, pl, true, B, lvl, ldb, es, ldes, spill, LS, slack, ldo, makespan, energy, slack_sum,
                       n_critical, nullptr, nullptr, status, st);
}

int emo_slack(const emo_graph *g, const uint8_t *lvl_one, int64_t *ES, int64_t *LS, int64_t *slack,
              int64_t *makespan, double *energy, void *ws, size_t ws_bytes, int32_t *status, void *stream)
{
    if (!g || !makespan || !lvl_one) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    size_t need = 0;
    emo_workspace_bytes(g, 1, 1, &need);
    if (!ws || ws_bytes < need) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    // re-pitch the level vector to [rows][16] so that the staged kernels can be used; the
    // per-node outputs are written at pitch 1 directly
    uint8_t *lv = (uint8_t *)ws + kSmallWs;
    const size_t rows = (size_t)std::max(g->h.rows, 1);
    EMO_CUDA(cudaMemcpy2DAsync(lv, 16, lvl_one, 1, 1, rows, cudaMemcpyDeviceToDevice, st));
    double *e = energy ? energy : (double *)((char *)ws + 1024);
    return emo_slack_batch(g, 1, lv, 16, ES, LS, slack, 1, makespan, e, nullptr, nullptr, nullptr, nullptr, ws, ws_bytes,
                           status, 0, stream);
}

int emo_baseline(const emo_graph *g, int64_t *T0, double *E0, void *ws, size_t ws_bytes, int32_t *status,
                 void *stream)
{
    if (!g || !T0 || !E0) return EMO_E_INVALID_ARG;
    return emo_eval_policies(g, 0, nullptr, 0, nullptr, nullptr, T0, E0, ws, ws_bytes, status, 0, stream);
}

int64_t emo_target_from_delta(int64_t T0, int64_t delta_ppm)
{
    return emo_budget(T0, delta_ppm);
}

int emo_select(int64_t B, const int64_t *makespan, const double *energy, int64_t target,
               const int64_t *target_dev, int64_t delta_ppm, int64_t *out_index, int64_t *out_T,
               double *out_E, void *ws, size_t ws_bytes, void *stream)
{
    if (B < 0 || !out_index) return EMO_E_INVALID_ARG;
    if (B > 0 && (!makespan || !energy)) return EMO_E_INVALID_ARG;
    if (!ws || ws_bytes < kSmallWs) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((B + 1023) / 1024, kSelectMaxBlocks));
    SelectPartial *part = (SelectPartial *)ws;
    emo_select_stage1<<<blocks, 256, 0, st>>>(B, makespan, energy, target, target_dev, delta_ppm, part);
    EMO_CUDA(cudaGetLastError());
    emo_select_stage2<<<1, 256, 0, st>>>(blocks, part, makespan, out_index, out_T, out_E);
    EMO_CUDA(cudaGetLastError());
    return EMO_OK;
}

// ---- selection without any allocation --------------------------------------------------------
// Scratch for emo_select_static: the stage-1 candidates (one per block) live in this file-scope
// device array instead of a caller workspace.  Every GPU that loads the library holds these 16 KiB
// until the process exits.  In host code the array's name is only a stand-in; the device address
// comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char emo_select_static_scratch[kSelectMaxBlocks * sizeof(SelectPartial)];
static void *g_select_static_ptr[64] = {nullptr};

int emo_select_static(int64_t B, const int64_t *makespan, const double *energy, int64_t target,
                      const int64_t *target_dev, int64_t delta_ppm, int64_t *out_index, int64_t *out_T,
                      double *out_E, void *stream)
{
    if (B < 0 || !out_index) return EMO_E_INVALID_ARG;
    if (B > EMO_SELECT_STATIC_MAX_B) return EMO_E_RANGE;
    if (B > 0 && (!makespan || !energy)) return EMO_E_INVALID_ARG;
    int dev = 0;
    EMO_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return EMO_E_UNSUPPORTED;
    if (!g_select_static_ptr[dev]) {
        // first call on this device (it is the current one): resolve the array's device address
        void *ptr = nullptr;
        EMO_CUDA(cudaGetSymbolAddress(&ptr, emo_select_static_scratch));
        if (!ptr) return EMO_E_CUDA;
        g_select_static_ptr[dev] = ptr;
    }
    SelectPartial *part = (SelectPartial *)g_select_static_ptr[dev];
    cudaStream_t st = (cudaStream_t)stream;
    int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((B + 1023) / 1024, kSelectMaxBlocks));
    // stage 1 overwrites the first `blocks` candidates and stage 2 reads exactly those, so nothing
    // left behind by an earlier call is ever read and nothing needs clearing
    emo_select_stage1<<<blocks, 256, 0, st>>>(B, makespan, energy, target, target_dev, delta_ppm, part);
    EMO_CUDA(cudaGetLastError());
    emo_select_stage2<<<1, 256, 0, st>>>(blocks, part, makespan, out_index, out_T, out_E);
    EMO_CUDA(cudaGetLastError());
    return EMO_OK;
}

int emo_transpose_policies(int64_t B, int64_t rows, const uint8_t *src, int64_t lds, uint8_t *dst,
                           int64_t ldb, void *stream)
{
    if (B < 0 || rows < 0) return EMO_E_INVALID_ARG;
    if (B == 0 || rows == 0) return EMO_OK;
    if (!src || !dst || lds < rows || ldb < B) return EMO_E_INVALID_ARG;
    dim3 grid((unsigned)((rows + 31) / 32), (unsigned)std::min<int64_t>((B + 31) / 32, 65535));
    emo_transpose_u8<<<grid, dim3(32, 8), 0, (cudaStream_t)stream>>>(B, rows, src, lds, dst, ldb);
    EMO_CUDA(cudaGetLastError());
    return EMO_OK;
}

namespace {
int repack(bool pack, int bits, int64_t rows, int64_t B, uint8_t *packed, int64_t ldp, uint8_t *bytes, int64_t ldb, cudaStream_t st)
{
    if (bits < 1 || bits > 8 || rows < 0 || B < 0) return EMO_E_INVALID_ARG;
    if (rows == 0 || B == 0) return EMO_OK;
    const int64_t groups = (B + 7) / 8;
    if (!packed || !bytes || ldp < groups * bits || ldb < groups * 8 || ldb % 8 != 0 || ((uintptr_t)bytes % 8) != 0) return EMO_E_INVALID_ARG;
    const int64_t total = rows * groups;
    const int grid = (int)std::min<int64_t>((total + 255) / 256, 148 * 32);
    if (pack) emo_repack_levels<true><<<grid, 256, 0, st>>>(bits, rows, groups, packed, ldp, bytes, ldb);
    else emo_repack_levels<false><<<grid, 256, 0, st>>>(bits, rows, groups, packed, ldp, bytes, ldb);
    EMO_CUDA(cudaGetLastError());
    return EMO_OK;
}
}  // namespace

int emo_pack_levels(int bits, int64_t rows, int64_t B, const uint8_t *lvl, int64_t ldb, uint8_t *packed, int64_t ldp, void *stream)
{
    return repack(true, bits, rows, B, packed, ldp, const_cast<uint8_t *>(lvl), ldb, (cudaStream_t)stream);
}

int emo_unpack_levels(int bits, int64_t rows, int64_t B, const uint8_t *packed, int64_t ldp, uint8_t *lvl, int64_t ldb, void *stream)
{
    return repack(false, bits, rows, B, const_cast<uint8_t *>(packed), ldp, lvl, ldb, (cudaStream_t)stream);
}

// The passes, the selection and the copies of the per-policy results to the host, once the levels are on the device:
// packed in dev_packed (bits < 8: spread to dev_lvl first) or as bytes in dev_lvl (bits = 8).
static int host_batch_tail(const emo_graph *g, int64_t B, int bits, const uint8_t *dev_packed, int64_t ld_packed, uint8_t *dev_lvl,
                           int64_t ldb, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm, int64_t *makespan_host,
                           double *energy_host, int64_t *slack_sum_host, int32_t *n_critical_host, int64_t *sel_host, void *ws,
                           size_t need, uint32_t flags, cudaStream_t st)
{
    size_t per_policy = round_up((size_t)B * 8, 256);
    char *tail = (char *)ws + need;
    int64_t *d_T = (int64_t *)tail;
    double *d_E = (double *)(tail + per_policy);
    int64_t *d_ss = (int64_t *)(tail + 2 * per_policy);
    int32_t *d_nc = (int32_t *)(tail + 3 * per_policy);
    int64_t *d_sel = (int64_t *)(tail + 4 * per_policy);      // {index, T, E bits, T0, E0 bits}
    int32_t *d_status = (int32_t *)(d_sel + 8);
    EMO_CUDA(cudaMemsetAsync(d_sel, 0, 128, st));
    if (bits < 8) {
        int rcu = emo_unpack_levels(bits, g->h.rows, B, dev_packed, ld_packed, dev_lvl, ldb, (void *)st);
        if (rcu) return rcu;
    }
    int rc = emo_slack_batch(g, B, dev_lvl, ldb, nullptr, nullptr, slack_dev, ldo, d_T, d_E,
                             slack_sum_host ? d_ss : nullptr, n_critical_host ? d_nc : nullptr, d_sel + 3,
                             (double *)(d_sel + 4), ws, need, d_status, flags, st);
    if (rc) return rc;
    rc = emo_select(B, d_T, d_E, 0, d_sel + 3, delta_ppm, d_sel, d_sel + 1, (double *)(d_sel + 2), ws, need, st);
    if (rc) return rc;
    EMO_CUDA(cudaMemcpyAsync(makespan_host, d_T, (size_t)B * 8, cudaMemcpyDeviceToHost, st));
    EMO_CUDA(cudaMemcpyAsync(energy_host, d_E, (size_t)B * 8, cudaMemcpyDeviceToHost, st));
    if (slack_sum_host) EMO_CUDA(cudaMemcpyAsync(slack_sum_host, d_ss, (size_t)B * 8, cudaMemcpyDeviceToHost, st));
    if (n_critical_host) EMO_CUDA(cudaMemcpyAsync(n_critical_host, d_nc, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    int64_t tmp[10];
    EMO_CUDA(cudaMemcpyAsync(tmp, d_sel, sizeof(tmp), cudaMemcpyDeviceToHost, st));
    EMO_CUDA(cudaStreamSynchronize(st));
    sel_host[0] = tmp[0];
    sel_host[1] = tmp[1];
    sel_host[2] = tmp[2];
    sel_host[3] = tmp[3];
    int32_t stc;
    std::memcpy(&stc, &tmp[8], sizeof stc);
    return stc < 0 ? stc : EMO_OK;
}

int emo_slack_batch_host_packed(const emo_graph *g, int64_t B, int bits, const uint8_t *lvl_host, int64_t ld_host,
                                uint8_t *dev_packed, uint8_t *dev_lvl, int64_t ldb, int64_t *slack_dev, int64_t ldo,
                                int64_t delta_ppm, int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                                int32_t *n_critical_host, int64_t *sel_host, void *ws, size_t ws_bytes, uint32_t flags,
                                void *stream)
{
    if (!g || B <= 0 || !lvl_host || !dev_lvl || !makespan_host || !energy_host || !sel_host || ldb < B)
        return EMO_E_INVALID_ARG;
    if (bits < 1 || bits > 8 || (bits < 8 && !dev_packed)) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    size_t need = 0, total = 0;
    const int aligned = (ldb % 16 == 0 && aligned16(dev_lvl)) ? 1 : 0;
    emo_workspace_bytes_for(g, B, 1, flags, aligned, &need);
    emo_workspace_bytes_for(g, B, 2, flags, aligned, &total);
    // per-policy result arrays live behind the slack workspace
    if (!ws || ws_bytes < total) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    if (bits == 8) {
        if (ld_host != ldb) return EMO_E_INVALID_ARG;
        EMO_CUDA(cudaMemcpyAsync(dev_lvl, lvl_host, (size_t)g->h.rows * (size_t)ldb, cudaMemcpyHostToDevice, st));
    } else {
        // the levels cross the bus packed and are spread to bytes on the device
        EMO_CUDA(cudaMemcpyAsync(dev_packed, lvl_host, (size_t)g->h.rows * (size_t)ld_host, cudaMemcpyHostToDevice, st));
    }
    return host_batch_tail(g, B, bits, dev_packed, ld_host, dev_lvl, ldb, slack_dev, ldo, delta_ppm, makespan_host, energy_host,
                           slack_sum_host, n_critical_host, sel_host, ws, need, flags, st);
}

int emo_levels_prefetch(const emo_graph *g, const uint8_t *lvl_host, int64_t ld_host, uint8_t *dev_packed, void *copy_stream,
                        void *ready)
{
    if (!g || !lvl_host || !dev_packed || !ready || ld_host <= 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    cudaStream_t cs = (cudaStream_t)copy_stream;
    EMO_CUDA(cudaMemcpyAsync(dev_packed, lvl_host, (size_t)g->h.rows * (size_t)ld_host, cudaMemcpyHostToDevice, cs));
    EMO_CUDA(cudaEventRecord((cudaEvent_t)ready, cs));
    return EMO_OK;
}

int emo_slack_batch_prefetched(const emo_graph *g, int64_t B, int bits, const uint8_t *dev_packed, int64_t ld_packed, void *ready,
                               uint8_t *dev_lvl, int64_t ldb, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm,
                               int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                               int32_t *n_critical_host, int64_t *sel_host, void *ws, size_t ws_bytes, uint32_t flags,
                               void *stream)
{
    if (!g || B <= 0 || !dev_packed || !dev_lvl || !makespan_host || !energy_host || !sel_host || ldb < B)
        return EMO_E_INVALID_ARG;
    if (bits < 1 || bits > 7) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    size_t need = 0, total = 0;
    const int aligned = (ldb % 16 == 0 && aligned16(dev_lvl)) ? 1 : 0;
    emo_workspace_bytes_for(g, B, 1, flags, aligned, &need);
    emo_workspace_bytes_for(g, B, 2, flags, aligned, &total);
    if (!ws || ws_bytes < total) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    if (ready) EMO_CUDA(cudaStreamWaitEvent(st, (cudaEvent_t)ready, 0));
    return host_batch_tail(g, B, bits, dev_packed, ld_packed, dev_lvl, ldb, slack_dev, ldo, delta_ppm, makespan_host, energy_host,
                           slack_sum_host, n_critical_host, sel_host, ws, need, flags, st);
}

int emo_slack_batch_host(const emo_graph *g, int64_t B, const uint8_t *lvl_host, int64_t ldb,
                         uint8_t *dev_lvl, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm,
                         int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                         int32_t *n_critical_host, int64_t *sel_host, void *ws, size_t ws_bytes,
                         uint32_t flags, void *stream)
{
    return emo_slack_batch_host_packed(g, B, 8, lvl_host, ldb, nullptr, dev_lvl, ldb, slack_dev, ldo, delta_ppm, makespan_host,
                                       energy_host, slack_sum_host, n_critical_host, sel_host, ws, ws_bytes, flags, stream);
}

}  // extern "C"
