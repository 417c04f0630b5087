// Pass kernel with the schedule lanes inside one thread (sm_100a).
//
// The step program gives every step W independent entries (one per schedule lane).  Here one thread
// carries ONE policy through ALL W lanes: the W running values live in registers, an exchange slot
// is a private 8-byte word of shared memory, and a value passes from one lane to another by a plain
// store and a later load of the same thread.  Nothing is synchronised between warps: no slot
// barriers, no group barriers, no phase parities - the program order of the thread is the order of
// the schedule.  The parallelism the W lanes offer is used as instruction-level parallelism: a step
// is written as phases over all W lanes (start values, slot operands, stores and additions, slot
// writes), the W entries of a phase are independent of each other, and everything a step reads from
// the stage is requested one step ahead.
//
// The program comes in a layout of its own (built at load time from the same step program):
//   entry  [Q][4 words]  word 0 = row of the per-node store (forward: row of the earliest-start
//                        spill; backward: node id) or kNone; word 1 = out slot (bits 0..7, 255 =
//                        none) | number of slot operands (bits 8..10) | terminal (bit 11) |
//                        operand slots 0 and 1 (bits 16..31); word 2 = mask applied to the lane's
//                        running value (0 = start from 0, ~0 = continue from the lane's last
//                        node); word 3 = operand slots 2..5
//   node   [Q]           node id (forward, for the caller's ES array)
//   table  [Q][Lp]       forward: {duration, 0, energy} in 16 bytes per level; backward: duration
//                        in 4 bytes.  Rows of nodes that ignore the policy hold one value Lp times.
// Q = padded steps x W; the padding steps are idle entries, so every stage holds whole steps.
//
// A block is up to kIlpMaxWarps consumer warps (32 policies each) and one producer warp that fills
// the ring of stages (emo_produce).  Used for programs of at most kIlpMaxLanes lanes; wider programs
// run on emo_pass_pair.  Included only by emo_lib.cu.
#pragma once
#include "emo_pass_staged.cuh"

constexpr int kIlpMaxLanes = 8;
constexpr int kIlpMaxWarps = 8;
constexpr int kIlpStepPad = 16;                 // programs are padded to a multiple of this many steps
constexpr unsigned kIlpNoSlot = 255u;
constexpr unsigned kIlpNpShift = 8, kIlpTerminal = 0x800u, kIlpOp0Shift = 16;

// offsets of the areas of one stage (records first, then what emo_produce addresses)
struct IlpStage {
    unsigned off_node, off_tab;                 // entries start at 0
};

struct IlpParams {
    StagedParams sp;
    IlpStage st;
    unsigned tab_entry;                         // bytes of one entry's table row
};

__device__ __forceinline__ long long emo_lds_s64(unsigned a)
{
    long long v;
    asm volatile("ld.shared.s64 %0, [%1];" : "=l"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void emo_sts_s64(unsigned a, long long v)
{
    asm volatile("st.shared.s64 [%0], %1;" ::"r"(a), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned emo_lds_u8(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// st.global / st.shared under a predicate (no branch): the store happens when row != kNone and ok != 0
__device__ __forceinline__ void emo_stg_row_if(long long *base, unsigned row, unsigned pitch_bytes, long long v, unsigned ok)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .u64 a;\n\t"
        "setp.ne.u32 q, %4, 0;\n\t"
        "setp.ne.and.u32 p, %1, 0xFFFFFFFF, q;\n\t"
        "mad.wide.u32 a, %1, %2, %0;\n\t"
        "@p st.global.s64 [a], %3;\n\t}"
        ::"l"(base), "r"(row), "r"(pitch_bytes), "l"(v), "r"(ok)
        : "memory");
}
__device__ __forceinline__ void emo_sts_s64_if(unsigned a, long long v, unsigned id, unsigned none)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, %3;\n\t@p st.shared.s64 [%0], %1;\n\t}" ::"r"(a), "l"(v), "r"(id), "r"(none)
                 : "memory");
}

// What one lane of one step reads from the stage.
struct EmoLaneIn {
    uint4 e;            // entry
    unsigned node;      // node id (only when the caller's ES array is written)
    unsigned lv;        // level byte of this thread's policy
    unsigned d;         // duration at that level
    double g;           // forward: energy at that level
    long long es;       // backward: earliest start of the node
};

template <bool BWD, bool EXTRA, int W>
__global__ void __launch_bounds__(32 * (kIlpMaxWarps + 1), 1) emo_pass_ilp(IlpParams ip)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const StagedParams &sp = ip.sp;
    const PassParams &p = sp.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int n_cons = p.groups;                         // consumer warps; the warp after them produces
    const bool producer = warp >= n_cons;
    const int steps = p.steps, nstages = sp.stages, sc = sp.sc;     // steps: padded, a multiple of sc
    const int ptile = sp.ptile;                          // 32 * n_cons
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = warp * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !producer && b < p.B;
    // column of the virtual all-max policy inside this block's tile (forward only), or -1
    const int base_col = (!BWD && p.want_base && p.B >= b0 && p.B < b0 + ptile) ? (int)(p.B - b0) : -1;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + sp.off_bar;           // full[k] at bar0 + 8k, empty[k] after them
    volatile int *abort_flag = reinterpret_cast<volatile int *>(emo_smem + sp.off_bar + 16 * kMaxStages);
    const unsigned stage0 = smem0 + sp.off_stage0;
    const unsigned stage_bytes = sp.stage_bytes;

    if (threadIdx.x == 0) {
        for (int k = 0; k < nstages; ++k) {
            emo_mbar_init(bar0 + 8 * k, 1 + 32);                       // expect-tx arrival + the producer lanes' cp.async arrivals
            emo_mbar_init(bar0 + 8 * (kMaxStages + k), n_cons);
        }
        abort_flag[0] = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    if (producer) {
        emo_produce(sp, stage0, bar0, abort_flag, lane, 0);
        return;
    }

    // ------------------------------------------------------------------------------- consumers
    const int n_chunks = steps / sc;
    long long h[W];
    double ea[W];
#pragma unroll
    for (int k = 0; k < W; ++k) {
        h[k] = 0;
        ea[k] = 0.0;
    }
    long long acc = 0;        // forward: running makespan; backward: slack sum
    int nc = 0;               // backward: critical nodes
    // private exchange slots: slot i of this thread at slot_a + i * slot_stride
    const unsigned slot_a = smem0 + (unsigned)col * 8u, slot_stride = (unsigned)ptile * 8u;
    const long long T0 = (BWD && act) ? p.makespan[b] : 0;
    const unsigned tab_entry = ip.tab_entry, lmask = (unsigned)p.Lp - 1u;
    const unsigned ldes8 = (unsigned)p.ldes * 8u, ldo8 = (unsigned)p.ldo * 8u;     // pitches below 2^28 elements
    long long *const es_lane = (!BWD && EXTRA && p.ES && act) ? reinterpret_cast<long long *>(p.ES) + b : nullptr;
    long long *const spill_lane = (!BWD && p.spill && act)
        ? reinterpret_cast<long long *>(p.spill) + (size_t)(b / p.spill_ptile) * p.spill_rows * p.spill_ptile + (b % p.spill_ptile)
        : nullptr;
    const unsigned spill8 = (unsigned)p.spill_ptile * 8u;
    long long *const ls_lane = (BWD && EXTRA && p.LS && act) ? reinterpret_cast<long long *>(p.LS) + b : nullptr;
    long long *const sl_lane = (BWD && p.slack && act) ? reinterpret_cast<long long *>(p.slack) + b : nullptr;
    const bool want_sums = BWD && EXTRA && sp.want_sums != 0 && act;
    const bool want_node = es_lane != nullptr;
    const unsigned spill_ok = spill_lane != nullptr, slack_ok = sl_lane != nullptr;

    // addresses inside the current stage; every step moves them on by one step's worth
    unsigned ent_a = 0, node_a = 0, tab_a = 0, lvl_a = 0, es_a = 0;
    const unsigned d_tab = (unsigned)W * tab_entry, d_lvl = (unsigned)W * ptile, d_es = d_lvl * 8u;

    // entry, level byte (and the backward pass's earliest start) of every lane of one step
    auto load_head = [&](EmoLaneIn (&x)[W]) {
#pragma unroll
        for (int k = 0; k < W; ++k) {
            x[k].e = emo_lds128(ent_a + 16u * k);
            if (EXTRA && !BWD && want_node) x[k].node = emo_lds_u32(node_a + 4u * k);
            x[k].lv = emo_lds_u8(lvl_a + (unsigned)k * ptile);
            if (BWD) x[k].es = emo_lds_s64(es_a + (unsigned)k * ptile * 8u);
        }
    };
    // the table look-ups, which need the level byte
    auto load_tables = [&](EmoLaneIn (&x)[W]) {
#pragma unroll
        for (int k = 0; k < W; ++k) {
            const unsigned l = x[k].lv & lmask;
            if (!BWD) {
                const uint4 t = emo_lds128(tab_a + (unsigned)k * tab_entry + l * 16u);
                x[k].d = t.x;
                x[k].g = __hiloint2double((int)t.w, (int)t.z);
            } else {
                x[k].d = emo_lds_u32(tab_a + (unsigned)k * tab_entry + l * 4u);
            }
        }
    };
    // One step, written as phases over the W lanes.  All slot reads of a step come before its slot
    // writes; operands always stem from earlier steps.
    auto step = [&](EmoLaneIn (&cur)[W], EmoLaneIn (&nxt)[W]) {
        ent_a += 16u * W;
        node_a += 4u * W;
        tab_a += d_tab;
        lvl_a += d_lvl;
        es_a += d_es;
        load_head(nxt);      // (after a stage's last step: bytes of the next stage or the pad, never used)
        long long v[W];
        // start value: the lane's running value (forward: completion time of the lane's last node;
        // backward: longest tail behind it) or 0
#pragma unroll
        for (int k = 0; k < W; ++k) v[k] = h[k] & (long long)(int)cur[k].e.z;
        // slot operands (most steps have none: one test per step)
        unsigned any_w1 = 0;
#pragma unroll
        for (int k = 0; k < W; ++k) any_w1 |= cur[k].e.y;
        if (any_w1 & (7u << kIlpNpShift))
#pragma unroll
        for (int k = 0; k < W; ++k) {
            const unsigned w1 = cur[k].e.y;
            if (w1 & (7u << kIlpNpShift)) {
                const unsigned np = (w1 >> kIlpNpShift) & 7u;
                unsigned ops = w1 >> kIlpOp0Shift;
                for (unsigned i = 0; i < np; ++i) {
                    if (i == 2) ops = cur[k].e.w;
                    v[k] = emo_max64(v[k], emo_lds_s64(slot_a + (ops & 255u) * slot_stride));
                    ops >>= 8;
                }
            }
        }
        load_tables(nxt);
        // here v is the node's start (forward: ES_v; backward: the longest tail behind v)
#pragma unroll
        for (int k = 0; k < W; ++k) {
            const unsigned row = cur[k].e.x;
            if (!BWD) {
                emo_stg_row_if(spill_lane, row, spill8, v[k], spill_ok);
                if (EXTRA && es_lane && row != emo::kNone) *emo_row_ptr(es_lane, cur[k].node, ldes8) = v[k];
                ea[k] += cur[k].g;
                v[k] = emo_add_dur(v[k], cur[k].d);
            } else {
                v[k] = emo_add_dur(v[k], cur[k].d);
                const long long ls = T0 - v[k], sl = ls - cur[k].es;
                emo_stg_row_if(sl_lane, row, ldo8, sl, slack_ok);
                if (EXTRA && row != emo::kNone) {
                    if (ls_lane) *emo_row_ptr(ls_lane, row, ldo8) = ls;
                    if (want_sums) {
                        acc += sl;
                        nc += (sl == 0);
                    }
                }
            }
        }
        // slot writes
#pragma unroll
        for (int k = 0; k < W; ++k) {
            const unsigned out = cur[k].e.y & 255u;
            emo_sts_s64_if(slot_a + out * slot_stride, v[k], out, kIlpNoSlot);
        }
        if (!BWD) {
            // makespan: terminal nodes are rare, one test per step
            if (any_w1 & kIlpTerminal) {
#pragma unroll
                for (int k = 0; k < W; ++k)
                    if (cur[k].e.y & kIlpTerminal) acc = emo_max64(acc, v[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < W; ++k) h[k] = v[k];
    };

    bool failed = false;
    for (int c = 0; c < n_chunks; ++c) {
        const int s = c % nstages;
        if (!emo_mbar_wait(bar0 + 8 * s, (c / nstages) & 1) || abort_flag[0]) {
            if (lane == 0) {
                abort_flag[0] = 1;
                if (p.status) atomicMin(p.status, -8);
            }
            failed = true;
            break;
        }
        const unsigned sta = stage0 + (unsigned)s * stage_bytes;
        if (base_col >= 0 && (base_col >> 5) == warp) {
            // the virtual all-max column: overwrite its byte in every level row of this stage (only
            // this warp reads that column)
            const unsigned char top = (unsigned char)(p.L - 1);
            for (int i = lane; i < sc * W; i += 32)
                emo_smem[sp.off_stage0 + (size_t)s * stage_bytes + sp.off_lvl + (size_t)i * ptile + (size_t)base_col] = top;
            __syncwarp();
        }
        ent_a = sta;
        node_a = sta + ip.st.off_node;
        tab_a = sta + ip.st.off_tab;
        lvl_a = sta + sp.off_lvl + (unsigned)col;
        es_a = sta + sp.off_es + (unsigned)col * 8u;
        EmoLaneIn x0[W], x1[W];
        load_head(x0);
        load_tables(x0);
        for (int j = 0; j < sc; j += 2) {       // sc is even
            step(x0, x1);
            step(x1, x0);
        }
        __syncwarp();
        if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kMaxStages + s));
    }
    if (failed) return;

    if (!BWD) {
        // lanes in a fixed order: run-to-run identical energy
        double e = 0.0;
#pragma unroll
        for (int k = 0; k < W; ++k) e += ea[k];
        if (act) {
            p.makespan[b] = acc;
            p.energy[b] = e;
        }
        if (base_col == col) {
            if (p.base_T) *p.base_T = acc;
            if (p.base_E) *p.base_E = e;
        }
    } else if (want_sums) {
        if (p.slack_sum) p.slack_sum[b] = acc;
        if (p.n_critical) p.n_critical[b] = (int32_t)nc;
    }
}
