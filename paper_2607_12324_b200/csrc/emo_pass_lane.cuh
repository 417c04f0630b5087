// Staged pass kernel, one warp per schedule lane and ONE policy per thread (sm_100a).
//
// A group of 32 policies is carried by `lanes` warps, one per schedule lane; a block holds several
// groups and the producer warps that fill the ring of stages (emo_produce).  Compared with two
// policies per thread this doubles the number of resident warps, which is what the path is short
// of: every warp is a serial chain of dependent steps, and only other warps can fill the issue slots
// it leaves.  The per-entry work is kept small by a program layout made for it (see
// emo_lane_layout.cuh: 32-byte entries with the running-value mask precomputed, one 12-byte table
// element per level: duration, energy high word, energy low word).
//
// The warps of a group do not run in lockstep.  Each walks its own column of the step program and
// waits only for the values it reads: every exchange slot (32 x 8 bytes) has an mbarrier whose phase
// completes when the slot's next value has been written, and the entry names the phase parity to
// wait for.  The group meets at a named barrier every `sync` steps, which bounds the drift
// between its warps; the host compiler reuses a slot only across such a barrier.
// (Tried and measured slower on the backward pass: carrying the parity in bit 63 of the value and
// polling the word itself instead of an mbarrier.)
// Included only by emo_lib.cu.
#pragma once
#include "emo_lane_layout.cuh"

constexpr unsigned kLaneSlotStride = 272;      // 8-byte mbarrier, 8 bytes unused, 32 lanes x 8 bytes

// What a step needs from its stage, independent of the recurrence; fetched one step ahead of its use.
struct EmoLaneFetched {
    uint4 e;            // entry words 0..3
    unsigned d;         // duration at the policy's level
    double g;           // forward: energy at that level
    long long es;       // backward: earliest start of the node
};

template <bool BWD, bool EXTRA, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) emo_pass_lane(LaneParams ip)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const StagedParams &sp = ip.sp;
    const PassParams &p = sp.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, nstages = sp.stages, sc = sp.sc, sync = p.sync;
    const int steps = p.steps;                          // padded: a multiple of sc
    const int n_cons = groups * lanes;                  // consumer warps; the warps after them produce
    const bool producer = warp >= n_cons;
    const int group = producer ? 0 : warp / lanes;
    const int chain = warp - group * lanes;
    const int ptile = sp.ptile;                         // 32 * groups
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !producer && b < p.B;
    // column of the virtual all-max policy inside this block's tile (forward only), or -1
    const int base_col = (!BWD && p.want_base && p.B >= b0 && p.B < b0 + ptile) ? (int)(p.B - b0) : -1;
    unsigned char *part_base = emo_smem + sp.off_part;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + sp.off_bar;           // full[k] at bar0 + 8k, empty[k] after them
    volatile int *abort_flag = reinterpret_cast<volatile int *>(emo_smem + sp.off_bar + 16 * kMaxStages);
    const unsigned stage0 = smem0 + sp.off_stage0;
    const unsigned stage_bytes = sp.stage_bytes;

    for (int i = threadIdx.x; i < groups * p.slots; i += blockDim.x) emo_mbar_init(smem0 + (unsigned)i * kLaneSlotStride, 1);
    if (threadIdx.x == 0) {
        for (int k = 0; k < nstages; ++k) {
            emo_mbar_init(bar0 + 8 * k, 1 + 32 * kProducerWarps);   // expect-tx arrival + every producer lane's cp.async arrival
            emo_mbar_init(bar0 + 8 * (kMaxStages + k), n_cons);
        }
        for (int k = 0; k <= groups; ++k) abort_flag[k] = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    long long h = 0;
    double ea = 0.0;
    long long acc = 0;        // forward: running makespan; backward: slack sum
    int nc = 0;               // backward: critical nodes

    if (producer) {
        emo_produce(sp, stage0, bar0, abort_flag + groups, lane, warp - n_cons);
    } else {
        const int n_chunks = steps / sc;
        const unsigned slotbar_base = smem0 + (unsigned)group * p.slots * kLaneSlotStride;
        const unsigned lane8 = 16u + (unsigned)lane * 8u;
        const long long T0 = (BWD && act) ? p.makespan[b] : 0;
        const unsigned tab_entry = ip.tab_entry, lmask = (unsigned)p.Lp - 1u;
        const unsigned d_ent = (unsigned)lanes * 32u, d_tab = (unsigned)lanes * tab_entry, d_lvl = (unsigned)lanes * ptile,
                       d_es = d_lvl * 8u;
        const unsigned ldes8 = (unsigned)p.ldes * 8u, ldo8 = (unsigned)p.ldo * 8u;     // pitches below 2^28 elements
        long long *const es_lane = (!BWD && EXTRA && p.ES && act) ? reinterpret_cast<long long *>(p.ES) + b : nullptr;
        long long *const spill_lane = (!BWD && p.spill && act)
            ? reinterpret_cast<long long *>(p.spill) + (size_t)(b / p.spill_ptile) * p.spill_rows * p.spill_ptile + (b % p.spill_ptile)
            : nullptr;
        const unsigned spill8 = (unsigned)p.spill_ptile * 8u;
        long long *const ls_lane = (BWD && EXTRA && p.LS && act) ? reinterpret_cast<long long *>(p.LS) + b : nullptr;
        long long *const sl_lane = (BWD && p.slack && act) ? reinterpret_cast<long long *>(p.slack) + b : nullptr;
        const bool want_sums = BWD && EXTRA && sp.want_sums != 0 && act;
        const unsigned spill_ok = spill_lane != nullptr, slack_ok = sl_lane != nullptr;
        const int gthreads = lanes * 32;
        volatile int *my_abort = abort_flag + group;
        bool dead = false;
        unsigned ent_a = 0, tab_a = 0, lvl_a = 0, es_a = 0;

        auto fetch = [&](EmoLaneFetched &x) {
            x.e = emo_lds128(ent_a);
            const unsigned l = emo_lds_u8(lvl_a) & lmask;
            if (BWD) x.es = emo_lds_s64(es_a);
            if (!BWD) {
                // three words per level, 12 bytes apart: with a stride of three words the 32 levels
                // of a row fall into 32 different banks, so each of these loads is one wavefront
                // whatever levels the lanes hold (one 16-byte load per lane cost about ten)
                const unsigned ta = tab_a + l * 12u;
                x.d = emo_lds_u32(ta);
                x.g = __hiloint2double((int)emo_lds_u32(ta + 4u), (int)emo_lds_u32(ta + 8u));
            } else {
                x.d = emo_lds_u32(tab_a + l * 4u);
            }
        };
        // a plain node: the lane's own value is its start and no slot is read (forward: none
        // is written either)
        auto simple = [&](const EmoLaneFetched &f) {
            if (!BWD) {
                // (an idle entry inside a run: row kNone, nothing stored, duration and energy 0)
                emo_stg_row_if(spill_lane, f.e.x, spill8, h, spill_ok);
                if (EXTRA && es_lane && f.e.x != emo::kNone) *emo_row_ptr(es_lane, emo_lds_u32(ent_a - d_ent + 20u), ldes8) = h;
                ea += f.g;
                h = emo_add_dur(h, f.d);
            } else {
                h = emo_add_dur(h, f.d);
                const unsigned out = f.e.y & 255u;
                const unsigned bar = slotbar_base + out * kLaneSlotStride;
                emo_sts_s64_if(bar + lane8, h, out, kLaneNoSlot);
                __syncwarp();
                emo_mbar_arrive_if(bar, out != kLaneNoSlot && lane == 0);
                const long long ls = T0 - h, sl = ls - f.es;
                if (sl_lane) *emo_row_ptr(sl_lane, f.e.x, ldo8) = sl;
                if (EXTRA) {
                    if (ls_lane) *emo_row_ptr(ls_lane, f.e.x, ldo8) = ls;
                    if (want_sums) {
                        acc += sl;
                        nc += (sl == 0);
                    }
                }
            }
        };
        // one node; ent is the address of its entry (for the rarely needed words 4 and 5)
        auto process = [&](const EmoLaneFetched &f, unsigned ent) {
            const unsigned fl = f.e.y;
            if ((fl & kLaneIdle) || dead) return;
            if (BWD && (fl & (15u << kLaneRunShift))) {
                // backward: most nodes are plain - skip every other test
                simple(f);
                return;
            }
            long long v = h & (long long)(int)f.e.z;
            if (fl & (7u << kLaneNpShift)) {
                const unsigned np = (fl >> kLaneNpShift) & 7u;
                unsigned ops = f.e.w, par = fl >> kLaneOpParShift;
                if (BWD && np == 4) {
                    // four operands (backward: a launch node waits for the four kernels it launched),
                    // straight-line: poll the four barriers, load the four values, take the maxima
                    const unsigned b0 = slotbar_base + (ops & 255u) * kLaneSlotStride, b1 = slotbar_base + ((ops >> 8) & 255u) * kLaneSlotStride,
                                   b2 = slotbar_base + ((ops >> 16) & 255u) * kLaneSlotStride, b3 = slotbar_base + (ops >> 24) * kLaneSlotStride;
                    if (!(fl & kLaneSettled) && !emo_mbar_test4(b0, b1, b2, b3, par)) {
                        if (!emo_slot_wait(b0, par & 1u, my_abort) || !emo_slot_wait(b1, (par >> 1) & 1u, my_abort) ||
                            !emo_slot_wait(b2, (par >> 2) & 1u, my_abort) || !emo_slot_wait(b3, (par >> 3) & 1u, my_abort)) {
                            *my_abort = 1;
                            dead = true;
                            return;
                        }
                    }
                    const long long x0 = emo_lds_s64(b0 + lane8), x1 = emo_lds_s64(b1 + lane8), x2 = emo_lds_s64(b2 + lane8),
                                    x3 = emo_lds_s64(b3 + lane8);
                    v = emo_max64(emo_max64(v, x0), emo_max64(emo_max64(x1, x2), x3));
                } else if (BWD && np > 1) {
                    // several operands (backward: a launch node waits for every kernel it launched):
                    // poll every slot's barrier, then load every value, then take the maxima - the
                    // latencies overlap instead of queuing behind one another
                    const unsigned ops_hi = np > 4 ? emo_lds_u32(ent + 16u) : 0u;
                    unsigned bars[emo::kMaxSlotPreds];
                    bool ready = true;
#pragma unroll
                    for (int k = 0; k < emo::kMaxSlotPreds; ++k) {
                        bars[k] = slotbar_base + (((k < 4 ? ops : ops_hi) >> (8 * (k & 3))) & 255u) * kLaneSlotStride;
                        if (k < (int)np) ready &= emo_mbar_test(bars[k], (par >> k) & 1u);
                    }
                    if (!ready) {
#pragma unroll 1
                        for (unsigned k = 0; k < np; ++k) {
                            const unsigned id = ((k < 4 ? ops : ops_hi) >> (8 * (k & 3))) & 255u;
                            if (!emo_slot_wait(slotbar_base + id * kLaneSlotStride, (par >> k) & 1u, my_abort)) {
                                *my_abort = 1;
                                dead = true;
                                return;
                            }
                        }
                    }
                    long long x[emo::kMaxSlotPreds];
#pragma unroll
                    for (int k = 0; k < emo::kMaxSlotPreds; ++k) x[k] = emo_lds_s64_if(bars[k] + lane8, k < (int)np);
#pragma unroll
                    for (int k = 0; k < emo::kMaxSlotPreds; ++k) v = emo_max64(v, x[k]);
                } else {
                    // a real loop (rare in the forward pass; unrolled and predicated it would be paid
                    // by every entry)
#pragma unroll 1
                    for (unsigned k = 0; k < np; ++k) {
                        if (k == 4) ops = emo_lds_u32(ent + 16u);
                        const unsigned bar = slotbar_base + (ops & 255u) * kLaneSlotStride;
                        if (!(fl & kLaneSettled) && !emo_mbar_test(bar, par & 1u) && !emo_slot_wait(bar, par & 1u, my_abort)) {
                            *my_abort = 1;
                            dead = true;
                            return;
                        }
                        v = emo_max64(v, emo_lds_s64(bar + lane8));
                        ops >>= 8;
                        par >>= 1;
                    }
                }
            }
            // here v is the node's start (forward: ES_v; backward: the longest tail behind v)
            const unsigned row = f.e.x;
            if (!BWD) {
                emo_stg_row_if(spill_lane, row, spill8, v, spill_ok);
                if (EXTRA && es_lane && row != emo::kNone) *emo_row_ptr(es_lane, emo_lds_u32(ent + 20u), ldes8) = v;
                ea += f.g;
            }
            v = emo_add_dur(v, f.d);
            if (!BWD || (fl & 255u) != kLaneNoSlot) {
                // slot write: store under a predicate, then lane 0 reports the value (backward: a
                // launch node writes nothing and skips this)
                const unsigned out = fl & 255u;
                const unsigned bar = slotbar_base + out * kLaneSlotStride;
                emo_sts_s64_if(bar + lane8, v, out, kLaneNoSlot);
                __syncwarp();
                emo_mbar_arrive_if(bar, out != kLaneNoSlot && lane == 0);
            }
            if (!BWD) {
                if (fl & kLaneTerminal) acc = emo_max64(acc, v);
            } else {
                const long long ls = T0 - v, sl = ls - f.es;
                emo_stg_row_if(sl_lane, row, ldo8, sl, slack_ok);
                if (EXTRA && row != emo::kNone) {
                    if (ls_lane) *emo_row_ptr(ls_lane, row, ldo8) = ls;
                    if (want_sums) {
                        acc += sl;
                        nc += (sl == 0);
                    }
                }
            }
            h = v;
        };

        for (int c = 0; c < n_chunks; ++c) {
            const int s = c % nstages;
            const bool ok = emo_mbar_test(bar0 + 8 * s, (c / nstages) & 1) || emo_mbar_wait(bar0 + 8 * s, (c / nstages) & 1);
            // a warp that gave up (or heard that the producer did) stops working but keeps walking
            // until the group's next meeting, where all its warps read one flag and leave together
            if (!ok || dead || (chain == 0 && abort_flag[groups])) {
                *my_abort = 1;
                dead = true;
            }
            const unsigned sta = stage0 + (unsigned)s * stage_bytes;
            if (base_col >= 0 && chain == 0 && (base_col >> 5) == group) {
                // the virtual all-max column: overwrite its byte in every level row of this stage
                const unsigned char top = (unsigned char)(p.L - 1);
                for (int i = lane; i < sc * lanes; i += 32)
                    emo_smem[sp.off_stage0 + (size_t)s * stage_bytes + sp.off_lvl + (size_t)i * ptile + (size_t)base_col] = top;
                __syncwarp();
            }
            // the group meets where a block of `sync` steps begins (stages may be shorter than that)
            const bool meet = lanes > 1 && ((c * sc) % sync == 0 || base_col >= 0);
            if (meet) emo_group_barrier(group + 1, gthreads);
            if ((meet || lanes == 1) && *my_abort) {
                if (lane == 0 && p.status) atomicMin(p.status, -8);
                break;
            }
            ent_a = sta + (unsigned)chain * 32u;
            tab_a = sta + ip.st.off_tab + (unsigned)chain * tab_entry;
            lvl_a = sta + sp.off_lvl + (unsigned)chain * ptile + (unsigned)col;
            es_a = sta + sp.off_es + ((unsigned)chain * ptile + (unsigned)col) * 8u;
            // everything a step reads from the stage is fetched one step ahead (after a stage's last
            // step: bytes of the next stage or the pad, never used)
            auto advance = [&]() {
                ent_a += d_ent;
                tab_a += d_tab;
                lvl_a += d_lvl;
                if (BWD) es_a += d_es;
            };
            auto step = [&](const EmoLaneFetched &cur, EmoLaneFetched &nxt) {
                const unsigned ent = ent_a;
                advance();
                fetch(nxt);
                process(cur, ent);
            };
            EmoLaneFetched x0, x1;
            fetch(x0);
            for (int j0 = 0; j0 < sc; j0 += sync) {
                if (j0 && lanes > 1) emo_group_barrier(group + 1, gthreads);
                const int n = min(sync, sc - j0);      // even
                if (BWD) {
#pragma unroll 1
                    for (int j = 0; j < n; j += 2) {
                        step(x0, x1);
                        step(x1, x0);
                    }
                } else {
                    // most entries are plain (the lane's own value is the node's start) and come in
                    // runs; the entry that starts a run says how long it is (a run ends with its block
                    // of `sync` steps, and here with the stage: the rest of it starts the next stage)
                    int j = 0;
#pragma unroll 1
                    while (j < n) {
                        int run = dead ? 0 : min((int)((x0.e.y >> kLaneRunShift) & 15u), n - j);
                        if (run) {
                            j += run;
#pragma unroll 1
                            for (; run >= 2; run -= 2) {
                                advance();
                                fetch(x1);
                                simple(x0);
                                advance();
                                fetch(x0);
                                simple(x1);
                            }
                            if (run) {
                                advance();
                                fetch(x1);
                                simple(x0);
                                x0 = x1;
                            }
                        } else {
                            step(x0, x1);
                            x0 = x1;
                            ++j;
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kMaxStages + s));
        }
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    // per (group, chain, lane): {energy | slack sum, makespan | critical count}
    if (!producer) {
        long long *pd = reinterpret_cast<long long *>(part_base) + ((size_t)(group * lanes + chain) * 32 + lane) * 2;
        pd[0] = BWD ? acc : __double_as_longlong(ea);
        pd[1] = BWD ? (long long)nc : acc;
    }
    __syncthreads();
    if (!producer && chain == 0) {
        const long long *g0 = reinterpret_cast<const long long *>(part_base) + ((size_t)(group * lanes) * 32 + lane) * 2;
        if (!BWD) {
            double e = 0.0;
            long long t = 0;
            for (int k = 0; k < lanes; ++k) {
                e += __longlong_as_double(g0[(size_t)k * 64]);
                t = emo_max64(t, g0[(size_t)k * 64 + 1]);
            }
            if (act) {
                p.makespan[b] = t;
                p.energy[b] = e;
            }
            if (base_col == col) {
                if (p.base_T) *p.base_T = t;
                if (p.base_E) *p.base_E = e;
            }
        } else if (sp.want_sums && act) {
            long long ssum = 0, cnt = 0;
            for (int k = 0; k < lanes; ++k) {
                ssum += g0[(size_t)k * 64];
                cnt += g0[(size_t)k * 64 + 1];
            }
            if (p.slack_sum) p.slack_sum[b] = ssum;
            if (p.n_critical) p.n_critical[b] = (int32_t)cnt;
        }
    }
}
