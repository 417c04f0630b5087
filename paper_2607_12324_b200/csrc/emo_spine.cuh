// The spine kernels (sm_100a): emo_spine_fwd and emo_spine_bwd walk the spine program of emo_flow.h.
// Included only by emo_lib.cu.
//
// A group of 32 policies (one per thread) has one spine warp and `workers` worker warps; a block holds
// `groups` groups and the producer warps of emo_flow.cuh, which bring one stage at a time into a ring of
// shared-memory buffers.  The recurrence of Eq. 1 runs through the spine warp alone: per segment it takes
// the maximum of two value slots, adds the segment's sum and stores the result, all in its own program
// order, so no value is ever waited for inside a stage; there is no branch in an operation (a taken branch
// costs a lone warp more than the operation itself).  Everything that does not depend on the recurrence is
// done by the workers, each of which walks whole lanes of the stage as streams of positions, four
// positions at a time so that the look-ups overlap: the level and table look-ups, the running sums per
// segment, the energy (forward) and, backward, the slack of every member (one number per segment) and the
// tails that nodes of much earlier stages read (folded into a slot of the reader with a maximum).  The
// workers run ahead of the spine with the sums and one stage behind it with the stores; mbarriers per group
// and buffer of sums order the three.  Forward, a worker also copies the spine's part of the stage
// (header, terminal bounds, operations) to a ring of the group, so that the stage buffer is free again as
// soon as the sums are taken and the loads run several stages ahead of the spine.
//
// Every wait is bounded (wait_cycles); a wait that runs out sets the block's abort word, which ends every
// other wait of the block early, and EMO_E_TIMEOUT goes to *status.  The spine polls tightly (its wake-up
// time is on the critical path), workers and producers nap between polls.
#pragma once
#include "emo_flow.cuh"

__device__ __noinline__ bool emo_spine_wait_slow(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < 4096u; ++i) {
            if (emo_mbar_test(bar, parity)) return true;
            if (i > 8u) __nanosleep(40);
        }
        if (*abort_word || clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ bool emo_spine_wait(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    if (emo_mbar_test(bar, parity)) return true;
    return emo_spine_wait_slow(bar, parity, abort_word, limit);
}
// The workers' waits: they run ahead of the spine (sums) or behind it (stores), so a late wake-up costs nothing,
// while every poll of the 20-odd waiting warps takes an issue slot from the spine.
__device__ __noinline__ bool emo_worker_wait_slow(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    // test_wait, not try_wait: try_wait spins inside (several barrier reads and naps per call)
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < 1024u; ++i) {
            __nanosleep(200);
            if (emo_mbar_test(bar, parity)) return true;
        }
        if (*abort_word || clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ bool emo_worker_wait(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    if (emo_mbar_test(bar, parity)) return true;
    return emo_worker_wait_slow(bar, parity, abort_word, limit);
}
__device__ __forceinline__ void emo_sts_u32(unsigned a, unsigned v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

// st.global of a 32-bit word under a predicate (no branch): base + row * pitch
__device__ __forceinline__ void emo_stg_u32_if(uint32_t *base, unsigned row, unsigned pitch_bytes, unsigned v, unsigned ok)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .u64 a;\n\t"
        "setp.ne.u32 p, %4, 0;\n\t"
        "mad.wide.u32 a, %1, %2, %0;\n\t"
        "@p st.global.u32 [a], %3;\n\t}"
        ::"l"(base), "r"(row), "r"(pitch_bytes), "r"(v), "r"(ok)
        : "memory");
}
__device__ __forceinline__ void emo_sts_u32_if(unsigned a, unsigned v, unsigned ok)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.u32 [%0], %1;\n\t}" ::"r"(a), "r"(v), "r"(ok) : "memory");
}
#define EMO_SCLK() (p.prof ? clock64() : 0LL)

// Barriers of group g and sums buffer a: workers -> spine (sums ready), spine -> workers (results ready),
// workers -> everybody (stores done).
__device__ __forceinline__ unsigned emo_spine_bar(const FlowParams &p, unsigned smem0, int g, int a, int which)
{
    return smem0 + p.off_sbar + (unsigned)(((g * kFlowMaxBuf + a) * 3 + which) * 8);
}

// Position of a stage in a ring of n buffers and the parity of its use of the buffer, kept by steps (no division).
struct SpineRing {
    int idx = 0, par = 0, n = 1;
    __device__ __forceinline__ void next()
    {
        if (++idx == n) {
            idx = 0;
            par ^= 1;
        }
    }
};

struct SpineRole {
    bool producer, spine;
    int group, widx;      // producer: widx = its index among the producers
};
// Which warp does what: the spine warps first, then the workers group by group, then the producers.  (Giving the
// spine and producer warps every fourth warp index, so that the workers sit on other schedulers, changed nothing:
// with four groups per block the spine waits on the shared-memory pipe, which all warps of the SM share.)
__device__ __forceinline__ SpineRole emo_spine_role(const FlowParams &p, int warp)
{
    SpineRole r;
    const int n_sp = p.groups, n_wk = p.groups * p.workers;
    r.producer = warp >= n_sp + n_wk;
    r.spine = warp < n_sp;
    r.group = r.spine ? warp : (r.producer ? 0 : (warp - n_sp) / p.workers);
    r.widx = r.spine ? 0 : (r.producer ? warp - n_sp - n_wk : (warp - n_sp) - r.group * p.workers);
    return r;
}
__device__ __forceinline__ void emo_spine_init(const FlowParams &p, unsigned smem0, unsigned char *smem, int n_cons)
{
    if (threadIdx.x == 0)
        for (int g = 0; g < p.groups; ++g)
            for (int a = 0; a < p.nacc; ++a) {
                emo_mbar_init(emo_spine_bar(p, smem0, g, a, 0), p.workers);
                emo_mbar_init(emo_spine_bar(p, smem0, g, a, 1), 1);
                emo_mbar_init(emo_spine_bar(p, smem0, g, a, 2), p.workers);
            }
    emo_flow_init(p, smem0, smem, n_cons);
}

// ---------------------------------------------------------------------------------------------------
// Forward pass (Eq. 1, Eq. 2): makespan and energy per policy, the restore list for the backward pass.
// Stage header (first 16 bytes of the blob): operations, segments, first restore row of the stage.
// ---------------------------------------------------------------------------------------------------
template <int MAXT>
__global__ void __launch_bounds__(MAXT, 1) emo_spine_fwd(FlowParams p)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, K = p.K, nbuf = p.nbuf, nacc = p.nacc, ptile = p.ptile, W = p.workers;
    const SpineRole role = emo_spine_role(p, warp);
    const int group = role.group;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !role.producer && b < p.B;
    const int base_col = (p.want_base && p.B >= b0 && p.B < b0 + ptile) ? (int)(p.B - b0) : -1;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + p.off_bar;
    volatile int *abort_word = reinterpret_cast<volatile int *>(emo_smem + p.off_bar + 16 * kFlowMaxBuf);
    const unsigned stage0 = smem0 + p.off_stage0;
    const long long limit = p.wait_cycles;
    emo_spine_init(p, smem0, emo_smem, groups * W);      // the spine reads its own copy: only the workers hold a stage buffer

    long long T = 0;
    double ea = 0.0;
    bool failed = false;
    if (role.producer) {
        emo_flow_produce<false, true>(p, stage0, bar0, abort_word, lane, role.widx);
    } else if (role.spine) {
        const unsigned slot_lane4 = smem0 + (unsigned)group * p.slot_bytes + (unsigned)lane * 4u;
        uint32_t *const rst_lane = p.restore ? p.restore + (size_t)blockIdx.x * p.restore_rows * ptile + col : nullptr;
        long long t_full = 0, t_pre = 0, t_loop = 0;
        const unsigned ptile4 = (unsigned)ptile * 4u;
        SpineRing ra;
        ra.n = nacc;
        const long long t_begin = EMO_SCLK();
        for (int cst = 0; cst < p.stages; ++cst) {
            const int a = ra.idx;
            const long long tw0 = EMO_SCLK();
            const long long tw1 = tw0;
            if (!emo_spine_wait(emo_spine_bar(p, smem0, group, a, 0), ra.par, abort_word, limit)) {
                failed = true;
                break;
            }
            const long long tw2 = EMO_SCLK();
            t_full += tw1 - tw0;
            t_pre += tw2 - tw1;
            const unsigned sta = smem0 + p.off_oring + (unsigned)(a * groups + group) * p.oring_bytes;      // the group's copy
            const uint4 hd = emo_lds128(sta);
            const int n_ops = (int)emo_uniform(hd.x);
            const unsigned acc_a = smem0 + p.off_acc + (unsigned)(a * groups + group) * p.acc_bytes + (unsigned)lane * 4u;
            unsigned op_a = sta + p.off_ops;
            uint4 d0 = emo_lds128(op_a), d1 = emo_lds128(op_a + 16u);
            // restore rows in the spine program's own numbering, or in that of the lane-stream program whose backward
            // kernel will read them (pair_rows)
            const unsigned push0 = p.pair_rows ? hd.w : hd.z, push_shift = p.pair_rows ? 20u : 8u;
            unsigned tcount = 0;
            const long long tl0 = EMO_SCLK();
            for (int i = 0; i < n_ops; ++i) {
                const uint4 c0 = d0, c1 = d1;
                op_a += 32u;
                d0 = emo_lds128(op_a);          // the next operation's words (one spare operation follows the last)
                d1 = emo_lds128(op_a + 16u);
                const unsigned x0 = emo_lds_u32(slot_lane4 + c0.x);
                const unsigned x1 = emo_lds_u32(slot_lane4 + c0.z);
                unsigned S = emo_lds_u32(acc_a + c1.z);
                const unsigned fl = c1.w;
                S = (fl & emo::kSp_NoSum) ? 0u : S;
                const unsigned y = max(emo_floor_sub(x0, c0.y), emo_floor_sub(x1, c0.w)) + S;
                // the lane's previous value (always the first operand) goes to the restore list where the backward pass cannot
                // derive it; no branch: a taken branch costs this lone warp more than the whole operation
                emo_stg_u32_if(rst_lane, push0 + ((fl >> push_shift) & 0xFFFu), ptile4, x0, (fl & emo::kSp_Push) && rst_lane);
                if (fl & emo::kSp_Terminal) {
                    const unsigned pa = sta + p.off_tpool + (tcount++) * 8u;
                    const long long lb = (long long)((unsigned long long)emo_lds_u32(pa) | ((unsigned long long)emo_lds_u32(pa + 4u) << 32));
                    T = emo_max64(T, lb + (long long)(unsigned long long)y);
                }
                emo_sts_u32(slot_lane4 + c1.x, y);
                emo_sts_u32(slot_lane4 + c1.y, y);
            }
            t_loop += EMO_SCLK() - tl0;
            __syncwarp();
            if (lane == 0) emo_mbar_arrive(emo_spine_bar(p, smem0, group, a, 1));
            ra.next();
        }
        if (!failed && rst_lane)
            for (int ln = 0; ln < lanes; ++ln) rst_lane[((size_t)p.pushes + ln) * ptile] = emo_lds_u32(slot_lane4 + (unsigned)ln * 128u);
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_full;
            pr[1] = t_pre;
            pr[2] = EMO_SCLK() - t_begin;
            pr[3] = t_loop;
        }
    } else {
        const unsigned lmask = (unsigned)p.Lp - 1u, tab_row = p.tab_row;
        const bool is_base = base_col == col;
        const unsigned top = (unsigned)(p.L - 1);
        long long t_full = 0, t_acc = 0;
        SpineRing rs, ra;
        rs.n = nbuf;
        ra.n = nacc;
        const long long t_begin = EMO_SCLK();
        for (int cst = 0; cst < p.stages; ++cst) {
            const int s = rs.idx, a = ra.idx;
            const long long tw0 = EMO_SCLK();
            const bool ok1 = emo_worker_wait(bar0 + 8 * s, rs.par, abort_word, limit);
            const long long tw1 = EMO_SCLK();
            if (!ok1 || (cst >= nacc && !emo_worker_wait(emo_spine_bar(p, smem0, group, a, 1), ra.par ^ 1, abort_word, limit))) {
                failed = true;
                break;
            }
            t_full += tw1 - tw0;
            t_acc += EMO_SCLK() - tw1;
            const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
            const unsigned acc_a = smem0 + p.off_acc + (unsigned)(a * groups + group) * p.acc_bytes + (unsigned)lane * 4u;
            if (role.widx == 0) {
                // the spine's part of the stage goes to the group's ring
                const unsigned dst = smem0 + p.off_oring + (unsigned)(a * groups + group) * p.oring_bytes;
                for (unsigned o = (unsigned)lane * 16u; o < p.oring_bytes; o += 512u) {
                    const uint4 v = emo_lds128(sta + o);
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + o), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                }
            }
            // A lane's positions of the stage are walked as one stream, four at a time (all look-ups of the four first, so
            // that they overlap): the running sum restarts where a segment begins and is stored where one ends.  Unused
            // positions have all-zero tables and store nothing.
            for (int ln = role.widx; ln < lanes; ln += W) {
                unsigned tab_a = sta + p.off_tab + (unsigned)(ln * K) * tab_row;
                unsigned lvl_a = sta + p.off_lvl + ((unsigned)((group * lanes + ln) * K) << 5) + (unsigned)lane;
                unsigned pos_a = sta + p.off_pos + (unsigned)(ln * K) * 4u;
                unsigned run = 0;
                for (int j0 = 0; j0 < K; j0 += 4) {
                    const uint4 pw = emo_lds128(pos_a);
                    unsigned lv[4], d[4];
                    double e[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) lv[i] = emo_lds_u8(lvl_a + 32u * i);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        lv[i] = (is_base ? top : lv[i]) & lmask;
                        const unsigned ta = tab_a + (unsigned)i * tab_row + lv[i] * 12u;
                        d[i] = emo_lds_u32(ta);
                        e[i] = __hiloint2double((int)emo_lds_u32(ta + 4u), (int)emo_lds_u32(ta + 8u));
                    }
                    const unsigned w4[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        run = (w4[i] & emo::kSpPos_First) ? d[i] : run + d[i];
                        emo_sts_u32_if(acc_a + (w4[i] >> 16) * 128u, run, w4[i] & emo::kSpPos_Last);
                        ea += e[i];
                    }
                    pos_a += 16u;
                    lvl_a += 128u;
                    tab_a += 4u * tab_row;
                }
            }
            __syncwarp();
            if (lane == 0) {
                emo_mbar_arrive(emo_spine_bar(p, smem0, group, a, 0));
                emo_mbar_arrive(bar0 + 8 * (kFlowMaxBuf + s));
            }
            rs.next();
            ra.next();
        }
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_full;
            pr[1] = t_acc;
            pr[2] = EMO_SCLK() - t_begin;
        }
    }
    if (failed && lane == 0) {
        *abort_word = 1;
        if (p.status) atomicMin(p.status, -8);
    }

    // combine the workers of a group in a fixed order (run-to-run identical energy)
    __syncthreads();
    double *part = reinterpret_cast<double *>(emo_smem + p.off_stage0);
    if (!role.producer && !role.spine) part[(size_t)(group * W + role.widx) * 32 + lane] = ea;
    __syncthreads();
    if (role.spine && !*abort_word) {
        double e = 0.0;
        for (int k = 0; k < W; ++k) e += part[(size_t)(group * W + k) * 32 + lane];
        if (act) {
            p.makespan[b] = T;
            p.energy[b] = e;
        }
        if (base_col == col) {
            if (p.base_T) *p.base_T = T;
            if (p.base_E) *p.base_E = e;
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Backward pass: slack of every node.  Stages are walked last to first.  The spine leaves per segment
// X = co + qin of its members (slack = T - A - X for all of them) and, where members are folded, the
// head's tail; the workers store the slack and fold the members' tails one stage behind the spine, which
// before a stage waits for the stores of the stage two back (folded values are read at least two stages
// after they are written).  EXTRA: also ES, LS, the slack sums and critical counts (ES_v = lbES_v + X - tail_v).
// ---------------------------------------------------------------------------------------------------
template <int MAXT, bool EXTRA>
__global__ void __launch_bounds__(MAXT, 1) emo_spine_bwd(FlowParams p)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, K = p.K, nbuf = p.nbuf, nacc = p.nacc, ptile = p.ptile, W = p.workers;
    const SpineRole role = emo_spine_role(p, warp);
    const int group = role.group;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !role.producer && b < p.B;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + p.off_bar;
    volatile int *abort_word = reinterpret_cast<volatile int *>(emo_smem + p.off_bar + 16 * kFlowMaxBuf);
    const unsigned stage0 = smem0 + p.off_stage0;
    const long long limit = p.wait_cycles;
    emo_spine_init(p, smem0, emo_smem, groups * (1 + W));
    const unsigned slot_lane4 = smem0 + (unsigned)group * p.slot_bytes + (unsigned)lane * 4u;

    bool failed = false;
    long long ssum = 0;
    int ncrit = 0;
    if (role.producer) {
        emo_flow_produce<true, true>(p, stage0, bar0, abort_word, lane, role.widx);
    } else if (role.spine) {
        // the lanes' last completion offsets: where the walk back begins
        for (int ln = 0; ln < lanes; ++ln)
            emo_sts_u32(slot_lane4 + (unsigned)(lanes + 2 + ln) * 128u,
                        p.restore[((size_t)blockIdx.x * p.restore_rows + p.pushes + ln) * ptile + col]);
        const unsigned col4 = (unsigned)col * 4u, ptile4 = (unsigned)ptile * 4u;
        long long t_full = 0, t_pre = 0, t_post = 0, t_loop = 0;
        SpineRing rs, ra, ra2;
        rs.n = nbuf;
        ra.n = ra2.n = nacc;
        const long long t_begin = EMO_SCLK();
        for (int cst = 0; cst < p.stages; ++cst) {
            const int s = rs.idx, a = ra.idx;
            const long long tw0 = EMO_SCLK();
            bool ok = emo_spine_wait(bar0 + 8 * s, rs.par, abort_word, limit);
            const long long tw1 = EMO_SCLK();
            ok = ok && emo_spine_wait(emo_spine_bar(p, smem0, group, a, 0), ra.par, abort_word, limit);
            const long long tw2 = EMO_SCLK();
            if (ok && cst >= 2) {
                ok = emo_spine_wait(emo_spine_bar(p, smem0, group, ra2.idx, 2), ra2.par, abort_word, limit);      // stage cst - 2
                ra2.next();
            }
            if (!ok) {
                failed = true;
                break;
            }
            const long long tw3 = EMO_SCLK();
            t_full += tw1 - tw0;
            t_pre += tw2 - tw1;
            t_post += tw3 - tw2;
            const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
            const uint4 hd = emo_lds128(sta);
            const int n_ops = (int)emo_uniform(hd.x);
            const unsigned acc_a = smem0 + p.off_acc + (unsigned)(a * groups + group) * p.acc_bytes + (unsigned)lane * 4u;
            const unsigned rst_a = sta + p.off_rst + col4;
            unsigned op_a = sta + p.off_ops;
            uint4 d0 = emo_lds128(op_a), d1 = emo_lds128(op_a + 16u), d2 = emo_lds128(op_a + 32u);
            for (int i = 0; i < n_ops; ++i) {
                const uint4 c0 = d0, c1 = d1, c2 = d2;
                op_a += 48u;
                d0 = emo_lds128(op_a);
                d1 = emo_lds128(op_a + 16u);
                d2 = emo_lds128(op_a + 32u);
                const unsigned x0 = emo_lds_u32(slot_lane4 + c0.x);
                const unsigned x1 = emo_lds_u32(slot_lane4 + c0.z);
                unsigned S = emo_lds_u32(acc_a + c1.z);
                const unsigned c = emo_lds_u32(slot_lane4 + c2.y);
                const unsigned fl = c1.w;
                S = (fl & emo::kSp_NoSum) ? 0u : S;
                const unsigned qin = max(emo_floor_sub(x0, c0.y), emo_floor_sub(x1, c0.w));
                const unsigned qo = qin + S;
                const unsigned cprev = emo_tld_u32_if(rst_a + ((fl >> 8) & 0xFFFu) * ptile4, 0u, fl & emo::kSp_Push, c - S);
                emo_sts_u32(acc_a + c1.z, c + qin);
                emo_sts_u32(acc_a + (EXTRA ? c2.w : c2.z), qo);      // EXTRA: every segment's head tail is kept, in a region of its own
                emo_sts_u32(slot_lane4 + c2.x, 0u);
                emo_sts_u32(slot_lane4 + c1.x, qo);
                emo_sts_u32(slot_lane4 + c1.y, qo);
                emo_sts_u32(slot_lane4 + c2.y, cprev);
            }
            t_loop += EMO_SCLK() - tw3;
            __syncwarp();
            if (lane == 0) {
                emo_mbar_arrive(emo_spine_bar(p, smem0, group, a, 1));
                emo_mbar_arrive(bar0 + 8 * (kFlowMaxBuf + s));
            }
            rs.next();
            ra.next();
        }
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_full;
            pr[1] = t_pre;
            pr[2] = EMO_SCLK() - t_begin;
            pr[3] = t_loop;
            pr[4] = t_post;
        }
    } else {
        const unsigned lmask = (unsigned)p.Lp - 1u, tab_row = p.tab_row;
        long long t_w1 = 0, t_w2 = 0, t_prew = 0, t_postw = 0;
        SpineRing rs, ra, rs1, ra1;
        rs.n = rs1.n = nbuf;
        ra.n = ra1.n = nacc;
        const long long t_begin = EMO_SCLK();
        const long long T = act ? p.makespan[b] : 0;
        const unsigned ldo8 = (unsigned)p.ldo * 8u;
        long long *const sl_lane = (p.slack && act) ? reinterpret_cast<long long *>(p.slack) + b : nullptr;
        const unsigned sl_ok = sl_lane != nullptr;
        long long *const es_lane = (EXTRA && p.ES && act) ? reinterpret_cast<long long *>(p.ES) + b : nullptr;
        long long *const ls_lane = (EXTRA && p.LS && act) ? reinterpret_cast<long long *>(p.LS) + b : nullptr;
        const unsigned es_ok = es_lane != nullptr, ls_ok = ls_lane != nullptr;
        for (int cst = 0; cst <= p.stages && !failed; ++cst) {
            if (cst < p.stages) {
                // the sums of stage cst
                const int s = rs.idx, a = ra.idx;
                const long long tq0 = EMO_SCLK();
                if (!emo_worker_wait(bar0 + 8 * s, rs.par, abort_word, limit) ||
                    (cst >= nacc && !emo_worker_wait(emo_spine_bar(p, smem0, group, a, 2), ra.par ^ 1, abort_word, limit))) {
                    failed = true;
                    break;
                }
                const long long tq1 = EMO_SCLK();
                t_w1 += tq1 - tq0;
                const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
                const unsigned acc_a = smem0 + p.off_acc + (unsigned)(a * groups + group) * p.acc_bytes + (unsigned)lane * 4u;
                // the sums per segment: every lane's positions as one stream, four at a time (see the forward kernel)
                for (int ln = role.widx; ln < lanes; ln += W) {
                    unsigned tab_a = sta + p.off_tab + (unsigned)(ln * K) * tab_row;
                    unsigned lvl_a = sta + p.off_lvl + ((unsigned)((group * lanes + ln) * K) << 5) + (unsigned)lane;
                    unsigned mem_a = sta + p.off_mem + (unsigned)(ln * K) * 32u + 12u;      // the position words
                    unsigned run = 0;
                    for (int j0 = 0; j0 < K; j0 += 4) {
                        unsigned w4[4], lv[4], d[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            w4[i] = emo_lds_u32(mem_a + 32u * i);
                            lv[i] = emo_lds_u8(lvl_a + 32u * i);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) d[i] = emo_lds_u32(tab_a + (unsigned)i * tab_row + (lv[i] & lmask) * 4u);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            run = (w4[i] & emo::kSpPos_First) ? d[i] : run + d[i];
                            emo_sts_u32_if(acc_a + (w4[i] >> 16) * 128u, run, w4[i] & emo::kSpPos_Last);
                        }
                        mem_a += 128u;
                        lvl_a += 128u;
                        tab_a += 4u * tab_row;
                    }
                }
                __syncwarp();
                if (lane == 0) emo_mbar_arrive(emo_spine_bar(p, smem0, group, a, 0));
                t_prew += EMO_SCLK() - tq1;
                rs.next();
                ra.next();
            }
            if (cst >= 1) {
                // the stores of stage cst - 1
                const int s = rs1.idx, a = ra1.idx;      // stage cst - 1
                const long long tq0 = EMO_SCLK();
                if (!emo_worker_wait(emo_spine_bar(p, smem0, group, a, 1), ra1.par, abort_word, limit)) {
                    failed = true;
                    break;
                }
                const long long tq1 = EMO_SCLK();
                t_w2 += tq1 - tq0;
                const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
                const unsigned acc_a = smem0 + p.off_acc + (unsigned)(a * groups + group) * p.acc_bytes + (unsigned)lane * 4u;
                // Every lane's positions as one stream, four at a time.  A member's slack is T - A - X of its segment
                // (A in its record, X where the spine left it); its tail, for the fold, is the head's tail minus the
                // durations of the members before it.  Unused positions have no node and fold into the unread slot.
                for (int ln = role.widx; ln < lanes; ln += W) {
                    unsigned tab_a = sta + p.off_tab + (unsigned)(ln * K) * tab_row;
                    unsigned lvl_a = sta + p.off_lvl + ((unsigned)((group * lanes + ln) * K) << 5) + (unsigned)lane;
                    unsigned mem_a = sta + p.off_mem + (unsigned)(ln * K) * 32u;
                    unsigned q = 0;
                    for (int j0 = 0; j0 < K; j0 += 4) {
                        uint4 m[4], n4[4];
                        unsigned lv[4], d[4], X[4], qh[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            m[i] = emo_lds128(mem_a + 32u * i);
                            n4[i] = emo_lds128(mem_a + 32u * i + 16u);
                            lv[i] = emo_lds_u8(lvl_a + 32u * i);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const unsigned xa = acc_a + (m[i].w >> 16) * 128u;
                            X[i] = emo_lds_u32(xa);
                            qh[i] = emo_lds_u32(EXTRA ? acc_a + p.acc_all_off + ((m[i].w >> 4) & 0xFFFu) * 128u : xa + 128u);
                            d[i] = emo_lds_u32(tab_a + (unsigned)i * tab_row + (lv[i] & lmask) * 4u);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const long long A = (long long)((unsigned long long)n4[i].x | ((unsigned long long)n4[i].y << 32));
                            const long long sl = (T - A) - (long long)(unsigned long long)X[i];
                            const unsigned real = (unsigned)(m[i].x != emo::kNone);
                            emo_stg_s64_if(sl_lane, m[i].x, ldo8, sl, sl_ok & real);
                            q = (m[i].w & emo::kSpPos_First) ? qh[i] : q;
                            if (EXTRA) {
                                // ES_v = lbES_v + eo_v with eo_v = X - tail_v (X = eo + tail for every member)
                                const long long lb = (long long)((unsigned long long)n4[i].z | ((unsigned long long)n4[i].w << 32));
                                const long long es = lb + (long long)(unsigned long long)(X[i] - q);
                                emo_stg_s64_if(es_lane, m[i].x, ldo8, es, es_ok & real);
                                emo_stg_s64_if(ls_lane, m[i].x, ldo8, es + sl, ls_ok & real);
                                ssum += real ? sl : 0;
                                ncrit += (real && sl == 0) ? 1 : 0;
                            }
                            emo_red_max_u32(slot_lane4 + m[i].y, emo_floor_sub(q, m[i].z));
                            q -= d[i];
                        }
                        mem_a += 128u;
                        lvl_a += 128u;
                        tab_a += 4u * tab_row;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    emo_mbar_arrive(emo_spine_bar(p, smem0, group, a, 2));
                    emo_mbar_arrive(bar0 + 8 * (kFlowMaxBuf + s));
                }
                t_postw += EMO_SCLK() - tq1;
                rs1.next();
                ra1.next();
            }
        }
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_w1;
            pr[1] = t_w2;
            pr[2] = EMO_SCLK() - t_begin;
            pr[3] = t_prew;
            pr[4] = t_postw;
        }
    }
    if (failed && lane == 0) {
        *abort_word = 1;
        if (p.status) atomicMin(p.status, -8);
    }
    if (EXTRA) {
        // per-policy sums: the workers' parts combined in worker order
        __syncthreads();
        long long *part = reinterpret_cast<long long *>(emo_smem + p.off_stage0);
        if (!role.producer && !role.spine) {
            long long *pd = part + ((size_t)(group * W + role.widx) * 32 + lane) * 2;
            pd[0] = ssum;
            pd[1] = (long long)ncrit;
        }
        __syncthreads();
        if (role.spine && act && !*abort_word) {
            long long s2 = 0, cnt = 0;
            for (int k = 0; k < W; ++k) {
                s2 += part[((size_t)(group * W + k) * 32 + lane) * 2];
                cnt += part[((size_t)(group * W + k) * 32 + lane) * 2 + 1];
            }
            if (p.slack_sum) p.slack_sum[b] = s2;
            if (p.n_critical) p.n_critical[b] = (int32_t)cnt;
        }
    }
}
#undef EMO_SCLK
