// The 32-bit pass kernels (sm_100a): emo_flow_fwd and emo_flow_bwd walk the lane-stream program of
// emo_flow.h.  Included only by emo_lib.cu.
//
// A group of 32 policies is carried by `lanes` warps, one per lane of the schedule, one policy per
// thread; a block holds `groups` groups and two producer warps.  The producers bring one stage at a
// time into a ring of shared-memory buffers: the stage's program blob (headers, records, operand
// pool, table rows) with one bulk copy (cp.async.bulk, completion counted on an mbarrier), backward
// also the stage's rows of the restore list with a second one, and the level rows of the block's
// policy tile, which lie scattered in the caller's matrix, as 16-byte cp.async pieces.  Nothing is
// multicast and nothing is read from another GPU.
//
// The warps of a group run at their own pace.  A value another lane needs travels through an
// exchange slot in shared memory: a tagged slot holds {value, tag} in one 64-bit word per policy and
// the reader polls until it finds the tag of the value it expects; a settled slot holds the value
// alone and is only read after a barrier of the group; a shared slot collects the maximum of several
// values for one reader (red.shared.max) and is reset by that reader.  The group meets at a named
// barrier where a period begins, and the compiler reuses a slot only across such a barrier.
//
// Every wait is bounded (wait_cycles): a wait that runs out marks the warp dead, the group learns
// of it at its next barrier (the barrier itself carries the flag, so all its warps decide alike),
// EMO_E_TIMEOUT goes to *status and the block winds down: consumers leave, the producers wait
// (bounded) for their copies in flight.
#pragma once
#include <type_traits>

#include "emo_flow.h"
#include "emo_pass_staged.cuh"

constexpr int kFlowMaxBuf = 8;
constexpr int kFlowRowRegs = 8;          // a stage holds at most 32 * kFlowRowRegs entries

struct FlowParams {
    const unsigned char *blob;           // [stages][blob_bytes]: header, records, pool, tables (, lbES)
    const uint32_t *rows;                // [stages][lanes][K] policy row of every entry (kNone: none)
    const uint32_t *push_base;           // [stages + 1] first restore row of every stage
    unsigned blob_bytes, off_seg, off_rec, off_pool, off_tab, off_lbes, tab_row;
    int stages, lanes, K, kshift, Lp, L;
    int groups, ptile, nbuf, nprod;      // nprod: producer warps (2 or 4)
    unsigned slot_bytes;                 // exchange slots of one group
    unsigned stage_bytes, off_lvl, off_rst, off_bar, off_stage0;
    int want_base;
    int64_t B;
    const uint8_t *lvl;
    int64_t ldb;
    uint32_t *restore;                   // [tiles][restore_rows][ptile]
    int64_t restore_rows;                // pushes + lanes
    int64_t pushes;
    int64_t *makespan;
    double *energy;
    int64_t *base_T;
    double *base_E;
    int64_t *ES, *LS, *slack;
    int64_t ldo;
    int64_t *slack_sum;
    int32_t *n_critical;
    int32_t *status;
    long long wait_cycles;               // bound of every device-side wait
    int stall_stage;                     // test hook: the producers stop before this stage (-1: off)
    long long *prof;                     // optional cycle counters, 8 per warp: waits for stages, group barriers, total, backward: special entries, runs
    // time-interval policies (forward kernel, INTV = true): the level of a pack comes from the interval that holds its
    // start time (uniform grid of change points, the block's columns of F in shared memory)
    const uint8_t *F;                    // [rowsF][I][ldF] levels
    int64_t ldF;
    int I, rowsF;
    long long delta;                     // the change points are i * delta
    float inv_mean;
    const long long *breaks;             // device [I]
    unsigned long long *busy;            // [rowsF][I][ldw] or NULL
    int64_t ldw;
    unsigned off_meta;                   // inside a stage: 16 bytes per entry {lbES_v (8), group, dmin_v}
    unsigned off_brk, off_Fs;            // inside the block's shared memory: change points, columns of F
    // spine kernels (emo_spine.cuh): inside a stage the operations, the segment list, the member records and the
    // terminal nodes' bounds; inside the block's shared memory the barriers of the groups and the segments' sums
    unsigned off_ops, off_mem, off_tpool, off_pos;   // off_pos: forward, one position word per lane position
    unsigned off_sbar, off_acc, acc_bytes;   // acc_bytes: one group's sums of one stage
    unsigned acc_all_off;                // backward with ES / LS / sums: where the heads' tails of all segments start inside them
    unsigned off_oring, oring_bytes;     // forward: per group and buffer of sums, a copy of the front of the stage (header, bounds, operations)
    int workers, nacc;                   // look-up / store warps per group, buffers of sums
    int pair_rows;                       // forward spine kernel: number the restore rows as the paired lane-stream program does
};

__device__ __forceinline__ unsigned long long emo_lds_b64v(unsigned a)
{
    unsigned long long v;
    asm volatile("ld.volatile.shared.b64 %0, [%1];" : "=l"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void emo_sts_b64v(unsigned a, unsigned long long v)
{
    asm volatile("st.volatile.shared.b64 [%0], %1;" ::"r"(a), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned emo_lds_u32v(unsigned a)
{
    unsigned v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void emo_sts_u32v(unsigned a, unsigned v)
{
    asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void emo_red_max_u32(unsigned a, unsigned v)
{
    asm volatile("red.shared.max.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
// named barrier of `nthreads` threads that also ORs a flag over them
__device__ __forceinline__ bool emo_group_barrier_or(int id, int nthreads, bool flag)
{
    unsigned r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbar.red.or.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"((unsigned)flag)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ unsigned emo_floor_sub(unsigned x, unsigned d) { return max(x, d) - d; }
// A control word that every lane of the warp loaded from the same address: the warp-wide OR gives the
// same value back, and the compiler now knows that it is uniform, so the branches on it need no
// divergence handling.
__device__ __forceinline__ unsigned emo_uniform(unsigned x)
{
    unsigned r;
    asm volatile("redux.sync.or.b32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(x));
    return r;
}

// Loads of staged data.  They are not volatile, so that the compiler may schedule them freely and
// early, but every one of them takes a token that is produced (by a volatile statement) after the
// wait that made the data visible: no load can move above that wait, and loads of the same address
// in different stages are different expressions.
__device__ __forceinline__ unsigned emo_token(unsigned x)
{
    unsigned t;
    asm volatile("mov.u32 %0, %1;" : "=r"(t) : "r"(x) : "memory");
    return t;
}
__device__ __forceinline__ unsigned emo_tld_u8(unsigned a, unsigned tok)
{
    unsigned v;
    asm("ld.shared.u8 %0, [%1]; // %2" : "=r"(v) : "r"(a), "r"(tok));
    return v;
}
// a byte of block-lifetime shared data (written once before the walk begins)
__device__ __forceinline__ unsigned emo_vld_u8(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ unsigned emo_tld_u32(unsigned a, unsigned tok)
{
    unsigned v;
    asm("ld.shared.u32 %0, [%1]; // %2" : "=r"(v) : "r"(a), "r"(tok));
    return v;
}
__device__ __forceinline__ long long emo_tld_s64(unsigned a, unsigned tok)
{
    long long v;
    asm("ld.shared.s64 %0, [%1]; // %2" : "=l"(v) : "r"(a), "r"(tok));
    return v;
}
// the staged word when `take` is set, else `other` (no access, no branch)
__device__ __forceinline__ unsigned emo_tld_u32_if(unsigned a, unsigned tok, unsigned take, unsigned other)
{
    unsigned v = other;
    asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p ld.shared.u32 %0, [%1]; // %3\n\t}" : "+r"(v) : "r"(a), "r"(take), "r"(tok));
    return v;
}
// st.global under a predicate (no branch)
__device__ __forceinline__ void emo_stg_s64_if(long long *base, unsigned row, unsigned pitch_bytes, long long v, unsigned ok)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .u64 a;\n\t"
        "setp.ne.u32 p, %4, 0;\n\t"
        "mad.wide.u32 a, %1, %2, %0;\n\t"
        "@p st.global.s64 [a], %3;\n\t}"
        ::"l"(base), "r"(row), "r"(pitch_bytes), "l"(v), "r"(ok)
        : "memory");
}
__device__ __forceinline__ uint4 emo_tld_128(unsigned a, unsigned tok)
{
    uint4 v;
    asm("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4]; // %5" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a), "r"(tok));
    return v;
}

// Bounded mbarrier wait that also gives up when the block's abort word is set.
__device__ __noinline__ bool emo_flow_wait_slow(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < 256u; ++i) {
            if (emo_mbar_test(bar, parity)) return true;      // one barrier read per poll (a try_wait spins inside)
            __nanosleep(400);      // polling costs issue slots that the working warps need
        }
        if (*abort_word || clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ bool emo_flow_wait(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    if (emo_mbar_test(bar, parity)) return true;
    return emo_flow_wait_slow(bar, parity, abort_word, limit);
}

// The same with one barrier read per poll (test_wait; a try_wait spins inside, several reads and naps per call): for
// kernels whose stages are short, where the polls of the waiting warps add up.
__device__ __noinline__ bool emo_flow_wait_fast_slow(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < 1024u; ++i) {
            __nanosleep(300);
            if (emo_mbar_test(bar, parity)) return true;
        }
        if (*abort_word || clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ bool emo_flow_wait_fast(unsigned bar, unsigned parity, volatile int *abort_word, long long limit)
{
    if (emo_mbar_test(bar, parity)) return true;
    return emo_flow_wait_fast_slow(bar, parity, abort_word, limit);
}

// Reads one operand: the slot word of this thread, polled for its tag when the descriptor asks.
// Returns false when the wait ran out.
__device__ __noinline__ unsigned long long emo_flow_poll_value(unsigned a, unsigned tag, volatile int *abort_word, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < 1024u; ++i) {
            const unsigned long long v = emo_lds_b64v(a);
            if ((unsigned)(v >> 32) == tag) return (v & 0xFFFFFFFFull) | (1ull << 32);
            if (i > 16u) __nanosleep(32);
        }
        if (*abort_word || clock64() - t0 > limit) return 0ull;
    }
}
// (The value travels in the result, not through a reference: a variable whose address is passed to a call that
// is not inlined lives in local memory for its whole life, and these sit on the critical path of every entry
// that reads a slot.)
__device__ __forceinline__ bool emo_flow_poll(unsigned a, unsigned tag, unsigned &x, volatile int *abort_word, long long limit)
{
    const unsigned long long r = emo_flow_poll_value(a, tag, abort_word, limit);
    if (r >> 32) x = (unsigned)r;
    return (r >> 32) != 0ull;
}
__device__ __forceinline__ unsigned emo_flow_operand(unsigned slot_base, int lane, unsigned w, unsigned tag, bool &dead,
                                                     volatile int *abort_word, long long limit)
{
    const unsigned off = w & emo::kOpOffMask;
    if (w & emo::kOpWord) {
        const unsigned a = slot_base + off + (unsigned)lane * 4u;
        const unsigned x = emo_lds_u32v(a);
        if (w & emo::kOpClear) emo_sts_u32v(a, 0u);
        return x;
    }
    const unsigned a = slot_base + off + (unsigned)lane * 8u;
    const unsigned long long v = emo_lds_b64v(a);
    unsigned x = (unsigned)v;
    if (!(w & emo::kOpNoPoll) && (unsigned)(v >> 32) != tag) {
        if (!emo_flow_poll(a, tag, x, abort_word, limit)) {
            dead = true;
            *abort_word = 1;      // the other waits of the block end early
        }
    }
    return x;
}
// Writes a node's value where its readers expect it.
__device__ __forceinline__ void emo_flow_out(unsigned slot_base, int lane, unsigned v, bool tagged, bool shared, unsigned off,
                                             unsigned aux)
{
    if (tagged) {
        emo_sts_b64v(slot_base + off + (unsigned)lane * 8u, (unsigned long long)v | ((unsigned long long)aux << 32));
    } else {
        const unsigned x = emo_floor_sub(v, aux);
        const unsigned a = slot_base + off + (unsigned)lane * 4u;
        if (shared) emo_red_max_u32(a, x);
        else emo_sts_u32v(a, x);
    }
}

// The same two steps without a branch, for the entries that need their record.  Every access is
// predicated on the descriptor's kind bits, so that an entry costs one straight run of instructions
// whatever it reads and writes; a branch costs a lone warp some forty cycles of fetch bubble, and these
// entries sit on the lanes' critical paths.
// Operand: x = the slot's value (0 when the operand is absent), tg = the tag found beside it (tagged
// slots only), a = the address read (for a later poll).
__device__ __forceinline__ void emo_flow_operand_u(unsigned slot_lane4, unsigned lane4, unsigned w, unsigned present, unsigned &x,
                                                   unsigned &tg, unsigned &a)
{
    asm volatile(
        "{\n\t.reg .pred pp, pw, pt, pc;\n\t.reg .b32 k;\n\t.reg .b64 t;\n\t"
        "setp.ne.u32 pp, %4, 0;\n\t"
        "and.b32 k, %3, 0x40000000;\n\t"
        "setp.ne.and.u32 pw, k, 0, pp;\n\t"
        "setp.eq.and.u32 pt, k, 0, pp;\n\t"
        "and.b32 k, %3, 0x20000000;\n\t"
        "setp.ne.and.u32 pc, k, 0, pp;\n\t"
        "and.b32 %2, %3, 0x1FFFFFFF;\n\t"
        "add.u32 %2, %2, %5;\n\t"
        "@pt add.u32 %2, %2, %6;\n\t"
        "mov.u32 %0, 0;\n\t"
        "mov.u32 %1, 0;\n\t"
        "@pw ld.volatile.shared.u32 %0, [%2];\n\t"
        "@pt ld.volatile.shared.b64 t, [%2];\n\t"
        "@pt mov.b64 {%0, %1}, t;\n\t"
        "@pc st.volatile.shared.u32 [%2], 0;\n\t}"
        : "=&r"(x), "=&r"(tg), "=&r"(a)
        : "r"(w), "r"(present), "r"(slot_lane4), "r"(lane4)
        : "memory");
}
// Output: tagged (value + tag), settled (corrected value) or shared (corrected value folded in), or none.
__device__ __forceinline__ void emo_flow_out_u(unsigned slot_lane4, unsigned lane4, unsigned v, unsigned off, unsigned aux, unsigned tagged,
                                               unsigned settled, unsigned shared)
{
    asm volatile(
        "{\n\t.reg .pred pt, ps, pa;\n\t.reg .b32 aw, at, xs;\n\t"
        "setp.ne.u32 pt, %5, 0;\n\t"
        "setp.ne.u32 pa, %7, 0;\n\t"
        "setp.ne.and.u32 ps, %6, 0, !pa;\n\t"
        "add.u32 aw, %0, %3;\n\t"
        "add.u32 at, aw, %1;\n\t"
        "max.u32 xs, %2, %4;\n\t"
        "sub.u32 xs, xs, %4;\n\t"
        "@pt st.volatile.shared.v2.u32 [at], {%2, %4};\n\t"
        "@ps st.volatile.shared.u32 [aw], xs;\n\t"
        "@pa red.shared.max.u32 [aw], xs;\n\t}"
        ::"r"(slot_lane4), "r"(lane4), "r"(v), "r"(off), "r"(aux), "r"(tagged), "r"(settled), "r"(shared)
        : "memory");
}

// The producer warps of both kernels.  Stages are issued in walking order (backward: last first).
template <bool BWD, bool FAST = false>
__device__ __forceinline__ void emo_flow_produce(const FlowParams &p, unsigned stage0, unsigned bar0, volatile int *abort_word,
                                                 int lane, int pw)
{
    const int stages = p.stages, nbuf = p.nbuf, lanes = p.lanes, K = p.K, ptile = p.ptile;
    const int ne = lanes * K;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int64_t lvl_left = p.ldb - b0;
    const unsigned lvl_bytes = lvl_left > 0 ? (unsigned)min((int64_t)ptile, lvl_left) : 0u;
    const int pieces = (int)(lvl_bytes >> 4);
    const unsigned inv_pieces = pieces > 1 ? (unsigned)((0x100000000ULL + pieces - 1) / pieces) : 0u;
    int pshift = -1;      // log2(pieces) when it is a power of two
    for (int q = 0; q < 6; ++q)
        if (pieces == (1 << q)) pshift = q;
    const int nprod = p.nprod;
    const uint8_t *const lvl0 = p.lvl + b0;
    int issued = 0;
    bool gave_up = false;
    unsigned rr[kFlowRowRegs], rr_next[kFlowRowRegs];
    auto load_rows = [&](int c, unsigned *dst) {
        const int st = BWD ? stages - 1 - c : c;
        const size_t q0 = (size_t)st * ne;
#pragma unroll
        for (int k = 0; k < kFlowRowRegs; ++k) {
            const int i = 32 * k + lane;
            dst[k] = (c < stages && i < ne) ? __ldg(p.rows + q0 + i) : emo::kNone;
        }
    };
    load_rows(0, rr);
    long long t_wait = 0, t_issue = 0;
    const long long t_begin = clock64();
    for (int c = 0; c < stages; ++c) {
        const int st = BWD ? stages - 1 - c : c;
        const int s = c % nbuf;
        load_rows(c + 1, rr_next);
        unsigned rst_rows = 0, rst_first = 0;
        if (BWD) {
            rst_first = __ldg(p.push_base + st);
            rst_rows = __ldg(p.push_base + st + 1) - rst_first;
        }
        const long long tw0 = clock64();
        if (c >= nbuf) {
            const unsigned eb = bar0 + 8 * (kFlowMaxBuf + s), ep = ((c / nbuf) - 1) & 1;
            if (!(FAST ? emo_flow_wait_fast(eb, ep, abort_word, p.wait_cycles) : emo_flow_wait(eb, ep, abort_word, p.wait_cycles))) {
                if (lane == 0) {
                    *abort_word = 1;
                    if (p.status) atomicMin(p.status, -8);
                }
                gave_up = true;
                break;
            }
        }
        if (*abort_word || c == p.stall_stage) { gave_up = true; break; }
        const long long tw1 = clock64();
        t_wait += tw1 - tw0;
        issued = c + 1;
        const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
        const unsigned full = bar0 + 8 * s;
        if (lane == 0 && pw == 0) {
            const unsigned rst_bytes = rst_rows * (unsigned)ptile * 4u;
            emo_mbar_expect_tx(full, p.blob_bytes + rst_bytes);
            emo_bulk_g2s(sta, p.blob + (size_t)st * p.blob_bytes, p.blob_bytes, full);
            if (BWD && rst_bytes)
                emo_bulk_g2s(sta + p.off_rst, p.restore + ((size_t)blockIdx.x * p.restore_rows + rst_first) * ptile, rst_bytes, full);
        }
        if (pieces) {
            // level rows: piece pc of entry i goes to [pc / 2][i][pc % 2] of the stage's level area (a group of
            // 32 policies has its 32 bytes of every entry side by side); the producer warps share the pieces
            const unsigned dst0 = sta + p.off_lvl;
            const unsigned gstride = (unsigned)(lanes * K) << 5;
#pragma unroll
            for (int k = 0; k < kFlowRowRegs; ++k) {
                if (32 * k < ne) {
                    for (int it = pw; it < pieces; it += nprod) {
                        const unsigned t = (unsigned)lane + 32u * (unsigned)it;
                        const unsigned e = pshift >= 0 ? t >> pshift : __umulhi(t, inv_pieces);   // t / pieces
                        const unsigned pc = t - e * (unsigned)pieces;
                        const unsigned row = __shfl_sync(0xFFFFFFFFu, rr[k], e & 31);
                        const unsigned i = 32u * (unsigned)k + e;                      // entry: lane i / K, position i % K
                        if ((int)i < ne && row != emo::kNone)
                            emo_cp_async16(dst0 + (pc >> 1) * gstride + (i << 5) + (pc & 1u) * 16u, lvl0 + (size_t)row * p.ldb + pc * 16u);
                    }
                }
            }
        }
        emo_cp_async_arrive(full);
#pragma unroll
        for (int k = 0; k < kFlowRowRegs; ++k) rr[k] = rr_next[k];
        t_issue += clock64() - tw1;
    }
    if (p.prof && lane == 0 && blockIdx.x < 512) {
        long long *pr = p.prof + ((size_t)blockIdx.x * 32 + (threadIdx.x >> 5)) * 8;
        pr[0] = t_wait;
        pr[1] = t_issue;
        pr[2] = clock64() - t_begin;
    }
    if (gave_up) {
        // do not leave the block while copies into its shared memory may still be in flight
        for (int c = max(0, issued - nbuf); c < issued; ++c)
            (void)emo_flow_wait(bar0 + 8 * (c % nbuf), (c / nbuf) & 1, abort_word + 1, p.wait_cycles);
    }
}

__device__ __forceinline__ void emo_flow_init(const FlowParams &p, unsigned smem0, unsigned char *smem, int n_cons)
{
    for (unsigned i = threadIdx.x; i < (unsigned)p.groups * p.slot_bytes / 4u; i += blockDim.x)
        reinterpret_cast<unsigned *>(smem)[i] = 0u;
    if (threadIdx.x == 0) {
        const unsigned bar0 = smem0 + p.off_bar;
        for (int k = 0; k < p.nbuf; ++k) {
            emo_mbar_init(bar0 + 8 * k, 1 + 32 * p.nprod);
            emo_mbar_init(bar0 + 8 * (kFlowMaxBuf + k), n_cons);
        }
        volatile int *abort_word = reinterpret_cast<volatile int *>(smem + p.off_bar + 16 * kFlowMaxBuf);
        abort_word[0] = 0;
        abort_word[1] = 0;      // never set: the drain after a failure waits its full time
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------------
// Forward pass (Eq. 1, Eq. 2): makespan and energy per policy, the restore list for the backward pass.
// A lane's entries come in segments (emo_flow.h): an optional entry that needs its record, then a run
// of plain entries.  The level and table look-ups of a run do not depend on the recurrence: they are
// issued together (one instantiation of the run per length, reached by one jump) and the run is
// then a sum.
// ---------------------------------------------------------------------------------------------------
template <int R>
__device__ __forceinline__ void emo_flow_fwd_run(unsigned la, unsigned ta0, unsigned tab_row, unsigned lmask, unsigned tok, unsigned &h,
                                                 double &ea)
{
    unsigned lv[R], d[R], ghi[R], glo[R];
#pragma unroll
    for (int i = 0; i < R; ++i) lv[i] = emo_tld_u8(la + 32u * i, tok);
#pragma unroll
    for (int i = 0; i < R; ++i) {
        const unsigned ta = ta0 + (unsigned)i * tab_row + (lv[i] & lmask) * 12u;
        d[i] = emo_tld_u32(ta, tok);
        ghi[i] = emo_tld_u32(ta + 4u, tok);
        glo[i] = emo_tld_u32(ta + 8u, tok);
    }
    double g[R];
#pragma unroll
    for (int i = 0; i < R; ++i) g[i] = __hiloint2double((int)ghi[i], (int)glo[i]);
    // pairwise sums: a short dependency chain, and a fixed order (run-to-run identical energy)
#pragma unroll
    for (int w = 1; w < R; w *= 2)
#pragma unroll
        for (int i = 0; i + w < R; i += 2 * w) {
            d[i] += d[i + w];
            g[i] += g[i + w];
        }
    h += d[0];
    ea += g[0];
}

// What the forward kernel carries for time-interval policies beside its parameters.
struct FlowIntv {
    const long long *brk;        // change points in shared memory
    unsigned Fs;                 // the block's columns of F in shared memory (shared-window address of this thread's column): [rowsF * I][ptile]
    int col;                     // this thread's column in the block
    int64_t b;                   // this thread's policy
    bool count;                  // this thread adds busy time (a live policy and a busy array)
    unsigned key;                // busy time collected for (row, interval) = key, not yet added to memory
    unsigned long long sum;
};
// The level of an entry whose start offset is eo (Alg. 1: the interval that holds the start time), then its
// table entry.  No branch on anything loaded here: a node outside every policy reads the last row and any
// level (its table row holds one value), the interval index is a float guess with one exact correction (uniform
// grid), and busy time is collected in a register while the (row, interval) stays the same.
__device__ __forceinline__ void emo_flow_intv_lookup(const FlowParams &p, FlowIntv &iv, const uint4 &meta, unsigned eo, unsigned ta0,
                                                     unsigned lmask, unsigned tok, unsigned &dd, double &e)
{
    const long long start = (long long)((unsigned long long)meta.x | ((unsigned long long)meta.y << 32)) + (long long)eo;
    const bool pack = meta.z != emo::kNone;
    const unsigned rowc = min(meta.z, (unsigned)p.rowsF - 1u);
    long long iend;
    const int i = emo_interval_index<true>(start, p.I, p.delta, p.inv_mean, iv.brk, iend);
    const unsigned key = rowc * (unsigned)p.I + (unsigned)i;
    const unsigned lv = emo_vld_u8(iv.Fs + key * (unsigned)p.ptile);
    const unsigned ta = ta0 + (lv & lmask) * 12u;
    dd = emo_tld_u32(ta, tok);
    e = __hiloint2double((int)emo_tld_u32(ta + 4u, tok), (int)emo_tld_u32(ta + 8u, tok));
    const long long dur = (long long)meta.w + (long long)dd;
    const bool on = pack && iv.count;
    if (on && key != iv.key) {      // rare: the lane moved on to another interval (or device)
        if (iv.sum) atomicAdd(p.busy + (size_t)iv.key * p.ldw + iv.b, iv.sum);
        iv.key = key;
        iv.sum = 0;
    }
    const bool single = start + dur <= iend;
    iv.sum += (on && single) ? (unsigned long long)dur : 0ull;
    if (on && !single) emo_interval_busy(p.busy, p.ldw, iv.b, rowc, p.I, i, iend, start, start + dur, iv.brk);      // rare
}
// A run of r plain entries: every start time depends on the entry before it, so the look-ups form one chain
// and there is nothing to gain from one instantiation per length (which would only crowd the instruction
// cache: the look-up is some sixty instructions); a loop, inlined so that the parameters and the lane's running
// values stay in registers, with the next entry's constants requested one entry ahead.
__device__ __forceinline__ void emo_flow_fwd_run_intv(const FlowParams &p, FlowIntv &iv, unsigned r, unsigned meta_a, unsigned ta0, unsigned tab_row,
                                                   unsigned lmask, unsigned tok, unsigned &h, double &ea)
{
    uint4 meta = emo_tld_128(meta_a, tok);
#pragma unroll 1
    for (unsigned i = 0; i < r; ++i) {
        const uint4 cur = meta;
        meta = emo_tld_128(meta_a + 16u * min(i + 1u, r - 1u), tok);      // never past the run: the last entry's constants end the stage buffer
        unsigned dd;
        double e;
        emo_flow_intv_lookup(p, iv, cur, h, ta0 + i * tab_row, lmask, tok, dd, e);
        h += dd;
        ea += e;
    }
}

// The consumers read the clock only in the instantiations that fill the cycle counters (PROF): the reads sit
// between the entries of the lanes' chains and cost the backward pass 6 % when they are always there.
#define EMO_CLK() (PROF ? clock64() : 0LL)

template <int MAXT, bool INTV, bool PROF>
__global__ void __launch_bounds__(MAXT, 1) emo_flow_fwd(FlowParams p)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, K = p.K, nbuf = p.nbuf, ptile = p.ptile;
    const int n_cons = groups * lanes;
    const bool producer = warp >= n_cons;
    const int group = producer ? 0 : warp / lanes;
    const int chain = warp - group * lanes;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !producer && b < p.B;
    const int base_col = (p.want_base && p.B >= b0 && p.B < b0 + ptile) ? (int)(p.B - b0) : -1;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + p.off_bar;
    volatile int *abort_word = reinterpret_cast<volatile int *>(emo_smem + p.off_bar + 16 * kFlowMaxBuf);
    const unsigned stage0 = smem0 + p.off_stage0;
    emo_flow_init(p, smem0, emo_smem, n_cons);
    FlowIntv iv{nullptr, 0u, col, b, act && p.busy != nullptr, 0u, 0ull};
    if (INTV) {
        long long *brk = reinterpret_cast<long long *>(emo_smem + p.off_brk);
        for (int i = threadIdx.x; i < p.I; i += blockDim.x) brk[i] = p.breaks[i];
        unsigned char *Fs = emo_smem + p.off_Fs;
        const int total = p.rowsF * p.I * ptile;
        for (int k2 = threadIdx.x; k2 < total; k2 += blockDim.x) {
            const int ri = k2 / ptile, c = k2 - ri * ptile;
            Fs[k2] = (b0 + c < p.B) ? p.F[(size_t)ri * p.ldF + b0 + c] : (unsigned char)0;
        }
        iv.brk = brk;
        iv.Fs = smem0 + p.off_Fs + (unsigned)col;
        __syncthreads();
    }

    unsigned h = 0;
    double ea = 0.0;
    long long acc = 0;
    if (producer) {
        emo_flow_produce<false>(p, stage0, bar0, abort_word, lane, warp - n_cons);
    } else {
        const unsigned slot_base = smem0 + (unsigned)group * p.slot_bytes;
        const unsigned lane4 = (unsigned)lane * 4u, slot_lane4 = slot_base + lane4;
        const unsigned lmask = (unsigned)p.Lp - 1u, tab_row = p.tab_row;
        const int gthreads = lanes * 32;
        const long long limit = p.wait_cycles;
        uint32_t *const rst_lane = p.restore ? p.restore + (size_t)blockIdx.x * p.restore_rows * ptile + col : nullptr;
        bool dead = false, leave = false;
        long long t_wait = 0, t_bar = 0;
        const long long t_begin = EMO_CLK();
        for (int st = 0; st < p.stages && !leave; ++st) {
            const int s = st % nbuf;
            const long long tw0 = EMO_CLK();
            if (!dead && !emo_flow_wait(bar0 + 8 * s, (st / nbuf) & 1, abort_word, limit)) {
                dead = true;
                *abort_word = 1;
            }
            t_wait += EMO_CLK() - tw0;
            const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
            const unsigned tok0 = emo_token((unsigned)st);
            uint4 hd0 = make_uint4(0, 0, 0, 0), hd1 = hd0;
            if (!dead) {
                hd0 = emo_tld_128(sta + (unsigned)chain * 32u, tok0);
                hd1 = emo_tld_128(sta + (unsigned)chain * 32u + 16u, tok0);
                if (base_col >= 0 && chain == 0 && (base_col >> 5) == group) {
                    // the virtual all-max column: overwrite its byte in every level row of this stage
                    unsigned char *lv = emo_smem + p.off_stage0 + (size_t)s * p.stage_bytes + p.off_lvl + ((size_t)group * lanes * K << 5) + (base_col & 31);
                    const unsigned char top = (unsigned char)(p.L - 1);
                    for (int i = lane; i < lanes * K; i += 32) lv[(size_t)i << 5] = top;
                    __syncwarp();
                }
            }
            const unsigned seg_a = sta + p.off_seg + (unsigned)chain * emo::kSegBytes;
            unsigned rec_a = sta + p.off_rec + (unsigned)(chain * K) * 32u;
            unsigned tab_a = sta + p.off_tab + (unsigned)(chain * K) * tab_row;
            unsigned lvl_a = sta + p.off_lvl + ((unsigned)((group * lanes + chain) * K) << 5) + (unsigned)lane;
            const unsigned pool_a = sta + p.off_pool;
            unsigned meta_a = sta + p.off_meta + (unsigned)(chain * K) * 16u;
            uint32_t *push = rst_lane ? rst_lane + ((size_t)hd1.z + hd1.y) * ptile : nullptr;
            hd0.x = emo_uniform(hd0.x);
            const int nseg = (int)(hd0.x & 255u);
            unsigned tok = tok0, segw = 0;
            for (int sgi = 0; sgi < nseg || dead; ++sgi) {
                if (dead) {
                    // a wait ran out: the group's next barrier tells every warp of the group to leave
                    if (lanes > 1) (void)emo_group_barrier_or(group + 1, gthreads, true);
                    leave = true;
                    break;
                }
                // segment bytes, four at a time
                if ((sgi & 3) == 0) segw = emo_uniform(emo_tld_u32(seg_a + (unsigned)sgi, tok0));
                const unsigned sg = segw & 255u;
                segw >>= 8;
                if (sg & emo::kSegBarrier) {
                    const long long tb0 = EMO_CLK();
                    if (lanes > 1 && emo_group_barrier_or(group + 1, gthreads, false)) { leave = true; break; }
                    t_bar += EMO_CLK() - tb0;
                }
                tok = emo_token(tok + 1u);
                const int r = (int)(sg & emo::kSegRunMask);
                const unsigned sp = (sg >> 4) & 1u;
                if (sp) {
                    // an entry that needs its record; everything it reads from the stage is requested at once, and
                    // the common shapes (at most one operand, any output) run without a branch
                    const uint4 r0 = emo_tld_128(rec_a, tok);
                    const uint4 r1 = emo_tld_128(rec_a + 16u, tok);
                    const unsigned fl = r0.x;
                    unsigned dd = 0;
                    double ee = 0.0;
                    uint4 meta = make_uint4(0, 0, 0, 0);
                    if (INTV) {
                        meta = emo_tld_128(meta_a, tok);
                    } else {
                        const unsigned lb = emo_tld_u8(lvl_a, tok);
                        const unsigned ta = tab_a + (lb & lmask) * 12u;
                        dd = emo_tld_u32(ta, tok);
                        ee = __hiloint2double((int)emo_tld_u32(ta + 4u, tok), (int)emo_tld_u32(ta + 8u, tok));
                    }
                    const unsigned nops = fl >> emo::kF_NopsShift;
                    unsigned v = emo_floor_sub((fl & emo::kF_HasReg) ? h : 0u, r1.w);
                    unsigned x0, t0, a0;
                    emo_flow_operand_u(slot_lane4, lane4, r1.x, nops, x0, t0, a0);
                    const bool retry0 = nops != 0u && (r1.x & (emo::kOpWord | emo::kOpNoPoll)) == 0u && t0 != r1.y;
                    unsigned pa = pool_a + r0.w * 4u;
                    bool term = false;
                    if (__any_sync(0xFFFFFFFFu, retry0 || nops > 1u || (fl & emo::kF_Terminal) != 0u)) {
                        // the rest: a value that was not there yet, further operands, a makespan candidate
                        if (retry0 && !emo_flow_poll(a0, r1.y, x0, abort_word, limit)) {
                            dead = true;
                            *abort_word = 1;
                        }
                        for (unsigned k = 1; k < nops; ++k) {
                            const unsigned x2 = emo_flow_operand(slot_base, lane, emo_tld_u32(pa, tok), emo_tld_u32(pa + 4u, tok), dead,
                                                                 abort_word, limit);
                            v = max(v, emo_floor_sub(x2, emo_tld_u32(pa + 8u, tok)));
                            pa += 12u;
                        }
                        dead = __any_sync(0xFFFFFFFFu, dead);
                        if (dead) continue;      // on to the group's next barrier
                        if (INTV) {
                            term = (fl & emo::kF_Terminal) != 0u;      // its duration is not known yet
                        } else if (fl & emo::kF_Terminal) {
                            // a node without successors: candidate for the makespan (its bound follows the operands in the pool)
                            const long long lbc = (long long)((unsigned long long)emo_tld_u32(pa, tok) | ((unsigned long long)emo_tld_u32(pa + 4u, tok) << 32));
                            const unsigned vt = max(v, emo_floor_sub(x0, r1.z)) + dd;
                            acc = emo_max64(acc, lbc + (long long)vt);
                        }
                    }
                    v = max(v, emo_floor_sub(x0, r1.z));
                    // time-interval policies: the level follows from the start time, which is known only now
                    if (INTV) emo_flow_intv_lookup(p, iv, meta, v, tab_a, lmask, tok, dd, ee);
                    if ((fl & emo::kF_Push) && push) {
                        *push = h;
                        push += ptile;
                    }
                    ea += ee;
                    v += dd;
                    emo_flow_out_u(slot_lane4, lane4, v, r0.y, r0.z, fl & emo::kF_OutTag, fl & emo::kF_OutSet, fl & emo::kF_OutAcc);
                    if (INTV && term) {
                        // a node without successors: candidate for the makespan (its bound follows the operands in the pool)
                        const long long lbc = (long long)((unsigned long long)emo_tld_u32(pa, tok) | ((unsigned long long)emo_tld_u32(pa + 4u, tok) << 32));
                        acc = emo_max64(acc, lbc + (long long)v);
                    }
                    h = v;
                    meta_a += 16u;
                    rec_a += 32u;
                    tab_a += tab_row;
                    lvl_a += 32u;
                }
                // the run: every entry continues from the lane's previous value
                if (INTV) {
                    if (r) emo_flow_fwd_run_intv(p, iv, (unsigned)r, meta_a, tab_a, tab_row, lmask, tok, h, ea);
                } else {
                    switch (r) {
                        case 1: emo_flow_fwd_run<1>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 2: emo_flow_fwd_run<2>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 3: emo_flow_fwd_run<3>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 4: emo_flow_fwd_run<4>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 5: emo_flow_fwd_run<5>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 6: emo_flow_fwd_run<6>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 7: emo_flow_fwd_run<7>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        case 8: emo_flow_fwd_run<8>(lvl_a, tab_a, tab_row, lmask, tok, h, ea); break;
                        default: break;
                    }
                }
                meta_a += (unsigned)r * 16u;
                rec_a += (unsigned)r * 32u;
                tab_a += (unsigned)r * tab_row;
                lvl_a += (unsigned)r * 32u;
            }
            if (leave) break;
            // everything read from the stage has been used before the buffer is handed back
            asm volatile("" ::"r"(h), "l"(__double_as_longlong(ea)), "l"(acc) : "memory");
            __syncwarp();
            if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kFlowMaxBuf + s));
        }
        if (INTV && iv.count && iv.sum) atomicAdd(p.busy + (size_t)iv.key * p.ldw + iv.b, iv.sum);
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_wait;
            pr[1] = t_bar;
            pr[2] = EMO_CLK() - t_begin;
        }
        if (leave) {
            if (lane == 0) {
                *abort_word = 1;
                if (p.status) atomicMin(p.status, -8);
            }
        } else if (rst_lane) {
            rst_lane[((size_t)p.pushes + chain) * ptile] = h;      // the lane's last value: where the backward walk begins
        }
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    __syncthreads();
    long long *part = reinterpret_cast<long long *>(emo_smem + p.off_stage0);
    if (!producer) {
        long long *pd = part + ((size_t)(group * lanes + chain) * 32 + lane) * 2;
        pd[0] = __double_as_longlong(ea);
        pd[1] = acc;
    }
    __syncthreads();
    if (!producer && chain == 0) {
        const long long *g0 = part + ((size_t)(group * lanes) * 32 + lane) * 2;
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
    }
}

// ---------------------------------------------------------------------------------------------------
// Backward pass: latest starts and slack.  Walks every stream from its last entry to its first, in
// segments like the forward pass; a run here is a stretch of simple entries (emo_flow.h) handled by
// straight-line code, one instantiation per length.  EXTRA = false is the lean instantiation (slack only).
// ---------------------------------------------------------------------------------------------------
template <bool EXTRA, int MAXT, bool PROF>
__global__ void __launch_bounds__(MAXT, 1) emo_flow_bwd(FlowParams p)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, K = p.K, nbuf = p.nbuf, ptile = p.ptile;
    const int n_cons = groups * lanes;
    const bool producer = warp >= n_cons;
    const int group = producer ? 0 : warp / lanes;
    const int chain = warp - group * lanes;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 32 + lane;
    const int64_t b = b0 + col;
    const bool act = !producer && b < p.B;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + p.off_bar;
    volatile int *abort_word = reinterpret_cast<volatile int *>(emo_smem + p.off_bar + 16 * kFlowMaxBuf);
    const unsigned stage0 = smem0 + p.off_stage0;
    emo_flow_init(p, smem0, emo_smem, n_cons);

    long long ssum = 0;
    int ncrit = 0;
    if (producer) {
        emo_flow_produce<true>(p, stage0, bar0, abort_word, lane, warp - n_cons);
    } else {
        const unsigned slot_lane = smem0 + (unsigned)group * p.slot_bytes + (unsigned)lane * 4u;
        const unsigned slot_base = smem0 + (unsigned)group * p.slot_bytes;
        const unsigned lane4 = (unsigned)lane * 4u, slot_lane4 = slot_lane;
        const unsigned lmask = (unsigned)p.Lp - 1u, tab_row = p.tab_row;
        const int gthreads = lanes * 32;
        const long long limit = p.wait_cycles;
        const long long T = act ? p.makespan[b] : 0;
        const unsigned ldo8 = (unsigned)p.ldo * 8u;
        const unsigned ptile4 = (unsigned)ptile * 4u;
        long long *const sl_lane = (p.slack && act) ? reinterpret_cast<long long *>(p.slack) + b : nullptr;
        const unsigned sl_ok = sl_lane != nullptr;
        long long *const es_lane = (EXTRA && p.ES && act) ? reinterpret_cast<long long *>(p.ES) + b : nullptr;
        long long *const ls_lane = (EXTRA && p.LS && act) ? reinterpret_cast<long long *>(p.LS) + b : nullptr;
        const bool want_sums = EXTRA && (p.slack_sum || p.n_critical) && act;
        unsigned q = 0;
        unsigned c = p.restore[((size_t)blockIdx.x * p.restore_rows + p.pushes + chain) * ptile + col];
        bool dead = false, leave = false;
        long long t_wait = 0, t_bar = 0;
        const long long t_begin = EMO_CLK();
        unsigned rec_a = 0, tab_a = 0, lvl_a = 0, xes_a = 0, pop_a = 0, tok = 0;
        long long t_spec = 0, t_run = 0;
        bool has_in = false, has_out = false;

        // what every entry does once the maximum over its successors (qin) is known
        auto finish = [&](unsigned qin, unsigned dd, unsigned row, unsigned a_lo, unsigned a_hi, unsigned xes_at) {
            // slack_v = T - (lbQ_v + lbES_v) - (qin_v + co_v)
            const long long A = (long long)((unsigned long long)a_lo | ((unsigned long long)a_hi << 32));
            const long long sl = (T - A) - (long long)((unsigned long long)qin + (unsigned long long)c);
            if (sl_lane) *emo_row_ptr(sl_lane, row, ldo8) = sl;
            if (EXTRA) {
                const long long es = emo_tld_s64(xes_at, tok) + (long long)(c - dd);
                if (es_lane) *emo_row_ptr(es_lane, row, ldo8) = es;
                if (ls_lane) *emo_row_ptr(ls_lane, row, ldo8) = sl + es;
                if (want_sums) {
                    ssum += sl;
                    ncrit += (sl == 0);
                }
            }
        };
        // R simple entries of one kind at positions o .. o + R - 1 of the run (lowest first in memory, walked
        // from the highest down).  Straight-line code without a branch (the kind is a compile-time parameter,
        // stores and the restore pop are predicated), so that the look-ups, the record loads and the slack
        // arithmetic of all R entries overlap and only the two running values form a chain.
        auto run = [&](auto rc, auto inc, auto outc, unsigned o) {
            constexpr int R = decltype(rc)::value;
            constexpr bool IN = decltype(inc)::value, OUT = decltype(outc)::value;
            const unsigned rec_o = rec_a + 64u * o, tab_o = tab_a + o * tab_row, lvl_o = lvl_a + 32u * o, xes_o = xes_a + 8u * o;
            unsigned lv[R], d[R];
#pragma unroll
            for (int j = 0; j < R; ++j) lv[j] = emo_tld_u8(lvl_o + 32u * j, tok);
#pragma unroll
            for (int j = 0; j < R; ++j) d[j] = emo_tld_u32(tab_o + (unsigned)j * tab_row + (lv[j] & lmask) * 4u, tok);
#pragma unroll
            for (int j = R - 1; j >= 0; --j) {
                const uint4 r0j = emo_tld_128(rec_o + 64u * j, tok);
                const uint4 r1j = emo_tld_128(rec_o + 64u * j + 16u, tok);
                unsigned qin = emo_floor_sub(q, r1j.w);
                if (IN) {
                    const unsigned a = slot_lane + r0j.w;
                    qin = max(qin, emo_lds_u32v(a));
                    emo_sts_u32v(a, 0u);
                }
                if (EXTRA) {
                    finish(qin, d[j], r1j.z, r1j.x, r1j.y, xes_o + 8u * j);
                } else {
                    // slack_v = T - (lbQ_v + lbES_v) - (qin_v + co_v)
                    const long long A = (long long)((unsigned long long)r1j.x | ((unsigned long long)r1j.y << 32));
                    const long long sl = (T - A) - (long long)((unsigned long long)qin + (unsigned long long)c);
                    emo_stg_s64_if(sl_lane, r1j.z, ldo8, sl, sl_ok);
                }
                q = qin + d[j];
                if (OUT) emo_red_max_u32(slot_lane + r0j.y, emo_floor_sub(q, r0j.z));
                const unsigned pops = r0j.x & emo::kB_Pop;
                pop_a -= pops ? ptile4 : 0u;
                c = emo_tld_u32_if(pop_a, tok, pops, c - d[j]);
            }
        };
        auto run_kind = [&](auto rc, unsigned o) {
            if (has_in) {
                if (has_out) run(rc, std::true_type{}, std::true_type{}, o);
                else run(rc, std::true_type{}, std::false_type{}, o);
            } else {
                if (has_out) run(rc, std::false_type{}, std::true_type{}, o);
                else run(rc, std::false_type{}, std::false_type{}, o);
            }
        };

        for (int cst = 0; cst < p.stages && !leave; ++cst) {
            const int s = cst % nbuf;
            const long long tw0 = EMO_CLK();
            if (!dead && !emo_flow_wait(bar0 + 8 * s, (cst / nbuf) & 1, abort_word, limit)) {
                dead = true;
                *abort_word = 1;
            }
            t_wait += EMO_CLK() - tw0;
            const unsigned sta = stage0 + (unsigned)s * p.stage_bytes;
            const unsigned tok0 = emo_token((unsigned)cst);
            uint4 hd0 = make_uint4(0, 0, 0, 0), hd1 = hd0;
            if (!dead) {
                hd0 = emo_tld_128(sta + (unsigned)chain * 32u, tok0);
                hd1 = emo_tld_128(sta + (unsigned)chain * 32u + 16u, tok0);
            }
            hd0.x = emo_uniform(hd0.x);
            const unsigned total = (hd0.x >> 16) & 255u;
            const unsigned seg_a = sta + p.off_seg + (unsigned)chain * emo::kSegBytes;
            // one past the lane's last entry of this stage; every segment steps down before it reads
            rec_a = sta + p.off_rec + ((unsigned)(chain * K) + total) * 64u;
            tab_a = sta + p.off_tab + ((unsigned)(chain * K) + total) * tab_row;
            lvl_a = sta + p.off_lvl + (((unsigned)((group * lanes + chain) * K) + total) << 5) + (unsigned)lane;
            xes_a = sta + p.off_lbes + ((unsigned)(chain * K) + total) * 8u;
            const unsigned pool_a = sta + p.off_pool;
            pop_a = sta + p.off_rst + ((hd1.y + hd1.x) * (unsigned)ptile + (unsigned)col) * 4u;
            const int nseg = (int)((hd0.x >> 8) & 255u);
            unsigned segw = 0;
            tok = tok0;
            for (int sgi = 0; sgi < nseg || dead; ++sgi) {
                if (dead) {
                    // a wait ran out: the group's next barrier tells every warp of the group to leave
                    if (lanes > 1) (void)emo_group_barrier_or(group + 1, gthreads, true);
                    leave = true;
                    break;
                }
                if ((sgi & 3) == 0) segw = emo_uniform(emo_tld_u32(seg_a + (unsigned)sgi, tok0));
                const unsigned sg = segw & 255u;
                segw >>= 8;
                if (sg & emo::kSegBarrier) {
                    const long long tb0 = EMO_CLK();
                    if (lanes > 1 && emo_group_barrier_or(group + 1, gthreads, false)) { leave = true; break; }
                    t_bar += EMO_CLK() - tb0;
                }
                tok = emo_token(tok + 1u);
                const int r = (int)(sg & emo::kSegRunMask);
                const long long ts0 = EMO_CLK();
                if (sg & emo::kSegSpecial) {
                    // an entry that needs its record: any operands, any kind of output.  Up to two operands
                    // and every kind of output run without a branch.
                    rec_a -= 64u;
                    tab_a -= tab_row;
                    lvl_a -= 32u;
                    xes_a -= 8u;
                    const uint4 r0 = emo_tld_128(rec_a, tok);
                    const uint4 r1 = emo_tld_128(rec_a + 16u, tok);
                    const uint4 r2 = emo_tld_128(rec_a + 32u, tok);
                    const uint4 r3 = emo_tld_128(rec_a + 48u, tok);
                    const unsigned lb = emo_tld_u8(lvl_a, tok);
                    const unsigned fl = r0.x;
                    const unsigned dd = emo_tld_u32(tab_a + (lb & lmask) * 4u, tok);
                    const unsigned nops = fl >> emo::kB_NopsShift;
                    unsigned qin = emo_floor_sub((fl & emo::kB_HasReg) ? q : 0u, r1.w);
                    unsigned x0, t0, a0, x1, t1, a1;
                    emo_flow_operand_u(slot_lane4, lane4, r2.x, nops, x0, t0, a0);
                    emo_flow_operand_u(slot_lane4, lane4, r3.x, nops > 1u, x1, t1, a1);
                    const bool retry0 = nops != 0u && (r2.x & (emo::kOpWord | emo::kOpNoPoll)) == 0u && t0 != r2.y;
                    const bool retry1 = nops > 1u && (r3.x & (emo::kOpWord | emo::kOpNoPoll)) == 0u && t1 != r3.y;
                    if (__any_sync(0xFFFFFFFFu, retry0 || retry1 || nops > 2u)) {
                        // the rest: values that were not there yet, further operands
                        if (retry0 && !emo_flow_poll(a0, r2.y, x0, abort_word, limit)) dead = true;
                        if (retry1 && !emo_flow_poll(a1, r3.y, x1, abort_word, limit)) dead = true;
                        if (dead) *abort_word = 1;      // the other waits of the block end early
                        unsigned pa = pool_a + r0.w * 4u;
                        for (unsigned k = 2; k < nops; ++k) {
                            const unsigned x2 = emo_flow_operand(slot_base, lane, emo_tld_u32(pa, tok), emo_tld_u32(pa + 4u, tok), dead,
                                                                 abort_word, limit);
                            qin = max(qin, emo_floor_sub(x2, emo_tld_u32(pa + 8u, tok)));
                            pa += 12u;
                        }
                        dead = __any_sync(0xFFFFFFFFu, dead);
                        if (dead) continue;      // on to the group's next barrier
                    }
                    qin = max(qin, max(emo_floor_sub(x0, r2.z), emo_floor_sub(x1, r3.z)));
                    if (EXTRA) {
                        finish(qin, dd, r1.z, r1.x, r1.y, xes_a);
                    } else {
                        const long long A = (long long)((unsigned long long)r1.x | ((unsigned long long)r1.y << 32));
                        const long long sl = (T - A) - (long long)((unsigned long long)qin + (unsigned long long)c);
                        emo_stg_s64_if(sl_lane, r1.z, ldo8, sl, sl_ok);
                    }
                    q = qin + dd;
                    emo_flow_out_u(slot_lane4, lane4, q, r0.y, r0.z, fl & emo::kB_OutTag, fl & emo::kB_OutSet, fl & emo::kB_OutAcc);
                    const unsigned pops = fl & emo::kB_Pop;
                    pop_a -= pops ? ptile4 : 0u;
                    c = emo_tld_u32_if(pop_a, tok, pops, c - dd);
                }
                const long long ts1 = EMO_CLK();
                t_spec += ts1 - ts0;
                // the run below it, from its highest position down
                rec_a -= (unsigned)r * 64u;
                tab_a -= (unsigned)r * tab_row;
                lvl_a -= (unsigned)r * 32u;
                xes_a -= (unsigned)r * 8u;
                has_in = (sg & emo::kSegIn) != 0;
                has_out = (sg & emo::kSegOut) != 0;
                {
                    // the run in pieces of 4, 2 and 1 entries, from its highest position down
                    unsigned rem = (unsigned)r;
                    while (rem >= 4u) {
                        rem -= 4u;
                        run_kind(std::integral_constant<int, 4>{}, rem);
                    }
                    if (rem >= 2u) {
                        rem -= 2u;
                        run_kind(std::integral_constant<int, 2>{}, rem);
                    }
                    if (rem) run_kind(std::integral_constant<int, 1>{}, 0u);
                }
                t_run += EMO_CLK() - ts1;
            }
            if (leave) break;
            asm volatile("" ::"r"(q), "r"(c) : "memory");
            __syncwarp();
            if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kFlowMaxBuf + s));
        }
        if (p.prof && lane == 0 && blockIdx.x < 512) {
            long long *pr = p.prof + ((size_t)blockIdx.x * 32 + warp) * 8;
            pr[0] = t_wait;
            pr[1] = t_bar;
            pr[2] = EMO_CLK() - t_begin;
            pr[3] = t_spec;
            pr[4] = t_run;
        }
        if (leave && lane == 0) {
            *abort_word = 1;
            if (p.status) atomicMin(p.status, -8);
        }
    }

    if (EXTRA) {
        __syncthreads();
        long long *part = reinterpret_cast<long long *>(emo_smem + p.off_stage0);
        if (!producer) {
            long long *pd = part + ((size_t)(group * lanes + chain) * 32 + lane) * 2;
            pd[0] = ssum;
            pd[1] = (long long)ncrit;
        }
        __syncthreads();
        if (!producer && chain == 0 && act) {
            const long long *g0 = part + ((size_t)(group * lanes) * 32 + lane) * 2;
            long long s2 = 0, cnt = 0;
            for (int k = 0; k < lanes; ++k) {
                s2 += g0[(size_t)k * 64];
                cnt += g0[(size_t)k * 64 + 1];
            }
            if (p.slack_sum) p.slack_sum[b] = s2;
            if (p.n_critical) p.n_critical[b] = (int32_t)cnt;
        }
    }
}

#undef EMO_CLK
