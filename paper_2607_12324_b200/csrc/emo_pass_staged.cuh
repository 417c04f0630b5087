// What the staged pass kernels share (PTX helpers, stage parameters, the producer emo_produce) and the
// staged pass kernel with two policies per thread, emo_pass_pair (sm_100a).
//
// A staged kernel is the step interpreter with everything a step reads brought into shared memory
// by producer warps with bulk asynchronous copies (TMA, cp.async.bulk) through a
// ring of stages guarded by full/empty mbarriers: the program records (entry + duration row +
// energy row) of a run of steps in one bulk copy, (backward) the earliest-start rows of those steps
// in a second bulk copy, and the level rows of the block's policy tile, which lie scattered in the
// caller's matrix, as 16-byte cp.async pieces issued by all lanes of the producer warps (a bulk copy
// per 128-byte row costs far more than it moves).  Each record and each level row is fetched once
// per block and used by every policy of the block.
//
// In emo_pass_pair a consumer thread carries TWO adjacent policies, so a warp covers 64 policies of one schedule
// lane: the entry decode and the address arithmetic are paid once per pair, the level pair is one
// 16-bit load, an exchange slot holds both values and moves with one 128-bit access, and the
// per-node outputs leave as 128-bit stores.
//
// The warps of a group do not run in lockstep.  Each walks its own column of the step program and
// waits only for the values it reads: every exchange slot has an mbarrier whose phase completes
// when the slot's next value has been written, and the entry names the phase parity to wait for.
// The group meets at a named barrier every `sync` steps, which bounds the drift between its
// warps; the host compiler reuses a slot only across such a barrier.  Included only by emo_lib.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "emo_compile.h"
#include "emo_kernels.cuh"

constexpr int kMaxStages = 8;
constexpr int kMaxBulk = 5;              // bulk copies per stage
constexpr int kRowRegs = 8;             // a stage holds at most 32 * kRowRegs records
constexpr int kProducerWarps = 2;       // warps that issue the copies (they share the level-row pieces)
constexpr unsigned kSlotStride = 528;   // 8-byte mbarrier, 8 bytes unused, 32 lanes x 16 bytes
constexpr long long kWaitCycles = 4000000000LL;   // about two seconds: a wait that long has failed
constexpr unsigned kSpinPolls = 1u << 14;          // polls between two looks at the clock

struct StagedParams {
    PassParams p;
    int sc;                    // steps per stage (a power of two, like the distance between group barriers)
    int stages;                // ring depth
    int ptile;                 // policies per block = 64 * groups
    int vec_es, vec_out;       // 128-bit global accesses allowed for ES / for LS and slack
    int want_sums;             // backward: accumulate slack sums and critical counts
    unsigned stage_bytes;      // bytes of one stage
    unsigned off_lvl, off_es;  // offsets inside a stage (records start at 0)
    unsigned off_part, off_bar, off_stage0;      // offsets inside dynamic shared memory
    // the bulk copies that fill a stage besides the level rows: per copy its global source, the
    // bytes one program entry takes in it, the offset of its area inside a stage and the distance
    // between the sources of consecutive blocks (0: all blocks read the same array)
    int nbulk;
    const unsigned char *bsrc[kMaxBulk];
    unsigned bentry[kMaxBulk], boff[kMaxBulk];
    unsigned long long bblock[kMaxBulk];
};

__device__ __forceinline__ unsigned emo_smem_addr(const void *p)
{
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void emo_mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void emo_mbar_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void emo_mbar_arrive(unsigned bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void emo_mbar_arrive_if(unsigned bar, bool cond)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar), "r"((unsigned)cond)
                 : "memory");
}
__device__ __forceinline__ bool emo_mbar_try(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitCycles and reports false (the caller raises EMO_E_TIMEOUT).
__device__ __noinline__ bool emo_mbar_wait_slow(unsigned bar, unsigned parity)
{
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < (1u << 12); ++i) {
            if (emo_mbar_try(bar, parity)) return true;
            __nanosleep(100);      // a waiting warp must not take issue slots from the warps that work
        }
        if (clock64() - t0 > kWaitCycles) return false;
    }
}
__device__ __forceinline__ bool emo_mbar_wait(unsigned bar, unsigned parity)
{
    if (emo_mbar_try(bar, parity)) return true;
    return emo_mbar_wait_slow(bar, parity);
}
// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void emo_bulk_g2s(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// 16-byte asynchronous copy global -> shared, and the arrival that reports a thread's copies done
__device__ __forceinline__ void emo_cp_async16(unsigned dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void emo_cp_async_arrive(unsigned bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// shared-memory accesses by 32-bit address
__device__ __forceinline__ uint4 emo_lds128(unsigned a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ unsigned emo_lds_u16(unsigned a)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ unsigned emo_lds_u32(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ double emo_lds_f64(unsigned a)
{
    double v;
    asm volatile("ld.shared.f64 %0, [%1];" : "=d"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void emo_lds_pair(unsigned a, long long &x0, long long &x1)
{
    asm volatile("ld.shared.v2.s64 {%0, %1}, [%2];" : "=l"(x0), "=l"(x1) : "r"(a));
}
__device__ __forceinline__ void emo_sts_pair(unsigned a, long long x0, long long x1)
{
    asm volatile("st.shared.v2.s64 [%0], {%1, %2};" ::"r"(a), "l"(x0), "l"(x1) : "memory");
}
__device__ __forceinline__ void emo_stg_pair(long long *p, long long x0, long long x1)
{
    asm volatile("st.global.v2.s64 [%0], {%1, %2};" ::"l"(p), "l"(x0), "l"(x1) : "memory");
}
__device__ __forceinline__ long long emo_max64(long long a, long long b) { return a > b ? a : b; }
// h + d with d an unsigned 32-bit duration: one wide multiply-add
__device__ __forceinline__ long long emo_add_dur(long long h, unsigned d)
{
    long long r;
    asm("mad.wide.u32 %0, %1, 1, %2;" : "=l"(r) : "r"(d), "l"(h));
    return r;
}

// What a step needs from its stage, independent of the recurrence; fetched one step ahead of its use.
struct EmoFetched {
    uint4 e;
    unsigned node;
    unsigned d0, d1;
    double g0, g1;
    long long es0, es1;
};
template <bool BWD>
__device__ __forceinline__ void emo_fetch(EmoFetched &x, unsigned rec_a, unsigned lvl_a, unsigned es_a, unsigned en_off,
                                          bool want_node)
{
    x.e = emo_lds128(rec_a);
    if (want_node) x.node = emo_lds_u32(rec_a + 16u);
    const unsigned lv2 = emo_lds_u16(lvl_a);
    const unsigned m = (x.e.y >> emo::kMaskShift) & 255u;
    const unsigned l0 = lv2 & m, l1 = (lv2 >> 8) & m;
    x.d0 = emo_lds_u32(rec_a + 32u + l0 * 4u);
    x.d1 = emo_lds_u32(rec_a + 32u + l1 * 4u);
    if (!BWD) {
        x.g0 = emo_lds_f64(rec_a + en_off + l0 * 8u);
        x.g1 = emo_lds_f64(rec_a + en_off + l1 * 8u);
    } else {
        emo_lds_pair(es_a, x.es0, x.es1);
    }
}
// base + row * pitch (bytes) as one wide multiply-add
__device__ __forceinline__ long long *emo_row_ptr(long long *base, unsigned row, unsigned pitch_bytes)
{
    unsigned long long r;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(r) : "r"(row), "r"(pitch_bytes), "l"(reinterpret_cast<unsigned long long>(base)));
    return reinterpret_cast<long long *>(r);
}
__device__ __forceinline__ bool emo_mbar_test(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// four barriers at once: true when every one of them has completed the phase with its parity
__device__ __forceinline__ bool emo_mbar_test4(unsigned b0, unsigned b1, unsigned b2, unsigned b3, unsigned par)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .u32 q0, q1, q2, q3;\n\t"
        "and.b32 q0, %5, 1;\n\tshr.u32 q1, %5, 1;\n\tand.b32 q1, q1, 1;\n\t"
        "shr.u32 q2, %5, 2;\n\tand.b32 q2, q2, 1;\n\tshr.u32 q3, %5, 3;\n\tand.b32 q3, q3, 1;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p0, [%1], q0;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p1, [%2], q1;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p2, [%3], q2;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p3, [%4], q3;\n\t"
        "and.pred p0, p0, p1;\n\tand.pred p2, p2, p3;\n\tand.pred p0, p0, p2;\n\t"
        "selp.u32 %0, 1, 0, p0;\n\t}"
        : "=r"(ok)
        : "r"(b0), "r"(b1), "r"(b2), "r"(b3), "r"(par)
        : "memory");
    return ok != 0;
}
// Wait until the slot's value with the given phase parity has been written.  Bounded; also gives
// up as soon as another warp of the group has raised the abort flag.
__device__ __noinline__ bool emo_slot_wait_slow(unsigned bar, unsigned parity, volatile int *abort_flag)
{
    // the clock is read rarely: reading it on every poll would keep the special-register path busy
    const long long t0 = clock64();
    for (;;) {
        for (unsigned i = 0; i < (1u << 12); ++i) {
            if (emo_mbar_try(bar, parity)) return true;
            __nanosleep(40);       // a waiting warp must not take issue slots from the warps that work
        }
        if (*abort_flag || clock64() - t0 > kWaitCycles) return false;
    }
}
__device__ __forceinline__ bool emo_slot_wait(unsigned bar, unsigned parity, volatile int *abort_flag)
{
    if (emo_mbar_try(bar, parity)) return true;
    return emo_slot_wait_slow(bar, parity, abort_flag);
}

// The producer warp: for every chunk of steps, the bulk copies the launch lists (program records,
// backward: the earliest-start rows) and the level rows of the block's policy tile as 16-byte pieces; then
// the arrivals that complete the stage's full barrier.  Waits for a free stage are bounded: on
// failure the warp raises *abort_all and EMO_E_TIMEOUT and returns once its copies have landed.
__device__ __forceinline__ void emo_produce(const StagedParams &sp, unsigned stage0, unsigned bar0, volatile int *abort_all,
                                            int lane, int pw)
{
    const PassParams &p = sp.p;
    const int steps = p.steps, nstages = sp.stages, sc = sp.sc, lanes = p.lanes, ptile = sp.ptile;
    const int n_chunks = (steps + sc - 1) / sc;
    const unsigned stage_bytes = sp.stage_bytes;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int64_t lvl_left = p.ldb - b0;
    const unsigned lvl_bytes = lvl_left > 0 ? (unsigned)min((int64_t)ptile, lvl_left) : 0u;
    const int pieces = (int)(lvl_bytes >> 4);
    const unsigned inv_pieces = pieces > 1 ? (unsigned)((0x100000000ULL + pieces - 1) / pieces) : 0u;
    int issued = 0;
    bool gave_up = false;
    // The level-row indices of a chunk are loaded one chunk ahead, 32 per register, so that no
    // copy waits on a dependent global load: entry i's row sits in lane i % 32 of rr[i / 32].
    unsigned rr[kRowRegs], rr_next[kRowRegs];
    auto load_rows = [&](int c, unsigned *dst) {
        const int step0 = c * sc;
        const int ne = (c < n_chunks) ? min(sc, steps - step0) * lanes : 0;
        const size_t q0 = (size_t)step0 * lanes;
#pragma unroll
        for (int k = 0; k < kRowRegs; ++k) {
            const int i = 32 * k + lane;
            dst[k] = (i < ne) ? __ldg(p.rows + q0 + i) : emo::kNone;
        }
    };
    load_rows(0, rr);
    for (int c = 0; c < n_chunks; ++c) {
        const int s = c % nstages;
        load_rows(c + 1, rr_next);
        if (c >= nstages) {
            if (!emo_mbar_wait(bar0 + 8 * (kMaxStages + s), ((c / nstages) - 1) & 1)) {
                if (lane == 0) {
                    *abort_all = 1;
                    if (p.status) atomicMin(p.status, -8);
                }
                gave_up = true;
                break;
            }
        }
        if (*abort_all) { gave_up = true; break; }      // the other producer warp gave up
        issued = c + 1;
        const int step0 = c * sc;
        const int ne = min(sc, steps - step0) * lanes;
        const size_t q0 = (size_t)step0 * lanes;
        const unsigned sta = stage0 + (unsigned)s * stage_bytes;
        const unsigned full = bar0 + 8 * s;
        if (lane == 0 && pw == 0) {
            unsigned total = 0;
            for (int i = 0; i < sp.nbulk; ++i) total += (unsigned)ne * sp.bentry[i];
            emo_mbar_expect_tx(full, total);
            for (int i = 0; i < sp.nbulk; ++i)
                emo_bulk_g2s(sta + sp.boff[i], sp.bsrc[i] + blockIdx.x * sp.bblock[i] + q0 * sp.bentry[i],
                             (unsigned)ne * sp.bentry[i], full);
        }
        // level rows: 32 entries x `pieces` 16-byte pieces per register of row indices; the
        // producer warps take alternate iterations
        if (pieces) {
#pragma unroll
            for (int k = 0; k < kRowRegs; ++k) {
                if (32 * k < ne) {
                    for (int it = pw; it < pieces; it += kProducerWarps) {
                        const unsigned t = (unsigned)lane + 32u * (unsigned)it;
                        const unsigned e = pieces > 1 ? __umulhi(t, inv_pieces) : t;   // t / pieces (t < 2^16)
                        const unsigned pc = t - e * (unsigned)pieces;
                        const unsigned row = __shfl_sync(0xFFFFFFFFu, rr[k], e & 31);
                        const int i = 32 * k + (int)e;
                        if (i < ne && row != emo::kNone)
                            emo_cp_async16(sta + sp.off_lvl + (unsigned)i * ptile + pc * 16u,
                                           p.lvl + (size_t)row * p.ldb + b0 + pc * 16);
                    }
                }
            }
        }
        emo_cp_async_arrive(full);
#pragma unroll
        for (int k = 0; k < kRowRegs; ++k) rr[k] = rr_next[k];
    }
    if (gave_up) {
        // do not leave the block while copies into its shared memory may still be in flight
        for (int c = max(0, issued - nstages); c < issued; ++c) (void)emo_mbar_wait(bar0 + 8 * (c % nstages), (c / nstages) & 1);
    }
}

// EXTRA = false is the lean instantiation for the common call (forward: ES only into the spill;
// backward: slack only, 16-byte aligned rows, no per-policy sums): the hot loop stays small, which
// matters because all warps of the block share the instruction cache.
template <bool BWD, bool EXTRA, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) emo_pass_pair(StagedParams sp)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const PassParams &p = sp.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int lanes = p.lanes, groups = p.groups, steps = p.steps, nstages = sp.stages, sc = sp.sc;
    const int n_cons = groups * lanes;                  // consumer warps; the warps after them produce
    const bool producer = warp >= n_cons;
    const int pw = warp - n_cons;                       // producer warp index
    const int group = producer ? 0 : warp / lanes;
    const int chain = warp - group * lanes;
    const int ptile = sp.ptile;
    const int64_t b0 = (int64_t)blockIdx.x * ptile;
    const int col = group * 64 + 2 * lane;
    const int64_t b = b0 + col;
    const bool act0 = !producer && b < p.B, act1 = !producer && b + 1 < p.B;
    // column of the virtual all-max policy inside this block's tile (fwd only), or -1
    const int base_col = (!BWD && p.want_base && p.B >= b0 && p.B < b0 + ptile) ? (int)(p.B - b0) : -1;
    unsigned char *part_base = emo_smem + sp.off_part;
    const unsigned smem0 = emo_smem_addr(emo_smem);
    const unsigned bar0 = smem0 + sp.off_bar;           // full[k] at bar0 + 8k, empty[k] after them
    volatile int *abort_flag = reinterpret_cast<volatile int *>(emo_smem + sp.off_bar + 16 * kMaxStages);
    const unsigned stage0 = smem0 + sp.off_stage0;
    const unsigned stage_bytes = sp.stage_bytes;

    for (int i = threadIdx.x; i < groups * p.slots; i += blockDim.x) emo_mbar_init(smem0 + (unsigned)i * kSlotStride, 1);
    if (threadIdx.x == 0) {
        for (int k = 0; k < nstages; ++k) {
            emo_mbar_init(bar0 + 8 * k, 1 + 32 * kProducerWarps);   // one expect-tx arrival + every producer lane's cp.async arrival
            emo_mbar_init(bar0 + 8 * (kMaxStages + k), n_cons);
        }
        for (int k = 0; k <= groups; ++k) abort_flag[k] = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    const int n_chunks = (steps + sc - 1) / sc;
    long long h0 = 0, h1 = 0;
    double ea0 = 0.0, ea1 = 0.0;
    long long acc0 = 0, acc1 = 0;      // forward: running makespan; backward: slack sums
    int nc0 = 0, nc1 = 0;

    if (producer) {
        emo_produce(sp, stage0, bar0, abort_flag + groups, lane, pw);
    } else {
        // --------------------------------------------------------------------------- consumers
        const unsigned slotbar_base = smem0 + (unsigned)group * p.slots * kSlotStride;
        const unsigned lane16 = 16u + (unsigned)lane * 16u;
        const long long T0 = (BWD && act0) ? p.makespan[b] : 0, T1 = (BWD && act1) ? p.makespan[b + 1] : 0;
        const unsigned d_rec = (unsigned)lanes * p.rec_bytes, d_lvl = (unsigned)lanes * ptile;
        const unsigned en_off = 32u + (unsigned)p.Lp * 4u;
        const unsigned ldes8 = (unsigned)p.ldes * 8u, ldo8 = (unsigned)p.ldo * 8u;     // pitches below 2^28 elements
        long long *const es_lane = (!BWD && p.ES) ? reinterpret_cast<long long *>(p.ES) + b : nullptr;
        // forward: this thread's column pair inside the spill tile it belongs to
        long long *const spill_lane = (!BWD && p.spill)
            ? reinterpret_cast<long long *>(p.spill) + (size_t)(b / p.spill_ptile) * p.spill_rows * p.spill_ptile + (b % p.spill_ptile)
            : nullptr;
        const unsigned spill8 = (unsigned)p.spill_ptile * 8u;
        long long *const ls_lane = p.LS ? reinterpret_cast<long long *>(p.LS) + b : nullptr;
        long long *const sl_lane = p.slack ? reinterpret_cast<long long *>(p.slack) + b : nullptr;
        const bool store_es = EXTRA && es_lane != nullptr && act0, store_spill = spill_lane != nullptr && act0;
        const bool vec_es = sp.vec_es && act1, vec_out = (!EXTRA || sp.vec_out) && act1;
        const bool want_sums = EXTRA && sp.want_sums != 0;
        const int gthreads = lanes * 32;
        volatile int *my_abort = abort_flag + group;
        bool dead = false;

        // one node for both policies of this thread
        auto process = [&](const EmoFetched &f) {
            const uint4 e = f.e;
            if (!(e.y & emo::kValid) || dead) return;
            if (!BWD) {
                ea0 += f.g0;
                ea1 += f.g1;
            }
            if (!(e.y & emo::kRegPred)) { h0 = 0; h1 = 0; }
            const unsigned np = (e.y >> emo::kNPredShift) & 7u;
            if (np && !BWD) {
                // forward programs have few slot operands: a plain loop keeps the code small
                unsigned ops = e.z, par = e.y >> emo::kOperandParityShift;
                for (unsigned k = 0; k < np; ++k) {
                    if (k == 4) ops = e.w;
                    const unsigned bar = slotbar_base + (ops & 255u) * kSlotStride;
                    if (!emo_slot_wait(bar, par & 1u, my_abort)) {
                        *my_abort = 1;
                        dead = true;
                        return;
                    }
                    long long x0, x1;
                    emo_lds_pair(bar + lane16, x0, x1);
                    ops >>= 8;
                    par >>= 1;
                    h0 = emo_max64(h0, x0);
                    h1 = emo_max64(h1, x1);
                }
            }
            if (np && BWD) {
                // all operands at once: poll every slot's barrier, then load every value, then take
                // the maxima - the loads overlap instead of queuing behind one another
                unsigned bars[emo::kMaxSlotPreds];
                bool ready = true;
#pragma unroll
                for (int k = 0; k < emo::kMaxSlotPreds; ++k) {
                    if (k < (int)np) {
                        const unsigned id = ((k < 4 ? e.z : e.w) >> (8 * (k & 3))) & 255u;
                        bars[k] = slotbar_base + id * kSlotStride;
                        ready &= emo_mbar_try(bars[k], (e.y >> (emo::kOperandParityShift + k)) & 1u);
                    }
                }
                if (!ready) {
#pragma unroll
                    for (int k = 0; k < emo::kMaxSlotPreds; ++k) {
                        if (k < (int)np && !dead) {
                            if (!emo_slot_wait(bars[k], (e.y >> (emo::kOperandParityShift + k)) & 1u, my_abort)) {
                                *my_abort = 1;
                                dead = true;
                            }
                        }
                    }
                    if (dead) return;
                }
                long long x0[emo::kMaxSlotPreds], x1[emo::kMaxSlotPreds];
#pragma unroll
                for (int k = 0; k < emo::kMaxSlotPreds; ++k)
                    if (k < (int)np) emo_lds_pair(bars[k] + lane16, x0[k], x1[k]);
#pragma unroll
                for (int k = 0; k < emo::kMaxSlotPreds; ++k) {
                    if (k < (int)np) {
                        h0 = emo_max64(h0, x0[k]);
                        h1 = emo_max64(h1, x1[k]);
                    }
                }
            }
            // here h is the node's start (forward: ES_v; backward: the longest tail behind v)
            if (!BWD && e.x != emo::kNone) {
                if (store_spill) {
                    long long *dst = emo_row_ptr(spill_lane, e.x, spill8);     // 16-byte aligned by construction
                    if (act1) {
                        emo_stg_pair(dst, h0, h1);
                    } else {
                        dst[0] = h0;
                    }
                }
                if (EXTRA && store_es) {
                    long long *dst = emo_row_ptr(es_lane, f.node, ldes8);
                    if (vec_es) {
                        emo_stg_pair(dst, h0, h1);
                    } else {
                        dst[0] = h0;
                        if (act1) dst[1] = h1;
                    }
                }
            }
            h0 = emo_add_dur(h0, f.d0);
            h1 = emo_add_dur(h1, f.d1);
            if (e.y & emo::kWriteSlot) {
                const unsigned bar = slotbar_base + ((e.y >> emo::kOutShift) & 255u) * kSlotStride;
                emo_sts_pair(bar + lane16, h0, h1);
                __syncwarp();
                if (lane == 0) emo_mbar_arrive(bar);
            }
            if (!BWD) {
                if (e.y & emo::kTerminal) {
                    acc0 = emo_max64(acc0, h0);
                    acc1 = emo_max64(acc1, h1);
                }
            } else if (e.x != emo::kNone && act0) {
                const long long ls0 = T0 - h0, ls1 = T1 - h1;
                const long long s0 = ls0 - f.es0, s1 = ls1 - f.es1;
                if (EXTRA && ls_lane) {
                    long long *dst = emo_row_ptr(ls_lane, e.x, ldo8);
                    if (vec_out) {
                        emo_stg_pair(dst, ls0, ls1);
                    } else {
                        dst[0] = ls0;
                        if (act1) dst[1] = ls1;
                    }
                }
                if (sl_lane) {
                    long long *dst = emo_row_ptr(sl_lane, e.x, ldo8);
                    if (vec_out) {
                        emo_stg_pair(dst, s0, s1);
                    } else {
                        dst[0] = s0;
                        if (act1) dst[1] = s1;
                    }
                }
                if (want_sums) {
                    acc0 += s0;
                    acc1 += s1;
                    nc0 += (s0 == 0);
                    nc1 += (s1 == 0);
                }
            }
        };

        for (int c = 0; c < n_chunks; ++c) {
            const int s = c % nstages;
            const bool ok = emo_mbar_wait(bar0 + 8 * s, (c / nstages) & 1);
            // the warps of a group must take the same decision: one flag, read after a barrier
            if (!ok || dead || (chain == 0 && abort_flag[groups])) *my_abort = 1;
            const unsigned sta = stage0 + (unsigned)s * stage_bytes;
            const int ns = min(sc, steps - c * sc);
            if (base_col >= 0 && chain == 0 && (base_col >> 6) == group) {
                // the virtual all-max column: overwrite its byte in every level row of this stage
                const unsigned char top = (unsigned char)(p.L - 1);
                for (int i = lane; i < ns * lanes; i += 32)
                    emo_smem[sp.off_stage0 + (size_t)s * stage_bytes + sp.off_lvl + (size_t)i * ptile + (size_t)base_col] = top;
                __syncwarp();
            }
            if (lanes > 1) emo_group_barrier(group + 1, gthreads);
            if (*my_abort) {
                if (lane == 0 && p.status) atomicMin(p.status, -8);
                break;
            }
            unsigned rec_a = sta + (unsigned)chain * p.rec_bytes;
            unsigned lvl_a = sta + sp.off_lvl + (unsigned)chain * ptile + col;
            unsigned es_a = sta + sp.off_es + ((unsigned)chain * ptile + col) * 8u;
            // everything a step reads from the stage is fetched one step ahead (one copy of the step
            // body: a small hot loop matters more than the few register moves)
            const unsigned d_es = d_lvl * 8u;
            EmoFetched cur, nxt;
            emo_fetch<BWD>(cur, rec_a, lvl_a, es_a, en_off, store_es);
            int j = 0;
            while (j < ns) {
                if (j && (j % p.sync) == 0 && lanes > 1) emo_group_barrier(group + 1, gthreads);
                if (!EXTRA && !BWD && (cur.e.y & emo::kSimple) && !dead) {
                    // a run of simple nodes: h += duration, nothing else to decide
                    // (a stage may end before the run does: the rest of it starts the next stage)
                    const int run = min((int)((cur.e.y >> emo::kRunShift) & 15u), ns - j);
                    const unsigned m = (cur.e.y >> emo::kMaskShift) & 255u;
                    for (int k = 0; k < run; ++k) {
                        const unsigned row = emo_lds_u32(rec_a);
                        const unsigned lv2 = emo_lds_u16(lvl_a);
                        const unsigned l0 = lv2 & m, l1 = (lv2 >> 8) & m;
                        const unsigned d0 = emo_lds_u32(rec_a + 32u + l0 * 4u), d1 = emo_lds_u32(rec_a + 32u + l1 * 4u);
                        if (!BWD) {
                            const double g0 = emo_lds_f64(rec_a + en_off + l0 * 8u), g1 = emo_lds_f64(rec_a + en_off + l1 * 8u);
                            if (store_spill) {
                                long long *dst = emo_row_ptr(spill_lane, row, spill8);
                                if (act1) {
                                    emo_stg_pair(dst, h0, h1);
                                } else {
                                    dst[0] = h0;
                                }
                            }
                            ea0 += g0;
                            ea1 += g1;
                            h0 = emo_add_dur(h0, d0);
                            h1 = emo_add_dur(h1, d1);
                        } else {
                            long long es0, es1;
                            emo_lds_pair(es_a, es0, es1);
                            h0 = emo_add_dur(h0, d0);
                            h1 = emo_add_dur(h1, d1);
                            if (act0 && sl_lane) {
                                long long *dst = emo_row_ptr(sl_lane, row, ldo8);
                                const long long s0 = T0 - h0 - es0, s1 = T1 - h1 - es1;
                                if (act1) {
                                    emo_stg_pair(dst, s0, s1);
                                } else {
                                    dst[0] = s0;
                                }
                            }
                        }
                        rec_a += d_rec;
                        lvl_a += d_lvl;
                        es_a += d_es;
                    }
                    j += run;
                    if (j < ns) emo_fetch<BWD>(cur, rec_a, lvl_a, es_a, en_off, store_es);
                    continue;
                }
                rec_a += d_rec;
                lvl_a += d_lvl;
                es_a += d_es;
                if (j + 1 < ns) emo_fetch<BWD>(nxt, rec_a, lvl_a, es_a, en_off, store_es);
                process(cur);
                cur = nxt;
                ++j;
            }
            __syncwarp();
            if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kMaxStages + s));
        }
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    // per (group, chain, lane): {energy0 | sum0, energy1 | sum1, makespan0 | count0, makespan1 | count1}
    if (!producer) {
        long long *pd = reinterpret_cast<long long *>(part_base) + ((size_t)(group * lanes + chain) * 32 + lane) * 4;
        if (!BWD) {
            pd[0] = __double_as_longlong(ea0);
            pd[1] = __double_as_longlong(ea1);
            pd[2] = acc0;
            pd[3] = acc1;
        } else {
            pd[0] = acc0;
            pd[1] = acc1;
            pd[2] = nc0;
            pd[3] = nc1;
        }
    }
    __syncthreads();
    if (!producer && chain == 0) {
        const long long *g0 = reinterpret_cast<const long long *>(part_base) + ((size_t)(group * lanes) * 32 + lane) * 4;
        if (!BWD) {
            double e0 = 0.0, e1 = 0.0;
            long long t0 = 0, t1 = 0;
            for (int k = 0; k < lanes; ++k) {
                e0 += __longlong_as_double(g0[(size_t)k * 128]);
                e1 += __longlong_as_double(g0[(size_t)k * 128 + 1]);
                t0 = emo_max64(t0, g0[(size_t)k * 128 + 2]);
                t1 = emo_max64(t1, g0[(size_t)k * 128 + 3]);
            }
            if (act0) { p.makespan[b] = t0; p.energy[b] = e0; }
            if (act1) { p.makespan[b + 1] = t1; p.energy[b + 1] = e1; }
            if (base_col == col) { if (p.base_T) *p.base_T = t0; if (p.base_E) *p.base_E = e0; }
            if (base_col == col + 1) { if (p.base_T) *p.base_T = t1; if (p.base_E) *p.base_E = e1; }
        } else if (sp.want_sums) {
            long long s0 = 0, s1 = 0, c0 = 0, c1 = 0;
            for (int k = 0; k < lanes; ++k) {
                s0 += g0[(size_t)k * 128];
                s1 += g0[(size_t)k * 128 + 1];
                c0 += g0[(size_t)k * 128 + 2];
                c1 += g0[(size_t)k * 128 + 3];
            }
            if (act0) { if (p.slack_sum) p.slack_sum[b] = s0; if (p.n_critical) p.n_critical[b] = (int32_t)c0; }
            if (act1) { if (p.slack_sum) p.slack_sum[b + 1] = s1; if (p.n_critical) p.n_critical[b + 1] = (int32_t)c1; }
        }
    }
}
