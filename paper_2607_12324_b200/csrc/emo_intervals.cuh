// Time-interval policies (Alg. 1): the level of a pack is the one of the interval that holds its start
// time, so the look-up depends on the recurrence and cannot be staged ahead of it.  Included only by
// emo_lib.cu.
#pragma once
#include "emo_kernels.cuh"

struct IntervalParams {
    PassParams p;              // the forward step program, the batch size, makespan / energy outputs (lvl unused)
    const uint8_t *F;          // [rows][I][ldb] levels
    int64_t ldb;
    int I;
    const int64_t *breaks;     // device, [I] change points, breaks[0] = 0
    float inv_mean;            // (I - 1) / breaks[I-1]: gives the first guess of the interval index
    long long delta;           // > 0: the change points are the uniform grid i * delta
    unsigned long long *busy;  // [rows][I][ldw] summed overlap of the row's packs with each interval (NULL: not wanted)
    int64_t ldw;
    unsigned slot_bytes;       // shared memory: slots and partial sums first, the change points after them,
    unsigned off_rec, rec_pad; // then four record buffers per warp (rec_pad bytes each: the record, then its group),
    unsigned off_F;            // then the block's columns of F when they fit (stage_F)
    int stage_F, rows;
};

// Forward pass of Eq. 1 with the level of every pack taken from its start time.  One warp = 32 policies of
// one schedule lane; `lanes` warps form a group and meet at a named barrier after every step (the layout of
// emo_pass_plain).  The look-up chain of a step is start -> interval -> level -> duration, all of it
// dependent, so everything it touches is brought on chip ahead of it: the change points and (when they fit)
// the block's columns of F sit in shared memory, and every warp copies the record of its next step (entry,
// duration row, energy row) into a buffer of its own while it works on the current one.
// Where busy is given, every pack adds its overlap with each interval it touches (integer atomics: the lanes
// of a group work on the same policies).
template <bool UNIFORM, bool STAGED>
__global__ void __launch_bounds__(1024) emo_pass_intervals(IntervalParams ip)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const PassParams &p = ip.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int group = warp / p.lanes;
    const int chain = warp - group * p.lanes;
    const int64_t b = ((int64_t)blockIdx.x * p.groups + group) * 32 + lane;
    const bool active = b < p.B;
    long long *slots = reinterpret_cast<long long *>(emo_smem) + (size_t)group * p.slots * 32 + lane;
    unsigned char *part_base = emo_smem + (size_t)p.groups * p.slots * 256;
    long long *brk = reinterpret_cast<long long *>(emo_smem + ip.slot_bytes);
    const int I = ip.I;
    unsigned char *recbuf = emo_smem + ip.off_rec + (size_t)warp * 4 * ip.rec_pad;      // four records per warp
    unsigned char *Fs = ip.stage_F ? emo_smem + ip.off_F : nullptr;                     // [rows * I][groups * 32]
    const int fcols = p.groups * 32;
    for (int i = threadIdx.x; i < I; i += blockDim.x) brk[i] = ip.breaks[i];
    if (Fs) {
        const int64_t b0 = (int64_t)blockIdx.x * fcols;
        const int total = ip.rows * I * fcols;
        for (int k = threadIdx.x; k < total; k += blockDim.x) {
            const int ri = k / fcols, c = k - ri * fcols;
            Fs[k] = (b0 + c < p.B) ? ip.F[(size_t)ri * ip.ldb + b0 + c] : (unsigned char)0;
        }
    }
    // The record of step t for this warp's lane (and the group it belongs to) is copied into a ring of four
    // buffers three steps ahead of its use with asynchronous copies, 16 bytes per thread: a step costs less
    // than a trip to L2, so one step ahead does not hide it.
    auto request = [&](int t) {
        if (t < p.steps) {
            const size_t q = (size_t)t * p.lanes + chain;
            const unsigned char *r = p.rec + q * p.rec_bytes;
            unsigned char *dst = recbuf + (size_t)(t & 3) * ip.rec_pad;
            for (int o = lane * 16; o < p.rec_bytes; o += 512)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(emo_smem_addr(dst + o)), "l"(r + o) : "memory");
            if (lane == 0)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(emo_smem_addr(dst + ip.rec_pad - 16)), "l"(p.rows + q) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    request(0);
    request(1);
    request(2);
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    __syncthreads();

    long long h = 0;
    double eacc = 0.0;
    long long tmax = 0;
    for (int t = 0; t < p.steps; ++t) {
        const unsigned char *r = recbuf + (size_t)(t & 3) * ip.rec_pad;
        request(t + 3);
        const uint32_t row = *reinterpret_cast<const uint32_t *>(r + ip.rec_pad - 16);
        const uint4 e = *reinterpret_cast<const uint4 *>(r);
        {
            // One straight run of instructions for every entry, idle steps included (their record is all zero: no
            // operands, zero duration and energy, no output; only the lane's value must survive them): a branch on
            // a freshly loaded word costs a lone warp far more than the few predicated instructions it would skip.
            const unsigned valid = e.y & emo::kValid;
            long long start = (e.y & emo::kRegPred) ? h : 0;
            const int np = (e.y >> emo::kNPredShift) & 7;
            unsigned long long ops = (unsigned long long)e.z | ((unsigned long long)e.w << 32);
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const long long x = slots[(unsigned)(ops & 255u) * 32];      // byte 0 where there is no operand: slot 0, ignored
                ops >>= 8;
                start = (k < np && x > start) ? x : start;
            }
            if (np > 3) {
                for (int k = 3; k < np; ++k) {
                    const long long x = slots[(unsigned)(ops & 255u) * 32];
                    ops >>= 8;
                    start = x > start ? x : start;
                }
            }
            // f <- F_i where start in [T_i, T_{i+1}); a node outside every policy reads row 0 and masks the level away
            const bool pack = row != emo::kNone;
            const unsigned rowc = pack ? row : 0u;
            long long iend;
            const int i = emo_interval_index<UNIFORM>(start, I, ip.delta, ip.inv_mean, brk, iend);
            unsigned lv;
            if (STAGED) lv = Fs[((size_t)rowc * I + i) * fcols + group * 32 + lane];
            else lv = active ? ip.F[((size_t)rowc * I + i) * ip.ldb + b] : 0u;
            lv &= (e.y >> emo::kMaskShift) & 255u;
            const long long dur = (long long)*(reinterpret_cast<const uint32_t *>(r + 32) + lv);
            const long long end = start + dur;
            h = valid ? end : h;
            eacc += *(reinterpret_cast<const double *>(r + 32 + p.Lp * 4) + lv);
            tmax = ((e.y & emo::kTerminal) && end > tmax) ? end : tmax;
            if (ip.busy) {
                // the pack's overlap with the intervals it touches: nearly always one
                const bool on = pack && active;
                if (on && end <= iend && dur) atomicAdd(ip.busy + ((size_t)rowc * I + i) * ip.ldw + b, (unsigned long long)dur);
                if (on && end > iend) emo_interval_busy(ip.busy, ip.ldw, b, rowc, I, i, iend, start, end, brk);
            }
            if (e.y & emo::kWriteSlot) slots[((e.y >> emo::kOutShift) & 255u) * 32] = end;
        }
        // the copy of the next step's record has landed; the barrier makes it visible to the whole warp
        asm volatile("cp.async.wait_group 2;" ::: "memory");
        if (p.lanes > 1) emo_group_barrier(group + 1, p.lanes * 32);
        else __syncwarp();
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    double *pd = reinterpret_cast<double *>(part_base) + ((size_t)(group * p.lanes + chain) * 32 + lane) * 2;
    pd[0] = eacc;
    reinterpret_cast<long long *>(pd)[1] = tmax;
    __syncthreads();
    if (chain == 0 && active) {
        const double *g0 = reinterpret_cast<const double *>(part_base) + ((size_t)(group * p.lanes) * 32 + lane) * 2;
        double es = 0.0;
        long long tm = 0;
        for (int k = 0; k < p.lanes; ++k) {
            es += g0[(size_t)k * 64];
            long long x = reinterpret_cast<const long long *>(g0)[(size_t)k * 64 + 1];
            tm = x > tm ? x : tm;
        }
        p.makespan[b] = tm;
        p.energy[b] = es;
    }
}

// E_i of Alg. 1: for every row (device) and interval, the interval's length below the makespan minus the
// busy time, not below zero, times the idle power of the interval's level; rows, then intervals, in order.
// One thread per policy.  Adds the idle energy to energy[b] and, if asked, stores it alone.
__global__ void __launch_bounds__(256) emo_idle_energy(int64_t B, int rows, int I, const int64_t *breaks, const uint8_t *F, int64_t ldb,
                                                       const unsigned long long *busy, int64_t ldw, const double *p_idle, int L,
                                                       const int64_t *makespan, double *energy, double *energy_idle)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const long long T = makespan[b];
    double sum = 0.0, comp = 0.0;      // compensated: many small terms
    for (int r = 0; r < rows; ++r)
        for (int i = 0; i < I; ++i) {
            const long long lo = breaks[i];
            long long hi = (i + 1 < I) ? breaks[i + 1] : T;
            hi = hi < T ? hi : T;
            const long long len = hi > lo ? hi - lo : 0;
            const long long bz = (long long)busy[((size_t)r * I + i) * ldw + b];
            const long long idle = len > bz ? len - bz : 0;
            unsigned f = F[((size_t)r * I + i) * ldb + b];
            f = f < (unsigned)L ? f : (unsigned)(L - 1);
            const double x = (double)idle * 1e-9 * p_idle[f];
            const double t = sum + x;
            comp += (fabs(sum) >= fabs(x)) ? (sum - t) + x : (x - t) + sum;
            sum = t;
        }
    const double ei = sum + comp;
    if (energy_idle) energy_idle[b] = ei;
    energy[b] += ei;
}
