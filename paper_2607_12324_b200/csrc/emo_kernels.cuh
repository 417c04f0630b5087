// CUDA kernels of the evaluator (sm_100a).  Included only by emo_lib.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "emo_compile.h"

// One pass (forward or backward) over the step program.
//
// Device layout of a program: an array of fixed-size records, one per (step, lane) in schedule
// order.  A record is the 32-byte entry, the node's duration row (Lp x uint32) and, in the forward
// program, its energy row (Lp x fp64).  `rows` holds, per record, the policy row whose level the
// entry reads (kNone: none).
//
// Earliest start times travel from the forward to the backward pass in one of two layouts: `ES`,
// [n][ldes] in the caller's numbering (also the caller-visible ES output), or `spill`, laid out
// [policy tile][row of the backward program][spill_ptile] so that the backward pass streams the
// rows of a run of steps with one contiguous copy.
//
// Columns: policies 0..B-1 come from the level matrix; when want_base is set, column B is a
// virtual policy with every row at level L-1 (the default, maximum-frequency policy P_0 of Alg. 2),
// whose makespan and energy go to base_T / base_E.
struct PassParams {
    const unsigned char *rec;  // records
    const uint32_t *rows;      // [steps*lanes]
    int rec_bytes;             // 32 + Lp*4 (+ Lp*8 forward)
    int steps, lanes, Lp, L, slots, groups;
    int sync;                  // staged kernels: the warps of a group meet every `sync` steps
    int want_base;
    int64_t B;
    const uint8_t *lvl;       // [rows][ldb]
    int64_t ldb;
    int64_t *ES;              // forward: written when not NULL; backward (plain kernel): read
    int64_t ldes;
    int64_t *spill;           // staged kernels: forward writes, backward reads
    int64_t spill_rows;       // rows of the backward program (steps * lanes)
    int spill_ptile;          // policies per tile of the spill
    int64_t *LS, *slack;      // backward outputs, optional
    int64_t ldo;
    int64_t *makespan;        // forward: written; backward: read
    double *energy;
    int64_t *slack_sum;
    int32_t *n_critical;
    int64_t *base_T;
    double *base_E;
    int32_t *status;
};

// T0 + floor(T0 * ppm / 10^6) without a 128-bit product: with T0 = q*10^6 + r the quotient is
// q*ppm + floor(r*ppm / 10^6), and r*ppm stays far below 2^63.
__host__ __device__ inline int64_t emo_budget(int64_t T0, int64_t ppm)
{
    const int64_t M = 1000000;
    int64_t q = T0 / M, r = T0 % M;
    return T0 + q * ppm + (r * ppm) / M;
}

// Alg. 1: "f <- F_i where start in [T_i, T_{i+1})".  Index of the interval that holds `start` among I change
// points brk[0] = 0 < brk[1] < ... (the last interval has no end); iend = where that interval ends.  A first
// guess from the mean interval length, one correction without a branch (exact on a uniform grid, delta > 0),
// then a search for whatever is left (uneven change points).
template <bool UNIFORM>
__device__ __forceinline__ int emo_interval_index(long long start, int I, long long delta, float inv_mean, const long long *brk,
                                                  long long &iend)
{
    int i = (int)((float)start * inv_mean);
    i = i < 0 ? 0 : (i > I - 1 ? I - 1 : i);
    iend = 0x7FFFFFFFFFFFFFFFLL;
    if (UNIFORM) {
        const long long r = start - (long long)i * delta;
        i += (r >= delta && i + 1 < I) ? 1 : 0;
        i -= (r < 0) ? 1 : 0;
        if (i + 1 < I) iend = (long long)(i + 1) * delta;
    } else {
        const long long lo = brk[i], hi = brk[i + 1 < I ? i + 1 : i];
        i += (i + 1 < I && hi <= start) ? 1 : 0;
        i -= (lo > start) ? 1 : 0;
        while (i + 1 < I && brk[i + 1] <= start) ++i;
        while (i > 0 && brk[i] > start) --i;
        if (i + 1 < I) iend = brk[i + 1];
    }
    return i;
}
// A pack's overlap with every interval it touches, added to busy[(row * I + i) * ldw + b]; nearly always one.
__device__ __forceinline__ void emo_interval_busy(unsigned long long *busy, int64_t ldw, int64_t b, unsigned row, int I, int i,
                                                  long long iend, long long start, long long end, const long long *brk)
{
    if (end <= iend) {
        if (end > start) atomicAdd(busy + ((size_t)row * I + i) * ldw + b, (unsigned long long)(end - start));
    } else {
        long long a = start;
        int j = i;
        while (a < end) {
            const long long hi = (j + 1 < I) ? brk[j + 1] : end;
            const long long z = hi < end ? hi : end;
            atomicAdd(busy + ((size_t)row * I + j) * ldw + b, (unsigned long long)(z - a));
            a = z;
            ++j;
        }
    }
}

__device__ __forceinline__ void emo_group_barrier(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Pass kernel, plain loads (used when the caller's pitches or pointers rule out bulk copies).
// One warp = 32 policies of one schedule lane; `lanes` warps form a group and meet at a named
// barrier after every step.  Forward (BWD = false): Eq. 1 with the value C_v kept in h; makespan
// over terminal nodes (equal to the maximum over all nodes because durations are >= 0), energy
// accumulated per warp in step order and combined in lane order.  Backward: the same recurrence on
// the reversed graph gives Q_v = t_v + max over successors of Q_u, so LS_v = T - Q_v and
// slack_v = LS_v - ES_v.
// ------------------------------------------------------------------------------------------------
template <bool BWD>
__global__ void __launch_bounds__(1024) emo_pass_plain(PassParams p)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int group = warp / p.lanes;
    const int chain = warp - group * p.lanes;
    const int64_t b = ((int64_t)blockIdx.x * p.groups + group) * 32 + lane;
    const bool active = b < p.B;
    const bool is_base = !BWD && p.want_base && b == p.B;
    long long *slots = reinterpret_cast<long long *>(emo_smem) + (size_t)group * p.slots * 32 + lane;
    unsigned char *part_base = emo_smem + (size_t)p.groups * p.slots * 256;

    long long h = 0;
    double eacc = 0.0;
    long long tmax = 0, ssum = 0;
    int ncrit = 0;
    const long long T = (BWD && active) ? p.makespan[b] : 0;
    for (int t = 0; t < p.steps; ++t) {
        const size_t q = (size_t)t * p.lanes + chain;
        const unsigned char *r = p.rec + q * p.rec_bytes;
        uint4 e = __ldg(reinterpret_cast<const uint4 *>(r));
        e.x = __ldg(reinterpret_cast<const unsigned *>(r + 16));      // the plain kernel addresses by node id
        if (e.y & emo::kValid) {
            unsigned lv = 0;
            const uint32_t row = __ldg(p.rows + q);
            if (row != emo::kNone && active) lv = p.lvl[(size_t)row * p.ldb + b];
            if (is_base) lv = (unsigned)(p.L - 1);
            lv &= (e.y >> emo::kMaskShift) & 255u;
            const long long dur = (long long)__ldg(reinterpret_cast<const uint32_t *>(r + 32) + lv);
            long long start = (e.y & emo::kRegPred) ? h : 0;
            const int np = (e.y >> emo::kNPredShift) & 7;
            unsigned long long ops = (unsigned long long)e.z | ((unsigned long long)e.w << 32);
            for (int k = 0; k < np; ++k) {
                long long x = slots[(unsigned)(ops & 255u) * 32];
                ops >>= 8;
                start = x > start ? x : start;
            }
            h = start + dur;
            if (!BWD) {
                eacc += __ldg(reinterpret_cast<const double *>(r + 32 + p.Lp * 4) + lv);
                if (e.y & emo::kTerminal) tmax = h > tmax ? h : tmax;
                if (p.ES && e.x != emo::kNone && active) p.ES[(size_t)e.x * p.ldes + b] = start;
            } else if (e.x != emo::kNone && active) {
                const long long ls = T - h;
                const long long es = p.ES[(size_t)e.x * p.ldes + b];
                const long long sl = ls - es;
                if (p.LS) p.LS[(size_t)e.x * p.ldo + b] = ls;
                if (p.slack) p.slack[(size_t)e.x * p.ldo + b] = sl;
                ssum += sl;
                ncrit += (sl == 0);
            }
            if (e.y & emo::kWriteSlot) slots[((e.y >> emo::kOutShift) & 255u) * 32] = h;
        }
        if (p.lanes > 1) emo_group_barrier(group + 1, p.lanes * 32);
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    double *pd = reinterpret_cast<double *>(part_base) + ((size_t)(group * p.lanes + chain) * 32 + lane) * 2;
    if (!BWD) {
        pd[0] = eacc;
        reinterpret_cast<long long *>(pd)[1] = tmax;
    } else {
        reinterpret_cast<long long *>(pd)[0] = ssum;
        reinterpret_cast<long long *>(pd)[1] = (long long)ncrit;
    }
    __syncthreads();
    if (chain == 0 && (active || is_base)) {
        const double *g0 = reinterpret_cast<const double *>(part_base) + ((size_t)(group * p.lanes) * 32 + lane) * 2;
        if (!BWD) {
            double es = 0.0;
            long long tm = 0;
            for (int k = 0; k < p.lanes; ++k) {
                es += g0[(size_t)k * 64];
                long long x = reinterpret_cast<const long long *>(g0)[(size_t)k * 64 + 1];
                tm = x > tm ? x : tm;
            }
            if (is_base) {
                if (p.base_T) *p.base_T = tm;
                if (p.base_E) *p.base_E = es;
            } else {
                p.makespan[b] = tm;
                p.energy[b] = es;
            }
        } else {
            long long ss = 0, nc = 0;
            for (int k = 0; k < p.lanes; ++k) {
                ss += reinterpret_cast<const long long *>(g0)[(size_t)k * 64];
                nc += reinterpret_cast<const long long *>(g0)[(size_t)k * 64 + 1];
            }
            if (p.slack_sum) p.slack_sum[b] = ss;
            if (p.n_critical) p.n_critical[b] = (int32_t)nc;
        }
    }
}

// Every level must be < L; the first offender sets *status to EMO_E_RANGE (-3).
__global__ void emo_validate_levels(const uint8_t *lvl, int64_t ldb, int64_t rows, int64_t B, int L, int32_t *status)
{
    const int64_t total = rows * B;
    bool bad = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / B, b = i - r * B;
        bad |= lvl[r * ldb + b] >= L;
    }
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicMin(status, -3);
}

// ------------------------------------------------------------------------------------------------
// Constrained arg-min (Eq. 4 over a finite batch): least energy among makespan <= target, equal
// energies to the lower index.  Stage 1 leaves one candidate per block, stage 2 finishes.
// ------------------------------------------------------------------------------------------------
struct SelectPartial {
    double e;
    long long idx;
};
constexpr int kSelectMaxBlocks = 1024;

__device__ __forceinline__ bool emo_better(double e1, long long i1, double e2, long long i2)
{
    // (e1, i1) beats (e2, i2); idx < 0 means "no candidate"
    if (i1 < 0) return false;
    if (i2 < 0) return true;
    return e1 < e2 || (e1 == e2 && i1 < i2);
}

__device__ __forceinline__ void emo_select_reduce(double &e, long long &idx, SelectPartial *sh)
{
    for (int off = 16; off > 0; off >>= 1) {
        double e2 = __shfl_down_sync(0xFFFFFFFFu, e, off);
        long long i2 = __shfl_down_sync(0xFFFFFFFFu, idx, off);
        if (emo_better(e2, i2, e, idx)) { e = e2; idx = i2; }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sh[warp].e = e; sh[warp].idx = idx; }
    __syncthreads();
    if (warp == 0) {
        const int nw = blockDim.x >> 5;
        e = lane < nw ? sh[lane].e : 0.0;
        idx = lane < nw ? sh[lane].idx : -1;
        for (int off = 16; off > 0; off >>= 1) {
            double e2 = __shfl_down_sync(0xFFFFFFFFu, e, off);
            long long i2 = __shfl_down_sync(0xFFFFFFFFu, idx, off);
            if (emo_better(e2, i2, e, idx)) { e = e2; idx = i2; }
        }
    }
}

__global__ void emo_select_stage1(int64_t B, const int64_t *makespan, const double *energy, int64_t target,
                                  const int64_t *target_dev, int64_t delta_ppm, SelectPartial *part)
{
    __shared__ SelectPartial sh[32];
    if (target_dev) target = emo_budget(target_dev[0], delta_ppm);
    double e = 0.0;
    long long idx = -1;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < B; b += (int64_t)gridDim.x * blockDim.x) {
        if (makespan[b] <= target) {
            const double x = energy[b];
            if (emo_better(x, b, e, idx)) { e = x; idx = b; }
        }
    }
    emo_select_reduce(e, idx, sh);
    if (threadIdx.x == 0) { part[blockIdx.x].e = e; part[blockIdx.x].idx = idx; }
}

__global__ void emo_select_stage2(int nparts, const SelectPartial *part, const int64_t *makespan,
                                  int64_t *out_index, int64_t *out_T, double *out_E)
{
    __shared__ SelectPartial sh[32];
    double e = 0.0;
    long long idx = -1;
    for (int i = threadIdx.x; i < nparts; i += blockDim.x) {
        if (emo_better(part[i].e, part[i].idx, e, idx)) { e = part[i].e; idx = part[i].idx; }
    }
    emo_select_reduce(e, idx, sh);
    if (threadIdx.x == 0) {
        *out_index = idx;
        if (out_T) *out_T = idx >= 0 ? makespan[idx] : 0;
        if (out_E) *out_E = idx >= 0 ? e : 0.0;
    }
}

// src [B][lds] -> dst [rows][ldb], 32x32 byte tiles through shared memory.
__global__ void emo_transpose_u8(int64_t B, int64_t rows, const uint8_t *src, int64_t lds, uint8_t *dst, int64_t ldb)
{
    __shared__ uint8_t tile[32][33];
    const int64_t r0 = (int64_t)blockIdx.x * 32;
    for (int64_t b0 = (int64_t)blockIdx.y * 32; b0 < B; b0 += (int64_t)gridDim.y * 32) {
        for (int j = threadIdx.y; j < 32; j += blockDim.y) {
            const int64_t b = b0 + j, r = r0 + threadIdx.x;
            if (b < B && r < rows) tile[j][threadIdx.x] = src[b * lds + r];
        }
        __syncthreads();
        for (int j = threadIdx.y; j < 32; j += blockDim.y) {
            const int64_t r = r0 + j, b = b0 + threadIdx.x;
            if (r < rows && b < B) dst[r * ldb + b] = tile[threadIdx.x][j];
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// What one warp alone pays, in cycles (clock64 around a loop, thread 0 reports): the pass kernels walk
// a dependency chain of tens of thousands of steps with a handful of warps per scheduler, so their
// speed is set by these latencies and not by a pipe's throughput.
//   0 dependent 32-bit add                      1 dependent max followed by subtract (one correction)
//   2 dependent shared-memory load              3 independent adds (issue interval)
//   4 loop body: shared load, four dependent operations, and a never-taken branch on the loaded word
//   5 the same body without the branch           6 redux.sync followed by an add (dependent)
//   7 named barrier of all warps of the block (run with five warps)
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ unsigned emo_cost_rare(unsigned a)
{
    for (int i = 0; i < 64; ++i) a = a * 3u + 1u;
    return a;
}
__global__ void emo_warp_costs(long long *out, const unsigned *zeros, int iters, unsigned seed)
{
    __shared__ unsigned s[1024];
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) s[i] = ((unsigned)i + 32u) & 1023u;
    __syncthreads();
    const bool warp0 = threadIdx.x < 32;
    long long t[8];
    unsigned keep = 0;
    if (warp0) {
        {
            unsigned a = seed;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 32; ++j) asm volatile("add.u32 %0, %0, %1;" : "+r"(a) : "r"(seed));
            t[0] = (clock64() - t0) / 32;
            keep ^= a;
        }
        {
            unsigned a = seed;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    asm volatile("max.u32 %0, %0, %1;" : "+r"(a) : "r"(seed + (unsigned)j));
                    asm volatile("sub.u32 %0, %0, %1;" : "+r"(a) : "r"(seed));
                }
            t[1] = (clock64() - t0) / 32;
            keep ^= a;
        }
        {
            unsigned q = threadIdx.x;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 32; ++j) q = *(volatile unsigned *)&s[q];
            t[2] = (clock64() - t0) / 32;
            keep ^= q;
        }
        {
            unsigned a[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) a[k] = seed + (unsigned)k;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int k = 0; k < 8; ++k) asm volatile("add.u32 %0, %0, %1;" : "+r"(a[k]) : "r"(seed));
            t[3] = (clock64() - t0) / 32;
#pragma unroll
            for (int k = 0; k < 8; ++k) keep ^= a[k];
        }
        for (int mode = 0; mode < 2; ++mode) {
            unsigned a = threadIdx.x, b = seed | 1u;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const unsigned f = *(volatile unsigned *)&s[(zeros[0] + (unsigned)(i + j)) & 1023u] >> 12;    // always 0
                    a = max(a, b) - b;
                    a += (unsigned)j;
                    a ^= 5u;
                    a += b;
                    if (mode == 0 && (f & 1u)) a = emo_cost_rare(a);
                    asm volatile("" : "+r"(a));
                }
            t[4 + mode] = (clock64() - t0) / 8;
            keep ^= a;
        }
        {
            unsigned a = threadIdx.x;
            const long long t0 = clock64();
            for (int i = 0; i < iters; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    asm volatile("redux.sync.or.b32 %0, %0, 0xffffffff;" : "+r"(a));
                    asm volatile("add.u32 %0, %0, 1;" : "+r"(a));
                }
            t[6] = (clock64() - t0) / 8;
            keep ^= a;
        }
    }
    {
        __syncthreads();
        const long long t0 = clock64();
        for (int i = 0; i < iters; ++i) asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");
        t[7] = clock64() - t0;
    }
    if (threadIdx.x == 0) {
        for (int k = 0; k < 8; ++k) out[k] = t[k];
        if (keep == 0x12345u) out[8] = keep;      // keeps the chains alive, (almost) never true
    }
}

// ------------------------------------------------------------------------------------------------
// Integer issue rate: eight independent dependent-chains per thread of one operation (OP 0: 32-bit
// add, 1: 32-bit max, 2: 64-bit add, 3: 64-bit max), enough warps to fill every SM.  The operations
// are volatile so that the compiler keeps every one of them.  Gives the denominator for "integer
// issue against peak": the forward and backward recurrences are one add per node and one max per edge.
// ------------------------------------------------------------------------------------------------
template <int OP>
__global__ void __launch_bounds__(256) emo_int_chains(unsigned long long *sink, int iters, unsigned seed)
{
    const unsigned tid = blockIdx.x * blockDim.x + threadIdx.x;
    if (OP < 2) {
        unsigned a[8], b = seed | 1u;
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = tid * 8u + (unsigned)k;
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (OP == 0) asm volatile("add.u32 %0, %0, %1;" : "+r"(a[k]) : "r"(b));
                    else asm volatile("max.u32 %0, %0, %1;" : "+r"(a[k]) : "r"(b + (unsigned)i));
                }
        }
        unsigned x = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) x ^= a[k];
        if (x == 0x12345u) sink[0] = x;      // keeps the chains alive, (almost) never true
    } else {
        unsigned long long a[8], b = ((unsigned long long)seed << 13) | 1ull;
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = (unsigned long long)tid * 8ull + (unsigned long long)k;
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (OP == 2) asm volatile("add.u64 %0, %0, %1;" : "+l"(a[k]) : "l"(b));
                    else asm volatile("max.s64 %0, %0, %1;" : "+l"(a[k]) : "l"(b + (unsigned long long)i));
                }
        }
        unsigned long long x = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) x ^= a[k];
        if (x == 0x12345ull) sink[0] = x;
    }
}

// ------------------------------------------------------------------------------------------------
// Levels packed at `bits` bits each (a frequency level needs ceil(log2 L) bits): eight levels of a row
// take `bits` consecutive bytes, lowest level in the lowest bits.  One thread converts one group of
// eight; rows of the byte matrix are 8-byte aligned.  PACK: bytes -> bits, else bits -> bytes.
// ------------------------------------------------------------------------------------------------
template <bool PACK>
__global__ void emo_repack_levels(int bits, int64_t rows, int64_t groups, uint8_t *packed, int64_t ldp, uint8_t *bytes, int64_t ldb)
{
    const unsigned long long mask = (1ull << bits) - 1ull;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * groups; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / groups, c = i - r * groups;
        uint8_t *pk = packed + r * ldp + c * bits;
        unsigned long long *by = reinterpret_cast<unsigned long long *>(bytes + r * ldb + c * 8);
        if (PACK) {
            const unsigned long long v = *by;
            unsigned long long w = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) w |= ((v >> (8 * k)) & mask) << (k * bits);
            for (int k = 0; k < bits; ++k) pk[k] = (uint8_t)(w >> (8 * k));
        } else {
            unsigned long long w = 0;
            for (int k = 0; k < bits; ++k) w |= (unsigned long long)pk[k] << (8 * k);
            unsigned long long v = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) v |= ((w >> (k * bits)) & mask) << (8 * k);
            *by = v;
        }
    }
}
