// Staged pass kernel (sm_100a): the same step interpreter as emo_pass_plain, but everything a step
// reads - program entries, the schedule-ordered duration and energy tables, the level rows of the
// block's policy tile and (backward) the earliest-start rows - is brought into shared memory by one
// producer warp with bulk asynchronous copies (TMA, cp.async.bulk) through a ring of stages guarded
// by full/empty mbarriers.  Each table chunk and each level row is fetched once per block and used
// by every policy of the block.  Included only by emo_lib.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "emo_compile.h"
#include "emo_kernels.cuh"

constexpr int kStages = 3;
constexpr long long kWaitCycles = 4000000000LL;   // about two seconds: a wait that long has failed

struct StagedParams {
    PassParams p;
    int sc;                    // steps per stage
    int ptile;                 // policies per block = 32 * groups
    unsigned stage_bytes;      // bytes of one stage
    unsigned off_lat, off_en, off_lvl, off_es;   // offsets inside a stage
    unsigned off_part, off_bar, off_stage0;      // offsets inside dynamic shared memory
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
__device__ __forceinline__ bool emo_mbar_wait(unsigned bar, unsigned parity)
{
    if (emo_mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (!emo_mbar_try(bar, parity)) {
        if (clock64() - t0 > kWaitCycles) return false;
    }
    return true;
}
// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void emo_bulk_g2s(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

template <bool BWD>
__global__ void __launch_bounds__(1024) emo_pass_staged(StagedParams sp)
{
    extern __shared__ __align__(128) unsigned char emo_smem[];
    const PassParams &p = sp.p;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int n_cons = p.groups * p.lanes;              // consumer warps; warp n_cons is the producer
    const bool producer = warp == n_cons;
    const int group = producer ? 0 : warp / p.lanes;
    const int chain = warp - group * p.lanes;
    const int64_t b0 = (int64_t)blockIdx.x * sp.ptile;
    const int64_t b = b0 + group * 32 + lane;
    const bool active = !producer && b < p.B;
    unsigned char *part_base = emo_smem + sp.off_part;
    const unsigned bar0 = emo_smem_addr(emo_smem + sp.off_bar);        // full[k] at bar0 + 8k, empty[k] after
    volatile int *abort_flag = reinterpret_cast<volatile int *>(emo_smem + sp.off_bar + 16 * kStages);
    unsigned char *stage0 = emo_smem + sp.off_stage0;

    if (threadIdx.x == 0) {
        for (int k = 0; k < kStages; ++k) {
            emo_mbar_init(bar0 + 8 * k, 1);
            emo_mbar_init(bar0 + 8 * (kStages + k), n_cons);
        }
        for (int k = 0; k <= p.groups; ++k) abort_flag[k] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int n_chunks = (p.steps + sp.sc - 1) / sp.sc;
    long long h = 0;
    double eacc = 0.0;
    long long tmax = 0, ssum = 0;
    int ncrit = 0;

    if (producer) {
        // ---------------------------------------------------------------------------- producer
        const unsigned lvl_bytes = (unsigned)min((int64_t)sp.ptile, p.ldb - b0);
        const unsigned es_bytes = BWD ? (unsigned)min((int64_t)sp.ptile, p.ldes - b0) * 8u : 0u;
        int issued = 0;
        bool gave_up = false;
        for (int c = 0; c < n_chunks; ++c) {
            const int s = c % kStages;
            if (c >= kStages) {
                if (!emo_mbar_wait(bar0 + 8 * (kStages + s), ((c / kStages) - 1) & 1)) {
                    if (lane == 0) {
                        abort_flag[p.groups] = 1;
                        if (p.status) atomicMin(p.status, -8);
                    }
                    gave_up = true;
                    break;
                }
            }
            issued = c + 1;
            const int step0 = c * sp.sc;
            const int ne = min(sp.sc, p.steps - step0) * p.lanes;
            const size_t q0 = (size_t)step0 * p.lanes;
            unsigned bytes = 0;
            for (int i = lane; i < ne; i += 32) {
                const uint4 e = __ldg(p.prog + q0 + i);
                if (e.z & emo::kValid) {
                    if (e.x != emo::kNone) bytes += lvl_bytes;
                    if (BWD && e.y != emo::kNone) bytes += es_bytes;
                }
            }
            for (int off = 16; off > 0; off >>= 1) bytes += __shfl_xor_sync(0xFFFFFFFFu, bytes, off);
            unsigned char *st = stage0 + (size_t)s * sp.stage_bytes;
            const unsigned sta = emo_smem_addr(st);
            const unsigned full = bar0 + 8 * s;
            if (lane == 0) {
                const unsigned fixed = (unsigned)ne * 16u + (unsigned)ne * p.Lp * 4u + (BWD ? 0u : (unsigned)ne * p.Lp * 8u);
                emo_mbar_expect_tx(full, bytes + fixed);
                emo_bulk_g2s(sta, p.prog + q0, (unsigned)ne * 16u, full);
                emo_bulk_g2s(sta + sp.off_lat, p.lat + q0 * p.Lp, (unsigned)ne * p.Lp * 4u, full);
                if (!BWD) emo_bulk_g2s(sta + sp.off_en, p.en + q0 * p.Lp, (unsigned)ne * p.Lp * 8u, full);
            }
            __syncwarp();
            for (int i = lane; i < ne; i += 32) {
                const uint4 e = __ldg(p.prog + q0 + i);
                if (e.z & emo::kValid) {
                    if (e.x != emo::kNone)
                        emo_bulk_g2s(sta + sp.off_lvl + (unsigned)i * sp.ptile, p.lvl + (size_t)e.x * p.ldb + b0, lvl_bytes, full);
                    if (BWD && e.y != emo::kNone)
                        emo_bulk_g2s(sta + sp.off_es + (unsigned)i * sp.ptile * 8u, p.ES + (size_t)e.y * p.ldes + b0, es_bytes, full);
                }
            }
        }
        if (gave_up) {
            // do not leave the block while copies into its shared memory may still be in flight
            for (int c = max(0, issued - kStages); c < issued; ++c) (void)emo_mbar_wait(bar0 + 8 * (c % kStages), (c / kStages) & 1);
        }
    } else {
        // --------------------------------------------------------------------------- consumers
        long long *slots = reinterpret_cast<long long *>(emo_smem) + (size_t)group * p.slots * 32 + lane;
        const long long T = (BWD && active) ? p.makespan[b] : 0;
        const int col = group * 32 + lane;
        bool failed = false;
        for (int c = 0; c < n_chunks && !failed; ++c) {
            const int s = c % kStages;
            const bool ok = emo_mbar_wait(bar0 + 8 * s, (c / kStages) & 1);
            // the warps of a group must take the same decision: one flag, read after a barrier
            if (!ok || (chain == 0 && abort_flag[p.groups])) abort_flag[group] = 1;
            if (p.lanes > 1) emo_group_barrier(group + 1, p.lanes * 32);
            if (abort_flag[group]) {
                if (lane == 0 && p.status) atomicMin(p.status, -8);
                failed = true;
                break;
            }
            const unsigned char *st = stage0 + (size_t)s * sp.stage_bytes;
            const uint4 *s_ent = reinterpret_cast<const uint4 *>(st);
            const uint32_t *s_lat = reinterpret_cast<const uint32_t *>(st + sp.off_lat);
            const double *s_en = reinterpret_cast<const double *>(st + sp.off_en);
            const unsigned char *s_lvl = st + sp.off_lvl;
            const long long *s_es = reinterpret_cast<const long long *>(st + sp.off_es);
            const int ns = min(sp.sc, p.steps - c * sp.sc);
            for (int j = 0; j < ns; ++j) {
                const int i = j * p.lanes + chain;
                const uint4 e = s_ent[i];
                if (e.z & emo::kValid) {
                    unsigned lv = 0;
                    if (e.x != emo::kNone) lv = s_lvl[i * sp.ptile + col];
                    lv &= (unsigned)p.Lmask;
                    const long long dur = (long long)s_lat[i * p.Lp + lv];
                    long long start = (e.z & emo::kRegPred) ? h : 0;
                    const int np = (e.z >> emo::kNPredShift) & 7;
                    unsigned long long ops = (unsigned long long)e.w | ((unsigned long long)(e.z >> 16) << 32);
                    for (int k = 0; k < np; ++k) {
                        long long x = slots[(unsigned)(ops & 255u) * 32];
                        ops >>= 8;
                        start = x > start ? x : start;
                    }
                    h = start + dur;
                    if (!BWD) {
                        eacc += s_en[i * p.Lp + lv];
                        if (e.z & emo::kTerminal) tmax = h > tmax ? h : tmax;
                        if (p.ES && e.y != emo::kNone && active) p.ES[(size_t)e.y * p.ldes + b] = start;
                    } else if (e.y != emo::kNone && active) {
                        const long long ls = T - h;
                        const long long es = s_es[i * sp.ptile + col];
                        const long long sl = ls - es;
                        if (p.LS) p.LS[(size_t)e.y * p.ldo + b] = ls;
                        if (p.slack) p.slack[(size_t)e.y * p.ldo + b] = sl;
                        ssum += sl;
                        ncrit += (sl == 0);
                    }
                    if (e.z & emo::kWriteSlot) slots[((e.z >> emo::kOutShift) & 255u) * 32] = h;
                }
                if (p.lanes > 1) emo_group_barrier(group + 1, p.lanes * 32);
            }
            if (lane == 0) emo_mbar_arrive(bar0 + 8 * (kStages + s));
        }
    }

    // combine the warps of a group in lane order (fixed order: run-to-run identical energy)
    if (!producer) {
        double *pd = reinterpret_cast<double *>(part_base) + ((size_t)(group * p.lanes + chain) * 32 + lane) * 2;
        if (!BWD) {
            pd[0] = eacc;
            reinterpret_cast<long long *>(pd)[1] = tmax;
        } else {
            reinterpret_cast<long long *>(pd)[0] = ssum;
            reinterpret_cast<long long *>(pd)[1] = (long long)ncrit;
        }
    }
    __syncthreads();
    if (!producer && chain == 0 && active) {
        const double *g0 = reinterpret_cast<const double *>(part_base) + ((size_t)(group * p.lanes) * 32 + lane) * 2;
        if (!BWD) {
            double es = 0.0;
            long long tm = 0;
            for (int k = 0; k < p.lanes; ++k) {
                es += g0[(size_t)k * 64];
                long long x = reinterpret_cast<const long long *>(g0)[(size_t)k * 64 + 1];
                tm = x > tm ? x : tm;
            }
            p.makespan[b] = tm;
            p.energy[b] = es;
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
