// Exact path for graphs that the schedule compilers cannot hold on chip (more simultaneously live exchanged
// values than there are slots): one thread per policy walks the nodes in index order (a topological numbering)
// with the completion times of all nodes in global memory, [n][ldw], so that the threads of a warp read and
// write consecutive words.  No cooperation between threads, no limits other than memory.  Eq. 1, Eq. 2 forward;
// the mirrored recurrence backward.  Included only by emo_lib.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

struct GenericParams {
    int n, L;
    const int64_t *row_ptr;    // predecessor CSR
    const int32_t *col;
    const int64_t *srow_ptr;   // successor CSR
    const int32_t *scol;
    const int32_t *group;      // policy row of every node, -1: none (level 0)
    const int64_t *lat;        // [n][L]
    const double *energy;      // [n][L]
    int64_t B;
    int want_base;             // forward: column B is the all-(L-1) policy
    const uint8_t *lvl;
    int64_t ldb;
    int64_t *C, *Q;            // [n][ldw] completion times / tails
    int64_t ldw;
    int64_t *ES, *LS, *slack;
    int64_t ldo;
    int64_t *makespan;
    double *energy_out;
    int64_t *slack_sum;
    int32_t *n_critical;
    int64_t *base_T;
    double *base_E;
};

__device__ __forceinline__ int emo_generic_level(const GenericParams &p, int v, int64_t b, bool is_base)
{
    const int row = p.group[v];
    if (row < 0) return 0;
    int lv = is_base ? p.L - 1 : (int)p.lvl[(size_t)row * p.ldb + b];
    return lv < p.L ? lv : p.L - 1;      // never read outside the table
}

__global__ void __launch_bounds__(128) emo_generic_fwd(GenericParams p)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool is_base = p.want_base && b == p.B;
    if (b >= p.B && !is_base) return;
    long long T = 0;
    double e = 0.0;
    for (int v = 0; v < p.n; ++v) {
        long long start = 0;
        for (int64_t k = p.row_ptr[v]; k < p.row_ptr[v + 1]; ++k) {
            const long long c = p.C[(size_t)p.col[k] * p.ldw + b];
            start = c > start ? c : start;
        }
        const int lv = emo_generic_level(p, v, b, is_base);
        const long long c = start + p.lat[(size_t)v * p.L + lv];
        e += p.energy[(size_t)v * p.L + lv];
        p.C[(size_t)v * p.ldw + b] = c;
        T = c > T ? c : T;
        if (p.ES && !is_base) p.ES[(size_t)v * p.ldo + b] = start;
    }
    if (is_base) {
        if (p.base_T) *p.base_T = T;
        if (p.base_E) *p.base_E = e;
    } else {
        p.makespan[b] = T;
        p.energy_out[b] = e;
    }
}

__global__ void __launch_bounds__(128) emo_generic_bwd(GenericParams p)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.B) return;
    const long long T = p.makespan[b];
    long long ssum = 0;
    int ncrit = 0;
    for (int v = p.n - 1; v >= 0; --v) {
        long long qin = 0;
        for (int64_t k = p.srow_ptr[v]; k < p.srow_ptr[v + 1]; ++k) {
            const long long q = p.Q[(size_t)p.scol[k] * p.ldw + b];
            qin = q > qin ? q : qin;
        }
        const int lv = emo_generic_level(p, v, b, false);
        const long long dur = p.lat[(size_t)v * p.L + lv];
        const long long q = qin + dur;
        p.Q[(size_t)v * p.ldw + b] = q;
        const long long ls = T - q;
        const long long es = p.C[(size_t)v * p.ldw + b] - dur;
        const long long sl = ls - es;
        if (p.LS) p.LS[(size_t)v * p.ldo + b] = ls;
        if (p.slack) p.slack[(size_t)v * p.ldo + b] = sl;
        ssum += sl;
        ncrit += (sl == 0);
    }
    if (p.slack_sum) p.slack_sum[b] = ssum;
    if (p.n_critical) p.n_critical[b] = ncrit;
}
