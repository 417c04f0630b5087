// C-ABI entry points (see include/emo.h) and the CUDA kernels behind them.  sm_100a only.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/emo.h"
#include "emo_compile.h"
#include "emo_kernels.cuh"
#include "emo_pass_staged.cuh"

using namespace emo;

struct DevProgram {
    uint4 *entries = nullptr;
    uint32_t *lat = nullptr;
    double *energy = nullptr;
};

struct emo_graph {
    HostGraph h;
    Program fwd, bwd;
    DevProgram dfwd, dbwd;
    bool host_only = false;
    int device = 0;
    int sm_count = 148;
    size_t smem_optin = 0;
};

namespace {

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
    int rc = upload(&d.entries, p.entries.data(), p.entries.size() * sizeof(uint32_t));
    if (rc) return rc;
    rc = upload(&d.lat, p.lat.data(), p.lat.size() * sizeof(uint32_t));
    if (rc) return rc;
    if (!p.energy.empty()) rc = upload(&d.energy, p.energy.data(), p.energy.size() * sizeof(double));
    return rc;
}

void free_program(DevProgram &d)
{
    if (d.entries) cudaFree(d.entries);
    if (d.lat) cudaFree(d.lat);
    if (d.energy) cudaFree(d.energy);
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
int shape_for(const emo_graph *g, const Program &p, int64_t B, LaunchShape &s)
{
    int64_t n_groups = (B + 31) / 32;
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

// Shape of the staged kernel: groups per block as above (one more warp produces), then as many
// steps per stage as fit beside the slots.  Returns false when the staged kernel cannot be used.
bool staged_shape(const emo_graph *g, const Program &p, bool backward, int64_t B, LaunchShape &s, StagedParams &sp)
{
    if (p.steps == 0 || !g->smem_optin) return false;
    int64_t n_groups = (B + 31) / 32;
    int gmax = std::min(31 / p.lanes, 15);
    if (gmax < 1) return false;
    int64_t want = (n_groups + g->sm_count - 1) / g->sm_count;
    int G = (int)std::max<int64_t>(1, std::min<int64_t>(gmax, want));
    const size_t budget = g->smem_optin;
    for (; G >= 1; --G) {
        const size_t P = 32 * (size_t)G;
        const size_t fixed = (size_t)G * p.slots * 256 + (size_t)G * p.lanes * 512 + 256;
        const size_t per_step = (size_t)p.lanes * (16 + (size_t)p.Lp * 4 + (backward ? 0 : (size_t)p.Lp * 8) + P + (backward ? P * 8 : 0));
        if (fixed + kStages * per_step > budget) continue;
        int sc = (int)std::min<size_t>(16, (budget - fixed) / (kStages * per_step));
        sc = std::min(sc, std::max(1, p.steps));
        const size_t ne = (size_t)sc * p.lanes;
        sp.sc = sc;
        sp.ptile = (int)P;
        sp.off_lat = (unsigned)(ne * 16);
        sp.off_en = sp.off_lat + (unsigned)(ne * p.Lp * 4);
        sp.off_lvl = sp.off_en + (backward ? 0u : (unsigned)(ne * p.Lp * 8));
        sp.off_es = sp.off_lvl + (unsigned)(ne * P);
        sp.stage_bytes = (unsigned)round_up(sp.off_es + (backward ? ne * P * 8 : 0), 128);
        sp.off_part = (unsigned)((size_t)G * p.slots * 256);
        sp.off_bar = sp.off_part + (unsigned)((size_t)G * p.lanes * 512);
        sp.off_stage0 = (unsigned)round_up(sp.off_bar + 256, 128);
        s.groups = G;
        s.grid = (int)((n_groups + G - 1) / G);
        s.threads = (G * p.lanes + 1) * 32;
        s.smem = sp.off_stage0 + (size_t)kStages * sp.stage_bytes;
        if (s.smem > budget) continue;
        return true;
    }
    return false;
}

int launch_pass(const emo_graph *g, bool backward, int64_t B, const uint8_t *lvl, int64_t ldb,
                int64_t *ES, int64_t ldes, int64_t *LS, int64_t *slack, int64_t ldo,
                int64_t *makespan, double *energy, int64_t *slack_sum, int32_t *n_critical,
                int32_t *status, cudaStream_t st, uint32_t flags = 0)
{
    const Program &p = backward ? g->bwd : g->fwd;
    const DevProgram &d = backward ? g->dbwd : g->dfwd;
    LaunchShape s;
    StagedParams sp;
    bool staged = !(flags & EMO_F_NO_STAGING) && ldb % 16 == 0 && ((uintptr_t)lvl % 16) == 0 &&
                  (!backward || (ldes % 2 == 0 && ((uintptr_t)ES % 16) == 0)) &&
                  staged_shape(g, p, backward, B, s, sp);
    if (!staged) {
        int rc = shape_for(g, p, B, s);
        if (rc) return rc;
    }
    PassParams a;
    a.prog = d.entries;
    a.lat = d.lat;
    a.en = d.energy;
    a.steps = p.steps;
    a.lanes = p.lanes;
    a.Lp = p.Lp;
    a.Lmask = p.Lp - 1;
    a.slots = p.slots;
    a.groups = s.groups;
    a.B = B;
    a.lvl = lvl;
    a.ldb = ldb;
    a.ES = ES;
    a.ldes = ldes;
    a.LS = LS;
    a.slack = slack;
    a.ldo = ldo;
    a.makespan = makespan;
    a.energy = energy;
    a.slack_sum = slack_sum;
    a.n_critical = n_critical;
    a.status = status;
    cudaEvent_t ev0 = g_pass_events[backward ? 2 : 0], ev1 = g_pass_events[backward ? 3 : 1];
    if (ev0) EMO_CUDA(cudaEventRecord(ev0, st));
    if (staged) {
        sp.p = a;
        if (backward) {
            EMO_CUDA(cudaFuncSetAttribute(emo_pass_staged<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem));
            emo_pass_staged<true><<<s.grid, s.threads, s.smem, st>>>(sp);
        } else {
            EMO_CUDA(cudaFuncSetAttribute(emo_pass_staged<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem));
            emo_pass_staged<false><<<s.grid, s.threads, s.smem, st>>>(sp);
        }
    } else if (backward) {
        if (s.smem > 48 * 1024) EMO_CUDA(cudaFuncSetAttribute(emo_pass_plain<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem));
        emo_pass_plain<true><<<s.grid, s.threads, s.smem, st>>>(a);
    } else {
        if (s.smem > 48 * 1024) EMO_CUDA(cudaFuncSetAttribute(emo_pass_plain<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s.smem));
        emo_pass_plain<false><<<s.grid, s.threads, s.smem, st>>>(a);
    }
    EMO_CUDA(cudaGetLastError());
    if (ev1) EMO_CUDA(cudaEventRecord(ev1, st));
    return EMO_OK;
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
        case EMO_E_UNSUPPORTED: return "graph needs more exchange slots than supported";
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
        if (n_levels < 0 || level_ptr[0] != 0 || level_ptr[n_levels] != n) return EMO_E_INVALID_ARG;
        std::vector<int32_t> lev((size_t)std::max(n, 1));
        for (int32_t l = 0; l < n_levels; ++l) {
            if (level_ptr[l + 1] < level_ptr[l]) return EMO_E_INVALID_ARG;
            for (int32_t v = level_ptr[l]; v < level_ptr[l + 1]; ++v) lev[v] = l;
        }
        for (int32_t v = 0; v < n; ++v)
            for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e)
                if (lev[col[e]] >= lev[v]) return EMO_E_NOT_TOPOLOGICAL;
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
        int rc = compile_program(h, lat, energy, false, lanes, look, g->fwd, err);
        if (rc == EMO_OK) rc = compile_program(h, lat, energy, true, g->fwd.lanes, look, g->bwd, err);
        if (rc != EMO_OK) { delete g; return rc; }
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
        int rc = upload_program(g->fwd, g->dfwd);
        if (rc == EMO_OK) rc = upload_program(g->bwd, g->dbwd);
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
    info->steps_fwd = g->fwd.steps;
    info->slots_fwd = g->fwd.slots;
    info->aux_fwd = g->fwd.aux;
    info->steps_bwd = g->bwd.steps;
    info->slots_bwd = g->bwd.slots;
    info->aux_bwd = g->bwd.aux;
    return EMO_OK;
}

int emo_graph_program(const emo_graph *g, int dir, int32_t *lanes, int32_t *steps, int32_t *slots,
                      int32_t *Lp, const uint32_t **entries, const uint32_t **lat)
{
    if (!g || (dir != 0 && dir != 1)) return EMO_E_INVALID_ARG;
    const Program &p = dir ? g->bwd : g->fwd;
    if (lanes) *lanes = p.lanes;
    if (steps) *steps = p.steps;
    if (slots) *slots = p.slots;
    if (Lp) *Lp = p.Lp;
    if (entries) *entries = p.entries.data();
    if (lat) *lat = p.lat.data();
    return EMO_OK;
}

int emo_workspace_bytes(const emo_graph *g, int64_t B, int need_slack, size_t *out)
{
    if (!g || !out || B < 0) return EMO_E_INVALID_ARG;
    size_t bytes = kSmallWs + lvl_area(g);
    if (need_slack) bytes += (size_t)g->h.n * round_up((size_t)B, 16) * sizeof(int64_t);
    if (need_slack == 2) bytes += 4 * round_up((size_t)B * 8, 256) + 256;
    *out = bytes;
    return EMO_OK;
}

int emo_eval_policies(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t *makespan,
                      double *energy, void *ws, size_t ws_bytes, int32_t *status, uint32_t flags,
                      void *stream)
{
    if (!g || B < 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (B == 0) return EMO_OK;
    if (!lvl || !makespan || !energy || ldb < B) return EMO_E_INVALID_ARG;
    (void)ws;
    (void)ws_bytes;
    cudaStream_t st = (cudaStream_t)stream;
    if (flags & EMO_F_VALIDATE) {
        int rc = launch_validate(g, B, lvl, ldb, status, st);
        if (rc) return rc;
    }
    return launch_pass(g, false, B, lvl, ldb, nullptr, 0, nullptr, nullptr, 0, makespan, energy, nullptr,
                       nullptr, status, st, flags);
}

int emo_slack_batch(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t *ES,
                    int64_t *LS, int64_t *slack, int64_t ldo, int64_t *makespan, double *energy,
                    int64_t *slack_sum, int32_t *n_critical, void *ws, size_t ws_bytes, int32_t *status,
                    uint32_t flags, void *stream)
{
    if (!g || B < 0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    if (B == 0) return EMO_OK;
    if (!lvl || !makespan || !energy || ldb < B) return EMO_E_INVALID_ARG;
    if ((ES || LS || slack) && ldo < B) return EMO_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int64_t *es = ES;
    int64_t ldes = ldo;
    if (!es) {
        size_t need = 0;
        emo_workspace_bytes(g, B, 1, &need);
        if (!ws || ws_bytes < need) return EMO_E_OOM;
        es = (int64_t *)((char *)ws + kSmallWs + lvl_area(g));
        ldes = (int64_t)round_up((size_t)B, 16);
    }
    if (flags & EMO_F_VALIDATE) {
        int rc = launch_validate(g, B, lvl, ldb, status, st);
        if (rc) return rc;
    }
    int rc = launch_pass(g, false, B, lvl, ldb, es, ldes, nullptr, nullptr, 0, makespan, energy, nullptr,
                         nullptr, status, st, flags);
    if (rc) return rc;
    return launch_pass(g, true, B, lvl, ldb, es, ldes, LS, slack, ldo, makespan, energy, slack_sum,
                       n_critical, status, st, flags);
}

int emo_slack(const emo_graph *g, const uint8_t *lvl_one, int64_t *ES, int64_t *LS, int64_t *slack,
              int64_t *makespan, double *energy, void *ws, size_t ws_bytes, int32_t *status, void *stream)
{
    if (!g || !makespan) return EMO_E_INVALID_ARG;
    size_t need = 0;
    emo_workspace_bytes(g, 1, 1, &need);
    if (!ws || ws_bytes < need) return EMO_E_OOM;
    double *e = energy ? energy : (double *)((char *)ws + 1024);
    return emo_slack_batch(g, 1, lvl_one, 1, ES, LS, slack, 1, makespan, e, nullptr, nullptr, ws, ws_bytes,
                           status, 0, stream);
}

int emo_baseline(const emo_graph *g, int64_t *T0, double *E0, void *ws, size_t ws_bytes, int32_t *status,
                 void *stream)
{
    if (!g || !T0 || !E0) return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    size_t need = 0;
    emo_workspace_bytes(g, 1, 0, &need);
    if (!ws || ws_bytes < need) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *lv = (uint8_t *)ws + kSmallWs;
    EMO_CUDA(cudaMemsetAsync(lv, g->h.L - 1, (size_t)std::max(g->h.rows, 1) * 16, st));
    return launch_pass(g, false, 1, lv, 16, nullptr, 0, nullptr, nullptr, 0, T0, E0, nullptr, nullptr, status, st);
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

int emo_slack_batch_host(const emo_graph *g, int64_t B, const uint8_t *lvl_host, int64_t ldb,
                         uint8_t *dev_lvl, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm,
                         int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                         int32_t *n_critical_host, int64_t *sel_host, void *ws, size_t ws_bytes,
                         uint32_t flags, void *stream)
{
    if (!g || B <= 0 || !lvl_host || !dev_lvl || !makespan_host || !energy_host || !sel_host)
        return EMO_E_INVALID_ARG;
    if (g->host_only) return EMO_E_CUDA;
    size_t need = 0, total = 0;
    emo_workspace_bytes(g, B, 1, &need);
    emo_workspace_bytes(g, B, 2, &total);
    // per-policy result arrays live behind the slack workspace
    size_t per_policy = round_up((size_t)B * 8, 256);
    if (!ws || ws_bytes < total) return EMO_E_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    char *tail = (char *)ws + need;
    int64_t *d_T = (int64_t *)tail;
    double *d_E = (double *)(tail + per_policy);
    int64_t *d_ss = (int64_t *)(tail + 2 * per_policy);
    int32_t *d_nc = (int32_t *)(tail + 3 * per_policy);
    int64_t *d_sel = (int64_t *)(tail + 4 * per_policy);      // {index, T, E bits, T0, E0 bits}
    int32_t *d_status = (int32_t *)(d_sel + 8);
    EMO_CUDA(cudaMemsetAsync(d_sel, 0, 128, st));
    EMO_CUDA(cudaMemcpyAsync(dev_lvl, lvl_host, (size_t)g->h.rows * (size_t)ldb, cudaMemcpyHostToDevice, st));
    int rc = emo_slack_batch(g, B, dev_lvl, ldb, nullptr, nullptr, slack_dev, ldo, d_T, d_E, d_ss, d_nc, ws,
                             need, d_status, flags, st);
    if (rc) return rc;
    rc = emo_baseline(g, d_sel + 3, (double *)(d_sel + 4), ws, need, d_status, st);
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

}  // extern "C"
