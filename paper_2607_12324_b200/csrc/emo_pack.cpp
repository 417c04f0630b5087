// Kernel packing (Sec. 4.4): critical predecessors at the default frequency (Eq. 5) and the dependency-aware
// greedy packing of GPU kernels into packs, with the packs' frequency tables.  Host code: the procedure is a
// sequential walk over the kernels of every stream and runs once per workload, before any policy is evaluated.
#include <algorithm>
#include <map>
#include <cstdint>
#include <new>
#include <vector>

#include "../../include/emo.h"

extern "C" {

int emo_pack_greedy(int32_t n, const int64_t *row_ptr, const int32_t *col, const uint8_t *is_kernel,
                    const int32_t *stream_of, const int64_t *t_default, int64_t delta_max, int32_t *crit_out,
                    int32_t *pack_of, int32_t *n_packs)
{
    if (n < 0 || !pack_of || (n > 0 && (!row_ptr || !is_kernel || !stream_of || !t_default))) return EMO_E_INVALID_ARG;
    if (n > 0 && row_ptr[n] > 0 && !col) return EMO_E_INVALID_ARG;
    try {
        // completion times at the default durations and, per node, the predecessor that finishes last
        // (Eq. 5); among equals the one with the lowest index, which is the one Alg. 1 meets first
        std::vector<int64_t> C((size_t)n, 0);
        std::vector<int32_t> crit((size_t)n, -1);
        for (int32_t v = 0; v < n; ++v) {
            if (row_ptr[v + 1] < row_ptr[v]) return EMO_E_INVALID_ARG;
            int64_t best = -1;
            for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
                const int32_t k = col[e];
                if (k < 0 || k >= v) return EMO_E_NOT_TOPOLOGICAL;
                if (C[k] > best || (C[k] == best && k < crit[v])) {
                    best = C[k];
                    crit[v] = k;
                }
            }
            if (t_default[v] < 0) return EMO_E_RANGE;
            C[v] = (best < 0 ? 0 : best) + t_default[v];
        }
        // rule 2 asks, for the last member u of a pack, whether every node whose critical predecessor is u
        // lies in u's stream: one flag per kernel, cleared by any critical successor elsewhere
        std::vector<char> followers_in_stream((size_t)n, 1);
        int32_t n_streams = 0;
        for (int32_t v = 0; v < n; ++v) {
            if (is_kernel[v]) {
                if (stream_of[v] < 0) return EMO_E_INVALID_ARG;
                n_streams = std::max(n_streams, stream_of[v] + 1);
            }
            const int32_t k = crit[v];
            if (k >= 0 && is_kernel[k] && !(is_kernel[v] && stream_of[v] == stream_of[k])) followers_in_stream[k] = 0;
        }
        // one pass over the nodes in index order; every stream keeps its open pack
        struct Open {
            int32_t last = -1, id = -1;
            int64_t duration = 0;
        };
        std::vector<Open> open((size_t)n_streams);
        int32_t count = 0;
        for (int32_t v = 0; v < n; ++v) {
            pack_of[v] = -1;
            if (!is_kernel[v]) continue;
            Open &o = open[(size_t)stream_of[v]];
            const int32_t k = crit[v];
            const bool same_stream_pred = k >= 0 && is_kernel[k] && stream_of[k] == stream_of[v];      // rule 1
            const bool joins = o.last >= 0 && same_stream_pred && followers_in_stream[o.last] &&       // rule 2
                               o.duration + t_default[v] < delta_max;                                    // rule 3
            if (joins) {
                o.duration += t_default[v];
            } else {
                o.id = count++;      // packs are numbered as they open, that is by their first member
                o.duration = t_default[v];
            }
            o.last = v;
            pack_of[v] = o.id;
        }
        if (n_packs) *n_packs = count;
        if (crit_out) std::copy(crit.begin(), crit.end(), crit_out);
    } catch (const std::bad_alloc &) {
        return EMO_E_OOM;
    }
    return EMO_OK;
}

int emo_pack_tables(int32_t n, int32_t L, const int64_t *lat, const double *energy, const int32_t *pack_of, int32_t n_packs,
                    int64_t *pack_lat, double *pack_energy)
{
    if (n < 0 || L < 1 || n_packs < 0 || !pack_of || !lat || !energy || !pack_lat || !pack_energy) return EMO_E_INVALID_ARG;
    for (int64_t i = 0; i < (int64_t)n_packs * L; ++i) {
        pack_lat[i] = 0;
        pack_energy[i] = 0.0;
    }
    // per level, the sum over the members in index order (fixed order: the same energies on every run)
    for (int32_t v = 0; v < n; ++v) {
        const int32_t p = pack_of[v];
        if (p < 0) continue;
        if (p >= n_packs) return EMO_E_RANGE;
        for (int32_t l = 0; l < L; ++l) {
            pack_lat[(int64_t)p * L + l] += lat[(int64_t)v * L + l];
            pack_energy[(int64_t)p * L + l] += energy[(int64_t)v * L + l];
        }
    }
    return EMO_OK;
}

int emo_pack_classes(int32_t n, const int32_t *pack_of, const int32_t *name_id, int32_t n_packs, int32_t *class_of_pack,
                     int32_t *n_classes)
{
    if (n < 0 || n_packs < 0 || !pack_of || !name_id || !class_of_pack) return EMO_E_INVALID_ARG;
    try {
        // the sequence of kernel names of every pack, members in index order
        std::vector<std::vector<int32_t>> seq((size_t)n_packs);
        for (int32_t v = 0; v < n; ++v) {
            const int32_t p = pack_of[v];
            if (p < 0) continue;
            if (p >= n_packs) return EMO_E_RANGE;
            seq[(size_t)p].push_back(name_id[v]);
        }
        // packs with the same sequence form a class; classes are numbered by their first pack
        std::map<std::vector<int32_t>, int32_t> seen;
        int32_t count = 0;
        for (int32_t p = 0; p < n_packs; ++p) {
            auto it = seen.find(seq[(size_t)p]);
            if (it == seen.end()) it = seen.emplace(seq[(size_t)p], count++).first;
            class_of_pack[p] = it->second;
        }
        if (n_classes) *n_classes = count;
    } catch (const std::bad_alloc &) {
        return EMO_E_OOM;
    }
    return EMO_OK;
}

}  // extern "C"
