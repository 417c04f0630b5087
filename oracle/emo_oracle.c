/*
 * CPU oracle for the what-if timing / energy evaluation over an execution DAG.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, one-policy-at-a-time restatement of
 * what the method computes; the CUDA library is checked against it.  It shares no code, header,
 * table or helper with the CUDA path and must never be linked into or called from it.  Only the
 * tests, the smoke check and the bench's CPU-baseline leg may call it.
 *
 * What each routine follows:
 *   durations / energies of a policy ........ Eq. 3 (frequency-indexed t_v, e_v; Alg. 1 "dur <- T_f[v], e <- E_f[v]")
 *   forward pass ............................. Eq. 1 (C_v = t_v + max over predecessors of C_k), Alg. 1 main loop
 *   makespan ................................. Eq. 2 (T_DAG = max over all v of C_v), Alg. 1 "T <- max comp[v]"
 *   energy ................................... Eq. 2 without E_idle (sum over v of e_v), Alg. 1 "E_a <- E_a + e"
 *   backward pass / slack .................... critical-path-method total float; the paper only
 *                                              describes slack in words (Sec. 1: the time a kernel
 *                                              can be delayed without touching the critical path), so
 *                                              the textbook recurrence is used: LF_v = min over successors of LS_u
 *                                              (T for sinks), LS_v = LF_v - t_v, slack_v = LS_v - ES_v
 *   target ................................... Sec. 4.6: T_0 is the makespan at maximum frequency and
 *                                              the budget is a fraction of it (2 %, 5 % in Sec. 5)
 *   selection ................................ Eq. 4 over a finite candidate set, with the feasibility
 *                                              and strict-improvement test of Alg. 2 (first best kept)
 *   critical predecessors, packing ........... Eq. 5 with Alg. 1's update rule; the dependency-aware greedy packing of
 *                                              Sec. 4.4 (three rules, its listing restated)
 *   pack modelling ........................... Eq. 6 (non-negative least squares, by its definition over all
 *                                              supports) and Eq. 7 (tables as weighted sums)
 *   policy search ............................ Alg. 2 (dynamic programming over the intervals, one prediction per
 *                                              candidate); a heuristic, pinned only in part: see its comment
 *   time-interval policies and idle energy ... Alg. 1 as printed (level from the interval that holds the
 *                                              start time, critical-predecessor tracking, E_a and E_i), Eq. 2
 *
 * Readings where the paper is silent: a node without predecessors starts at 0; edges carry no lag;
 * the maximum in Eq. 2 runs over all nodes; energies are summed in node order with Neumaier
 * compensation in fp64; times are int64 nanoseconds.
 *
 * Graph format: predecessor CSR (row_ptr[n+1], col[m]).  The oracle derives its own topological
 * order (Kahn) and its own successor lists; it never relies on the caller's numbering.
 *
 * Parity pins: every routine here is pinned by tests/test_oracle_pins.py (brute-force path
 * enumeration, closed forms, reversal duality, invariants, a hand-worked example).  Of this file only
 * the policy search (Alg. 2) has a part that is "parity unpinned": which of two candidates of one time bin
 * survives (its comment lists the pins, among them the exhaustive optimum where no bin is shared).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORACLE_OK 0
#define ORACLE_E_CYCLE (-1)
#define ORACLE_E_RANGE (-2)
#define ORACLE_E_ARG (-3)
#define ORACLE_E_NOMEM (-4)

/* Kahn's algorithm on the predecessor CSR.  order[i] = i-th node of a topological order. */
int emo_oracle_topo(int32_t n, const int64_t *row_ptr, const int32_t *col, int32_t *order)
{
    if (n < 0) return ORACLE_E_ARG;
    if (n == 0) return ORACLE_OK;
    int64_t m = row_ptr[n];
    int32_t *outdeg = calloc((size_t)n, sizeof *outdeg);
    int64_t *sp = calloc((size_t)n + 1, sizeof *sp);
    int32_t *succ = malloc(sizeof *succ * (size_t)(m > 0 ? m : 1));
    int32_t *indeg = malloc(sizeof *indeg * (size_t)n);
    if (!outdeg || !sp || !succ || !indeg) { free(outdeg); free(sp); free(succ); free(indeg); return ORACLE_E_NOMEM; }
    for (int32_t v = 0; v < n; ++v) {
        indeg[v] = (int32_t)(row_ptr[v + 1] - row_ptr[v]);
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            if (col[e] < 0 || col[e] >= n) { free(outdeg); free(sp); free(succ); free(indeg); return ORACLE_E_RANGE; }
            outdeg[col[e]]++;
        }
    }
    for (int32_t v = 0; v < n; ++v) sp[v + 1] = sp[v] + outdeg[v];
    memset(outdeg, 0, sizeof *outdeg * (size_t)n);
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            int32_t k = col[e];
            succ[sp[k] + outdeg[k]++] = v;
        }
    int32_t head = 0, tail = 0;
    for (int32_t v = 0; v < n; ++v) if (indeg[v] == 0) order[tail++] = v;
    while (head < tail) {
        int32_t v = order[head++];
        for (int64_t e = sp[v]; e < sp[v + 1]; ++e) {
            int32_t u = succ[e];
            if (--indeg[u] == 0) order[tail++] = u;
        }
    }
    free(outdeg); free(sp); free(succ); free(indeg);
    return tail == n ? ORACLE_OK : ORACLE_E_CYCLE;
}

/* Eq. 3: the duration and energy a policy gives each node.  Node v reads the level of policy row
 * group_of[v] (v itself when group_of is NULL); a negative group means the node ignores the
 * policy and uses table column 0.  lvl points at the first row of one policy column, rows are
 * ld bytes apart. */
int emo_oracle_durations(int32_t n, int32_t L, const int64_t *lat, const double *energy,
                         const int32_t *group_of, const uint8_t *lvl, int64_t ld,
                         int64_t *dur, double *e)
{
    for (int32_t v = 0; v < n; ++v) {
        int32_t r = group_of ? group_of[v] : v;
        int32_t l = 0;
        if (r >= 0) {
            l = lvl[(int64_t)r * ld];
            if (l >= L) return ORACLE_E_RANGE;
        }
        dur[v] = lat[(int64_t)v * L + l];
        if (e) e[v] = energy[(int64_t)v * L + l];
    }
    return ORACLE_OK;
}

/* Eq. 1 in topological order.  ES_v = max(0, max_k C_k), C_v = ES_v + dur_v.  Returns the
 * makespan of Eq. 2, the maximum of C_v over ALL nodes. */
int64_t emo_oracle_forward(int32_t n, const int64_t *row_ptr, const int32_t *col,
                           const int32_t *order, const int64_t *dur, int64_t *ES, int64_t *C)
{
    int64_t T = 0;
    for (int32_t i = 0; i < n; ++i) {
        int32_t v = order[i];
        int64_t start = 0;
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            int64_t ck = C[col[e]];
            if (ck > start) start = ck;
        }
        ES[v] = start;
        C[v] = start + dur[v];
        if (C[v] > T) T = C[v];
    }
    return T;
}

/* Backward pass, written independently of the forward one: explicit successor lists, nodes in
 * reverse topological order.  LF_v = T for a node without successors, else min over successors
 * of LS_u;  LS_v = LF_v - dur_v. */
int emo_oracle_backward(int32_t n, const int64_t *row_ptr, const int32_t *col,
                        const int32_t *order, const int64_t *dur, int64_t T, int64_t *LS)
{
    int64_t m = n > 0 ? row_ptr[n] : 0;
    int64_t *sp = calloc((size_t)n + 2, sizeof *sp);
    int32_t *succ = malloc(sizeof *succ * (size_t)(m > 0 ? m : 1));
    int64_t *fill = calloc((size_t)n + 1, sizeof *fill);
    if (!sp || !succ || !fill) { free(sp); free(succ); free(fill); return ORACLE_E_NOMEM; }
    for (int64_t e = 0; e < m; ++e) sp[col[e] + 1]++;
    for (int32_t v = 0; v < n; ++v) sp[v + 1] += sp[v];
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            int32_t k = col[e];
            succ[sp[k] + fill[k]++] = v;
        }
    for (int32_t i = n - 1; i >= 0; --i) {
        int32_t v = order[i];
        int64_t lf;
        if (sp[v + 1] == sp[v]) {
            lf = T;
        } else {
            lf = LS[succ[sp[v]]];
            for (int64_t e = sp[v] + 1; e < sp[v + 1]; ++e) {
                int64_t x = LS[succ[e]];
                if (x < lf) lf = x;
            }
        }
        LS[v] = lf - dur[v];
    }
    free(sp); free(succ); free(fill);
    return ORACLE_OK;
}

/* Sum of the node energies in node order, Neumaier-compensated, fp64. */
double emo_oracle_energy(int32_t n, const double *e)
{
    double sum = 0.0, comp = 0.0;   /* built without -ffast-math: no reassociation */
    for (int32_t v = 0; v < n; ++v) {
        double x = e[v];
        double t = sum + x;
        if (fabs(sum) >= fabs(x)) comp += (sum - t) + x;
        else comp += (x - t) + sum;
        sum = t;
    }
    return sum + comp;
}

/* Policies b0 <= b < b1 of a level matrix lvl[rows][ldb], one at a time.
 * Outputs (each may be NULL): makespan[B], energy_out[B] indexed by b; ES/LS/slack laid out
 * [n][ldo] with column b - ocol0 (so a caller can ask for a slab of columns); slack_sum[B],
 * n_critical[B] (nodes with slack 0). */
int emo_oracle_batch(int32_t n, const int64_t *row_ptr, const int32_t *col, int32_t L,
                     const int64_t *lat, const double *energy, const int32_t *group_of,
                     const uint8_t *lvl, int64_t ldb, int64_t b0, int64_t b1,
                     int64_t *makespan, double *energy_out,
                     int64_t *ES_out, int64_t *LS_out, int64_t *slack_out, int64_t ldo, int64_t ocol0,
                     int64_t *slack_sum, int32_t *n_critical)
{
    if (n < 0 || L < 1 || b0 < 0 || b1 < b0) return ORACLE_E_ARG;
    size_t nn = (size_t)(n > 0 ? n : 1);
    int32_t *order = malloc(sizeof *order * nn);
    int64_t *dur = malloc(sizeof *dur * nn), *ES = malloc(sizeof *ES * nn);
    int64_t *C = malloc(sizeof *C * nn), *LS = malloc(sizeof *LS * nn);
    double *e = malloc(sizeof *e * nn);
    int rc = ORACLE_OK;
    if (!order || !dur || !ES || !C || !LS || !e) { rc = ORACLE_E_NOMEM; goto done; }
    rc = emo_oracle_topo(n, row_ptr, col, order);
    if (rc) goto done;
    int need_back = ES_out || LS_out || slack_out || slack_sum || n_critical;
    for (int64_t b = b0; b < b1; ++b) {
        rc = emo_oracle_durations(n, L, lat, energy, group_of, lvl + b, ldb, dur, e);
        if (rc) goto done;
        int64_t T = emo_oracle_forward(n, row_ptr, col, order, dur, ES, C);
        if (makespan) makespan[b] = T;
        if (energy_out) energy_out[b] = emo_oracle_energy(n, e);
        if (need_back) {
            rc = emo_oracle_backward(n, row_ptr, col, order, dur, T, LS);
            if (rc) goto done;
            int64_t ssum = 0;
            int32_t ncrit = 0;
            for (int32_t v = 0; v < n; ++v) {
                int64_t s = LS[v] - ES[v];
                ssum += s;
                ncrit += (s == 0);
                int64_t o = (int64_t)v * ldo + (b - ocol0);
                if (ES_out) ES_out[o] = ES[v];
                if (LS_out) LS_out[o] = LS[v];
                if (slack_out) slack_out[o] = s;
            }
            if (slack_sum) slack_sum[b] = ssum;
            if (n_critical) n_critical[b] = ncrit;
        }
    }
done:
    free(order); free(dur); free(ES); free(C); free(LS); free(e);
    return rc;
}

/* T_set = T_0 + floor(T_0 * delta_ppm / 10^6): the latency budget relative to the
 * maximum-frequency makespan (Sec. 4.6; budgets of 2 % and 5 % in Sec. 5). */
int64_t emo_oracle_target(int64_t T0, int64_t delta_ppm)
{
    __int128 x = (__int128)T0 * (__int128)delta_ppm;
    return T0 + (int64_t)(x / 1000000);
}

/* Eq. 4 over a finite batch: the feasible policy (T <= target) of least energy; a later policy
 * replaces the incumbent only if strictly better (Alg. 2), so ties go to the lowest index.
 * Returns -1 when no policy is feasible. */
int64_t emo_oracle_select(int64_t B, const int64_t *makespan, const double *energy, int64_t target)
{
    int64_t best = -1;
    for (int64_t b = 0; b < B; ++b) {
        if (makespan[b] <= target && (best < 0 || energy[b] < energy[best])) best = b;
    }
    return best;
}

/* ------------------------------------------------------------------------------------------------
 * Alg. 1 with a time-interval policy P = {<T_i, F_i>}: the frequency of a pack is the one of the
 * interval that holds its START time (Alg. 1: "f <- F_i where start in [T_i, T_{i+1})"; Eq. 4's
 * side condition puts max over predecessors of C_k in the interval), plus the idle energy of Eq. 2.
 * The steps are taken in the algorithm's order and notation: comp[], the critical predecessor
 * pred[] updated from every finished node to its successors, start = comp[pred[v]], E_a, E_i.
 *
 * Inputs beyond the per-node-level routines:
 *   dev_of[n]   device whose policy governs node v (each GPU has its own policy, Sec. 4.3);
 *               -1 = not a pack: the policy does not touch it, dur = lat[v][0], e = energy[v][0]
 *               (the tables hold the fixed t_v and the zero energy that Alg. 1 gives such nodes)
 *   breaks[I]   the change points T_1 < T_2 < ... (nanoseconds), breaks[0] = 0; the last interval
 *               has no end
 *   F           levels, [D][I][ldb]: device d, interval i, policy b at F[(d*I + i)*ldb + b]
 *   p_idle[L]   idle power at each level in watts (NULL: no idle energy)
 *
 * Readings where the paper is silent: idle_time of an interval, per device, is the interval's
 * length inside [0, T) minus the summed overlap of that device's packs with it, not below zero
 * (packs of several streams can overlap); the last interval ends at T; a pack that starts at or
 * after the last change point uses the last level; E_i sums devices, then intervals, in order,
 * compensated like E_a.
 *
 * Outputs (each may be NULL): makespan[b], e_active[b], e_idle[b]; level_out[v*ldo + (b - b0)] =
 * the level the policy gave node v (0 for a node outside every policy).
 * ------------------------------------------------------------------------------------------------ */
int emo_oracle_intervals(int32_t n, const int64_t *row_ptr, const int32_t *col, int32_t L,
                         const int64_t *lat, const double *energy, const int32_t *dev_of, int32_t D,
                         int32_t I, const int64_t *breaks, const uint8_t *F, int64_t ldb,
                         int64_t b0, int64_t b1, const double *p_idle,
                         int64_t *makespan, double *e_active, double *e_idle,
                         uint8_t *level_out, int64_t ldo)
{
    if (n < 0 || L < 1 || D < 1 || I < 1 || b0 < 0 || b1 < b0 || !breaks || breaks[0] != 0) return ORACLE_E_ARG;
    for (int32_t i = 1; i < I; ++i)
        if (breaks[i] <= breaks[i - 1]) return ORACLE_E_ARG;
    size_t nn = (size_t)(n > 0 ? n : 1);
    int64_t m = n > 0 ? row_ptr[n] : 0;
    int32_t *order = malloc(sizeof *order * nn), *pred = malloc(sizeof *pred * nn);
    int64_t *comp = malloc(sizeof *comp * nn), *start_of = malloc(sizeof *start_of * nn);
    int64_t *succ_ptr = calloc(nn + 1, sizeof *succ_ptr);
    int32_t *succ = malloc(sizeof *succ * (size_t)(m > 0 ? m : 1));
    double *e = malloc(sizeof *e * nn), *ei = malloc(sizeof *ei * (size_t)D * (size_t)I);
    int rc = ORACLE_OK;
    if (!order || !pred || !comp || !start_of || !succ_ptr || !succ || !e || !ei) { rc = ORACLE_E_NOMEM; goto done; }
    rc = emo_oracle_topo(n, row_ptr, col, order);
    if (rc) goto done;
    /* successor lists from the predecessor CSR */
    for (int32_t v = 0; v < n; ++v)
        for (int64_t k = row_ptr[v]; k < row_ptr[v + 1]; ++k) succ_ptr[col[k] + 1]++;
    for (int32_t v = 0; v < n; ++v) succ_ptr[v + 1] += succ_ptr[v];
    {
        int64_t *fill = malloc(sizeof *fill * nn);
        if (!fill) { rc = ORACLE_E_NOMEM; goto done; }
        memcpy(fill, succ_ptr, sizeof *fill * nn);
        for (int32_t v = 0; v < n; ++v)
            for (int64_t k = row_ptr[v]; k < row_ptr[v + 1]; ++k) succ[fill[col[k]]++] = v;
        free(fill);
    }
    for (int32_t v = 0; v < n; ++v)
        if (dev_of[v] >= D) { rc = ORACLE_E_RANGE; goto done; }

    for (int64_t b = b0; b < b1; ++b) {
        for (int32_t v = 0; v < n; ++v) { comp[v] = 0; pred[v] = -1; }
        for (int32_t k = 0; k < n; ++k) {
            int32_t v = order[k];
            int64_t start = pred[v] >= 0 ? comp[pred[v]] : 0;
            int64_t dur;
            int32_t f = 0;
            if (dev_of[v] >= 0) {
                /* f <- F_i where start in [T_i, T_{i+1}) */
                int32_t i = 0;
                while (i + 1 < I && breaks[i + 1] <= start) ++i;
                f = F[((int64_t)dev_of[v] * I + i) * ldb + b];
                if (f >= L) { rc = ORACLE_E_RANGE; goto done; }
            }
            dur = lat[(int64_t)v * L + f];
            e[v] = energy[(int64_t)v * L + f];
            start_of[v] = start;
            comp[v] = start + dur;
            if (level_out) level_out[(int64_t)v * ldo + (b - b0)] = (uint8_t)f;
            for (int64_t s = succ_ptr[v]; s < succ_ptr[v + 1]; ++s) {
                int32_t u = succ[s];
                if (pred[u] < 0 || comp[v] > comp[pred[u]]) pred[u] = v;
            }
        }
        int64_t T = 0;
        for (int32_t v = 0; v < n; ++v)
            if (comp[v] > T) T = comp[v];
        /* E_i <- E_i + idle_time of [T_i, T_{i+1}) x p_idle[F_i], per device */
        double Ei = 0.0;
        if (p_idle) {
            for (int32_t d = 0; d < D; ++d)
                for (int32_t i = 0; i < I; ++i) {
                    int64_t lo = breaks[i], hi = (i + 1 < I) ? breaks[i + 1] : T;
                    if (hi > T) hi = T;
                    int64_t len = hi > lo ? hi - lo : 0;
                    int64_t busy = 0;
                    for (int32_t v = 0; v < n; ++v) {
                        if (dev_of[v] != d) continue;
                        int64_t a = start_of[v] > lo ? start_of[v] : lo;
                        int64_t z = comp[v] < hi ? comp[v] : hi;
                        if (z > a) busy += z - a;
                    }
                    int64_t idle = len > busy ? len - busy : 0;
                    ei[(size_t)d * I + i] = (double)idle * 1e-9 * p_idle[F[((int64_t)d * I + i) * ldb + b]];
                }
            Ei = emo_oracle_energy(D * I, ei);
        }
        if (makespan) makespan[b] = T;
        if (e_active) e_active[b] = emo_oracle_energy(n, e);
        if (e_idle) e_idle[b] = Ei;
    }
done:
    free(order); free(pred); free(comp); free(start_of); free(succ_ptr); free(succ); free(e); free(ei);
    return rc;
}

/* ------------------------------------------------------------------------------------------------
 * Alg. 2: search for a near-optimal time-interval policy by dynamic programming over the intervals.
 * dp[i] maps an end-to-end time to the least energy (and its policy) seen after the first i intervals
 * have been decided; every state is extended by every level for interval i, each candidate is
 * predicted by Alg. 1 (emo_oracle_intervals: active + idle energy), kept if it meets T_max and
 * improves its time's entry strictly.  The steps are taken in the algorithm's order.
 *
 * Readings where the paper is silent: the DP is keyed by the discretised time floor(t / bin_ns) (Sec. 4.6
 * discretises the constraint, "e.g., 1 ms"; bin_ns = 1 keeps exact times); the states of dp[i] are visited
 * in ascending time and the levels in ascending order, so that with the strict test the first candidate
 * of least energy in a bin stays; one policy governs every device (the paper drops the GPU index in
 * Alg. 2 and replicates one GPU's policy, Sec. 6.2); the answer is the entry of dp[I] of least energy,
 * the earliest time among equals; the default policy P_0 is the maximum level L-1 everywhere.  If even
 * P_0 misses T_max, dp[0] is still seeded with it (Alg. 2 line 3 has no test) and the search may end
 * with an empty dp[I]: then *found = 0.
 *
 * Pins (tests/test_oracle_search.py): the exhaustive optimum for one interval; for several intervals the
 * exhaustive optimum (policy, time, energy, number of predictions) whenever no two policies end in one
 * time bin, with a constraint that admits all of them and with one that cuts into the set (lower levels
 * never faster there); bounds otherwise (never worse than P_0, never better than the exhaustive optimum,
 * always feasible); consistency of the reported (T, E) with Alg. 1 on the reported policy; L = 1;
 * T_max = t_0.  Where two candidates do end in one bin the DP is a heuristic (one of them survives) and
 * has no independent definition to compare with: for that choice alone it is "parity unpinned".
 *
 * Outputs: F_best[I] levels of the chosen policy, T_best, E_best, n_pred = calls of Alg. 1, found.
 * ------------------------------------------------------------------------------------------------ */
typedef struct {
    int64_t key;      /* floor(t / bin) */
    int64_t t;
    double E;
    uint8_t *P;       /* I levels */
} dp_state;

static int dp_cmp(const void *a, const void *b)
{
    int64_t x = ((const dp_state *)a)->key, y = ((const dp_state *)b)->key;
    return x < y ? -1 : (x > y ? 1 : 0);
}

int emo_oracle_search_dp(int32_t n, const int64_t *row_ptr, const int32_t *col, int32_t L,
                         const int64_t *lat, const double *energy, const int32_t *dev_of, int32_t D,
                         int32_t I, const int64_t *breaks, const double *p_idle,
                         int64_t T_max, int64_t bin_ns,
                         uint8_t *F_best, int64_t *T_best, double *E_best, int64_t *n_pred, int32_t *found)
{
    if (I < 1 || L < 1 || D < 1 || bin_ns < 1) return ORACLE_E_ARG;
    int rc = ORACLE_OK;
    size_t cap = 16, cnt = 0, ncap = 16, ncnt = 0;
    dp_state *cur = calloc(cap, sizeof *cur), *nxt = calloc(ncap, sizeof *nxt);
    uint8_t *Fd = malloc((size_t)D * (size_t)I);      /* one candidate: [D][I][1] */
    uint8_t *P2 = malloc((size_t)I);
    int64_t calls = 0;
    if (!cur || !nxt || !Fd || !P2) { rc = ORACLE_E_NOMEM; goto done; }
#define PRED(Pol, tt, ee)                                                                                   \
    do {                                                                                                    \
        for (int32_t d_ = 0; d_ < D; ++d_) memcpy(Fd + (size_t)d_ * I, (Pol), (size_t)I);                    \
        double ea_ = 0.0, ei_ = 0.0;                                                                        \
        rc = emo_oracle_intervals(n, row_ptr, col, L, lat, energy, dev_of, D, I, breaks, Fd, 1, 0, 1, p_idle, \
                                  &(tt), &ea_, &ei_, NULL, 0);                                              \
        (ee) = ea_ + ei_;                                                                                   \
        ++calls;                                                                                            \
    } while (0)
    /* P_0 = default frequency in all intervals; (t_0, E_0) = Pred(P_0); dp[0][t_0] = (E_0, P_0) */
    {
        uint8_t *P0 = malloc((size_t)I);
        if (!P0) { rc = ORACLE_E_NOMEM; goto done; }
        memset(P0, L - 1, (size_t)I);
        int64_t t0 = 0;
        double E0 = 0.0;
        PRED(P0, t0, E0);
        if (rc) { free(P0); goto done; }
        cur[0].key = t0 / bin_ns; cur[0].t = t0; cur[0].E = E0; cur[0].P = P0;
        cnt = 1;
    }
    for (int32_t i = 0; i < I; ++i) {
        qsort(cur, cnt, sizeof *cur, dp_cmp);      /* ascending time */
        ncnt = 0;
        for (size_t s = 0; s < cnt; ++s) {
            for (int32_t f = 0; f < L; ++f) {
                /* P' <- set level f in [p_i, p_{i+1}) in P;  (t', E') <- Pred(P') */
                memcpy(P2, cur[s].P, (size_t)I);
                P2[i] = (uint8_t)f;
                int64_t t2 = 0;
                double E2 = 0.0;
                PRED(P2, t2, E2);
                if (rc) goto done;
                if (t2 > T_max) continue;
                int64_t key = t2 / bin_ns;
                size_t k = 0;
                while (k < ncnt && nxt[k].key != key) ++k;
                if (k == ncnt) {
                    if (ncnt == ncap) {
                        dp_state *g2 = realloc(nxt, 2 * ncap * sizeof *nxt);
                        if (!g2) { rc = ORACLE_E_NOMEM; goto done; }
                        nxt = g2;
                        memset(nxt + ncap, 0, ncap * sizeof *nxt);
                        ncap *= 2;
                    }
                    nxt[k].P = malloc((size_t)I);
                    if (!nxt[k].P) { rc = ORACLE_E_NOMEM; goto done; }
                    nxt[k].key = key; nxt[k].t = t2; nxt[k].E = E2;
                    memcpy(nxt[k].P, P2, (size_t)I);
                    ++ncnt;
                } else if (E2 < nxt[k].E) {
                    nxt[k].t = t2; nxt[k].E = E2;
                    memcpy(nxt[k].P, P2, (size_t)I);
                }
            }
        }
        /* dp[i] is no longer needed */
        for (size_t s = 0; s < cnt; ++s) { free(cur[s].P); cur[s].P = NULL; }
        dp_state *tmp = cur; cur = nxt; nxt = tmp;
        size_t tc = cap; cap = ncap; ncap = tc;
        cnt = ncnt; ncnt = 0;
    }
    /* (E*, P*) <- min over t <= T_max of dp[N][t] */
    qsort(cur, cnt, sizeof *cur, dp_cmp);
    {
        size_t best = cnt;
        for (size_t s = 0; s < cnt; ++s)
            if (best == cnt || cur[s].E < cur[best].E) best = s;
        if (found) *found = best < cnt;
        if (best < cnt) {
            if (F_best) memcpy(F_best, cur[best].P, (size_t)I);
            if (T_best) *T_best = cur[best].t;
            if (E_best) *E_best = cur[best].E;
        }
    }
    if (n_pred) *n_pred = calls;
done:
    if (cur) for (size_t s = 0; s < cap; ++s) free(cur[s].P);
    if (nxt) for (size_t s = 0; s < ncap; ++s) free(nxt[s].P);
    free(cur); free(nxt); free(Fd); free(P2);
    return rc;
#undef PRED
}

/* ------------------------------------------------------------------------------------------------
 * Eq. 5: the critical predecessor k*_v = argmax over predecessors of C_k, tracked as Alg. 1 does it:
 * every finished node offers itself to its successors and replaces their entry only if it finishes
 * strictly later, so among equals the predecessor that is processed first stays.
 *
 * Reading: nodes are processed in index order (the caller's numbering must be topological: every
 * predecessor has a lower index), which makes "processed first" = "lowest index".  dur[v] is the
 * duration of v under the policy in question (the default frequency for packing).
 * Outputs: C[v] completion times, crit[v] = k*_v or -1 for a node without predecessors.
 * ------------------------------------------------------------------------------------------------ */
int emo_oracle_crit_pred(int32_t n, const int64_t *row_ptr, const int32_t *col, const int64_t *dur,
                         int64_t *C, int32_t *crit)
{
    if (n < 0) return ORACLE_E_ARG;
    for (int32_t v = 0; v < n; ++v) crit[v] = -1;
    /* successor lists */
    int64_t m = n > 0 ? row_ptr[n] : 0;
    int64_t *sp = calloc((size_t)n + 2, sizeof *sp);
    int32_t *sc = malloc(sizeof *sc * (size_t)(m > 0 ? m : 1));
    int64_t *fill = malloc(sizeof *fill * (size_t)(n > 0 ? n : 1));
    if (!sp || !sc || !fill) { free(sp); free(sc); free(fill); return ORACLE_E_NOMEM; }
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            if (col[e] >= v) { free(sp); free(sc); free(fill); return ORACLE_E_CYCLE; }
            sp[col[e] + 1]++;
        }
    for (int32_t v = 0; v < n; ++v) sp[v + 1] += sp[v];
    memcpy(fill, sp, sizeof *fill * (size_t)n);
    for (int32_t v = 0; v < n; ++v)
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) sc[fill[col[e]]++] = v;
    for (int32_t v = 0; v < n; ++v) {
        int64_t start = crit[v] >= 0 ? C[crit[v]] : 0;
        C[v] = start + dur[v];
        for (int64_t s = sp[v]; s < sp[v + 1]; ++s) {
            int32_t u = sc[s];
            if (crit[u] < 0 || C[v] > C[crit[u]]) crit[u] = v;
        }
    }
    free(sp); free(sc); free(fill);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------------
 * Dependency-aware greedy packing (Sec. 4.4, its listing): walk the kernels of one stream in order and
 * keep adding the next kernel v to the current pack (last member u) while
 *   rule 1  v and its critical predecessor are in the same stream,
 *   rule 2  every critical successor of u is in u's stream,
 *   rule 3  the pack's duration at the default frequency plus t_v stays below delta_max (strict);
 * otherwise the pack is closed and v starts a new one.
 *
 * Readings: the listing's sorted kernel list V is taken per (device, stream): a pack is a stretch of one
 * stream (the rules speak of "the same stream", and only the first member's incoming and the last
 * member's outgoing dependencies survive, which presupposes that the members follow each other on one
 * stream); kernels are visited in index order; a node that is not a GPU kernel (is_kernel[v] = 0) is in
 * no pack and in no stream, so a kernel whose critical predecessor is a launch or a collective starts a
 * new pack; a kernel without predecessors has no critical predecessor and fails rule 1.
 * stream_of[v] identifies the stream globally (device and stream together).
 * Output: pack_of[v] = pack number (0, 1, ... in order of their first member) or -1; returns the count
 * in *n_packs.
 * ------------------------------------------------------------------------------------------------ */
int emo_oracle_pack_greedy(int32_t n, const int64_t *row_ptr, const int32_t *col, const uint8_t *is_kernel,
                           const int32_t *stream_of, const int64_t *t_default, const int32_t *crit,
                           int64_t delta_max, int32_t *pack_of, int32_t *n_packs)
{
    if (n < 0) return ORACLE_E_ARG;
    (void)row_ptr; (void)col;
    int32_t max_stream = -1;
    for (int32_t v = 0; v < n; ++v) {
        pack_of[v] = -1;
        if (is_kernel[v] && stream_of[v] > max_stream) max_stream = stream_of[v];
    }
    /* rule 2 needs, for every node, whether all its critical successors share its stream */
    uint8_t *succ_ok = malloc((size_t)(n > 0 ? n : 1));
    if (!succ_ok) return ORACLE_E_NOMEM;
    for (int32_t v = 0; v < n; ++v) succ_ok[v] = 1;
    for (int32_t v = 0; v < n; ++v) {
        int32_t k = crit[v];
        if (k < 0 || !is_kernel[k]) continue;
        if (!is_kernel[v] || stream_of[v] != stream_of[k]) succ_ok[k] = 0;
    }
    /* pack numbers are handed out in order of the first member's index: collect (first member) per pack */
    int32_t *first = malloc(sizeof *first * (size_t)(n > 0 ? n : 1));
    int32_t *tmp_pack = malloc(sizeof *tmp_pack * (size_t)(n > 0 ? n : 1));
    if (!first || !tmp_pack) { free(succ_ok); free(first); free(tmp_pack); return ORACLE_E_NOMEM; }
    int32_t count = 0;
    for (int32_t s = 0; s <= max_stream; ++s) {
        int32_t u = -1;            /* last node in the current pack */
        int64_t dur_pack = 0;
        for (int32_t v = 0; v < n; ++v) {
            if (!is_kernel[v] || stream_of[v] != s) continue;
            int ok = 0;
            if (u >= 0) {
                int r1 = crit[v] >= 0 && is_kernel[crit[v]] && stream_of[crit[v]] == stream_of[v];
                int r2 = succ_ok[u];
                int r3 = dur_pack + t_default[v] < delta_max;
                ok = r1 && r2 && r3;
            }
            if (ok) {
                tmp_pack[v] = tmp_pack[u];
                dur_pack += t_default[v];
            } else {
                first[count] = v;
                tmp_pack[v] = count++;
                dur_pack = t_default[v];
            }
            u = v;
        }
    }
    /* renumber by first member */
    {
        int32_t *order = malloc(sizeof *order * (size_t)(count > 0 ? count : 1));
        int32_t *newid = malloc(sizeof *newid * (size_t)(count > 0 ? count : 1));
        if (!order || !newid) { free(order); free(newid); free(succ_ok); free(first); free(tmp_pack); return ORACLE_E_NOMEM; }
        for (int32_t p = 0; p < count; ++p) order[p] = p;
        for (int32_t i = 1; i < count; ++i) {          /* insertion sort by first member */
            int32_t x = order[i], j = i - 1;
            while (j >= 0 && first[order[j]] > first[x]) { order[j + 1] = order[j]; --j; }
            order[j + 1] = x;
        }
        for (int32_t i = 0; i < count; ++i) newid[order[i]] = i;
        for (int32_t v = 0; v < n; ++v)
            if (is_kernel[v]) pack_of[v] = newid[tmp_pack[v]];
        free(order); free(newid);
    }
    if (n_packs) *n_packs = count;
    free(succ_ok); free(first); free(tmp_pack);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------------
 * Pack modelling (Sec. 4.5): a pack's feature vector b (n metrics at the default frequency) is
 * written as a non-negative combination of m micro-benchmarks, x = argmin ||B x - b||^2 subject to
 * x >= 0 (Eq. 6), and its tables follow as T_f[P] = sum_i x_i T_f[B_i], E_f[P] = sum_i x_i E_f[B_i]
 * (Eq. 7).
 *
 * The minimiser has a plain definition, and that is what is written out here: every subset S of the m
 * columns is tried, the unconstrained least-squares solution on S is computed (normal equations,
 * Cholesky, long double), subsets whose solution has a negative entry or whose columns are dependent
 * are skipped, and the feasible candidate of least residual wins (ties: the first subset in counting
 * order).  The constrained optimum is among the candidates and every candidate is a feasible point, so
 * the least residual is the optimum.  Exponential in m (m <= 16): for tests only.
 * ------------------------------------------------------------------------------------------------ */
int emo_oracle_nnls(int32_t n, int32_t m, const double *B /*[n][m]*/, const double *b /*[n]*/, double *x /*[m]*/, double *resid2)
{
    if (n < 1 || m < 1 || m > 16) return ORACLE_E_ARG;
    long double G[16][16], c[16], bb = 0.0L;
    for (int i = 0; i < m; ++i) {
        c[i] = 0.0L;
        for (int r = 0; r < n; ++r) c[i] += (long double)B[r * m + i] * b[r];
        for (int j = 0; j < m; ++j) {
            G[i][j] = 0.0L;
            for (int r = 0; r < n; ++r) G[i][j] += (long double)B[r * m + i] * B[r * m + j];
        }
    }
    for (int r = 0; r < n; ++r) bb += (long double)b[r] * b[r];
    long double best = bb;              /* the empty subset: x = 0 */
    for (int i = 0; i < m; ++i) x[i] = 0.0;
    for (uint32_t S = 1; S < (1u << m); ++S) {
        int idx[16], k = 0;
        for (int i = 0; i < m; ++i)
            if (S & (1u << i)) idx[k++] = i;
        /* Cholesky of G_SS */
        long double Lc[16][16], z[16], y[16];
        int ok = 1;
        for (int i = 0; i < k && ok; ++i)
            for (int j = 0; j <= i; ++j) {
                long double s = G[idx[i]][idx[j]];
                for (int q = 0; q < j; ++q) s -= Lc[i][q] * Lc[j][q];
                if (i == j) {
                    if (s <= 1e-18L * G[idx[i]][idx[i]]) { ok = 0; break; }      /* dependent columns */
                    Lc[i][i] = sqrtl(s);
                } else {
                    Lc[i][j] = s / Lc[j][j];
                }
            }
        if (!ok) continue;
        for (int i = 0; i < k; ++i) {
            long double s = c[idx[i]];
            for (int q = 0; q < i; ++q) s -= Lc[i][q] * y[q];
            y[i] = s / Lc[i][i];
        }
        for (int i = k - 1; i >= 0; --i) {
            long double s = y[i];
            for (int q = i + 1; q < k; ++q) s -= Lc[q][i] * z[q];
            z[i] = s / Lc[i][i];
        }
        int feas = 1;
        for (int i = 0; i < k; ++i)
            if (z[i] < 0.0L) { feas = 0; break; }
        if (!feas) continue;
        /* residual^2 = b.b - 2 c_S.z + z.G_SS.z = b.b - c_S.z at the least-squares solution */
        long double r2 = bb;
        for (int i = 0; i < k; ++i) r2 -= c[idx[i]] * z[i];
        if (r2 < best) {
            best = r2;
            for (int i = 0; i < m; ++i) x[i] = 0.0;
            for (int i = 0; i < k; ++i) x[idx[i]] = (double)z[i];
        }
    }
    if (resid2) *resid2 = (double)(best > 0.0L ? best : 0.0L);
    return ORACLE_OK;
}

/* Eq. 6 for every pack, then Eq. 7: T_out, E_out [n_packs][L] from the micro-benchmark tables Tb, Eb [m][L]. */
int emo_oracle_pack_model(int32_t n_packs, int32_t n, int32_t m, int32_t L, const double *B, const double *feat /*[n_packs][n]*/,
                          const double *Tb, const double *Eb, double *x /*[n_packs][m]*/, double *T_out, double *E_out)
{
    for (int32_t p = 0; p < n_packs; ++p) {
        int rc = emo_oracle_nnls(n, m, B, feat + (int64_t)p * n, x + (int64_t)p * m, NULL);
        if (rc) return rc;
        for (int32_t l = 0; l < L; ++l) {
            double t = 0.0, e = 0.0;
            for (int32_t i = 0; i < m; ++i) {
                t += x[(int64_t)p * m + i] * Tb[(int64_t)i * L + l];
                e += x[(int64_t)p * m + i] * Eb[(int64_t)i * L + l];
            }
            T_out[(int64_t)p * L + l] = t;
            E_out[(int64_t)p * L + l] = e;
        }
    }
    return ORACLE_OK;
}
