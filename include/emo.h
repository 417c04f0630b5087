/*
 * emo.h - C ABI of the batched what-if timing and energy evaluator for kernel dependency graphs.
 *
 * The library evaluates many candidate frequency-level policies at once on one execution graph:
 * earliest start times by a max-plus forward pass (Eq. 1) giving the makespan (Eq. 2), latest
 * start times by a backward pass giving per-node slack, total energy from frequency-indexed
 * per-node tables (Eq. 2, Eq. 3), and the least-energy policy within a latency budget (Eq. 4).
 * All of it runs in CUDA kernels for sm_100a; there is no CPU fallback.
 *
 * Conventions
 *   - Every function returns an int: EMO_OK (0) or a negative EMO_E_* code.  Nothing throws or
 *     aborts across this boundary.  Output parameters are written only on success.
 *   - "host" / "device" on a pointer says where the memory lives.  Device pointers are borrowed
 *     until the work queued on `stream` has completed; the library never frees caller memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls that take a
 *     stream are asynchronous: they queue kernels and return.
 *   - A graph handle is immutable after emo_graph_load and may be shared by concurrent calls that
 *     use distinct workspaces and streams.
 *   - Notation: n nodes, m edges, L frequency levels (level L-1 = maximum frequency, the
 *     default), B policies.  A policy assigns a level to every policy row; node v reads row
 *     group_of[v] (row v when no grouping was given).  Times are int64 nanoseconds, energies
 *     fp64 joules.
 *   - Level matrix layout: lvl[r * ldb + b] is the level policy b gives row r (uint8, row-major
 *     over rows, policies contiguous).  Per-node outputs use the same shape: X[v * ldo + b].
 */
#ifndef EMO_H_
#define EMO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EMO_OK 0
#define EMO_E_INVALID_ARG (-1)     /* NULL where a pointer is required, negative size, bad ld */
#define EMO_E_NOT_TOPOLOGICAL (-2) /* an edge does not go from a lower to a higher node number */
#define EMO_E_RANGE (-3)           /* value outside the supported range (level >= L, lat >= 2^32, ...) */
#define EMO_E_OVERFLOW (-4)        /* the slowest-level makespan does not stay below 2^62 ns */
#define EMO_E_NONFINITE (-5)       /* NaN or infinity in the energy table */
#define EMO_E_OOM (-6)             /* host or device allocation failed, or workspace too small */
#define EMO_E_CUDA (-7)            /* a CUDA runtime call failed (no device, launch error, ...) */
#define EMO_E_TIMEOUT (-8)         /* a bounded device-side wait ran out; results are invalid */
#define EMO_E_UNSUPPORTED (-9)     /* the call has no path for these arguments (for example time-interval policies on a graph
                                      that only the generic kernels can take) */

/* flags of emo_graph_load */
#define EMO_F_HOST_ONLY 0x1u       /* build the handle without touching a device (inspection) */
#define EMO_F_LANES(c) (((uint32_t)(c) & 0xFFu) << 8)      /* force c cooperating warps per policy group */
#define EMO_F_LOOKAHEAD(d) (((uint32_t)(d) & 0xFFu) << 16) /* scheduling look-ahead in steps */
#define EMO_F_FLOW_SYNC(s) ((((uint32_t)(s) / 8u) & 0xFu) << 4)  /* lane-stream program: steps between group barriers (8, 16, 32;
                                                                  * default: one per stage where four policy groups then still fit a block, else 16) */
#define EMO_F_FLOW_STAGE(k) (((uint32_t)(k) & 0x3Fu) << 24)      /* lane-stream program: steps per stage (8, 16, 32) */
#define EMO_F_SPINE_STAGE(k) ((uint32_t)((k) == 8 ? 1u : ((k) == 32 ? 3u : 2u)) << 30)   /* spine program: steps per stage (8, 16, 32) */
#define EMO_F_INTERVALS 0x2u       /* also prepare the lane-stream form of emo_eval_intervals (a second copy of the forward program on
                                      the device); without it that call runs its step-program kernel */
#define EMO_F_GENERIC 0x4u         /* skip the schedule compilers: the generic kernels evaluate the graph (they also take every
                                      graph whose simultaneously live values exceed the on-chip exchange slots) */
/* flags of the evaluation calls */
#define EMO_F_VALIDATE 0x1u        /* check every level < L first; EMO_E_RANGE goes to *status */
#define EMO_F_NO_STAGING 0x2u      /* use the plain-load kernels instead of the staged ones */
#define EMO_F_PAIR_KERNEL 0x4u     /* staged pass kernel with two policies per thread (default only for very large batches) */
#define EMO_F_LANE_KERNEL 0x8u     /* staged pass kernel with one policy per thread (the default otherwise) */
#define EMO_F_FLOW_KERNEL 0x10u    /* the 32-bit lane-stream kernels (the default for large batches: n * B >= 2^31, or more than three
                                    * policy groups of 32 per SM on a graph of at most eight lanes) */
#define EMO_F_SPINE_KERNEL 0x20u   /* the spine kernels (the default on graphs of at most eight lanes while the batch leaves at most
                                    * three policy groups of 32 to an SM, or the graph has at most 8 192 nodes) */
#define EMO_F_TEST_STALL 0x100u    /* test hook of the 32-bit kernels: the producer warps stop half way, so that the
                                      consumers' bounded waits run out and EMO_E_TIMEOUT is reported */

typedef struct emo_graph emo_graph;

typedef struct emo_info {
    int32_t n;          /* nodes */
    int64_t m;          /* edges as given (duplicates included) */
    int32_t L;          /* frequency levels */
    int32_t rows;       /* policy rows (max group + 1, or n) */
    int32_t depth;      /* number of hop-count levels */
    int32_t max_span;   /* largest v - pred(v) in the caller's numbering */
    int64_t T_worst;    /* makespan with every node at its slowest level */
    int64_t T_best;     /* makespan with every node at its fastest level */
    int32_t lanes;      /* warps that cooperate on one group of policies, forward program */
    int32_t steps_fwd, slots_fwd, aux_fwd;   /* forward program: steps, exchange slots, helper ops */
    int32_t steps_bwd, slots_bwd, aux_bwd;   /* backward program */
    int32_t lanes_bwd;  /* cooperating warps of the backward program */
    int32_t sync_fwd, sync_bwd;   /* steps between two barriers of a group's warps (8, 16 or 32) */
} emo_info;

/* Human-readable text for a status code (static storage). */
const char *emo_strerror(int code);

/*
 * emo_graph_load - take an execution graph (Sec. 4.3: nodes are execution primitives, an edge
 * (i, j) means i must finish before j starts) with its frequency-indexed tables (Eq. 3) and
 * prepare it for evaluation.
 *   n, row_ptr[n+1], col[m]   host. Predecessor CSR: predecessors of v are col[row_ptr[v] ..
 *                             row_ptr[v+1]).  Nodes must be numbered topologically (every
 *                             predecessor < v); level-ordered numbering is the usual case.
 *                             Duplicate edges and isolated nodes are allowed.
 *   level_ptr[n_levels+1]     host, optional (NULL): node ranges of the caller's levels; when given
 *                             it is checked (every predecessor in a strictly lower level).
 *   L                         1..255 levels.
 *   lat[n][L]                 host, int64 ns, 0 <= lat < 2^32.
 *   energy[n][L]              host, fp64, finite.
 *   group_of[n]               host, optional: policy row of each node; -1 = the node ignores the
 *                             policy and uses table column 0.
 *   flags                     EMO_F_* of emo_graph_load.
 *   out                       receives the handle.
 * Everything is copied; the caller may free its arrays on return.  The device copies belong to
 * the handle until emo_graph_free.  Not asynchronous: it synchronises the device copies it makes.
 * A graph whose simultaneously live exchanged values exceed what the on-chip schedules can hold still loads:
 * the generic kernels (one thread per policy, completion times in the workspace, [n][B] int64 per pass)
 * evaluate it, exactly but slower; emo_call_path reports 3 for such a handle, emo_eval_intervals and
 * emo_search_dp return EMO_E_UNSUPPORTED on it.
 * Errors: INVALID_ARG, NOT_TOPOLOGICAL, RANGE, OVERFLOW, NONFINITE, OOM, CUDA.
 */
int emo_graph_load(int32_t n, const int64_t *row_ptr, const int32_t *col,
                   const int32_t *level_ptr, int32_t n_levels, int32_t L,
                   const int64_t *lat, const double *energy, const int32_t *group_of,
                   uint32_t flags, emo_graph **out);

/* Release a handle and its device memory.  NULL is allowed. */
int emo_graph_free(emo_graph *g);

/* Sizes and derived facts of a loaded graph. */
int emo_graph_info(const emo_graph *g, emo_info *info);

/*
 * emo_workspace_bytes - device scratch a call on B policies needs.  need_slack = 0 gives the size
 * for emo_eval_policies, emo_baseline and emo_select; 1 the size emo_slack_batch needs when the
 * caller passes no ES array (the earliest start times are then kept in the workspace between the
 * two passes); 2 the size emo_slack_batch_host needs.  The caller allocates; no call allocates
 * device memory per invocation.
 */
int emo_workspace_bytes(const emo_graph *g, int64_t B, int need_slack, size_t *out);

/*
 * emo_workspace_bytes_for - the same for a call that passes `flags` (EMO_F_* of the evaluation calls:
 * they choose the kernels, and the kernels differ in what they keep between the two passes) and a
 * level matrix that is (aligned = 1) or is not (aligned = 0) fetchable in 16-byte pieces: pointer
 * 16-byte aligned and ldb a multiple of 16.  emo_workspace_bytes assumes no flags and an aligned
 * matrix.  A workspace that is too small for what the call ends up running gives EMO_E_OOM.
 */
int emo_workspace_bytes_for(const emo_graph *g, int64_t B, int need_slack, uint32_t flags, int aligned,
                            size_t *out);

/*
 * emo_eval_policies - Alg. 1 without the idle-energy loop, for B policies at once:
 * makespan[b] = max_v C_v (Eq. 1, Eq. 2) and energy[b] = sum_v e_v (Eq. 2) under policy b.
 *   lvl          device uint8 [rows][ldb], ldb >= B.
 *   makespan     device int64 [B];  energy  device fp64 [B].
 *   ws, ws_bytes device scratch of at least emo_workspace_bytes(g, B, 0).
 *   T0, E0       device int64 [1] / fp64 [1], optional: when given, the default policy P_0 (every
 *                row at level L-1, Alg. 2 line 1) is evaluated in the same launch as one more
 *                column and its makespan and energy are written here.
 *   status       device int32, optional: set to a negative code if a kernel detected an error
 *                (left untouched otherwise; the caller zeroes it).
 * B == 0 writes nothing but T0 / E0.  Asynchronous on `stream`.
 */
int emo_eval_policies(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb,
                      int64_t *makespan, double *energy, int64_t *T0, double *E0,
                      void *ws, size_t ws_bytes, int32_t *status, uint32_t flags, void *stream);

/*
 * emo_eval_intervals - Alg. 1 with time-interval policies P = {<T_i, F_i>} and the idle energy of Eq. 2,
 * for B policies at once.  The level of a node is the one of the interval that holds its START time
 * (Alg. 1: "f <- F_i where start in [T_i, T_{i+1})"; half-open, the last interval has no end), so a node's
 * duration depends on the recurrence of Eq. 1 itself.  Each device has its own policy (Sec. 4.3): the graph's
 * group_of (emo_graph_load) names the device row of every pack; a node with group_of = -1 is outside every
 * policy and uses column 0 of its tables (the fixed t_v and the zero energy Alg. 1 gives such nodes).
 *   F            device uint8 [rows][I][ldb]: row r, interval i, policy b at F[(r*I + i)*ldb + b]; ldb >= B;
 *                levels must be < L (a larger value is masked into the table, never read out of bounds).
 *   I, breaks    number of intervals (1..4096) and their change points T_1 < T_2 < ..., HOST int64 [I] in
 *                nanoseconds with breaks[0] = 0; the same for every policy of the batch.  Copied by the call.
 *   p_idle       device fp64 [L], idle power in watts at each level, or NULL (no idle energy).
 *   makespan     device int64 [B]: max_v C_v (Eq. 2).
 *   energy       device fp64 [B]: sum_v e_v + E_idle (Eq. 2; E_idle = 0 without p_idle).
 *   energy_idle  device fp64 [B], optional: E_idle alone.  Requires p_idle.
 *   ws           device scratch of at least emo_workspace_bytes_intervals(g, B, I, p_idle != NULL).
 * E_idle (Alg. 1, last loop) = sum over rows and intervals of idle_time x p_idle[F_i], where idle_time is the
 * part of the interval below the makespan minus the summed overlap of the row's packs with it, not below zero
 * (exact when the packs of a device do not overlap in time, as packs of one device timeline do not; the paper
 * does not define idle_time further).
 * Kernels: a graph loaded with EMO_F_INTERVALS runs the 32-bit lane-stream kernel when the change points are a
 * uniform grid and the columns of F fit shared memory; otherwise, or with EMO_F_NO_STAGING in flags, the
 * step-program kernel runs.  Both give the same results.
 * Errors: EMO_E_INVALID_ARG (sizes, breaks not increasing from 0, energy_idle without p_idle), EMO_E_OOM
 * (workspace too small), EMO_E_UNSUPPORTED (change points and exchange slots do not fit shared memory).
 * Asynchronous on `stream` after the change points are copied.
 */
int emo_eval_intervals(const emo_graph *g, int64_t B, const uint8_t *F, int64_t ldb, int32_t I,
                       const int64_t *breaks, const double *p_idle, int64_t *makespan, double *energy,
                       double *energy_idle, void *ws, size_t ws_bytes, int32_t *status, uint32_t flags,
                       void *stream);
int emo_workspace_bytes_intervals(const emo_graph *g, int64_t B, int32_t I, int with_idle, size_t *out);

/*
 * emo_pack_greedy - kernel packing (Sec. 4.4): the critical predecessor of every node at the default frequency
 * (Eq. 5: k*_v = argmax over predecessors of C_k; among equals the lowest index, the one Alg. 1's update meets
 * first) and the dependency-aware greedy packing of GPU kernels.  The kernels of every stream are walked in
 * index order; kernel v joins the open pack of its stream (last member u) while (1) v's critical predecessor is
 * a kernel of v's stream, (2) every node whose critical predecessor is u is a kernel of u's stream, and (3) the
 * pack's duration at the default frequency plus t_v stays below delta_max; otherwise v opens a new pack.
 * Host function, host arrays; nothing touches a device.
 *   row_ptr, col   predecessor CSR in a topological numbering (every predecessor has a lower index).
 *   is_kernel      uint8 [n]: 1 for GPU kernels (only they are packed).
 *   stream_of      int32 [n]: global stream id (device and stream together) of every kernel, >= 0; ignored elsewhere.
 *   t_default      int64 [n]: durations at the default frequency, ns.
 *   delta_max      granularity bound in ns (the paper uses 5 ms).
 *   crit_out       int32 [n], optional: the critical predecessors (-1: none).
 *   pack_of        int32 [n]: pack number of every kernel (0, 1, ... in order of the packs' first members), -1
 *                  for other nodes.  Usable as group_of of emo_graph_load for per-pack policies after the
 *                  non-kernel nodes are given rows of their own (or -1).
 *   n_packs        number of packs.
 * Errors: EMO_E_INVALID_ARG, EMO_E_NOT_TOPOLOGICAL, EMO_E_RANGE (negative duration), EMO_E_OOM.
 */
int emo_pack_greedy(int32_t n, const int64_t *row_ptr, const int32_t *col, const uint8_t *is_kernel,
                    const int32_t *stream_of, const int64_t *t_default, int64_t delta_max, int32_t *crit_out,
                    int32_t *pack_of, int32_t *n_packs);
/*
 * emo_pack_tables - the packs' frequency tables: per level the sum of the members' table entries (a pack's
 * kernels run one after the other on their stream).  pack_lat int64 [n_packs][L], pack_energy fp64 [n_packs][L];
 * members are added in index order.  Host function.
 */
int emo_pack_tables(int32_t n, int32_t L, const int64_t *lat, const double *energy, const int32_t *pack_of,
                    int32_t n_packs, int64_t *pack_lat, double *pack_energy);

/*
 * emo_pack_model - pack modelling (Sec. 4.5) for a batch of packs on the GPU.  Eq. 6: the weights of pack p are
 * x_p = argmin ||B x - b_p||^2 subject to x >= 0, with B the metric matrix of the m micro-benchmarks and b_p the
 * pack's feature vector at the default frequency; Eq. 7: its tables are T_f[P] = sum_i x_i T_f[B_i] and
 * E_f[P] = sum_i x_i E_f[B_i].  One thread per pack (active-set method on the normal equations, fp64).
 *   Bmat   device fp64 [n_metrics][m], m <= 16;  feat  device fp64 [n_packs][n_metrics].
 *   Tb, Eb device fp64 [m][L]: the micro-benchmarks' latency (ns) and energy (J) at every level.
 *   x      device fp64 [n_packs][m];  T_out, E_out  device fp64 [n_packs][L] (the caller rounds latencies to
 *          whole ns for emo_graph_load).
 *   status device int32, optional: EMO_E_UNSUPPORTED (-9) if a fit did not settle within its iteration bound.
 * The minimiser is unique when B has independent columns (n_metrics >= m in practice); otherwise any minimiser
 * may come out.  Errors: EMO_E_INVALID_ARG, EMO_E_UNSUPPORTED (tables and matrices beyond 48 KB of shared
 * memory).  Asynchronous on `stream`.
 */
int emo_pack_model(int32_t n_packs, int32_t n_metrics, int32_t m, int32_t L, const double *Bmat, const double *feat,
                   const double *Tb, const double *Eb, double *x, double *T_out, double *E_out, int32_t *status,
                   void *stream);

/*
 * emo_pack_classes - pack-level sampling (Sec. 4.4, last paragraph): packs whose kernels carry the same sequence
 * of names are one class, and only the first pack of every class needs profiling.  name_id int32 [n] gives every
 * kernel's name as a number (the caller interns the strings); class_of_pack int32 [n_packs] receives the class of
 * every pack, classes numbered by their first pack; n_classes their count.  Exact comparison of the sequences (the
 * paper hashes them; a hash collision would merge different packs).  Host function.
 */
int emo_pack_classes(int32_t n, const int32_t *pack_of, const int32_t *name_id, int32_t n_packs, int32_t *class_of_pack,
                     int32_t *n_classes);

/*
 * emo_search_dp - Alg. 2: search for a near-optimal time-interval policy by dynamic programming over the
 * intervals, with emo_eval_intervals (Alg. 1) as the predictor.  dp[i] maps an end-to-end time to the least
 * energy and its policy after the first i intervals are decided; every state is extended by every level in
 * interval i, the |dp[i]| x L candidates of a stage are predicted as one batch on the GPU (in chunks of
 * max_batch), and a candidate replaces its time's entry only if it meets T_max and is strictly better
 * (candidates in the order of Alg. 2: states by ascending time, levels ascending).  The answer is the entry of
 * dp[I] of least energy (Alg. 2, last line).
 *   I, breaks     the intervals [p_i, p_{i+1}) as change points, HOST int64 [I], breaks[0] = 0 (as in
 *                 emo_eval_intervals); one policy governs every device row (the paper drops the GPU index here
 *                 and replicates one GPU's policy, Sec. 6.2).
 *   p_idle        device fp64 [L] or NULL, as in emo_eval_intervals.
 *   T_max         the constraint in ns (emo_target_from_delta gives it from T_0 and a budget).
 *   bin_ns        >= 1: times are keyed as floor(t / bin_ns) (Sec. 4.6 discretises the constraint, "e.g., 1 ms";
 *                 1 keeps exact times).  The number of states per stage is at most (T_max - t_min) / bin_ns + 1.
 *   max_batch     candidates per evaluation call (0: 16384); sizes the workspace.
 *   F_best        HOST uint8 [I]: the chosen level of every interval; T_best, E_best HOST scalars; n_pred HOST:
 *                 predictions made; found HOST: 0 when no candidate met T_max (the other outputs are then untouched).
 *   ws            device scratch of at least emo_workspace_bytes_search(g, I, max_batch, p_idle != NULL).
 * The default policy P_0 is level L-1 everywhere; dp[0] is seeded with it without a test (Alg. 2 line 3).
 * Synchronous: the call waits for every stage's results.  Errors as emo_eval_intervals.
 */
int emo_search_dp(const emo_graph *g, int32_t I, const int64_t *breaks, const double *p_idle, int64_t T_max,
                  int64_t bin_ns, int64_t max_batch, uint8_t *F_best, int64_t *T_best, double *E_best,
                  int64_t *n_pred, int32_t *found, void *ws, size_t ws_bytes, void *stream);
int emo_workspace_bytes_search(const emo_graph *g, int32_t I, int64_t max_batch, int with_idle, size_t *out);

/*
 * emo_slack_batch - forward and backward pass for B policies: earliest start ES, latest start LS
 * (critical-path backward pass: LF_v = min over successors of LS_u, the makespan for nodes
 * without successors; LS_v = LF_v - t_v) and slack = LS - ES per node and policy.
 *   ES, LS, slack   device int64 [n][ldo], each optional (NULL); ldo >= B.
 *   makespan, energy device [B] (required).
 *   slack_sum       device int64 [B], optional: sum of slack over nodes.
 *   n_critical      device int32 [B], optional: number of nodes with slack 0.
 *   T0, E0          optional, as in emo_eval_policies.
 *   ws              at least emo_workspace_bytes(g, B, ES == NULL).
 * Asynchronous on `stream`.
 */
int emo_slack_batch(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb,
                    int64_t *ES, int64_t *LS, int64_t *slack, int64_t ldo,
                    int64_t *makespan, double *energy, int64_t *slack_sum, int32_t *n_critical,
                    int64_t *T0, double *E0,
                    void *ws, size_t ws_bytes, int32_t *status, uint32_t flags, void *stream);

/*
 * emo_slack - one policy: lvl_one is device uint8 [rows]; ES, LS, slack are device int64 [n]
 * (each optional); makespan device int64 [1], energy device fp64 [1] (optional).
 */
int emo_slack(const emo_graph *g, const uint8_t *lvl_one, int64_t *ES, int64_t *LS, int64_t *slack,
              int64_t *makespan, double *energy, void *ws, size_t ws_bytes, int32_t *status,
              void *stream);

/*
 * emo_baseline - T_0 and E_0 of the default policy, every row at level L-1 (Alg. 2 line 1-2:
 * P_0 = default frequency everywhere; Sec. 4.6: T_0 is the latency at maximum frequency).
 * T0 device int64 [1], E0 device fp64 [1].
 */
int emo_baseline(const emo_graph *g, int64_t *T0, double *E0, void *ws, size_t ws_bytes,
                 int32_t *status, void *stream);

/* T_set = T0 + floor(T0 * delta_ppm / 10^6), exact in 128-bit.  Pure host function. */
int64_t emo_target_from_delta(int64_t T0, int64_t delta_ppm);

/*
 * emo_select - Eq. 4 over the batch: the index of the least-energy policy among those with
 * makespan[b] <= target; equal energies go to the lowest index (the strict-improvement test of
 * Alg. 2 keeps the incumbent).  out_index receives -1 when no policy is feasible (still EMO_OK).
 *   makespan, energy  device [B];  out_index device int64 [1];  out_T device int64 [1] and
 *   out_E device fp64 [1] (optional) receive the selected policy's values.
 *   target_dev        optional device int64 [1]: when not NULL the target is read from it on the
 *                     device (so a budget computed from emo_baseline needs no host round trip)
 *                     as target_dev[0] + floor(target_dev[0] * delta_ppm / 10^6) and `target` is
 *                     ignored; when NULL, `target` is used and delta_ppm ignored.
 */
int emo_select(int64_t B, const int64_t *makespan, const double *energy, int64_t target,
               const int64_t *target_dev, int64_t delta_ppm,
               int64_t *out_index, int64_t *out_T, double *out_E,
               void *ws, size_t ws_bytes, void *stream);

/*
 * emo_select_static - emo_select for callers that must not allocate.  (The paper has no counterpart;
 * this is a packaging variant of the selection above.)  Some callers cannot call cudaMalloc or any
 * allocating routine: code running inside a latency-critical control loop that must not take the
 * driver's allocation lock, a plug-in that was handed a stream but owns no memory pool, or a process
 * whose device memory is fully pre-partitioned.  For them the scratch that emo_select takes as `ws`
 * (one candidate per thread block) lives in a 16 KiB array inside the library, held by every GPU
 * that loads the library until the process exits.
 *   Arguments as emo_select, without ws.  B must not exceed EMO_SELECT_STATIC_MAX_B
 *   (else EMO_E_RANGE); inputs and outputs are still the caller's device arrays.
 *   The first call on a device looks up the array's device address (with that device current);
 *   make that first call before any stream capture.  The call itself allocates nothing.
 *   All calls on a device share the one array: calls whose kernels may overlap on the GPU (two
 *   streams, two threads) race and give wrong results; serialise them.  The array keeps the last
 *   call's candidates; every call overwrites what it later reads, so no clearing is needed.
 */
#define EMO_SELECT_STATIC_MAX_B 1048576
int emo_select_static(int64_t B, const int64_t *makespan, const double *energy, int64_t target,
                      const int64_t *target_dev, int64_t delta_ppm,
                      int64_t *out_index, int64_t *out_T, double *out_E, void *stream);

/*
 * emo_transpose_policies - layout helper: src device uint8 [B][lds] (one policy per row) to
 * dst device uint8 [rows][ldb].
 */
int emo_transpose_policies(int64_t B, int64_t rows, const uint8_t *src, int64_t lds,
                           uint8_t *dst, int64_t ldb, void *stream);

/*
 * emo_slack_batch_host - the same computation as emo_slack_batch followed by emo_baseline and
 * emo_select, driven from host memory: lvl_host is host uint8 [rows][ldb] (pinned memory gives
 * the best copy rate); makespan_host, energy_host, slack_sum_host, n_critical_host are host
 * arrays [B] (the last two optional); sel_host receives {index, T, E-bits, T0} as 4 int64.
 * slack_dev (device int64 [n][ldo], optional) stays on the device.  dev_lvl is a device buffer
 * of rows*ldb bytes and ws a device workspace of emo_workspace_bytes(g, B, 2).
 * The call copies the levels in, runs the passes, copies the per-policy results out and waits
 * for the stream.
 */
int emo_slack_batch_host(const emo_graph *g, int64_t B, const uint8_t *lvl_host, int64_t ldb,
                         uint8_t *dev_lvl, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm,
                         int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                         int32_t *n_critical_host, int64_t *sel_host,
                         void *ws, size_t ws_bytes, uint32_t flags, void *stream);

/*
 * Levels packed at `bits` bits each (1..8; a level needs ceil(log2 L) bits): a layout for moving
 * policies over the bus.  In a packed row, eight consecutive levels take `bits` consecutive bytes, the
 * first level in the lowest bits; a row of B levels takes ceil(B / 8) * bits bytes (pitch ldp).
 * emo_pack_levels: device byte matrix lvl [rows][ldb] -> device packed [rows][ldp];
 * emo_unpack_levels the other way (levels beyond B up to the next multiple of 8 are written too).
 * ldb a multiple of 8, lvl 8-byte aligned.  Layout helpers: no counterpart in the method.
 */
int emo_pack_levels(int bits, int64_t rows, int64_t B, const uint8_t *lvl, int64_t ldb,
                    uint8_t *packed, int64_t ldp, void *stream);
int emo_unpack_levels(int bits, int64_t rows, int64_t B, const uint8_t *packed, int64_t ldp,
                      uint8_t *lvl, int64_t ldb, void *stream);

/*
 * emo_slack_batch_host_packed - emo_slack_batch_host with the levels in host memory packed at `bits`
 * bits each (see emo_pack_levels; bits = 8: plain bytes, ld_host must equal ldb and dev_packed is not
 * used): lvl_host is host [rows][ld_host], dev_packed a device buffer of rows * ld_host bytes, dev_lvl
 * the device byte matrix [rows][ldb] the levels are spread into before the passes run.  With 5 bits
 * (32 levels) 0.625 bytes per level cross the bus instead of 1.  Everything else as emo_slack_batch_host.
 */
int emo_slack_batch_host_packed(const emo_graph *g, int64_t B, int bits, const uint8_t *lvl_host, int64_t ld_host,
                                uint8_t *dev_packed, uint8_t *dev_lvl, int64_t ldb, int64_t *slack_dev, int64_t ldo,
                                int64_t delta_ppm, int64_t *makespan_host, double *energy_host,
                                int64_t *slack_sum_host, int32_t *n_critical_host, int64_t *sel_host,
                                void *ws, size_t ws_bytes, uint32_t flags, void *stream);

/*
 * The same in two halves, so that the copy of the next batch runs under the kernels of the current one
 * (two device buffers of packed levels, a copy stream of the caller's):
 * emo_levels_prefetch enqueues the host -> device copy of packed levels (rows * ld_host bytes, bits < 8 as in
 * emo_slack_batch_host_packed; lvl_host should be pinned) on copy_stream and records `ready` (a cudaEvent_t as
 * void*) behind it; it returns at once.
 * emo_slack_batch_prefetched is emo_slack_batch_host_packed without the copy: `stream` waits for `ready`, then the
 * levels in dev_packed (pitch ld_packed) are spread to dev_lvl and everything else follows as there, including the
 * wait for the stream at the end.  The caller must not start a prefetch into a buffer before the call that reads it
 * has returned.
 */
int emo_levels_prefetch(const emo_graph *g, const uint8_t *lvl_host, int64_t ld_host, uint8_t *dev_packed, void *copy_stream,
                        void *ready);
int emo_slack_batch_prefetched(const emo_graph *g, int64_t B, int bits, const uint8_t *dev_packed, int64_t ld_packed, void *ready,
                               uint8_t *dev_lvl, int64_t ldb, int64_t *slack_dev, int64_t ldo, int64_t delta_ppm,
                               int64_t *makespan_host, double *energy_host, int64_t *slack_sum_host,
                               int32_t *n_critical_host, int64_t *sel_host, void *ws, size_t ws_bytes, uint32_t flags,
                               void *stream);

/*
 * emo_set_pass_events - measurement hook (no counterpart in the method): four cudaEvent_t handles
 * (as void*, any may be NULL) that later emo_slack_batch / emo_eval_policies / emo_baseline calls
 * record on their stream immediately before and after the forward pass kernel and before and after
 * the backward pass kernel.  Pass four NULLs to switch it off.  Process-wide, not thread-safe.
 */
int emo_set_pass_events(void *fwd_start, void *fwd_stop, void *bwd_start, void *bwd_stop);

/*
 * emo_call_path - which kernels emo_eval_policies (need_slack = 0) or emo_slack_batch (need_slack = 1)
 * would run for these arguments: 4 = the spine kernels, 5 = the forward spine kernel followed by the lane-stream backward
 * kernel, 2 = the 32-bit lane-stream kernels, 1 = the staged 64-bit kernels,
 * 0 = the plain-load 64-bit kernels, 3 = the generic kernels (a graph beyond the on-chip schedules' limits, or
 * loaded with EMO_F_GENERIC); negative = an EMO_E_* code.  lvl may be any pointer with the
 * alignment of the real one.  For tests and reports; it launches nothing.
 */
int emo_call_path(const emo_graph *g, int64_t B, const uint8_t *lvl, int64_t ldb, int64_t ldo,
                  int need_slack, uint32_t flags);

/*
 * emo_measure_int_issue - measurement helper (no counterpart in the method): the rate at which this GPU
 * issues the integer operations of the recurrences (Eq. 1 is one add per node and one max per edge).
 * Runs four small kernels of independent dependent-chains that fill every SM and writes warp-level
 * operations per second to ops_per_s[4] (host): 32-bit add, 32-bit max, 64-bit add, 64-bit max.
 * scratch_dev: device memory of at least 8 bytes.  Synchronises the stream.
 */
int emo_measure_int_issue(double *ops_per_s, void *scratch_dev, void *stream);

/*
 * emo_measure_warp_costs - measurement helper (no counterpart in the method): what one warp alone pays, in
 * SM cycles, for the steps the pass kernels are made of.  The recurrences (Eq. 1 and its mirror) are walked
 * as a dependency chain of as many steps as the graph is deep, with a few warps per scheduler, so these
 * latencies and not a pipe's throughput set the kernels' speed.  Writes cycles[8] (host): dependent 32-bit
 * add; dependent max then subtract; dependent shared-memory load; independent adds (issue interval); a loop
 * body of one shared load and four dependent operations with a never-taken branch on the loaded word; the
 * same body without the branch; redux.sync then add; a named barrier of five warps.
 * scratch_dev: device memory of at least 128 bytes.  Synchronises the stream.
 */
int emo_measure_warp_costs(double *cycles, void *scratch_dev, void *stream);

/*
 * emo_set_flow_counters - measurement hook (no counterpart in the method): a device array of 262144
 * int64 that later calls of the 32-bit kernels fill with cycle counts, 8 per warp at
 * [((pass * 512 + block) * 32 + warp) * 8] for the first 512 blocks (pass 0 forward, 1 backward): consumer
 * warps {cycles waiting for staged data, cycles at group barriers, total, backward only: cycles in
 * entries that need their record, cycles in runs of simple entries}, producer warps {cycles waiting
 * for a free buffer, cycles issuing copies, total}; the other words are spare.  The spine kernels fill the same
 * array: spine warps {waiting for staged data, waiting for the workers' sums, total, inside the operation loop,
 * backward: waiting for the stores two stages back}, forward workers {waiting for staged data, waiting for a free
 * buffer of sums, total}, backward workers {both of those, waiting for the spine, total, sums, stores}.
 * NULL switches it off.  Process-wide.
 */
int emo_set_flow_counters(void *dev);

/*
 * emo_set_wait_limit - bound, in SM clock cycles, of every device-side wait of the 32-bit pass kernels
 * (a wait on a stage of staged data or on a value another warp produces).  A wait that runs out ends
 * the kernel with EMO_E_TIMEOUT in *status instead of hanging.  Default 4 * 10^9 (about two seconds);
 * tests use a small value.  Process-wide; applies to calls made afterwards.
 */
int emo_set_wait_limit(int64_t cycles);

/*
 * Inspection of the compiled evaluation program (host memory owned by the handle; valid until
 * emo_graph_free).  dir 0 = forward, 1 = backward.  entries is [steps][lanes][8] uint32, rows is
 * uint32 [steps*lanes] (policy row read by the entry, 0xFFFFFFFF = none), lat is uint32
 * [steps*lanes][Lp], Lp = row stride (a power of two >= max(L, 4)).  Used by host-side tests of
 * the scheduler; not needed to evaluate anything.
 */
int emo_graph_program(const emo_graph *g, int dir, int32_t *lanes, int32_t *steps, int32_t *slots,
                      int32_t *Lp, const uint32_t **entries, const uint32_t **rows, const uint32_t **lat);

/*
 * Inspection of the lane-stream program that the 32-bit pass kernels walk (host memory owned by the
 * handle; valid until emo_graph_free).  ok32 = 0 means the graph's spread of start times over all
 * policies does not fit 32 bits (or it needs more than 30 lanes) and the 64-bit kernels serve it;
 * the arrays are then empty.  Layouts: hdr [stages][lanes][8], rows / node / step [stages][lanes][K],
 * tab_fwd [stages][lanes][K][Lp][3], tab_bwd [stages][lanes][K][Lp], rec_fwd [stages][lanes][K][8],
 * rec_bwd [stages][lanes][K][12], pool_* [stages][pool_stride_*], seg_* [stages][lanes][40] (bytes),
 * lbes [stages][lanes][K],
 * push_base [stages + 1].  Used by host-side tests of the compiler; not needed to evaluate anything.
 */
typedef struct emo_flow_view {
    int32_t ok32, lanes, K, sync, stages, steps, Lp;
    int32_t slots_tag_fwd, slots_set_fwd, pool_stride_fwd;
    int32_t slots_tag_bwd, slots_set_bwd, pool_stride_bwd;
    int64_t pushes, pruned_fwd, pruned_bwd;
    const uint32_t *hdr, *rows, *node, *step, *tab_fwd, *tab_bwd;
    const uint32_t *rec_fwd, *pool_fwd, *rec_bwd, *pool_bwd;
    const uint8_t *seg_fwd, *seg_bwd;
    const int64_t *lbes, *push_base;
} emo_flow_view;
int emo_graph_flow(const emo_graph *g, emo_flow_view *out);

/* Sizes of the spine program (the form of the schedule that the spine kernels walk: consecutive nodes of a
 * lane that are linked only to each other form a segment, whose members share one slack; Eq. 1 runs through
 * one operation per segment).  out[0] = 1 if the program exists (else the rest is 0), then lanes, steps per
 * stage, stages, segments, forward operations, backward operations, forward value slots, backward value
 * slots, most segments of a stage, 4-byte words of sums per policy and stage, restore rows.  Host memory. */
int emo_graph_spine(const emo_graph *g, int64_t out[12]);

/* The spine program itself, as pointers into the handle's host memory (valid until emo_graph_free; for the host-side
 * tests of the compiler, which interpret it).  Arrays: n_ops_fwd / n_ops_bwd [stages]; ops_fwd [stages][max_ops_fwd][8]
 * = {operand slot 0, its correction, operand slot 1, its correction, the lane's slot, published slot, offset of the
 * segment's sum, flags (1 = sum is zero, 2 = push to the restore list, 4 = terminal) | restore row in the stage << 8 |
 * index of the terminal bound << 20}, slots and sums as byte offsets in units of 128; ops_bwd [stages][max_ops_bwd][12]
 * = the same eight (2 = pop), then {slot to clear, slot of the lane's completion offset, offset where the head's tail
 * goes, spare}; mem [stages][lanes * K][8] = {node (0xFFFFFFFF: unused position), fold slot, fold correction, position
 * word (bit 0 first member, bit 1 last member of its segment, bits 16..31 offset of the segment's sum in units of 128
 * bytes), A_v low, high, lbES_v low, high}; pos [stages][lanes * K] the position words alone; pool [stages][max_pool]
 * lower bounds of terminal completions; push_base [stages + 1]; rows [stages][lanes][K] policy row of a position
 * (0xFFFFFFFF: none); tab_fwd [stages][lanes][K][Lp][3] = {duration - dmin, energy high word, low word};
 * tab_bwd [stages][lanes][K][Lp]. */
typedef struct emo_spine_view {
    int32_t ok, lanes, K, stages, Lp, max_ops_fwd, max_ops_bwd, max_pool, acc_words, slots_fwd, slots_bwd;
    int64_t pushes;
    const uint32_t *n_ops_fwd, *ops_fwd, *n_ops_bwd, *ops_bwd, *mem, *pos, *rows, *tab_fwd, *tab_bwd;
    const uint64_t *pool;
    const int64_t *push_base;
} emo_spine_view;
int emo_graph_spine_view(const emo_graph *g, emo_spine_view *out);

#ifdef __cplusplus
}
#endif
#endif /* EMO_H_ */
