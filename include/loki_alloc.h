/*
 * loki_alloc -- candidate-scoring allocation search of Loki's Resource Manager
 * (Loki, HPDC '24, Section 4 "Resource Manager") as a CUDA library for sm_100a.
 *
 * The paper states the allocation problem as two mixed-integer programs
 * (Section 4.1, Eqs. 1-12).  This library solves the same constraint set over a
 * finite candidate space by exhaustive scoring on the GPU:
 *
 *   candidate   per task one option = (model variant, batch size), or in split
 *               mode an unordered pair of distinct options with a k/16 traffic
 *               split, k = 1..15 (the allocation plan of Section 2.2.1:
 *               variants, replica counts, maximum batch sizes);
 *   accuracy    product of task accuracies along each root-to-leaf path of the
 *               pipeline tree, averaged over the leaves (Section 2.1; objective
 *               Eq. 12);
 *   latency     for every root-to-leaf path  2 * sum lat <= slo_us - hops*comm_us
 *               (Eqs. 6-7, the halved SLO, and "Communication latency", Sec. 4.2);
 *   demand      stage demand = root demand times the fan-out factors of the edges
 *               above the task, rounded up per edge (Eq. 1);
 *   workers     per part ceil(demand_mqps * share/16 * lat_us / (batch * 1e9))
 *               -- Eq. 2 with throughput q = batch / lat from Eq. 5;
 *   cluster     sum of workers <= cluster_size (Eq. 3);
 *   objective   highest accuracy, then fewest workers, then lowest candidate
 *               index (Eqs. 8-11 and Eq. 12 folded into one order).
 *
 * Candidate index: c = sum_i o_i * prod_{j<i} O_j, task 0 least significant.
 * Option index of a task with nS = n_variants*n_batches single options:
 *   o <  nS : single option, variant o / n_batches, batch index o % n_batches;
 *   o >= nS : split option, pair rank (o-nS)/15 in lexicographic order of
 *             (o1 < o2), share k = (o-nS)%15 + 1 sixteenths to o1, the rest to o2.
 * Split task accuracy is A2 + (k/16)*(A1 - A2) in three rounded double
 * operations; split task latency is the larger of the two parts.
 *
 * All functions return LOKI_OK or a negative error code; nothing is thrown and
 * no function terminates the process.  Unless stated, pointers are HOST memory.
 * The library has no CPU fallback: without a usable CUDA device
 * loki_alloc_create returns LOKI_ERR_CUDA.
 */
#ifndef LOKI_ALLOC_H_
#define LOKI_ALLOC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LOKI_MAX_TASKS 8

enum {
  LOKI_OK = 0,
  LOKI_ERR_INVALID_ARG = -1,   /* null pointer, count <= 0, value out of range        */
  LOKI_ERR_INVALID_GRAPH = -2, /* not a rooted tree in topological order (Sec. 2.1)   */
  LOKI_ERR_RANGE = -3,         /* the 64-bit overflow proof fails or the space is too big */
  LOKI_ERR_CUDA = -4,          /* a CUDA call failed (no device, launch error, ...)   */
  LOKI_ERR_NOMEM = -5          /* host or device allocation failed                    */
};

/* per-level status in loki_config_t */
enum {
  LOKI_LEVEL_FEASIBLE = 0,
  LOKI_LEVEL_INFEASIBLE = 1,   /* no candidate meets SLO and cluster size ("Effect of SLOs
                                  on system performance": demand that cannot be served) */
  LOKI_LEVEL_BAD_DEMAND = 2,   /* demand < 0 or > max_demand_mqps                     */
  LOKI_LEVEL_INTERNAL_ERROR = 3 /* self-check failed: the winning key and the plan decoded
                                   from it disagree on the worker count (never expected) */
};

/* scoring kernels selectable with loki_alloc_set_path */
enum {
  LOKI_PATH_AUTO = 0,     /* the default; decided per solve by this library's measurements: PREFIX
                             (HOISTED for a single task) wherever the class tables fit the shared-memory bound (72 KB for the
                             largest class tuple at 32 levels), except sweeps of at most 16 levels
                             over 2^20 candidates or more, where DIRECT is quicker; where the
                             tables do not fit, UNIFORM for 256 levels or more if its conditions
                             hold, else DIRECT; GENERIC where DIRECT's exactness and range
                             conditions fail.  With per-variant factors: UNIFORM, else GENERIC   */
  LOKI_PATH_GENERIC = 1,  /* 64-bit arithmetic with plain division; any accepted input          */
  LOKI_PATH_DIRECT = 2,   /* one FP64 fma (rounded down) per option part and pair for every
                             candidate within the latency bound; the key of the running argmax
                             is the worker sum, the index tie-break is resolved per level
                             after the cross-block reduction                                      */
  LOKI_PATH_HOISTED = 3,  /* per-option worker tables in shared memory, one add per pair: with one
                             fan-out factor per edge Eq. 2 depends on (level, task, option) only   */
  LOKI_PATH_UNIFORM = 4,  /* the DIRECT arithmetic with lanes holding demand levels and the
                             candidate uniform across the warp, the tasks walked root first: a
                             stage demand is derived from the parent's chosen option (so per-
                             variant factors are served), an outer task's workers are evaluated
                             once per move of its digit, latency-infeasible candidates are never
                             reached.  DIRECT's conditions, exact demand ratios and 12 KB of
                             shared memory for the largest class tuple                            */
  LOKI_PATH_FASTEST = 5,  /* the older name of what LOKI_PATH_AUTO does                           */
  LOKI_PATH_PREFIX = 6,   /* HOISTED's tables with the innermost loop replaced by one read: the
                             members of a class are laid out in ascending latency, so those that
                             fit the slack the outer tasks leave are a prefix, and the fewest
                             workers (lowest index on ties) over every prefix are tabulated once
                             per class tuple.  Same plans; the candidates of the innermost task
                             (or pair of tasks) are no longer visited one by one.  Where HOISTED
                             applies.  Sweeps of 2^28 (candidate, level) pairs or more take the
                             tables of LOKI_PATH_SHARED, shorter ones a table per class tuple      */
  LOKI_PATH_SHARED = 7    /* PREFIX with tables shared by all class tuples: one kernel tabulates,
                             per level tile, the workers of every member of every class (the
                             innermost rows as prefix minima) in global memory, a second one
                             walks the class tuples, a warp each.  Two tasks or more, one fan-out
                             factor per edge, tables of at most 256 MB for the longest sweep       */
};

typedef struct loki_alloc loki_alloc_t; /* opaque; owns device tables and scratch */

/* Problem statement: the inputs of Section 4.1 ("Inputs", Table 1).  Every array
 * is copied by loki_alloc_create; the caller may free it on return. */
typedef struct {
  int32_t n_tasks;              /* |T|, 1..LOKI_MAX_TASKS                                   */
  const int32_t* parent;        /* [n_tasks] parent[0] = -1, 0 <= parent[i] < i (rooted tree) */
  const int32_t* fanout_milli;  /* [n_tasks] multiplicative factor of edge parent[i]->i in
                                   thousandths (1000 = x1), >= 1; entry 0 is ignored        */
  const int32_t* n_variants;    /* [n_tasks] |V_i| >= 1                                     */
  int32_t n_batches;            /* |B| >= 1                                                 */
  const int32_t* batch_sizes;   /* [n_batches] strictly ascending, >= 1 (the set B, Eq. 4)  */
  const double* accuracy;       /* [sum n_variants] task-major A(v_ik); finite, > 0, <= 1   */
  const int64_t* latency_us;    /* [sum n_variants][n_batches] l(i,k) for each batch size in
                                   microseconds, > 0 (Eq. 5: l = b / q)                     */
  int64_t slo_us;               /* L, end-to-end latency SLO, >= 0                          */
  int64_t comm_us;              /* per-hop communication latency, >= 0                      */
  int32_t cluster_size;         /* S, 0 <= S < 2^24                                         */
  int32_t split_mode;           /* 0: one option per task; 1: also pairs with k/16 splits   */
  int64_t max_demand_mqps;      /* declared upper bound on demand (milli-queries/s), >= 0;
                                   used for the overflow proof                              */
  int32_t max_levels;           /* largest n_levels a solve call may pass, >= 1             */
  const int32_t* variant_fanout_milli; /* [sum n_variants] task-major r(i,k) of Eq. 1 in thousandths,
                                   1..2^20, or NULL for 1000 everywhere: every outgoing edge of a
                                   task carries parent demand x fanout_milli x r of the parent's
                                   chosen variant (k/16-weighted mean of the two in a split option).
                                   With factors other than 1000 AUTO resolves to the root-first
                                   level-lane kernel (UNIFORM), or to GENERIC where its conditions
                                   do not hold; DIRECT and HOISTED are refused.               */
} loki_alloc_desc_t;

/* One allocation plan (the output x(i,k), y(i,k) of Section 4.1) per demand level. */
typedef struct {
  int64_t cand_index;           /* winning candidate, -1 if none                            */
  double accuracy;              /* end-to-end accuracy, 0.0 if none                         */
  int32_t total_workers;        /* sum of workers, 0 if none                                */
  int32_t status;               /* LOKI_LEVEL_*                                             */
  int32_t variant[LOKI_MAX_TASKS][2]; /* variant of part 0 / part 1 (-1 if unused)          */
  int32_t batch[LOKI_MAX_TASKS][2];   /* maximum batch size y(i,k) of each part (0 if unused) */
  int32_t workers[LOKI_MAX_TASKS][2]; /* replicas x(i,k) of each part                       */
  int32_t split_k[LOKI_MAX_TASKS];    /* 16 = single option, else sixteenths routed to part 0;
                                         0 for tasks >= n_tasks or when there is no plan    */
  int64_t latency_budget_us[LOKI_MAX_TASKS]; /* execution time of the chosen (variant, batch):
                                         the task's latency budget (Sec. 4.2)               */
} loki_config_t;

/* Facts about a handle, for harnesses and tests. */
typedef struct {
  int64_t n_candidates;         /* N                                                        */
  int32_t path_auto;            /* what LOKI_PATH_AUTO falls back to where HOISTED is not taken */
  int32_t path_current;         /* path set with loki_alloc_set_path (LOKI_PATH_AUTO at first) */
  int32_t direct_ok;            /* 1 if the DIRECT path's conditions hold                   */
  int32_t direct_level_tile;    /* most demand levels per DIRECT launch                     */
  int32_t n_blocks;             /* thread blocks of the scoring kernel                      */
  int32_t n_launches_last;      /* kernels + device copies enqueued by the last solve       */
  int32_t hoisted_ok;           /* 1 if the HOISTED path's conditions hold                  */
  int32_t path_last;            /* kernel the last solve used (what AUTO resolved to); 0 before */
  int32_t uniform_ok;           /* 1 if the UNIFORM path's conditions hold                  */
  int32_t level_tile_last;      /* demand levels per scoring tile in the last solve; 0 before    */
  int64_t scratch_bytes;        /* device scratch owned by the handle                       */
  int64_t table_bytes;          /* device tables owned by the handle                        */
} loki_alloc_info_t;

/* Checks `desc` exactly as loki_alloc_create does before it touches the device
 * (argument checks; the rooted-tree requirement of Section 2.1; range checks).
 * Needs no GPU.  Returns LOKI_OK or the error loki_alloc_create would return. */
int loki_alloc_validate(const loki_alloc_desc_t* desc);

/* Host-only diagnostic of the planner.  Sets *direct_ok to 1 if the DIRECT path's
 * exactness and range conditions hold for `desc`; if so, replays that path's
 * fixed-point worker arithmetic on the host for every option part at demands on
 * both sides of the points where ceil(demand*lat/(batch*1e9)) (Eq. 2 with Eq. 5)
 * steps, and counts evaluations and disagreements with exact division.  Needs no
 * GPU.  Returns LOKI_OK or the validation error. */
int loki_alloc_plan_selfcheck(const loki_alloc_desc_t* desc, int32_t* direct_ok,
                              int64_t* n_checked, int64_t* n_mismatch);

/* Builds a handle on the current CUDA device for the problem of Section 4.1
 * ("Inputs"): validates, copies the tables to the device, computes every
 * option's task accuracy there, sizes scratch for max_levels, and solves the
 * demand-free zero-demand case once (a few kernel launches on the default
 * stream, then a synchronise).  *out is set only on success.  The handle is
 * immutable afterwards except for loki_alloc_set_path / loki_alloc_set_timing. */
int loki_alloc_create(const loki_alloc_desc_t* desc, loki_alloc_t** out);

/* Scores every candidate for each of n_levels demand levels and writes one plan
 * per level (Section 4.1, both steps; Section 4.2 "Solving the MILP" for the
 * periodic re-solve over a demand history that the batched form serves).
 *   d_demand_mqps  DEVICE pointer, int64[n_levels], milli-queries/s, caller-owned
 *   d_out          DEVICE pointer, loki_config_t[n_levels], caller-owned, 8-byte aligned
 *   cuda_stream    a cudaStream_t (0 = default stream)
 * Work is enqueued on the stream and the call returns without synchronising.
 * At most one solve per handle may be in flight (scratch is per handle).  DIRECT
 * solves of different handles on different streams are serialised on the device by
 * the library (they share one constant-memory demand tile); the other kernels run
 * concurrently.  n_levels must be 1..max_levels.  Per-level problems (infeasible, bad
 * demand) are reported in loki_config_t.status, never as an error code. */
int loki_alloc_solve(loki_alloc_t* h, const int64_t* d_demand_mqps, int32_t n_levels,
                     void* cuda_stream, loki_config_t* d_out);

/* The same search (Section 4.1) with HOST buffers: copies the demands to the
 * device, solves, copies the plans back and synchronises the stream before
 * returning.  h_demand_mqps: int64[n_levels]; h_out: loki_config_t[n_levels];
 * pinned host memory makes the copies asynchronous but is not required. */
int loki_alloc_solve_host(loki_alloc_t* h, const int64_t* h_demand_mqps, int32_t n_levels,
                          void* cuda_stream, loki_config_t* h_out);

/* The same search for callers that are not allowed to allocate device memory
 * (the paper has no counterpart).  Typical cases: a control loop inside a serving
 * process whose memory pool has already claimed the whole GPU, so cudaMalloc
 * fails or is forbidden by policy; code that runs between latency-critical
 * kernels and must avoid the device-wide stall cudaMalloc/cudaFree can cause.
 * Such a caller builds the handle once at start-up, while allocating is still
 * allowed, and from then on calls this function: it allocates nothing (no
 * cudaMalloc, cudaFree or allocating library routine), loads nothing onto the
 * device and touches none of the handle's scratch.  Its working memory is one
 * fixed 267,520-byte array inside the library, which every GPU that loads the
 * library holds until the process exits.  Limits: n_levels <= 64 per call (more
 * returns LOKI_ERR_RANGE); the scoring grid is capped at 256 blocks.  It always
 * uses the GENERIC scoring kernel and produces the same plans as loki_alloc_solve.
 *   d_demand_mqps, d_out, cuda_stream: as for loki_alloc_solve (DEVICE pointers).
 * The array's device address is looked up by loki_alloc_create (once per device,
 * with that device current): that lookup is what makes the driver place the array
 * on the device, so it happens while the caller may still allocate, and the handle
 * must have been created on the device the call runs on (LOKI_ERR_CUDA otherwise).
 * Create the handle before any stream capture begins.  All calls, from every handle
 * and stream, share the one array: calls that overlap on the GPU race on it and
 * give wrong plans, so order them (same stream, or events).  The array keeps the
 * previous call's contents; every word a call reads it has written itself first, so
 * nothing needs clearing between calls.  Enqueues on the stream and returns without
 * synchronising. */
int loki_alloc_solve_static(const loki_alloc_t* h, const int64_t* d_demand_mqps, int32_t n_levels,
                            void* cuda_stream, loki_config_t* d_out);

/* Request routing for the plans of a demand sweep: MostAccurateFirst, Algorithm 1
 * of Section 5.1 ("Request Routing"), the step the Load Balancer runs every time
 * the Resource Manager changes the allocation.  For each level: the workers of
 * every task are taken in non-increasing order of the single-model accuracy of
 * the variant they host; starting from the Frontend (source id -1, sending the
 * level's demand to the root task) and then worker by worker in that order, the
 * requests a worker sends to a child task -- incoming x the multiplicative factor
 * of its variant x the edge's factor -- are handed to the child's workers, most
 * accurate first, each up to its remaining capacity (peak throughput q = b / l of
 * Eq. 5, in queries/s); a routing-table entry holds the share routed / outgoing.
 * Capacity left over at the end is reported per worker (the list the paper gives
 * upstream workers for opportunistic rerouting, Section 5.2).
 *   d_demand_mqps  DEVICE, int64[n_levels]: the demands the plans were solved for
 *   d_plans        DEVICE, loki_config_t[n_levels] as written by loki_alloc_solve
 *   d_headers      DEVICE, loki_route_header_t[n_levels]
 *   d_workers      DEVICE, loki_route_worker_t[n_levels][max_workers]; worker ids are
 *                  indices into a level's row: task by task, most accurate first
 *   d_entries      DEVICE, loki_route_entry_t[n_levels][max_entries], in the order
 *                  Algorithm 1 adds them
 * max_workers = cluster_size and max_entries = 2 * cluster_size + n_tasks are always
 * enough; a level that needs more gets status LOKI_ROUTE_TABLE_FULL.  A level without a
 * plan gets LOKI_ROUTE_NO_PLAN and empty tables.  Requests that find no capacity (by
 * rounding, or when demand exceeds what the plan was made for) are summed in
 * unrouted_qps.  All buffers are caller-owned; the call enqueues one kernel on the
 * stream and returns without synchronising; it uses none of the handle's scratch. */
enum { LOKI_ROUTE_OK = 0, LOKI_ROUTE_NO_PLAN = 1, LOKI_ROUTE_TABLE_FULL = 2 };
typedef struct {
  int32_t status;               /* LOKI_ROUTE_*                                             */
  int32_t n_workers;            /* workers of the plan                                      */
  int32_t n_entries;            /* routing-table entries written                            */
  int32_t reserved;
  double unrouted_qps;          /* requests no worker had capacity for                      */
} loki_route_header_t;
typedef struct {
  int32_t task, variant, batch, reserved;
  double capacity_qps;          /* Eq. 5                                                    */
  double incoming_qps;          /* requests routed to this worker                           */
  double leftover_qps;          /* capacity - incoming                                      */
} loki_route_worker_t;
typedef struct {
  int32_t src_worker;           /* -1 = Frontend                                            */
  int32_t dst_worker;
  double probability;           /* share of src's requests for dst's task that go to dst    */
} loki_route_entry_t;
int loki_alloc_route(const loki_alloc_t* h, const int64_t* d_demand_mqps, const loki_config_t* d_plans,
                     int32_t n_levels, int32_t max_workers, int32_t max_entries, void* cuda_stream,
                     loki_route_header_t* d_headers, loki_route_worker_t* d_workers,
                     loki_route_entry_t* d_entries);

/* Frees the handle's device and host memory (waits for the device first).
 * loki_alloc_destroy(NULL) is a no-op. */
int loki_alloc_destroy(loki_alloc_t* h);

/* Selects the scoring kernel (LOKI_PATH_*).  LOKI_PATH_DIRECT, LOKI_PATH_UNIFORM and
 * LOKI_PATH_HOISTED are refused with LOKI_ERR_RANGE when their conditions do not hold for this
 * problem (HOISTED also needs its per-class worker tables to fit in shared memory). */
int loki_alloc_set_path(loki_alloc_t* h, int32_t path);

/* Replaces the latency SLO L and the per-hop communication latency of the handle
 * (the knob of the paper's "Effect of SLOs on system performance" study: the same
 * pipeline and profiles solved under a range of SLOs).  Only the per-path latency
 * limits change; no table is rebuilt.  Waits for the device, re-solves the
 * demand-free zero-demand case on the default stream and synchronises.  Must not
 * overlap a solve of this handle. */
int loki_alloc_set_slo(loki_alloc_t* h, int64_t slo_us, int64_t comm_us);

/* One demand sweep under a sweep of latency SLOs, the two axes of the paper's
 * "Effect of SLOs on system performance" study (Section 6.4) in one call:
 * d_out[s * n_levels + l] is the plan of demand level l under slo_us[s]; the
 * handle's own SLO, communication latency and everything else stay as they are.
 *   slo_us         HOST pointer, int64[n_slos], each 0..2^60; n_slos <= 64 (more
 *                  returns LOKI_ERR_RANGE)
 *   d_demand_mqps  DEVICE, int64[n_levels]; d_out DEVICE, loki_config_t[n_slos * n_levels]
 * No table is rebuilt and nothing is synchronised.  Where the sweep takes the HOISTED
 * kernel the SLOs are a second batched axis of the same launches (the SLO only sets the
 * latency slack the walk starts from, the worker tables are shared): one launch pair
 * answers the zero-demand levels of all SLOs, then one scoring launch and one finishing
 * launch cover as many (SLO, level tile) pairs as the partial-key scratch holds -- the
 * whole study for small problems.  On the other kernels the call enqueues, per SLO, the
 * demand-free pass and then the kernels of loki_alloc_solve with that SLO's per-path
 * latency limits in their launch parameters.  Same rules as loki_alloc_solve otherwise. */
int loki_alloc_solve_slos(loki_alloc_t* h, const int64_t* d_demand_mqps, int32_t n_levels,
                          const int64_t* slo_us, int32_t n_slos, void* cuda_stream,
                          loki_config_t* d_out);

/* Timing of the scoring kernel (the paper has no counterpart; measurement aid).
 * With timing enabled every scoring launch of the following solves is bracketed
 * by a CUDA event pair on the solve's stream.  loki_alloc_last_score_ms waits for
 * the last solve's scoring launches and returns their summed device time and
 * their number; call it only after a solve, from the thread that issued it. */
int loki_alloc_set_timing(loki_alloc_t* h, int32_t enable);
int loki_alloc_last_score_ms(loki_alloc_t* h, float* total_ms, int32_t* n_launches);

/* Work the DIRECT kernel executed in the last solve (the paper has no counterpart;
 * measurement aid): the number of FP64 fused multiply-adds of the worker arithmetic
 * (Eq. 2 with Eq. 5), one per (staged candidate, level of the tile, option part).  Only
 * candidates within the latency bound of Eqs. 6-7 are staged, a ragged last row of 32
 * is padded with copies, and a tile's unused levels are scored like the others, so the
 * count is what ran, not N x n_levels x parts.  Waits for the device copy of one
 * counter; *executed is 0 when the last solve used another kernel. */
int loki_alloc_last_fma_count(loki_alloc_t* h, int64_t* executed);

/* Status of the checked build (the paper has no counterpart; a debugging aid that stands in
 * for a memory checker).  The library is also built as libloki_alloc_debug.so with every index
 * into its device tables, its shared-memory stages and tables and its partial-key scratch
 * bounds-checked inside the kernels: an index out of range is recorded and replaced by a valid
 * one, so the kernel runs on and nothing faults.  *checked_build is 1 for that build, 0 for the
 * release build (which records nothing); *site_mask has one bit per kind of index that was ever
 * out of range on this handle, *n_violations their number.  Waits for the device copy of the
 * status words. */
int loki_alloc_debug_status(const loki_alloc_t* h, int32_t* checked_build, uint32_t* site_mask,
                            uint32_t* n_violations);

/* Number of candidates N = prod_i O_i (the root-to-sink paths of the augmented
 * graph of Section 4.1 times the batch choices). */
int loki_alloc_num_candidates(const loki_alloc_t* h, int64_t* out);

/* Fills *out with facts about the handle. */
int loki_alloc_get_info(const loki_alloc_t* h, loki_alloc_info_t* out);

/* Static, never-null description of an error code. */
const char* loki_alloc_strerror(int code);

/* sizeof(loki_config_t) as compiled into the library (layout check for bindings). */
int32_t loki_alloc_config_size(void);

#ifdef __cplusplus
}
#endif
#endif /* LOKI_ALLOC_H_ */
