/*
 * galv.h — C boundary of the B200 strategy-search library (libgalv.so).
 *
 * The library runs the hot path of a hybrid-parallel strategy selector for
 * transformer training (the "Dynamic Strategy Selector" of the paper's
 * Section 3: profiler statistics -> performance model -> dynamic-programming
 * search for a per-layer plan; per-layer strategies are the paper's Section 2,
 * "Layer-Specific Parallelism Optimization"):
 *
 *   galv_eval_costs   cost model for every (instance, layer, strategy), fp64 -> int32
 *   galv_dp_search    layer-wise min-plus recurrence under a memory budget
 *   galv_backtrack    optimum at a budget and the per-layer plan
 *
 * for a batch of B independent search instances on one GPU (sm_100a).
 *
 * Conventions
 *  - Every function returning int returns GALV_OK (0) or a negative error code.
 *    No exceptions, no exit(), no device trap.
 *  - Unless a parameter says "host", array pointers are DEVICE pointers owned by
 *    the caller, 16-byte aligned.  The library allocates no device memory;
 *    scratch comes from a caller-provided workspace sized by a query call.
 *  - Work is enqueued on the caller's stream (a cudaStream_t passed as void*,
 *    NULL = default stream) and is asynchronous; errors the host can detect are
 *    returned at once, conditions found on the device land in status[B].
 *  - A context belongs to one host thread at a time.
 *
 * Notation: instance i has L[i] <= Lmax layers; S strategies; budget columns
 * m = 0..M inclusive, stored with pitch m_pitch (multiple of 32, >= M+1).
 * Integer tables: time_q, mem_q [B][Lmax][S]; trans_q [B][S][S] with row = the
 * previous layer's strategy s', column = this layer's strategy s.
 * DP tables: C int32 [B][Lmax][S][m_pitch] (m fastest), A uint8 same dims.
 */
#ifndef GALV_H
#define GALV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GALV_INF 1073741823 /* 2^30-1: +infinity of the cost tables, absorbing */

/* return codes */
#define GALV_OK 0
#define GALV_ERR_INVALID_ARG (-1) /* NULL required pointer, limits violated, flags inconsistent with tables */
#define GALV_ERR_UNSUPPORTED (-2) /* device is not compute capability 10.x */
#define GALV_ERR_WORKSPACE (-3)   /* workspace NULL, misaligned or too small */
#define GALV_ERR_CUDA (-4)        /* a CUDA call failed; text in galv_last_error */
#define GALV_ERR_TIMEOUT (-5)     /* a bounded device-side wait ran out */

/* per-instance status bits (status[B], device) */
#define GALV_STATUS_INFEASIBLE 1    /* no plan fits the budget (not an error) */
#define GALV_STATUS_BAD_INPUT 2     /* negative entry, L[i] out of 1..Lmax, bad descriptor */
#define GALV_STATUS_OVERFLOW_RISK 4 /* a path sum could reach GALV_INF */
#define GALV_STATUS_TIMEOUT 8       /* a bounded device-side wait ran out while this batch ran */

/* shape.flags */
#define GALV_STORE_C_FULL 1 /* keep every layer of C (needed to backtrack without A) */
#define GALV_STORE_ARGMIN 2 /* write the argmin table A */
#define GALV_TRANS_PER_LAYER 4 /* trans_q is [B][Lmax][S][S]: matrix l is paid between layers l-1 and l (matrix 0 unused);
                                  for galv_dp_search, galv_backtrack, galv_plan_cost, galv_search_host, galv_graph_create */
#define GALV_KERNEL_REFERENCE 256 /* run the recurrence with the simple one-thread-per-cell kernel (slow; cross-checks) */
#define GALV_KERNEL_PER_LAYER 512 /* one launch per layer instead of one cooperative launch over all layers */
#define GALV_KERNEL_NO_PACKED 4096 /* never take the packed 16-bit path (two relaxations per instruction on rebased
                                      costs; taken on its own when S <= 64, S % 4 == 0, no argmin table, all layers in
                                      one launch and every transition entry <= 32767; same results) */
#define GALV_KERNEL_NO_CLUSTER 16384 /* never take the cluster kernel (small batches: one thread-block cluster per instance,
                                        the table slice kept in shared memory; taken on its own when the device can hold
                                        one cluster per instance at once, no argmin table is asked for, S <= 128 and the
                                        slice fits in shared memory; same results) */
#define GALV_KERNEL_CLUSTER 32768 /* take the cluster kernel whenever the shape allows it, also for batches that need
                                     several rounds of clusters (at most 512 instances then) */
#define GALV_CLUSTER_SIZE(n) (((n) & 31) << 16) /* the cluster kernel with clusters of n CTAs (1..16), where that size is possible
                                                   for the shape (by default the size is chosen from the shape, the batch
                                                   and what the device can hold at once) */
#define GALV_DEBUG_WITHHOLD_LOAD 2048 /* test hook for the time-out path: one CTA never receives its first stage, every
                                         bounded wait that depends on it runs out (about a second each), status gets
                                         GALV_STATUS_TIMEOUT and the call's results are void; nothing faults or hangs */
#define GALV_SKIP_INFEASIBLE 1024 /* tiles wholly below the previous layer's feasibility frontier (sum of the
                                     layers' smallest mem) read only +inf: write their +inf results without
                                     loading or relaxing anything.  Same tables, less work on tight budgets. */
#define GALV_SKIP_DOMINATED 8192 /* a candidate more than the largest transition entry above its column's best
                                    previous-layer value cannot win or tie; rows (row pairs in the packed loop) that
                                    are such in all 128 columns of a warp group's tile are left out of the inner
                                    loop.  Same tables (argmin table included); the work then depends on the spread
                                    of the costs.  Honoured when S <= 64 and, in the 32-bit loop, a tile's S rows fit
                                    one stage; ignored elsewhere (GALV_KERNEL_REFERENCE among them). */

typedef struct galv_ctx galv_ctx;

/* limits: 1<=B, 1<=S<=256, 1<=Lmax<=65535, 0<=M<2^24, m_pitch>=M+1, m_pitch%32==0 */
typedef struct { int32_t B, Lmax, S, M, m_pitch, flags; } galv_shape;

/* One layer as the model profiler would describe it (80 bytes).
 * FLOPs forward = c_lin*b*seq*h^2 + c_attn*b*seq^2*h; parameters = p_coef*h^2;
 * n_ar tensor-parallel all-reduces per step; activation bytes
 * seq*b*h*(act_rep + act_tp/tp) + act_attn*heads*seq^2*b/tp. */
typedef struct { double h, seq, heads, c_lin, c_attn, p_coef, n_ar, act_rep, act_tp, act_attn; } galv_layer_desc;
/* One candidate strategy (32 bytes): tensor-parallel ways, data-parallel replicas,
 * ZeRO stage 0..3, activation checkpointing 0/1, sequence parallelism 0/1,
 * and the divisor that turns the instance batch b into the per-replica batch. */
typedef struct { int32_t tp, dp, zero, ckpt, sp, _pad; double batch_div; } galv_strategy_desc;
/* One search instance (64 bytes): micro-batch, in-flight micro-batches held in
 * memory, FLOP/s, tp and dp link bytes/s, bytes per element, bytes per memory
 * bin, nanoseconds per integer time unit. */
typedef struct { double b, act_mult, flops_rate, bw_tp, bw_dp, bytes_per_elem, bin_bytes, time_unit_ns; } galv_inst_params;

/* Create a context on CUDA device `device_ordinal` (must be compute capability
 * 10.x).  Allocates host memory only.  Destroy with galv_destroy. */
int galv_create(galv_ctx** out, int device_ordinal);
int galv_destroy(galv_ctx* ctx);
/* Static text for a return code. */
const char* galv_strerror(int code);
/* Detail of the last failure on this context (valid until the next call on it). */
const char* galv_last_error(const galv_ctx* ctx);

/*
 * Cost model (Section 3: the selector combines the model profiler's per-layer
 * shapes/FLOPs, the hardware profiler's memory and bandwidth and the dataset
 * profiler's batch into a performance model).  For every instance i, layer
 * l < L[i] and strategy s, in IEEE double without fused multiply-add:
 *   time_s    = compute/(tp*flops_rate) + tensor-parallel ring all-reduce + gradient ring all-reduce
 *   mem_bytes = optimizer/parameter state under the ZeRO stage + act_mult * activations
 *   time_q = rint(time_s*1e9/time_unit_ns), mem_q = ceil(mem_bytes/bin_bytes), both saturating at 2^30
 * and for every (s', s): trans_q = rint(reshard_s*1e9/time_unit_ns), the time to
 * re-lay-out one activation of layer 0's shape between the two tensor-parallel layouts.
 *
 * L [B] layers per instance; layers [B][Lmax] with layer_stride_B = Lmax, or one
 * shared row with layer_stride_B = 0; strat [S]; inst [B].
 * time_s, mem_bytes [B][Lmax][S] may be NULL.  Entries of layers l >= L[i] are left untouched.
 * status[i] is set to 0, or GALV_STATUS_BAD_INPUT when L[i] is outside 1..Lmax
 * (nothing is written for that instance) or when a descriptor is one no profiler
 * could have produced: an instance parameter, h, seq or batch_div that is not a
 * positive finite number, a negative or non-finite layer coefficient, tp or dp
 * below 1, a ZeRO stage outside 0..3, ckpt or sp other than 0/1.  Such an
 * instance (every instance, when the strategy table is at fault) gets -1 in all
 * its time_q, mem_q and trans_q entries, which galv_dp_search flags in turn;
 * its time_s / mem_bytes are left untouched.
 */
int galv_eval_costs(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                    const galv_layer_desc* layers, int64_t layer_stride_B,
                    const galv_strategy_desc* strat, const galv_inst_params* inst,
                    double* time_s, double* mem_bytes,
                    int32_t* time_q, int32_t* mem_q, int32_t* trans_q,
                    int32_t* status, void* stream);

/* Bytes of workspace galv_dp_search needs for `shape` (0 on invalid shape). */
size_t galv_dp_workspace_bytes(const galv_ctx* ctx, const galv_shape* shape);

/*
 * The search (Section 3: "a dynamic programming algorithm to find an optimal
 * strategy given a performance model"), for every instance:
 *   C[0][m][s] = time(0,s)                      if mem(0,s) <= m, else GALV_INF
 *   C[l][m][s] = time(l,s) + min_{s'} ( C[l-1][m-mem(l,s)][s'] + trans(s',s) )
 * GALV_INF where m < mem(l,s) or every candidate is GALV_INF.  A[l][m][s] is the
 * lowest minimising s' (255 for GALV_INF cells and on layer 0; with S = 256 the
 * value 255 is also a strategy index: read A only where C is finite, as
 * galv_backtrack does).
 *
 * Before the recurrence every instance is validated: entries >= 0, L[i] in
 * 1..Lmax, and sum_l max_s time + (L-1)*max trans < GALV_INF.  status[i] is set
 * to 0 or to BAD_INPUT / OVERFLOW_RISK; flagged instances are skipped (their
 * tables are left untouched) and never cause an out-of-range access.
 *
 * C       [B][Lmax][S][m_pitch] iff GALV_STORE_C_FULL, else NULL
 * A       same dims, uint8, iff GALV_STORE_ARGMIN, else NULL (with S <= 64 and transition entries below 2^24 the
 *         argmin loop runs one fused add-min per relaxation on keys, rebased cost << 6 | row; same table)
 * C_last  [B][S][m_pitch], always written: layer L[i]-1 of instance i
 * Pad columns M < m < m_pitch are written as GALV_INF / 255.
 * workspace: 256-byte aligned, at least galv_dp_workspace_bytes(shape) bytes,
 * overwritten by every call (calls sharing a workspace must not overlap).
 * Without GALV_STORE_C_FULL two layers roll in the workspace (which then holds
 * 2*B*S*m_pitch more int32): with GALV_STORE_ARGMIN the plan comes from A, with
 * neither flag the search yields the optimum only (C_last, and opt_cost from
 * galv_backtrack with plan = NULL) at a two-layer memory footprint.
 * Without an argmin table all layers run in ONE cooperative launch (its CTAs hand
 * finished tiles to one another through counters in the workspace, with bounded
 * waits; on the rolling buffer a tile also waits for the readers of the cells it
 * overwrites); so does the argmin table where its loop can work on keys (S <= 64, entries
 * below 2^24, no GALV_SKIP_DOMINATED).  Otherwise with an argmin table, and with
 * GALV_KERNEL_PER_LAYER, one launch per layer.
 * Nothing synchronises the host, so the call may be captured in a CUDA graph.
 */
int galv_dp_search(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                   const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                   int32_t* C, uint8_t* A, int32_t* C_last,
                   void* workspace, size_t workspace_bytes,
                   int32_t* status, void* stream);

/*
 * Which kernel the most recent galv_dp_search on `workspace` ran: *packed = 1 for the tiled kernel
 * with the packed 16-bit inner loop (two relaxations per instruction; see GALV_KERNEL_NO_PACKED),
 * 0 for the tiled kernel with the 32-bit one, 2 for the cluster kernel (32-bit loop; see
 * GALV_KERNEL_NO_CLUSTER).  The choice between the two inner loops is made on the device; this
 * call waits for `stream` and reads the answer back (host pointer).
 */
int galv_dp_search_path(galv_ctx* ctx, const galv_shape* shape, const void* workspace, int32_t* packed, void* stream);

/*
 * The same search without any caller-provided scratch (the paper has no
 * counterpart; this exists for deployment).  Some callers cannot call
 * cudaMalloc at all: a plugin running inside a host application that owns the
 * device heap, code on a latency path where an allocation (which may
 * synchronise the device) is forbidden, or a process whose memory pool was
 * sized up front and is full.  For them the scratch that galv_dp_search takes
 * as `workspace` lives in a fixed array of GALV_STATIC_WORKSPACE_BYTES inside
 * the library's device image; every GPU that loads the library carries that
 * array until the process exits.  Inputs and outputs are still the caller's.
 *
 * Arguments, results and status bits are those of galv_dp_search.  Shapes whose
 * galv_dp_workspace_bytes exceeds GALV_STATIC_WORKSPACE_BYTES are refused with
 * GALV_ERR_WORKSPACE.  What the scratch holds: a few int32 per instance and per
 * layer; 4 bytes per (instance, layer) and per (instance, tile of 128 budget
 * columns); B*S*S*2 bytes of packed transition rows when the packed 16-bit
 * loop may run (S <= 64, S % 4 == 0, neither GALV_KERNEL_NO_PACKED nor
 * GALV_STORE_ARGMIN nor GALV_KERNEL_PER_LAYER; times Lmax with
 * GALV_TRANS_PER_LAYER), or B*S*S*4 bytes of shifted transition entries with
 * GALV_STORE_ARGMIN and S <= 64 (the argmin loop on keys); and 2*B*S*m_pitch*4
 * bytes when the full table is not kept.  So batches of a few hundred instances with the full table fit; large
 * batches fit only with GALV_KERNEL_NO_PACKED (B = 1024, S = 32 needs 2 MiB
 * for the packed rows alone), and the rolling two-layer mode only for small
 * B*S*m_pitch.  Ask galv_dp_workspace_bytes.  The call itself allocates
 * nothing, on the host or the device.
 *
 * The first call on a device looks up the array's device address and, like the
 * first launch of any kernel, makes the CUDA runtime load the library's device
 * code (once per device); make that first call outside any stream capture.  All calls share
 * the one array: what has to start from zero is cleared by each call, and two
 * calls that overlap on the GPU (different streams, or different contexts on
 * the same device) race on it — serialise them.
 */
#define GALV_STATIC_WORKSPACE_BYTES (1 << 20)
int galv_dp_search_static(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                          const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                          int32_t* C, uint8_t* A, int32_t* C_last,
                          int32_t* status, void* stream);

/*
 * Optimum and plan (Section 3: the selector's output is a per-layer
 * parallelism plan).  For every instance, at budget[i] (NULL: M):
 *   opt_cost = min_s C_last[budget][s], lowest s on ties (GALV_INF if none is finite);
 *   plan walks back from the last layer taking, at each layer, the lowest s'
 *   that attains the cell's minimum (read from A when given, otherwise found
 *   again from C); mem_used = sum_l mem(l, plan[l]).
 * Needs A, or C with GALV_STORE_C_FULL; with neither, plan must be NULL and
 * only opt_cost is produced.  status[i]: the INFEASIBLE bit is set or cleared;
 * instances flagged by the search get opt_cost = GALV_INF and plan = -1.
 * plan [B][Lmax], -1 beyond L[i] and when infeasible; budget values must be in 0..M.
 */
int galv_backtrack(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                   const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                   const int32_t* C, const uint8_t* A, const int32_t* C_last,
                   const int32_t* budget,
                   int32_t* opt_cost, int32_t* plan, int32_t* mem_used,
                   int32_t* status, void* stream);

/*
 * Outer selection over the instance batch (Section 3: the emitted plan also fixes the number of
 * pipeline stages and the micro-batch; Section 2: pipelines run with many micro-batches).  Every
 * instance is one candidate (micro-batch, pipeline degree) whose per-stage optimum opt_cost[i] the
 * search has found.  An iteration of a pp-stage pipeline fed with n_micro micro-batches lasts
 * (n_micro + pp - 1) stage times; within each group of candidates (same global batch) the
 * feasible one (status 0, finite cost) with the shortest iteration wins, the lowest index on ties.
 * opt_cost, status, n_micro, pp, group: int32 [B]; group values 0..G-1 (others, and n_micro < 1 or
 * pp < 1, are ignored).  best_time int64 [G] (time units; -1 if the group has no feasible
 * candidate), best_inst int32 [G] (-1 likewise).  All device pointers.
 */
int galv_select_best(galv_ctx* ctx, int32_t B, int32_t G, const int32_t* opt_cost, const int32_t* status,
                     const int32_t* n_micro, const int32_t* pp, const int32_t* group,
                     int64_t* best_time, int32_t* best_inst, void* stream);

/*
 * Dominated-strategy prune (Section 3: a prune of the candidates precedes the dynamic program).
 * Strategy s is dropped when another strategy d is at least as good in every layer of every
 * instance of the batch (time and memory) and in every transition (trans(x,d) <= trans(x,s) and
 * trans(d,x) <= trans(s,x) for all x), and either d < s or d is strictly faster at every layer.
 * Under this rule the search on the remaining strategies returns the same optimal cost and, after
 * galv_expand_plan, the same plan as the search on all of them, at every budget.
 * keep int32 [S]: 1 kept, 0 dropped; map int32 [S]: original indices of the kept strategies in
 * ascending order, -1 beyond; S_kept int32 [1].  All device pointers; read S_kept back (after
 * synchronising the stream) to size the compacted tables.  shape.M, m_pitch and flags are not used.
 */
int galv_prune_strategies(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                          const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                          int32_t* keep, int32_t* map, int32_t* S_kept, void* stream);
/* Gather the kept strategies: time_out, mem_out [B][Lmax][S_kept], trans_out [B][S_kept][S_kept]. */
int galv_compact_tables(galv_ctx* ctx, const galv_shape* shape, int32_t S_kept, const int32_t* map,
                        const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                        int32_t* time_out, int32_t* mem_out, int32_t* trans_out, void* stream);
/* Turn a plan over kept strategies back into original indices, in place: plan[e] = map[plan[e]] where >= 0. */
int galv_expand_plan(galv_ctx* ctx, int32_t B, int32_t Lmax, const int32_t* map, int32_t* plan, void* stream);

/*
 * Cost and memory of GIVEN plans under the current tables (Sections 3-4: when the selector
 * re-evaluates during training it weighs the running plan against the new optimum):
 * cost[i] = sum_l time(l,p_l) + sum_{l>=1} trans(p_{l-1},p_l), mem_total[i] = sum_l mem(l,p_l)
 * over the L[i] layers of instance i, as int64; both -1 when L[i] is out of range or the plan
 * has an entry outside 0..S-1 among those layers.  plan int32 [B][Lmax].  All device pointers.
 */
int galv_plan_cost(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                   const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                   const int32_t* plan, int64_t* cost, int64_t* mem_total, void* stream);

/*
 * Plan switch (Sections 3-4: the running job is resharded when the selector finds a better plan;
 * the paper gives no rule for when that pays, this is the reading taken).
 * galv_add_switch_cost: time_out(i,l,s) = time_q(i,l,s) + trans_l(cur_plan[i][l], s) / horizon[i]
 * (integer division; saturating at GALV_INF): resharding layer l from its current strategy to s
 * is paid once and spread over horizon[i] >= 1 iterations (smaller values count as 1).  Entries
 * of cur_plan outside 0..S-1 (no plan yet) and layers l >= L[i] add nothing.  With
 * GALV_TRANS_PER_LAYER layer l uses matrix l (matrix 0 for layer 0).  Searching time_out instead
 * of time_q weighs iteration time against the price of getting there.  time_out may not alias
 * time_q.  cur_plan int32 [B][Lmax], horizon int32 [B], time_out int32 [B][Lmax][S]; device.
 * galv_switch_decision: decision[i] = 1 when new_cost[i] * (1000 + hysteresis_permille) <
 * cur_cost[i] * 1000, i.e. the new optimum beats staying by the margin; also 1 when the running
 * plan no longer fits (cur_cost[i] < 0 or >= GALV_INF) and the new one does; 0 when new_status[i]
 * != 0 or new_cost[i] >= GALV_INF.  cur_cost int64 [B] (as written by galv_plan_cost), new_cost,
 * new_status, decision int32 [B]; device.  hysteresis_permille >= 0.
 */
int galv_add_switch_cost(galv_ctx* ctx, const galv_shape* shape, const int32_t* L, const int32_t* time_q,
                         const int32_t* trans_q, const int32_t* cur_plan, const int32_t* horizon,
                         int32_t* time_out, void* stream);
int galv_switch_decision(galv_ctx* ctx, int32_t B, const int64_t* cur_cost, const int32_t* new_cost,
                         const int32_t* new_status, int32_t hysteresis_permille, int32_t* decision, void* stream);

/*
 * Re-search pipeline (Sections 3-4: the selector re-runs at intervals from fresh measurements).
 * galv_graph_create captures galv_eval_costs (when layers != NULL) -> galv_dp_search ->
 * galv_backtrack on the given device buffers into a CUDA graph; galv_graph_launch replays it on
 * a stream.  Between replays the caller may overwrite the CONTENTS of any input buffer (typically
 * inst: measured FLOP rate, link bandwidth, micro-batch); pointers and shape are frozen.
 * Arguments are those of the three calls; `stream` must be a non-default stream that is not
 * capturing; the galv_graph holds no device memory.  One replay in flight at a time.
 */
typedef struct galv_graph galv_graph;
int galv_graph_create(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                      const galv_layer_desc* layers, int64_t layer_stride_B,
                      const galv_strategy_desc* strat, const galv_inst_params* inst,
                      int32_t* time_q, int32_t* mem_q, int32_t* trans_q,
                      int32_t* C, uint8_t* A, int32_t* C_last, void* workspace, size_t workspace_bytes,
                      const int32_t* budget, int32_t* opt_cost, int32_t* plan, int32_t* mem_used,
                      int32_t* status, void* stream, galv_graph** out);
int galv_graph_launch(galv_ctx* ctx, galv_graph* graph, void* stream);
int galv_graph_destroy(galv_graph* graph);

/*
 * Stage partitioning (Sections 2-3: layers are spread over pipeline stages so that the stages are
 * balanced, and re-cut when one becomes the bottleneck).  Build the batch with one instance per
 * start layer a (its layers are a, a+1, ..., so B = Lmax = Lm and L[a] = Lm - a) and search it with
 * the full table kept; galv_layer_optima then reads out, for every instance and layer,
 *   opt_l[i][l] = min_s C[i][l][s][budget_i]      (GALV_INF beyond L[i] and for flagged instances),
 * i.e. opt_l[a][n-1] = optimum of the stage made of layers a .. a+n-1.  budget NULL: M.
 * galv_stage_partition cuts layers 0..Lm-1 into P consecutive stages minimising the slowest stage:
 *   f[1][b] = opt(0,b),  f[k][b] = min_{k-1 <= a < b} max(f[k-1][a], opt(a,b)),  range_opt = opt_l.
 * cuts int32 [P+1]: 0 = cuts[0] < ... < cuts[P] = Lm (walking back from the end, the lowest a that
 * attains f[k][b]); bottleneck int32 [1] = f[P][Lm]; GALV_INF and cuts = -1 when nothing is
 * feasible or P > Lm.  (P+1)*(Lm+1) must fit one CTA's shared memory (about 28 000 entries).
 * All device pointers.
 */
int galv_layer_optima(galv_ctx* ctx, const galv_shape* shape, const int32_t* L, const int32_t* C,
                      const int32_t* budget, const int32_t* status, int32_t* opt_l, void* stream);
int galv_stage_partition(galv_ctx* ctx, int32_t Lm, int32_t P, const int32_t* range_opt,
                         int32_t* cuts, int32_t* bottleneck, void* stream);

/*
 * What GALV_SKIP_INFEASIBLE and GALV_SKIP_DOMINATED would leave out of a search, estimated from its inputs (the
 * paper has no counterpart; the flags never change a result, only the work, and how much depends on the data).
 * counts int64 [4], device: [0] tiles of the tiled kernel that lie wholly below the previous layer's feasibility
 * frontier (the running sum of the layers' smallest mem) out of [1] tiles in all, over layers 1 .. L[i]-1 of every
 * instance: the exact share GALV_SKIP_INFEASIBLE skips; [2] rows of layer 0 that cannot win in layer 1 (they never
 * fit, or their time exceeds the layer's smallest by more than the largest transition entry) out of [3] rows: an
 * indication of what GALV_SKIP_DOMINATED finds, which in later layers depends on the tables themselves.
 * Instances with L[i] outside 1..Lmax are not counted.  Same table arguments as galv_dp_search.
 */
int galv_skip_estimate(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                       const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                       int64_t* counts, void* stream);

/* Bytes of device arena galv_search_host needs (0 on invalid shape). */
size_t galv_search_host_arena_bytes(const galv_ctx* ctx, const galv_shape* shape, int with_model);

/*
 * The whole path from HOST buffers: copies the inputs to the device arena, runs
 * galv_eval_costs (when layers != NULL) or takes the host integer tables, then
 * galv_dp_search and galv_backtrack, copies opt_cost / plan / mem_used / status
 * back and synchronises the stream before returning.
 * Host pointers (pinned memory makes the copies asynchronous): L, layers, strat,
 * inst, or time_q/mem_q/trans_q; outputs opt_cost [B], plan [B][Lmax], mem_used [B],
 * status [B].  arena: device, 256-byte aligned, galv_search_host_arena_bytes bytes.
 * shape.flags selects the table mode as in galv_dp_search (tables live in the arena).
 */
int galv_search_host(galv_ctx* ctx, const galv_shape* shape, const int32_t* L,
                     const galv_layer_desc* layers, int64_t layer_stride_B,
                     const galv_strategy_desc* strat, const galv_inst_params* inst,
                     const int32_t* time_q, const int32_t* mem_q, const int32_t* trans_q,
                     int32_t* opt_cost, int32_t* plan, int32_t* mem_used, int32_t* status,
                     void* arena, size_t arena_bytes, void* stream);

/*
 * Integer-ALU throughput probe (the denominator of the roofline the bench
 * reports; the paper has no counterpart).  Runs a register-only kernel of
 * dependent-chain-free integer operations on every SM and returns operations
 * per second in *ops_per_s (host pointer).  kind 0: fused add-then-min, counted
 * as one operation per min-plus relaxation; kind 1: add then min written as two
 * C statements (however the compiler lowers them), counted per relaxation;
 * kind 2: add then xor, two plain int32 operations, both counted; kind 3: the
 * packed add-then-min on two unsigned 16-bit halves (the instruction of the
 * packed 16-bit inner loop), counted as the two relaxations it performs;
 * kind 4: three-input minimum, counted per instruction.  Synchronises.
 */
int galv_probe_int_alu(galv_ctx* ctx, int kind, int iters, double* ops_per_s, void* stream);

/*
 * Timing hook for benchmarks (the paper has no counterpart).  While profiling is
 * on, galv_dp_search records one CUDA event before its first layer launch and
 * one after its last; galv_last_layer_loop_ms waits for the second and returns
 * the milliseconds between them for the most recent search (host pointer).
 * galv_layer_loop_ms_stats does the same for every search since profiling was
 * switched on (the most recent 64 at most): mean, shortest and longest span in
 * milliseconds and the number of searches they cover (host pointers).
 * Switching profiling on or off forgets the spans.  Leave it off when capturing
 * a CUDA graph.
 */
int galv_set_profiling(galv_ctx* ctx, int on);
int galv_last_layer_loop_ms(galv_ctx* ctx, float* ms);
int galv_layer_loop_ms_stats(galv_ctx* ctx, float* mean_ms, float* min_ms, float* max_ms, int* searches);

#ifdef __cplusplus
}
#endif
#endif /* GALV_H */
