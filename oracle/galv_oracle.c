/*
 * CPU oracle for the layer-wise strategy search.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the search computes, used
 * by the tests, by the smoke check and by the bench's CPU-baseline leg to judge
 * the CUDA library.  It shares no code with that library and is never on the
 * product path.
 *
 * What it follows.  The paper's selector (Section 3, "Dynamic Strategy
 * Selector"; Section 2, "Dynamic Strategy Selection" and "Layer-Specific
 * Parallelism Optimization") picks, per layer, one hybrid-parallel strategy so
 * that a performance model's time is smallest within GPU memory, by dynamic
 * programming.  The paper prints no formula; the problem is taken in its plain
 * form:
 *
 *   over all plans p in {0..S-1}^L with  sum_l mem(l,p_l) <= budget, minimise
 *   cost(p) = sum_l time(l,p_l) + sum_{l>=1} trans(p_{l-1}, p_l);
 *   among optimal plans report the one smallest in the order of
 *   (p_{L-1}, p_{L-2}, ..., p_0)  (lowest index wins every tie, last layer first).
 *
 * orc_brute_force() is that definition written out.  orc_dp() is the min-plus
 * recurrence
 *   C[l][m][s] = time(l,s) + min_{s'} ( C[l-1][m-mem(l,s)][s'] + trans(s',s) )
 * with C[0][m][s] = time(0,s) when mem(0,s) <= m; C[l][m][s] is the best cost
 * of layers 0..l that ends in strategy s and uses at most m bins.  m runs over
 * 0..M inclusive.  +inf is ORC_INF = 2^30-1, absorbing.
 *
 * Layout here is the recurrence's own index order, C[l][m][s] with s fastest.
 * trans is one S x S matrix, or one per layer: tl is the number of entries between
 * the matrices of consecutive layers (0: one matrix; S*S: matrix l is paid between
 * layers l-1 and l, matrix 0 is unused).
 *
 * Parity pins (tests, CPU only): brute force on tiny shapes, monotonicity in m,
 * hand-derived worked example, S=1 closed form, trans=0 multiple-choice
 * knapsack, mem=0 layered shortest path against a graph library.
 * Cost model: FLOP count, x3/x4 factor, ring all-reduce byte counts and unit
 * conversion are pinned by closed forms; the memory-state, activation,
 * ZeRO-3 traffic, sequence-parallel and transition formulas are this build's
 * own accounting (the paper gives none): the code is pinned to the stated
 * formulas by hand-worked values, the formulas themselves have no outside
 * truth and are "parity unpinned" in that sense.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORC_INF 1073741823

enum { ORC_INFEASIBLE = 1, ORC_BAD_INPUT = 2, ORC_OVERFLOW_RISK = 4 };

/* Input check: entries non-negative, and no finite path sum can reach ORC_INF:
 * sum_l max_s time(l,s) + (L-1) * max trans < ORC_INF. */
int orc_validate(int L, int S, const int32_t *time, const int32_t *mem, const int32_t *trans, int64_t tl)
{
    int st = 0;
    int64_t sum = 0, tmax = 0;
    if (L < 1 || S < 1) return ORC_BAD_INPUT;
    for (int l = 0; l < L; l++) {
        int64_t mx = 0;
        for (int s = 0; s < S; s++) {
            if (time[l * S + s] < 0 || mem[l * S + s] < 0) st |= ORC_BAD_INPUT;
            if (time[l * S + s] > mx) mx = time[l * S + s];
        }
        sum += mx;
    }
    for (int l = (tl ? 1 : 0); l < (tl ? L : 1); l++)
        for (int k = 0; k < S * S; k++) {
            if (trans[l * tl + k] < 0) st |= ORC_BAD_INPUT;
            if (trans[l * tl + k] > tmax) tmax = trans[l * tl + k];
        }
    if (!(st & ORC_BAD_INPUT) && sum + (int64_t)(L - 1) * tmax >= ORC_INF) st |= ORC_OVERFLOW_RISK;
    return st;
}

/* The recurrence.  C and A are [L][M+1][S]; A may be NULL.  A holds the lowest
 * minimising s' (255 where the cell is +inf and on layer 0). */
void orc_dp(int L, int S, int M, const int32_t *time, const int32_t *mem, const int32_t *trans, int64_t tl,
            int32_t *C, uint8_t *A)
{
    const int64_t W = (int64_t)(M + 1) * S;
    for (int m = 0; m <= M; m++)
        for (int s = 0; s < S; s++) {
            C[(int64_t)m * S + s] = (mem[s] <= m) ? time[s] : ORC_INF;
            if (A) A[(int64_t)m * S + s] = 255;
        }
    for (int l = 1; l < L; l++)
        for (int m = 0; m <= M; m++)
            for (int s = 0; s < S; s++) {
                int64_t best = ORC_INF;
                int arg = 255;
                int64_t mp = (int64_t)m - mem[l * S + s];
                if (mp >= 0) {
                    const int32_t *prev = C + (l - 1) * W + mp * S;
                    for (int sp = 0; sp < S; sp++)
                        if (prev[sp] < ORC_INF) {
                            int64_t v = (int64_t)prev[sp] + trans[l * tl + sp * S + s];
                            if (v < best) { best = v; arg = sp; }
                        }
                }
                C[l * W + (int64_t)m * S + s] = (best < ORC_INF) ? (int32_t)(best + time[l * S + s]) : ORC_INF;
                if (A) A[l * W + (int64_t)m * S + s] = (uint8_t)arg;
            }
}

/* Optimum at `budget` and the plan, walking back from the last layer.  With A
 * the walk reads the stored argmin, without it the argmin is found again from
 * C (lowest s' whose candidate equals the cell's pre-time value).
 * Returns status bits; plan[l] = -1 everywhere when infeasible. */
int orc_backtrack(int L, int S, int M, const int32_t *time, const int32_t *mem, const int32_t *trans, int64_t tl,
                  const int32_t *C, const uint8_t *A, int budget,
                  int32_t *opt_cost, int32_t *plan, int32_t *mem_used)
{
    const int64_t W = (int64_t)(M + 1) * S;
    int s = -1;
    int32_t best = ORC_INF;
    for (int l = 0; l < L; l++) plan[l] = -1;
    *mem_used = 0;
    for (int k = 0; k < S; k++) {
        int32_t v = C[(L - 1) * W + (int64_t)budget * S + k];
        if (v < best) { best = v; s = k; }
    }
    *opt_cost = best;
    if (s < 0) return ORC_INFEASIBLE;
    int64_t m = budget, used = 0;
    for (int l = L - 1; l >= 0; l--) {
        plan[l] = s;
        used += mem[l * S + s];
        if (l == 0) break;
        int64_t mp = m - mem[l * S + s];
        int prev_s = -1;
        if (A) {
            prev_s = A[l * W + m * S + s];
        } else {
            int64_t target = (int64_t)C[l * W + m * S + s] - time[l * S + s];
            for (int sp = 0; sp < S; sp++) {
                int32_t c = C[(l - 1) * W + mp * S + sp];
                if (c < ORC_INF && (int64_t)c + trans[l * tl + sp * S + s] == target) { prev_s = sp; break; }
            }
        }
        m = mp;
        s = prev_s;
    }
    *mem_used = (int32_t)used;
    return 0;
}

/* cost(p) and memory of one plan, straight from the definition. */
void orc_plan_cost(int L, int S, const int32_t *time, const int32_t *mem, const int32_t *trans, int64_t tl,
                   const int32_t *plan, int64_t *cost, int64_t *mem_total)
{
    int64_t c = 0, u = 0;
    for (int l = 0; l < L; l++) {
        c += time[l * S + plan[l]];
        u += mem[l * S + plan[l]];
        if (l >= 1) c += trans[l * tl + plan[l - 1] * S + plan[l]];
    }
    *cost = c;
    *mem_total = u;
}

/* The definition itself: enumerate all S^L plans.  The counter runs with p_0 as
 * the fastest digit, so plans are visited in increasing (p_{L-1},...,p_0) order
 * and "strictly better" keeps the first, i.e. the smallest in that order.
 * Returns the number of feasible plans; opt_cost = ORC_INF and plan = -1 if none. */
int64_t orc_brute_force(int L, int S, int budget, const int32_t *time, const int32_t *mem,
                        const int32_t *trans, int64_t tl, int32_t *opt_cost, int32_t *plan, int32_t *mem_used)
{
    int32_t *p = (int32_t *)calloc((size_t)L, sizeof(int32_t));
    int64_t best = -1, best_mem = 0, feasible = 0;
    for (int l = 0; l < L; l++) plan[l] = -1;
    for (;;) {
        int64_t c, u;
        orc_plan_cost(L, S, time, mem, trans, tl, p, &c, &u);
        if (u <= budget) {
            feasible++;
            if (best < 0 || c < best) {
                best = c; best_mem = u;
                memcpy(plan, p, (size_t)L * sizeof(int32_t));
            }
        }
        int d = 0;
        while (d < L && ++p[d] == S) p[d++] = 0;
        if (d == L) break;
    }
    free(p);
    *opt_cost = best < 0 ? ORC_INF : (int32_t)best;
    *mem_used = (int32_t)best_mem;
    return feasible;
}

/* ------------------------------------------------------------------ cost model
 *
 * The paper states only that a performance model built from per-layer shapes
 * and FLOPs, memory and interconnect bandwidth, and the batch, is searched
 * (Section 3, profilers and selector).  The accounting below is the standard
 * published one: transformer layer FLOPs 24 b s h^2 + 4 b s^2 h, x3 for
 * forward+backward and x4 with activation recomputation; ring all-reduce moves
 * 2(n-1)/n of the buffer; mixed-precision Adam keeps 2+2+12 bytes per
 * parameter, sharded by ZeRO stage; activation bytes per layer
 * s b h (10 + 24/tp) + 5 a s^2 b / tp.  All in IEEE double, evaluated in the
 * order written, no fused multiply-add (compile with -ffp-contract=off).
 */
typedef struct { double h, seq, heads, c_lin, c_attn, p_coef, n_ar, act_rep, act_tp, act_attn; } orc_layer;
typedef struct { int32_t tp, dp, zero, ckpt, sp, pad; double batch_div; } orc_strategy;
typedef struct { double b, act_mult, flops_rate, bw_tp, bw_dp, bytes_per_elem, bin_bytes, time_unit_ns; } orc_inst;

void orc_cost(const orc_layer *ly, const orc_strategy *st, const orc_inst *in,
              double *time_s, double *mem_bytes)
{
    const double tp = st->tp, dp = st->dp;
    const double bq = in->b / st->batch_div;
    const double sbh = ly->seq * bq * ly->h;
    const double fwd = ly->c_lin * bq * ly->seq * ly->h * ly->h + ly->c_attn * bq * ly->seq * ly->seq * ly->h;
    const double t_comp = fwd * (3.0 + st->ckpt) / tp / in->flops_rate;
    const double t_tp = ly->n_ar * (2.0 * (tp - 1.0) / tp) * (bq * ly->seq * ly->h * in->bytes_per_elem) / in->bw_tp;
    const double zmul = st->zero == 3 ? 1.5 : 1.0;
    const double t_dp = zmul * (2.0 * (dp - 1.0) / dp) * (ly->p_coef * ly->h * ly->h * in->bytes_per_elem / tp) / in->bw_dp;
    *time_s = (t_comp + t_tp) + t_dp;

    const double psi = ly->p_coef * ly->h * ly->h / tp;
    double zb;
    switch (st->zero) {
    case 0: zb = 16.0; break;
    case 1: zb = 4.0 + 12.0 / dp; break;
    case 2: zb = 2.0 + 14.0 / dp; break;
    default: zb = 16.0 / dp; break;
    }
    const double state = psi * zb;
    double act;
    if (st->ckpt)
        act = st->sp ? 2.0 * sbh / tp : 2.0 * sbh;
    else if (st->sp)
        act = sbh * (ly->act_rep + ly->act_tp) / tp + ly->act_attn * ly->heads * ly->seq * ly->seq * bq / tp;
    else
        act = sbh * (ly->act_rep + ly->act_tp / tp) + ly->act_attn * ly->heads * ly->seq * ly->seq * bq / tp;
    *mem_bytes = state + in->act_mult * act;
}

/* Resharding time when the previous layer ran strategy `a` and this one runs
 * `c`: the activation of the first layer's shape is regathered in proportion
 * to the change of tensor-parallel layout; ZeRO and checkpointing changes are free. */
double orc_trans_cost(const orc_layer *ly0, const orc_strategy *a, const orc_strategy *c, const orc_inst *in)
{
    const double tpa = a->tp, tpc = c->tp;
    const double bq = in->b / c->batch_div;
    const double bytes = bq * ly0->seq * ly0->h * in->bytes_per_elem;
    const double k = (tpa > tpc ? tpa : tpc) / (tpa < tpc ? tpa : tpc);
    const double spterm = (a->sp != c->sp) ? (tpc - 1.0) / tpc : 0.0;
    return ((k - 1.0) / k + spterm) * bytes / in->bw_tp;
}

/* Time to integer units: round half to even of seconds*1e9/unit.  Memory to
 * bins: ceiling.  Both saturate at 2^30 so the conversion is always defined. */
int32_t orc_quant_time(double t_s, double time_unit_ns)
{
    double q = rint(t_s * 1e9 / time_unit_ns);
    if (!(q < 1073741824.0)) q = 1073741824.0;
    if (q < 0.0) q = 0.0;
    return (int32_t)q;
}

int32_t orc_quant_mem(double bytes, double bin_bytes)
{
    double q = ceil(bytes / bin_bytes);
    if (!(q < 1073741824.0)) q = 1073741824.0;
    if (q < 0.0) q = 0.0;
    return (int32_t)q;
}

/* Descriptors the profilers cannot have produced (the paper's model, hardware and dataset profilers report
 * sizes, rates and counts: Section 3): a rate, size or divisor that is not a positive finite number, a degree
 * below 1, a ZeRO stage outside 0..3, a flag that is not 0/1, a negative coefficient.  An instance with any such
 * descriptor among its own parameters, the strategy table or its L layers is flagged ORC_BAD_INPUT as a whole. */
static int pos_finite(double x) { return x > 0.0 && x < INFINITY; }
static int nonneg_finite(double x) { return x >= 0.0 && x < INFINITY; }
int orc_check_descriptors(int L, int S, const orc_layer *layers, const orc_strategy *strat, const orc_inst *in)
{
    int ok = pos_finite(in->b) && pos_finite(in->act_mult) && pos_finite(in->flops_rate) && pos_finite(in->bw_tp) &&
             pos_finite(in->bw_dp) && pos_finite(in->bytes_per_elem) && pos_finite(in->bin_bytes) && pos_finite(in->time_unit_ns);
    for (int s = 0; s < S; s++)
        ok = ok && strat[s].tp >= 1 && strat[s].dp >= 1 && strat[s].zero >= 0 && strat[s].zero <= 3 &&
             (strat[s].ckpt == 0 || strat[s].ckpt == 1) && (strat[s].sp == 0 || strat[s].sp == 1) && pos_finite(strat[s].batch_div);
    for (int l = 0; l < L; l++)
        ok = ok && pos_finite(layers[l].h) && pos_finite(layers[l].seq) && nonneg_finite(layers[l].heads) &&
             nonneg_finite(layers[l].c_lin) && nonneg_finite(layers[l].c_attn) && nonneg_finite(layers[l].p_coef) &&
             nonneg_finite(layers[l].n_ar) && nonneg_finite(layers[l].act_rep) && nonneg_finite(layers[l].act_tp) &&
             nonneg_finite(layers[l].act_attn);
    return ok ? 0 : ORC_BAD_INPUT;
}

/* One instance: every (layer, strategy) and every (s', s). Outputs may be NULL.  Returns 0, or ORC_BAD_INPUT for
 * a bad descriptor: the integer tables are then filled with -1 (which the search's validation flags in turn)
 * and the double outputs are left untouched. */
int orc_eval_costs(int L, int S, const orc_layer *layers, const orc_strategy *strat, const orc_inst *in,
                   double *time_s, double *mem_bytes, int32_t *time_q, int32_t *mem_q, int32_t *trans_q)
{
    if (orc_check_descriptors(L, S, layers, strat, in)) {
        for (int e = 0; e < L * S; e++) {
            if (time_q) time_q[e] = -1;
            if (mem_q) mem_q[e] = -1;
        }
        if (trans_q)
            for (int e = 0; e < S * S; e++) trans_q[e] = -1;
        return ORC_BAD_INPUT;
    }
    for (int l = 0; l < L; l++)
        for (int s = 0; s < S; s++) {
            double t, b;
            orc_cost(&layers[l], &strat[s], in, &t, &b);
            if (time_s) time_s[l * S + s] = t;
            if (mem_bytes) mem_bytes[l * S + s] = b;
            if (time_q) time_q[l * S + s] = orc_quant_time(t, in->time_unit_ns);
            if (mem_q) mem_q[l * S + s] = orc_quant_mem(b, in->bin_bytes);
        }
    if (trans_q)
        for (int a = 0; a < S; a++)
            for (int c = 0; c < S; c++)
                trans_q[a * S + c] = orc_quant_time(orc_trans_cost(&layers[0], &strat[a], &strat[c], in),
                                                    in->time_unit_ns);
    return 0;
}

/* ------------------------------------------------------------------ outer selection
 *
 * The plan the selector finally emits also fixes the number of pipeline stages and the
 * micro-batch (Section 3, "Dynamic Strategy Selector"; Section 2 on pipelines run with many
 * micro-batches).  Each search instance is one candidate (micro-batch, pipeline degree) whose
 * per-stage optimum the DP has found; one training iteration of a pp-stage pipeline fed with
 * n_micro micro-batches lasts (n_micro + pp - 1) stage times (fill and drain).  Within each group
 * of candidates (same global batch, so the shortest iteration is the highest throughput) pick
 * the feasible instance with the smallest iteration time, the lowest index on ties.
 * best_time[g] = -1 and best_inst[g] = -1 when the group has no feasible candidate.
 * Candidates with n_micro < 1, pp < 1 or a group outside 0..G-1 are ignored.
 */
void orc_select_best(int B, int G, const int32_t *opt_cost, const int32_t *status, const int32_t *n_micro,
                     const int32_t *pp, const int32_t *group, int64_t *best_time, int32_t *best_inst)
{
    for (int g = 0; g < G; g++) { best_time[g] = -1; best_inst[g] = -1; }
    for (int i = 0; i < B; i++) {
        if (status[i] != 0 || opt_cost[i] >= ORC_INF || opt_cost[i] < 0) continue;
        if (n_micro[i] < 1 || pp[i] < 1 || group[i] < 0 || group[i] >= G) continue;
        int64_t t = ((int64_t)n_micro[i] + pp[i] - 1) * (int64_t)opt_cost[i];
        int g = group[i];
        if (best_inst[g] < 0 || t < best_time[g]) { best_time[g] = t; best_inst[g] = i; }
    }
}

/* ------------------------------------------------------------------ dominated-strategy prune
 *
 * The paper prunes the candidate strategies before the dynamic program (Section 3: a decision-tree
 * prune precedes the search).  The rule here is the one that provably leaves the search result
 * untouched, plan included: strategy s goes when some other strategy d is at least as good in every
 * respect, in every instance of the batch -
 *    time(l,d) <= time(l,s) and mem(l,d) <= mem(l,s) for every layer l < L,
 *    trans(x,d) <= trans(x,s) and trans(d,x) <= trans(s,x) for every strategy x -
 * and either d < s (then swapping s for d in a plan never costs more and makes the plan smaller in
 * the (p_{L-1},..,p_0) order, so the reported plan never holds s), or d is strictly faster at every
 * layer (then a plan holding s is never optimal).  keep[s] = 1 for the survivors.
 */
void orc_prune(int B, int Lmax, int S, const int32_t *L, const int32_t *time, const int32_t *mem,
               const int32_t *trans, int32_t *keep)
{
    for (int s = 0; s < S; s++) {
        keep[s] = 1;
        for (int d = 0; d < S && keep[s]; d++) {
            if (d == s) continue;
            int dominated = 1, strict = 1;
            for (int i = 0; i < B && dominated; i++) {
                if (L[i] < 1 || L[i] > Lmax) continue;
                const int32_t *t = time + (int64_t)i * Lmax * S, *m = mem + (int64_t)i * Lmax * S;
                const int32_t *x = trans + (int64_t)i * S * S;
                for (int l = 0; l < L[i]; l++) {
                    if (t[l * S + d] > t[l * S + s] || m[l * S + d] > m[l * S + s]) { dominated = 0; break; }
                    if (t[l * S + d] >= t[l * S + s]) strict = 0;
                }
                for (int k = 0; k < S && dominated; k++)
                    if (x[k * S + d] > x[k * S + s] || x[d * S + k] > x[s * S + k]) dominated = 0;
            }
            if (dominated && (d < s || strict)) keep[s] = 0;
        }
    }
}

/* ------------------------------------------------------------------ stage partitioning
 *
 * The model's layers are cut into P consecutive pipeline stages (Section 2 and Section 3 of the
 * paper: layers are distributed over stages so that the work per stage is balanced, and re-cut when
 * a stage becomes the bottleneck).  range_opt[a][n-1] is the optimum of the layer-wise search for the
 * stage made of layers a .. a+n-1 (ORC_INF when nothing fits); a pipeline runs at the pace of its
 * slowest stage, so the cut minimises the largest stage optimum:
 *   f[1][b] = opt(0,b),   f[k][b] = min_{k-1 <= a < b} max( f[k-1][a], opt(a,b) ).
 * cuts[0] = 0 < cuts[1] < ... < cuts[P] = Lm.  Several cut sets can share the optimal bottleneck.
 * The one reported, stated without the recurrence: among the cut sets whose every prefix (the first
 * k stages, k = 1..P) has the smallest bottleneck that any k-stage cut of the same layers can have,
 * the one smallest in the order (cuts[P-1], cuts[P-2], ..., cuts[1]).  The walk back from the end
 * that takes the lowest a attaining f[k][b] yields exactly that set (the tests enumerate all cut
 * sets on tie-heavy models and compare the cuts themselves).
 * bottleneck = ORC_INF and cuts = -1 when no partition is feasible or P > Lm.
 */
void orc_stage_partition(int Lm, int P, const int32_t *range_opt, int32_t *cuts, int32_t *bottleneck)
{
    for (int k = 0; k <= P; k++) cuts[k] = -1;
    *bottleneck = ORC_INF;
    if (P < 1 || P > Lm) return;
    int32_t *f = (int32_t *)malloc((size_t)(P + 1) * (Lm + 1) * sizeof(int32_t));
    int32_t *g = (int32_t *)malloc((size_t)(P + 1) * (Lm + 1) * sizeof(int32_t));
    for (int k = 1; k <= P; k++)
        for (int b = 0; b <= Lm; b++) {
            int32_t best = ORC_INF, arg = -1;
            if (b >= k) {
                if (k == 1) { best = range_opt[0 * Lm + (b - 1)]; arg = 0; }
                else
                    for (int a = k - 1; a < b; a++) {
                        int32_t left = f[(k - 1) * (Lm + 1) + a], here = range_opt[a * Lm + (b - a - 1)];
                        int32_t v = left > here ? left : here;
                        if (v < best) { best = v; arg = a; }
                    }
            }
            if (best >= ORC_INF) { best = ORC_INF; arg = -1; }
            f[k * (Lm + 1) + b] = best;
            g[k * (Lm + 1) + b] = arg;
        }
    *bottleneck = f[P * (Lm + 1) + Lm];
    if (*bottleneck < ORC_INF) {
        int b = Lm;
        for (int k = P; k >= 1; k--) { cuts[k] = b; b = g[k * (Lm + 1) + b]; }
        cuts[0] = 0;
    }
    free(f);
    free(g);
}

/* ------------------------------------------------------------------ plan switch
 *
 * Runtime adaptation (Sections 3 and 4 of the paper: the monitor re-evaluates, the optimiser
 * proposes a plan, the manager reshards the running job).  The paper gives no rule for when a
 * switch pays; the reading taken here:
 *   - moving layer l from its current strategy c_l to s reshards that layer once, at the price the
 *     cost model puts on that change of layout, trans_l(c_l, s); spread over `horizon` iterations
 *     the price per iteration is trans_l(c_l, s) / horizon (integer division), added to time(l,s);
 *     c_l < 0 (no plan yet) adds nothing; a horizon below 1 counts as 1; sums saturate at ORC_INF;
 *   - the job switches when the new optimum, raised by hysteresis_permille / 1000, is still below
 *     the cost of staying: new * (1000 + h) < cur * 1000.  A current plan that no longer fits
 *     (cost >= ORC_INF) is left whenever the new one is feasible; an infeasible new plan never wins.
 */
void orc_add_switch_cost(int L, int S, const int32_t *time, const int32_t *trans, int64_t tl,
                         const int32_t *cur_plan, int32_t horizon, int32_t *time_out)
{
    const int64_t H = horizon < 1 ? 1 : horizon;
    for (int l = 0; l < L; l++)
        for (int s = 0; s < S; s++) {
            int64_t v = time[l * S + s];
            const int c = cur_plan[l];
            if (c >= 0 && c < S) v += (int64_t)trans[l * tl + c * S + s] / H;
            time_out[l * S + s] = v >= ORC_INF ? ORC_INF : (int32_t)v;
        }
}

int orc_switch_decision(int64_t cur_cost, int64_t new_cost, int32_t hysteresis_permille)
{
    if (new_cost >= ORC_INF) return 0;
    if (cur_cost >= ORC_INF) return 1;
    return new_cost * (1000 + (int64_t)hysteresis_permille) < cur_cost * 1000;
}
