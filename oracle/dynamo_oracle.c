/*
 * CPU oracle for the configuration-selection hot path of DynamoLLM (arXiv 2408.00741).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain C, fp64, one loop per step of the definition, no blocking and
 * no reordering.  It shares no code, header, table or constant with the CUDA library; only the
 * tests, the smoke check and the benchmark's CPU-baseline / reference arms may call it.
 *
 * What it computes (paper passages in brackets):
 *   orc_bin_trace     requests (timestamp, input tokens, output tokens) [Sec. 3, trace fields] are
 *                     assigned a time window and one of KI*KO length classes [Sec. 3.1 and its
 *                     thresholds table] and counted per (window, class) [Sec. 3.1 "Request loads",
 *                     Sec. 3.2 load over time].
 *   orc_load          count / window length = requests per second per (window, class).
 *   orc_resolve       the profile function (load, class, TP, frequency) -> TTFT, TBT, power is a
 *                     table over a few profiled frequencies and load levels with linear
 *                     interpolation in between [Sec. 4.1 "Generating LLM profiles"; Sec. 5
 *                     implementation: linear 1-D interpolation].
 *   orc_eval_tile     for every candidate (N instances, TP, f): fair-share per-instance load,
 *                     expected TBT and power, the constraints of Eq. 1 (GPU budget, load covered,
 *                     performance within SLO) and the objective N x Energy^{TP,f}(L/N) [Sec. 4.1,
 *                     Eq. 1]; infeasible candidates get +inf [Sec. 4.2 scale-up/down: filter out
 *                     SLO-violating settings, then pick the minimum-energy one].
 *   orc_select_row    minimum-energy feasible candidate, lowest index on ties [Sec. 4.2]; also the
 *                     runner-up energy (for near-tie exemptions in parity tests).
 *   orc_totals        cluster energy per scenario and per window, GPUs in use per window, histogram
 *                     of chosen configurations [Sec. 6 cluster-level energy, GPUs per sharding].
 *   orc_mixed_select  Eq. 1 in full: a pool that mixes tensor parallelisms (counts per TP under a GPU
 *                     budget, load split by capacity, one frequency per TP), by enumeration.
 *   orc_reconf_select selection that counts the cost of re-configuring between windows (overhead table):
 *                     a shortest path over the windows, states = shardings, frequency free per window.
 *   orc_bin_tokens    token sums per (window, class): the load in tokens per second of Sec. 3.
 *   orc_carbon        operational carbon: window energies times a carbon-intensity trace [Sec. 6.4].
 *   orc_hier_select   the controller hierarchy of Sec. 4.2 on the same models: nodes per pool from the
 *                     epoch's peak load and the per-node maximum load (ceil(PL/ML)), sharding at the
 *                     highest frequency within those GPUs, then the frequency per window.
 *
 * Readings of points the paper leaves open: class = number of edges <= value; window =
 * t_ms / window_ms (unsigned integer division); utilisation u = (L/n)/cap with u > 1 infeasible; tables sampled at u_m = m/(M-1);
 * config index j = ((n-1)*T + t)*F + q; no feasible candidate -> index -1, energy +inf, excluded
 * from totals and counted in n_infeasible; energy in Wh per window.
 *
 * Parity pins (tests/ -m "not gpu"): closed forms of the synthetic profiles, Tables 1-3 of the
 * paper as energy rows for orc_select_row, boundary values of the thresholds table, invariants and
 * tiny-grid brute force.  Absolute energies versus the paper's Wh numbers: parity unpinned (the
 * measured H100 profiles behind them are not available).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_EINVAL (-1)

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---- stage (a): classify, window, count -------------------------------------------------- */

/* class of one length: how many ascending edges are <= the value */
static int32_t edge_class(uint32_t v, const uint32_t *edges, int32_t n_edges) {
    int32_t k = 0;
    for (int32_t e = 0; e < n_edges; ++e)
        if (edges[e] <= v) ++k;
    return k;
}

int orc_bin_trace(const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok, uint64_t n_req,
                  uint32_t window_ms, uint32_t n_windows,
                  const uint32_t *in_edges, int32_t n_in_edges,
                  const uint32_t *out_edges, int32_t n_out_edges,
                  uint32_t *counts /* [W][C] */, uint64_t *dropped) {
    if (window_ms == 0 || n_in_edges < 0 || n_out_edges < 0) return ORC_EINVAL;
    const int32_t KO = n_out_edges + 1;
    const int32_t C = (n_in_edges + 1) * KO;
    memset(counts, 0, (size_t)n_windows * (size_t)C * sizeof(uint32_t));
    uint64_t drop = 0;
    for (uint64_t i = 0; i < n_req; ++i) {
        uint32_t w = t_ms[i] / window_ms;
        if (w >= n_windows) { ++drop; continue; }
        int32_t ci = edge_class(in_tok[i], in_edges, n_in_edges);
        int32_t co = edge_class(out_tok[i], out_edges, n_out_edges);
        counts[(size_t)w * C + (size_t)(ci * KO + co)] += 1u;
    }
    *dropped = drop;
    return ORC_OK;
}

/* load in requests/s, computed and rounded in fp32: this fp32 number is the input of stage (b) */
void orc_load(const uint32_t *counts, uint64_t n_bins, float window_s, float *load) {
    for (uint64_t i = 0; i < n_bins; ++i) load[i] = (float)counts[i] / window_s;
}

/* ---- stage (b): profile lookup, feasibility, energy -------------------------------------- */

typedef struct {
    int32_t C, T, R, M;
    const int32_t *tp;         /* [T] */
    const float *f_grid;       /* [R] ascending */
    const float *ttft;         /* [C][T][R] */
    const float *cap;          /* [C][T][R] */
    const float *tbt;          /* [C][T][R][M] */
    const float *pw;           /* [C][T][R][M] */
} orc_profile;

typedef struct {
    int32_t F, Nmax;
    const float *f_cand;       /* [F] */
    const float *slo_ttft;     /* [C] */
    const float *slo_tbt;      /* [C] */
    int32_t gpu_budget;        /* <= 0: none */
    float window_s;
} orc_space;

/* position of candidate frequency q in the table grid: row r and weight w in [0,1] */
int orc_resolve(const float *f_grid, int32_t R, const float *f_cand, int32_t F,
                int32_t *row, double *weight) {
    if (R < 2) return ORC_EINVAL;
    for (int32_t q = 0; q < F; ++q) {
        double f = (double)f_cand[q];
        if (f < (double)f_grid[0] || f > (double)f_grid[R - 1]) return ORC_EINVAL;
        int32_t r = 0;
        for (int32_t i = 0; i <= R - 2; ++i)
            if ((double)f_grid[i] <= f) r = i;
        row[q] = r;
        weight[q] = (f - (double)f_grid[r]) / ((double)f_grid[r + 1] - (double)f_grid[r]);
    }
    return ORC_OK;
}

static double lerp(double a, double b, double w) { return (1.0 - w) * a + w * b; }

/* value of a [R][M] table at (row r, weight om) x (knot m, weight nu): bilinear */
static double table_at(const float *tab, int32_t M, int32_t r, double om, int32_t m, double nu) {
    double lo = lerp((double)tab[(size_t)r * M + m], (double)tab[(size_t)r * M + m + 1], nu);
    double hi = lerp((double)tab[(size_t)(r + 1) * M + m], (double)tab[(size_t)(r + 1) * M + m + 1], nu);
    return lerp(lo, hi, om);
}

/*
 * All J = Nmax*T*F candidates of one (window, class) tile with total load `load` (requests/s).
 * E[j] in Wh (+inf if infeasible).  Optional outputs (NULL to skip): per-candidate TBT, power,
 * utilisation; *margin = smallest relative distance of any deciding quantity to its bound
 * (|TBT-slo|/slo, |u-1|, |TTFT-slo|/slo) over the candidates of the tile.
 */
void orc_eval_tile(const orc_profile *p, const orc_space *sp, const int32_t *row, const double *weight,
                   int32_t c, double load, double *E, double *tbt_out, double *pow_out, double *u_out,
                   double *margin) {
    const int32_t T = p->T, R = p->R, M = p->M, F = sp->F;
    double mg = INFINITY;
    for (int32_t n = 1; n <= sp->Nmax; ++n) {
        for (int32_t t = 0; t < T; ++t) {
            for (int32_t q = 0; q < F; ++q) {
                const size_t j = ((size_t)(n - 1) * T + t) * F + q;
                const size_t ct = ((size_t)c * T + t) * R;
                const int32_t r = row[q];
                const double om = weight[q];
                const double ttft = lerp((double)p->ttft[ct + r], (double)p->ttft[ct + r + 1], om);
                const double cap = lerp((double)p->cap[ct + r], (double)p->cap[ct + r + 1], om);
                const double l = load / (double)n;                 /* fair share per instance */
                const double u = l / cap;                          /* utilisation */
                const double x = fmin(u, 1.0) * (double)(M - 1);
                int32_t m = (int32_t)floor(x);
                if (m > M - 2) m = M - 2;
                const double nu = x - (double)m;
                const double tbt = table_at(p->tbt + ct * M, M, r, om, m, nu);
                const double pw = table_at(p->pw + ct * M, M, r, om, m, nu);
                const double slo_a = (double)sp->slo_ttft[c], slo_b = (double)sp->slo_tbt[c];
                int ok = (ttft <= slo_a) && (tbt <= slo_b) && (u <= 1.0);
                if (sp->gpu_budget > 0 && n * p->tp[t] > sp->gpu_budget) ok = 0;
                E[j] = ok ? (double)n * pw * (double)sp->window_s / 3600.0 : INFINITY;
                if (tbt_out) tbt_out[j] = tbt;
                if (pow_out) pow_out[j] = pw;
                if (u_out) u_out[j] = u;
                double d1 = fabs(tbt - slo_b) / slo_b, d2 = fabs(u - 1.0), d3 = fabs(ttft - slo_a) / slo_a;
                if (d1 < mg) mg = d1;
                if (d2 < mg) mg = d2;
                if (d3 < mg) mg = d3;
            }
        }
    }
    if (margin) *margin = mg;
}

/* ---- stage (c): masked argmin, totals ----------------------------------------------------- */

/* smallest j attaining the minimum of E[0..J); -1 if the minimum is +inf.  *E2 = minimum over
   the other indices (+inf if none). */
void orc_select_row(const double *E, int64_t J, int32_t *best_idx, double *best_E, double *E2) {
    int64_t jb = -1;
    double eb = INFINITY;
    for (int64_t j = 0; j < J; ++j)
        if (E[j] < eb) { eb = E[j]; jb = j; }
    double e2 = INFINITY;
    for (int64_t j = 0; j < J; ++j)
        if (j != jb && E[j] < e2) e2 = E[j];
    *best_idx = (int32_t)jb;
    *best_E = eb;
    if (E2) *E2 = e2;
}

/* E tensor [S][W][C][J] for loads [S][W][C] */
int orc_eval_configs(const orc_profile *p, const orc_space *sp, const float *load, int64_t S, int64_t W,
                     double *E) {
    const int32_t C = p->C;
    const int64_t J = (int64_t)sp->Nmax * p->T * sp->F;
    int32_t *row = (int32_t *)malloc(sizeof(int32_t) * (size_t)sp->F);
    double *wt = (double *)malloc(sizeof(double) * (size_t)sp->F);
    int rc = orc_resolve(p->f_grid, p->R, sp->f_cand, sp->F, row, wt);
    if (rc == ORC_OK) {
        const int64_t tiles = S * W * C;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < tiles; ++i)
            orc_eval_tile(p, sp, row, wt, (int32_t)(i % C), (double)load[i], E + i * J, NULL, NULL, NULL, NULL);
    }
    free(row); free(wt);
    return rc;
}

/* per tile: argmin of a materialised E tensor */
void orc_select(const double *E, int64_t tiles, int64_t J, int32_t *best_idx, double *best_E, double *E2) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < tiles; ++i)
        orc_select_row(E + i * J, J, best_idx + i, best_E + i, E2 ? E2 + i : NULL);
}

/* evaluate then select, tile by tile (the row of J energies lives only inside the loop body) */
int orc_eval_select(const orc_profile *p, const orc_space *sp, const float *load, int64_t S, int64_t W,
                    int32_t *best_idx, double *best_E, double *E2, double *margin) {
    const int32_t C = p->C;
    const int64_t J = (int64_t)sp->Nmax * p->T * sp->F;
    int32_t *row = (int32_t *)malloc(sizeof(int32_t) * (size_t)sp->F);
    double *wt = (double *)malloc(sizeof(double) * (size_t)sp->F);
    int rc = orc_resolve(p->f_grid, p->R, sp->f_cand, sp->F, row, wt);
    if (rc == ORC_OK) {
        const int64_t tiles = S * W * C;
#pragma omp parallel
        {
            double *Erow = (double *)malloc(sizeof(double) * (size_t)J);
#pragma omp for schedule(static)
            for (int64_t i = 0; i < tiles; ++i) {
                orc_eval_tile(p, sp, row, wt, (int32_t)(i % C), (double)load[i], Erow, NULL, NULL, NULL,
                              margin ? margin + i : NULL);
                orc_select_row(Erow, J, best_idx + i, best_E + i, E2 ? E2 + i : NULL);
            }
            free(Erow);
        }
    }
    free(row); free(wt);
    return rc;
}

/*
 * Totals per scenario, summed in (w, c) order in fp64 over tiles that have a feasible candidate.
 * E_window[S][W], hist[S][J], gpus[S][W] optional (NULL to skip); n_of_j / tp_of_j give the
 * instance count and TP degree of candidate j (needed for gpus only).
 */
void orc_totals(const int32_t *best_idx, const double *best_E, int64_t S, int64_t W, int32_t C, int64_t J,
                const int32_t *n_of_j, const int32_t *tp_of_j,
                double *E_total, uint32_t *n_infeasible, double *E_window, uint32_t *hist, uint32_t *gpus) {
    if (hist) memset(hist, 0, sizeof(uint32_t) * (size_t)(S * J));
    for (int64_t s = 0; s < S; ++s) {
        double tot = 0.0;
        uint32_t bad = 0;
        for (int64_t w = 0; w < W; ++w) {
            double ew = 0.0;
            uint32_t g = 0;
            for (int32_t c = 0; c < C; ++c) {
                const int64_t i = (s * W + w) * C + c;
                const int32_t j = best_idx[i];
                if (j < 0) { ++bad; continue; }
                tot += best_E[i];
                ew += best_E[i];
                if (hist) hist[s * J + j] += 1u;
                if (gpus && n_of_j && tp_of_j) g += (uint32_t)(n_of_j[j] * tp_of_j[j]);
            }
            if (E_window) E_window[s * W + w] = ew;
            if (gpus) gpus[s * W + w] = g;
        }
        E_total[s] = tot;
        n_infeasible[s] = bad;
    }
}

/* ---- hierarchical control (Sec. 4.2): nodes per pool, then sharding, then frequency ---------- */

/*
 * One candidate of class c at total load `load`: energy (+inf if infeasible) and the smallest
 * relative distance of a deciding quantity to its bound.  Same arithmetic as orc_eval_tile.
 */
static double eval_candidate(const orc_profile *p, const orc_space *sp, const int32_t *row, const double *weight,
                             int32_t c, double load, int32_t n, int32_t t, int32_t q, int32_t budget, double *margin) {
    const int32_t R = p->R, M = p->M;
    const size_t ct = ((size_t)c * p->T + t) * R;
    const int32_t r = row[q];
    const double om = weight[q];
    const double ttft = lerp((double)p->ttft[ct + r], (double)p->ttft[ct + r + 1], om);
    const double cap = lerp((double)p->cap[ct + r], (double)p->cap[ct + r + 1], om);
    const double u = load / (double)n / cap;
    const double x = fmin(u, 1.0) * (double)(M - 1);
    int32_t m = (int32_t)floor(x);
    if (m > M - 2) m = M - 2;
    const double nu = x - (double)m;
    const double tbt = table_at(p->tbt + ct * M, M, r, om, m, nu);
    const double pw = table_at(p->pw + ct * M, M, r, om, m, nu);
    const double slo_a = (double)sp->slo_ttft[c], slo_b = (double)sp->slo_tbt[c];
    int ok = (ttft <= slo_a) && (tbt <= slo_b) && (u <= 1.0);
    if (budget > 0 && n * p->tp[t] > budget) ok = 0;
    if (margin) {
        double d = fabs(tbt - slo_b) / slo_b;
        if (fabs(u - 1.0) < d) d = fabs(u - 1.0);
        if (d < *margin) *margin = d;
    }
    return ok ? (double)n * pw * (double)sp->window_s / 3600.0 : INFINITY;
}

/*
 * ML of class c: the largest load one instance of the highest-performance configuration (largest TP,
 * highest candidate frequency) sustains with TTFT, TBT and capacity within bounds [Sec. 4.2
 * scale-out/in].  TBT is piecewise linear in the utilisation, so the largest feasible utilisation is
 * found segment by segment from the top.  0 if no load is feasible.
 */
double orc_max_load(const orc_profile *p, const orc_space *sp, const int32_t *row, const double *weight, int32_t c) {
    const int32_t t = p->T - 1, q = sp->F - 1, R = p->R, M = p->M;
    const size_t ct = ((size_t)c * p->T + t) * R;
    const int32_t r = row[q];
    const double om = weight[q];
    const double ttft = lerp((double)p->ttft[ct + r], (double)p->ttft[ct + r + 1], om);
    const double cap = lerp((double)p->cap[ct + r], (double)p->cap[ct + r + 1], om);
    const double slo_b = (double)sp->slo_tbt[c];
    if (!(ttft <= (double)sp->slo_ttft[c]) || !(cap > 0.0)) return 0.0;
    for (int32_t m = M - 2; m >= 0; --m) {
        const double a = table_at(p->tbt + ct * M, M, r, om, m, 0.0);
        const double b = table_at(p->tbt + ct * M, M, r, om, m, 1.0);
        if (b <= slo_b) return (double)(m + 1) / (double)(M - 1) * cap;
        if (a <= slo_b) return ((double)m + (slo_b - a) / (b - a)) / (double)(M - 1) * cap;
    }
    return 0.0;
}

/*
 * Hierarchical selection for loads [S][W][C].  Epoch lengths in windows: e1 (nodes per pool), e2
 * (sharding), 1 (frequency); e1 must be a multiple of e2.  The load predictor is the epoch's own peak.
 *   nodes[s][k1][c]  = max(1, ceil(PL / ML_c)), PL = peak load of the scale epoch; -1 if ML_c == 0
 *   shard[s][k2][c]  = (n-1)*T + t minimising the energy at the highest candidate frequency and the
 *                      shard epoch's peak load, over n*TP <= nodes*TP_max (and the space's own GPU
 *                      budget), lowest index on ties; -1 if none is feasible
 *   best_idx/best_E  per window: with (n, t) of its shard epoch, the feasible frequency of least
 *                      energy at the window's load (lowest on ties); -1 / +inf if none
 * Optional diagnostics for parity tests (NULL to skip): nodes_frac = PL/ML; shard_margin / shard_gap =
 * margin and relative runner-up gap of the sharding decision; freq_margin / freq_gap likewise per tile.
 */
int orc_hier_select(const orc_profile *p, const orc_space *sp, int32_t e1, int32_t e2, const float *load,
                    int64_t S, int64_t W, int32_t *nodes, int32_t *shard, int32_t *best_idx, double *best_E,
                    double *max_load, double *nodes_frac, double *shard_margin, double *shard_gap,
                    double *freq_margin, double *freq_gap) {
    if (e1 < 1 || e2 < 1 || e1 % e2 != 0) return ORC_EINVAL;
    const int32_t C = p->C, T = p->T, F = sp->F;
    int32_t *row = (int32_t *)malloc(sizeof(int32_t) * (size_t)F);
    double *wt = (double *)malloc(sizeof(double) * (size_t)F);
    int rc = orc_resolve(p->f_grid, p->R, sp->f_cand, F, row, wt);
    if (rc != ORC_OK) { free(row); free(wt); return rc; }
    const int64_t K1 = (W + e1 - 1) / e1, K2 = (W + e2 - 1) / e2;
    const int32_t gpus_per_node = p->tp[T - 1];
    double *ml = (double *)malloc(sizeof(double) * (size_t)C);
    for (int32_t c = 0; c < C; ++c) {
        ml[c] = orc_max_load(p, sp, row, wt, c);
        if (max_load) max_load[c] = ml[c];
    }
#pragma omp parallel for schedule(static) collapse(2)
    for (int64_t s = 0; s < S; ++s) {
        for (int32_t c = 0; c < C; ++c) {
            for (int64_t k1 = 0; k1 < K1; ++k1) {
                /* scale-out/in: nodes for the peak of the epoch */
                const int64_t w1a = k1 * e1, w1b = (w1a + e1 < W) ? w1a + e1 : W;
                double PL = 0.0;
                for (int64_t w = w1a; w < w1b; ++w) {
                    const double L = (double)load[(s * W + w) * C + c];
                    if (L > PL) PL = L;
                }
                int32_t nn = -1;
                if (ml[c] > 0.0) {
                    nn = (int32_t)ceil(PL / ml[c]);
                    if (nn < 1) nn = 1;
                }
                nodes[(s * K1 + k1) * C + c] = nn;
                if (nodes_frac) nodes_frac[(s * K1 + k1) * C + c] = ml[c] > 0.0 ? PL / ml[c] : INFINITY;
                int32_t budget = nn > 0 ? nn * gpus_per_node : 0;
                if (sp->gpu_budget > 0 && budget > sp->gpu_budget) budget = sp->gpu_budget;

                /* shard-up/down: instances x TP at the highest frequency, peak of the shard epoch */
                for (int64_t w2a = w1a; w2a < w1b; w2a += e2) {
                    const int64_t k2 = w2a / e2, w2b = (w2a + e2 < w1b) ? w2a + e2 : w1b;
                    double PL2 = 0.0;
                    for (int64_t w = w2a; w < w2b; ++w) {
                        const double L = (double)load[(s * W + w) * C + c];
                        if (L > PL2) PL2 = L;
                    }
                    int32_t best_nt = -1;
                    double eb = INFINITY, e2nd = INFINITY, mg = INFINITY;
                    if (nn > 0) {
                        for (int32_t n = 1; n <= sp->Nmax; ++n)
                            for (int32_t t = 0; t < T; ++t) {
                                const double E = eval_candidate(p, sp, row, wt, c, PL2, n, t, F - 1, budget, &mg);
                                if (E < eb) { e2nd = eb; eb = E; best_nt = (n - 1) * T + t; }
                                else if (E < e2nd) e2nd = E;
                            }
                    }
                    shard[(s * K2 + k2) * C + c] = best_nt;
                    if (shard_margin) shard_margin[(s * K2 + k2) * C + c] = mg;
                    if (shard_gap) shard_gap[(s * K2 + k2) * C + c] = best_nt >= 0 ? (e2nd - eb) / eb : INFINITY;

                    /* scale-up/down: frequency per window for the chosen sharding */
                    for (int64_t w = w2a; w < w2b; ++w) {
                        const int64_t i = (s * W + w) * C + c;
                        int32_t bq = -1;
                        double fb = INFINITY, f2 = INFINITY, fm = INFINITY;
                        if (best_nt >= 0) {
                            const int32_t n = best_nt / T + 1, t = best_nt % T;
                            for (int32_t q = 0; q < F; ++q) {
                                const double E = eval_candidate(p, sp, row, wt, c, (double)load[i], n, t, q, 0, &fm);
                                if (E < fb) { f2 = fb; fb = E; bq = q; }
                                else if (E < f2) f2 = E;
                            }
                        }
                        best_idx[i] = bq >= 0 ? best_nt * F + bq : -1;
                        best_E[i] = fb;
                        if (freq_margin) freq_margin[i] = fm;
                        if (freq_gap) freq_gap[i] = bq >= 0 ? (f2 - fb) / fb : INFINITY;
                    }
                }
            }
        }
    }
    free(row); free(wt); free(ml);
    return ORC_OK;
}

/* ---- pools that mix tensor parallelisms (Sec. 4.1, Eq. 1 in full) ------------------------------- */

/*
 * Eq. 1 lets one pool hold instances of several tensor parallelisms at once: counts N^{TP_i}, one
 * frequency f^{TP_i} per parallelism, a load L^{TP_i} per instance, under the GPU budget
 * sum_i TP_i * N^{TP_i} <= N, with all the load served and every instance within the SLO; the objective
 * is sum_i N^{TP_i} * Energy^{TP_i, f_i}(L^{TP_i}).  The paper hands this to a solver; here the count
 * tuples are enumerated.  Readings (the paper leaves the split and the enumeration open):
 *   - counts n_t = 0..Nmax per TP index t, not all zero, sum_t n_t*TP_t <= gpu_budget (required > 0);
 *   - the load is split in proportion to the capacity at the highest candidate frequency: the group
 *     of type t gets L * n_t*capH_t / A, A = sum_j n_j*capH_j, capH_t = cap(c, t, highest candidate f),
 *     so every instance runs at the same fraction L/A of its top-frequency capacity;
 *   - each group then takes, on its own, the feasible frequency of least energy for its share (fair
 *     share inside the group, TTFT / TBT / capacity as for a single-type pool), lowest q on ties; a
 *     tuple with a group that has no feasible frequency is infeasible;
 *   - energy of the tuple = sum over groups in ascending t; the tuple of least energy wins, ties go to
 *     the lowest tuple number, tuples being numbered in odometer order with n_0 (smallest TP) the
 *     fastest digit.
 * Outputs per tile (s, w, c): counts[T], freq[T] (-1 where the count is 0; all -1 and E = +inf if no
 * tuple is feasible), tuple number (position among the budget-feasible tuples in odometer order, -1 if
 * none), energy.  Optional diagnostics (NULL to skip): E2 = least energy over the other tuples, margin =
 * smallest relative distance of a deciding quantity to its bound over everything evaluated for the tile.
 */
int orc_mixed_select(const orc_profile *p, const orc_space *sp, const float *load, int64_t S, int64_t W,
                     int32_t *counts, int32_t *freq, int32_t *tuple_no, double *best_E, double *E2, double *margin) {
    const int32_t C = p->C, T = p->T, F = sp->F, Nmax = sp->Nmax, B = sp->gpu_budget;
    if (B <= 0 || T > 8) return ORC_EINVAL;
    int32_t *row = (int32_t *)malloc(sizeof(int32_t) * (size_t)F);
    double *wt = (double *)malloc(sizeof(double) * (size_t)F);
    int rc = orc_resolve(p->f_grid, p->R, sp->f_cand, F, row, wt);
    if (rc != ORC_OK) { free(row); free(wt); return rc; }
    const int64_t tiles = S * W * C;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < tiles; ++i) {
        const int32_t c = (int32_t)(i % C);
        const double L = (double)load[i];
        double capH[8];
        for (int32_t t = 0; t < T; ++t) {
            const size_t ct = ((size_t)c * T + t) * p->R;
            capH[t] = lerp((double)p->cap[ct + row[F - 1]], (double)p->cap[ct + row[F - 1] + 1], wt[F - 1]);
        }
        int32_t n[8] = {0}, bn[8], bq[8];
        for (int32_t t = 0; t < T; ++t) { bn[t] = -1; bq[t] = -1; }
        double eb = INFINITY, e2nd = INFINITY, mg = INFINITY;
        int32_t number = -1, bnum = -1;
        for (;;) {
            /* next tuple in odometer order, n_0 fastest */
            int32_t t = 0;
            while (t < T && n[t] == Nmax) n[t++] = 0;
            if (t == T) break;
            ++n[t];
            int64_t gpus = 0;
            for (int32_t k = 0; k < T; ++k) gpus += (int64_t)n[k] * p->tp[k];
            if (gpus > B) continue;
            ++number;
            double A = 0.0;
            for (int32_t k = 0; k < T; ++k) A += (double)n[k] * capH[k];
            double E = 0.0;
            int32_t qs[8];
            for (int32_t k = 0; k < T; ++k) {
                qs[k] = -1;
                if (n[k] == 0) continue;
                const double share = L * ((double)n[k] * capH[k]) / A;      /* load of the whole group */
                double eg = INFINITY;
                for (int32_t q = 0; q < F; ++q) {
                    const double e = eval_candidate(p, sp, row, wt, c, share, n[k], k, q, 0, &mg);
                    if (e < eg) { eg = e; qs[k] = q; }
                }
                E += eg;                                                     /* +inf if the group has no frequency */
            }
            if (E < eb) {
                e2nd = eb; eb = E; bnum = number;
                for (int32_t k = 0; k < T; ++k) { bn[k] = n[k]; bq[k] = qs[k]; }
            } else if (E < e2nd) {
                e2nd = E;
            }
        }
        for (int32_t k = 0; k < T; ++k) {
            counts[i * T + k] = bnum >= 0 ? bn[k] : -1;
            freq[i * T + k] = bnum >= 0 ? bq[k] : -1;
        }
        tuple_no[i] = bnum;
        best_E[i] = eb;
        if (E2) E2[i] = e2nd;
        if (margin) margin[i] = mg;
    }
    free(row); free(wt);
    return ORC_OK;
}

/* ---- selection that accounts for the cost of re-configuring (Sec. 4.2, "Accounting for the overheads") ---- */

/*
 * The controllers weigh the energy a new configuration saves against the cost of getting there, which they
 * read from an Overhead Table [Sec. 4.2]; changing the sharding of an instance costs transfer time that depends
 * on the source and destination parallelism [Sec. 4.3, table of re-sharding overheads], changing the frequency
 * costs next to nothing [Sec. 4.3, "Scaling up/down the frequency"].  Here that trade-off is solved exactly for
 * one (scenario, class) over the whole horizon.  Readings:
 *   - a state is a sharding sigma = (n, TP index t), numbered sigma = (n-1)*T + t, NS = Nmax*T states;
 *   - the frequency is free in every window: the cost of state sigma in window w is
 *     cost_w(sigma) = min over q of E(w, n, t, q) (the evaluation of Eq. 1), lowest q on ties, +inf if none;
 *   - moving from sigma' in window w-1 to sigma in window w costs R[sigma'][sigma] (Wh, the caller's overhead
 *     table, NS x NS, used as given); the first window is free to start anywhere;
 *   - the schedule minimises  sum_w cost_w(sigma_w) + sum_{w>=1} R[sigma_{w-1}][sigma_w]  (a shortest path
 *     through the windows); forward recursion D_w(sigma) = cost_w(sigma) + min_{sigma'} (D_{w-1}(sigma') +
 *     R[sigma'][sigma]) with the lowest sigma' on ties, last state the lowest sigma attaining the minimum;
 *   - a (scenario, class) with a window in which no state is feasible has no schedule: indices -1, total +inf.
 * Outputs: best_idx[S][W][C] = sigma_w*F + q_w (or -1), best_E[S][W][C] = cost_w(sigma_w) (+inf if none),
 * path_total[S][C] = the minimised sum (window energies plus transition costs).
 */
int orc_reconf_select(const orc_profile *p, const orc_space *sp, const float *R, const float *load, int64_t S, int64_t W,
                      int32_t *best_idx, double *best_E, double *path_total) {
    const int32_t C = p->C, T = p->T, F = sp->F, Nmax = sp->Nmax;
    const int64_t NS = (int64_t)Nmax * T;
    int32_t *row = (int32_t *)malloc(sizeof(int32_t) * (size_t)F);
    double *wt = (double *)malloc(sizeof(double) * (size_t)F);
    int rc = orc_resolve(p->f_grid, p->R, sp->f_cand, F, row, wt);
    if (rc != ORC_OK) { free(row); free(wt); return rc; }
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (int64_t s = 0; s < S; ++s) {
        for (int32_t c = 0; c < C; ++c) {
            double *cost = (double *)malloc(sizeof(double) * (size_t)(W * NS));
            int32_t *qb = (int32_t *)malloc(sizeof(int32_t) * (size_t)(W * NS));
            int32_t *from = (int32_t *)malloc(sizeof(int32_t) * (size_t)(W * NS));
            double *D = (double *)malloc(sizeof(double) * (size_t)NS), *Dn = (double *)malloc(sizeof(double) * (size_t)NS);
            /* window costs: the frequency of least energy for every sharding */
            for (int64_t w = 0; w < W; ++w) {
                const double L = (double)load[(s * W + w) * C + c];
                for (int64_t g = 0; g < NS; ++g) {
                    const int32_t n = (int32_t)(g / T) + 1, t = (int32_t)(g % T);
                    double eb = INFINITY;
                    int32_t bq = -1;
                    for (int32_t q = 0; q < F; ++q) {
                        const double e = eval_candidate(p, sp, row, wt, c, L, n, t, q, sp->gpu_budget, NULL);
                        if (e < eb) { eb = e; bq = q; }
                    }
                    cost[w * NS + g] = eb;
                    qb[w * NS + g] = bq;
                }
            }
            /* shortest path through the windows */
            for (int64_t g = 0; g < NS; ++g) { D[g] = W > 0 ? cost[g] : 0.0; from[g] = -1; }
            for (int64_t w = 1; w < W; ++w) {
                for (int64_t g = 0; g < NS; ++g) {
                    double best = INFINITY;
                    int32_t arg = -1;
                    for (int64_t h = 0; h < NS; ++h) {
                        const double v = D[h] + (double)R[h * NS + g];
                        if (v < best) { best = v; arg = (int32_t)h; }
                    }
                    Dn[g] = cost[w * NS + g] + best;
                    from[w * NS + g] = arg;
                }
                double *tmp = D; D = Dn; Dn = tmp;
            }
            double tot = INFINITY;
            int64_t g = -1;
            for (int64_t h = 0; h < NS; ++h)
                if (D[h] < tot) { tot = D[h]; g = h; }
            path_total[s * C + c] = W > 0 ? tot : 0.0;
            for (int64_t w = W - 1; w >= 0; --w) {
                const int64_t i = (s * W + w) * C + c;
                if (g < 0) { best_idx[i] = -1; best_E[i] = INFINITY; continue; }
                best_idx[i] = (int32_t)(g * F + qb[w * NS + g]);
                best_E[i] = cost[w * NS + g];
                g = from[w * NS + g];
            }
            free(cost); free(qb); free(from); free(D); free(Dn);
        }
    }
    free(row); free(wt);
    return ORC_OK;
}

/* ---- token-weighted loads and carbon (Sec. 3 load in tokens per second; Sec. 6.4 carbon) ------------ */

/*
 * The paper states loads in tokens per second (TPS) [Sec. 3, characterisation tables; Sec. 3.2].  Per (window,
 * class) the sums of input tokens and of output tokens of the requests that fall there; window and class as in
 * orc_bin_trace; requests past the last window add nothing.  Exact 64-bit integer sums.
 */
int orc_bin_tokens(const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok, uint64_t n_req,
                   uint32_t window_ms, uint32_t n_windows, const uint32_t *in_edges, int32_t n_in_edges,
                   const uint32_t *out_edges, int32_t n_out_edges, uint64_t *tok_in, uint64_t *tok_out) {
    if (window_ms == 0 || n_in_edges < 0 || n_out_edges < 0) return ORC_EINVAL;
    const int32_t KO = n_out_edges + 1, C = (n_in_edges + 1) * KO;
    memset(tok_in, 0, sizeof(uint64_t) * (size_t)n_windows * (size_t)C);
    memset(tok_out, 0, sizeof(uint64_t) * (size_t)n_windows * (size_t)C);
    for (uint64_t i = 0; i < n_req; ++i) {
        const uint32_t w = t_ms[i] / window_ms;
        if (w >= n_windows) continue;
        const int32_t c = edge_class(in_tok[i], in_edges, n_in_edges) * KO + edge_class(out_tok[i], out_edges, n_out_edges);
        tok_in[(size_t)w * C + c] += in_tok[i];
        tok_out[(size_t)w * C + c] += out_tok[i];
    }
    return ORC_OK;
}

/* tokens per second of a (window, class), computed and rounded in fp32 like orc_load */
void orc_load_tps(const uint64_t *tok_in, const uint64_t *tok_out, uint64_t n_bins, float window_s, float *tps) {
    for (uint64_t i = 0; i < n_bins; ++i) tps[i] = (float)(tok_in[i] + tok_out[i]) / window_s;
}

/*
 * Operational carbon of a scenario: the energy of every window times the carbon intensity of the grid in that
 * window, summed over the windows in order [Sec. 6.4: energy over time combined with an intensity trace].
 * E_window[S][W] in Wh, intensity[W] in gCO2 per kWh; carbon[S] in gCO2.
 */
void orc_carbon(const double *E_window, const float *intensity, int64_t S, int64_t W, double *carbon) {
    for (int64_t s = 0; s < S; ++s) {
        double acc = 0.0;
        for (int64_t w = 0; w < W; ++w) acc += E_window[s * W + w] * (double)intensity[w] / 1000.0;
        carbon[s] = acc;
    }
}
