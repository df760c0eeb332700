/*
 * dynamo.h -- C ABI of the B200 configuration-sweep library (libdynamo.so).
 *
 * The library evaluates, on one GPU, the search that DynamoLLM (arXiv 2408.00741) states in
 * Sec. 4.1 / Eq. 1 and Sec. 4.2: for every request class and time window, every candidate
 * (number of instances N, tensor-parallel degree TP, GPU frequency f) is checked against the
 * profile-derived latency model and the SLOs, its energy is computed, and the minimum-energy
 * feasible candidate is chosen.  Three stages:
 *
 *   (a) dyn_bin_trace     trace (timestamp, input tokens, output tokens) -> per-(window, class)
 *                         request counts and loads                      [Sec. 3, Sec. 3.1, Sec. 3.2]
 *   (b) dyn_eval_configs  loads x candidates -> energy tensor with +inf where a constraint of Eq. 1
 *                         fails                                         [Sec. 4.1, Eq. 1]
 *   (c) dyn_select        masked argmin per (window, class) + cluster totals      [Sec. 4.2, Sec. 6]
 *       dyn_eval_select   (b)+(c) fused, no energy tensor
 *
 * Conventions for every call
 *   - returns DYN_OK (0) or a negative dyn_status; never throws, never aborts, never traps the GPU;
 *   - work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream) and the
 *     call returns without synchronising; results are valid once the stream reaches that point;
 *   - pointers named d_* are DEVICE pointers owned by the caller; all other pointers are HOST
 *     pointers that are read before the call returns; the library allocates nothing;
 *   - tensors are dense, row-major, in the index order written in brackets;
 *   - candidate index  j = ((n-1)*T + t)*F + q  with n = 1..Nmax (slowest), t = TP index, q =
 *     frequency index (fastest); J = Nmax*T*F.  Ties in energy go to the lowest j.
 *   - argument errors are detected on the host before anything is enqueued.
 */
#ifndef DYNAMO_H_
#define DYNAMO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DYN_OK = 0,
    DYN_EINVAL = -1,        /* NULL required pointer, bad size, non-ascending edges / grids, ... */
    DYN_ECUDA = -2,         /* a CUDA runtime call failed; see dyn_last_cuda_error() */
    DYN_EUNSUPPORTED = -3,  /* valid request outside the built limits (see each call) */
    DYN_EWORKSPACE = -4     /* workspace missing, misaligned (256 B) or smaller than dyn_workspace_bytes() */
} dyn_status;

/* Static, human-readable text for a status code. */
const char *dyn_strerror(int status);

/* cudaError_t (as int) behind the most recent DYN_ECUDA returned on the calling thread, else 0. */
int dyn_last_cuda_error(void);

/* Limits the library was built with. */
#define DYN_MAX_EDGES 15      /* per axis: at most 16 x 16 classes */
#define DYN_MAX_F 256         /* candidate frequencies */
#define DYN_MAX_T 16          /* TP degrees */

/* ---------------------------------------------------------------------------------------------
 * (a) Trace binning.  [Sec. 3: a trace record is (timestamp, #input tokens, #output tokens);
 *     Sec. 3.1 and its thresholds table: 3 x 3 length classes; Sec. 3.2: load per class over time]
 *
 * Request i falls in window w = t_ms[i] / window_ms (unsigned integer division) and class
 * c = ci*KO + co, where ci = number of in_edges <= in_tok[i], co likewise, KI = n_in_edges+1,
 * KO = n_out_edges+1, C = KI*KO.  With in_edges {256, 1024} and out_edges {100, 350} this is the
 * paper's SS, SM, SL, MS, ..., LL order.  Requests with w >= n_windows are counted in *d_dropped.
 * The trace need not be sorted; a time-sorted trace is the fast case.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    uint32_t window_ms;          /* > 0 */
    uint32_t n_windows;          /* W > 0 */
    int32_t n_in_edges;          /* 0 .. DYN_MAX_EDGES */
    int32_t n_out_edges;         /* 0 .. DYN_MAX_EDGES */
    const uint32_t *in_edges;    /* host, strictly ascending */
    const uint32_t *out_edges;   /* host, strictly ascending */
} dyn_bin_spec;

/*
 * d_t_ms, d_in_tok, d_out_tok : device, uint32 [n_req] each (structure of arrays), read only.
 * d_counts  : device, uint32 [W][C], overwritten (exact counts; W*C must be < 2^31).
 * d_load    : device, float  [W][C] = (float)count / (window_ms/1000 as float), or NULL to skip.
 * d_dropped : device, uint64 [1], overwritten.
 * n_req may be 0.  Errors: DYN_EINVAL (NULL pointer, window_ms or n_windows 0, edges not strictly
 * ascending, too many edges, W*C >= 2^31), DYN_ECUDA.
 */
int dyn_bin_trace(const dyn_bin_spec *spec, const uint32_t *d_t_ms, const uint32_t *d_in_tok,
                  const uint32_t *d_out_tok, uint64_t n_req, uint32_t *d_counts, float *d_load,
                  uint64_t *d_dropped, void *stream);

/*
 * Token-weighted loads.  [Sec. 3 and Sec. 3.2 state loads in tokens per second (TPS); the characterisation
 * tables quote a medium load as 2K TPS.]  Same windows and classes as dyn_bin_trace; per (window, class) the sum
 * of the input tokens and the sum of the output tokens of its requests, exact in 64 bits for any values and any
 * order of the trace; requests past the last window add nothing.
 * d_tok_in, d_tok_out : device, uint64 [W][C], overwritten.
 * d_load_tps          : device, float [W][C] = (float)(tok_in + tok_out) / (window_ms/1000 as float), or NULL.
 * Errors: as dyn_bin_trace.
 */
int dyn_bin_tokens(const dyn_bin_spec *spec, const uint32_t *d_t_ms, const uint32_t *d_in_tok,
                   const uint32_t *d_out_tok, uint64_t n_req, uint64_t *d_tok_in, uint64_t *d_tok_out,
                   float *d_load_tps, void *stream);

/* ---------------------------------------------------------------------------------------------
 * (b) Profiles and the candidate space.  [Sec. 4.1 "Generating LLM profiles": the profile maps
 *     (load, request class, TP, frequency) to energy/power and TTFT/TBT, measured at a few
 *     frequencies and load levels and interpolated linearly in between.]
 *
 * Tables hold, per class c, TP index t and profiled frequency row r:
 *   ttft[c][t][r]      time to first token (s)
 *   cap[c][t][r]       largest per-instance load the instance sustains (requests/s), > 0
 *   tbt[c][t][r][m]    time between tokens (s) at utilisation u_m = m/(M-1), m = 0..M-1
 *   pow[c][t][r][m]    power of one instance (W) at utilisation u_m
 * A candidate frequency between two rows is interpolated linearly in f, utilisation linearly in
 * u (bilinear overall).  NaN table entries give unspecified results.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t C, T, R, M;          /* classes, TP degrees (<= DYN_MAX_T), frequency rows (>= 2), knots (>= 2) */
    const int32_t *tp;           /* host [T], strictly ascending, > 0 */
    const float *f_grid_mhz;     /* host [R], strictly ascending */
    const float *d_ttft;         /* device [C][T][R] */
    const float *d_cap;          /* device [C][T][R] */
    const float *d_tbt;          /* device [C][T][R][M] */
    const float *d_pow;          /* device [C][T][R][M] */
} dyn_profile;

typedef struct {
    int32_t F, Nmax;             /* 1 <= F <= DYN_MAX_F; Nmax >= 1; Nmax*T*F < 2^31 */
    const float *f_cand_mhz;     /* host [F], strictly ascending, inside [f_grid[0], f_grid[R-1]] */
    const float *slo_ttft_s;     /* host [C] */
    const float *slo_tbt_s;      /* host [C] */
    int32_t gpu_budget;          /* Eq. 1 first constraint: n*TP <= gpu_budget; <= 0 means no budget */
    float window_s;              /* window length in seconds (energy is Wh per window) */
} dyn_space;

/*
 * Evaluation of one candidate for a tile (s, w, c) with load L = d_load[s][w][c]   [Eq. 1]:
 *   l = L/n (fair share),  u = l / cap(c,t,f),  TBT and P interpolated at (f, min(u,1));
 *   feasible  <=>  TTFT(c,t,f) <= slo_ttft[c]  and  TBT <= slo_tbt[c]  and  u <= 1
 *                  and (gpu_budget <= 0 or n*TP_t <= gpu_budget);
 *   E = n * P * window_s / 3600  (Wh)  if feasible, +inf otherwise.
 * Arithmetic is fp32; results agree with an fp64 evaluation to about 1e-6 relative, and the
 * feasibility decision can differ where a deciding quantity is within rounding of its bound.
 */

/* Scratch memory (bytes, multiple of 256) that dyn_eval_configs / dyn_select / dyn_eval_select need
 * for this problem shape; d_ws must be 256-byte aligned.  The scratch holds the candidate-resolved
 * tables and partial sums; its contents are meaningless between calls.  Returns 0 on bad input. */
size_t dyn_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W);

/*
 * d_load : device float [S][W][C] (requests/s, >= 0).   d_E : device float [S][W][C][J], overwritten.
 * Errors: DYN_EINVAL, DYN_EUNSUPPORTED (F > DYN_MAX_F, T > DYN_MAX_T, candidate frequency outside the
 * grid), DYN_EWORKSPACE, DYN_ECUDA.
 */
int dyn_eval_configs(const dyn_profile *profile, const dyn_space *space, const float *d_load,
                     int64_t S, int64_t W, float *d_E, void *d_ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * (c) Selection and totals.  [Sec. 4.2 scale-up/down: drop the settings that violate the SLO, then
 *     take the one with the least energy; Sec. 6: cluster energy over time, GPUs in use.]
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t *d_best_idx;         /* [S][W][C] chosen j, -1 if no candidate is feasible; required */
    float *d_best_E;             /* [S][W][C] its energy (Wh), +inf if none; required */
    double *d_E_total;           /* [S] sum of chosen energies over feasible tiles; required */
    uint32_t *d_n_infeasible;    /* [S] tiles without a feasible candidate; required */
    double *d_E_window;          /* [S][W] energy per window, or NULL */
    uint32_t *d_hist;            /* [S][J] how often each candidate was chosen, or NULL */
    uint32_t *d_gpus;            /* [S][W] sum over classes of n* x TP*, or NULL */
} dyn_select_out;

/*
 * Argmin over a materialised energy tensor d_E [S][W][C][J] (+inf = infeasible).
 * n_of_j, tp_of_j : host int32 [J], instance count and TP degree of candidate j; needed only when
 * out->d_gpus is set (else may be NULL).  They are copied with cudaMemcpyAsync on `stream`: pageable arrays are
 * staged before the call returns (which makes the call wait for earlier work on the stream), pinned arrays
 * are read when the stream reaches the copy and must stay valid until then.  dyn_eval_select needs neither.  Sums are fp64, accumulated in a fixed order: results are
 * bit-identical from run to run.  Workspace: dyn_select_workspace_bytes(S, W, J).
 */
size_t dyn_select_workspace_bytes(int64_t S, int64_t W, int64_t J);
int dyn_select(const float *d_E, int64_t S, int64_t W, int32_t C, int32_t J, const int32_t *n_of_j,
               const int32_t *tp_of_j, const dyn_select_out *out, void *d_ws, size_t ws_bytes,
               void *stream);

/* (b)+(c) in one pass: same results as dyn_eval_configs followed by dyn_select, without the
 * [S][W][C][J] tensor (which need not fit in memory).  Workspace: dyn_workspace_bytes(). */
int dyn_eval_select(const dyn_profile *profile, const dyn_space *space, const float *d_load,
                    int64_t S, int64_t W, const dyn_select_out *out, void *d_ws, size_t ws_bytes,
                    void *stream);

/*
 * Operational carbon.  [Sec. 6.4: the energy over time is combined with the carbon intensity of the grid over
 * time.]  d_carbon[s] = sum over windows, in a fixed order, of d_E_window[s][w] (Wh, e.g. dyn_select_out.d_E_window)
 * x d_intensity[w] (gCO2 per kWh) / 1000, in fp64 (gCO2); bit-identical from run to run.
 */
int dyn_carbon(const double *d_E_window, const float *d_intensity, int64_t S, int64_t W, double *d_carbon, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Hierarchical control.  [Sec. 4.2: instead of the joint search, three controllers set one knob each
 * at their own time scale -- scale-out/in: the number of nodes of a pool for the epoch's peak load PL,
 * ceil(PL / ML) with ML the largest load one node sustains in the highest-performance configuration;
 * shard-up/down: how the machine's GPUs are split into instances x TP, decided at the highest frequency;
 * scale-up/down: the frequency, per window, among those that keep the SLO.]
 *
 * Epoch lengths are in windows: scale_epoch_windows (nodes), shard_epoch_windows (sharding), 1
 * (frequency); scale_epoch_windows must be a multiple of shard_epoch_windows.  The load "prediction"
 * of an epoch is its own peak.  A node has TP_max = tp[T-1] GPUs.  Per scenario s and class c:
 *   d_nodes[s][k1][c] = max(1, ceil(PL / ML_c)), PL = max load over scale epoch k1; -1 if no load is
 *                       feasible at (TP_max, highest candidate frequency);
 *   d_shard[s][k2][c] = (n-1)*T + t of least energy at the highest candidate frequency and the peak
 *                       load of shard epoch k2, over n*TP_t <= nodes*TP_max (and space->gpu_budget when
 *                       set), lowest index on ties; -1 if none is feasible;
 *   out->d_best_idx / d_best_E [s][w][c]: for that (n, t), the feasible frequency of least energy at
 *                       the window's load (lowest on ties), as candidate index j; -1 / +inf if none.
 * The totals in `out` are as in dyn_select.  K1 = ceil(W / scale_epoch_windows), K2 likewise.
 * Workspace: dyn_hier_workspace_bytes().  Errors: as dyn_eval_select, plus DYN_EINVAL for bad epochs
 * or NULL d_nodes / d_shard.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t scale_epoch_windows;
    int32_t shard_epoch_windows;
} dyn_hier_spec;

size_t dyn_hier_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W);
int dyn_hier_select(const dyn_profile *profile, const dyn_space *space, const dyn_hier_spec *hier,
                    const float *d_load, int64_t S, int64_t W, int32_t *d_nodes, int32_t *d_shard,
                    const dyn_select_out *out, void *d_ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Pools that mix tensor parallelisms.  [Sec. 4.1, Eq. 1 in full: the pool may hold N^{TP_i} instances of
 * several parallelisms at once, each parallelism at its own frequency f^{TP_i} and with its own per-instance
 * load L^{TP_i}, under  sum_i TP_i * N^{TP_i} <= N,  sum_i N^{TP_i} * L^{TP_i} >= L  and the SLO for every
 * instance; the objective is  sum_i N^{TP_i} * Energy^{TP_i, f_i}(L^{TP_i}).]
 *
 * The paper leaves the search to a solver; this call enumerates.  Per tile (s, w, c) with load L:
 *   - count tuples (n_0, ..., n_{T-1}), n_t = 0 .. space->Nmax instances of TP index t, not all zero, with
 *     sum_t n_t * tp[t] <= space->gpu_budget (the budget is REQUIRED here, > 0);
 *   - the load is split in proportion to capacity at the highest candidate frequency: the group of TP index t
 *     serves L * n_t*capH_t / sum_j n_j*capH_j, capH_t = cap(c, t, f_cand[F-1]);
 *   - every group takes, on its own, the feasible candidate frequency of least energy for its share (fair
 *     share within the group; TTFT, TBT and capacity as in the single-type evaluation above), lowest
 *     frequency index on ties; a tuple with a group that has none is infeasible;
 *   - the tuple's energy is the sum over its groups; the tuple of least energy is chosen, lowest tuple
 *     number on ties.  Tuples are numbered 0, 1, ... in odometer order with n_0 the fastest digit, counting
 *     only tuples within the budget.
 * Limits: T <= 4, Nmax <= 255, at most 2^20 tuples within the budget (else DYN_EUNSUPPORTED).
 * Workspace: dyn_mixed_workspace_bytes().  Errors: as dyn_eval_select, plus DYN_EINVAL for gpu_budget <= 0.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t *d_counts;           /* [S][W][C][T] chosen n_t; -1 in every slot if no tuple is feasible; required */
    int32_t *d_freq;             /* [S][W][C][T] chosen frequency index of TP index t, -1 where n_t is 0; required */
    int32_t *d_tuple;            /* [S][W][C] number of the chosen tuple, -1 if none; required */
    float *d_best_E;             /* [S][W][C] its energy (Wh), +inf if none; required */
    double *d_E_total;           /* [S] sum over feasible tiles; required */
    uint32_t *d_n_infeasible;    /* [S] tiles without a feasible tuple; required */
} dyn_mixed_out;

size_t dyn_mixed_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W);
/* Number of count tuples within the budget (0 on bad input): the work per tile is this times T*F evaluations. */
int64_t dyn_mixed_tuple_count(const dyn_profile *profile, const dyn_space *space);
int dyn_mixed_select(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                     const dyn_mixed_out *out, void *d_ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Selection that counts the cost of re-configuring.  [Sec. 4.2 "Accounting for the overheads": the transition
 * overheads are kept in an Overhead Table, and a controller sets the energy a new configuration saves against the
 * cost of getting there; Sec. 4.3: what a re-sharding costs depends on the source and destination parallelism
 * (table of re-sharding overheads), a frequency change costs next to nothing.]
 *
 * Per scenario s and class c the call finds the schedule over all W windows of least total cost:
 *   - a state is a sharding sigma = (n-1)*T + t (n instances of TP index t), NS = Nmax*T states (NS <= 1024);
 *   - the cost of state sigma in window w is the least energy over the candidate frequencies q of candidate
 *     (n, t, q) at the window's load (evaluation and constraints as for dyn_eval_configs, gpu_budget included),
 *     lowest q on ties, +inf if none is feasible;
 *   - moving from sigma' in window w-1 to sigma in window w costs d_R[sigma'][sigma] (Wh; the caller's overhead
 *     table, device float [NS][NS], used as given, entries >= 0 expected); the first window starts anywhere;
 *   - minimise  sum_w cost_w(sigma_w) + sum_{w>=1} d_R[sigma_{w-1}][sigma_w];  among schedules of equal cost the
 *     forward recursion keeps the lowest predecessor and the lowest final state.
 * Results: out->d_best_idx[s][w][c] = sigma_w*F + q_w and out->d_best_E = cost_w(sigma_w); if some window of
 * (s, c) has no feasible state there is no schedule: -1 / +inf in all its windows.  Totals in `out` as in
 * dyn_select (window energies only); d_path_total[s][c] (double, required) is the minimised sum including the
 * transition costs (+inf without a schedule).  Arithmetic: fp32 window costs; the running path costs are held as
 * fp32 differences to their minimum, the minimum itself in fp64.
 * Workspace: dyn_reconf_workspace_bytes() (9 bytes per (s, c, w, sigma) plus the resolved tables).
 * Errors: as dyn_eval_select, plus DYN_EINVAL for NULL d_R / d_path_total, DYN_EUNSUPPORTED for NS > 1024 or
 * F > 256.
 * ------------------------------------------------------------------------------------------- */
size_t dyn_reconf_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W);
int dyn_reconf_select(const dyn_profile *profile, const dyn_space *space, const float *d_R, const float *d_load,
                      int64_t S, int64_t W, const dyn_select_out *out, double *d_path_total, void *d_ws,
                      size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Whole path from HOST buffers: (a) -> (b) -> (c) in one call.  [Sec. 3 trace -> Sec. 3.2 loads ->
 * Sec. 4.1 / Eq. 1 evaluation -> Sec. 4.2 selection -> Sec. 6 totals]
 *
 * Copies the trace and the profile tables to the device, bins the trace into the loads of scenario 0,
 * appends S_extra further load scenarios given by the caller (e.g. resampled loads), runs the fused
 * evaluate+select and the totals, and copies the requested results back.  All device memory comes
 * from the caller's arena (256-byte aligned, at least dyn_pipeline_arena_bytes()); nothing is
 * allocated.  Copies are cudaMemcpyAsync on `stream`: with pinned host buffers the call returns before
 * the results have arrived, so synchronise the stream before reading them; the host input buffers
 * must stay valid until then.
 * ------------------------------------------------------------------------------------------- */
typedef struct {                 /* as dyn_profile, with the four tables in HOST memory */
    int32_t C, T, R, M;
    const int32_t *tp;
    const float *f_grid_mhz;
    const float *ttft, *cap, *tbt, *pow;
} dyn_profile_host;

typedef struct {
    const uint32_t *t_ms, *in_tok, *out_tok;   /* host [n_req] each */
    uint64_t n_req;
    const float *extra_load;                   /* host [S_extra][W][C] requests/s, or NULL */
    int64_t S_extra;                           /* scenarios after scenario 0 (the binned trace); S = 1 + S_extra */
    void *copy_stream;                         /* optional second cudaStream_t (NULL = none): extra_load is then copied on
                                                  it in up to 16 pieces, each evaluated on `stream` as soon as it has
                                                  arrived, and each piece's results are copied back on it while the
                                                  next piece is evaluated (the trace is copied on it too, behind
                                                  the first piece, and scenario 0 is evaluated last); `stream` waits for the last of these copies,
                                                  so synchronising `stream` is still all the caller does; the two streams
                                                  are ordered by events the library creates once per thread and device */
} dyn_host_in;

typedef struct {                 /* host result buffers; any of them may be NULL to skip that copy */
    uint32_t *counts;            /* [W][C] */
    uint64_t *dropped;           /* [1] */
    int32_t *best_idx;           /* [S][W][C] */
    float *best_E;               /* [S][W][C] */
    double *E_total;             /* [S] */
    uint32_t *n_infeasible;      /* [S] */
    double *E_window;            /* [S][W] */
    uint32_t *hist;              /* [S][J] */
    uint32_t *gpus;              /* [S][W] */
} dyn_host_out;

/* Arena size in bytes for this problem (0 on bad input).  spec->n_windows is W, C must equal
 * (n_in_edges+1)*(n_out_edges+1), S = 1 + S_extra. */
size_t dyn_pipeline_arena_bytes(const dyn_bin_spec *spec, const dyn_profile_host *profile, const dyn_space *space,
                                uint64_t n_req, int64_t S);

/* Errors: as the stage calls, plus DYN_EINVAL when profile->C differs from the class count of spec, and
 * DYN_EWORKSPACE for a missing, misaligned or short arena. */
int dyn_pipeline_host(const dyn_bin_spec *spec, const dyn_profile_host *profile, const dyn_space *space,
                      const dyn_host_in *in, const dyn_host_out *out, void *d_arena, size_t arena_bytes,
                      void *stream);

/* ---------------------------------------------------------------------------------------------
 * Instrumentation (no counterpart in the paper).  With two non-NULL cudaEvent_t handles (created by
 * the caller with timing enabled), every later stage call on the calling thread records `start`
 * right before and `stop` right after its main kernel on the call's stream: the histogram kernel of
 * dyn_bin_trace, the sweep kernel of dyn_eval_configs / dyn_eval_select, the argmin kernel of
 * dyn_select.  cudaEventElapsedTime(start, stop) after a synchronise is then that kernel's duration.
 * Pass NULL, NULL to switch it off (the default).
 * ------------------------------------------------------------------------------------------- */
void dyn_set_timing_events(void *start_event, void *stop_event);

/* ---------------------------------------------------------------------------------------------
 * Checking build (no counterpart in the paper).  The library can be built a second time with index checks
 * (libdynamo_check.so): every computed index into a global array, a shared-memory bin or a table is tested
 * against its extent before use, and every table address that the sweep forms arithmetically against the
 * range it staged; an index out of range is recorded and replaced by 0, so that the access stays in bounds and
 * the kernel runs to its end -- nothing traps, nothing waits.  This call WAITS for the device, then reports
 * and clears what the kernels of this process recorded since the last call: the number of violations and, of
 * the first one, the site (translation unit number * 65536 + source line), the offending index and the extent
 * it was tested against (both saturate at 2^32 - 1).  Any of the four pointers may be NULL.
 * Returns DYN_OK in a checking build, DYN_EUNSUPPORTED (and zeros) in the ordinary build, which has no checks.
 * ------------------------------------------------------------------------------------------- */
int dyn_debug_status(uint32_t *violations, uint32_t *site, uint32_t *index, uint32_t *extent);
/* Checking build only (DYN_EUNSUPPORTED otherwise): enqueues a one-thread kernel that indexes a three-element
 * local array with 5 through the check, which must record {site in probe.cu, index 5, extent 3} and read
 * element 0 instead (d_out, device int32 [1], receives 7).  It shows that the reporting path works; no access
 * leaves its array. */
int dyn_debug_selftest(int32_t *d_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Start-up self-check (no counterpart in the paper).  The sweep forms table addresses as subnormal
 * floating-point numbers; a library built with flush-to-zero arithmetic (-ftz=true, --use_fast_math) would
 * read entry 0 for every candidate and return plausible but wrong results.  This call runs one tiny kernel on
 * `stream`, WAITS for it (the only call here that synchronises) and returns DYN_OK when the device computes
 * such an address exactly, DYN_EUNSUPPORTED when it does not (rebuild without those flags), DYN_ECUDA on a
 * runtime error.  Call it once per process at start-up; the stage calls do not call it.
 * ------------------------------------------------------------------------------------------- */
int dyn_self_check(void *stream);

/* ---------------------------------------------------------------------------------------------
 * Measured ceilings (instrumentation; no counterpart in the paper).  Each call enqueues one short
 * kernel on `stream` and records the events of dyn_set_timing_events around it; the caller divides
 * the returned amount of work by the measured time.  d_sink: device float [1], required, never
 * written for the values the kernels use (it only keeps their arithmetic alive).  `iters` >= 1 scales
 * the run time (about 1 ms per 500 on a B200 for the first, per 100 for the second).
 *
 *   dyn_probe_fma          every thread advances eight independent fp32 multiply-add chains; *fp32_ops
 *                          (host, may be NULL) receives the fp32 operations executed, 2 per lane and
 *                          multiply-add.  ops / time is the fp32 peak of this GPU at the clock it runs at;
 *                          one warp-wide multiply-add is 64 operations, so peak / 64 is the ceiling of
 *                          instruction issue (warp instructions per second).
 *   dyn_probe_sweep_inner  the inner (TP, f) loop of dyn_eval_select's kernel on the load-threshold path,
 *                          the same device code on a synthetic table in shared memory, 8 candidates per
 *                          lane and pair, without any per-tile work; `feasible_share` in [0, 1] is the
 *                          share of candidates whose load is within the pair's limit (an infeasible
 *                          candidate skips its table lookup, so the rate depends on it); *candidates
 *                          (host, may be NULL) receives the candidates evaluated.  candidates / time is
 *                          the rate the instruction mix of that loop reaches on this GPU.
 * Errors: DYN_EINVAL (iters < 1, NULL d_sink, share outside [0, 1]), DYN_ECUDA.
 * ------------------------------------------------------------------------------------------- */
int dyn_probe_fma(int32_t iters, float *d_sink, double *fp32_ops, void *stream);
int dyn_probe_sweep_inner(int32_t iters, float feasible_share, float *d_sink, double *candidates, void *stream);

/* ---------------------------------------------------------------------------------------------
 * dyn_eval_select without a workspace argument (the paper has no counterpart; this is a packaging
 * variant of dyn_eval_select for callers that cannot obtain device memory).
 *
 * Who needs it: a controller that runs as a guest inside a serving process which has already handed
 * the whole GPU to its own memory pool (weights + KV cache), a plug-in that is allowed to launch
 * kernels but not to call the CUDA allocator, or a few-second control loop that must not risk the
 * device-wide synchronisation an allocation can cause.  Such a caller still owns its input and
 * output buffers (it got them from its host application) but has nowhere to get scratch from.
 *
 * The scratch (candidate-resolved tables and partial sums, the same content dyn_eval_select puts in
 * d_ws) lives in a fixed array of DYN_STATIC_WS_BYTES inside the library image.  Every GPU on which
 * the library is loaded holds that array from load until the process exits, used or not.
 *
 *   - Limit: the call serves a problem only if dyn_workspace_bytes(profile, space, S, W) is at most
 *     DYN_STATIC_WS_BYTES; a larger problem is refused with DYN_EUNSUPPORTED and nothing is enqueued
 *     (use dyn_eval_select with your own workspace instead).
 *   - The first call on each device is a warm-up: it looks up the array's device address (once per device,
 *     with that device current) and keeps it.  With lazy module loading that look-up is also the moment the
 *     CUDA runtime loads this library's device code onto the device, array included, which can take device
 *     memory and synchronise the device once.  Make that first call at start-up, before any stream capture
 *     begins.  A cudaDeviceReset invalidates the kept address: do not reset a device this call has been used on.
 *   - Every later call performs no allocation of any kind, frees nothing and does not synchronise.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left there.
 *     That is harmless for back-to-back calls on one stream, because every word the kernels read from
 *     the scratch is written earlier in the same call (nothing relies on zero-initialised scratch).
 *     Two calls whose GPU work overlaps (different streams, or different host threads on different
 *     streams) race on the array and give undefined results: serialise them.
 *   - Everything else (arguments, results, errors, tolerances) is exactly dyn_eval_select's.
 * ------------------------------------------------------------------------------------------- */
#define DYN_STATIC_WS_BYTES (4u << 20)   /* 4 MiB: coarse frequency grids fit with thousands of scenarios; a
                                            79-frequency, 64-knot grid (5 MB of resolved tables) does not */
int dyn_eval_select_static(const dyn_profile *profile, const dyn_space *space, const float *d_load,
                           int64_t S, int64_t W, const dyn_select_out *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DYNAMO_H_ */
