// Internal declarations shared by the translation units of libdynamo.so (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dynamo.h"
#include "check.cuh"

namespace dyn {

// ---- error plumbing -----------------------------------------------------------------------
void set_last_cuda_error(cudaError_t e);

#define DYN_CUDA_TRY(expr)                              \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) {                       \
            ::dyn::set_last_cuda_error(e__);            \
            return DYN_ECUDA;                           \
        }                                               \
    } while (0)

// ---- unsigned division by a run-time invariant (Granlund & Montgomery 1994, Fig. 4.1) -------
// q = floor(n / d) for every 32-bit n and every d >= 1:
//   l = ceil(log2 d), m' = floor(2^32 (2^l - d) / d) + 1, t1 = mulhi(m', n),
//   q = (t1 + ((n - t1) >> min(l,1))) >> max(l-1, 0)
struct FastDiv {
    uint32_t mul, sh1, sh2, d;
};

inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    uint32_t l = 0;
    while (l < 32 && (uint64_t(1) << l) < d) ++l;
    f.mul = uint32_t(((uint64_t(1) << 32) * ((uint64_t(1) << l) - d)) / d + 1);
    f.sh1 = l < 1 ? l : 1;
    f.sh2 = l > 0 ? l - 1 : 0;
    f.d = d;
    return f;
}

__device__ __forceinline__ uint32_t fastdiv(uint32_t n, const FastDiv &f) {
    uint32_t t1 = __umulhi(f.mul, n);
    return (t1 + ((n - t1) >> f.sh1)) >> f.sh2;
}

// ---- resolved candidate tables (scratch memory) ----------------------------------------------
// For class c and pair p = t*F + q (P = T*F pairs), with x = u*(M-1) the table position and
// v = x/M = sat(L/n * ic):
//   rows[c][p][m]   m = 0..M, float4 {tbt_a, -tbt_d, e_a, -e_d}: on segment m (x in [m, m+1])
//                   TBT(x) = tbt_a + (x-m)*tbt_d and the window energy of ONE instance is
//                   e(x) = e_a + (x-m)*e_d (Wh); slopes are stored negated.  Entry M-1 is the last
//                   knot with a huge TBT slope and entry M has TBT = +inf, so u > 1 shows up as an SLO
//                   violation; a pair whose TTFT misses its SLO has TBT = +inf everywhere.
//   pairc[c][p]     float2 {ic, vlim}: ic = (M-1)/(M*cap(c,t,f_q)) (0 for a never-feasible pair);
//                   vlim = largest v with TBT <= slo_tbt[c] and u <= 1 when TBT does not decrease
//                   along the row (-1 for a never-feasible pair), NaN when it does decrease somewhere.
//   slo[c]          slo_tbt[c]
//   pair2[c][p]     float4 {icm, icm, llim, cap} for the threshold path (cap: the pair's interpolated capacity): icm = (M-1)/cap, the table position per
//                   unit of per-instance load l (x = l*icm); llim = largest l with TBT <= slo_tbt[c] and
//                   u <= 1 (-1 for a never-feasible pair)
//   rows2[c][p][m]  m = 0..M, float2 {a, b}: the energy line of segment m in l, e = a + l*b (a = e_a - m*e_d,
//                   b = e_d*(M-1)/cap; flat at the last knot's energy for m >= M-1), for the threshold path
struct ResolvedLayout {
    int32_t C, T, F, P, M, Nmax, J;
    int32_t row_stride;          // entries per pair row (M + 1)
    size_t off_rows, off_pairc, off_slo, off_pair2, off_rows2, off_tp, off_partial, total;
};

ResolvedLayout resolved_layout(int32_t C, int32_t T, int32_t F, int32_t M, int32_t Nmax, int64_t S, int64_t W);

struct ResolveParams {
    int32_t C, T, R, M, F;
    const float *d_ttft, *d_cap, *d_tbt, *d_pow;
    float window_s;
    int16_t row[DYN_MAX_F];
    float weight[DYN_MAX_F];
    float slo_ttft[256], slo_tbt[256];
    int32_t tp[DYN_MAX_T];
};

// launchers (each enqueues on `st` and returns the launch error, if any)
cudaError_t launch_resolve(const ResolveParams &rp, const ResolvedLayout &lay, void *d_ws, cudaStream_t st);

struct SelectOut {
    int32_t *best_idx;
    float *best_E;
    double *E_total;
    uint32_t *n_infeasible;
    double *E_window;
    uint32_t *hist;
    uint32_t *gpus;
};

cudaError_t launch_eval_configs(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                                int32_t gpu_budget, float *d_E, cudaStream_t st);
cudaError_t launch_eval_select(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                               int32_t gpu_budget, int32_t *best_idx, float *best_E, cudaStream_t st);
cudaError_t launch_select(const float *d_E, int64_t tiles, int32_t J, int32_t *best_idx, float *best_E,
                          cudaStream_t st);
// n/tp of candidate j: either from device tables (d_nj, d_tj) or, when those are NULL, from
// j = ((n-1)*T + t)*F + q with the TP list d_tp.
cudaError_t launch_totals(const SelectOut &o, int64_t S, int64_t W, int32_t C, int32_t J, const int32_t *d_nj,
                          const int32_t *d_tj, int32_t T, int32_t F, const int32_t *d_tp, double *d_partial,
                          uint32_t *d_partial_bad, cudaStream_t st);
int64_t totals_chunks(int64_t W);
cudaError_t launch_hier(const ResolveParams &rp, const ResolvedLayout &lay, void *d_ws, size_t off_ml, const float *d_load,
                        int64_t S, int64_t W, int32_t e1, int32_t e2, int32_t space_budget, int32_t *d_nodes,
                        int32_t *d_shard, int32_t *best_idx, float *best_E, cudaStream_t st);

// pools that mix tensor parallelisms: `tuples` holds K count tuples, 8 bits per TP index
// `pairs` (n_pairs entries, 0: none): tuple index | count << 16 | TP index << 24, by TP index, every index padded to
// whole chunks of kMixedPairsChunk entries; built for lists of at most kMixedPairsMaxTuples tuples
constexpr int64_t kMixedPairsMaxTuples = 512;
constexpr int kMixedPairsChunk = 64;
cudaError_t launch_mixed(const ResolvedLayout &lay, void *d_ws, size_t off_tuples, size_t off_caph, size_t off_inva, size_t off_pairs,
                         int64_t n_pairs, int64_t K, const float *d_load, int64_t tiles, int32_t *d_counts, int32_t *d_freq,
                         int32_t *d_tuple, float *d_best_E, cudaStream_t st);

// selection with re-configuration costs (shortest path over the windows)
cudaError_t launch_reconf(const ResolvedLayout &lay, void *d_ws, size_t off_cost, size_t off_q, size_t off_from, size_t off_rt,
                          const float *d_R, const float *d_load, int64_t S, int64_t W, int32_t budget, int32_t *best_idx,
                          float *best_E, double *path_total, cudaStream_t st);

struct BinParams {
    FastDiv win;
    uint32_t n_windows;
    int32_t n_in, n_out, C;
    uint32_t in_edges[DYN_MAX_EDGES], out_edges[DYN_MAX_EDGES];
    float window_s;
};
cudaError_t launch_bin_trace(const BinParams &bp, const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok,
                             uint64_t n_req, uint32_t *counts, float *load, unsigned long long *dropped,
                             cudaStream_t st);

cudaError_t launch_bin_tokens(const BinParams &bp, const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok,
                              uint64_t n_req, unsigned long long *tok_in, unsigned long long *tok_out, float *tps,
                              cudaStream_t st);
cudaError_t launch_carbon(const double *E_window, const float *intensity, int64_t S, int64_t W, double *carbon, cudaStream_t st);

int sm_count();
// device ordinal of the calling thread's current device, clamped to [0, kMaxDevices): index of per-device caches
constexpr int kMaxDevices = 64;
int device_slot();

int eval_select_impl(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                     const dyn_select_out *out, void *d_ws, size_t ws_bytes, cudaStream_t st, bool resolve);

#ifdef __CUDACC__
// general-path evaluation of one candidate from the resolved rows (used by the small restricted searches)
// energy of the pool (n instances) for pair row `row` at per-instance load ln; ok = TBT within the SLO
// (u > 1 and never-feasible pairs read as TBT = huge or +inf through the sentinel entries of the row)
__device__ __forceinline__ float eval_pair(const float4 *__restrict__ row, float ic, float Mf, float ln, float nf,
                                           float slo, bool &ok) {
    const float x = __saturatef(ln * ic) * Mf;
    const int m = int(x);
    const float nu = x - float(m);
    const float4 e = __ldg(row + DYN_IDX(m, int(Mf) + 1));
    ok = fmaf(-nu, e.y, e.x) <= slo;
    return nf * fmaf(-nu, e.w, e.z);
}
#endif

// optional caller-owned events recorded around a stage's main kernel (thread-local; NULL = off)
struct TimingEvents { cudaEvent_t start, stop; };
TimingEvents timing_events();
inline cudaError_t record_start(cudaStream_t st) {
    const TimingEvents t = timing_events();
    return (t.start && t.stop) ? cudaEventRecord(t.start, st) : cudaSuccess;
}
inline cudaError_t record_stop(cudaStream_t st) {
    const TimingEvents t = timing_events();
    return (t.start && t.stop) ? cudaEventRecord(t.stop, st) : cudaSuccess;
}

}  // namespace dyn
