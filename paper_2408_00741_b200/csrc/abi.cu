// Host side of the C ABI declared in include/dynamo.h: argument validation and launch sequencing.
// Every step of the path runs in the kernels of this library; nothing here computes results.
#define DYN_TU_ID 1
#include "dyn_internal.cuh"

#include <cmath>
#include <algorithm>
#include <cstring>
#include <vector>

namespace dyn {

static thread_local int tls_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { tls_cuda_error = int(e); }

static thread_local TimingEvents tls_events = {nullptr, nullptr};
TimingEvents timing_events() { return tls_events; }

int sm_count() {
    // per device, cached on first use
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached = v;
        cached_dev = dev;
    }
    return cached;
}

#ifdef DYN_CHECK
namespace check {
namespace {
constexpr int kMaxReaders = 32;
Reader g_readers[kMaxReaders];
int g_n_readers = 0;
}  // namespace
void register_reader(Reader r) {
    if (g_n_readers < kMaxReaders) g_readers[g_n_readers++] = r;
}
}  // namespace check
#endif

int device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 0;
    return dev < kMaxDevices ? dev : kMaxDevices - 1;
}

namespace {

bool strictly_ascending_u32(const uint32_t *v, int n) {
    for (int i = 1; i < n; ++i)
        if (!(v[i - 1] < v[i])) return false;
    return true;
}

bool strictly_ascending_f32(const float *v, int n) {
    for (int i = 0; i < n; ++i)
        if (!std::isfinite(v[i])) return false;
    for (int i = 1; i < n; ++i)
        if (!(v[i - 1] < v[i])) return false;
    return true;
}

// shape checks shared by the evaluation entry points; fills the resolve parameters
int check_problem(const dyn_profile *p, const dyn_space *sp, int64_t S, int64_t W, ResolveParams *rp) {
    if (!p || !sp) return DYN_EINVAL;
    if (p->C < 1 || p->T < 1 || p->R < 2 || p->M < 2 || sp->F < 1 || sp->Nmax < 1) return DYN_EINVAL;
    if (S < 0 || W < 0) return DYN_EINVAL;
    if (!p->tp || !p->f_grid_mhz || !p->d_ttft || !p->d_cap || !p->d_tbt || !p->d_pow) return DYN_EINVAL;
    if (!sp->f_cand_mhz || !sp->slo_ttft_s || !sp->slo_tbt_s) return DYN_EINVAL;
    if (!(sp->window_s > 0.f) || !std::isfinite(sp->window_s)) return DYN_EINVAL;
    if (p->T > DYN_MAX_T || sp->F > DYN_MAX_F || p->C > 256 || sp->Nmax > 256 || p->M > 4096 || p->R > 32767)
        return DYN_EUNSUPPORTED;
    for (int t = 0; t < p->T; ++t) {
        if (p->tp[t] <= 0) return DYN_EINVAL;
        if (t > 0 && !(p->tp[t - 1] < p->tp[t])) return DYN_EINVAL;
    }
    if (!strictly_ascending_f32(p->f_grid_mhz, p->R) || !strictly_ascending_f32(sp->f_cand_mhz, sp->F))
        return DYN_EINVAL;
    const int64_t J = int64_t(sp->Nmax) * p->T * sp->F;
    if (J >= (int64_t(1) << 31)) return DYN_EINVAL;
    if (int64_t(p->C) * p->T * sp->F * (p->M + 1) >= (int64_t(1) << 26)) return DYN_EUNSUPPORTED;   // table entries
    if (S > 0 && W > 0 && (S > (int64_t(1) << 40) / W || S * W > (int64_t(1) << 40) / p->C)) return DYN_EINVAL;
    if (sp->f_cand_mhz[0] < p->f_grid_mhz[0] || sp->f_cand_mhz[sp->F - 1] > p->f_grid_mhz[p->R - 1])
        return DYN_EUNSUPPORTED;
    if (!rp) return DYN_OK;

    std::memset(rp, 0, sizeof(*rp));
    rp->C = p->C; rp->T = p->T; rp->R = p->R; rp->M = p->M; rp->F = sp->F;
    rp->d_ttft = p->d_ttft; rp->d_cap = p->d_cap; rp->d_tbt = p->d_tbt; rp->d_pow = p->d_pow;
    rp->window_s = sp->window_s;
    for (int q = 0; q < sp->F; ++q) {
        // largest row r <= R-2 whose frequency is <= the candidate; weight in [0, 1]
        const double f = double(sp->f_cand_mhz[q]);
        int r = 0;
        for (int i = 0; i <= p->R - 2; ++i)
            if (double(p->f_grid_mhz[i]) <= f) r = i;
        rp->row[q] = int16_t(r);
        rp->weight[q] = float((f - double(p->f_grid_mhz[r])) / (double(p->f_grid_mhz[r + 1]) - double(p->f_grid_mhz[r])));
    }
    for (int c = 0; c < p->C; ++c) {
        rp->slo_ttft[c] = sp->slo_ttft_s[c];
        rp->slo_tbt[c] = sp->slo_tbt_s[c];
    }
    for (int t = 0; t < p->T; ++t) rp->tp[t] = p->tp[t];
    return DYN_OK;
}

// required outputs may be NULL only when they would hold nothing
int check_out(const dyn_select_out *o, int64_t S, int64_t tiles) {
    if (!o) return DYN_EINVAL;
    if (tiles > 0 && (!o->d_best_idx || !o->d_best_E)) return DYN_EINVAL;
    if (S > 0 && (!o->d_E_total || !o->d_n_infeasible)) return DYN_EINVAL;
    return DYN_OK;
}

SelectOut to_out(const dyn_select_out *o) {
    SelectOut s;
    s.best_idx = o->d_best_idx; s.best_E = o->d_best_E; s.E_total = o->d_E_total;
    s.n_infeasible = o->d_n_infeasible; s.E_window = o->d_E_window; s.hist = o->d_hist; s.gpus = o->d_gpus;
    return s;
}

int check_ws(const void *d_ws, size_t ws_bytes, size_t need) {
    if (need == 0) return DYN_OK;
    if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255u) != 0 || ws_bytes < need) return DYN_EWORKSPACE;
    return DYN_OK;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// validation of a binning request shared by dyn_bin_trace and dyn_bin_tokens; fills the kernel parameters
int make_bin_params(const dyn_bin_spec *spec, const uint32_t *d_t_ms, const uint32_t *d_in_tok, const uint32_t *d_out_tok,
                    uint64_t n_req, BinParams *out) {
    if (!spec) return DYN_EINVAL;
    if (n_req > 0 && (!d_t_ms || !d_in_tok || !d_out_tok)) return DYN_EINVAL;
    if (spec->window_ms == 0 || spec->n_windows == 0) return DYN_EINVAL;
    if (spec->n_in_edges < 0 || spec->n_out_edges < 0 || spec->n_in_edges > DYN_MAX_EDGES ||
        spec->n_out_edges > DYN_MAX_EDGES)
        return DYN_EINVAL;
    if ((spec->n_in_edges > 0 && !spec->in_edges) || (spec->n_out_edges > 0 && !spec->out_edges)) return DYN_EINVAL;
    if (!strictly_ascending_u32(spec->in_edges, spec->n_in_edges) ||
        !strictly_ascending_u32(spec->out_edges, spec->n_out_edges))
        return DYN_EINVAL;
    BinParams bp;
    std::memset(&bp, 0, sizeof(bp));
    bp.win = make_fastdiv(spec->window_ms);
    bp.n_windows = spec->n_windows;
    bp.n_in = spec->n_in_edges;
    bp.n_out = spec->n_out_edges;
    bp.C = (bp.n_in + 1) * (bp.n_out + 1);
    if (uint64_t(spec->n_windows) * uint64_t(bp.C) >= (uint64_t(1) << 31)) return DYN_EINVAL;
    for (int e = 0; e < bp.n_in; ++e) bp.in_edges[e] = spec->in_edges[e];
    for (int e = 0; e < bp.n_out; ++e) bp.out_edges[e] = spec->out_edges[e];
    bp.window_s = float(spec->window_ms) / 1000.0f;
    *out = bp;
    return DYN_OK;
}

// count tuples within the GPU budget in odometer order (n_0 fastest): {counts, 8 bits per TP index; number};
// with out == nullptr only counts.  Returns -1 when there are more than `limit` tuples.
int64_t enumerate_tuples(const dyn_profile *p, const dyn_space *sp, int64_t limit, uint2 *out) {
    const int T = p->T, Nmax = sp->Nmax;
    int n[4] = {0, 0, 0, 0};
    int64_t K = 0;
    for (;;) {
        int t = 0;
        while (t < T && n[t] == Nmax) n[t++] = 0;
        if (t == T) break;
        ++n[t];                                              // the digits below t are zero now
        int64_t gpus = 0;
        for (int k = 0; k < T; ++k) gpus += int64_t(n[k]) * p->tp[k];
        if (gpus > sp->gpu_budget) {
            n[t] = Nmax;                                     // larger values of this digit only add GPUs: carry next
            continue;
        }
        if (K >= limit) return -1;
        if (out) out[K] = make_uint2(uint32_t(n[0]) | (uint32_t(n[1]) << 8) | (uint32_t(n[2]) << 16) | (uint32_t(n[3]) << 24),
                                     uint32_t(K));
        ++K;
    }
    return K;
}

constexpr int64_t kMaxTuples = int64_t(1) << 20;

// entries the list of (tuple, TP index) pairs can take: one per tuple and index, plus at most one padded-out chunk per
// index and at the end
size_t mixed_pairs_capacity(int64_t K, int T) {
    return K <= kMixedPairsMaxTuples ? size_t(K) * size_t(T) + size_t(T + 1) * size_t(kMixedPairsChunk) : 0;
}

int check_mixed(const dyn_profile *p, const dyn_space *sp, int64_t S, int64_t W, ResolveParams *rp) {
    const int rc = check_problem(p, sp, S, W, rp);
    if (rc != DYN_OK) return rc;
    if (sp->gpu_budget <= 0) return DYN_EINVAL;
    if (p->T > 4 || sp->Nmax > 255) return DYN_EUNSUPPORTED;
    return DYN_OK;
}

}  // namespace

// dyn_eval_select; with resolve == false the tables in d_ws are taken as resolved by an earlier call for the same
// profile, space and W (the host pipeline evaluates its pieces that way)
int eval_select_impl(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                     const dyn_select_out *out, void *d_ws, size_t ws_bytes, cudaStream_t st, bool resolve) {
    ResolveParams rp;
    int rc = check_problem(profile, space, S, W, &rp);
    if (rc != DYN_OK) return rc;
    const int64_t tiles = S * W * profile->C;
    rc = check_out(out, S, tiles);
    if (rc != DYN_OK) return rc;
    if (tiles > 0 && !d_load) return DYN_EINVAL;
    const ResolvedLayout lay = resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W);
    rc = check_ws(d_ws, ws_bytes, lay.total);
    if (rc != DYN_OK) return rc;
    char *ws = static_cast<char *>(d_ws);
    if (resolve) DYN_CUDA_TRY(launch_resolve(rp, lay, d_ws, st));
    DYN_CUDA_TRY(record_start(st));
    DYN_CUDA_TRY(launch_eval_select(lay, d_ws, d_load, tiles, space->gpu_budget, out->d_best_idx, out->d_best_E, st));
    DYN_CUDA_TRY(record_stop(st));
    const int64_t chunks = totals_chunks(W);
    double *partial = reinterpret_cast<double *>(ws + lay.off_partial);
    uint32_t *partial_bad = reinterpret_cast<uint32_t *>(ws + lay.off_partial + size_t(S) * size_t(chunks) * sizeof(double));
    DYN_CUDA_TRY(launch_totals(to_out(out), S, W, profile->C, lay.J, nullptr, nullptr, profile->T, space->F,
                               reinterpret_cast<const int32_t *>(ws + lay.off_tp), partial, partial_bad, st));
    return DYN_OK;
}

}  // namespace dyn

using namespace dyn;

extern "C" {

const char *dyn_strerror(int status) {
    switch (status) {
        case DYN_OK: return "success";
        case DYN_EINVAL: return "invalid argument";
        case DYN_ECUDA: return "CUDA runtime error (see dyn_last_cuda_error)";
        case DYN_EUNSUPPORTED: return "request outside the built limits";
        case DYN_EWORKSPACE: return "workspace missing, misaligned or too small";
        default: return "unknown status";
    }
}

int dyn_last_cuda_error(void) { return tls_cuda_error; }

int dyn_debug_status(uint32_t *violations, uint32_t *site, uint32_t *index, uint32_t *extent) {
#ifdef DYN_CHECK
    DYN_CUDA_TRY(cudaDeviceSynchronize());
    uint32_t total = 0, s0 = 0, i0 = 0, n0 = 0;
    for (int k = 0; k < check::g_n_readers; ++k) {
        check::Record r = {0u, 0u, 0u, 0u};
        DYN_CUDA_TRY(check::g_readers[k](&r));
        if (r.count && !total) { s0 = r.site; i0 = r.index; n0 = r.extent; }
        total += r.count;
    }
    if (violations) *violations = total;
    if (site) *site = s0;
    if (index) *index = i0;
    if (extent) *extent = n0;
    return DYN_OK;
#else
    if (violations) *violations = 0;
    if (site) *site = 0;
    if (index) *index = 0;
    if (extent) *extent = 0;
    return DYN_EUNSUPPORTED;
#endif
}

void dyn_set_timing_events(void *start_event, void *stop_event) {
    tls_events.start = static_cast<cudaEvent_t>(start_event);
    tls_events.stop = static_cast<cudaEvent_t>(stop_event);
}

int dyn_bin_trace(const dyn_bin_spec *spec, const uint32_t *d_t_ms, const uint32_t *d_in_tok,
                  const uint32_t *d_out_tok, uint64_t n_req, uint32_t *d_counts, float *d_load,
                  uint64_t *d_dropped, void *stream) {
    if (!d_counts || !d_dropped) return DYN_EINVAL;
    BinParams bp;
    const int rc = make_bin_params(spec, d_t_ms, d_in_tok, d_out_tok, n_req, &bp);
    if (rc != DYN_OK) return rc;
    DYN_CUDA_TRY(launch_bin_trace(bp, d_t_ms, d_in_tok, d_out_tok, n_req, d_counts, d_load,
                                  reinterpret_cast<unsigned long long *>(d_dropped),
                                  static_cast<cudaStream_t>(stream)));
    return DYN_OK;
}

size_t dyn_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W) {
    if (!profile || !space) return 0;
    if (profile->C < 1 || profile->T < 1 || profile->M < 2 || space->F < 1 || space->Nmax < 1 || S < 0 || W < 0)
        return 0;
    return resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W).total;
}

int dyn_eval_configs(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                     float *d_E, void *d_ws, size_t ws_bytes, void *stream) {
    ResolveParams rp;
    int rc = check_problem(profile, space, S, W, &rp);
    if (rc != DYN_OK) return rc;
    const int64_t tiles = S * W * profile->C;
    if (tiles > 0 && (!d_load || !d_E)) return DYN_EINVAL;
    const ResolvedLayout lay = resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W);
    rc = check_ws(d_ws, ws_bytes, lay.total);
    if (rc != DYN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DYN_CUDA_TRY(launch_resolve(rp, lay, d_ws, st));
    DYN_CUDA_TRY(record_start(st));
    DYN_CUDA_TRY(launch_eval_configs(lay, d_ws, d_load, tiles, space->gpu_budget, d_E, st));
    DYN_CUDA_TRY(record_stop(st));
    return DYN_OK;
}

size_t dyn_select_workspace_bytes(int64_t S, int64_t W, int64_t J) {
    if (S < 0 || W < 0 || J < 0) return 0;
    const size_t partial = align256(size_t(S) * size_t(totals_chunks(W)) * (sizeof(double) + sizeof(uint32_t)));
    return partial + 2 * align256(size_t(J) * sizeof(int32_t));
}

int dyn_select(const float *d_E, int64_t S, int64_t W, int32_t C, int32_t J, const int32_t *n_of_j,
               const int32_t *tp_of_j, const dyn_select_out *out, void *d_ws, size_t ws_bytes, void *stream) {
    if (S < 0 || W < 0 || C < 1 || J < 1 || !out) return DYN_EINVAL;
    if (out->d_gpus && (!n_of_j || !tp_of_j)) return DYN_EINVAL;
    if (S > 0 && W > 0 && (S > (int64_t(1) << 40) / W || S * W > (int64_t(1) << 40) / C)) return DYN_EINVAL;
    const int64_t tiles = S * W * C;
    int rc = check_out(out, S, tiles);
    if (rc != DYN_OK) return rc;
    if (tiles > 0 && !d_E) return DYN_EINVAL;
    rc = check_ws(d_ws, ws_bytes, dyn_select_workspace_bytes(S, W, J));
    if (rc != DYN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(d_ws);
    const int64_t chunks = totals_chunks(W);
    double *partial = reinterpret_cast<double *>(ws);
    uint32_t *partial_bad = reinterpret_cast<uint32_t *>(ws + size_t(S) * size_t(chunks) * sizeof(double));
    const size_t off_nj = align256(size_t(S) * size_t(chunks) * (sizeof(double) + sizeof(uint32_t)));
    int32_t *d_nj = nullptr, *d_tj = nullptr;
    if (out->d_gpus) {
        d_nj = reinterpret_cast<int32_t *>(ws + off_nj);
        d_tj = reinterpret_cast<int32_t *>(ws + off_nj + align256(size_t(J) * sizeof(int32_t)));
        // pageable host arrays are staged before cudaMemcpyAsync returns (the call then waits for earlier work
        // on the stream); pinned arrays are read when the stream gets here and must stay valid until then
        DYN_CUDA_TRY(cudaMemcpyAsync(d_nj, n_of_j, size_t(J) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        DYN_CUDA_TRY(cudaMemcpyAsync(d_tj, tp_of_j, size_t(J) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    }
    DYN_CUDA_TRY(record_start(st));
    DYN_CUDA_TRY(launch_select(d_E, tiles, J, out->d_best_idx, out->d_best_E, st));
    DYN_CUDA_TRY(record_stop(st));
    DYN_CUDA_TRY(launch_totals(to_out(out), S, W, C, J, d_nj, d_tj, 1, 1, nullptr, partial, partial_bad, st));
    return DYN_OK;
}

int dyn_eval_select(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                    const dyn_select_out *out, void *d_ws, size_t ws_bytes, void *stream) {
    return eval_select_impl(profile, space, d_load, S, W, out, d_ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

size_t dyn_hier_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W) {
    const size_t base = dyn_workspace_bytes(profile, space, S, W);
    return base ? base + align256(size_t(profile->C) * sizeof(double)) : 0;
}

int dyn_hier_select(const dyn_profile *profile, const dyn_space *space, const dyn_hier_spec *hier,
                    const float *d_load, int64_t S, int64_t W, int32_t *d_nodes, int32_t *d_shard,
                    const dyn_select_out *out, void *d_ws, size_t ws_bytes, void *stream) {
    ResolveParams rp;
    int rc = check_problem(profile, space, S, W, &rp);
    if (rc != DYN_OK) return rc;
    if (!hier || hier->scale_epoch_windows < 1 || hier->shard_epoch_windows < 1 ||
        hier->scale_epoch_windows % hier->shard_epoch_windows != 0)
        return DYN_EINVAL;
    if (W * profile->C >= (int64_t(1) << 31)) return DYN_EUNSUPPORTED;      // 32-bit indices inside a scenario
    const int64_t tiles = S * W * profile->C;
    rc = check_out(out, S, tiles);
    if (rc != DYN_OK) return rc;
    if (tiles > 0 && (!d_load || !d_nodes || !d_shard)) return DYN_EINVAL;
    const ResolvedLayout lay = resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W);
    rc = check_ws(d_ws, ws_bytes, lay.total + align256(size_t(profile->C) * sizeof(double)));
    if (rc != DYN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(d_ws);
    DYN_CUDA_TRY(launch_resolve(rp, lay, d_ws, st));
    DYN_CUDA_TRY(launch_hier(rp, lay, d_ws, lay.total, d_load, S, W, hier->scale_epoch_windows,
                             hier->shard_epoch_windows, space->gpu_budget, d_nodes, d_shard, out->d_best_idx,
                             out->d_best_E, st));
    const int64_t chunks = totals_chunks(W);
    double *partial = reinterpret_cast<double *>(ws + lay.off_partial);
    uint32_t *partial_bad = reinterpret_cast<uint32_t *>(ws + lay.off_partial + size_t(S) * size_t(chunks) * sizeof(double));
    DYN_CUDA_TRY(launch_totals(to_out(out), S, W, profile->C, lay.J, nullptr, nullptr, profile->T, space->F,
                               reinterpret_cast<const int32_t *>(ws + lay.off_tp), partial, partial_bad, st));
    return DYN_OK;
}

int64_t dyn_mixed_tuple_count(const dyn_profile *profile, const dyn_space *space) {
    if (check_mixed(profile, space, 0, 0, nullptr) != DYN_OK) return 0;
    const int64_t K = enumerate_tuples(profile, space, kMaxTuples, nullptr);
    return K < 0 ? 0 : K;
}

size_t dyn_mixed_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W) {
    const size_t base = dyn_workspace_bytes(profile, space, S, W);
    const int64_t K = dyn_mixed_tuple_count(profile, space);
    if (!base || K <= 0) return 0;
    return base + align256(size_t(K) * sizeof(uint2)) + align256(size_t(profile->C) * profile->T * sizeof(float)) +
           align256(size_t(profile->C) * size_t(K) * sizeof(float)) + align256(mixed_pairs_capacity(K, profile->T) * sizeof(uint32_t));
}

int dyn_mixed_select(const dyn_profile *profile, const dyn_space *space, const float *d_load, int64_t S, int64_t W,
                     const dyn_mixed_out *out, void *d_ws, size_t ws_bytes, void *stream) {
    ResolveParams rp;
    int rc = check_mixed(profile, space, S, W, &rp);
    if (rc != DYN_OK) return rc;
    const int64_t tiles = S * W * profile->C;
    if (!out) return DYN_EINVAL;
    if (tiles > 0 && (!out->d_counts || !out->d_freq || !out->d_tuple || !out->d_best_E || !d_load)) return DYN_EINVAL;
    if (S > 0 && (!out->d_E_total || !out->d_n_infeasible)) return DYN_EINVAL;
    const int64_t K = enumerate_tuples(profile, space, kMaxTuples, nullptr);
    if (K < 0) return DYN_EUNSUPPORTED;
    if (K == 0) return DYN_EINVAL;                           // the budget admits no instance at all
    static thread_local std::vector<uint2> tuples;           // host list, rebuilt per call (cheap next to the search)
    tuples.resize(size_t(K));
    enumerate_tuples(profile, space, K, tuples.data());
    // group the tuples by the set of TP indices in use (stable: number order inside a group), so that the
    // tuples a warp evaluates side by side take the same branches
    auto mask_of = [](const uint2 &u) {
        return ((u.x & 0xffu) ? 1u : 0u) | ((u.x & 0xff00u) ? 2u : 0u) | ((u.x & 0xff0000u) ? 4u : 0u) | ((u.x >> 24) ? 8u : 0u);
    };
    std::stable_sort(tuples.begin(), tuples.end(), [&](const uint2 &x, const uint2 &y) { return mask_of(x) < mask_of(y); });
    const ResolvedLayout lay = resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W);
    const size_t off_tuples = lay.total, off_caph = off_tuples + align256(size_t(K) * sizeof(uint2));
    const size_t off_inva = off_caph + align256(size_t(profile->C) * profile->T * sizeof(float));
    const size_t off_pairs = off_inva + align256(size_t(profile->C) * size_t(K) * sizeof(float));
    const size_t need = off_pairs + align256(mixed_pairs_capacity(K, profile->T) * sizeof(uint32_t));
    rc = check_ws(d_ws, ws_bytes, need);
    if (rc != DYN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(d_ws);
    // pageable host memory: the copy is staged before the call returns
    DYN_CUDA_TRY(cudaMemcpyAsync(ws + off_tuples, tuples.data(), size_t(K) * sizeof(uint2), cudaMemcpyHostToDevice, st));
    // short lists: the (tuple, TP index) pairs that hold instances, by TP index and padded per index to whole
    // chunks of a warp, so that the search spends no evaluation on a parallelism a tuple does not use
    int64_t n_pairs = 0;
    if (K <= kMixedPairsMaxTuples) {
        static thread_local std::vector<uint32_t> pairs;
        pairs.clear();
        // A lane takes two neighbouring entries, which must share their TP index (every index is padded to an even
        // count); a chunk of kMixedPairsChunk entries may run over from one index into the next as long as no tuple
        // appears in it twice (the sums of a chunk are added without looking at each other): where one would, the
        // chunk is padded out.  Padding entries hold no instance and are never evaluated.
        static thread_local std::vector<uint8_t> in_chunk;
        in_chunk.assign(size_t(K), 0);
        size_t chunk_begin = 0;
        auto new_chunk_if_full = [&]() {
            if (pairs.size() - chunk_begin == size_t(kMixedPairsChunk)) {
                for (size_t e = chunk_begin; e < pairs.size(); ++e) in_chunk[pairs[e] & 0xffffu] = 0;
                chunk_begin = pairs.size();
            }
        };
        for (int t = 0; t < profile->T; ++t) {
            for (int64_t k = 0; k < K; ++k) {
                const uint32_t n = (tuples[size_t(k)].x >> (8 * t)) & 255u;
                if (!n) continue;
                if (in_chunk[size_t(k)]) {                   // the tuple is in this chunk already (at a lower index): pad it out
                    while (pairs.size() - chunk_begin < size_t(kMixedPairsChunk)) pairs.push_back(uint32_t(t) << 24);
                    new_chunk_if_full();
                }
                pairs.push_back(uint32_t(k) | (n << 16) | (uint32_t(t) << 24));
                in_chunk[size_t(k)] = 1;
                new_chunk_if_full();
            }
            if (pairs.size() & 1u) {                         // an even count per index; the padding entry names tuple 0 with no instance
                pairs.push_back(uint32_t(t) << 24);
                new_chunk_if_full();
            }
        }
        while (pairs.size() % size_t(kMixedPairsChunk)) pairs.push_back(uint32_t(profile->T - 1) << 24);
        n_pairs = pairs.size() <= mixed_pairs_capacity(K, profile->T) ? int64_t(pairs.size()) : 0;     // (0: the kernel for long lists)
        if (n_pairs > 0)
            DYN_CUDA_TRY(cudaMemcpyAsync(ws + off_pairs, pairs.data(), pairs.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, st));
    }
    DYN_CUDA_TRY(launch_resolve(rp, lay, d_ws, st));
    DYN_CUDA_TRY(launch_mixed(lay, d_ws, off_tuples, off_caph, off_inva, off_pairs, n_pairs, K, d_load, tiles, out->d_counts,
                              out->d_freq, out->d_tuple, out->d_best_E, st));
    SelectOut so{};
    so.best_idx = out->d_tuple; so.best_E = out->d_best_E; so.E_total = out->d_E_total; so.n_infeasible = out->d_n_infeasible;
    const int64_t chunks = totals_chunks(W);
    double *partial = reinterpret_cast<double *>(ws + lay.off_partial);
    uint32_t *partial_bad = reinterpret_cast<uint32_t *>(ws + lay.off_partial + size_t(S) * size_t(chunks) * sizeof(double));
    DYN_CUDA_TRY(launch_totals(so, S, W, profile->C, 1, nullptr, nullptr, 1, 1, nullptr, partial, partial_bad, st));
    return DYN_OK;
}

size_t dyn_reconf_workspace_bytes(const dyn_profile *profile, const dyn_space *space, int64_t S, int64_t W) {
    const size_t base = dyn_workspace_bytes(profile, space, S, W);
    if (!base) return 0;
    const size_t n = size_t(S) * size_t(profile->C) * size_t(W) * size_t(space->Nmax) * size_t(profile->T);
    const size_t ns = size_t(space->Nmax) * size_t(profile->T);
    return base + align256(n * sizeof(float)) + align256(n) + align256(n * sizeof(float)) + align256(ns * ns * sizeof(float));
}

int dyn_reconf_select(const dyn_profile *profile, const dyn_space *space, const float *d_R, const float *d_load,
                      int64_t S, int64_t W, const dyn_select_out *out, double *d_path_total, void *d_ws,
                      size_t ws_bytes, void *stream) {
    ResolveParams rp;
    int rc = check_problem(profile, space, S, W, &rp);
    if (rc != DYN_OK) return rc;
    const int64_t NS = int64_t(space->Nmax) * profile->T;
    if (NS > 1024 || space->F > 256) return DYN_EUNSUPPORTED;
    const int64_t tiles = S * W * profile->C;
    rc = check_out(out, S, tiles);
    if (rc != DYN_OK) return rc;
    if (!d_R || (S > 0 && !d_path_total) || (tiles > 0 && !d_load)) return DYN_EINVAL;
    const ResolvedLayout lay = resolved_layout(profile->C, profile->T, space->F, profile->M, space->Nmax, S, W);
    const size_t n = size_t(S) * size_t(profile->C) * size_t(W) * size_t(NS);
    const size_t off_cost = lay.total, off_q = off_cost + align256(n * sizeof(float)), off_from = off_q + align256(n);
    const size_t off_rt = off_from + align256(n * sizeof(float));
    rc = check_ws(d_ws, ws_bytes, off_rt + align256(size_t(NS) * size_t(NS) * sizeof(float)));
    if (rc != DYN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(d_ws);
    DYN_CUDA_TRY(launch_resolve(rp, lay, d_ws, st));
    DYN_CUDA_TRY(launch_reconf(lay, d_ws, off_cost, off_q, off_from, off_rt, d_R, d_load, S, W, space->gpu_budget, out->d_best_idx,
                               out->d_best_E, d_path_total, st));
    const int64_t chunks = totals_chunks(W);
    double *partial = reinterpret_cast<double *>(ws + lay.off_partial);
    uint32_t *partial_bad = reinterpret_cast<uint32_t *>(ws + lay.off_partial + size_t(S) * size_t(chunks) * sizeof(double));
    DYN_CUDA_TRY(launch_totals(to_out(out), S, W, profile->C, lay.J, nullptr, nullptr, profile->T, space->F,
                               reinterpret_cast<const int32_t *>(ws + lay.off_tp), partial, partial_bad, st));
    return DYN_OK;
}

int dyn_bin_tokens(const dyn_bin_spec *spec, const uint32_t *d_t_ms, const uint32_t *d_in_tok, const uint32_t *d_out_tok,
                   uint64_t n_req, uint64_t *d_tok_in, uint64_t *d_tok_out, float *d_load_tps, void *stream) {
    if (!d_tok_in || !d_tok_out) return DYN_EINVAL;
    BinParams bp;
    const int rc = make_bin_params(spec, d_t_ms, d_in_tok, d_out_tok, n_req, &bp);
    if (rc != DYN_OK) return rc;
    DYN_CUDA_TRY(launch_bin_tokens(bp, d_t_ms, d_in_tok, d_out_tok, n_req, reinterpret_cast<unsigned long long *>(d_tok_in),
                                   reinterpret_cast<unsigned long long *>(d_tok_out), d_load_tps,
                                   static_cast<cudaStream_t>(stream)));
    return DYN_OK;
}

int dyn_carbon(const double *d_E_window, const float *d_intensity, int64_t S, int64_t W, double *d_carbon, void *stream) {
    if (S < 0 || W < 0) return DYN_EINVAL;
    if (S > 0 && (!d_carbon || (W > 0 && (!d_E_window || !d_intensity)))) return DYN_EINVAL;
    DYN_CUDA_TRY(launch_carbon(d_E_window, d_intensity, S, W, d_carbon, static_cast<cudaStream_t>(stream)));
    return DYN_OK;
}

}  // extern "C"
