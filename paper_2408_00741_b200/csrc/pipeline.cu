// Whole path from host buffers: copy in, bin, evaluate + select, totals, copy out.  Device memory is
// carved from the caller's arena; nothing is allocated here.
#define DYN_TU_ID 6
#include "dyn_internal.cuh"

namespace {

size_t a256(size_t x) { return (x + 255) / 256 * 256; }

struct Arena {
    size_t t, a, b, counts, dropped, load, ttft, cap, tbt, pw, idx, be, etot, ninf, ewin, hist, gpus, ws, total;
    size_t ws_bytes;
};

bool plan(const dyn_bin_spec *spec, const dyn_profile_host *p, const dyn_space *sp, uint64_t n_req, int64_t S, Arena *ar) {
    if (!spec || !p || !sp || S < 1) return false;
    if (spec->n_in_edges < 0 || spec->n_out_edges < 0 || spec->n_windows == 0) return false;
    if (p->C < 1 || p->T < 1 || p->R < 2 || p->M < 2 || sp->F < 1 || sp->Nmax < 1) return false;
    const size_t C = size_t(p->C), W = spec->n_windows;
    const size_t tiles = size_t(S) * W * C;
    const size_t J = size_t(sp->Nmax) * size_t(p->T) * size_t(sp->F);
    const size_t ctr = C * size_t(p->T) * size_t(p->R);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = a256(off + bytes); return o; };
    ar->t = take(n_req * 4); ar->a = take(n_req * 4); ar->b = take(n_req * 4);
    ar->counts = take(W * C * 4); ar->dropped = take(8);
    ar->load = take(tiles * 4);
    ar->ttft = take(ctr * 4); ar->cap = take(ctr * 4);
    ar->tbt = take(ctr * size_t(p->M) * 4); ar->pw = take(ctr * size_t(p->M) * 4);
    ar->idx = take(tiles * 4); ar->be = take(tiles * 4);
    ar->etot = take(size_t(S) * 8); ar->ninf = take(size_t(S) * 4);
    ar->ewin = take(size_t(S) * W * 8); ar->hist = take(size_t(S) * J * 4); ar->gpus = take(size_t(S) * W * 4);
    dyn_profile dp{p->C, p->T, p->R, p->M, p->tp, p->f_grid_mhz, nullptr, nullptr, nullptr, nullptr};
    ar->ws_bytes = dyn_workspace_bytes(&dp, sp, S, int64_t(W));
    if (ar->ws_bytes == 0) return false;
    ar->ws = take(ar->ws_bytes);
    ar->total = off;
    return true;
}

constexpr int kPieces = 16;      // pieces the scenario loads are copied in when a copy stream is given
constexpr int kEvents = 2 * kPieces + 3;         // [k]: loads of piece k are in; [kPieces]: arena free / results out;
                                                 // [kPieces + 1 + k]: piece k is evaluated; [2 kPieces + 2]: trace is in
constexpr int kTraceEvent = 2 * kPieces + 2;

// events that order the copy stream against the caller's stream: created on first use per thread and device,
// kept for the life of the process (they hold no device memory)
cudaEvent_t *overlap_events() {
    constexpr int kMaxDev = 64;
    static thread_local cudaEvent_t ev[kMaxDev][kEvents];
    static thread_local bool made[kMaxDev] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
    if (!made[dev]) {
        for (int i = 0; i < kEvents; ++i) {
            const cudaError_t e = cudaEventCreateWithFlags(&ev[dev][i], cudaEventDisableTiming);
            if (e != cudaSuccess) {                      // give back what was created and report why
                for (int k = 0; k < i; ++k) cudaEventDestroy(ev[dev][k]);
                dyn::set_last_cuda_error(e);
                return nullptr;
            }
        }
        made[dev] = true;
    }
    return ev[dev];
}

}  // namespace

extern "C" {

size_t dyn_pipeline_arena_bytes(const dyn_bin_spec *spec, const dyn_profile_host *profile, const dyn_space *space,
                                uint64_t n_req, int64_t S) {
    Arena ar;
    return plan(spec, profile, space, n_req, S, &ar) ? ar.total : 0;
}

int dyn_pipeline_host(const dyn_bin_spec *spec, const dyn_profile_host *p, const dyn_space *sp, const dyn_host_in *in,
                      const dyn_host_out *out, void *d_arena, size_t arena_bytes, void *stream) {
    if (!spec || !p || !sp || !in || !out) return DYN_EINVAL;
    if (in->S_extra < 0 || (in->S_extra > 0 && !in->extra_load)) return DYN_EINVAL;
    if (in->n_req > 0 && (!in->t_ms || !in->in_tok || !in->out_tok)) return DYN_EINVAL;
    if (!p->ttft || !p->cap || !p->tbt || !p->pow) return DYN_EINVAL;
    if (spec->n_in_edges < 0 || spec->n_out_edges < 0 ||
        int64_t(spec->n_in_edges + 1) * int64_t(spec->n_out_edges + 1) != int64_t(p->C))
        return DYN_EINVAL;
    const int64_t S = 1 + in->S_extra;
    Arena ar;
    if (!plan(spec, p, sp, in->n_req, S, &ar)) return DYN_EINVAL;
    if (!d_arena || (reinterpret_cast<uintptr_t>(d_arena) & 255u) != 0 || arena_bytes < ar.total) return DYN_EWORKSPACE;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *base = static_cast<char *>(d_arena);
    auto dptr = [&](size_t off) { return static_cast<void *>(base + off); };
    const size_t C = size_t(p->C), W = spec->n_windows;
    const size_t wc = W * C, tiles = size_t(S) * wc;
    const size_t J = size_t(sp->Nmax) * size_t(p->T) * size_t(sp->F);
    const size_t ctr = C * size_t(p->T) * size_t(p->R);
    const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;

    // the caller's scenario loads: on `stream`, or in pieces on the copy stream so that a piece is evaluated while
    // the next ones are still on their way
    cudaStream_t cs = static_cast<cudaStream_t>(in->copy_stream);
    const int pieces = (cs && cs != st && in->S_extra > 0) ? int(in->S_extra < kPieces ? in->S_extra : kPieces) : 0;
    // the trace travels on `stream`, or, with a copy stream, behind the first piece of loads: scenario 0 (the binned
    // trace) is then evaluated last, and the first piece does not wait for the trace
    auto copy_trace = [&](cudaStream_t on) -> int {
        if (in->n_req > 0) {
            DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.t), in->t_ms, in->n_req * 4, H2D, on));
            DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.a), in->in_tok, in->n_req * 4, H2D, on));
            DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.b), in->out_tok, in->n_req * 4, H2D, on));
        }
        return DYN_OK;
    };
    if (pieces == 0) {
        const int rt = copy_trace(st);
        if (rt != DYN_OK) return rt;
    }
    DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.ttft), p->ttft, ctr * 4, H2D, st));
    DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.cap), p->cap, ctr * 4, H2D, st));
    DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.tbt), p->tbt, ctr * size_t(p->M) * 4, H2D, st));
    DYN_CUDA_TRY(cudaMemcpyAsync(dptr(ar.pw), p->pow, ctr * size_t(p->M) * 4, H2D, st));
    cudaEvent_t *ev = nullptr;
    if (pieces > 0) {
        ev = overlap_events();
        if (!ev) return DYN_ECUDA;
        // the arena may still be in use by work enqueued earlier on `stream`
        DYN_CUDA_TRY(cudaEventRecord(ev[kPieces], st));
        DYN_CUDA_TRY(cudaStreamWaitEvent(cs, ev[kPieces], 0));
        for (int k = 0; k < pieces; ++k) {
            const size_t e0 = size_t(in->S_extra) * k / pieces, e1 = size_t(in->S_extra) * (k + 1) / pieces;
            DYN_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(dptr(ar.load)) + (1 + e0) * wc * 4, in->extra_load + e0 * wc,
                                         (e1 - e0) * wc * 4, H2D, cs));
            DYN_CUDA_TRY(cudaEventRecord(ev[k], cs));
            if (k == 0) {
                const int rt = copy_trace(cs);
                if (rt != DYN_OK) return rt;
                DYN_CUDA_TRY(cudaEventRecord(ev[kTraceEvent], cs));
            }
        }
    } else if (in->S_extra > 0) {
        DYN_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(dptr(ar.load)) + wc * 4, in->extra_load,
                                     size_t(in->S_extra) * wc * 4, H2D, st));
    }

    // (a): scenario 0 of the load tensor is the binned trace
    auto bin = [&]() {
        return dyn_bin_trace(spec, static_cast<const uint32_t *>(dptr(ar.t)), static_cast<const uint32_t *>(dptr(ar.a)),
                             static_cast<const uint32_t *>(dptr(ar.b)), in->n_req, static_cast<uint32_t *>(dptr(ar.counts)),
                             static_cast<float *>(dptr(ar.load)), static_cast<uint64_t *>(dptr(ar.dropped)), stream);
    };
    int rc = DYN_OK;

    // (b)+(c)
    dyn_profile dp{p->C, p->T, p->R, p->M, p->tp, p->f_grid_mhz, static_cast<const float *>(dptr(ar.ttft)),
                   static_cast<const float *>(dptr(ar.cap)), static_cast<const float *>(dptr(ar.tbt)),
                   static_cast<const float *>(dptr(ar.pw))};
    dyn_select_out so{};
    so.d_best_idx = static_cast<int32_t *>(dptr(ar.idx));
    so.d_best_E = static_cast<float *>(dptr(ar.be));
    so.d_E_total = static_cast<double *>(dptr(ar.etot));
    so.d_n_infeasible = static_cast<uint32_t *>(dptr(ar.ninf));
    so.d_E_window = out->E_window ? static_cast<double *>(dptr(ar.ewin)) : nullptr;
    so.d_hist = out->hist ? static_cast<uint32_t *>(dptr(ar.hist)) : nullptr;
    so.d_gpus = out->gpus ? static_cast<uint32_t *>(dptr(ar.gpus)) : nullptr;
    if (pieces == 0) {
        if ((rc = bin()) != DYN_OK) return rc;
        rc = dyn_eval_select(&dp, sp, static_cast<const float *>(dptr(ar.load)), S, int64_t(W), &so, dptr(ar.ws),
                             ar.ws_bytes, stream);
        if (rc != DYN_OK) return rc;
    } else {
        // piece k: scenarios [s0, s1) of the caller's loads, evaluated once they are in; piece `pieces` is scenario 0,
        // binned and evaluated once the trace is in
        for (int k = 0; k <= pieces; ++k) {
            const size_t s0 = k == pieces ? 0 : 1 + size_t(in->S_extra) * k / pieces;
            const size_t s1 = k == pieces ? 1 : 1 + size_t(in->S_extra) * (k + 1) / pieces;
            DYN_CUDA_TRY(cudaStreamWaitEvent(st, ev[k == pieces ? kTraceEvent : k], 0));
            if (k == pieces && (rc = bin()) != DYN_OK) return rc;
            dyn_select_out sk = so;
            sk.d_best_idx += s0 * wc; sk.d_best_E += s0 * wc; sk.d_E_total += s0; sk.d_n_infeasible += s0;
            if (sk.d_E_window) sk.d_E_window += s0 * W;
            if (sk.d_hist) sk.d_hist += s0 * J;
            if (sk.d_gpus) sk.d_gpus += s0 * W;
            // the tables are resolved once, by the first piece; the others run the sweep and the totals on them
            rc = dyn::eval_select_impl(&dp, sp, static_cast<const float *>(dptr(ar.load)) + s0 * wc, int64_t(s1 - s0), int64_t(W),
                                       &sk, dptr(ar.ws), ar.ws_bytes, st, k == 0);
            if (rc != DYN_OK) return rc;
            // the piece's results go back on the copy stream (behind the loads, which are long in by then) while
            // the next piece is evaluated
            DYN_CUDA_TRY(cudaEventRecord(ev[kPieces + 1 + k], st));
            DYN_CUDA_TRY(cudaStreamWaitEvent(cs, ev[kPieces + 1 + k], 0));
            const size_t ns = s1 - s0;
            if (out->best_idx) DYN_CUDA_TRY(cudaMemcpyAsync(out->best_idx + s0 * wc, sk.d_best_idx, ns * wc * 4, D2H, cs));
            if (out->best_E) DYN_CUDA_TRY(cudaMemcpyAsync(out->best_E + s0 * wc, sk.d_best_E, ns * wc * 4, D2H, cs));
            if (out->E_total) DYN_CUDA_TRY(cudaMemcpyAsync(out->E_total + s0, sk.d_E_total, ns * 8, D2H, cs));
            if (out->n_infeasible) DYN_CUDA_TRY(cudaMemcpyAsync(out->n_infeasible + s0, sk.d_n_infeasible, ns * 4, D2H, cs));
            if (out->E_window) DYN_CUDA_TRY(cudaMemcpyAsync(out->E_window + s0 * W, sk.d_E_window, ns * W * 8, D2H, cs));
            if (out->hist) DYN_CUDA_TRY(cudaMemcpyAsync(out->hist + s0 * J, sk.d_hist, ns * J * 4, D2H, cs));
            if (out->gpus) DYN_CUDA_TRY(cudaMemcpyAsync(out->gpus + s0 * W, sk.d_gpus, ns * W * 4, D2H, cs));
        }
        // the caller's stream is done when the last results have left
        DYN_CUDA_TRY(cudaEventRecord(ev[kPieces], cs));
        DYN_CUDA_TRY(cudaStreamWaitEvent(st, ev[kPieces], 0));
    }

    if (out->counts) DYN_CUDA_TRY(cudaMemcpyAsync(out->counts, dptr(ar.counts), wc * 4, D2H, st));
    if (out->dropped) DYN_CUDA_TRY(cudaMemcpyAsync(out->dropped, dptr(ar.dropped), 8, D2H, st));
    if (pieces == 0) {
        if (out->best_idx) DYN_CUDA_TRY(cudaMemcpyAsync(out->best_idx, dptr(ar.idx), tiles * 4, D2H, st));
        if (out->best_E) DYN_CUDA_TRY(cudaMemcpyAsync(out->best_E, dptr(ar.be), tiles * 4, D2H, st));
        if (out->E_total) DYN_CUDA_TRY(cudaMemcpyAsync(out->E_total, dptr(ar.etot), size_t(S) * 8, D2H, st));
        if (out->n_infeasible) DYN_CUDA_TRY(cudaMemcpyAsync(out->n_infeasible, dptr(ar.ninf), size_t(S) * 4, D2H, st));
        if (out->E_window) DYN_CUDA_TRY(cudaMemcpyAsync(out->E_window, dptr(ar.ewin), size_t(S) * W * 8, D2H, st));
        if (out->hist) DYN_CUDA_TRY(cudaMemcpyAsync(out->hist, dptr(ar.hist), size_t(S) * J * 4, D2H, st));
        if (out->gpus) DYN_CUDA_TRY(cudaMemcpyAsync(out->gpus, dptr(ar.gpus), size_t(S) * W * 4, D2H, st));
    }
    return DYN_OK;
}

}  // extern "C"
