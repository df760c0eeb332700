// Stage (a): trace -> per-(window, class) request counts and loads.
//
// Each request (timestamp, input tokens, output tokens) [Sec. 3] gets a time window and one of the
// KI x KO length classes of the thresholds table [Sec. 3.1]; the per-class load over time [Sec. 3.2]
// is the count per (window, class) divided by the window length.
//
// Memory-bound: 12 bytes are read per request and nothing else scales with the trace.  A CTA owns a
// contiguous slice of the trace; on a time-sorted trace that slice covers few windows, so its bins
// live in shared memory.  A warp takes 128 consecutive requests (one 16-byte load per lane and
// array), reduces the requests of one window to per-class counts with packed 8-bit counters and
// warp-wide integer reductions, and issues at most C shared-memory atomics per window present.
// Requests outside the CTA's window range (unsorted input) go to global atomics, so the counts are
// exact for any order.
#include "dyn_internal.cuh"

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kSmemBins = 4096;       // uint32 bins per CTA
constexpr int kBatch = 128;           // requests per warp step (4 per lane)
constexpr int kMaxRounds = 4;         // distinct windows reduced per batch before falling back
constexpr unsigned kFull = 0xffffffffu;

template <int NI, int NO>
__device__ __forceinline__ uint32_t classify(const BinParams &bp, uint32_t in, uint32_t out) {
    uint32_t ci = 0, co = 0;
    if (NI >= 0) {
#pragma unroll
        for (int e = 0; e < NI; ++e) ci += (bp.in_edges[e] <= in) ? 1u : 0u;
#pragma unroll
        for (int e = 0; e < NO; ++e) co += (bp.out_edges[e] <= out) ? 1u : 0u;
        return ci * uint32_t(NO + 1) + co;
    } else {
        for (int e = 0; e < bp.n_in; ++e) ci += (bp.in_edges[e] <= in) ? 1u : 0u;
        for (int e = 0; e < bp.n_out; ++e) co += (bp.out_edges[e] <= out) ? 1u : 0u;
        return ci * uint32_t(bp.n_out + 1) + co;
    }
}

// NI/NO: compile-time edge counts (or -1: read them from the parameters).
// PACKED: C <= 16, per-class counts of a window travel as 4 x 8-bit fields in up to 4 words.
// VEC: the three arrays are 16-byte aligned.
template <int NI, int NO, bool PACKED, bool VEC>
__global__ void __launch_bounds__(kThreads)
bin_trace_kernel(const BinParams bp, const uint32_t *__restrict__ t_ms, const uint32_t *__restrict__ in_tok,
                 const uint32_t *__restrict__ out_tok, const uint64_t n_req, const uint64_t chunk,
                 uint32_t *__restrict__ counts, unsigned long long *__restrict__ dropped) {
    __shared__ uint32_t sbins[kSmemBins];

    const uint64_t begin = uint64_t(blockIdx.x) * chunk;
    if (begin >= n_req) return;
    const uint64_t end = (begin + chunk < n_req) ? begin + chunk : n_req;
    const uint32_t C = uint32_t(bp.C);
    const uint32_t W = bp.n_windows;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;

    // window range kept in shared memory: starts at the window of the slice's first (or last,
    // if that is earlier) request
    const uint32_t wa = fastdiv(t_ms[begin], bp.win);
    const uint32_t wb = fastdiv(t_ms[end - 1], bp.win);
    const uint32_t w_lo = wa < wb ? wa : wb;
    uint32_t nwin = 0;
    if (w_lo < W) {
        const uint32_t span = (wa < wb ? wb - wa : wa - wb) + 1u;
        const uint32_t cap = uint32_t(kSmemBins) / C;
        nwin = span < cap ? span : cap;
        if (nwin > W - w_lo) nwin = W - w_lo;
    }
    const uint32_t nbins = nwin * C;
    for (uint32_t i = threadIdx.x; i < nbins; i += kThreads) sbins[i] = 0u;
    __syncthreads();

    auto add_bin = [&](uint32_t w, uint32_t c, uint32_t v) {
        const uint32_t rel = w - w_lo;                       // wraps for w < w_lo: then rel >= nwin
        if (rel < nwin) atomicAdd(&sbins[rel * C + c], v);
        else atomicAdd(&counts[size_t(w) * C + c], v);
    };

    uint32_t my_dropped = 0;
    for (uint64_t base = begin + uint64_t(warp) * kBatch; base < end; base += uint64_t(kWarps) * kBatch) {
        const uint64_t i0 = base + uint64_t(lane) * 4;
        uint32_t t[4], a[4], b[4];
        uint32_t live = 0;
        if (VEC && i0 + 4 <= end) {
            const uint4 vt = *reinterpret_cast<const uint4 *>(t_ms + i0);
            const uint4 va = *reinterpret_cast<const uint4 *>(in_tok + i0);
            const uint4 vb = *reinterpret_cast<const uint4 *>(out_tok + i0);
            t[0] = vt.x; t[1] = vt.y; t[2] = vt.z; t[3] = vt.w;
            a[0] = va.x; a[1] = va.y; a[2] = va.z; a[3] = va.w;
            b[0] = vb.x; b[1] = vb.y; b[2] = vb.z; b[3] = vb.w;
            live = 0xfu;
        } else {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                t[r] = a[r] = b[r] = 0u;
                if (i0 + r < end) {
                    t[r] = t_ms[i0 + r];
                    a[r] = in_tok[i0 + r];
                    b[r] = out_tok[i0 + r];
                    live |= 1u << r;
                }
            }
        }
        uint32_t w[4], c[4];
        uint32_t ndrop = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            w[r] = fastdiv(t[r], bp.win);
            c[r] = classify<NI, NO>(bp, a[r], b[r]);
            if ((live >> r & 1u) && w[r] >= W) {
                live &= ~(1u << r);
                ++ndrop;
            }
        }
        my_dropped += ndrop;

        if (PACKED) {
            // one round per distinct window present in the batch, earliest first
            for (int round = 0; round < kMaxRounds; ++round) {
                uint32_t wmin = 0xffffffffu;
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if (live >> r & 1u) wmin = w[r] < wmin ? w[r] : wmin;
                wmin = __reduce_min_sync(kFull, wmin);
                if (wmin == 0xffffffffu) break;              // warp-uniform
                uint32_t pk0 = 0, pk1 = 0, pk2 = 0, pk3 = 0;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if ((live >> r & 1u) && w[r] == wmin) {
                        const uint32_t inc = 1u << ((c[r] & 3u) * 8u);
                        const uint32_t g = c[r] >> 2;
                        pk0 += g == 0 ? inc : 0u;
                        pk1 += g == 1 ? inc : 0u;
                        pk2 += g == 2 ? inc : 0u;
                        pk3 += g == 3 ? inc : 0u;
                        live &= ~(1u << r);
                    }
                }
                // at most 4 requests x 32 lanes = 128 per 8-bit field: no carry between fields
                uint32_t s0 = __reduce_add_sync(kFull, pk0), s1 = 0, s2 = 0, s3 = 0;
                if (C > 4) s1 = __reduce_add_sync(kFull, pk1);
                if (C > 8) s2 = __reduce_add_sync(kFull, pk2);
                if (C > 12) s3 = __reduce_add_sync(kFull, pk3);
                if (uint32_t(lane) < C) {
                    const uint32_t g = uint32_t(lane) >> 2;
                    const uint32_t word = g == 0 ? s0 : g == 1 ? s1 : g == 2 ? s2 : s3;
                    const uint32_t cnt = (word >> ((uint32_t(lane) & 3u) * 8u)) & 0xffu;
                    if (cnt) add_bin(wmin, uint32_t(lane), cnt);
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (live >> r & 1u) add_bin(w[r], c[r], 1u);
        } else {
            // many classes: lanes holding the same bin elect one leader that adds the group size
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const bool on = live >> r & 1u;
                const uint32_t key = on ? w[r] * C + c[r] : (0x80000000u | uint32_t(lane));
                const unsigned peers = __match_any_sync(kFull, key);
                if (on && lane == __ffs(peers) - 1) add_bin(w[r], c[r], uint32_t(__popc(peers)));
            }
        }
    }

    my_dropped = __reduce_add_sync(kFull, my_dropped);
    if (lane == 0 && my_dropped) atomicAdd(dropped, (unsigned long long)my_dropped);

    __syncthreads();
    for (uint32_t i = threadIdx.x; i < nbins; i += kThreads) {
        const uint32_t v = sbins[i];
        if (v) atomicAdd(&counts[size_t(w_lo) * C + i], v);
    }
}

__global__ void counts_to_load_kernel(const uint32_t *__restrict__ counts, float *__restrict__ load, uint64_t n,
                                      float window_s) {
    for (uint64_t i = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += uint64_t(gridDim.x) * blockDim.x)
        load[i] = __fdiv_rn(float(counts[i]), window_s);
}

template <int NI, int NO, bool PACKED>
cudaError_t launch_variant(bool vec, int grid, const BinParams &bp, const uint32_t *t, const uint32_t *a,
                           const uint32_t *b, uint64_t n, uint64_t chunk, uint32_t *counts,
                           unsigned long long *dropped, cudaStream_t st) {
    if (vec) bin_trace_kernel<NI, NO, PACKED, true><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
    else bin_trace_kernel<NI, NO, PACKED, false><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bin_trace(const BinParams &bp, const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok,
                             uint64_t n_req, uint32_t *counts, float *load, unsigned long long *dropped,
                             cudaStream_t st) {
    const uint64_t n_bins = uint64_t(bp.n_windows) * uint64_t(bp.C);
    cudaError_t e = cudaMemsetAsync(counts, 0, n_bins * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(dropped, 0, sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;

    if (n_req > 0) {
        const uint64_t batches = (n_req + kBatch - 1) / kBatch;
        uint64_t grid = (batches + kWarps - 1) / kWarps;
        const uint64_t max_grid = uint64_t(sm_count()) * 8;
        if (grid > max_grid) grid = max_grid;
        const uint64_t chunk = ((batches + grid - 1) / grid) * kBatch;     // multiple of 128: keeps 16-byte alignment
        grid = (n_req + chunk - 1) / chunk;
        const bool vec = ((reinterpret_cast<uintptr_t>(t_ms) | reinterpret_cast<uintptr_t>(in_tok) |
                           reinterpret_cast<uintptr_t>(out_tok)) & 15u) == 0;
        const int g = int(grid);
        e = record_start(st);
        if (e != cudaSuccess) return e;
        if (bp.C <= 16) {
            if (bp.n_in == 2 && bp.n_out == 2)
                e = launch_variant<2, 2, true>(vec, g, bp, t_ms, in_tok, out_tok, n_req, chunk, counts, dropped, st);
            else
                e = launch_variant<-1, -1, true>(vec, g, bp, t_ms, in_tok, out_tok, n_req, chunk, counts, dropped, st);
        } else {
            e = launch_variant<-1, -1, false>(vec, g, bp, t_ms, in_tok, out_tok, n_req, chunk, counts, dropped, st);
        }
        if (e != cudaSuccess) return e;
        e = record_stop(st);
        if (e != cudaSuccess) return e;
    }
    if (load) {
        const int threads = 256;
        uint64_t blocks = (n_bins + threads - 1) / threads;
        const uint64_t cap = uint64_t(sm_count()) * 8;
        if (blocks > cap) blocks = cap;
        counts_to_load_kernel<<<int(blocks), threads, 0, st>>>(counts, load, n_bins, bp.window_s);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace dyn
