// Stage (a): trace -> per-(window, class) request counts and loads.
//
// Each request (timestamp, input tokens, output tokens) [Sec. 3] gets a time window and one of the
// KI x KO length classes of the thresholds table [Sec. 3.1]; the per-class load over time [Sec. 3.2]
// is the count per (window, class) divided by the window length.
//
// Memory-bound: 12 bytes are read per request and nothing else scales with the trace, so the kernel
// is written for few instructions per request.  A CTA owns a contiguous slice of the trace; on a
// time-sorted trace that slice covers few windows, so its bins live in shared memory, four copies of
// each bin side by side (lane l adds to copy l mod 4) so that the lanes of one warp instruction that
// hit the same (window, class) spread over four banks.  A warp takes 128 consecutive requests (one
// 16-byte load per lane and array, two batches in flight).  When a lane's four timestamps are in order
// and both ends fall inside the CTA's window range (the rule on a sorted trace) nothing has to be
// tested per request, and two divisions serve all four unless a window boundary falls among them; the
// window is a multiply-shift division by the invariant window length.  Requests outside the CTA's
// window range (unsorted input) go to global atomics, so the counts are exact for any order.
#define DYN_TU_ID 2
#include "dyn_internal.cuh"

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCopies = 4;            // copies of every shared-memory bin
constexpr int kSmemBins = 6144;       // uint32 words of bins per CTA (copies included)
constexpr int kBatch = 128;           // requests per warp step (4 per lane)
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
// VEC: the three arrays are 16-byte aligned.
// PIECES: a slice may be taken in several pieces (chosen by the host for long slices); without it the
// slice is one piece and the code is the plain straight-line form.
template <int NI, int NO, bool VEC, bool PIECES>
__global__ void __launch_bounds__(kThreads)
bin_trace_kernel(const BinParams bp, const uint32_t *__restrict__ t_ms, const uint32_t *__restrict__ in_tok,
                 const uint32_t *__restrict__ out_tok, const uint64_t n_req, const uint64_t chunk,
                 uint32_t *__restrict__ counts, unsigned long long *__restrict__ dropped) {
    __shared__ __align__(16) uint32_t sbins[kSmemBins];

    const uint64_t cta_begin = uint64_t(blockIdx.x) * chunk;
    if (cta_begin >= n_req) return;
    const uint64_t cta_end = (cta_begin + chunk < n_req) ? cta_begin + chunk : n_req;
    const uint32_t C = uint32_t(bp.C);
    const uint32_t W = bp.n_windows;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t copy = uint32_t(lane) & (kCopies - 1);
    const uint32_t cap = uint32_t(kSmemBins / kCopies) / C;  // windows whose bins fit in shared memory
    const uint64_t step = uint64_t(kWarps) * kBatch;

    // A slice that spans more windows than fit (a long sparse trace) is taken in pieces sized from its
    // average density; whatever still falls outside a piece's window range goes to global atomics.
    uint64_t piece = cta_end - cta_begin;
    const uint32_t cta_wa = fastdiv(t_ms[cta_begin], bp.win), cta_wb = fastdiv(t_ms[cta_end - 1], bp.win);
    {
        const uint32_t wa = cta_wa, wb = cta_wb;
        const uint64_t span = uint64_t(wa < wb ? wb - wa : wa - wb) + 1u;
        if (PIECES && span > cap) {
            piece = piece * cap / span * 3 / 4;
            piece = piece / (2 * step) * (2 * step);         // whole double-batch passes of the CTA
            if (piece < 2 * step) piece = 2 * step;
        }
    }
    uint32_t my_dropped = 0;

    auto run_piece = [&](const uint64_t begin, const uint64_t end, const uint32_t wa, const uint32_t wb) {
    // window range kept in shared memory: starts at the window of the piece's first (or last,
    // if that is earlier) request
    const uint32_t w_lo = wa < wb ? wa : wb;
    uint32_t nwin = 0;
    if (w_lo < W) {
        const uint32_t span = (wa < wb ? wb - wa : wa - wb) + 1u;
        nwin = span < cap ? span : cap;
        if (nwin > W - w_lo) nwin = W - w_lo;
    }
    const uint32_t nbins = nwin * C;                         // distinct bins held here
    for (uint32_t i = threadIdx.x; i < nbins * kCopies; i += kThreads) sbins[DYN_IDX(i, kSmemBins)] = 0u;
    __syncthreads();

    // any request, any order: window by division, dropped / shared / global by range
    auto count_one = [&](uint32_t t, uint32_t a, uint32_t b, uint32_t &ndrop) {
        const uint32_t w = fastdiv(t, bp.win);
        if (w >= W) {
            ++ndrop;
            return;
        }
        const uint32_t c = classify<NI, NO>(bp, a, b);
        const uint32_t rel = w - w_lo;                       // wraps for w < w_lo: then rel >= nwin
        if (rel < nwin) atomicAdd(&sbins[DYN_IDX((rel * C + c) * kCopies + copy, kSmemBins)], 1u);
        else atomicAdd(&counts[DYN_IDX(size_t(w) * C + c, size_t(W) * C)], 1u);
    };

    // four consecutive requests of one lane
    auto count_four = [&](const uint4 vt, const uint4 va, const uint4 vb, uint32_t &ndrop) {
        // the rule on a sorted trace: timestamps in order and both ends inside the CTA's window range;
        // then no request is dropped or out of range, and the middle windows are the end windows
        // unless a window boundary falls between the lane's four requests
        const uint32_t w0 = fastdiv(vt.x, bp.win), w3 = fastdiv(vt.w, bp.win);
        const uint32_t r0 = w0 - w_lo, r3 = w3 - w_lo;
        const bool fast = (vt.x <= vt.y) && (vt.y <= vt.z) && (vt.z <= vt.w) && (r0 < nwin) && (r3 < nwin);
        if (fast) {
            uint32_t r1 = r0, r2 = r0;
            if (r0 != r3) {
                r1 = fastdiv(vt.y, bp.win) - w_lo;
                r2 = fastdiv(vt.z, bp.win) - w_lo;
            }
            uint32_t *row = sbins + copy;
            const uint32_t stride = C * kCopies;
            atomicAdd(row + DYN_IDX((r0 * stride + classify<NI, NO>(bp, va.x, vb.x) * kCopies), uint32_t(kSmemBins) - copy), 1u);
            atomicAdd(row + DYN_IDX((r1 * stride + classify<NI, NO>(bp, va.y, vb.y) * kCopies), uint32_t(kSmemBins) - copy), 1u);
            atomicAdd(row + DYN_IDX((r2 * stride + classify<NI, NO>(bp, va.z, vb.z) * kCopies), uint32_t(kSmemBins) - copy), 1u);
            atomicAdd(row + DYN_IDX((r3 * stride + classify<NI, NO>(bp, va.w, vb.w) * kCopies), uint32_t(kSmemBins) - copy), 1u);
        } else {
            count_one(vt.x, va.x, vb.x, ndrop);
            count_one(vt.y, va.y, vb.y, ndrop);
            count_one(vt.z, va.z, vb.z, ndrop);
            count_one(vt.w, va.w, vb.w, ndrop);
        }
    };

    uint64_t base = begin + uint64_t(warp) * kBatch;
    if (VEC) {
        // two full batches per pass: six 16-byte loads in flight per lane before any of them is used
        for (; base + step + kBatch <= end; base += 2 * step) {
            const uint64_t i0 = DYN_IDX(base + uint64_t(lane) * 4, n_req - 3), i1 = DYN_IDX(i0 + step, n_req - 3);
            const uint4 t0 = __ldcs(reinterpret_cast<const uint4 *>(t_ms + i0));
            const uint4 a0 = __ldcs(reinterpret_cast<const uint4 *>(in_tok + i0));
            const uint4 b0 = __ldcs(reinterpret_cast<const uint4 *>(out_tok + i0));
            const uint4 t1 = __ldcs(reinterpret_cast<const uint4 *>(t_ms + i1));
            const uint4 a1 = __ldcs(reinterpret_cast<const uint4 *>(in_tok + i1));
            const uint4 b1 = __ldcs(reinterpret_cast<const uint4 *>(out_tok + i1));
            count_four(t0, a0, b0, my_dropped);
            count_four(t1, a1, b1, my_dropped);
        }
        for (; base + kBatch <= end; base += step) {
            const uint64_t i0 = DYN_IDX(base + uint64_t(lane) * 4, n_req - 3);
            count_four(__ldcs(reinterpret_cast<const uint4 *>(t_ms + i0)),
                       __ldcs(reinterpret_cast<const uint4 *>(in_tok + i0)),
                       __ldcs(reinterpret_cast<const uint4 *>(out_tok + i0)), my_dropped);
        }
    }
    // ragged tail of the slice (and everything, when the arrays are not 16-byte aligned)
    for (; base < end; base += step) {
        const uint64_t i0 = base + uint64_t(lane) * 4;
#pragma unroll
        for (int r = 0; r < 4; ++r)
            if (i0 + r < end) {
                const uint64_t ir = DYN_IDX(i0 + r, n_req);
                count_one(t_ms[ir], in_tok[ir], out_tok[ir], my_dropped);
            }
    }

    __syncthreads();
    for (uint32_t i = threadIdx.x; i < nbins; i += kThreads) {
        const uint4 v = *reinterpret_cast<const uint4 *>(&sbins[DYN_IDX(i * kCopies, kSmemBins - 3)]);
        const uint32_t sum = v.x + v.y + v.z + v.w;
        if (sum) atomicAdd(&counts[DYN_IDX(size_t(w_lo) * C + i, size_t(W) * C)], sum);
    }
    };   // run_piece

    if (!PIECES || piece == cta_end - cta_begin) {           // one piece, ends already read
        run_piece(cta_begin, cta_end, cta_wa, cta_wb);
    } else {
        for (uint64_t begin = cta_begin; begin < cta_end; begin += piece) {
            const uint64_t end = (begin + piece < cta_end) ? begin + piece : cta_end;
            run_piece(begin, end, fastdiv(t_ms[begin], bp.win), fastdiv(t_ms[end - 1], bp.win));
            __syncthreads();                                 // the bins are cleared again for the next piece
        }
    }

    my_dropped = __reduce_add_sync(kFull, my_dropped);
    if (lane == 0 && my_dropped) atomicAdd(dropped, (unsigned long long)my_dropped);
}

__global__ void counts_to_load_kernel(const uint32_t *__restrict__ counts, float *__restrict__ load, uint64_t n,
                                      float window_s) {
    for (uint64_t i = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += uint64_t(gridDim.x) * blockDim.x)
        load[DYN_IDX(i, n)] = __fdiv_rn(float(counts[DYN_IDX(i, n)]), window_s);
}

template <int NI, int NO>
cudaError_t launch_variant(bool vec, int grid, const BinParams &bp, const uint32_t *t, const uint32_t *a,
                           const uint32_t *b, uint64_t n, uint64_t chunk, uint32_t *counts,
                           unsigned long long *dropped, cudaStream_t st) {
    // slices longer than this may span more windows than the shared-memory bins hold
    const bool pieces = chunk > 12288;
    if (vec && pieces) bin_trace_kernel<NI, NO, true, true><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
    else if (vec) bin_trace_kernel<NI, NO, true, false><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
    else if (pieces) bin_trace_kernel<NI, NO, false, true><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
    else bin_trace_kernel<NI, NO, false, false><<<grid, kThreads, 0, st>>>(bp, t, a, b, n, chunk, counts, dropped);
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
        // two whole waves of resident CTAs (a whole number of waves keeps every SM slot busy to the end; worth a
        // few percent on 14 M requests) for traces up to a few tens of millions of requests; beyond that more CTAs rather than longer slices (a slice of about 24 K requests streams best:
        // measured 6.7 TB/s on 112 M requests against 5.5 TB/s with slices of 95 K)
        static thread_local int resident_of[kMaxDevices] = {};      // per device
        int &resident = resident_of[device_slot()];
        if (resident == 0) {
            int r = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, bin_trace_kernel<2, 2, true, false>, kThreads, 0) !=
                    cudaSuccess || r < 1)
                r = 4;
            resident = r;
        }
        uint64_t max_grid = uint64_t(sm_count()) * uint64_t(resident) * 2;
        const uint64_t by_slice = (n_req + 24575) / 24576;
        if (max_grid < by_slice) max_grid = by_slice;
        if (max_grid > (uint64_t(1) << 30)) max_grid = uint64_t(1) << 30;
        if (grid > max_grid) grid = max_grid;
        const uint64_t chunk = ((batches + grid - 1) / grid) * kBatch;     // multiple of 128: keeps 16-byte alignment
        grid = (n_req + chunk - 1) / chunk;
        const bool vec = ((reinterpret_cast<uintptr_t>(t_ms) | reinterpret_cast<uintptr_t>(in_tok) |
                           reinterpret_cast<uintptr_t>(out_tok)) & 15u) == 0;
        const int g = int(grid);
        e = record_start(st);
        if (e != cudaSuccess) return e;
        if (bp.n_in == 2 && bp.n_out == 2)
            e = launch_variant<2, 2>(vec, g, bp, t_ms, in_tok, out_tok, n_req, chunk, counts, dropped, st);
        else
            e = launch_variant<-1, -1>(vec, g, bp, t_ms, in_tok, out_tok, n_req, chunk, counts, dropped, st);
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
