// Token-weighted loads and carbon.
//
// bin_tokens: the paper states loads in tokens per second [Sec. 3, Sec. 3.2]; per (window, class) this sums the
// input tokens and the output tokens of the requests that fall there (window and class as in the trace binning).
// Exact 64-bit sums for any token values and any order of the trace.  A CTA owns a contiguous slice of requests;
// on a time-sorted trace the slice covers few windows, whose sums live in shared memory and are flushed once;
// whatever falls outside that range goes to global atomics.  Shared-memory sums are 32-bit (64-bit shared
// atomics are slow): the low and the high 16 bits of a token count are added to separate words, which cannot
// overflow within a slice (65536 x 65535 < 2^32).  Every word exists in up to 32 copies, a lane adding to the copy
// of its lane number: with 32 copies no two lanes of a warp meet on a word or on a bank (the four words of a
// bin are in four arrays, copies adjacent), so the atomics of a warp take one pass.  Reads 12 bytes per request,
// four requests per thread and load when the arrays are 16-byte aligned.
//
// carbon: window energies times the grid's carbon intensity, summed over the windows in a fixed order
// [Sec. 6.4]; fp64, one warp per scenario, bit-identical from run to run.
#define DYN_TU_ID 11
#include "dyn_internal.cuh"

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kSliceStep = 1024;              // slices are multiples of this (whole 16-byte loads per thread)
constexpr int kSliceMax = 16384;              // requests per CTA at most
constexpr int kWords = 3072;                  // bins x copies that a CTA holds in shared memory, per word array
static_assert(uint64_t(kSliceMax) * 65535ull < (1ull << 32), "16-bit halves must not overflow a 32-bit word within a slice");

struct TokenBins {
    uint32_t w_lo, nwin, C, W, copies_log2, stride;          // stride = bins x copies: length of one word array
};

// NI/NO: compile-time numbers of class edges (or -1: read them from the parameters)
template <int NI, int NO>
__device__ __forceinline__ uint32_t token_class(const BinParams &bp, uint32_t in, uint32_t out) {
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

// the same for a request whose token counts are known to be below 65536: the high halves add nothing
__device__ __forceinline__ void add_shared_low(uint32_t *p, uint32_t stride, uint32_t a, uint32_t b) {
    atomicAdd(p, a);
    atomicAdd(p + 2 * stride, b);
}

// adds one request's tokens to the sums of shared-memory bin `p` (the lane's copy)
__device__ __forceinline__ void add_shared(uint32_t *p, uint32_t stride, uint32_t a, uint32_t b) {
    atomicAdd(p, a & 0xffffu);
    atomicAdd(p + 2 * stride, b & 0xffffu);
    if ((a | b) >> 16) {                                     // token counts below 65536 (the usual case) add nothing here
        atomicAdd(p + stride, a >> 16);
        atomicAdd(p + 3 * stride, b >> 16);
    }
}

// any request, any order: window by division; dropped, shared or global by range
template <int NI, int NO>
__device__ __forceinline__ void add_request(const BinParams &bp, const TokenBins &tb, uint32_t *s_lane, uint32_t t, uint32_t a,
                                            uint32_t b, unsigned long long *tok_in, unsigned long long *tok_out) {
    const uint32_t w = fastdiv(t, bp.win);
    if (w >= tb.W) return;
    const uint32_t c = token_class<NI, NO>(bp, a, b);
    const uint32_t rel = w - tb.w_lo;                        // wraps for w < w_lo: then rel >= nwin
    if (rel < tb.nwin) {
        add_shared(s_lane + DYN_IDX((rel * tb.C + c) << tb.copies_log2, tb.stride), tb.stride, a, b);
    } else {
        atomicAdd(&tok_in[DYN_IDX(size_t(w) * tb.C + c, size_t(tb.W) * tb.C)], (unsigned long long)a);
        atomicAdd(&tok_out[DYN_IDX(size_t(w) * tb.C + c, size_t(tb.W) * tb.C)], (unsigned long long)b);
    }
}

// four consecutive requests of one lane.  The rule on a sorted trace: timestamps in order and both ends inside
// the CTA's window range; then nothing is out of range, and the middle windows are the end windows unless a
// window boundary falls among the four
template <int NI, int NO>
__device__ __forceinline__ void add_four(const BinParams &bp, const TokenBins &tb, uint32_t *s_lane, const uint4 vt, const uint4 va,
                                         const uint4 vb, unsigned long long *tok_in, unsigned long long *tok_out) {
    const uint32_t r0 = fastdiv(vt.x, bp.win) - tb.w_lo, r3 = fastdiv(vt.w, bp.win) - tb.w_lo;
    if ((vt.x <= vt.y) && (vt.y <= vt.z) && (vt.z <= vt.w) && (r0 < tb.nwin) && (r3 < tb.nwin)) {
        uint32_t r1 = r0, r2 = r0;
        if (r0 != r3) {
            r1 = fastdiv(vt.y, bp.win) - tb.w_lo;
            r2 = fastdiv(vt.z, bp.win) - tb.w_lo;
        }
        uint32_t *p0 = s_lane + DYN_IDX(((r0 * tb.C + token_class<NI, NO>(bp, va.x, vb.x)) << tb.copies_log2), tb.stride);
        uint32_t *p1 = s_lane + DYN_IDX(((r1 * tb.C + token_class<NI, NO>(bp, va.y, vb.y)) << tb.copies_log2), tb.stride);
        uint32_t *p2 = s_lane + DYN_IDX(((r2 * tb.C + token_class<NI, NO>(bp, va.z, vb.z)) << tb.copies_log2), tb.stride);
        uint32_t *p3 = s_lane + DYN_IDX(((r3 * tb.C + token_class<NI, NO>(bp, va.w, vb.w)) << tb.copies_log2), tb.stride);
        if (((va.x | va.y | va.z | va.w | vb.x | vb.y | vb.z | vb.w) >> 16) == 0u) {      // one test for all eight counts
            add_shared_low(p0, tb.stride, va.x, vb.x);
            add_shared_low(p1, tb.stride, va.y, vb.y);
            add_shared_low(p2, tb.stride, va.z, vb.z);
            add_shared_low(p3, tb.stride, va.w, vb.w);
        } else {
            add_shared(p0, tb.stride, va.x, vb.x);
            add_shared(p1, tb.stride, va.y, vb.y);
            add_shared(p2, tb.stride, va.z, vb.z);
            add_shared(p3, tb.stride, va.w, vb.w);
        }
    } else {
        add_request<NI, NO>(bp, tb, s_lane, vt.x, va.x, vb.x, tok_in, tok_out);
        add_request<NI, NO>(bp, tb, s_lane, vt.y, va.y, vb.y, tok_in, tok_out);
        add_request<NI, NO>(bp, tb, s_lane, vt.z, va.z, vb.z, tok_in, tok_out);
        add_request<NI, NO>(bp, tb, s_lane, vt.w, va.w, vb.w, tok_in, tok_out);
    }
}

template <int NI, int NO, bool VEC>
__global__ void __launch_bounds__(kThreads)
bin_tokens_kernel(const BinParams bp, const uint32_t *__restrict__ t_ms, const uint32_t *__restrict__ in_tok,
                  const uint32_t *__restrict__ out_tok, const uint64_t n_req, const uint32_t slice,
                  unsigned long long *__restrict__ tok_in, unsigned long long *__restrict__ tok_out) {
    __shared__ __align__(16) uint32_t s_sum[4 * kWords];     // {in low, in high, out low, out high}[bin][copy]
    const uint64_t begin = uint64_t(blockIdx.x) * slice;
    if (begin >= n_req) return;
    const uint32_t len = uint32_t(begin + slice < n_req ? slice : n_req - begin);
    t_ms += begin;
    in_tok += begin;
    out_tok += begin;
    TokenBins tb;
    tb.C = uint32_t(bp.C);
    tb.W = bp.n_windows;
    const uint32_t cap = uint32_t(kWords) / tb.C;            // windows that fit with one copy
    const uint32_t wa = fastdiv(t_ms[0], bp.win), wb = fastdiv(t_ms[len - 1], bp.win);
    tb.w_lo = wa < wb ? wa : wb;
    tb.nwin = 0;
    if (tb.w_lo < tb.W) {
        const uint32_t span = (wa < wb ? wb - wa : wa - wb) + 1u;
        tb.nwin = span < cap ? span : cap;
        if (tb.nwin > tb.W - tb.w_lo) tb.nwin = tb.W - tb.w_lo;
    }
    const uint32_t nbins = tb.nwin * tb.C;
    tb.copies_log2 = 0;
    while (tb.copies_log2 < 5 && (nbins << (tb.copies_log2 + 1)) <= uint32_t(kWords)) ++tb.copies_log2;
    tb.stride = DYN_IDX(nbins << tb.copies_log2, uint32_t(kWords) + 1u);      // four word arrays of this length fit in s_sum
    for (uint32_t i = threadIdx.x; i < tb.stride; i += kThreads)
        s_sum[i] = s_sum[i + tb.stride] = s_sum[i + 2 * tb.stride] = s_sum[i + 3 * tb.stride] = 0u;
    __syncthreads();
    uint32_t *s_lane = s_sum + (threadIdx.x & ((1u << tb.copies_log2) - 1u));          // this lane's copies
    uint32_t done = 0;
    if (VEC) {
        // the slice starts at a multiple of 1024 requests: 16-byte loads of four consecutive requests, two
        // batches (six loads) in flight per thread before any of them is used
        const uint32_t n4 = len >> 2;
        const uint4 *t4 = reinterpret_cast<const uint4 *>(t_ms), *a4 = reinterpret_cast<const uint4 *>(in_tok),
                    *b4 = reinterpret_cast<const uint4 *>(out_tok);
        uint32_t i = threadIdx.x;
        for (; i + kThreads < n4; i += 2 * kThreads) {
            const uint32_t j0 = DYN_IDX(i, n4), j1 = DYN_IDX(i + kThreads, n4);
            const uint4 t0 = __ldcs(t4 + j0), a0 = __ldcs(a4 + j0), b0 = __ldcs(b4 + j0);
            const uint4 t1 = __ldcs(t4 + j1), a1 = __ldcs(a4 + j1), b1 = __ldcs(b4 + j1);
            add_four<NI, NO>(bp, tb, s_lane, t0, a0, b0, tok_in, tok_out);
            add_four<NI, NO>(bp, tb, s_lane, t1, a1, b1, tok_in, tok_out);
        }
        if (i < n4) add_four<NI, NO>(bp, tb, s_lane, __ldcs(t4 + i), __ldcs(a4 + i), __ldcs(b4 + i), tok_in, tok_out);
        done = n4 << 2;
    }
    // ragged tail of the slice (and everything, when the arrays are not 16-byte aligned)
    for (uint32_t i = done + threadIdx.x; i < len; i += kThreads)
        add_request<NI, NO>(bp, tb, s_lane, t_ms[i], in_tok[i], out_tok[i], tok_in, tok_out);
    __syncthreads();
    // add the copies of every word (the slice's total of a 16-bit half fits 32 bits), then join the halves
    const uint32_t copies = 1u << tb.copies_log2;
    for (uint32_t i = threadIdx.x; i < 4 * nbins; i += kThreads) {
        uint32_t *q = s_sum + (i << tb.copies_log2);                        // word array i / nbins, bin i % nbins
        uint32_t sum = 0;
        for (uint32_t k = 0; k < copies; ++k) sum += q[(k + threadIdx.x) & (copies - 1u)];
        q[0] = sum;                                          // this thread alone reads and writes these copies
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < nbins; i += kThreads) {
        const uint32_t *q = s_sum + (i << tb.copies_log2);
        const unsigned long long si = (unsigned long long)q[0] + ((unsigned long long)q[tb.stride] << 16);
        const unsigned long long so = (unsigned long long)q[2 * tb.stride] + ((unsigned long long)q[3 * tb.stride] << 16);
        if (si) atomicAdd(&tok_in[DYN_IDX(size_t(tb.w_lo) * tb.C + i, size_t(tb.W) * tb.C)], si);
        if (so) atomicAdd(&tok_out[DYN_IDX(size_t(tb.w_lo) * tb.C + i, size_t(tb.W) * tb.C)], so);
    }
}

__global__ void tokens_to_tps_kernel(const unsigned long long *__restrict__ tok_in, const unsigned long long *__restrict__ tok_out,
                                     float *__restrict__ tps, uint64_t n, float window_s) {
    for (uint64_t i = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += uint64_t(gridDim.x) * blockDim.x)
        tps[DYN_IDX(i, n)] = __fdiv_rn(float(tok_in[DYN_IDX(i, n)] + tok_out[DYN_IDX(i, n)]), window_s);
}

// one warp per scenario; lane l sums windows l, l+32, ... in order, then the lanes are added in a fixed tree
__global__ void __launch_bounds__(kThreads) carbon_kernel(const double *__restrict__ E_window, const float *__restrict__ intensity,
                                                          int64_t S, int64_t W, double *__restrict__ carbon) {
    const int lane = threadIdx.x & 31;
    const int64_t s = int64_t(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    if (s >= S) return;
    double acc = 0.0;
    for (int64_t w = lane; w < W; w += 32) acc += E_window[DYN_IDX(s * W + w, S * W)] * double(intensity[DYN_IDX(w, W)]) / 1000.0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, off);
    if (lane == 0) carbon[s] = acc;
}

}  // namespace

cudaError_t launch_bin_tokens(const BinParams &bp, const uint32_t *t_ms, const uint32_t *in_tok, const uint32_t *out_tok,
                              uint64_t n_req, unsigned long long *tok_in, unsigned long long *tok_out, float *tps,
                              cudaStream_t st) {
    const uint64_t n_bins = uint64_t(bp.n_windows) * uint64_t(bp.C);
    cudaError_t e = cudaMemsetAsync(tok_in, 0, n_bins * sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(tok_out, 0, n_bins * sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;
    if (n_req > 0) {
        // slices sized for whole waves of resident CTAs, as few waves as the slice limit allows
        static thread_local int resident_of[kMaxDevices] = {};      // per device
        int &resident = resident_of[device_slot()];
        if (resident == 0) {
            int r = 0;
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, bin_tokens_kernel<2, 2, true>, kThreads, 0);
            if (e != cudaSuccess) return e;
            resident = r > 0 ? r : 1;
        }
        const uint64_t slots = uint64_t(sm_count()) * uint64_t(resident);
        const uint64_t waves = (n_req + slots * kSliceMax - 1) / (slots * kSliceMax);
        uint64_t slice = (n_req + waves * slots - 1) / (waves * slots);
        slice = (slice + kSliceStep - 1) / kSliceStep * kSliceStep;
        if (slice > uint64_t(kSliceMax)) slice = kSliceMax;
        const uint64_t grid = (n_req + slice - 1) / slice;
        if (grid > (uint64_t(1) << 31) - 1) return cudaErrorInvalidValue;
        const bool vec = ((reinterpret_cast<uintptr_t>(t_ms) | reinterpret_cast<uintptr_t>(in_tok) |
                           reinterpret_cast<uintptr_t>(out_tok)) & 15u) == 0;
        e = record_start(st);
        if (e != cudaSuccess) return e;
        const unsigned g = unsigned(grid);
        const uint32_t sl = uint32_t(slice);
        if (bp.n_in == 2 && bp.n_out == 2) {                 // the 3 x 3 classes of the thresholds table
            if (vec) bin_tokens_kernel<2, 2, true><<<g, kThreads, 0, st>>>(bp, t_ms, in_tok, out_tok, n_req, sl, tok_in, tok_out);
            else bin_tokens_kernel<2, 2, false><<<g, kThreads, 0, st>>>(bp, t_ms, in_tok, out_tok, n_req, sl, tok_in, tok_out);
        } else {
            if (vec) bin_tokens_kernel<-1, -1, true><<<g, kThreads, 0, st>>>(bp, t_ms, in_tok, out_tok, n_req, sl, tok_in, tok_out);
            else bin_tokens_kernel<-1, -1, false><<<g, kThreads, 0, st>>>(bp, t_ms, in_tok, out_tok, n_req, sl, tok_in, tok_out);
        }
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        e = record_stop(st);
        if (e != cudaSuccess) return e;
    }
    if (tps) {
        uint64_t blocks = (n_bins + 255) / 256;
        const uint64_t cap = uint64_t(sm_count()) * 8;
        if (blocks > cap) blocks = cap;
        tokens_to_tps_kernel<<<unsigned(blocks), 256, 0, st>>>(tok_in, tok_out, tps, n_bins, bp.window_s);
        e = cudaGetLastError();
    }
    return e;
}

cudaError_t launch_carbon(const double *E_window, const float *intensity, int64_t S, int64_t W, double *carbon, cudaStream_t st) {
    if (S == 0) return cudaSuccess;
    carbon_kernel<<<unsigned((S + kThreads / 32 - 1) / (kThreads / 32)), kThreads, 0, st>>>(E_window, intensity, S, W, carbon);
    return cudaGetLastError();
}

}  // namespace dyn
