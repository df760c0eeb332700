// Token-weighted loads and carbon.
//
// bin_tokens: the paper states loads in tokens per second [Sec. 3, Sec. 3.2]; per (window, class) this sums the
// input tokens and the output tokens of the requests that fall there (window and class as in the trace binning).
// Exact 64-bit sums for any token values and any order of the trace.  A CTA owns a contiguous slice of 8192
// requests; on a time-sorted trace the slice covers few windows, whose sums live in shared memory and are flushed
// once; whatever falls outside that range goes to global atomics.  Shared-memory sums are 32-bit (64-bit shared
// atomics are slow): the low and the high 16 bits of a token count are added to separate words, which cannot
// overflow within a slice (8192 x 65535 < 2^32), and two copies of every word halve the collisions of
// neighbouring lanes.  Reads 12 bytes per request.
//
// carbon: window energies times the grid's carbon intensity, summed over the windows in a fixed order
// [Sec. 6.4]; fp64, one warp per scenario, bit-identical from run to run.
#include "dyn_internal.cuh"

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kSlice = 8192;                  // requests per CTA
constexpr int kBins = 1024;                   // (window, class) pairs whose sums a CTA holds in shared memory
static_assert(uint64_t(kSlice) * 65535ull < (1ull << 32), "16-bit halves must not overflow a 32-bit word within a slice");

__global__ void __launch_bounds__(kThreads)
bin_tokens_kernel(const BinParams bp, const uint32_t *__restrict__ t_ms, const uint32_t *__restrict__ in_tok,
                  const uint32_t *__restrict__ out_tok, const uint64_t n_req, unsigned long long *__restrict__ tok_in,
                  unsigned long long *__restrict__ tok_out) {
    __shared__ __align__(16) uint32_t s_sum[kBins][2][4];                  // [bin][copy]{in low, in high, out low, out high}
    const uint64_t begin = uint64_t(blockIdx.x) * kSlice;
    if (begin >= n_req) return;
    const uint64_t end = begin + kSlice < n_req ? begin + kSlice : n_req;
    const uint32_t C = uint32_t(bp.C), W = bp.n_windows;
    const uint32_t cap = uint32_t(kBins) / C;                // windows that fit
    const uint32_t wa = fastdiv(t_ms[begin], bp.win), wb = fastdiv(t_ms[end - 1], bp.win);
    const uint32_t w_lo = wa < wb ? wa : wb;
    uint32_t nwin = 0;
    if (w_lo < W) {
        const uint32_t span = (wa < wb ? wb - wa : wa - wb) + 1u;
        nwin = span < cap ? span : cap;
        if (nwin > W - w_lo) nwin = W - w_lo;
    }
    const uint32_t nbins = nwin * C;
    for (uint32_t i = threadIdx.x; i < nbins * 8; i += kThreads) (&s_sum[0][0][0])[i] = 0u;
    __syncthreads();
    const uint32_t copy = threadIdx.x & 1u;
    for (uint64_t i = begin + threadIdx.x; i < end; i += kThreads) {
        const uint32_t a = in_tok[i], b = out_tok[i];
        const uint32_t w = fastdiv(t_ms[i], bp.win);
        if (w >= W) continue;
        uint32_t ci = 0, co = 0;
        for (int e = 0; e < bp.n_in; ++e) ci += (bp.in_edges[e] <= a) ? 1u : 0u;
        for (int e = 0; e < bp.n_out; ++e) co += (bp.out_edges[e] <= b) ? 1u : 0u;
        const uint32_t c = ci * uint32_t(bp.n_out + 1) + co;
        const uint32_t rel = w - w_lo;                       // wraps for w < w_lo: then rel >= nwin
        if (rel < nwin) {
            uint32_t *p = s_sum[rel * C + c][copy];
            atomicAdd(p + 0, a & 0xffffu);
            atomicAdd(p + 1, a >> 16);
            atomicAdd(p + 2, b & 0xffffu);
            atomicAdd(p + 3, b >> 16);
        } else {
            atomicAdd(&tok_in[size_t(w) * C + c], (unsigned long long)a);
            atomicAdd(&tok_out[size_t(w) * C + c], (unsigned long long)b);
        }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < nbins; i += kThreads) {
        const uint4 x = *reinterpret_cast<const uint4 *>(s_sum[i][0]), y = *reinterpret_cast<const uint4 *>(s_sum[i][1]);
        const unsigned long long si = (unsigned long long)x.x + y.x + (((unsigned long long)x.y + y.y) << 16);
        const unsigned long long so = (unsigned long long)x.z + y.z + (((unsigned long long)x.w + y.w) << 16);
        if (si) atomicAdd(&tok_in[size_t(w_lo) * C + i], si);
        if (so) atomicAdd(&tok_out[size_t(w_lo) * C + i], so);
    }
}

__global__ void tokens_to_tps_kernel(const unsigned long long *__restrict__ tok_in, const unsigned long long *__restrict__ tok_out,
                                     float *__restrict__ tps, uint64_t n, float window_s) {
    for (uint64_t i = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += uint64_t(gridDim.x) * blockDim.x)
        tps[i] = __fdiv_rn(float(tok_in[i] + tok_out[i]), window_s);
}

// one warp per scenario; lane l sums windows l, l+32, ... in order, then the lanes are added in a fixed tree
__global__ void __launch_bounds__(kThreads) carbon_kernel(const double *__restrict__ E_window, const float *__restrict__ intensity,
                                                          int64_t S, int64_t W, double *__restrict__ carbon) {
    const int lane = threadIdx.x & 31;
    const int64_t s = int64_t(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    if (s >= S) return;
    double acc = 0.0;
    for (int64_t w = lane; w < W; w += 32) acc += E_window[s * W + w] * double(intensity[w]) / 1000.0;
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
        const uint64_t grid = (n_req + kSlice - 1) / kSlice;
        if (grid > (uint64_t(1) << 31) - 1) return cudaErrorInvalidValue;
        e = record_start(st);
        if (e != cudaSuccess) return e;
        bin_tokens_kernel<<<unsigned(grid), kThreads, 0, st>>>(bp, t_ms, in_tok, out_tok, n_req, tok_in, tok_out);
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
