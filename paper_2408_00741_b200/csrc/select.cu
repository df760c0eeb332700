// Stage (c): per-tile masked argmin over a materialised energy tensor, and cluster totals.
//
// The chosen configuration of a tile is the minimum-energy candidate among those that meet the
// SLO [Sec. 4.2]; infeasible candidates carry +inf.  Ties go to the lowest candidate index.  Totals
// per scenario (cluster energy, energy per window, GPUs in use, how often each candidate is chosen)
// follow the cluster-level quantities of the evaluation [Sec. 6].
//
// select: one warp per tile, lanes stride over the candidates with 16-byte streaming loads, each
// lane keeps its first minimum, then two warp-wide integer min-reductions pick (energy, index).
// totals: fp64 sums in a fixed order (thread: the classes of its window in order; block: a fixed tree
// over 256 windows; scenario: chunks in order), so results repeat bit for bit.
#define DYN_TU_ID 5
#include "dyn_internal.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kChunkWindows = 256;           // one window per thread; must match totals_chunks()

__device__ __forceinline__ uint32_t float_key(float v) {
    const uint32_t b = __float_as_uint(v);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}

template <bool VEC4>
__global__ void __launch_bounds__(kThreads)
select_kernel(const float *__restrict__ E, int64_t tiles, int J, int32_t *__restrict__ best_idx,
              float *__restrict__ best_E) {
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t i = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); i < tiles; i += nwarps) {
        const float *row = E + size_t(DYN_IDX(i, tiles)) * size_t(J);
        float best = CUDART_INF_F;
        int bj = 0x7fffffff;
        if (VEC4) {
            const float4 *row4 = reinterpret_cast<const float4 *>(row);
            const int J4 = J >> 2;
#pragma unroll 4
            for (int q = lane; q < J4; q += 32) {
                const float4 v = __ldcs(row4 + DYN_IDX(q, J4));
                const int j = q << 2;
                if (v.x < best) { best = v.x; bj = j; }
                if (v.y < best) { best = v.y; bj = j + 1; }
                if (v.z < best) { best = v.z; bj = j + 2; }
                if (v.w < best) { best = v.w; bj = j + 3; }
            }
        } else {
#pragma unroll 4
            for (int j = lane; j < J; j += 32) {
                const float v = __ldcs(row + DYN_IDX(j, J));
                if (v < best) { best = v; bj = j; }
            }
        }
        best += 0.f;                                       // -0 -> +0
        const uint32_t key = float_key(best);
        const uint32_t kmin = __reduce_min_sync(kFull, key);
        const uint32_t jmin = __reduce_min_sync(kFull, key == kmin ? uint32_t(bj) : 0xffffffffu);
        if (kmin != float_key(CUDART_INF_F)) {
            if (key == kmin && uint32_t(bj) == jmin) {
                best_idx[i] = bj;
                best_E[i] = best;
            }
        } else if (lane == 0) {
            best_idx[i] = -1;
            best_E[i] = CUDART_INF_F;
        }
    }
}

struct TotalsArgs {
    SelectOut o;
    int64_t S, W, chunks;
    int32_t C, J, T, F;
    const int32_t *nj, *tj, *tp;
    double *partial;
    uint32_t *partial_bad;
};

// One CTA per (scenario, chunk of kChunkWindows windows), one window per thread.
__global__ void __launch_bounds__(kThreads) totals_partial_kernel(const TotalsArgs a) {
    __shared__ double s_sum[kThreads];
    __shared__ uint32_t s_bad[kThreads];
    const int64_t s = blockIdx.x / a.chunks;
    const int64_t ch = blockIdx.x % a.chunks;
    const int64_t w = ch * kChunkWindows + threadIdx.x;
    const bool have = threadIdx.x < kChunkWindows && w < a.W;
    const int lane = threadIdx.x & 31;
    const int TF = a.T * a.F;
    const size_t base = size_t(s * a.W + (have ? w : 0)) * size_t(a.C);
    double ew = 0.0;
    uint32_t bad = 0, g = 0;
    for (int c = 0; c < a.C; ++c) {                 // every lane takes every trip: the match below is warp-wide
        int32_t j = -1;
        if (have) {
            j = a.o.best_idx[DYN_IDX(base + c, size_t(a.S) * a.W * a.C)];
            if (j < 0) ++bad;
            else ew += double(a.o.best_E[DYN_IDX(base + c, size_t(a.S) * a.W * a.C)]);
        }
        if (a.o.hist) {
            // neighbouring windows of a class often choose the same candidate: one atomic per distinct
            // candidate in the warp, by the lowest lane that holds it
            const unsigned peers = __match_any_sync(kFull, j);
            if (j >= 0 && lane == __ffs(peers) - 1)
                atomicAdd(&a.o.hist[size_t(s) * size_t(a.J) + size_t(DYN_IDX(j, a.J))], uint32_t(__popc(peers)));
        }
        if (a.o.gpus && j >= 0) {
            if (a.nj) g += uint32_t(a.nj[DYN_IDX(j, a.J)] * a.tj[DYN_IDX(j, a.J)]);
            else g += uint32_t((j / TF + 1) * a.tp[DYN_IDX((j / a.F) % a.T, a.T)]);
        }
    }
    if (have) {
        if (a.o.E_window) a.o.E_window[s * a.W + w] = ew;
        if (a.o.gpus) a.o.gpus[s * a.W + w] = g;
    }
    s_sum[threadIdx.x] = ew;
    s_bad[threadIdx.x] = bad;
    __syncthreads();
    for (int h = kThreads / 2; h > 0; h >>= 1) {
        if (threadIdx.x < h) {
            s_sum[threadIdx.x] += s_sum[threadIdx.x + h];
            s_bad[threadIdx.x] += s_bad[threadIdx.x + h];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        a.partial[blockIdx.x] = s_sum[0];
        a.partial_bad[blockIdx.x] = s_bad[0];
    }
}

__global__ void totals_final_kernel(const TotalsArgs a) {
    const int64_t s = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (s >= a.S) return;
    double sum = 0.0;
    uint32_t bad = 0;
    for (int64_t ch = 0; ch < a.chunks; ++ch) {
        sum += a.partial[DYN_IDX(s * a.chunks + ch, a.S * a.chunks)];
        bad += a.partial_bad[DYN_IDX(s * a.chunks + ch, a.S * a.chunks)];
    }
    a.o.E_total[s] = sum;
    a.o.n_infeasible[s] = bad;
}

}  // namespace

cudaError_t launch_select(const float *d_E, int64_t tiles, int32_t J, int32_t *best_idx, float *best_E,
                          cudaStream_t st) {
    if (tiles == 0) return cudaSuccess;
    int64_t grid = (tiles + kWarps - 1) / kWarps;
    const int64_t cap = int64_t(sm_count()) * 8;
    if (grid > cap) grid = cap;
    const bool vec = (J % 4 == 0) && (reinterpret_cast<uintptr_t>(d_E) & 15u) == 0;
    if (vec) select_kernel<true><<<int(grid), kThreads, 0, st>>>(d_E, tiles, J, best_idx, best_E);
    else select_kernel<false><<<int(grid), kThreads, 0, st>>>(d_E, tiles, J, best_idx, best_E);
    return cudaGetLastError();
}

cudaError_t launch_totals(const SelectOut &o, int64_t S, int64_t W, int32_t C, int32_t J, const int32_t *d_nj,
                          const int32_t *d_tj, int32_t T, int32_t F, const int32_t *d_tp, double *d_partial,
                          uint32_t *d_partial_bad, cudaStream_t st) {
    if (S == 0) return cudaSuccess;
    TotalsArgs a{};
    a.o = o;
    a.S = S; a.W = W; a.chunks = totals_chunks(W);
    a.C = C; a.J = J; a.T = T; a.F = F;
    a.nj = d_nj; a.tj = d_tj; a.tp = d_tp;
    a.partial = d_partial;
    a.partial_bad = d_partial_bad;
    cudaError_t e;
    if (o.hist) {
        e = cudaMemsetAsync(o.hist, 0, size_t(S) * size_t(J) * sizeof(uint32_t), st);
        if (e != cudaSuccess) return e;
    }
    if (a.chunks > 0) {
        totals_partial_kernel<<<unsigned(S * a.chunks), kThreads, 0, st>>>(a);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    totals_final_kernel<<<unsigned((S + 127) / 128), 128, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace dyn
