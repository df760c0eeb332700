// Pools that mix tensor parallelisms [Sec. 4.1, Eq. 1 in full]: counts N^{TP_i} per parallelism under the GPU
// budget sum_i TP_i*N^{TP_i} <= N, one frequency per parallelism, the load shared out over the groups, the
// objective sum_i N^{TP_i} * Energy^{TP_i, f_i}(L^{TP_i}).  The paper gives this to a solver; here the count
// tuples are enumerated: the host lists the tuples within the budget (odometer order, smallest TP fastest),
// a warp takes a tile, its lanes take every 32nd tuple.  For a tuple the load is split in proportion to the
// groups' capacity at the highest candidate frequency, each group then picks its own feasible frequency of
// least energy (the single-type evaluation at fixed n and TP), and the tuple's energy is the sum.  The warp
// keeps the tuple of least energy, lowest tuple number on ties.
//
// Work per tile is (tuples) x (TP degrees in use) x F single-type evaluations on the general-path tables,
// read through L1 (they are a few tens of KB); the loads and results are 4 + 12 + 8T bytes per tile.
#include "dyn_internal.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;

struct MixedArgs {
    const float4 *rows;       // [C][P][M+1]
    const float2 *pairc;      // [C][P]
    const float *slo;         // [C]
    float *caph;              // [C][T] capacity at the highest candidate frequency
    const uint32_t *tuples;   // [K]
    const float *load;        // [tiles]
    int64_t tiles, K;
    int32_t C, T, F, M;
    int32_t *counts, *freq, *tuple;
    float *best_E;
};

// capacity at the highest candidate frequency, from the resolved pair constant ic = (M-1)/(M*cap)
__global__ void mixed_caph_kernel(const MixedArgs a) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.C * a.T) return;
    const int c = i / a.T, t = i - c * a.T;
    const float ic = a.pairc[c * (a.T * a.F) + t * a.F + a.F - 1].x;
    a.caph[i] = ic > 0.f ? float(double(a.M - 1) / (double(a.M) * double(ic))) : 0.f;
}

template <int T>
__global__ void __launch_bounds__(kThreads) mixed_select_kernel(const MixedArgs a) {
    const int lane = threadIdx.x & 31;
    const int P = T * a.F, RS = a.M + 1;
    const float Mf = float(a.M);
    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t i = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); i < a.tiles; i += nwarps) {
        const int c = int(i % a.C);
        const float L = fmaxf(a.load[i], 0.f);              // negative / NaN -> 0
        const float slo = a.slo[c];
        float caph[T];
#pragma unroll
        for (int t = 0; t < T; ++t) caph[t] = a.caph[c * T + t];
        float best = CUDART_INF_F;
        int64_t bk = a.K;                                    // tuple number of the lane's best
        uint32_t bq = 0;                                     // its frequencies, 8 bits per TP index
        for (int64_t k = lane; k < a.K; k += 32) {
            const uint32_t tup = __ldg(a.tuples + k);
            float A = 0.f;
#pragma unroll
            for (int t = 0; t < T; ++t) A = fmaf(float((tup >> (8 * t)) & 255u), caph[t], A);
            const float frac = L / A;                        // every instance at this fraction of its top-frequency capacity
            float E = 0.f;
            uint32_t qs = 0;
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const uint32_t n = (tup >> (8 * t)) & 255u;
                if (n == 0) continue;
                const float l = frac * caph[t], nf = float(n);
                const float4 *rows_t = a.rows + (size_t(c) * P + t * a.F) * RS;
                const float2 *pc_t = a.pairc + c * P + t * a.F;
                float eg = CUDART_INF_F;
                uint32_t qg = 0;
                for (int q = 0; q < a.F; ++q) {
                    bool ok;
                    const float e = eval_pair(rows_t + size_t(q) * RS, __ldg(pc_t + q).x, Mf, l, nf, slo, ok);
                    if (ok && e < eg) {                      // ascending q: strict compare keeps the lowest
                        eg = e;
                        qg = uint32_t(q);
                    }
                }
                E += eg;                                     // ascending TP index; +inf if the group has no frequency
                qs |= qg << (8 * t);
            }
            if (E < best) {                                  // ascending tuple number per lane
                best = E;
                bk = k;
                bq = qs;
            }
        }
        best += 0.f;                                         // -0 -> +0
        float Emin;
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(Emin) : "f"(best));
        // lowest tuple number among the lanes that hold the minimum (numbers fit 32 bits: K <= 2^20)
        const uint32_t kmin = __reduce_min_sync(kFull, best == Emin ? uint32_t(bk) : 0xffffffffu);
        if (Emin == CUDART_INF_F) {
            if (lane < T) {
                a.counts[i * T + lane] = -1;
                a.freq[i * T + lane] = -1;
            }
            if (lane == 0) {
                a.tuple[i] = -1;
                a.best_E[i] = CUDART_INF_F;
            }
            continue;
        }
        if (best == Emin && uint32_t(bk) == kmin) {          // exactly one lane: tuple numbers are distinct
            const uint32_t tup = __ldg(a.tuples + bk);
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const uint32_t n = (tup >> (8 * t)) & 255u;
                a.counts[i * T + t] = int32_t(n);
                a.freq[i * T + t] = n ? int32_t((bq >> (8 * t)) & 255u) : -1;
            }
            a.tuple[i] = int32_t(kmin);
            a.best_E[i] = Emin;
        }
    }
}

}  // namespace

cudaError_t launch_mixed(const ResolvedLayout &lay, void *d_ws, size_t off_tuples, size_t off_caph, int64_t K,
                         const float *d_load, int64_t tiles, int32_t *d_counts, int32_t *d_freq, int32_t *d_tuple,
                         float *d_best_E, cudaStream_t st) {
    char *ws = static_cast<char *>(d_ws);
    MixedArgs a{};
    a.rows = reinterpret_cast<const float4 *>(ws + lay.off_rows);
    a.pairc = reinterpret_cast<const float2 *>(ws + lay.off_pairc);
    a.slo = reinterpret_cast<const float *>(ws + lay.off_slo);
    a.caph = reinterpret_cast<float *>(ws + off_caph);
    a.tuples = reinterpret_cast<const uint32_t *>(ws + off_tuples);
    a.load = d_load;
    a.tiles = tiles; a.K = K;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.M = lay.M;
    a.counts = d_counts; a.freq = d_freq; a.tuple = d_tuple; a.best_E = d_best_E;
    mixed_caph_kernel<<<(lay.C * lay.T + 127) / 128, 128, 0, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || tiles == 0) return e;
    int64_t grid = (tiles + kWarps - 1) / kWarps;
    const int64_t cap = int64_t(sm_count()) * 8;
    if (grid > cap) grid = cap;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    switch (lay.T) {
        case 1: mixed_select_kernel<1><<<int(grid), kThreads, 0, st>>>(a); break;
        case 2: mixed_select_kernel<2><<<int(grid), kThreads, 0, st>>>(a); break;
        case 3: mixed_select_kernel<3><<<int(grid), kThreads, 0, st>>>(a); break;
        case 4: mixed_select_kernel<4><<<int(grid), kThreads, 0, st>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
