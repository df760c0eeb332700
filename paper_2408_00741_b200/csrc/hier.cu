// Hierarchical control [Sec. 4.2]: nodes per pool from the epoch's peak load (scale-out/in), sharding
// at the highest frequency within those GPUs (shard-up/down), frequency per window (scale-up/down).
// Same models and the same resolved tables as the joint sweep; each level is a small restricted search.
// When every TBT row is monotone in load (the resolve step's flags) and the threshold tables fit in shared
// memory, the sharding and frequency kernels evaluate candidates as the sweep's threshold path does (compare on
// the per-instance load, 8-byte lookup of the energy line in shared memory); otherwise from the general-path
// tables through L1.  Both variants are launched; each looks at the flags and only the selected one works.
#include "dyn_internal.cuh"
#include "eval_dev.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

__device__ __forceinline__ double lerp64(double a, double b, double w) { return (1.0 - w) * a + w * b; }

// ML of each class: the largest load one instance of (largest TP, highest candidate frequency) sustains
// within TTFT, TBT and capacity; TBT is piecewise linear in the utilisation, searched from the top.
__global__ void hier_max_load_kernel(const ResolveParams rp, double *__restrict__ ml) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= rp.C) return;
    const int t = rp.T - 1, q = rp.F - 1, M = rp.M;
    const int r = rp.row[q];
    const double w = double(rp.weight[q]);
    const size_t ct = (size_t(c) * rp.T + t) * rp.R;
    const float *tb0 = rp.d_tbt + (ct + r) * M, *tb1 = tb0 + M;
    const double ttft = lerp64(rp.d_ttft[ct + r], rp.d_ttft[ct + r + 1], w);
    const double cap = lerp64(rp.d_cap[ct + r], rp.d_cap[ct + r + 1], w);
    const double slo = double(rp.slo_tbt[c]);
    double out = 0.0;
    if (ttft <= double(rp.slo_ttft[c]) && cap > 0.0) {
        for (int m = M - 2; m >= 0; --m) {
            const double a = lerp64(tb0[m], tb1[m], w), b = lerp64(tb0[m + 1], tb1[m + 1], w);
            if (b <= slo) { out = double(m + 1) / double(M - 1) * cap; break; }
            if (a <= slo) { out = (double(m) + (slo - a) / (b - a)) / double(M - 1) * cap; break; }
        }
    }
    ml[c] = out;
}

struct HierArgs {
    const float4 *rows;      // [C][P][M+1]
    const float2 *pairc;     // [C][P]
    const float *slo;        // [C]
    const char *ws;          // scratch block (threshold tables at off_pair2 .. off_end)
    int32_t off_pair2, off_rows2, off_end;
    int32_t use_fast;        // the threshold tables fit in shared memory
    const double *ml;        // [C]
    const float *load;       // [S][W][C]
    int64_t S;
    int32_t W, K1, K2;       // W*C < 2^31: indices inside one scenario are 32-bit
    int32_t C, T, F, M, Nmax, e1, e2, space_budget;
    FastDiv divC, divE1, divE2, divT;
    int32_t tp[DYN_MAX_T];
    int32_t *nodes, *shard, *best_idx;
    float *best_E;
};


// true when every pair row has a load threshold (vlim is NaN for a row whose TBT decreases somewhere)
__device__ __forceinline__ bool rows_monotone(const HierArgs &a) {
    int bad = 0;
    for (int i = threadIdx.x; i < a.C * a.T * a.F; i += blockDim.x) bad |= isnan(__ldg(a.pairc + i).y) ? 1 : 0;
    return __syncthreads_or(bad) == 0;
}

// FAST kernels do the work iff the tables are monotone (and staged); the others iff not.  Returns false when
// this kernel has nothing to do; for FAST it also stages pair2 | rows2 into shared memory.
template <bool FAST>
__device__ __forceinline__ bool hier_begin(const HierArgs &a) {
    const bool mono = rows_monotone(a);
    if (FAST) {
        if (!mono) return false;
        extern __shared__ float4 smem[];
        const float4 *src = reinterpret_cast<const float4 *>(a.ws + a.off_pair2);
        const int n16 = (a.off_end - a.off_pair2) / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) smem[i] = src[i];
        __syncthreads();
        return true;
    }
    return !(a.use_fast && mono);
}

// pool energy of n instances of pair p (class c) at per-instance load ln; ok = within SLO and capacity
template <bool FAST>
__device__ __forceinline__ float hier_eval(const HierArgs &a, uint32_t origin, int c, int p, float ln, float nf, float slo,
                                           bool &ok) {
    const int P = a.T * a.F, RS = a.M + 1;
    if (FAST) {
        const float4 pc = load16<true>(a.ws, origin + uint32_t(c * P + p) * 16u);
        float e;
        fast_one<true>(a.ws, origin + uint32_t(a.off_rows2 - a.off_pair2) + uint32_t((c * P + p) * RS) * 8u, ln, pc.x, pc.z,
                       e, ok);
        return nf * e;
    }
    return eval_pair(a.rows + (size_t(c) * P + p) * RS, __ldg(&a.pairc[c * P + p]).x, float(a.M), ln, nf, slo, ok);
}


// Index of the (epoch or window, class) pair a thread serves among `n_items` epochs/windows.  The plain
// variants take x = item*C + c in thread order (neighbouring threads read neighbouring loads).  The
// staging variants give a warp ONE class and 32 consecutive items, so that the lanes of a lookup read the same
// few table rows in shared memory instead of rows of nine classes (bank conflicts); the strided loads and
// stores of the nine warps that share a block of items meet in L1 / L2.
template <bool FAST>
__device__ __forceinline__ bool hier_item(const HierArgs &a, uint32_t n_items, uint32_t &item, uint32_t &c) {
    const uint32_t y = blockIdx.x * blockDim.x + threadIdx.x;
    if (FAST) {
        const uint32_t g = y >> 5;
        const uint32_t blk = fastdiv(g, a.divC);
        c = g - blk * a.C;
        item = blk * 32u + (y & 31u);
        return item < n_items;
    }
    if (y >= n_items * uint32_t(a.C)) return false;
    item = fastdiv(y, a.divC);
    c = y - item * a.C;
    return true;
}

// grid: x over the (epoch or window, class) pairs of one scenario, y over scenarios (strided)

__global__ void __launch_bounds__(256) hier_nodes_kernel(const HierArgs a) {
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;              // k1 * C + c
    if (x >= uint32_t(a.K1 * a.C)) return;
    const uint32_t k1 = fastdiv(x, a.divC), c = x - k1 * a.C;
    const int w0 = int(k1) * a.e1, w1 = min(w0 + a.e1, a.W);
    const double ml = a.ml[c];
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const float *ld = a.load + size_t(s) * size_t(a.W) * a.C + c;
        float PL = 0.f;
        for (int w = w0; w < w1; ++w) PL = fmaxf(PL, ld[size_t(w) * a.C]);
        int nn = -1;
        if (ml > 0.0) {
            const double q = ceil(double(PL) / ml);
            nn = q < 1.0 ? 1 : (q > 1e9 ? 1000000000 : int(q));
        }
        a.nodes[size_t(s) * size_t(a.K1) * a.C + x] = nn;
    }
}

// one thread per (s, k2, c): neighbouring threads are neighbouring classes, so the loads coalesce; the
// node budget cuts the (n, TP) space to a few dozen candidates, walked in index order
template <bool FAST>
__global__ void __launch_bounds__(256) hier_shard_kernel(const HierArgs a) {
    if (!hier_begin<FAST>(a)) return;
    uint32_t origin = table_origin<FAST>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    uint32_t k2, c;
    if (!hier_item<FAST>(a, uint32_t(a.K2), k2, c)) return;
    const uint32_t x = k2 * a.C + c;
    const int w0 = int(k2) * a.e2, w1 = min(w0 + a.e2, a.W);
    const uint32_t k1 = fastdiv(uint32_t(w0), a.divE1);
    const float slo = a.slo[c];
    const int tpmax = a.tp[a.T - 1];
    const int cap_budget = a.Nmax * tpmax;            // a larger budget changes nothing
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const float *ld = a.load + size_t(s) * size_t(a.W) * a.C + c;
        float PL = 0.f;
        for (int w = w0; w < w1; ++w) PL = fmaxf(PL, ld[size_t(w) * a.C]);
        const int nn = a.nodes[size_t(s) * size_t(a.K1) * a.C + k1 * a.C + c];
        int budget = nn > 0 ? (nn > a.Nmax ? cap_budget : nn * tpmax) : 0;
        if (a.space_budget > 0 && budget > a.space_budget) budget = a.space_budget;
        int nmax = budget / a.tp[0];                  // no n above this fits even the smallest TP
        if (nmax > a.Nmax) nmax = a.Nmax;
        float best = CUDART_INF_F;
        int bnt = -1;
        if (FAST && a.T <= 4) {
            // the constants of the (at most four) highest-frequency pairs stay in registers for the whole walk
            float icm[4], llim[4];
            uint32_t row[4];
            int nlim[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int tt = t < a.T ? t : 0;
                const int p = tt * a.F + a.F - 1;
                const float4 pc = load16<true>(a.ws, origin + uint32_t(int(c) * a.T * a.F + p) * 16u);
                icm[t] = pc.x;
                llim[t] = t < a.T ? pc.z : -1.f;
                row[t] = origin + uint32_t(a.off_rows2 - a.off_pair2) + uint32_t((int(c) * a.T * a.F + p) * (a.M + 1)) * 8u;
                nlim[t] = t < a.T ? budget / a.tp[tt] : 0;  // TP ascending: the limits descend
            }
            for (int n = 1; n <= nmax; ++n) {
                const float nf = float(n), ln = PL * (1.0f / nf);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (n > nlim[t]) break;
                    float e;
                    bool ok;
                    fast_one<true>(a.ws, row[t], ln, icm[t], llim[t], e, ok);
                    const float E = nf * e;
                    if (ok && E < best) {             // ascending (n, t): strict compare keeps the lowest index
                        best = E;
                        bnt = (n - 1) * a.T + t;
                    }
                }
            }
        } else
        for (int n = 1; n <= nmax; ++n) {
            const float nf = float(n), ln = PL * (1.0f / nf);
            for (int t = 0; t < a.T; ++t) {
                if (n * a.tp[t] > budget) break;      // TP ascending
                const int p = t * a.F + a.F - 1;
                bool ok;
                const float E = hier_eval<FAST>(a, origin, int(c), p, ln, nf, slo, ok);
                if (ok && E < best) {                 // ascending (n, t): strict compare keeps the lowest index
                    best = E;
                    bnt = (n - 1) * a.T + t;
                }
            }
        }
        a.shard[size_t(s) * size_t(a.K2) * a.C + x] = bnt;
    }
}

// one thread per (s, w, c): the frequency for the sharding of its shard epoch
template <bool FAST>
__global__ void __launch_bounds__(256) hier_freq_kernel(const HierArgs a) {
    if (!hier_begin<FAST>(a)) return;
    uint32_t origin = table_origin<FAST>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    uint32_t w, c;
    if (!hier_item<FAST>(a, uint32_t(a.W), w, c)) return;
    const uint32_t x = w * a.C + c;
    const uint32_t k2 = fastdiv(w, a.divE2);
    const float slo = a.slo[c];
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const size_t i = size_t(s) * size_t(a.W) * a.C + x;
        const int nt = a.shard[size_t(s) * size_t(a.K2) * a.C + k2 * a.C + c];
        int32_t bj = -1;
        float best = CUDART_INF_F;
        if (nt >= 0) {
            const int n1 = int(fastdiv(uint32_t(nt), a.divT)), t = nt - n1 * a.T;
            const float nf = float(n1 + 1);
            const float ln = fmaxf(a.load[i], 0.f) * (1.0f / nf);
            for (int q = 0; q < a.F; ++q) {
                bool ok;
                const float E = hier_eval<FAST>(a, origin, int(c), t * a.F + q, ln, nf, slo, ok);
                if (ok && E < best) {
                    best = E;
                    bj = nt * a.F + q;
                }
            }
        }
        a.best_idx[i] = bj;
        a.best_E[i] = best;
    }
}

}  // namespace

cudaError_t launch_hier(const ResolveParams &rp, const ResolvedLayout &lay, void *d_ws, size_t off_ml, const float *d_load,
                        int64_t S, int64_t W, int32_t e1, int32_t e2, int32_t space_budget, int32_t *d_nodes,
                        int32_t *d_shard, int32_t *best_idx, float *best_E, cudaStream_t st) {
    char *ws = static_cast<char *>(d_ws);
    double *ml = reinterpret_cast<double *>(ws + off_ml);
    hier_max_load_kernel<<<(rp.C + 63) / 64, 64, 0, st>>>(rp, ml);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || S == 0 || W == 0) return e;
    HierArgs a{};
    a.rows = reinterpret_cast<const float4 *>(ws + lay.off_rows);
    a.pairc = reinterpret_cast<const float2 *>(ws + lay.off_pairc);
    a.slo = reinterpret_cast<const float *>(ws + lay.off_slo);
    a.ml = ml;
    a.load = d_load;
    a.S = S; a.W = int32_t(W); a.K1 = int32_t((W + e1 - 1) / e1); a.K2 = int32_t((W + e2 - 1) / e2);
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.M = lay.M; a.Nmax = lay.Nmax; a.e1 = e1; a.e2 = e2;
    a.space_budget = space_budget;
    a.divC = make_fastdiv(uint32_t(lay.C)); a.divE1 = make_fastdiv(uint32_t(e1));
    a.divE2 = make_fastdiv(uint32_t(e2)); a.divT = make_fastdiv(uint32_t(lay.T));
    for (int t = 0; t < lay.T; ++t) a.tp[t] = rp.tp[t];
    a.nodes = d_nodes; a.shard = d_shard; a.best_idx = best_idx; a.best_E = best_E;
    const unsigned gy = unsigned(S < 32768 ? S : 32768);
    const int64_t n1 = int64_t(a.K1) * lay.C, n2 = int64_t(a.K2) * lay.C, n3 = W * lay.C;
    a.ws = ws;
    a.off_pair2 = int32_t(lay.off_pair2); a.off_rows2 = int32_t(lay.off_rows2); a.off_end = int32_t(lay.off_tp);
    const size_t fast_bytes = lay.off_tp - lay.off_pair2;
    a.use_fast = fast_bytes <= 96 * 1024 ? 1 : 0;
    // the staging variants run about eight CTAs per SM, each walking many scenarios, so that the tables are
    // staged a few thousand times per call rather than once per 256 tiles
    auto few = [&](int64_t blocks_x) {
        int64_t g = (int64_t(sm_count()) * 8 + blocks_x - 1) / blocks_x;
        return unsigned(g < 1 ? 1 : (g > int64_t(gy) ? int64_t(gy) : g));
    };
    if (a.use_fast) {
        if ((e = cudaFuncSetAttribute(hier_shard_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(fast_bytes))) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(hier_freq_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(fast_bytes))) != cudaSuccess) return e;
    }
    hier_nodes_kernel<<<dim3(unsigned((n1 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // staging variants: a warp per (32 items, class)
    const int64_t f2 = ((int64_t(a.K2) + 31) / 32 * lay.C * 32 + 255) / 256, f3 = ((W + 31) / 32 * lay.C * 32 + 255) / 256;
    if (a.use_fast) {
        hier_shard_kernel<true><<<dim3(unsigned(f2), few(f2)), 256, fast_bytes, st>>>(a);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    hier_shard_kernel<false><<<dim3(unsigned((n2 + 255) / 256), a.use_fast ? few((n2 + 255) / 256) : gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    if (a.use_fast) {
        hier_freq_kernel<true><<<dim3(unsigned(f3), few(f3)), 256, fast_bytes, st>>>(a);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    hier_freq_kernel<false><<<dim3(unsigned((n3 + 255) / 256), a.use_fast ? few((n3 + 255) / 256) : gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
