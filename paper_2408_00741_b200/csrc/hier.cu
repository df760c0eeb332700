// Hierarchical control [Sec. 4.2]: nodes per pool from the epoch's peak load (scale-out/in), sharding
// at the highest frequency within those GPUs (shard-up/down), frequency per window (scale-up/down).
// Same models and the same resolved tables as the joint sweep; each level is a small restricted search,
// so these kernels are bound by reading the load matrix, not by arithmetic.
#include "dyn_internal.cuh"

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
__global__ void __launch_bounds__(256) hier_shard_kernel(const HierArgs a) {
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;              // k2 * C + c
    if (x >= uint32_t(a.K2 * a.C)) return;
    const uint32_t k2 = fastdiv(x, a.divC), c = x - k2 * a.C;
    const int w0 = int(k2) * a.e2, w1 = min(w0 + a.e2, a.W);
    const uint32_t k1 = fastdiv(uint32_t(w0), a.divE1);
    const int P = a.T * a.F, RS = a.M + 1;
    const float Mf = float(a.M), slo = a.slo[c];
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
        for (int n = 1; n <= nmax; ++n) {
            const float nf = float(n), ln = PL * (1.0f / nf);
            for (int t = 0; t < a.T; ++t) {
                if (n * a.tp[t] > budget) break;      // TP ascending
                const int p = t * a.F + a.F - 1;
                bool ok;
                const float E = eval_pair(a.rows + (size_t(c) * P + p) * RS, __ldg(&a.pairc[c * P + p]).x, Mf, ln, nf, slo, ok);
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
__global__ void __launch_bounds__(256) hier_freq_kernel(const HierArgs a) {
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;              // w * C + c
    if (x >= uint32_t(a.W * a.C)) return;
    const uint32_t w = fastdiv(x, a.divC), c = x - w * a.C;
    const uint32_t k2 = fastdiv(w, a.divE2);
    const int P = a.T * a.F, RS = a.M + 1;
    const float Mf = float(a.M), slo = a.slo[c];
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const size_t i = size_t(s) * size_t(a.W) * a.C + x;
        const int nt = a.shard[size_t(s) * size_t(a.K2) * a.C + k2 * a.C + c];
        int32_t bj = -1;
        float best = CUDART_INF_F;
        if (nt >= 0) {
            const int n1 = int(fastdiv(uint32_t(nt), a.divT)), t = nt - n1 * a.T;
            const float nf = float(n1 + 1);
            const float ln = fmaxf(a.load[i], 0.f) * (1.0f / nf);
            const float4 *rows_t = a.rows + (size_t(c) * P + t * a.F) * RS;
            const float2 *pc_t = a.pairc + c * P + t * a.F;
            for (int q = 0; q < a.F; ++q) {
                bool ok;
                const float E = eval_pair(rows_t + size_t(q) * RS, __ldg(pc_t + q).x, Mf, ln, nf, slo, ok);
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
    hier_nodes_kernel<<<dim3(unsigned((n1 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    hier_shard_kernel<<<dim3(unsigned((n2 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    hier_freq_kernel<<<dim3(unsigned((n3 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
