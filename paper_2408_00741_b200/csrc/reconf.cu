// Selection that counts the cost of re-configuring [Sec. 4.2 "Accounting for the overheads": the controllers set
// the energy a new configuration saves against the cost of the transition, read from an Overhead Table; Sec. 4.3:
// re-sharding costs depend on source and destination parallelism, frequency changes cost next to nothing].
//
// Per (scenario, class) this is a shortest path through the windows: a state is a sharding sigma = (n, TP),
// the cost of a state in a window is the least energy over the candidate frequencies (the evaluation of Eq. 1),
// a move sigma' -> sigma between consecutive windows costs R[sigma'][sigma] (the caller's table, Wh).
//   reconf_cost_kernel  cost[s][c][w][sigma] and the frequency that attains it: one thread per entry, a warp
//                       covers 32 shardings of one tile (one load, the table rows of T degrees), F evaluations each
//   reconf_path_kernel  one CTA per (scenario, class): forward recursion over the windows, a thread per target
//                       state scanning all source states (min-plus product of the state vector with R, R read
//                       through L1, the state vector in shared memory), back pointers to global memory; then the
//                       walk back, 32 windows of pointers staged per step.  The running values are kept relative
//                       to their minimum, which is accumulated in fp64, so that fp32 holds only differences.
#include "dyn_internal.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kBack = 32;                       // windows of back pointers staged per step of the walk back

struct ReconfArgs {
    const float4 *rows;       // [C][P][M+1]
    const float2 *pairc;      // [C][P]
    const float *slo;         // [C]
    const int32_t *tp;        // [T]
    const float *R;           // [NS][NS]
    const float *load;        // [S][W][C]
    float *cost;              // [S][C][W][NS]
    uint8_t *qbest;           // [S][C][W][NS]
    uint16_t *from;           // [S][C][W][NS]
    int64_t S, W;
    int32_t C, T, F, M, Nmax, NS, budget;
    int32_t *best_idx;
    float *best_E;
    double *path_total;       // [S][C]
};

__global__ void __launch_bounds__(kThreads) reconf_cost_kernel(const ReconfArgs a) {
    const int64_t total = a.S * a.C * a.W * a.NS;
    const int P = a.T * a.F, RS = a.M + 1;
    const float Mf = float(a.M);
    for (int64_t e = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; e < total; e += int64_t(gridDim.x) * blockDim.x) {
        const int g = int(e % a.NS);
        const int64_t scw = e / a.NS;
        const int64_t w = scw % a.W;
        const int64_t sc = scw / a.W;
        const int c = int(sc % a.C);
        const int64_t s = sc / a.C;
        const int n = g / a.T + 1, t = g - (n - 1) * a.T;
        const float L = fmaxf(a.load[(s * a.W + w) * a.C + c], 0.f);
        const float nf = float(n), ln = L * (1.0f / nf);
        const float slo = a.slo[c];
        float best = CUDART_INF_F;
        int bq = 0;
        if (a.budget <= 0 || int64_t(n) * a.tp[t] <= int64_t(a.budget)) {
            const float4 *rows_t = a.rows + (size_t(c) * P + t * a.F) * RS;
            const float2 *pc_t = a.pairc + c * P + t * a.F;
            for (int q = 0; q < a.F; ++q) {
                bool ok;
                const float E = eval_pair(rows_t + size_t(q) * RS, __ldg(pc_t + q).x, Mf, ln, nf, slo, ok);
                if (ok && E < best) {                        // ascending q: strict compare keeps the lowest
                    best = E;
                    bq = q;
                }
            }
        }
        a.cost[e] = best;
        a.qbest[e] = uint8_t(bq);
    }
}

// block-wide minimum of v (all threads get it); `red` holds kThreads / 32 floats
__device__ __forceinline__ float block_min(float v, float *red) {
    float m;
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
    __syncthreads();                                         // `red` may still be read from the previous call
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int i = 1; i < kThreads / 32; ++i) r = fminf(r, red[i]);
    return r;
}

// dynamic shared memory: D[2][NS] floats | back[kBack][NS] uint16 | path[kBack] int32
__global__ void __launch_bounds__(kThreads) reconf_path_kernel(const ReconfArgs a) {
    extern __shared__ float4 smem4[];
    __shared__ float red[kThreads / 32];
    __shared__ int s_last;
    const int NS = a.NS;
    float *D0 = reinterpret_cast<float *>(smem4), *D1 = D0 + NS;
    uint16_t *back = reinterpret_cast<uint16_t *>(D1 + NS);
    int32_t *path = reinterpret_cast<int32_t *>(back + size_t(kBack) * NS);
    const int64_t sc = blockIdx.x;                           // s * C + c
    const int c = int(sc % a.C);
    const int64_t s = sc / a.C;
    const int64_t W = a.W;
    const float *cost = a.cost + sc * W * NS;
    uint16_t *from = a.from + sc * W * NS;
    const int tid = threadIdx.x;

    // forward: D_w(g) = cost_w(g) + min_h (D_{w-1}(h) + R[h][g]), lowest h on ties; values relative to `base`
    double base = 0.0;
    float *Dp = D0, *Dn = D1;
    float lmin = CUDART_INF_F;
    for (int g = tid; g < NS; g += kThreads) {
        const float v = W > 0 ? cost[g] : 0.f;
        Dp[g] = v;
        lmin = fminf(lmin, v);
    }
    float m = block_min(lmin, red);                          // also orders the writes of Dp before the reads below
    for (int64_t w = 1; w < W; ++w) {
        // renormalise: keep differences only (the minimum goes to the fp64 base); all +inf stays +inf
        const float shift = (m < CUDART_INF_F) ? m : 0.f;
        base += double(shift);
        lmin = CUDART_INF_F;
        for (int g = tid; g < NS; g += kThreads) {
            float best = CUDART_INF_F;
            int arg = 0;
            const float *Rg = a.R + g;
#pragma unroll 8
            for (int h = 0; h < NS; ++h) {
                const float v = (Dp[h] - shift) + __ldg(Rg + size_t(h) * NS);
                if (v < best) {
                    best = v;
                    arg = h;
                }
            }
            const float d = cost[w * NS + g] + best;
            Dn[g] = d;
            from[w * NS + g] = uint16_t(arg);
            lmin = fminf(lmin, d);
        }
        m = block_min(lmin, red);                            // its barriers separate this window's writes from the next reads
        float *tmp = Dp; Dp = Dn; Dn = tmp;
    }
    // last state: lowest g attaining the minimum
    if (tid == 0) {
        int last = -1;
        if (m < CUDART_INF_F && W > 0)
            for (int g = 0; g < NS; ++g)
                if (Dp[g] == m) { last = g; break; }
        s_last = last;
        a.path_total[sc] = W > 0 ? ((m < CUDART_INF_F) ? base + double(m) : double(CUDART_INF_F)) : 0.0;
    }
    __syncthreads();
    int cur = s_last;
    // walk back, kBack windows per step: stage their back pointers, one thread follows them, all write results
    for (int64_t hi = W; hi > 0; hi -= kBack) {
        const int64_t lo = hi > kBack ? hi - kBack : 0;
        const int nw = int(hi - lo);
        if (cur >= 0) {
            for (int i = tid; i < nw * NS; i += kThreads) back[i] = from[lo * NS + i];
        }
        __syncthreads();
        if (tid == 0) {
            int g = cur;
            for (int k = nw - 1; k >= 0; --k) {
                path[k] = g;
                if (g >= 0 && lo + k > 0) g = back[k * NS + g];       // pointer of window lo+k leads to window lo+k-1
            }
            s_last = g;
        }
        __syncthreads();
        for (int k = tid; k < nw; k += kThreads) {
            const int g = path[k];
            const int64_t w = lo + k;
            const int64_t i = (s * W + w) * a.C + c;
            if (g >= 0) {
                a.best_idx[i] = g * a.F + int(a.qbest[sc * W * NS + w * NS + g]);
                a.best_E[i] = cost[w * NS + g];
            } else {
                a.best_idx[i] = -1;
                a.best_E[i] = CUDART_INF_F;
            }
        }
        cur = s_last;
        __syncthreads();
    }
}

}  // namespace

size_t reconf_smem_bytes(int32_t NS) {
    return size_t(2) * NS * sizeof(float) + size_t(kBack) * NS * sizeof(uint16_t) + size_t(kBack) * sizeof(int32_t) + 16;
}

cudaError_t launch_reconf(const ResolvedLayout &lay, void *d_ws, size_t off_cost, size_t off_q, size_t off_from,
                          const float *d_R, const float *d_load, int64_t S, int64_t W, int32_t budget, int32_t *best_idx,
                          float *best_E, double *path_total, cudaStream_t st) {
    char *ws = static_cast<char *>(d_ws);
    ReconfArgs a{};
    a.rows = reinterpret_cast<const float4 *>(ws + lay.off_rows);
    a.pairc = reinterpret_cast<const float2 *>(ws + lay.off_pairc);
    a.slo = reinterpret_cast<const float *>(ws + lay.off_slo);
    a.tp = reinterpret_cast<const int32_t *>(ws + lay.off_tp);
    a.R = d_R; a.load = d_load;
    a.cost = reinterpret_cast<float *>(ws + off_cost);
    a.qbest = reinterpret_cast<uint8_t *>(ws + off_q);
    a.from = reinterpret_cast<uint16_t *>(ws + off_from);
    a.S = S; a.W = W;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.M = lay.M; a.Nmax = lay.Nmax; a.NS = lay.Nmax * lay.T; a.budget = budget;
    a.best_idx = best_idx; a.best_E = best_E; a.path_total = path_total;
    if (S == 0) return cudaSuccess;
    const int64_t total = S * lay.C * W * a.NS;
    if (total > 0) {
        int64_t grid = (total + kThreads - 1) / kThreads;
        const int64_t cap = int64_t(sm_count()) * 16;
        if (grid > cap) grid = cap;
        reconf_cost_kernel<<<unsigned(grid), kThreads, 0, st>>>(a);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const size_t smem = reconf_smem_bytes(a.NS);
    cudaError_t e = cudaFuncSetAttribute(reconf_path_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    reconf_path_kernel<<<unsigned(S * lay.C), kThreads, smem, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
