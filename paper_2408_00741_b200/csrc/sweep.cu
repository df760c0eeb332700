// Stage (b) and fused (b)+(c): evaluate every candidate (n instances, TP, f) of every (window, class)
// tile against the latency/power profile and the SLOs [Sec. 4.1, Eq. 1], and keep the
// minimum-energy feasible one [Sec. 4.2].
//
// Work is plain fp32 arithmetic (no dense contraction, so no tensor cores).  A warp owns one tile at
// a time: lanes hold instance counts n (several per lane when Nmax > 32), the (TP, f) pairs are the
// inner loop, so the per-pair constants and the table row are warp-uniform and the per-lane work is
// one multiply, one table lookup indexed by floor(x), two fused multiply-adds, the feasibility
// compares and the running minimum.  floor(x) comes from adding 2^23 with round-toward-zero: the low
// mantissa bits are the segment number, and subtracting 2^23 gives it back as a float, so no
// float-to-int conversion is issued.  The resolved tables of all classes are staged in shared memory
// once per CTA when they fit; larger tables are read through L1.
#include "dyn_internal.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kTwo23 = 8388608.0f;

struct SweepArgs {
    const float4 *rows;      // [C][P][M]
    const float *icm;        // [C][P]
    const float *slo;        // [C]
    const int32_t *tp;       // [T]
    const float *load;       // [tiles]
    int64_t tiles;
    int32_t C, T, F, P, M, Nmax, J;
    int32_t budget;          // <= 0: none
    int32_t ln_log2;         // lanes per n-group = 1 << ln_log2
    int64_t tiles_per_warp;
    size_t stage_bytes;      // bytes of [rows | icm | slo] staged in shared memory (0: read from global)
    size_t off_icm, off_slo; // offsets of icm / slo inside the staged block
};

// order-preserving map float -> uint32 (smaller float <=> smaller key), and back
__device__ __forceinline__ uint32_t float_key(float v) {
    const uint32_t b = __float_as_uint(v);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}

// one candidate: x = u*(M-1); returns energy of the whole pool (n instances) and its feasibility
__device__ __forceinline__ void eval_one(const float4 *__restrict__ row, float x, float mm1, float slo, float nf,
                                         float &E, bool &ok) {
    const float xc = fminf(x, mm1);                       // NaN/inf -> last entry: a safe address
    const float y = __fadd_rz(xc, kTwo23);                // 2^23 + floor(xc), exactly
    const int m = __float_as_int(y) - 0x4b000000;
    const float nu = xc - (y - kTwo23);
    const float4 e = row[m];
    const float tbt = fmaf(nu, e.y, e.x);
    const float ew = fmaf(nu, e.w, e.z);
    ok = (x <= mm1) && (tbt <= slo);                      // u <= 1 and TBT within its SLO
    E = nf * ew;
}

// ---------------------------------------------------------------------------------------------
// fused evaluate + select
// ---------------------------------------------------------------------------------------------
template <int NPL, bool BUDGET, bool SMEM>
__global__ void __launch_bounds__(kThreads)
eval_select_kernel(const SweepArgs a, int32_t *__restrict__ best_idx, float *__restrict__ best_E) {
    extern __shared__ float4 smem[];
    const float4 *rows = a.rows;
    const float *icm = a.icm;
    const float *slo = a.slo;
    if (SMEM) {
        // the staged block has the layout of the scratch block: rows, then icm, then slo
        const float4 *src = a.rows;
        const int n16 = int(a.stage_bytes / 16);
        for (int i = threadIdx.x; i < n16; i += kThreads) smem[i] = src[i];
        __syncthreads();
        rows = smem;
        icm = reinterpret_cast<const float *>(reinterpret_cast<const char *>(smem) + a.off_icm);
        slo = reinterpret_cast<const float *>(reinterpret_cast<const char *>(smem) + a.off_slo);
    }

    const int lane = threadIdx.x & 31;
    const int64_t gwarp = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const int LN = 1 << a.ln_log2;
    const int G = 32 >> a.ln_log2;                  // pair groups inside the warp
    const int nl = lane & (LN - 1);
    const int g = lane >> a.ln_log2;
    const int P = a.P, M = a.M;
    const float mm1 = float(M - 1);

    float nf[NPL], rn[NPL];
    int pmax[NPL];
#pragma unroll
    for (int k = 0; k < NPL; ++k) {
        const int n = nl + 1 + LN * k;
        nf[k] = float(n);
        rn[k] = n <= a.Nmax ? 1.0f / float(n) : CUDART_INF_F;     // n beyond Nmax: never feasible
        pmax[k] = P;
        if (BUDGET) {
            int nt = 0;
            for (int t = 0; t < a.T; ++t) nt += (int64_t(n) * a.tp[t] <= int64_t(a.budget)) ? 1 : 0;
            pmax[k] = nt * a.F;                      // TP ascending: allowed pairs are a prefix
        }
    }

    int64_t i = gwarp * a.tiles_per_warp;
    int64_t i_end = i + a.tiles_per_warp;
    if (i_end > a.tiles) i_end = a.tiles;
    if (i >= i_end) return;
    int c = int(i % a.C);

    for (; i < i_end; ++i) {
        const float L = fmaxf(a.load[i], 0.f);      // negative or NaN load counts as zero
        const float4 *crow = rows + size_t(c) * P * M;
        const float *cicm = icm + size_t(c) * P;
        const float slo_c = slo[c];
        float Ln[NPL], best[NPL];
        int bp[NPL];
#pragma unroll
        for (int k = 0; k < NPL; ++k) {
            Ln[k] = L * rn[k];
            best[k] = CUDART_INF_F;
            bp[k] = 0;
        }
#pragma unroll 4
        for (int p = g; p < P; p += G) {
            const float ic = cicm[p];
            const float4 *row = crow + size_t(p) * M;
#pragma unroll
            for (int k = 0; k < NPL; ++k) {
                float E;
                bool ok;
                eval_one(row, Ln[k] * ic, mm1, slo_c, nf[k], E, ok);
                if (BUDGET) ok = ok && (p < pmax[k]);
                if (ok && E < best[k]) {            // strict: keeps the lowest pair index on ties
                    best[k] = E;
                    bp[k] = p;
                }
            }
        }
        // the lane's chains in ascending n: strict compare keeps the lower n on ties
        float E = best[0] + 0.f;                    // -0 -> +0 so that keys order like floats
        int j = nl * P + bp[0];
#pragma unroll
        for (int k = 1; k < NPL; ++k) {
            const float Ek = best[k] + 0.f;
            if (Ek < E) {
                E = Ek;
                j = (nl + LN * k) * P + bp[k];
            }
        }
        // warp argmin on (E, j): smallest energy, then smallest index
        const uint32_t key = float_key(E);
        const uint32_t kmin = __reduce_min_sync(kFull, key);
        const uint32_t jmin = __reduce_min_sync(kFull, key == kmin ? uint32_t(j) : 0xffffffffu);
        if (kmin != float_key(CUDART_INF_F)) {
            if (key == kmin && uint32_t(j) == jmin) {           // exactly one lane: j is unique per lane
                best_idx[i] = j;
                best_E[i] = E;
            }
        } else if (lane == 0) {                                 // no feasible candidate
            best_idx[i] = -1;
            best_E[i] = CUDART_INF_F;
        }
        if (++c == a.C) c = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// evaluate only: E[tile][j]
// ---------------------------------------------------------------------------------------------
template <bool SMEM>
__global__ void __launch_bounds__(kThreads)
eval_configs_kernel(const SweepArgs a, const FastDiv divP, float *__restrict__ E_out) {
    extern __shared__ float4 smem[];
    const float4 *rows = a.rows;
    const float *icm = a.icm;
    const float *slo = a.slo;
    if (SMEM) {
        const float4 *src = a.rows;
        const int n16 = int(a.stage_bytes / 16);
        for (int i = threadIdx.x; i < n16; i += kThreads) smem[i] = src[i];
        __syncthreads();
        rows = smem;
        icm = reinterpret_cast<const float *>(reinterpret_cast<const char *>(smem) + a.off_icm);
        slo = reinterpret_cast<const float *>(reinterpret_cast<const char *>(smem) + a.off_slo);
    }
    const int P = a.P, M = a.M, J = a.J;
    const float mm1 = float(M - 1);
    // a CTA takes whole tiles; threads stride over j so that the row of E is written coalesced
    for (int64_t i = blockIdx.x; i < a.tiles; i += gridDim.x) {
        const int c = int(i % a.C);
        const float L = fmaxf(a.load[i], 0.f);
        const float4 *crow = rows + size_t(c) * P * M;
        const float *cicm = icm + size_t(c) * P;
        const float slo_c = slo[c];
        float *out = E_out + size_t(i) * size_t(J);
        for (int j = threadIdx.x; j < J; j += kThreads) {
            const int n1 = int(fastdiv(uint32_t(j), divP));      // n - 1
            const int p = j - n1 * P;
            const float nf = float(n1 + 1);
            float E;
            bool ok;
            eval_one(crow + size_t(p) * M, (L / nf) * cicm[p], mm1, slo_c, nf, E, ok);
            if (a.budget > 0) {
                const int t = p / a.F;
                ok = ok && (int64_t(n1 + 1) * a.tp[t] <= int64_t(a.budget));
            }
            out[j] = ok ? E : CUDART_INF_F;
        }
    }
}

size_t smem_limit() {
    static size_t lim = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return size_t(48 * 1024);
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return size_t(48 * 1024);
        return size_t(v);
    }();
    return lim;
}

SweepArgs make_args(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles, int32_t budget) {
    const char *ws = static_cast<const char *>(d_ws);
    SweepArgs a{};
    a.rows = reinterpret_cast<const float4 *>(ws + lay.off_rows);
    a.icm = reinterpret_cast<const float *>(ws + lay.off_icm);
    a.slo = reinterpret_cast<const float *>(ws + lay.off_slo);
    a.tp = reinterpret_cast<const int32_t *>(ws + lay.off_tp);
    a.load = d_load;
    a.tiles = tiles;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.P = lay.P; a.M = lay.M; a.Nmax = lay.Nmax; a.J = lay.J;
    a.budget = budget;
    // rows, icm and slo are consecutive in the scratch block: stage them as one piece when it fits
    const size_t block = lay.off_tp - lay.off_rows;
    a.stage_bytes = block <= 96 * 1024 && block <= smem_limit() ? block : 0;
    a.off_icm = lay.off_icm - lay.off_rows;
    a.off_slo = lay.off_slo - lay.off_rows;
    return a;
}

template <int NPL>
cudaError_t launch_es(const SweepArgs &a, int grid, int32_t *best_idx, float *best_E, cudaStream_t st) {
    const bool smem = a.stage_bytes > 0;
    const bool budget = a.budget > 0;
    cudaError_t e = cudaSuccess;
#define DYN_LAUNCH_ES(B, S)                                                                                       \
    do {                                                                                                          \
        if (S) e = cudaFuncSetAttribute(eval_select_kernel<NPL, B, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                        int(a.stage_bytes));                                                      \
        if (e == cudaSuccess) {                                                                                   \
            eval_select_kernel<NPL, B, S><<<grid, kThreads, S ? a.stage_bytes : 0, st>>>(a, best_idx, best_E);    \
            e = cudaGetLastError();                                                                               \
        }                                                                                                         \
    } while (0)
    if (budget && smem) DYN_LAUNCH_ES(true, true);
    else if (budget) DYN_LAUNCH_ES(true, false);
    else if (smem) DYN_LAUNCH_ES(false, true);
    else DYN_LAUNCH_ES(false, false);
#undef DYN_LAUNCH_ES
    return e;
}

}  // namespace

cudaError_t launch_eval_select(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                               int32_t gpu_budget, int32_t *best_idx, float *best_E, cudaStream_t st) {
    if (tiles == 0) return cudaSuccess;
    SweepArgs a = make_args(lay, d_ws, d_load, tiles, gpu_budget);
    // lanes per n-group: smallest power of two covering Nmax, at most 32
    int ln = 0;
    while ((1 << ln) < lay.Nmax && ln < 5) ++ln;
    a.ln_log2 = ln;
    const int npl = (lay.Nmax + 31) / 32;           // instance counts per lane
    // resident CTAs: 4 per SM; each warp takes a contiguous run of tiles
    int64_t grid = int64_t(sm_count()) * 4;
    const int64_t need = (tiles + kWarps - 1) / kWarps;
    if (grid > need) grid = need;
    a.tiles_per_warp = (tiles + grid * kWarps - 1) / (grid * kWarps);
    grid = (tiles + a.tiles_per_warp * kWarps - 1) / (a.tiles_per_warp * kWarps);
    if (npl <= 1) return launch_es<1>(a, int(grid), best_idx, best_E, st);
    if (npl <= 2) return launch_es<2>(a, int(grid), best_idx, best_E, st);
    if (npl <= 4) return launch_es<4>(a, int(grid), best_idx, best_E, st);
    if (npl <= 8) return launch_es<8>(a, int(grid), best_idx, best_E, st);
    return cudaErrorInvalidValue;                   // Nmax > 256 is rejected by the caller
}

cudaError_t launch_eval_configs(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                                int32_t gpu_budget, float *d_E, cudaStream_t st) {
    if (tiles == 0) return cudaSuccess;
    SweepArgs a = make_args(lay, d_ws, d_load, tiles, gpu_budget);
    int64_t grid = int64_t(sm_count()) * 8;
    if (grid > tiles) grid = tiles;
    const FastDiv divP = make_fastdiv(uint32_t(lay.P));
    cudaError_t e = cudaSuccess;
    if (a.stage_bytes > 0) {
        e = cudaFuncSetAttribute(eval_configs_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(a.stage_bytes));
        if (e != cudaSuccess) return e;
        eval_configs_kernel<true><<<int(grid), kThreads, a.stage_bytes, st>>>(a, divP, d_E);
    } else {
        eval_configs_kernel<false><<<int(grid), kThreads, 0, st>>>(a, divP, d_E);
    }
    return cudaGetLastError();
}

}  // namespace dyn
