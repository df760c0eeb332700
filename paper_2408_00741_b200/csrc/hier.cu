// Hierarchical control [Sec. 4.2]: nodes per pool from the epoch's peak load (scale-out/in), sharding
// at the highest frequency within those GPUs (shard-up/down), frequency per window (scale-up/down).
// Same models and the same resolved tables as the joint sweep; each level is a small restricted search.
// When the threshold tables fit in shared memory, the sharding and frequency kernels stage them and evaluate
// candidates as the sweep's threshold path does (compare on the per-instance load, 8-byte lookup of the energy
// line in shared memory); a warp serves one class there, and a class with a table row that has no load
// threshold (the resolve step's flags) is evaluated from the general-path tables through L1 instead, as is
// everything when the tables do not fit.
#define DYN_TU_ID 8
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


// true when some pair row of class c has no load threshold (vlim is NaN there); warp-uniform
__device__ __forceinline__ bool class_without_threshold(const HierArgs &a, int c) {
    const int P = a.T * a.F, lane = threadIdx.x & 31;
    bool bad = false;
    for (int p0 = 0; p0 < P; p0 += 32)
        bad |= __any_sync(kFull, p0 + lane < P && isnan(__ldg(a.pairc + c * P + p0 + lane).y));
    return bad;
}

// FAST kernels stage pair2 | rows2 into shared memory
template <bool FAST>
__device__ __forceinline__ void hier_begin(const HierArgs &a) {
    if (FAST) {
        extern __shared__ float4 smem[];
        const float4 *src = reinterpret_cast<const float4 *>(a.ws + a.off_pair2);
        const int n16 = (a.off_end - a.off_pair2) / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) smem[i] = src[i];
        __syncthreads();
        DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)), uint32_t(__cvta_generic_to_shared(smem)) + uint32_t(n16) * 16u,
                       uint32_t(a.off_end));
    } else {
        DYN_SET_RANGES(0u, 0u, uint32_t(a.off_end));
    }
}

// pool energy of n instances of pair p (class c) at per-instance load ln; ok = within SLO and capacity
template <bool FAST>
__device__ __forceinline__ float hier_eval(const HierArgs &a, uint32_t origin, int c, int p, float ln, float nf, float slo,
                                           bool general, bool &ok) {
    const int P = a.T * a.F, RS = a.M + 1;
    if (FAST && !general) {
        const float4 pc = load16<true>(a.ws, origin + uint32_t(c * P + p) * 16u);
        float e;
        fast_one<true>(a.ws, origin + uint32_t(a.off_rows2 - a.off_pair2) + uint32_t((c * P + p) * RS) * 8u, ln, pc.x, pc.z,
                       e, ok);
        return nf * e;
    }
    return eval_pair(a.rows + size_t(DYN_IDX(c * P + p, a.C * P)) * RS, __ldg(&a.pairc[DYN_IDX(c * P + p, a.C * P)]).x, float(a.M), ln,
                     nf, slo, ok);
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
        for (int w = w0; w < w1; ++w) PL = fmaxf(PL, *DYN_PTR(ld + size_t(w) * a.C, a.load, a.S * a.W * a.C));
        int nn = -1;
        if (ml > 0.0) {
            const double q = ceil(double(PL) / ml);
            nn = q < 1.0 ? 1 : (q > 1e9 ? 1000000000 : int(q));
        }
        a.nodes[DYN_IDX(size_t(s) * size_t(a.K1) * a.C + x, size_t(a.S) * a.K1 * a.C)] = nn;
    }
}

// one thread per (s, k2, c).  Staging variant: lanes are 32 consecutive shard epochs of one class.  With at most
// four TP degrees the constants of the highest-frequency pairs stay in registers; instance counts are walked two
// at a time with the sweep's packed evaluation (the two counts are the two chains, the TP degrees the pairs),
// the running minimum is kept on the energy of one instance and multiplied by n once per count; counts below
// the smallest one that can carry the load at any degree are skipped; the TP degree of the winning count is found
// again afterwards with bit-identical arithmetic (lowest degree first).
template <bool FAST>
__global__ void __launch_bounds__(256, FAST ? 4 : 1) hier_shard_kernel(const HierArgs a) {
    __shared__ float s_rn[257];                          // 1/n
    for (int n = threadIdx.x; n <= 256; n += blockDim.x) s_rn[n] = n ? 1.0f / float(n) : 0.f;
    hier_begin<FAST>(a);
    if (!FAST) __syncthreads();
    uint32_t origin = table_origin<FAST>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    uint32_t k2, c;
    const bool have = hier_item<FAST>(a, uint32_t(a.K2), k2, c);
    const bool general = FAST ? class_without_threshold(a, int(c)) : true;   // (c is warp-uniform in the staging variant)
    if (!have) return;
    const uint32_t x = k2 * a.C + c;
    const int w0 = int(k2) * a.e2, w1 = min(w0 + a.e2, a.W);
    const uint32_t k1 = fastdiv(uint32_t(w0), a.divE1);
    const float slo = a.slo[c];
    const int tpmax = a.tp[a.T - 1];
    const int cap_budget = a.Nmax * tpmax;            // a larger budget changes nothing
    const bool packed = FAST && !general && a.T <= 4;
    // constants of the (at most four) highest-frequency pairs
    uint64_t icm2[4], off2[4];
    float llim[4], icm[4], inv_llim[4];
    uint32_t row[4];
    if (packed) {
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int tt = t < a.T ? t : 0;
            const int p = tt * a.F + a.F - 1;
            const float4 pc = load16<true>(a.ws, origin + uint32_t(int(c) * a.T * a.F + p) * 16u);
            icm[t] = pc.x;
            icm2[t] = pack2(pc.x, pc.x);
            llim[t] = t < a.T ? pc.z : -1.f;
            inv_llim[t] = llim[t] > 0.f ? 1.0f / llim[t] : (llim[t] == 0.f ? 0.f : CUDART_INF_F);   // limit 0: no pruning
            row[t] = origin + uint32_t(a.off_rows2 - a.off_pair2) + uint32_t((int(c) * a.T * a.F + p) * (a.M + 1)) * 8u;
            const float off = row_offset_units(row[t]);
            off2[t] = pack2(off, off);
        }
    }
    // The energy of one instance never falls below the least knot energy of its row (the rows are piecewise
    // linear), so a pool of n instances costs at least n * e_floor whatever the load: once that reaches the best
    // energy found, no larger count can improve on it and the walk over n stops.  (Taken a little low, so that
    // rounding cannot cut off a candidate.)
    float e_floor = CUDART_INF_F;
    if (packed) {
        for (int t = 0; t < a.T; ++t) {
            if (!(llim[t] >= 0.f)) continue;
            for (int m = 0; m < a.M; ++m) {
                const float2 en = load8<true>(a.ws, row[t] + uint32_t(m) * 8u);
                const float l0 = float(m) / icm[t], l1 = float(m + 1) / icm[t];
                e_floor = fminf(e_floor, fminf(fmaf(l0, en.y, en.x), m + 1 < a.M ? fmaf(l1, en.y, en.x) : en.x));
            }
        }
        e_floor *= 0.99999f;
        if (!(e_floor > 0.f)) e_floor = 0.f;          // no positive floor: no pruning
    }
    // A sharper bound per degree: a line under the row's energy, e_t(l) >= alpha_t + beta_t * l on [0, limit] (beta_t the
    // row's secant slope, alpha_t the least knot value of e - beta_t * l; the rows are piecewise linear, so the knots
    // decide).  A pool of n instances at the epoch's peak PL then costs at least n * alpha_t + PL * beta_t at degree t
    // (n * e_t(PL / n)), whatever segment PL / n falls in: a candidate whose bound reaches the best energy found is
    // skipped, and once that holds for every degree and every alpha_t is non-negative (the bounds grow with n) the
    // walk stops.  For a power model that is linear in the load the bound is the energy itself, so the walk ends
    // right after the first feasible count.  (Both coefficients are taken a little low against rounding.)
    float alpha[4], beta[4];
    bool grows = true;                                // every bound is non-decreasing in n
#pragma unroll
    for (int t = 0; t < 4; ++t) { alpha[t] = 0.f; beta[t] = 0.f; }
    if (packed) {
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (t >= a.T || !(llim[t] >= 0.f)) continue;
            // knot m sits at l_m = m / icm; its energy is the segment's line there (the last knot closes segment M-2)
            const float2 e0 = load8<true>(a.ws, row[t]);
            const float2 eL = load8<true>(a.ws, row[t] + uint32_t(a.M - 2) * 8u);
            const float lL = float(a.M - 1) / icm[t];
            const float first = e0.x, last = fmaf(lL, eL.y, eL.x);
            float b = lL > 0.f ? (last - first) / lL : 0.f;
            if (!(b > 0.f) || !(b < CUDART_INF_F)) b = 0.f;
            b *= 0.9999f;
            float al = CUDART_INF_F;
            for (int m = 0; m < a.M; ++m) {
                const int seg = m < a.M - 1 ? m : a.M - 2;
                const float2 en = load8<true>(a.ws, row[t] + uint32_t(seg) * 8u);
                const float lm = float(m) / icm[t];
                al = fminf(al, fmaf(lm, en.y, en.x) - b * lm);
            }
            al = al > 0.f ? al * 0.9999f : al * 1.0001f;
            if (!(al > -CUDART_INF_F) || !(al < CUDART_INF_F)) { al = 0.f; b = 0.f; }
            alpha[t] = al;
            beta[t] = b;
            grows = grows && al >= 0.f;
        }
    }
    const uint64_t two23_2 = pack2(kTwo23, kTwo23), eight2 = pack2(units(8u), units(8u));
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const float *ld = a.load + size_t(s) * size_t(a.W) * a.C + c;
        float PL = 0.f;
        for (int w = w0; w < w1; ++w) PL = fmaxf(PL, *DYN_PTR(ld + size_t(w) * a.C, a.load, a.S * a.W * a.C));
        const int nn = a.nodes[DYN_IDX(size_t(s) * size_t(a.K1) * a.C + k1 * a.C + c, size_t(a.S) * a.K1 * a.C)];
        int budget = nn > 0 ? (nn > a.Nmax ? cap_budget : nn * tpmax) : 0;
        if (a.space_budget > 0 && budget > a.space_budget) budget = a.space_budget;
        int nmax = budget / a.tp[0];                  // no n above this fits even the smallest TP
        if (nmax > a.Nmax) nmax = a.Nmax;
        float best = CUDART_INF_F;
        int bnt = -1;
        if (packed) {
            // Degree by degree: counts below the least one that carries PL at the degree are infeasible there and are
            // not visited; from there on the counts are walked two at a time with the sweep's packed evaluation until
            // the degree's bound (see above) or the energy floor reaches the best energy found.  Ties go to the lowest
            // index (n - 1) * T + t, as in a walk in index order.
            int bidx = 0x7fffffff;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                if (t >= a.T || !(llim[t] >= 0.f)) continue;
                int nl = budget / a.tp[t];
                if (nl > a.Nmax) nl = a.Nmax;
                const float plb = PL * beta[t];
                float xf = PL * inv_llim[t] * 0.9999f;       // a little below the least count that carries PL here
                if (!(xf < 1e9f)) xf = 1e9f;
                int n = xf < 1.f ? 1 : (xf < 300.f ? int(xf) : nl + 1);
                for (; n <= nl; n += 2) {
                    const float nf = float(n);
                    if (nf * e_floor >= best) break;         // n and every larger count cost more than `best`
                    if (alpha[t] >= 0.f && fmaf(fmaxf(nf, xf), alpha[t], plb) >= best) break;   // so does every count from n on at this degree
                    const bool two = n + 1 <= nl;
                    const uint64_t ln2 = pack2(PL * s_rn[DYN_IDX(n, 257)], two ? PL * s_rn[DYN_IDX(n + 1, 257)] : CUDART_INF_F);
                    float eA = CUDART_INF_F, eB = CUDART_INF_F;
                    fast_two(ln2, icm2[t], off2[t], two23_2, eight2, llim[t], two ? llim[t] : -1.f, eA, eB);
                    const float EA = nf * eA, EB = (nf + 1.0f) * eB;
                    const int iA = (n - 1) * a.T + t, iB = n * a.T + t;
                    if (EA < best || (EA == best && EA < CUDART_INF_F && iA < bidx)) { best = EA; bidx = iA; }
                    if (EB < best || (EB == best && EB < CUDART_INF_F && iB < bidx)) { best = EB; bidx = iB; }
                }
            }
            if (best < CUDART_INF_F) bnt = bidx;
        } else
        for (int n = 1; n <= nmax; ++n) {
            const float nf = float(n), ln = PL * s_rn[n];
            for (int t = 0; t < a.T; ++t) {
                if (n * a.tp[t] > budget) break;      // TP ascending
                const int p = t * a.F + a.F - 1;
                bool ok;
                const float E = hier_eval<FAST>(a, origin, int(c), p, ln, nf, slo, general, ok);
                if (ok && E < best) {                 // ascending (n, t): strict compare keeps the lowest index
                    best = E;
                    bnt = (n - 1) * a.T + t;
                }
            }
        }
        a.shard[DYN_IDX(size_t(s) * size_t(a.K2) * a.C + x, size_t(a.S) * a.K2 * a.C)] = bnt;
    }
}

// one thread per (s, w, c): the frequency for the sharding of its shard epoch.  Staging variant: lanes are 32
// consecutive windows of one class; whatever depends on (window, class) only is formed once per thread, the
// walk over the scenarios keeps the F pairs of (class, TP) as running addresses (16 bytes of constants and one
// table row apart) and the minimum on the energy of one instance.
template <bool FAST>
__global__ void __launch_bounds__(256) hier_freq_kernel(const HierArgs a) {
    __shared__ float s_rn[257];                          // 1/n
    for (int n = threadIdx.x; n <= 256; n += blockDim.x) s_rn[n] = n ? 1.0f / float(n) : 0.f;
    hier_begin<FAST>(a);
    if (!FAST) __syncthreads();
    uint32_t origin = table_origin<FAST>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    uint32_t w, c;
    const bool have = hier_item<FAST>(a, uint32_t(a.W), w, c);
    const bool general = FAST ? class_without_threshold(a, int(c)) : true;   // (c is warp-uniform in the staging variant)
    if (!have) return;
    const uint32_t x = w * a.C + c;
    const uint32_t k2 = fastdiv(w, a.divE2);
    const float slo = a.slo[c];
    const size_t tile_stride = size_t(a.W) * a.C, shard_stride = size_t(a.K2) * a.C;
    const uint32_t pair_c = origin + uint32_t(int(c) * a.T * a.F) * 16u;
    const uint32_t rows_c = origin + uint32_t(a.off_rows2 - a.off_pair2) + uint32_t(int(c) * a.T * a.F * (a.M + 1)) * 8u;
    const uint32_t row_step = uint32_t(a.M + 1) * 8u;
    const float *ld = a.load + x;
    const int32_t *sh = a.shard + (k2 * a.C + c);
    int32_t *out_idx = a.best_idx + x;
    float *out_E = a.best_E + x;
    for (int64_t s = blockIdx.y; s < a.S; s += gridDim.y) {
        const int nt = *DYN_PTR(sh + size_t(s) * shard_stride, a.shard, a.S * int64_t(shard_stride));
        int32_t bj = -1;
        float best = CUDART_INF_F;
        if (nt >= 0) {
            const int n1 = int(fastdiv(uint32_t(nt), a.divT)), t = nt - n1 * a.T;
            const float nf = float(n1 + 1);
            const float ln = fmaxf(*DYN_PTR(ld + size_t(s) * tile_stride, a.load, a.S * int64_t(tile_stride)), 0.f) *
                             (n1 < 256 ? s_rn[DYN_IDX(n1 + 1, 257)] : 1.0f / nf);
            if (FAST && !general) {
                uint32_t pc_addr = pair_c + uint32_t(t * a.F) * 16u;
                uint32_t row = rows_c + uint32_t(t * a.F) * row_step;
                float emin = CUDART_INF_F;
                int bq = -1;
#pragma unroll 4
                for (int q = 0; q < a.F; ++q, pc_addr += 16u, row += row_step) {
                    const float4 pc = load16<true>(a.ws, pc_addr);
                    float e;
                    bool ok;
                    fast_one<true>(a.ws, row, ln, pc.x, pc.z, e, ok);
                    if (ok && e < emin) {            // ascending q: strict compare keeps the lowest
                        emin = e;
                        bq = q;
                    }
                }
                if (bq >= 0) {
                    best = nf * emin;
                    bj = nt * a.F + bq;
                }
            } else
            for (int q = 0; q < a.F; ++q) {
                bool ok;
                const float E = hier_eval<FAST>(a, origin, int(c), t * a.F + q, ln, nf, slo, general, ok);
                if (ok && E < best) {
                    best = E;
                    bj = nt * a.F + q;
                }
            }
        }
        out_idx[DYN_IDX(size_t(s) * tile_stride, size_t(a.S) * tile_stride - x)] = bj;
        out_E[DYN_IDX(size_t(s) * tile_stride, size_t(a.S) * tile_stride - x)] = best;
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
    const int64_t n1 = int64_t(a.K1) * lay.C, n2 = int64_t(a.K2) * lay.C;
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
    }
    hier_nodes_kernel<<<dim3(unsigned((n1 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // staging variants: a warp per (32 items, class)
    const int64_t f2 = ((int64_t(a.K2) + 31) / 32 * lay.C * 32 + 255) / 256;
    if (a.use_fast) hier_shard_kernel<true><<<dim3(unsigned(f2), few(f2)), 256, fast_bytes, st>>>(a);
    else hier_shard_kernel<false><<<dim3(unsigned((n2 + 255) / 256), gy), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    const int64_t f3 = ((W + 31) / 32 * lay.C * 32 + 255) / 256, n3 = W * lay.C;
    if (a.use_fast) {
        if ((e = cudaFuncSetAttribute(hier_freq_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(fast_bytes))) != cudaSuccess) return e;
        hier_freq_kernel<true><<<dim3(unsigned(f3), few(f3)), 256, fast_bytes, st>>>(a);
    } else {
        hier_freq_kernel<false><<<dim3(unsigned((n3 + 255) / 256), gy), 256, 0, st>>>(a);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
