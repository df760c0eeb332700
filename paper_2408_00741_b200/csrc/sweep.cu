// Stage (b) and fused (b)+(c): evaluate every candidate (n instances, TP, f) of every (window, class)
// tile against the latency/power profile and the SLOs [Sec. 4.1, Eq. 1], and keep the
// minimum-energy feasible one [Sec. 4.2].
//
// Work is plain fp32 arithmetic (no dense contraction, so no tensor cores); the kernel is bound by
// instruction issue.  The design keeps the instructions per candidate low:
//   * a warp owns tiles of ONE class; lanes hold instance counts n (several per lane when Nmax > 32),
//     the (TP, f) pairs are the inner loop, so per-pair constants and the table row are warp-uniform
//     and shared by all candidates of the pair;
//   * within one (tile, n) chain the instance count is fixed, so the running minimum is kept on the
//     energy of ONE instance and multiplied by n once per chain after the pair loop (rounding is
//     monotone, so the minimum of the products is the product of the minimum, bit for bit);
//   * for a table row whose TBT, once above the SLO, never returns to it as the load grows (the resolve
//     step checks each row; every row that rises with load qualifies), "TBT <= SLO and u <= 1" is a
//     threshold on the per-instance load l = L/n (the largest load an instance sustains within the SLO,
//     cf. ML in Sec. 4.2): one compare, no TBT interpolation.  The energy of the
//     segment is stored as a line in l (intercept, slope), so one FMA on l gives it and no fraction is
//     formed.  The segment number is floor(l*icm), taken from a fused multiply-add with 2^23 rounded
//     toward zero (the low mantissa bits are the integer; no float-to-int conversion); a second fused
//     multiply-add by 2^-146 with a per-pair offset turns 2^23 + m into the subnormal number whose bit
//     pattern IS the shared-memory byte address of entry m of the pair's row (subnormal floats count
//     in units of 2^-149, entries are 8 bytes apart).  Both run two candidates at a time on the packed
//     two-wide fp32 instructions of sm_100.  Per candidate that leaves: compare, 2 x half a packed
//     FMA, lookup, FMA, predicated min.  Infeasible candidates skip the lookup (same predicate), so
//     no clamp of the table position is needed;
//   * a row without that property (a measured profile with a dip at the SLO) takes the general path: TBT
//     and energy are interpolated from the segment's left knot for every candidate (16-byte lookups,
//     saturating multiply as clamp, sentinel entries for u > 1).  The choice is made per ROW: with few
//     such rows the threshold loop runs over all pairs (a row without a threshold has the limit -1 there
//     and accepts nothing) and a second loop serves only those rows, from the tables in global memory;
//     when more than a quarter of the rows lack a threshold, all rows take the general path on staged
//     tables;
//   * only the running minimum is kept; the pair that attained it is recovered once per tile by
//     re-evaluating that instance count for 32 pairs at a time with bit-identical arithmetic.
// The resolved tables of all classes are staged in shared memory once per CTA when they fit; larger
// tables are read through L1 or staged per class.
#define DYN_TU_ID 4
#include "dyn_internal.cuh"
#include "eval_dev.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

#ifndef DYN_SW_UNROLL
#define DYN_SW_UNROLL 8
#endif
constexpr int kPairUnroll = DYN_SW_UNROLL;
#ifndef DYN_SW_MINB4
#define DYN_SW_MINB4 5
#endif
#ifndef DYN_SW_TT1
#define DYN_SW_TT1 8
#endif
#ifndef DYN_SW_TT2
#define DYN_SW_TT2 4
#endif
#ifndef DYN_SW_MINB16
#define DYN_SW_MINB16 2
#endif
#ifndef DYN_SW_MINB8
#define DYN_SW_MINB8 4
#endif

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct SweepArgs {
    const char *ws;          // scratch block: rows (float4) | pairc (float2) | slo | pair2 (float4) | rows2 (float2) | tp ...
    const float *load;       // [rows_total][C]
    const int32_t *tp;       // [T]
    int64_t tiles;
    int64_t rows_total;      // S*W
    int64_t rows_per_warp;   // multiple of the tiles a warp takes per pass
    int64_t blocks;          // row blocks; work units = blocks * C
    int32_t C, T, F, P, M, Nmax, J;
    int32_t budget;          // <= 0: none
    int32_t ln_log2;         // lanes per n-group = 1 << ln_log2
    int32_t off_rows, off_pairc, off_slo, off_pair2, off_rows2, off_end;   // byte offsets inside ws
    int32_t smem_bytes;      // dynamic shared memory of the launch (0: tables are read from global)
};

// where the tables of this CTA live: byte offsets from `smem` when staged, else from a.ws
struct Tables {
    uint32_t rows, pairc, slo, pair2, rows2;
};

// copy [ws + from, ws + to) into shared memory (16-byte pieces)
__device__ __forceinline__ void stage(const SweepArgs &a, int from, int to) {
    extern __shared__ float4 smem[];
    const float4 *src = reinterpret_cast<const float4 *>(a.ws + from);
    const int n16 = (to - from) / 16;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) smem[DYN_IDX(i, a.smem_bytes / 16)] = src[i];
    __syncthreads();
    // (checking build) the range the arithmetically formed table addresses must stay in
    DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)), uint32_t(__cvta_generic_to_shared(smem)) + uint32_t(to - from),
                   uint32_t(a.off_end));
}

// number of pair rows among [first, first + n) without a load threshold (the resolve step stores NaN as
// their vlim); the same value in every thread of the CTA
__device__ __forceinline__ int rows_without_threshold(const SweepArgs &a, int first, int n) {
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const float2 *pc = reinterpret_cast<const float2 *>(a.ws + a.off_pairc) + first;
    int bad = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) bad += isnan(__ldg(pc + i).y) ? 1 : 0;
    if (bad) atomicAdd(&s_bad, bad);
    __syncthreads();
    return s_bad;
}

// what the general-path evaluation of one class's rows needs, formed at the point of use from values the
// compiler cannot trace (so that none of it is kept in registers across the threshold loop)
struct MixedRows {
    const float2 *flags;     // pairc of the class: {ic, vlim}; vlim is NaN for a row without a load threshold
    uint32_t rows;           // byte offset of the class's general-path rows in the scratch block
    int P, RS;
    float Mf, slo;
    Consts2 k2;
};
__device__ __forceinline__ int opaque(int v) {
    asm volatile("mov.b32 %0, %0;" : "+r"(v));
    return v;
}
__device__ __forceinline__ MixedRows mixed_rows(const SweepArgs &a, int c) {
    MixedRows g;
    const int co = opaque(c), M = opaque(a.M);
    g.P = opaque(a.P);
    g.RS = M + 1;
    g.Mf = float(M);
    g.flags = reinterpret_cast<const float2 *>(a.ws + opaque(a.off_pairc)) + co * g.P;
    g.rows = uint32_t(opaque(a.off_rows)) + uint32_t(co * g.P * g.RS) * 16u;
    g.slo = __ldg(reinterpret_cast<const float *>(a.ws + opaque(a.off_slo)) + co);
    g.k2.M = make_float2(g.Mf, g.Mf);
    g.k2.negM = make_float2(-g.Mf, -g.Mf);
    g.k2.two23 = make_float2(kTwo23, kTwo23);
    g.k2.neg23 = make_float2(-kTwo23, -kTwo23);
    return g;
}

// ---------------------------------------------------------------------------------------------
// fused evaluate + select
//   NPL  instance counts per lane (Nmax <= 32*NPL)
//   TT   tiles (rows of the same class) a warp evaluates per pass over the pairs
//   CLS  the CTA serves one class (blockIdx.y) and `tb` points at that class's tables alone
//   MIXED (threshold path only) some rows have no load threshold: a second loop and the pair recovery
//        evaluate those rows on the general path from the tables in global memory
// ---------------------------------------------------------------------------------------------
template <int NPL, int TT, bool BUDGET, bool SMEM, bool FAST, bool FULL, bool CLS = false, bool MIXED = false>
__device__ __forceinline__ void sweep_body(const SweepArgs &a, const Tables tb, int32_t *__restrict__ best_idx,
                                           float *__restrict__ best_E) {
    const int lane = threadIdx.x & 31;
    const int64_t unit = int64_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (unit >= (CLS ? a.blocks : a.blocks * a.C)) return;
    const int c = CLS ? int(blockIdx.y) : int(unit % a.C);
    const int64_t r_begin = (CLS ? unit : unit / a.C) * a.rows_per_warp;
    const int64_t r_end = r_begin + a.rows_per_warp < a.rows_total ? r_begin + a.rows_per_warp : a.rows_total;

    // FULL: the 32 lanes are 32 instance counts of the same tiles.  Otherwise (Nmax <= 16) the warp splits
    // into TG groups of LN lanes; the lanes of a group are the instance counts, and every group takes its own
    // TT tiles of a pass, so the per-tile reductions and the pair recovery of all groups share their instructions
    const int LN = FULL ? 32 : 1 << a.ln_log2;
    const int TG = FULL ? 1 : 32 >> a.ln_log2;
    const int nl = lane & (LN - 1);
    const int g = FULL ? 0 : lane >> a.ln_log2;
    const int gsh = g * LN;                          // first lane of the group
    const unsigned lowmask = FULL ? kFull : (1u << LN) - 1u;
    const unsigned gmask = lowmask << gsh;           // the lanes of this group
    const int P = a.P, RS = a.M + 1, C = a.C;
    const float Mf = float(a.M);
    const char *ws = a.ws;

    // chain k of the lane evaluates n = nl + 1 + LN*k.  A lane whose n exceeds Nmax: on the threshold path its
    // per-instance load is made +inf (or NaN), which no pair accepts; on the general path it is dropped
    // after the pair loop
    float nf[NPL], rn[NPL];
    int pmax[NPL];
    bool keep[NPL];
#pragma unroll
    for (int k = 0; k < NPL; ++k) {
        const int n = nl + 1 + LN * k;
        const bool valid = n <= a.Nmax;
        keep[k] = (FAST && !MIXED) || valid;
        nf[k] = float(n);
        rn[k] = valid ? 1.0f / float(n) : (FAST ? CUDART_INF_F : 0.f);
        pmax[k] = P;
        if (BUDGET) {
            int nt = 0;
            for (int t = 0; t < a.T; ++t) nt += (int64_t(n) * a.tp[t] <= int64_t(a.budget)) ? 1 : 0;
            pmax[k] = nt * a.F;                      // TP ascending: allowed pairs are a prefix
        }
    }

    // class constants
    constexpr uint32_t ESZ = FAST ? 8u : 16u;
    uint32_t origin = table_origin<SMEM>();
    // every table address below derives from `origin`: this keeps the (side-effect free) inline-assembly
    // loads from being scheduled ahead of the barrier that ends the staging
    asm volatile("" : "+r"(origin) : : "memory");
    const int ct = CLS ? 0 : c;                      // class offset inside the tables `tb` points at
    // pair constants: threshold path pair2 (16 bytes), general path pairc (8 bytes)
    const uint32_t cpair = origin + (FAST ? tb.pair2 + uint32_t(ct * P) * 16u : tb.pairc + uint32_t(ct * P) * 8u);
    const uint32_t crow = origin + (FAST ? tb.rows2 : tb.rows) + uint32_t(ct * P * RS) * ESZ;   // row of pair 0
    const uint32_t pstep = uint32_t(RS) * ESZ;
    float slo_c = 0.f;
    if (!FAST) {
        if (SMEM && !CLS) {
            extern __shared__ float4 smem[];
            slo_c = reinterpret_cast<const float *>(reinterpret_cast<const char *>(smem) + tb.slo)[c];
        } else {
            slo_c = __ldg(reinterpret_cast<const float *>(ws + a.off_slo) + c);
        }
    }
    Consts2 k2;
    k2.M = make_float2(Mf, Mf);
    k2.negM = make_float2(-Mf, -Mf);
    k2.two23 = make_float2(kTwo23, kTwo23);
    k2.neg23 = make_float2(-kTwo23, -kTwo23);
    // threshold path with staged tables: row offsets as subnormal floats (see fast_two)
    const uint64_t two23_2 = pack2(kTwo23, kTwo23);
    const uint64_t eight2 = pack2(units(8u), units(8u));
    const float off0 = row_offset_units(crow);
    const float offs = float(int(pstep)) * units(1u);
    const uint64_t off2_first = pack2(off0, off0), off2_step = pack2(offs, offs);
    constexpr int NCH = TT * NPL;                    // candidates per lane and pair, an even number
    static_assert(NCH % 2 == 0, "candidates are evaluated two at a time");

    // per-lane constants of the pair recovery: lane p re-evaluates pair p0 + p.  With at most 32 pairs and
    // no GPU budget there is one round, and the lane's pair constants stay in registers for all tiles
    const uint32_t cpair_lane = cpair + uint32_t(nl) * (FAST ? 16u : 8u);
    const uint32_t crow_lane = crow + uint32_t(nl) * pstep;
    const bool one_round = !BUDGET && P <= LN;
    float rc_ic = 0.f, rc_lim = FAST ? -1.f : -CUDART_INF_F;          // a lane without a pair never hits
    if (one_round && nl < P) {
        if (FAST) {
            const float4 pc = load16<SMEM>(ws, cpair_lane);
            rc_ic = pc.x;
            rc_lim = pc.z;
        } else {
            rc_ic = load8<SMEM>(ws, cpair_lane).x;
            rc_lim = slo_c;
        }
    }
    const uint32_t rc_row = (one_round && nl < P) ? crow_lane : crow;
    // Rows of this class without a load threshold: their general-path tables are read from global memory.
    // Only this flag (and the class number) stays live across the pair loop; whatever else those rows need
    // is formed where it is used, behind opaque moves, so that the threshold loop keeps its registers.
    bool class_mixed = false;
    if (MIXED) {
        const float2 *flags = reinterpret_cast<const float2 *>(ws + a.off_pairc) + c * P;
        for (int p0 = 0; p0 < P; p0 += 32)
            class_mixed |= __any_sync(kFull, p0 + lane < P && isnan(__ldg(flags + p0 + lane).y));
    }
    const int sh_n = FULL ? 5 : a.ln_log2;           // n - 1 = (chain number << sh_n) + lane number
    const int tpp = TT * TG;                         // tiles of a pass
    const float *lp = a.load + ((r_begin + g * TT) * C + c);          // load of the group's first tile; tiles are C floats apart
    int64_t oi = (r_begin + g * TT) * C + c;         // its index in the outputs

    for (int64_t r = r_begin; r < r_end; r += tpp, lp += tpp * C, oi += int64_t(tpp) * C) {
        const int64_t left = r_end - (r + g * TT);
        const int nt = left < TT ? (FULL || left > 0 ? int(left) : 0) : TT;          // tiles of this group in this pass
        // chain q = t*NPL + k: tile t of this pass, k-th instance count of the lane; `best` is the least
        // energy of ONE instance over the feasible pairs of the chain
        float best[NCH];
        uint64_t ln2[NCH / 2];                       // per-instance loads L/n of chains (q, q+1), packed
        {
            float ln[NCH];
#pragma unroll
            for (int t = 0; t < TT; ++t) {
                const float L = t < nt ? fmaxf(*DYN_PTR(lp + t * C, a.load, a.tiles), 0.f) : 0.f;   // negative / NaN -> 0
#pragma unroll
                for (int k = 0; k < NPL; ++k) {
                    ln[t * NPL + k] = L * rn[k];
                    best[t * NPL + k] = CUDART_INF_F;
                }
            }
#pragma unroll
            for (int q = 0; q < NCH; q += 2) ln2[q / 2] = pack2(ln[q], ln[q + 1]);
        }
#define DYN_LN(q) half_of(ln2[(q) / 2], (q) & 1)
        if (FAST && SMEM) {
            uint64_t off2 = off2_first;
#pragma unroll kPairUnroll
            for (int p = 0; p < P; ++p) {
                uint64_t icm2, lim2;
                asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(icm2), "=l"(lim2) : "r"(DYN_SMEM_ADDR(cpair + uint32_t(p) * 16u, 16u)));
                const float lim = __uint_as_float(uint32_t(lim2));
#pragma unroll
                for (int q = 0; q < NCH; q += 2)
                    fast_two(ln2[q / 2], icm2, off2, two23_2, eight2,
                             (!BUDGET || p < pmax[q % NPL]) ? lim : -1.f,
                             (!BUDGET || p < pmax[(q + 1) % NPL]) ? lim : -1.f, best[q], best[q + 1]);
                off2 = add2(off2, off2_step);
            }
        } else if (FAST) {
#pragma unroll 4
            for (int p = 0; p < P; ++p) {
                const float4 pc = load16<SMEM>(ws, cpair + uint32_t(p) * 16u);
                const uint32_t row = crow + uint32_t(p) * pstep;
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    float e;
                    bool ok;
                    fast_one<SMEM>(ws, row, DYN_LN(q), pc.x, pc.z, e, ok);
                    if (ok && (!BUDGET || p < pmax[q % NPL])) best[q] = fminf(best[q], e);
                }
            }
        } else {
#pragma unroll 8
            for (int p = 0; p < P; ++p) {
                const float2 pc = load8<SMEM>(ws, cpair + uint32_t(p) * 8u);
                const uint32_t base = crow + uint32_t(p) * pstep - kTwo23Bits * 16u;
#pragma unroll
                for (int q = 0; q < NCH; q += 2)
                    general_two<SMEM>(ws, base, DYN_LN(q), DYN_LN(q + 1), pc.x, slo_c, k2, !BUDGET || p < pmax[q % NPL],
                                      !BUDGET || p < pmax[(q + 1) % NPL], best[q], best[q + 1]);
            }
        }
        if (MIXED && class_mixed) {
            // the rows without a threshold, one by one (warp-uniform), on the general path
            const MixedRows g = mixed_rows(a, c);
            for (int p0 = 0; p0 < g.P; p0 += 32) {
                unsigned todo = __ballot_sync(kFull, p0 + lane < g.P && isnan(__ldg(g.flags + p0 + lane).y));
                while (todo) {
                    const int p = p0 + __ffs(todo) - 1;
                    todo &= todo - 1;
                    const float ic = __ldg(g.flags + p).x;
                    const uint32_t base = g.rows + uint32_t(p * g.RS) * 16u - kTwo23Bits * 16u;
#pragma unroll
                    for (int q = 0; q < NCH; q += 2)
                        general_two<false>(ws, base, DYN_LN(q), DYN_LN(q + 1), ic, g.slo, g.k2,
                                           !BUDGET || p < pmax[q % NPL], !BUDGET || p < pmax[(q + 1) % NPL],
                                           best[q], best[q + 1]);
                }
            }
        }
        // per tile: warp argmin on (pool energy, n), then the pair; lane t keeps the result of tile t
        int32_t my_idx = -1;
        float my_E = CUDART_INF_F;
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            if (FULL && t >= nt) break;              // one group: uniform (several groups: the idle ones run along)
            // the lane's chains in ascending n: strict compare keeps the lower n on ties.  Pool energy =
            // n * (energy of one instance); the zero addend turns -0 into +0, so equal energies have equal bits
            float E = keep[0] ? fmaf(best[t * NPL], nf[0], 0.f) : CUDART_INF_F;
            int kk = 0;
#pragma unroll
            for (int k = 1; k < NPL; ++k) {
                const float Ek = keep[k] ? fmaf(best[t * NPL + k], nf[k], 0.f) : CUDART_INF_F;
                if (Ek < E) {
                    E = Ek;
                    kk = k;
                }
            }
            // smallest energy of the tile, then the fewest instances that attain it (lowest index: n is the
            // slowest digit of j); lanes of different pair groups may hold the same n.  A tile without a
            // feasible candidate (minimum +inf) runs through the same steps and finds no pair: -1 / +inf
            const float Emin = FULL ? warp_min(E) : group_min(E, gmask);
            const uint32_t n1 = uint32_t(kk << sh_n) + uint32_t(nl);              // n - 1
            const uint32_t n1min = __reduce_min_sync(FULL ? kFull : gmask, E == Emin ? n1 : 0xffffffffu);
            const float nfm = float(n1min + 1u);
            // L/n of the winning instance count, from the lane that holds it (bit-identical by construction)
            float lnk = DYN_LN(t * NPL);
            if (NPL > 1) {
                const int kstar = int(n1min >> sh_n);
#pragma unroll
                for (int k = 1; k < NPL; ++k) lnk = (k == kstar) ? DYN_LN(t * NPL + k) : lnk;
            }
            const float lnm = __shfl_sync(kFull, lnk, gsh + (int(n1min) & (LN - 1)));
            // recover the pair: lanes re-evaluate (nmin, p) for 32 pairs at a time, same arithmetic, and the
            // first pair that reproduces the minimum bit for bit is the lowest-index one
            int pstar = -1;
            if (one_round) {
                float e;
                bool ok;
                if (FAST) fast_one<SMEM>(ws, rc_row, lnm, rc_ic, rc_lim, e, ok);
                else general_one<SMEM>(ws, rc_row - kTwo23Bits * 16u, lnm, rc_ic, rc_lim, Mf, e, ok);
                if (MIXED && class_mixed && nl < P) {                // a lane whose row has no threshold: general path
                    const MixedRows g = mixed_rows(a, c);
                    const float2 gp = __ldg(g.flags + nl);
                    if (isnan(gp.y))
                        general_one<false>(ws, g.rows + uint32_t(nl * g.RS) * 16u - kTwo23Bits * 16u, lnm, gp.x, g.slo,
                                           g.Mf, e, ok);
                }
                pstar = __ffs((__ballot_sync(kFull, ok && (fmaf(e, nfm, 0.f) == Emin)) >> gsh) & lowmask) - 1;
            } else {
                int pm = P;
                if (BUDGET) {
                    int ntp = 0;
                    for (int tt = 0; tt < a.T; ++tt) ntp += (int64_t(n1min + 1u) * a.tp[tt] <= int64_t(a.budget)) ? 1 : 0;
                    pm = ntp * a.F;
                }
                // one group stops at its first hit; several groups walk all rounds together (their bounds differ)
                for (int p0 = 0; p0 < (FULL ? pm : P); p0 += LN) {
                    bool hit = false;
                    if (pstar < 0 && p0 + nl < pm) {
                        float e;
                        bool ok;
                        float2 gp = make_float2(0.f, 0.f);
                        MixedRows g;
                        if (MIXED && class_mixed) {
                            g = mixed_rows(a, c);
                            gp = __ldg(g.flags + p0 + nl);
                        }
                        if (MIXED && class_mixed && isnan(gp.y)) {
                            general_one<false>(ws, g.rows + uint32_t((p0 + nl) * g.RS) * 16u - kTwo23Bits * 16u, lnm, gp.x,
                                               g.slo, g.Mf, e, ok);
                        } else if (FAST) {
                            const float4 pc = load16<SMEM>(ws, cpair_lane + uint32_t(p0) * 16u);
                            fast_one<SMEM>(ws, crow_lane + uint32_t(p0) * pstep, lnm, pc.x, pc.z, e, ok);
                        } else {
                            const float2 pc = load8<SMEM>(ws, cpair_lane + uint32_t(p0) * 8u);
                            general_one<SMEM>(ws, crow_lane + uint32_t(p0) * pstep - kTwo23Bits * 16u, lnm, pc.x, slo_c, Mf, e, ok);
                        }
                        hit = ok && (fmaf(e, nfm, 0.f) == Emin);
                    }
                    const unsigned m = (__ballot_sync(kFull, hit) >> gsh) & lowmask;
                    if (m && pstar < 0) pstar = p0 + __ffs(m) - 1;
                    if (FULL && m) break;
                }
            }
            if (nl == t) {
                my_idx = pstar >= 0 ? int32_t(n1min * uint32_t(P) + uint32_t(pstar)) : -1;
                my_E = Emin;
            }
        }
        if (nl < nt) {
            best_idx[DYN_IDX(oi + nl * C, a.tiles)] = my_idx;
            best_E[DYN_IDX(oi + nl * C, a.tiles)] = my_E;
        }
    }
}

#undef DYN_LN

template <int NPL, int TT, bool BUDGET, bool SMEM, bool FULL>
__global__ void __launch_bounds__(kThreads, (NPL * TT <= 4 ? DYN_SW_MINB4 : (NPL * TT <= 8 && NPL <= 2 ? (NPL == 1 ? DYN_SW_MINB4 : DYN_SW_MINB8) : (NPL * TT <= 16 && NPL <= 2 ? DYN_SW_MINB16 : 2))))
eval_select_kernel(const SweepArgs a, int32_t *__restrict__ best_idx, float *__restrict__ best_E) {
    Tables tb;
    tb.rows = a.off_rows; tb.pairc = a.off_pairc; tb.slo = a.off_slo; tb.pair2 = a.off_pair2; tb.rows2 = a.off_rows2;
    const int bad = rows_without_threshold(a, 0, a.C * a.P);     // uniform over the grid: every CTA reads the same flags
    if (!SMEM) DYN_SET_RANGES(0u, 0u, uint32_t(a.off_end));
    if (bad * 4 <= a.C * a.P) {
        if (SMEM) {
            stage(a, a.off_pair2, a.off_end);        // pair2 | rows2
            tb.pair2 = 0; tb.rows2 = a.off_rows2 - a.off_pair2;
        }
        if (bad == 0) sweep_body<NPL, TT, BUDGET, SMEM, true, FULL>(a, tb, best_idx, best_E);
        else sweep_body<NPL, TT, BUDGET, SMEM, true, FULL, false, true>(a, tb, best_idx, best_E);
    } else {
        if (SMEM) {
            stage(a, a.off_rows, a.off_pair2);       // rows | pairc | slo
            tb.rows = 0; tb.pairc = a.off_pairc - a.off_rows; tb.slo = a.off_slo - a.off_rows;
        }
        sweep_body<NPL, TT, BUDGET, SMEM, false, FULL>(a, tb, best_idx, best_E);
    }
}

// Tables too large to stage for all classes at once (fine frequency grids): a CTA serves ONE class
// (blockIdx.y) and stages that class's threshold tables, pair2_c | rows2_c, in shared memory; one CTA
// of 16 warps per SM.  The rows of the class that have no load threshold are served from the tables in global
// memory; when they are more than a quarter of the class's rows the general path serves all of them.
template <int NPL, int TT, bool BUDGET>
__global__ void __launch_bounds__(512, 1)
eval_select_class_kernel(const SweepArgs a, int32_t *__restrict__ best_idx, float *__restrict__ best_E) {
    Tables tb;
    tb.rows = tb.pairc = tb.slo = tb.pair2 = tb.rows2 = 0;
    const int bad = rows_without_threshold(a, int(blockIdx.y) * a.P, a.P);
    if (bad * 4 <= a.P) {
        extern __shared__ float4 smem[];
        const int c = blockIdx.y;
        const int pair_bytes = a.P * 16, rows2_bytes = a.P * (a.M + 1) * 8;
        const float4 *src_p = reinterpret_cast<const float4 *>(a.ws + a.off_pair2 + size_t(c) * pair_bytes);
        const float4 *src_r = reinterpret_cast<const float4 *>(a.ws + a.off_rows2 + size_t(c) * rows2_bytes);
        const int np16 = pair_bytes / 16, nr16 = (rows2_bytes + 15) / 16;   // rounding up stays inside the scratch block
        for (int i = threadIdx.x; i < np16; i += blockDim.x) smem[i] = src_p[i];
        for (int i = threadIdx.x; i < nr16; i += blockDim.x) smem[np16 + i] = src_r[i];
        __syncthreads();
        DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)), uint32_t(__cvta_generic_to_shared(smem)) + uint32_t((np16 + nr16) * 16),
                       uint32_t(a.off_end));
        tb.pair2 = 0; tb.rows2 = uint32_t(pair_bytes);
        if (bad == 0) sweep_body<NPL, TT, BUDGET, true, true, true, true>(a, tb, best_idx, best_E);
        else sweep_body<NPL, TT, BUDGET, true, true, true, true, true>(a, tb, best_idx, best_E);
    } else {
        DYN_SET_RANGES(0u, 0u, uint32_t(a.off_end));
        const int c = blockIdx.y;
        tb.rows = a.off_rows + uint32_t(c) * uint32_t(a.P * (a.M + 1)) * 16u;
        tb.pairc = a.off_pairc + uint32_t(c) * uint32_t(a.P) * 8u;
        tb.slo = a.off_slo;
        sweep_body<NPL, TT, BUDGET, false, false, true, true>(a, tb, best_idx, best_E);
    }
}

// ---------------------------------------------------------------------------------------------
// evaluate only: E[tile][j], j = (n-1)*P + p.  A warp takes one tile and 32 consecutive pairs: lanes
// are pairs (their constants stay in registers), the loop runs over n two at a time, and each pass
// writes two coalesced runs of 32 energies.  Threshold or general path as in the fused kernel, with
// the same arithmetic per candidate; MIXED: a lane whose row has no load threshold evaluates it on the
// general path from the tables in global memory.
// ---------------------------------------------------------------------------------------------
template <bool BUDGET, bool SMEM, bool FAST, bool MIXED = false>
__device__ __forceinline__ void configs_body(const SweepArgs &a, const Tables tb, const float2 *s_n, const int64_t units_total,
                                             float *__restrict__ E_out) {
    const int lane = threadIdx.x & 31;
    const int P = a.P, RS = a.M + 1, Nmax = a.Nmax;
    const int PG = (P + 31) / 32;                     // pair groups per tile
    const float Mf = float(a.M);
    constexpr uint32_t ESZ = FAST ? 8u : 16u;
    uint32_t origin = table_origin<SMEM>();
    asm volatile("" : "+r"(origin) : : "memory");        // as in sweep_body: table loads stay behind the staging barrier
    const char *ws = a.ws;
    const float4 *s_n4 = reinterpret_cast<const float4 *>(s_n);   // per pair of counts: {1/n, 1/(n+1), n, n+1}
    const uint32_t sn_addr = uint32_t(__cvta_generic_to_shared(s_n));

    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t u = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); u < units_total; u += nwarps) {
        const int64_t i = u / PG;
        const int p = int(u - i * PG) * 32 + lane;
        const int c = int(i % a.C);
        const bool active = p < P;
        const int pp = active ? p : 0;
        const float L = fmaxf(a.load[DYN_IDX(i, a.tiles)], 0.f);
        const float slo_c = __ldg(reinterpret_cast<const float *>(ws + a.off_slo) + c);
        const uint32_t row = origin + (FAST ? tb.rows2 : tb.rows) + uint32_t((c * P + pp) * RS) * ESZ;
        float ic, lim;                                // threshold path: {icm, llim}; general: {ic, slo}
        if (FAST) {
            const float4 pc = load16<SMEM>(ws, origin + tb.pair2 + uint32_t(c * P + pp) * 16u);
            ic = pc.x;
            lim = pc.z;
        } else {
            ic = load8<SMEM>(ws, origin + tb.pairc + uint32_t(c * P + pp) * 8u).x;
            lim = slo_c;
        }
        bool lane_general = false;
        float gic = 0.f;
        if (MIXED) {
            const float2 gp = __ldg(reinterpret_cast<const float2 *>(ws + a.off_pairc) + (c * P + pp));
            lane_general = isnan(gp.y);
            gic = gp.x;
        }
        const uint32_t grow = uint32_t(a.off_rows) + uint32_t((c * P + pp) * RS) * 16u - kTwo23Bits * 16u;
        int nlim = Nmax;                              // Eq. 1 GPU budget: n * TP <= budget
        if (BUDGET) {
            const int64_t q = int64_t(a.budget) / a.tp[pp / a.F];
            nlim = q < Nmax ? int(q) : Nmax;
        }
        float *out = E_out + size_t(DYN_IDX(i, a.tiles)) * size_t(a.J) + (active ? p : 0);     // candidates of this pair are P floats apart
        if (FAST && SMEM) {
            // two instance counts per trip with the packed form of the fused kernel (same arithmetic)
            const uint64_t L2 = pack2(L, L), icm2 = pack2(ic, ic);
            const float off = row_offset_units(row);
            const uint64_t off2 = pack2(off, off);
            const uint64_t two23_2 = pack2(kTwo23, kTwo23), eight2 = pack2(units(8u), units(8u));
            const int pairs = Nmax >> 1;
#pragma unroll 4
            for (int h = 0; h < pairs; ++h, out += 2 * P) {
                uint64_t rn2, nf2;                            // {1/n, 1/(n+1)}, {n, n+1}
                asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(rn2), "=l"(nf2) : "r"(sn_addr + uint32_t(DYN_IDX(h, 129)) * 16u));
                const float limA = (!BUDGET || 2 * h + 1 <= nlim) ? lim : -1.f;
                const float limB = (!BUDGET || 2 * h + 2 <= nlim) ? lim : -1.f;
                float EA, EB;
                fast_two_energy(mul2(L2, rn2), icm2, off2, two23_2, eight2, limA, limB, half_of(nf2, 0), half_of(nf2, 1),
                                EA, EB);
                if (MIXED && lane_general) {
                    float eA, eB;
                    bool okA, okB;
                    general_one<false>(ws, grow, L * half_of(rn2, 0), gic, slo_c, Mf, eA, okA);
                    general_one<false>(ws, grow, L * half_of(rn2, 1), gic, slo_c, Mf, eB, okB);
                    EA = (okA && (!BUDGET || 2 * h + 1 <= nlim)) ? eA * half_of(nf2, 0) : CUDART_INF_F;
                    EB = (okB && (!BUDGET || 2 * h + 2 <= nlim)) ? eB * half_of(nf2, 1) : CUDART_INF_F;
                }
                if (active) {
                    __stcs(out, EA);
                    __stcs(out + P, EB);
                }
            }
            if (Nmax & 1) {                               // odd count: the last n alone
                const float4 nn = s_n4[pairs];
                float e;
                bool ok;
                fast_one<SMEM>(ws, row, L * nn.x, ic, (!BUDGET || Nmax <= nlim) ? lim : -1.f, e, ok);
                if (MIXED && lane_general) {
                    general_one<false>(ws, grow, L * nn.x, gic, slo_c, Mf, e, ok);
                    ok = ok && (!BUDGET || Nmax <= nlim);
                }
                if (active) __stcs(out, ok ? e * nn.z : CUDART_INF_F);
            }
        } else
        for (int n1 = 0; n1 < Nmax; n1 += 2, out += 2 * P) {
            const float4 nn = s_n4[n1 >> 1];                       // {1/n, 1/(n+1), n, n+1}
            const float lnA = L * nn.x, lnB = L * nn.y;
            float eA, eB;
            bool okA, okB;
            if (MIXED && lane_general) {
                general_one<false>(ws, grow, lnA, gic, slo_c, Mf, eA, okA);
                general_one<false>(ws, grow, lnB, gic, slo_c, Mf, eB, okB);
            } else if (FAST) {
                fast_one<SMEM>(ws, row, lnA, ic, lim, eA, okA);
                fast_one<SMEM>(ws, row, lnB, ic, lim, eB, okB);
            } else {
                general_one<SMEM>(ws, row - kTwo23Bits * 16u, lnA, ic, lim, Mf, eA, okA);
                general_one<SMEM>(ws, row - kTwo23Bits * 16u, lnB, ic, lim, Mf, eB, okB);
            }
            if (BUDGET) {
                okA = okA && n1 + 1 <= nlim;
                okB = okB && n1 + 2 <= nlim;
            }
            if (active) {
                __stcs(out, okA ? eA * nn.z : CUDART_INF_F);
                if (n1 + 1 < Nmax) __stcs(out + P, okB ? eB * nn.w : CUDART_INF_F);
            }
        }
    }
}

template <bool BUDGET, bool SMEM>
__global__ void __launch_bounds__(kThreads)
eval_configs_kernel(const SweepArgs a, const int64_t units_total, float *__restrict__ E_out) {
    // for the counts (2h+1, 2h+2), h = 0..Nmax/2: {1/n, 1/(n+1), n, n+1} (Nmax <= 256)
    __shared__ __align__(16) float2 s_n[258];
    for (int h = threadIdx.x; h <= a.Nmax / 2; h += kThreads) {
        const float n0 = float(2 * h + 1), n1 = float(2 * h + 2);
        s_n[2 * h] = make_float2(1.0f / n0, 1.0f / n1);
        s_n[2 * h + 1] = make_float2(n0, n1);
    }
    Tables tb;
    tb.rows = a.off_rows; tb.pairc = a.off_pairc; tb.slo = a.off_slo; tb.pair2 = a.off_pair2; tb.rows2 = a.off_rows2;
    const int bad = rows_without_threshold(a, 0, a.C * a.P);     // (also a barrier for s_n)
    if (!SMEM) DYN_SET_RANGES(0u, 0u, uint32_t(a.off_end));
    if (bad * 4 <= a.C * a.P) {                      // load-threshold path: 8-byte lookups
        if (SMEM) {
            stage(a, a.off_pair2, a.off_end);
            tb.pair2 = 0; tb.rows2 = a.off_rows2 - a.off_pair2;
        }
        if (bad == 0) configs_body<BUDGET, SMEM, true>(a, tb, s_n, units_total, E_out);
        else configs_body<BUDGET, SMEM, true, true>(a, tb, s_n, units_total, E_out);
    } else {
        if (SMEM) {
            stage(a, a.off_rows, a.off_pair2);
            tb.rows = 0; tb.pairc = a.off_pairc - a.off_rows; tb.slo = a.off_slo - a.off_rows;
        }
        configs_body<BUDGET, SMEM, false>(a, tb, s_n, units_total, E_out);
    }
}

size_t smem_limit() {
    // opt-in shared memory per block of the current device (cached per device)
    static thread_local size_t lim[kMaxDevices] = {};
    const int slot = device_slot();
    if (lim[slot] == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess || v <= 0)
            v = 48 * 1024;
        lim[slot] = size_t(v);
    }
    return lim[slot];
}

SweepArgs make_args(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles, int32_t budget) {
    SweepArgs a{};
    a.ws = static_cast<const char *>(d_ws);
    a.tp = reinterpret_cast<const int32_t *>(a.ws + lay.off_tp);
    a.load = d_load;
    a.tiles = tiles;
    a.rows_total = tiles / lay.C;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.P = lay.P; a.M = lay.M; a.Nmax = lay.Nmax; a.J = lay.J;
    a.budget = budget;
    a.off_rows = int32_t(lay.off_rows);
    a.off_pairc = int32_t(lay.off_pairc);
    a.off_slo = int32_t(lay.off_slo);
    a.off_pair2 = int32_t(lay.off_pair2);
    a.off_rows2 = int32_t(lay.off_rows2);
    a.off_end = int32_t(lay.off_tp);
    // the general path stages rows | pairc | slo, the threshold path pair2 | rows2 (smaller): one piece each
    const size_t general = lay.off_pair2 - lay.off_rows;
    a.smem_bytes = general <= 96 * 1024 && general <= smem_limit() ? int32_t(general) : 0;
    return a;
}

template <int NPL, int TT, bool B, bool S, bool FULL>
cudaError_t launch_es_variant(SweepArgs &a, int32_t *best_idx, float *best_E, cudaStream_t st) {
    auto kernel = eval_select_kernel<NPL, TT, B, S, FULL>;
    cudaError_t e = cudaSuccess;
    if (S) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, a.smem_bytes);
        if (e != cudaSuccess) return e;
    }
    int resident = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kThreads, S ? size_t(a.smem_bytes) : 0);
    if (e != cudaSuccess) return e;
    if (resident < 1) resident = 1;
    // about four work units per resident warp: all units cost the same, so the tail is short
    const int64_t want_units = int64_t(sm_count()) * resident * kWarps * 4;
    int64_t rpw = (a.tiles + want_units - 1) / want_units;          // rows of one class per unit
    const int tpp = TT * (FULL ? 1 : 32 >> a.ln_log2);               // tiles of a pass
    rpw = (rpw + tpp - 1) / tpp * tpp;
    a.rows_per_warp = rpw;
    a.blocks = (a.rows_total + rpw - 1) / rpw;
    const int64_t units = a.blocks * a.C;
    const int64_t grid = (units + kWarps - 1) / kWarps;
    kernel<<<unsigned(grid), kThreads, S ? size_t(a.smem_bytes) : 0, st>>>(a, best_idx, best_E);
    return cudaGetLastError();
}

// one class per CTA, 512 threads, the class's threshold tables in shared memory
template <int NPL, int TT, bool B>
cudaError_t launch_es_class(SweepArgs &a, size_t class_bytes, int32_t *best_idx, float *best_E, cudaStream_t st) {
    auto kernel = eval_select_class_kernel<NPL, TT, B>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(class_bytes));
    if (e != cudaSuccess) return e;
    const int warps = 16;
    // about four work units per resident warp
    const int64_t want_units = int64_t(sm_count()) * warps * 4;
    int64_t rpw = (a.tiles + want_units - 1) / want_units;          // rows of one class per unit
    rpw = (rpw + TT - 1) / TT * TT;
    a.rows_per_warp = rpw;
    a.blocks = (a.rows_total + rpw - 1) / rpw;                      // units per class
    const int64_t gx = (a.blocks + warps - 1) / warps;
    kernel<<<dim3(unsigned(gx), unsigned(a.C)), warps * 32, class_bytes, st>>>(a, best_idx, best_E);
    return cudaGetLastError();
}

template <int NPL, int TT>
cudaError_t launch_es(SweepArgs &a, int32_t *best_idx, float *best_E, cudaStream_t st) {
    const bool smem = a.smem_bytes > 0;
    const bool budget = a.budget > 0;
    if (!smem && NPL > 1) {
        // pair2_c and rows2_c (rounded up to 16 bytes)
        const size_t class_bytes = size_t(a.P) * 16 + (size_t(a.P) * size_t(a.M + 1) * 8 + 15) / 16 * 16;
        if (a.P % 2 == 0 && class_bytes + 1024 <= smem_limit())       // even P: class blocks stay 16-byte aligned
            return budget ? launch_es_class<NPL, TT, true>(a, class_bytes, best_idx, best_E, st)
                          : launch_es_class<NPL, TT, false>(a, class_bytes, best_idx, best_E, st);
    }
    constexpr bool FULL = NPL > 1;                   // more than 32 instance counts: one pair group
    if (NPL == 1 && a.ln_log2 == 5) {                // exactly 17..32 instance counts
        if (budget && smem) return launch_es_variant<NPL, TT, true, true, true>(a, best_idx, best_E, st);
        if (budget) return launch_es_variant<NPL, TT, true, false, true>(a, best_idx, best_E, st);
        if (smem) return launch_es_variant<NPL, TT, false, true, true>(a, best_idx, best_E, st);
        return launch_es_variant<NPL, TT, false, false, true>(a, best_idx, best_E, st);
    }
    if (budget && smem) return launch_es_variant<NPL, TT, true, true, FULL>(a, best_idx, best_E, st);
    if (budget) return launch_es_variant<NPL, TT, true, false, FULL>(a, best_idx, best_E, st);
    if (smem) return launch_es_variant<NPL, TT, false, true, FULL>(a, best_idx, best_E, st);
    return launch_es_variant<NPL, TT, false, false, FULL>(a, best_idx, best_E, st);
}

}  // namespace

cudaError_t launch_eval_select(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                               int32_t gpu_budget, int32_t *best_idx, float *best_E, cudaStream_t st) {
    if (tiles == 0) return cudaSuccess;
    SweepArgs a = make_args(lay, d_ws, d_load, tiles, gpu_budget);
    // lanes per n-group: smallest power of two covering Nmax, at most 32
    int ln = 0;
    while ((1 << ln) < lay.Nmax && ln < 5) ++ln;
    if (ln < 3) ln = 3;                             // a group of lanes also holds the results of its 8 tiles
    a.ln_log2 = ln;
    const int npl = (lay.Nmax + 31) / 32;           // instance counts per lane
    // four candidates per lane share each pair's constants
    if (npl <= 1) return launch_es<1, DYN_SW_TT1>(a, best_idx, best_E, st);
    if (npl <= 2) return launch_es<2, DYN_SW_TT2>(a, best_idx, best_E, st);
    if (npl <= 4) return launch_es<4, 1>(a, best_idx, best_E, st);
    if (npl <= 8) return launch_es<8, 1>(a, best_idx, best_E, st);
    return cudaErrorInvalidValue;                   // Nmax > 256 is rejected by the caller
}

cudaError_t launch_eval_configs(const ResolvedLayout &lay, const void *d_ws, const float *d_load, int64_t tiles,
                                int32_t gpu_budget, float *d_E, cudaStream_t st) {
    if (tiles == 0) return cudaSuccess;
    SweepArgs a = make_args(lay, d_ws, d_load, tiles, gpu_budget);
    const int64_t units = tiles * ((lay.P + 31) / 32);          // (tile, group of 32 pairs) per warp
    int64_t grid = int64_t(sm_count()) * 8;
    const int64_t need = (units + kWarps - 1) / kWarps;
    if (grid > need) grid = need;
    const bool smem = a.smem_bytes > 0, budget = gpu_budget > 0;
    const size_t dyn_smem = smem ? size_t(a.smem_bytes) : 0;
    cudaError_t e = cudaSuccess;
#define DYN_LAUNCH_EC(B, S)                                                                                        \
    do {                                                                                                           \
        if (S) e = cudaFuncSetAttribute(eval_configs_kernel<B, S>, cudaFuncAttributeMaxDynamicSharedMemorySize,     \
                                        a.smem_bytes);                                                             \
        if (e == cudaSuccess) {                                                                                    \
            eval_configs_kernel<B, S><<<int(grid), kThreads, dyn_smem, st>>>(a, units, d_E);                       \
            e = cudaGetLastError();                                                                                \
        }                                                                                                          \
    } while (0)
    if (budget && smem) DYN_LAUNCH_EC(true, true);
    else if (budget) DYN_LAUNCH_EC(true, false);
    else if (smem) DYN_LAUNCH_EC(false, true);
    else DYN_LAUNCH_EC(false, false);
#undef DYN_LAUNCH_EC
    return e;
}

}  // namespace dyn
