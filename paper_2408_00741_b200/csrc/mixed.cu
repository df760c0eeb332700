// Pools that mix tensor parallelisms [Sec. 4.1, Eq. 1 in full]: counts N^{TP_i} per parallelism under the GPU
// budget sum_i TP_i*N^{TP_i} <= N, one frequency per parallelism, the load shared out over the groups, the
// objective sum_i N^{TP_i} * Energy^{TP_i, f_i}(L^{TP_i}).  The paper gives this to a solver; here the count
// tuples are enumerated: the host lists the tuples within the budget (numbered in odometer order, smallest TP
// fastest) and sorts the list by the set of parallelisms in use, so that the 32 tuples a warp handles at once
// mostly take the same branches; a warp takes a tile, lane l takes tuples l, l + 32, ... of the sorted list.  For a tuple the load is split in proportion to the
// groups' capacity at the highest candidate frequency, each group then picks its own feasible frequency of
// least energy (the single-type evaluation at fixed n and TP), and the tuple's energy is the sum.  The warp
// keeps the tuple of least energy, lowest tuple number on ties.
//
// Work per tile is (tuples) x (TP degrees in use) x F single-type evaluations; the loads and results are
// 4 + 12 + 8T bytes per tile.  The energy of a group is n x (energy of one instance at its per-instance load l),
// and l = (L/A) x capH_t, so for one TP degree the 32 x 4 tuples a warp holds are 128 per-instance loads run
// against that degree's F table rows: the inner loop of the single-type sweep.  When the threshold tables fit
// in shared memory, the kernel uses
// that loop (compare on l, segment address from a subnormal FMA, one FMA per candidate, predicated min) and
// recovers the frequencies of the winning tuple afterwards with the same arithmetic.  A class with a table row
// that has no load threshold is evaluated tile by tile from the general-path tables through L1 (the same
// kernel, a warp-uniform choice per tile), as is everything when the tables do not fit.
#define DYN_TU_ID 9
#include "dyn_internal.cuh"
#include "eval_dev.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

#ifndef DYN_MIXED_SHORT
#define DYN_MIXED_SHORT 0
#endif
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct MixedArgs {
    const float4 *rows;       // [C][P][M+1]
    const float2 *pairc;      // [C][P]
    const char *ws;           // scratch block (threshold tables at off_pair2 .. off_end)
    int32_t off_pair2, off_rows2, off_end;
    int32_t use_fast;         // threshold tables fit in shared memory
    const float *slo;         // [C]
    float *caph;              // [C][T] capacity at the highest candidate frequency
    float *inva;              // [C][K] 1 / (sum_t n_t * capH_t) of every tuple (threshold variant)
    const uint2 *tuples;      // [K] {counts, 8 bits per TP index; tuple number}, sorted by the set of TP indices in use
    const uint32_t *pairs;    // [n_pairs] tuple index | count << 16 | TP index << 24, by TP index, padded per index to whole chunks
    int64_t n_pairs;
    const float *load;        // [tiles]
    int64_t tiles, K;
    int32_t C, T, F, M;
    int32_t *counts, *freq, *tuple;
    float *best_E;
};

// capacity at the highest candidate frequency, as interpolated from the profile (whether or not that pair meets its
// TTFT SLO: the split of the load does not depend on feasibility)
__global__ void mixed_caph_kernel(const MixedArgs a) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.C * a.T) return;
    const int c = i / a.T, t = i - c * a.T;
    const float4 *pair2 = reinterpret_cast<const float4 *>(a.ws + a.off_pair2);
    a.caph[i] = pair2[DYN_IDX(c * (a.T * a.F) + t * a.F + a.F - 1, a.C * a.T * a.F)].w;
}

// 1 / A of every (class, tuple): A = sum_t n_t * capH_t, the pool's capacity at the highest candidate frequency
__global__ void mixed_inva_kernel(const MixedArgs a) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= int64_t(a.C) * a.K) return;
    const int c = int(i / a.K);
    const uint32_t tup = a.tuples[DYN_IDX(i - int64_t(c) * a.K, a.K)].x;
    double A = 0.0;
    for (int t = 0; t < a.T; ++t) A += double((tup >> (8 * t)) & 255u) * double(a.caph[c * a.T + t]);
    a.inva[i] = float(1.0 / A);                              // +inf when no degree of the tuple has capacity: infeasible
}

// one tile on the general-path tables (through L1): lane l takes tuples l, l + 32, ... of the list
template <int T>
__device__ __noinline__ void mixed_tile_plain(const MixedArgs &a, const int64_t i, const int lane) {
    const int P = T * a.F, RS = a.M + 1;
    const float Mf = float(a.M);
    {
        const int c = int(i % a.C);
        const float L = fmaxf(a.load[DYN_IDX(i, a.tiles)], 0.f);              // negative / NaN -> 0
        const float slo = a.slo[DYN_IDX(c, a.C)];
        float caph[T];
#pragma unroll
        for (int t = 0; t < T; ++t) caph[t] = a.caph[c * T + t];
        float best = CUDART_INF_F;
        uint32_t bnum = 0xffffffffu, btup = 0;               // number and counts of the lane's best tuple
        uint32_t bq = 0;                                     // its frequencies, 8 bits per TP index
        for (int64_t k = lane; k < a.K; k += 32) {
            const uint2 tk = __ldg(a.tuples + DYN_IDX(k, a.K));
            const uint32_t tup = tk.x;
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
                const float4 *rows_t = a.rows + size_t(DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1)) * RS;
                const float2 *pc_t = a.pairc + DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1);
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
            if (E < best || (E == best && tk.y < bnum)) {    // the list is not in number order: lowest number on ties
                best = E;
                bnum = tk.y;
                btup = tup;
                bq = qs;
            }
        }
        best += 0.f;                                         // -0 -> +0
        float Emin;
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(Emin) : "f"(best));
        // lowest tuple number among the lanes that hold the minimum
        const uint32_t kmin = __reduce_min_sync(kFull, best == Emin ? bnum : 0xffffffffu);
        if (Emin == CUDART_INF_F) {
            if (lane < T) {
                a.counts[DYN_IDX(i * T + lane, a.tiles * T)] = -1;
                a.freq[DYN_IDX(i * T + lane, a.tiles * T)] = -1;
            }
            if (lane == 0) {
                a.tuple[DYN_IDX(i, a.tiles)] = -1;
                a.best_E[i] = CUDART_INF_F;
            }
            return;
        }
        if (best == Emin && bnum == kmin) {                  // exactly one lane: tuple numbers are distinct
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const uint32_t n = (btup >> (8 * t)) & 255u;
                a.counts[DYN_IDX(i * T + t, a.tiles * T)] = int32_t(n);
                a.freq[i * T + t] = n ? int32_t((bq >> (8 * t)) & 255u) : -1;
            }
            a.tuple[DYN_IDX(i, a.tiles)] = int32_t(kmin);
            a.best_E[i] = Emin;
        }
    }
}

template <int T>
__global__ void __launch_bounds__(kThreads) mixed_select_kernel(const MixedArgs a) {
    DYN_SET_RANGES(0u, 0u, uint32_t(a.off_end));
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t i = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); i < a.tiles; i += nwarps) mixed_tile_plain<T>(a, i, lane);
}


// End of a tile in the threshold variants: the warp's best tuple (least energy, lowest tuple number among equals)
// from the lanes' candidates, its frequencies recovered with the arithmetic of the search, the results written.
template <int T>
__device__ __forceinline__ void finish_tile(const MixedArgs &a, const int64_t i, const int c, const int lane, float best,
                                            const uint32_t bnum, const uint32_t btup, const float bfrac, const float (&caph)[T],
                                            const uint32_t origin, const uint32_t rows2) {
    const int F = a.F, P = T * F, RS = a.M + 1;
    best += 0.f;                                         // -0 -> +0
    const float Emin = warp_min(best);
    const uint32_t kmin = __reduce_min_sync(kFull, best == Emin ? bnum : 0xffffffffu);
    if (Emin == CUDART_INF_F) {
        if (lane < T) {
            a.counts[DYN_IDX(i * T + lane, a.tiles * T)] = -1;
            a.freq[DYN_IDX(i * T + lane, a.tiles * T)] = -1;
        }
        if (lane == 0) {
            a.tuple[DYN_IDX(i, a.tiles)] = -1;
            a.best_E[i] = CUDART_INF_F;
        }
        return;
    }
    // the winning tuple and its load fraction, from the lane that holds it (tuple numbers are distinct)
    const int wl = __ffs(__ballot_sync(kFull, best == Emin && bnum == kmin)) - 1;
    const uint32_t wt = __shfl_sync(kFull, btup, wl);
    const float wf = __shfl_sync(kFull, bfrac, wl);
    // its frequencies: lane p re-evaluates pair (t, q) = (p / F, p % F) with the same arithmetic; per degree
    // the least energy, lowest q among equals
    float gmin[T];
    int gq[T];
#pragma unroll
    for (int t = 0; t < T; ++t) { gmin[t] = CUDART_INF_F; gq[t] = -1; }
    for (int p0 = 0; p0 < P; p0 += 32) {
        const int p = p0 + lane;
        const int tp = p < P ? p / F : 0;
        float val = CUDART_INF_F;
        if (p < P && ((wt >> (8 * tp)) & 255u)) {
            float ctp = caph[0];
#pragma unroll
            for (int t = 1; t < T; ++t) ctp = (t == tp) ? caph[t] : ctp;
            const float4 pc = load16<true>(a.ws, origin + uint32_t(c * P + p) * 16u);
            float e;
            bool ok;
            fast_one<true>(a.ws, rows2 + uint32_t((c * P + p) * RS) * 8u, wf * ctp, pc.x, pc.z, e, ok);
            if (ok) val = e;
        }
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const bool mine = p < P && tp == t;
            const float m = warp_min(mine ? val : CUDART_INF_F);
            if (m < gmin[t]) {                           // strictly better than the earlier rounds (lower q)
                gmin[t] = m;
                gq[t] = p0 + __ffs(__ballot_sync(kFull, mine && val == m)) - 1 - t * F;
            }
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const uint32_t n = (wt >> (8 * t)) & 255u;
            a.counts[DYN_IDX(i * T + t, a.tiles * T)] = int32_t(n);
            a.freq[i * T + t] = n ? gq[t] : -1;
        }
        a.tuple[DYN_IDX(i, a.tiles)] = int32_t(kmin);
        a.best_E[i] = Emin;
    }
}

// threshold variant: tables of all classes in shared memory, SL tuples per lane and pass (32 * SL tuples side by side;
// the list is sorted by the set of degrees in use, and a pass skips the degrees none of its tuples uses: short
// passes skip more, long ones share a pair's constants among more candidates)
template <int T, int SL>
__global__ void __launch_bounds__(kThreads, 3) mixed_fast_kernel(const MixedArgs a) {
    // classes with a table row that has no load threshold (the resolve step's flags) take the general path
    __shared__ unsigned char s_general[256];
    for (int c = threadIdx.x; c < a.C; c += blockDim.x) {
        bool bad = false;
        for (int p = 0; p < a.T * a.F; ++p) bad |= isnan(__ldg(a.pairc + c * a.T * a.F + p).y);
        s_general[c] = bad ? 1 : 0;
    }
    extern __shared__ float4 smem[];
    {
        const float4 *src = reinterpret_cast<const float4 *>(a.ws + a.off_pair2);
        const int n16 = (a.off_end - a.off_pair2) / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) smem[i] = src[i];
        __syncthreads();
        DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)), uint32_t(__cvta_generic_to_shared(smem)) + uint32_t(n16) * 16u,
                       uint32_t(a.off_end));
    }
    uint32_t origin = table_origin<true>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    const int lane = threadIdx.x & 31;
    const int F = a.F, P = T * F, RS = a.M + 1;
    const uint32_t pstep = uint32_t(RS) * 8u;
    const uint32_t rows2 = origin + uint32_t(a.off_rows2 - a.off_pair2);
    const uint64_t two23_2 = pack2(kTwo23, kTwo23);
    const uint64_t eight2 = pack2(units(8u), units(8u));
    const float offs = float(int(pstep)) * units(1u);
    const uint64_t off2_step = pack2(offs, offs);
    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t i = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); i < a.tiles; i += nwarps) {
        const int c = int(i % a.C);
        if (s_general[c]) {                                  // warp-uniform
            mixed_tile_plain<T>(a, i, lane);
            continue;
        }
        const float L = fmaxf(a.load[DYN_IDX(i, a.tiles)], 0.f);              // negative / NaN -> 0
        float caph[T];
#pragma unroll
        for (int t = 0; t < T; ++t) caph[t] = a.caph[c * T + t];
        float best = CUDART_INF_F, bfrac = 0.f;
        uint32_t bnum = 0xffffffffu, btup = 0;
        for (int64_t base = 0; base < a.K; base += 32 * SL) {
            uint32_t tup[SL], num[SL];
            float frac[SL], E[SL];
#pragma unroll
            for (int j = 0; j < SL; ++j) {
                const int64_t k = base + j * 32 + lane;
                const uint2 tk = k < a.K ? __ldg(a.tuples + k) : make_uint2(0u, 0xffffffffu);
                tup[j] = tk.x;
                num[j] = tk.y;
                // every instance runs at this fraction of its top-frequency capacity
                frac[j] = k < a.K ? L * __ldg(a.inva + DYN_IDX(int64_t(c) * a.K + k, int64_t(a.C) * a.K)) : 0.f;
                E[j] = tk.x ? 0.f : CUDART_INF_F;            // a slot past the end of the list never wins
            }
#pragma unroll
            for (int t = 0; t < T; ++t) {
                uint32_t n[SL];
                float ln[SL], e1[SL];
                uint32_t any = 0;
#pragma unroll
                for (int j = 0; j < SL; ++j) {
                    n[j] = (tup[j] >> (8 * t)) & 255u;
                    any |= n[j];
                    ln[j] = n[j] ? frac[j] * caph[t] : CUDART_INF_F;      // no instance of this degree: nothing to serve
                    e1[j] = CUDART_INF_F;
                }
                if (!__any_sync(kFull, any != 0)) continue;              // no tuple of the pass uses this degree
                uint64_t ln2[SL / 2];
#pragma unroll
                for (int j = 0; j < SL; j += 2) ln2[j / 2] = pack2(ln[j], ln[j + 1]);
                const uint32_t cpair = origin + uint32_t(c * P + t * F) * 16u;
                const float off0 = row_offset_units(rows2 + uint32_t((c * P + t * F) * RS) * 8u);
                uint64_t off2 = pack2(off0, off0);
#pragma unroll 4
                for (int q = 0; q < F; ++q) {
                    uint64_t icm2, lim2;
                    asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(icm2), "=l"(lim2) : "r"(DYN_SMEM_ADDR(cpair + uint32_t(q) * 16u, 16u)));
                    const float lim = __uint_as_float(uint32_t(lim2));
#pragma unroll
                    for (int j = 0; j < SL; j += 2) fast_two(ln2[j / 2], icm2, off2, two23_2, eight2, lim, lim, e1[j], e1[j + 1]);
                    off2 = add2(off2, off2_step);
                }
#pragma unroll
                for (int j = 0; j < SL; ++j)
                    if (n[j]) E[j] += float(n[j]) * e1[j];   // ascending TP index; +inf if the group has no frequency
            }
#pragma unroll
            for (int j = 0; j < SL; ++j)
                if (E[j] < best || (E[j] == best && num[j] < bnum)) {     // lowest tuple number on ties
                    best = E[j];
                    bnum = num[j];
                    btup = tup[j];
                    bfrac = frac[j];
                }
        }
        finish_tile<T>(a, i, c, lane, best, bnum, btup, bfrac, caph, origin, rows2);
    }
}

// threshold variant for short lists: the (tuple, TP index) pairs that hold instances are listed by TP index, a warp
// takes a chunk of 64 at a time, two neighbouring pairs per lane, against the F table rows of the lane's index, and
// adds n x (energy of one instance) to the tuple's sum in a per-warp array in shared memory.  A chunk may run over
// from one index into the next, but holds no tuple twice (the host sees to that).  Chunks come in ascending TP index, so a tuple's sum forms in the same order as in the other
// variants; no evaluation is spent on a parallelism that a tuple does not use.  Then the lanes scan the sums.
template <int T>
__global__ void __launch_bounds__(kThreads, 3) mixed_pairs_kernel(const MixedArgs a, const int table_bytes) {
    __shared__ unsigned char s_general[256];
    for (int c = threadIdx.x; c < a.C; c += blockDim.x) {
        bool bad = false;
        for (int p = 0; p < a.T * a.F; ++p) bad |= isnan(__ldg(a.pairc + c * a.T * a.F + p).y);
        s_general[c] = bad ? 1 : 0;
    }
    extern __shared__ float4 smem[];
    {
        const float4 *src = reinterpret_cast<const float4 *>(a.ws + a.off_pair2);
        const int n16 = (a.off_end - a.off_pair2) / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) smem[i] = src[i];
        __syncthreads();
        DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)), uint32_t(__cvta_generic_to_shared(smem)) + uint32_t(n16) * 16u,
                       uint32_t(a.off_end));
    }
    uint32_t origin = table_origin<true>();
    asm volatile("" : "+r"(origin) : : "memory");        // table loads stay behind the staging barrier
    const int lane = threadIdx.x & 31;
    const int K = int(a.K), Kpad = (K + 31) & ~31;
    float *Es = reinterpret_cast<float *>(reinterpret_cast<char *>(smem) + table_bytes) + (threadIdx.x >> 5) * Kpad;   // this warp's sums
    const int F = a.F, P = T * F, RS = a.M + 1;
    const uint32_t pstep = uint32_t(RS) * 8u;
    const uint32_t rows2 = origin + uint32_t(a.off_rows2 - a.off_pair2);
    const uint64_t two23_2 = pack2(kTwo23, kTwo23);
    const uint64_t eight2 = pack2(units(8u), units(8u));
    const float offs = float(int(pstep)) * units(1u);
    const uint64_t off2_step = pack2(offs, offs);
    const int64_t nwarps = int64_t(gridDim.x) * kWarps;
    for (int64_t i = int64_t(blockIdx.x) * kWarps + (threadIdx.x >> 5); i < a.tiles; i += nwarps) {
        const int c = int(i % a.C);
        if (s_general[c]) {                                  // warp-uniform
            mixed_tile_plain<T>(a, i, lane);
            continue;
        }
        const float L = fmaxf(a.load[DYN_IDX(i, a.tiles)], 0.f);              // negative / NaN -> 0
        float caph[T];
#pragma unroll
        for (int t = 0; t < T; ++t) caph[t] = a.caph[c * T + t];
        const float *inva_c = a.inva + int64_t(c) * a.K;
        for (int k = lane; k < Kpad; k += 32) Es[DYN_IDX(k, Kpad)] = 0.f;
        __syncwarp();
        for (int64_t e0 = 0; e0 < a.n_pairs; e0 += kMixedPairsChunk) {
            // a lane's two neighbouring entries share their TP index; the chunk may run over from one index into the next
            const uint2 ent = __ldg(reinterpret_cast<const uint2 *>(a.pairs + DYN_IDX(e0 + 2 * lane, a.n_pairs - 1)));
            const int t = int(ent.x >> 24);
            const uint32_t kA = ent.x & 0xffffu, kB = ent.y & 0xffffu, nA = (ent.x >> 16) & 255u, nB = (ent.y >> 16) & 255u;
            float ct = caph[0];
#pragma unroll
            for (int u = 1; u < T; ++u) ct = (u == t) ? caph[u] : ct;
            // every instance of a tuple runs at the fraction L / A of its top-frequency capacity
            const float lA = nA ? (L * __ldg(inva_c + DYN_IDX(kA, a.K))) * ct : CUDART_INF_F;
            const float lB = nB ? (L * __ldg(inva_c + DYN_IDX(kB, a.K))) * ct : CUDART_INF_F;
            const uint64_t ln2 = pack2(lA, lB);
            float eA = CUDART_INF_F, eB = CUDART_INF_F;
            uint32_t cpair = origin + uint32_t(c * P + t * F) * 16u;
            const float off0 = row_offset_units(rows2 + uint32_t((c * P + t * F) * RS) * 8u);
            uint64_t off2 = pack2(off0, off0);
#pragma unroll 4
            for (int q = 0; q < F; ++q, cpair += 16u) {
                uint64_t icm2, lim2;
                asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(icm2), "=l"(lim2) : "r"(DYN_SMEM_ADDR(cpair, 16u)));
                const float lim = __uint_as_float(uint32_t(lim2));
                fast_two(ln2, icm2, off2, two23_2, eight2, lim, lim, eA, eB);
                off2 = add2(off2, off2_step);
            }
            // no tuple appears twice in a chunk (the host pads a chunk out where one would): no two lanes meet on a sum
            if (nA) Es[DYN_IDX(kA, Kpad)] += float(nA) * eA;                  // +inf if the group has no frequency
            if (nB) Es[DYN_IDX(kB, Kpad)] += float(nB) * eB;
            __syncwarp();
        }
        float best = CUDART_INF_F, bfrac = 0.f;
        uint32_t bnum = 0xffffffffu, btup = 0;
        for (int k = lane; k < K; k += 32) {
            const float E = Es[DYN_IDX(k, Kpad)];
            const uint2 tk = __ldg(a.tuples + k);
            if (E < best || (E == best && tk.y < bnum)) {    // lowest tuple number on ties
                best = E;
                bnum = tk.y;
                btup = tk.x;
                bfrac = L * __ldg(inva_c + k);
            }
        }
        __syncwarp();                                        // the sums are read before the next tile clears them
        finish_tile<T>(a, i, c, lane, best, bnum, btup, bfrac, caph, origin, rows2);
    }
}

}  // namespace

cudaError_t launch_mixed(const ResolvedLayout &lay, void *d_ws, size_t off_tuples, size_t off_caph, size_t off_inva, size_t off_pairs,
                         int64_t n_pairs, int64_t K, const float *d_load, int64_t tiles, int32_t *d_counts, int32_t *d_freq,
                         int32_t *d_tuple, float *d_best_E, cudaStream_t st) {
    char *ws = static_cast<char *>(d_ws);
    MixedArgs a{};
    a.rows = reinterpret_cast<const float4 *>(ws + lay.off_rows);
    a.pairc = reinterpret_cast<const float2 *>(ws + lay.off_pairc);
    a.slo = reinterpret_cast<const float *>(ws + lay.off_slo);
    a.caph = reinterpret_cast<float *>(ws + off_caph);
    a.inva = reinterpret_cast<float *>(ws + off_inva);
    a.tuples = reinterpret_cast<const uint2 *>(ws + off_tuples);
    a.pairs = reinterpret_cast<const uint32_t *>(ws + off_pairs);
    a.n_pairs = n_pairs;
    a.load = d_load;
    a.tiles = tiles; a.K = K;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.M = lay.M;
    a.counts = d_counts; a.freq = d_freq; a.tuple = d_tuple; a.best_E = d_best_E;
    a.ws = ws;
    a.off_pair2 = int32_t(lay.off_pair2); a.off_rows2 = int32_t(lay.off_rows2); a.off_end = int32_t(lay.off_tp);
    mixed_caph_kernel<<<(lay.C * lay.T + 127) / 128, 128, 0, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || tiles == 0) return e;
    mixed_inva_kernel<<<unsigned((int64_t(lay.C) * K + 255) / 256), 256, 0, st>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    int64_t grid = (tiles + kWarps - 1) / kWarps;
    const int64_t cap = int64_t(sm_count()) * 8;
    if (grid > cap) grid = cap;
    a.ws = ws;
    a.off_pair2 = int32_t(lay.off_pair2); a.off_rows2 = int32_t(lay.off_rows2); a.off_end = int32_t(lay.off_tp);
    const size_t fast_bytes = lay.off_tp - lay.off_pair2;
    a.use_fast = fast_bytes <= 96 * 1024 ? 1 : 0;
    // (passes of 64 tuples skip more degrees than passes of 128 but share a pair's constants among fewer candidates:
    // measured slower at 200 tuples, so the long passes serve every list)
    const bool short_passes = K <= DYN_MIXED_SHORT;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    // short lists: the compact list of (tuple, TP index) pairs; per-warp sums behind the tables in shared memory
    const size_t pairs_bytes = fast_bytes + size_t(kWarps) * size_t((K + 31) & ~int64_t(31)) * sizeof(float);
    const bool use_pairs = a.use_fast && n_pairs > 0 && K <= kMixedPairsMaxTuples && K <= 0xffff;
#define DYN_MIXED_LAUNCH(TT)                                                                                      \
    do {                                                                                                          \
        if (use_pairs) {                                                                                          \
            e = cudaFuncSetAttribute(mixed_pairs_kernel<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                                     int(pairs_bytes));                                                           \
            if (e != cudaSuccess) return e;                                                                       \
            mixed_pairs_kernel<TT><<<int(grid), kThreads, pairs_bytes, st>>>(a, int(fast_bytes));                 \
        } else if (a.use_fast) {                                                                                  \
            if (short_passes) {                                                                                   \
                e = cudaFuncSetAttribute(mixed_fast_kernel<TT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                         int(fast_bytes));                                                        \
                if (e != cudaSuccess) return e;                                                                   \
                mixed_fast_kernel<TT, 2><<<int(grid), kThreads, fast_bytes, st>>>(a);                             \
            } else {                                                                                              \
                e = cudaFuncSetAttribute(mixed_fast_kernel<TT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                         int(fast_bytes));                                                        \
                if (e != cudaSuccess) return e;                                                                   \
                mixed_fast_kernel<TT, 4><<<int(grid), kThreads, fast_bytes, st>>>(a);                             \
            }                                                                                                     \
        } else {                                                                                                  \
            mixed_select_kernel<TT><<<int(grid), kThreads, 0, st>>>(a);                                           \
        }                                                                                                         \
    } while (0)
    switch (lay.T) {
        case 1: DYN_MIXED_LAUNCH(1); break;
        case 2: DYN_MIXED_LAUNCH(2); break;
        case 3: DYN_MIXED_LAUNCH(3); break;
        case 4: DYN_MIXED_LAUNCH(4); break;
        default: return cudaErrorInvalidValue;
    }
#undef DYN_MIXED_LAUNCH
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
