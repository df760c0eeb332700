// Selection that counts the cost of re-configuring [Sec. 4.2 "Accounting for the overheads": the controllers set
// the energy a new configuration saves against the cost of the transition, read from an Overhead Table; Sec. 4.3:
// re-sharding costs depend on source and destination parallelism, frequency changes cost next to nothing].
//
// Per (scenario, class) this is a shortest path through the windows: a state is a sharding sigma = (n, TP),
// the cost of a state in a window is the least energy over the candidate frequencies (the evaluation of Eq. 1),
// a move sigma' -> sigma between consecutive windows costs R[sigma'][sigma] (the caller's table, Wh).
//   reconf_cost_kernel  cost[s][c][w][sigma] and the frequency that attains it: one thread per entry, a warp
//                       covers 32 shardings of one tile (one load, the table rows of T degrees), F evaluations each
//   reconf_cost_fast_kernel  the same on the threshold tables in shared memory, the form the sweep uses: a warp takes a
//                       tile, lanes hold instance counts, the (TP, f) pairs are the inner loop (packed evaluation of
//                       two counts), the frequency is noted whenever the running minimum falls; classes with a row
//                       that has no load threshold are evaluated as in reconf_cost_kernel
//   reconf_path_kernel  one CTA per (scenario, class): forward recursion over the windows (min-plus product of the
//                       state vector with R: add + min per step; R in shared memory as far as it fits, the state
//                       vector too), the vectors written to global memory.  The running values are kept relative
//                       to their minimum, which is accumulated in fp64, so that fp32 holds only differences.
//   reconf_back_kernel  the walk back, one warp per (scenario, class): it finds each predecessor again with the
//                       same addition (lowest source on ties) and writes the chosen candidates.
#define DYN_TU_ID 10
#include "dyn_internal.cuh"
#include "eval_dev.cuh"

#include <cuda_pipeline.h>
#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kThreads = 256;

struct ReconfArgs {
    const float4 *rows;       // [C][P][M+1]
    const float2 *pairc;      // [C][P]
    const float *slo;         // [C]
    const int32_t *tp;        // [T]
    const float *R;           // [NS][NS]
    float *Rt;                // [NS][NS] transposed copy: Rt[g][h] = R[h][g] (the walk back reads columns of R)
    const float *load;        // [S][W][C]
    float *cost;              // [S][C][W][NS]
    uint8_t *qbest;           // [S][C][W][NS]
    float *hist;              // [S][C][W][NS] running values relative to their minimum, window by window
    int64_t S, W;
    int32_t C, T, F, M, Nmax, NS, budget;
    int32_t *best_idx;
    float *best_E;
    double *path_total;       // [S][C]
    const char *ws;           // scratch block (threshold tables at off_pair2 .. off_end)
    int32_t off_pair2, off_rows2, off_end;
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
        const float L = fmaxf(a.load[DYN_IDX((s * a.W + w) * a.C + c, a.S * a.W * a.C)], 0.f);
        const float nf = float(n), ln = L * (1.0f / nf);
        const float slo = a.slo[c];
        float best = CUDART_INF_F;
        int bq = 0;
        if (a.budget <= 0 || int64_t(n) * a.tp[t] <= int64_t(a.budget)) {
            const float4 *rows_t = a.rows + size_t(DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1)) * RS;
            const float2 *pc_t = a.pairc + DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1);
            for (int q = 0; q < a.F; ++q) {
                bool ok;
                const float E = eval_pair(rows_t + size_t(q) * RS, __ldg(pc_t + q).x, Mf, ln, nf, slo, ok);
                if (ok && E < best) {                        // ascending q: strict compare keeps the lowest
                    best = E;
                    bq = q;
                }
            }
        }
        a.cost[DYN_IDX(e, total)] = best;
        a.qbest[DYN_IDX(e, total)] = uint8_t(bq);
    }
}

// one entry of the cost tensor from the general-path tables (any class)
__device__ __forceinline__ void cost_entry_general(const ReconfArgs &a, int c, float L, int g, float &best, int &bq) {
    const int P = a.T * a.F, RS = a.M + 1;
    const int n = g / a.T + 1, t = g - (n - 1) * a.T;
    const float nf = float(n), ln = L * (1.0f / nf);
    const float slo = a.slo[c];
    best = CUDART_INF_F;
    bq = 0;
    if (a.budget <= 0 || int64_t(n) * a.tp[t] <= int64_t(a.budget)) {
        const float4 *rows_t = a.rows + size_t(DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1)) * RS;
        const float2 *pc_t = a.pairc + DYN_IDX(c * P + t * a.F, a.C * P - a.F + 1);
        for (int q = 0; q < a.F; ++q) {
            bool ok;
            const float E = eval_pair(rows_t + size_t(q) * RS, __ldg(pc_t + q).x, float(a.M), ln, nf, slo, ok);
            if (ok && E < best) {                            // ascending q: strict compare keeps the lowest
                best = E;
                bq = q;
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) reconf_cost_fast_kernel(const ReconfArgs a, const int table_bytes) {
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
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = kThreads / 32;
    const int NS = a.NS, NS4 = (NS + 3) & ~3;
    // this warp's results of a tile: NS costs, then NS frequencies
    float *oc = reinterpret_cast<float *>(reinterpret_cast<char *>(smem) + table_bytes) + size_t(warp) * NS4;
    unsigned char *oq = reinterpret_cast<unsigned char *>(reinterpret_cast<float *>(reinterpret_cast<char *>(smem) + table_bytes) +
                                                          size_t(warps) * NS4) + size_t(warp) * NS4;
    const int F = a.F, T = a.T, P = T * F, RS = a.M + 1;
    const uint32_t pstep = uint32_t(RS) * 8u;
    const uint32_t rows2 = origin + uint32_t(a.off_rows2 - a.off_pair2);
    const uint64_t two23_2 = pack2(kTwo23, kTwo23);
    const uint64_t eight2 = pack2(units(8u), units(8u));
    const float offs = float(int(pstep)) * units(1u);
    const uint64_t off2_step = pack2(offs, offs);
    const int64_t tiles = a.S * a.C * a.W;
    for (int64_t i = int64_t(blockIdx.x) * warps + warp; i < tiles; i += int64_t(gridDim.x) * warps) {
        const int64_t w = i % a.W, sc = i / a.W;
        const int c = int(sc % a.C);
        const int64_t s = sc / a.C;
        const float L = fmaxf(a.load[DYN_IDX((s * a.W + w) * a.C + c, a.S * a.W * a.C)], 0.f);
        float *cost_i = a.cost + i * NS;
        uint8_t *q_i = a.qbest + i * NS;
        if (s_general[c]) {                                  // warp-uniform
            for (int g = lane; g < NS; g += 32) {
                float best;
                int bq;
                cost_entry_general(a, c, L, g, best, bq);
                cost_i[DYN_IDX(g, NS)] = best;
                q_i[DYN_IDX(g, NS)] = uint8_t(bq);
            }
            continue;
        }
        for (int k0 = 0; k0 < a.Nmax; k0 += 64) {
            const int nA = k0 + lane + 1, nB = nA + 32;
            const bool inA = nA <= a.Nmax, inB = nB <= a.Nmax;
            const float nfA = float(nA), nfB = float(nB);
            const uint64_t ln2 = pack2(inA ? L * (1.0f / nfA) : CUDART_INF_F, inB ? L * (1.0f / nfB) : CUDART_INF_F);
            for (int t = 0; t < T; ++t) {
                const int tpt = __ldg(a.tp + t);
                const bool okA = inA && (a.budget <= 0 || int64_t(nA) * tpt <= int64_t(a.budget));
                const bool okB = inB && (a.budget <= 0 || int64_t(nB) * tpt <= int64_t(a.budget));
                float eA = CUDART_INF_F, eB = CUDART_INF_F;
                int qA = 0, qB = 0;
                const uint32_t cpair = origin + uint32_t(c * P + t * F) * 16u;
                const float off0 = row_offset_units(rows2 + uint32_t((c * P + t * F) * RS) * 8u);
                uint64_t off2 = pack2(off0, off0);
#pragma unroll 4
                for (int q = 0; q < F; ++q) {
                    uint64_t icm2, lim2;
                    asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(icm2), "=l"(lim2) : "r"(DYN_SMEM_ADDR(cpair + uint32_t(q) * 16u, 16u)));
                    const float lim = __uint_as_float(uint32_t(lim2));
                    const float pA = eA, pB = eB;
                    fast_two(ln2, icm2, off2, two23_2, eight2, okA ? lim : -1.f, okB ? lim : -1.f, eA, eB);
                    qA = eA < pA ? q : qA;                   // ascending q: the lowest frequency that attains the minimum
                    qB = eB < pB ? q : qB;
                    off2 = add2(off2, off2_step);
                }
                if (inA) {
                    oc[DYN_IDX((nA - 1) * T + t, NS4)] = nfA * eA;           // +inf where no frequency is feasible
                    oq[DYN_IDX((nA - 1) * T + t, NS4)] = (unsigned char)qA;
                }
                if (inB) {
                    oc[DYN_IDX((nB - 1) * T + t, NS4)] = nfB * eB;
                    oq[DYN_IDX((nB - 1) * T + t, NS4)] = (unsigned char)qB;
                }
            }
        }
        __syncwarp();
        for (int g = lane; g < NS; g += 32) {
            cost_i[DYN_IDX(g, NS)] = oc[g];
            q_i[DYN_IDX(g, NS)] = oq[g];
        }
        __syncwarp();                                        // the tile is out before the next one overwrites it
    }
}

// smallest of three (one instruction on this architecture; exact, so equal to two nested minima)
__device__ __forceinline__ float min3f(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Two sources A, B (their values, relative to the minimum, in d) against the running minima of four neighbouring
// targets.  v0 = {R[A][t0], R[B][t0], R[A][t1], R[B][t1]}, v1 the same for t2, t3: a packed addition forms both
// sums of a target (each the same round-to-nearest sum as a single addition), one three-input minimum takes them in
__device__ __forceinline__ void relax_pair(float &b0, float &b1, float &b2, float &b3, const float2 d, const float4 v0,
                                           const float4 v1) {
    const float2 s0 = __fadd2_rn(d, make_float2(v0.x, v0.y)), s1 = __fadd2_rn(d, make_float2(v0.z, v0.w));
    const float2 s2 = __fadd2_rn(d, make_float2(v1.x, v1.y)), s3 = __fadd2_rn(d, make_float2(v1.z, v1.w));
    b0 = min3f(b0, s0.x, s0.y);
    b1 = min3f(b1, s1.x, s1.y);
    b2 = min3f(b2, s2.x, s2.y);
    b3 = min3f(b3, s3.x, s3.y);
}

constexpr int kPathThreads = 256;
constexpr int kRegRows = 40;                    // rows of R a thread keeps in registers (its four columns of them); whole quads
constexpr int kOwn = 4;                         // entries of the state vector a thread owns outside the scan (NS <= 1024)

// R[h][g]: rows_s rows sit in shared memory, NS4 + 4 floats per row (NS4 = NS rounded up to a multiple of 4; the
// pieces stay 16-byte aligned), pairs of rows interleaved as described at the copy loop
// One CTA per (scenario, class).  Dynamic shared memory: Dp[NS4] | part[G][NS4] | rlo[NS4] | Rs[rows_s / 2][2][NS4 + 4].
// Sources that cannot attain any minimum are skipped, four at a time: with a reference state h0 every target g has
// min_h (D(h) + R[h][g]) <= D(h0) + R[h0][g] <= D(h0) + max_g R[h0][g] =: bound, while source h offers at least
// D(h) + min_g R[h][g] =: D(h) + rlo(h); a quad of sources whose four values D(h) + rlo(h) all exceed the bound is not
// scanned (rounding is monotone, so the comparison of the rounded sums decides the same way as the exact one would for
// the rounded candidates: the minima formed are bit for bit those of the full scan).  h0 is the state that attained
// the last gathered minimum; any state gives a valid bound.  Where transitions cost little next to the spread of the
// window costs over the shardings -- the regime of the paper's overhead table -- most quads are skipped; with a
// prohibitive table none is, and the test costs a few instructions per quad.
// Forward: D_w(g) = cost_w(g) + min_h (D_{w-1}(h) + R[h][g]).  Only the minimum is formed here (half a packed add and half a three-input min per
// step): a thread takes four neighbouring targets and a share of the sources, four sources per trip (one 16-byte
// read of the state vector, four of R).  The values D_{w-1}, as held (relative to the running base), are written to `hist`,
// and the walk back finds each predecessor again as the lowest h that attains the minimum, with the same addition.
__global__ void __launch_bounds__(kPathThreads) reconf_path_kernel(const ReconfArgs a, const int rows_s) {
    extern __shared__ float4 smem4[];
    const int NS = a.NS, NS4 = (NS + 3) & ~3, RSd = NS4 + 4;
    const int TG = NS4 / 4;                                  // groups of four targets
    const int lanes_t = (TG + 31) / 32 * 32;                 // threads side by side over the target groups (<= 256)
    const int G = kPathThreads / lanes_t;                    // thread groups that split the sources
    float *Dp = reinterpret_cast<float *>(smem4);
    float *part = Dp + NS4;
    float *rlo = part + size_t(G) * NS4;                   // [NS4] least entry of every row of R (+inf past NS)
    float *Rs = rlo + NS4;
    __shared__ float s_rhi[1024];                            // largest entry of every row of R (NS <= 1024)
    const int64_t sc = blockIdx.x;                           // s * C + c
    const int64_t W = a.W;
    const float *cost = a.cost + sc * W * NS;
    float *hist = a.hist + sc * W * NS;
    const int tid = threadIdx.x;
    const int hg = tid / lanes_t, tg = tid - hg * lanes_t;
    const bool worker = hg < G && tg < TG;
    const int SQ = rows_s / 4;                               // quads of rows held in shared memory
    const int q_lo = int(int64_t(hg) * SQ / G), q_hi = worker ? int(int64_t(hg + 1) * SQ / G) : q_lo;   // this group's share

    // rows A = 2k and B = 2k + 1 are interleaved (a packed addition takes {R[A][g], R[B][g]}): per pair of rows two
    // planes of RSd floats, plane 0 holding {R[A][t0], R[B][t0], R[A][t1], R[B][t1]} of every group of four targets
    // t0..t3 and plane 1 the same for t2, t3, so that the lanes of a warp read neighbouring 16-byte pieces
    for (int i = tid; i < rows_s * RSd; i += kPathThreads) {
        const int h = i / RSd, g = i - h * RSd, j = g & 3;
        Rs[DYN_IDX(size_t(h >> 1) * (2 * RSd) + (j >> 1) * RSd + (g & ~3) + (j & 1) * 2 + (h & 1), size_t(rows_s) * RSd)] =
            g < NS ? a.R[DYN_IDX(size_t(h) * NS + g, size_t(NS) * NS)] : 0.f;
    }
    // least and largest entry of every row: a warp per row, lanes across it
    for (int h = tid >> 5; h < NS4; h += kPathThreads / 32) {
        float lo = CUDART_INF_F, hi = -CUDART_INF_F;
        if (h < NS)
            for (int g = tid & 31; g < NS; g += 32) {
                const float v = __ldg(a.R + DYN_IDX(size_t(h) * NS + g, size_t(NS) * NS));
                lo = fminf(lo, v);
                hi = fmaxf(hi, v);
            }
        float wlo, whi;
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(wlo) : "f"(lo));
        asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(whi) : "f"(hi));
        if ((tid & 31) == 0) {
            rlo[h] = wlo;                                    // +inf past NS: such a source is never scanned
            if (h < 1024) s_rhi[h] = whi;
        }
    }
    // rows of R that do not fit in shared memory: the first G * kRegRows of them stay in registers, each source
    // group holding kRegRows rows (its four columns of them); any further rows are read through L1 / L2
    float4 rp0[kRegRows / 2], rp1[kRegRows / 2];             // per pair of rows, interleaved like the shared-memory copy
    const int h_reg = rows_s + hg * kRegRows;                // this group's first register row (a multiple of 4)
#pragma unroll
    for (int k = 0; k < kRegRows / 2; ++k) {
        float v[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int h = h_reg + 2 * k + i;
            const bool have = worker && h < NS;              // no such row: +inf never wins
            const float *row = a.R + size_t(h) * NS + 4 * tg;
#pragma unroll
            for (int j = 0; j < 4; ++j) v[i][j] = have ? (4 * tg + j < NS ? __ldg(DYN_PTR(row + j, a.R, int64_t(NS) * NS)) : 0.f) : CUDART_INF_F;
        }
        rp0[k] = make_float4(v[0][0], v[1][0], v[0][1], v[1][1]);
        rp1[k] = make_float4(v[0][2], v[1][2], v[0][3], v[1][3]);
    }
    const int rows_sr = rows_s + G * kRegRows;               // rows below this are in shared memory or registers
    // the rest, split evenly over the source groups
    const int n_rest = NS > rows_sr ? NS - rows_sr : 0;
    const int g_lo = rows_sr + int(int64_t(hg) * n_rest / G), g_hi = worker ? rows_sr + int(int64_t(hg + 1) * n_rest / G) : g_lo;
    // Two barriers per window.  Dp holds the vector of the previous window as computed.  Its minimum and a state that
    // attains it are gathered without atomics: every warp leaves the minimum of its threads' entries and where it
    // sits in a slot of its own, and at the start of the next window every thread takes the least of the
    // kPathThreads / 32 slots.  The minimum comes off the vector of the window after (one window late); the state is
    // the reference of the bound that lets the scan skip sources.  A thread owns entries tid, tid + kPathThreads, ...
    // (kOwn of them) of the vector outside the scan and writes them to `hist` as it forms them.  Padding entries past
    // NS are sources that never win: +inf.
    constexpr int kPW = kPathThreads / 32;
    __shared__ __align__(16) float s_wmin[kPW];
    __shared__ __align__(16) int s_warg[kPW];
    auto publish_min = [&](float lmin, int larg) {           // larg: an entry of this thread that holds lmin (any valid state if none)
        float wm;
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(wm) : "f"(lmin));
        if (lmin == wm) {                                    // some lane holds it (no NaNs here); any of them will do
            s_wmin[tid >> 5] = wm;
            s_warg[tid >> 5] = larg;
        }
    };
    auto gathered_min = [&](int &arg) {                      // least slot (the lowest warp among equals) and its state
        float m = s_wmin[0];
        arg = s_warg[0];
#pragma unroll
        for (int k = 1; k < kPW; ++k) {
            const float v = s_wmin[k];
            if (v < m) {
                m = v;
                arg = s_warg[k];
            }
        }
        return m;
    };
    __syncthreads();
    double base = 0.0;
    {
        float lmin = CUDART_INF_F;
        int larg = 0;
        for (int g = tid; g < NS4; g += kPathThreads) {
            const float v = g < NS ? (W > 0 ? cost[g] : 0.f) : CUDART_INF_F;
            Dp[g] = v;
            if (g < NS && W > 0) hist[g] = v;                // row 0: the first window's vector as held
            if (v < lmin) {
                lmin = v;
                larg = g;
            }
        }
        publish_min(lmin, larg);
    }
    // The window costs come from DRAM: a thread loads its own entries of the NEXT window at the start of a window and
    // uses them a whole window later, so the recursion does not wait for memory.
    float cnow[kOwn], cnext[kOwn];
#pragma unroll
    for (int o = 0; o < kOwn; ++o) {
        const int g = tid + o * kPathThreads;
        cnow[o] = (g < NS && W > 1) ? __ldg(cost + NS + g) : 0.f;
        cnext[o] = 0.f;
    }
    __syncthreads();                                         // publishes Dp, the minimum and Rs
    for (int64_t w = 1; w < W; ++w) {
        // keep differences only: the minimum of the previous vector goes to the fp64 base (all +inf stays +inf) and
        // is taken off the vector computed in this window
        int h0;
        const float mprev = gathered_min(h0);
        const float shift = (mprev < CUDART_INF_F) ? mprev : 0.f;
        base += double(shift);
        const float bound = mprev + s_rhi[DYN_IDX(h0, 1024)];               // D(h0) = mprev
        if (w + 1 < W) {
#pragma unroll
            for (int o = 0; o < kOwn; ++o) {
                const int g = tid + o * kPathThreads;
                if (g < NS) cnext[o] = __ldg(cost + DYN_IDX((w + 1) * NS + g, W * NS));
            }
        }
        auto quad_live = [&](int qd) {                       // some source of quad qd can still attain a minimum
            const float4 d4 = reinterpret_cast<const float4 *>(Dp)[DYN_IDX(qd, TG)];
            const float4 m4 = reinterpret_cast<const float4 *>(rlo)[DYN_IDX(qd, TG)];
            return fminf(fminf(d4.x + m4.x, d4.y + m4.y), fminf(d4.z + m4.z, d4.w + m4.w)) <= bound;
        };
        // which quads of this warp's source group are live: one lane per quad, gathered by a vote (bit b of live_s:
        // shared-memory quad q_lo + b, the first 32 of them; bit j of live_r: register quad j)
        uint32_t live_s = 0xffffffffu, live_r = 0xffffffffu;
        if (hg < G) {                                        // the same in every thread of a warp
            const int lane = tid & 31;
            const int nsm = int(int64_t(hg + 1) * SQ / G) - q_lo;
            if (nsm + kRegRows / 4 <= 32) {
                // one vote serves both kinds: lanes 0 .. nsm-1 the shared-memory quads, the next ten the register quads
                const int jr = lane - nsm;
                const int qd = lane < nsm ? q_lo + lane : h_reg / 4 + jr;
                const bool have = lane < nsm || (jr < kRegRows / 4 && qd < TG);
                const uint32_t bal = __ballot_sync(0xffffffffu, quad_live(have ? qd : 0) && have);
                live_s = bal & ((1u << nsm) - 1u);
                live_r = (bal >> nsm) & ((1u << (kRegRows / 4)) - 1u);
            } else {
                live_s = __ballot_sync(0xffffffffu, lane < nsm && quad_live(q_lo + lane));
                const int hq = h_reg / 4 + lane;
                live_r = __ballot_sync(0xffffffffu, lane < kRegRows / 4 && hq < TG && quad_live(hq));
            }
        }
        if (worker) {
            float b0 = CUDART_INF_F, b1 = CUDART_INF_F, b2 = CUDART_INF_F, b3 = CUDART_INF_F;
            // only the live quads are visited: the set bits of the votes, then any shared-memory quads beyond the 32
            // a vote covers (those are scanned in full)
            for (uint32_t m = live_s; m; m &= m - 1u) {
                const int q = q_lo + __ffs(int(m)) - 1;
                const float4 d4 = reinterpret_cast<const float4 *>(Dp)[DYN_IDX(q, TG)];
                const float *rq = Rs + DYN_IDX(size_t(2 * q) * (2 * RSd) + 4 * tg, size_t(rows_s) * RSd - 3 * RSd - 3);
                relax_pair(b0, b1, b2, b3, make_float2(d4.x, d4.y), *reinterpret_cast<const float4 *>(rq),
                           *reinterpret_cast<const float4 *>(rq + RSd));
                relax_pair(b0, b1, b2, b3, make_float2(d4.z, d4.w), *reinterpret_cast<const float4 *>(rq + 2 * RSd),
                           *reinterpret_cast<const float4 *>(rq + 3 * RSd));
            }
#pragma unroll 1
            for (int q = q_lo + 32; q < q_hi; ++q) {
                const float4 d4 = reinterpret_cast<const float4 *>(Dp)[DYN_IDX(q, TG)];
                const float *rq = Rs + DYN_IDX(size_t(2 * q) * (2 * RSd) + 4 * tg, size_t(rows_s) * RSd - 3 * RSd - 3);
                relax_pair(b0, b1, b2, b3, make_float2(d4.x, d4.y), *reinterpret_cast<const float4 *>(rq),
                           *reinterpret_cast<const float4 *>(rq + RSd));
                relax_pair(b0, b1, b2, b3, make_float2(d4.z, d4.w), *reinterpret_cast<const float4 *>(rq + 2 * RSd),
                           *reinterpret_cast<const float4 *>(rq + 3 * RSd));
            }
            // register quads: a jump per live quad into the code that names its registers
            static_assert(kRegRows == 40, "ten register quads are spelled out below");
            for (uint32_t m = live_r; m; m &= m - 1u) {
                const int j4 = __ffs(int(m)) - 1;
                const float4 d4 = reinterpret_cast<const float4 *>(Dp)[DYN_IDX(h_reg / 4 + j4, TG)];
                const float2 dA = make_float2(d4.x, d4.y), dB = make_float2(d4.z, d4.w);
                switch (j4) {
#define DYN_REG_QUAD(J)                                              \
    case J:                                                          \
        relax_pair(b0, b1, b2, b3, dA, rp0[2 * J], rp1[2 * J]);         \
        relax_pair(b0, b1, b2, b3, dB, rp0[2 * J + 1], rp1[2 * J + 1]); \
        break;
                    DYN_REG_QUAD(0) DYN_REG_QUAD(1) DYN_REG_QUAD(2) DYN_REG_QUAD(3) DYN_REG_QUAD(4)
                    DYN_REG_QUAD(5) DYN_REG_QUAD(6) DYN_REG_QUAD(7) DYN_REG_QUAD(8) DYN_REG_QUAD(9)
#undef DYN_REG_QUAD
                    default: break;
                }
            }
            for (int h = g_lo; h < g_hi; ++h) {
                const float d = Dp[h];
                if (!(d + rlo[h] <= bound)) continue;
                const float *row = a.R + size_t(h) * NS + 4 * tg;
                b0 = fminf(b0, d + __ldg(row));
                if (4 * tg + 1 < NS) b1 = fminf(b1, d + __ldg(row + 1));
                if (4 * tg + 2 < NS) b2 = fminf(b2, d + __ldg(row + 2));
                if (4 * tg + 3 < NS) b3 = fminf(b3, d + __ldg(row + 3));
            }
            reinterpret_cast<float4 *>(part + size_t(DYN_IDX(hg, G)) * NS4)[DYN_IDX(tg, TG)] = make_float4(b0, b1, b2, b3);
        }
        __syncthreads();                                     // every reader of Dp is done; the partial minima are in
        float lmin = CUDART_INF_F;
        int larg = 0;
#pragma unroll
        for (int o = 0; o < kOwn; ++o) {
            const int g = tid + o * kPathThreads;
            if (g < NS) {
                float best = part[DYN_IDX(g, NS4)];               // G is 1, 2, 4 or 8: independent loads
                if (G >= 2) best = fminf(best, part[DYN_IDX(NS4 + g, G * NS4)]);
                if (G >= 4) best = min3f(best, part[DYN_IDX(2 * NS4 + g, G * NS4)], part[DYN_IDX(3 * NS4 + g, G * NS4)]);
                if (G >= 8)
                    best = fminf(min3f(best, part[DYN_IDX(4 * NS4 + g, G * NS4)], part[DYN_IDX(5 * NS4 + g, G * NS4)]),
                                 fminf(part[DYN_IDX(6 * NS4 + g, G * NS4)], part[DYN_IDX(7 * NS4 + g, G * NS4)]));
                // the minimum of the PREVIOUS vector comes off here, one window late: one subtraction per entry
                // instead of one per source in the scan; the values stay within two windows' growth of zero
                const float d = (cnow[o] + best) - shift;
                Dp[DYN_IDX(g, NS4)] = d;
                hist[DYN_IDX(w * NS + g, W * NS)] = d;       // the vector as held: the walk back reads it
                if (d < lmin) {
                    lmin = d;
                    larg = g;
                }
            }
        }
        publish_min(lmin, larg);
#pragma unroll
        for (int o = 0; o < kOwn; ++o) cnow[o] = cnext[o];
        __syncthreads();                                     // publishes Dp and the minimum
    }
    int h_last;
    const float m = W > 0 ? gathered_min(h_last) : 0.f;      // minimum of the last vector (relative to `base`)
    if (W == 0) {
        if (tid == 0) a.path_total[sc] = 0.0;
        return;
    }
    // (every window's vector, the last one included, went to `hist` as it was formed; the walk back starts at the last)
    if (tid == 0) a.path_total[sc] = (m < CUDART_INF_F) ? base + double(m) : double(CUDART_INF_F);
}

// The walk back: one warp per (scenario, class), four of them per CTA.  At window w in state g the predecessor is
// the lowest h that attains min_h hist[w-1][h] + R[h][g] (the same addition as in the forward scan).  R is read
// from a transposed copy (a column of R is then one contiguous row) through L1.  With at most 256 states
// a lane keeps its eight entries of the vectors of the next eight windows in registers: they do not depend on the
// state, and asking for them eight steps ahead hides the memory latency of the walk.  The states of a stretch of
// windows are noted in shared memory, then the lanes write the results of those windows side by side.
__global__ void reconf_transpose_kernel(const ReconfArgs a) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= int64_t(a.NS) * a.NS) return;
    const int g = int(i / a.NS), h = int(i - int64_t(g) * a.NS);
    a.Rt[i] = a.R[DYN_IDX(size_t(h) * a.NS + g, size_t(a.NS) * a.NS)];
}

constexpr int kBackWarps = 1;
constexpr int kBackThreads = 256;               // threads of a CTA: all copy the table, one warp walks
constexpr int kBackChunk = 512;                 // windows per stretch
constexpr int kBackRing = 12;                   // windows whose vectors are on their way into shared memory

__global__ void __launch_bounds__(kBackThreads) reconf_back_kernel(const ReconfArgs a, const int rows_b) {
    __shared__ int path_all[kBackWarps][kBackChunk];
    extern __shared__ float4 smem4[];
    const int NS = a.NS;
    // the first rows_b rows of the transposed table (columns of R) in shared memory: the walk reads one of them per
    // window, and which one is known only when the previous window is done
    float *Rts = reinterpret_cast<float *>(smem4);
    if ((NS & 3) == 0) {
        const float4 *src = reinterpret_cast<const float4 *>(a.Rt);
        for (int i = threadIdx.x; i < rows_b * (NS / 4); i += kBackThreads) smem4[i] = __ldg(src + i);
    } else {
        for (int i = threadIdx.x; i < rows_b * NS; i += kBackThreads) Rts[i] = __ldg(a.Rt + i);
    }
    __syncthreads();
    if (threadIdx.x >= kBackWarps * 32) return;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const int64_t sc = int64_t(blockIdx.x) * kBackWarps + wi;
    if (sc >= a.S * a.C) return;
    int *path = path_all[wi];
    const int c = int(sc % a.C);
    const int64_t s = sc / a.C;
    const int64_t W = a.W;
    if (W == 0) return;
    const float *cost = a.cost + sc * W * NS;
    const float *hist = a.hist + sc * W * NS;
    const float *Rt = a.Rt;
    // last state: the lowest g that attains the minimum of the final vector
    int cur = -1;
    {
        float best = CUDART_INF_F;
        uint32_t arg = 0xffffffffu;
        for (int g = lane; g < NS; g += 32) {
            const float v = hist[(W - 1) * NS + g];
            if (v < best) {
                best = v;
                arg = uint32_t(g);
            }
        }
        float mm;
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(mm) : "f"(best));
        if (mm < CUDART_INF_F) cur = int(__reduce_min_sync(0xffffffffu, best == mm ? arg : 0xffffffffu));
    }
    // With at most 256 states a lane owns eight entries h = lane + 32 j of every vector.  The vectors of the next
    // kBackRing windows do not depend on the state: a lane asks for its own entries that many windows ahead with
    // asynchronous copies into a ring in shared memory and later reads only what it copied itself, so no barrier
    // is needed and the walk does not wait for DRAM.  (Loads into registers that far ahead do not work: a warp
    // can wait only for all of its outstanding loads at once.)
    const bool ahead = NS <= 256;
    float *ring = Rts + size_t(rows_b) * NS;                 // [kBackRing][256]
    auto ask = [&](int64_t row, int slot) {                  // entries of vector `row` (clamped; rows < 0 are never used)
        const float *src = hist + DYN_IDX(row > 0 ? row : 0, W) * NS;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (lane + 32 * j < NS) __pipeline_memcpy_async(ring + DYN_IDX(slot, kBackRing) * 256 + lane + 32 * j, src + lane + 32 * j, 4);
        __pipeline_commit();
    };
    if (ahead)
        for (int k = 0; k < kBackRing; ++k) ask(W - 2 - k, k);         // slot k: the vector used at window W-1-k
    // the column of R that leads into the current state (a row of the transposed copy), a lane's eight entries of
    // it: it is read again only when the state changes
    float rcol[8];
    int rcol_of = -1;
    int64_t seg_hi = W;                                      // windows [w, seg_hi) are noted in path[seg_hi - 1 - w]
    int slot = 0;
    for (int64_t wb = W - 1; wb >= 0; wb -= 8) {
#pragma unroll 1
        for (int k = 0; k < 8; ++k) {
            const int64_t w = wb - k;
            if (w >= 0) {
                if (lane == 0) path[DYN_IDX(seg_hi - 1 - w, kBackChunk)] = cur;
                if (ahead) __pipeline_wait_prior(kBackRing - 1);        // this window's vector has arrived
                if (cur >= 0 && w > 0) {
                    float mm;
                    uint32_t arg = 0xffffffffu;
                    if (ahead) {
                        if (rcol_of != cur) {                // warp-uniform
                            const float *col = cur < rows_b ? Rts + size_t(cur) * NS : Rt + size_t(DYN_IDX(cur, NS)) * NS;
#pragma unroll
                            for (int j = 0; j < 8; ++j) rcol[j] = lane + 32 * j < NS ? col[lane + 32 * j] : CUDART_INF_F;
                            rcol_of = cur;
                        }
                        float v[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = lane + 32 * j < NS ? ring[slot * 256 + lane + 32 * j] + rcol[j] : CUDART_INF_F;
                        const float best = fminf(min3f(min3f(v[0], v[1], v[2]), v[3], v[4]), min3f(v[5], v[6], v[7]));
                        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(mm) : "f"(best));
                        // lowest h that attains the minimum: descending j, so the lowest matching entry stays
#pragma unroll
                        for (int j = 7; j >= 0; --j) arg = (v[j] == mm) ? uint32_t(lane + 32 * j) : arg;
                    } else {
                        float best = CUDART_INF_F;
                        const float *hp = hist + (w - 1) * NS;
                        for (int h = lane; h < NS; h += 32) {
                            const float x = hp[h] + __ldg(Rt + size_t(cur) * NS + h);
                            if (x < best) {              // ascending h per lane: strict compare keeps the lowest
                                best = x;
                                arg = uint32_t(h);
                            }
                        }
                        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(mm) : "f"(best));
                        if (best != mm) arg = 0xffffffffu;
                    }
                    cur = int(__reduce_min_sync(0xffffffffu, arg));
                }
                if (ahead) {                                 // the slot is free: the vector used kBackRing windows further down
                    ask(w - 1 - kBackRing, slot);
                    slot = slot + 1 == kBackRing ? 0 : slot + 1;
                }
            }
        }
        const int64_t lo = wb - 7 > 0 ? wb - 7 : 0;          // lowest window handled so far
        if (seg_hi - lo >= kBackChunk || lo == 0) {
            __syncwarp();
            for (int64_t w = lo + lane; w < seg_hi; w += 32) {
                const int g = path[DYN_IDX(seg_hi - 1 - w, kBackChunk)];
                const int64_t i = DYN_IDX((s * W + w) * a.C + c, a.S * W * a.C);
                if (g >= 0) {
                    a.best_idx[i] = g * a.F + int(a.qbest[DYN_IDX(sc * W * NS + w * NS + g, a.S * a.C * W * NS)]);
                    a.best_E[i] = cost[DYN_IDX(w * NS + g, W * NS)];
                } else {
                    a.best_idx[i] = -1;
                    a.best_E[i] = CUDART_INF_F;
                }
            }
            __syncwarp();
            seg_hi = lo;
        }
    }
}

}  // namespace

// rows of R kept in shared memory for NS states, given the device's limit
static size_t reconf_fixed_floats(int32_t NS) {
    const int NS4 = (NS + 3) & ~3, TG = NS4 / 4, lanes_t = (TG + 31) / 32 * 32, G = kPathThreads / lanes_t;
    return size_t(1 + G + 1) * NS4;
}
static int reconf_rows_in_smem(int32_t NS, size_t limit) {
    const int NS4 = (NS + 3) & ~3;
    const size_t fixed = reconf_fixed_floats(NS) * sizeof(float) + 6144;      // the kernel's static shared memory on top
    if (limit <= fixed) return 0;
    int64_t rows = int64_t((limit - fixed) / (size_t(NS4 + 4) * sizeof(float)));
    // the registers come first (no shared-memory traffic): shared memory holds what they leave
    const int TG = NS4 / 4, lanes_t = (TG + 31) / 32 * 32, G = kPathThreads / lanes_t;
    const int64_t left = NS4 > G * kRegRows ? NS4 - G * kRegRows : 0;
    if (rows > left) rows = left;
    return int(rows) & ~3;                                   // whole quads of rows
}

cudaError_t launch_reconf(const ResolvedLayout &lay, void *d_ws, size_t off_cost, size_t off_q, size_t off_from, size_t off_rt,
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
    a.hist = reinterpret_cast<float *>(ws + off_from);
    a.Rt = reinterpret_cast<float *>(ws + off_rt);
    a.S = S; a.W = W;
    a.C = lay.C; a.T = lay.T; a.F = lay.F; a.M = lay.M; a.Nmax = lay.Nmax; a.NS = lay.Nmax * lay.T; a.budget = budget;
    a.best_idx = best_idx; a.best_E = best_E; a.path_total = path_total;
    if (S == 0) return cudaSuccess;
    reconf_transpose_kernel<<<unsigned((int64_t(a.NS) * a.NS + 255) / 256), 256, 0, st>>>(a);
    const int64_t total = S * lay.C * W * a.NS;
    if (total > 0) {
        int64_t grid = (total + kThreads - 1) / kThreads;
        const int64_t cap = int64_t(sm_count()) * 16;
        if (grid > cap) grid = cap;
        // threshold tables and a tile's results per warp in shared memory when they fit
        const size_t table_bytes = lay.off_tp - lay.off_pair2;
        const int NS4c = (a.NS + 3) & ~3;
        const size_t fast_smem = table_bytes + size_t(kThreads / 32) * NS4c * (sizeof(float) + 1);
        cudaError_t e;
        if (fast_smem <= 96 * 1024 && lay.F <= 256) {
            a.ws = ws;
            a.off_pair2 = int32_t(lay.off_pair2); a.off_rows2 = int32_t(lay.off_rows2); a.off_end = int32_t(lay.off_tp);
            if ((e = cudaFuncSetAttribute(reconf_cost_fast_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(fast_smem))) != cudaSuccess)
                return e;
            int64_t g2 = (S * lay.C * W + kThreads / 32 - 1) / (kThreads / 32);
            const int64_t cap2 = int64_t(sm_count()) * 4;
            if (g2 > cap2) g2 = cap2;
            reconf_cost_fast_kernel<<<unsigned(g2), kThreads, fast_smem, st>>>(a, int(table_bytes));
        } else {
            reconf_cost_kernel<<<unsigned(grid), kThreads, 0, st>>>(a);
        }
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    int dev = 0, lim = 48 * 1024;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (cudaDeviceGetAttribute(&lim, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) lim = 48 * 1024;
    const int rows_s = reconf_rows_in_smem(a.NS, size_t(lim));
    const int NS4 = (a.NS + 3) & ~3;
    const size_t smem = (reconf_fixed_floats(a.NS) + size_t(rows_s) * (NS4 + 4)) * sizeof(float) + 16;
    e = cudaFuncSetAttribute(reconf_path_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    e = record_start(st);
    if (e != cudaSuccess) return e;
    reconf_path_kernel<<<unsigned(S * lay.C), kPathThreads, smem, st>>>(a, rows_s);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    {
        // as many columns of R as fit beside the kernel's static shared memory
        const size_t ring_b = size_t(kBackRing) * 256 * sizeof(float);
        const size_t room = size_t(lim) > 8192 + ring_b ? size_t(lim) - 8192 - ring_b : 0;
        int rows_b = int(room / (size_t(a.NS) * sizeof(float)));
        if (rows_b > a.NS) rows_b = a.NS;
        const size_t smem_b = size_t(rows_b) * a.NS * sizeof(float) + ring_b;
        e = cudaFuncSetAttribute(reconf_back_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_b));
        if (e != cudaSuccess) return e;
        reconf_back_kernel<<<unsigned((S * lay.C + kBackWarps - 1) / kBackWarps), kBackThreads, smem_b, st>>>(a, rows_b);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return record_stop(st);
}

}  // namespace dyn
