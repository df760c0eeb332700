// Stage (b0): resolve the candidate frequencies against the profile tables.
//
// The profile is measured at a few frequencies and load levels and interpolated linearly in between
// [Sec. 4.1 "Generating LLM profiles"].  Everything that depends only on (class, TP, candidate
// frequency) is computed here once per call, in fp64, and stored in scratch memory in the form the
// sweep kernels read: per (class, TP, frequency) pair one row of utilisation segments, each holding
// value and slope of TBT and of the per-instance window energy, plus the scale from per-instance load
// to table position.  Interpolating in f here and in u inside the sweep equals the bilinear
// interpolation of the definition.
#define DYN_TU_ID 3
#include "dyn_internal.cuh"

namespace dyn {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int64_t totals_chunks(int64_t W) {
    const int64_t per = 256;             // windows per partial sum (one CTA, one window per thread)
    return (W + per - 1) / per;
}

ResolvedLayout resolved_layout(int32_t C, int32_t T, int32_t F, int32_t M, int32_t Nmax, int64_t S, int64_t W) {
    ResolvedLayout l{};
    l.C = C; l.T = T; l.F = F; l.P = T * F; l.M = M; l.Nmax = Nmax;
    l.J = Nmax * T * F;
    l.row_stride = M + 1;
    const size_t entries = size_t(C) * size_t(l.P) * size_t(l.row_stride);
    size_t off = 0;
    // rows | pairc | slo and pair2 | rows2 are contiguous: the sweep stages one or the other as one piece
    l.off_rows = off;   off = align_up(off + entries * sizeof(float4), 256);
    l.off_pairc = off;  off = align_up(off + size_t(C) * size_t(l.P) * sizeof(float2), 256);
    l.off_slo = off;    off = align_up(off + size_t(C) * sizeof(float), 256);
    l.off_pair2 = off;  off = align_up(off + size_t(C) * size_t(l.P) * sizeof(float4), 256);
    l.off_rows2 = off;  off = align_up(off + entries * sizeof(float2), 256);
    l.off_tp = off;     off = align_up(off + size_t(T) * sizeof(int32_t), 256);
    l.off_partial = off;
    off = align_up(off + size_t(S) * size_t(totals_chunks(W)) * (sizeof(double) + sizeof(uint32_t)), 256);
    l.total = off;
    return l;
}

namespace {

__device__ __forceinline__ double lerp64(double a, double b, double w) { return (1.0 - w) * a + w * b; }

// One thread per table entry (class c, pair p = t*F + q, entry m = 0..M):
//   m <= M-2  segment m: value and NEGATED slope of TBT and of the per-instance window energy (the
//             sweep multiplies them by minus the fraction)
//   m == M-1  the last knot, reached with nu == 0 only at u == 1; its TBT slope is huge, so that any
//             x above M-1 (u > 1) reads as an SLO violation without a separate capacity test
//   m == M    x saturated (u >= M/(M-1)): TBT = +inf
// A pair whose TTFT misses its SLO, or whose capacity is not positive, gets TBT = +inf in every entry.
__global__ void resolve_kernel(const ResolveParams rp, float4 *__restrict__ rows, float2 *__restrict__ pairc,
                               float *__restrict__ slo, float4 *__restrict__ pair2, float2 *__restrict__ rows2,
                               int32_t *__restrict__ tp) {
    const int P = rp.T * rp.F;
    const int M = rp.M;
    const int RS = M + 1;
    const long long total = (long long)rp.C * P * RS;
    const double scale = double(rp.window_s) / 3600.0;
    const float kInf = __int_as_float(0x7f800000);
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int m = int(e % RS);
        const long long cp = e / RS;
        const int p = int(cp % P);
        const int c = int(cp / P);
        const int t = p / rp.F, q = p - t * rp.F;
        const int r = rp.row[q];
        const double w = double(rp.weight[q]);
        const size_t ct = (size_t(c) * rp.T + t) * rp.R;
        (void)DYN_IDX(ct + r + 1, size_t(rp.C) * rp.T * rp.R);        // rows r and r + 1 of the profile tables exist
        const float *tb0 = rp.d_tbt + (ct + r) * M, *tb1 = tb0 + M;
        const float *pw0 = rp.d_pow + (ct + r) * M, *pw1 = pw0 + M;
        const double ttft = lerp64(rp.d_ttft[ct + r], rp.d_ttft[ct + r + 1], w);
        const double cap = lerp64(rp.d_cap[ct + r], rp.d_cap[ct + r + 1], w);
        // a non-positive (or NaN) capacity can serve no load: the pair is never feasible
        const bool pair_ok = (ttft <= double(rp.slo_ttft[c])) && (cap > 0.0);
        const int mk = m < M ? m : M - 1;
        const double tb_m = lerp64(tb0[mk], tb1[mk], w);
        const double pw_m = lerp64(pw0[mk], pw1[mk], w) * scale;
        float4 v;
        if (m < M - 1) {
            const double tb_n = lerp64(tb0[m + 1], tb1[m + 1], w);
            const double pw_n = lerp64(pw0[m + 1], pw1[m + 1], w) * scale;
            v = make_float4(float(tb_m), float(tb_m - tb_n), float(pw_m), float(pw_m - pw_n));
        } else if (m == M - 1) {
            v = make_float4(float(tb_m), -1e30f, float(pw_m), 0.f);
        } else {
            v = make_float4(kInf, 0.f, float(pw_m), 0.f);
        }
        if (!pair_ok) v.x = kInf;
        rows[DYN_IDX((size_t(c) * P + p) * RS + m, size_t(total))] = v;
        // threshold path: the same energy as a line in the per-instance load l, e(l) = a + l*b (x = l*(M-1)/cap);
        // the lines of neighbouring segments meet at the knots, so a position that rounding puts on
        // either side of a knot gets the same value
        float2 line = make_float2(float(pw_m), 0.f);
        if (m < M - 1 && pair_ok) {
            const double d = lerp64(pw0[m + 1], pw1[m + 1], w) * scale - pw_m;
            line = make_float2(float(pw_m - double(m) * d), float(d * double(M - 1) / cap));
        }
        rows2[DYN_IDX((size_t(c) * P + p) * RS + m, size_t(total))] = line;
        if (m == 0) {
            // Load threshold of the pair.  TBT is piecewise linear along the row, so {x : TBT(x) <= slo} is a
            // union of intervals; when it is empty or one interval that starts at x = 0, "TBT <= slo and
            // u <= 1" holds exactly for x in [0, xlim] and the sweep tests the load against a threshold.
            // That is the case whenever TBT, walking up the row, never comes back to or below the SLO after
            // having exceeded it (a row that rises with load always qualifies; so does a row with dips that
            // do not reach the SLO again).  NaN marks a row without that property: its candidates interpolate
            // TBT one by one.
            const double slo_c = double(rp.slo_tbt[c]);
            double vlim = -1.0;
            bool single = true;                  // the feasible set is empty or [0, xlim]
            bool closed = false;                 // an infeasible position has been passed
            double prev = lerp64(tb0[0], tb1[0], w);
            double xlim = -1.0;
            if (prev <= slo_c) xlim = 0.0;
            else closed = true;
            for (int k = 1; k < M; ++k) {
                const double cur = lerp64(tb0[k], tb1[k], w);
                if (cur <= slo_c) {
                    if (closed || !(prev <= slo_c)) single = false;      // feasible again after an infeasible stretch
                    xlim = double(k);
                } else {
                    if (prev <= slo_c && !closed) xlim = double(k - 1) + (slo_c - prev) / (cur - prev);
                    closed = true;
                    if (!(cur > slo_c)) single = false;                  // NaN entry: no threshold
                }
                prev = cur;
            }
            if (!pair_ok) single = true;         // never feasible: the empty set
            if (!single) xlim = -1.0;            // the threshold path skips this row; the general path serves it
            if (pair_ok && xlim >= 0.0) vlim = xlim / double(M);
            // x = u*(M-1) is formed as sat(L/n * ic) * M, so that saturation at 1 means x = M
            pairc[DYN_IDX(size_t(c) * P + p, size_t(rp.C) * P)] = make_float2(pair_ok ? float(double(M - 1) / (double(M) * cap)) : 0.f,
                                                   single ? float(vlim) : __int_as_float(0x7fc00000));
            // threshold path: table position per unit of per-instance load (twice: the sweep uses it as a
            // packed pair) and the largest per-instance load within the SLO and the capacity
            const float icm = pair_ok ? float(double(M - 1) / cap) : 0.f;
            const float llim = (pair_ok && xlim >= 0.0) ? float(xlim / double(M - 1) * cap) : -1.f;
            pair2[DYN_IDX(size_t(c) * P + p, size_t(rp.C) * P)] = make_float4(icm, icm, llim, float(cap));   // cap as interpolated, feasible or not
            if (p == 0) slo[c] = rp.slo_tbt[c];
            if (c == 0 && p < rp.T) tp[p] = rp.tp[p];
        }
    }
}

}  // namespace

cudaError_t launch_resolve(const ResolveParams &rp, const ResolvedLayout &lay, void *d_ws, cudaStream_t st) {
    char *ws = static_cast<char *>(d_ws);
    const long long total = (long long)rp.C * lay.P * (rp.M + 1);
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    const long long cap = (long long)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    resolve_kernel<<<int(blocks), threads, 0, st>>>(rp, reinterpret_cast<float4 *>(ws + lay.off_rows),
                                                    reinterpret_cast<float2 *>(ws + lay.off_pairc),
                                                    reinterpret_cast<float *>(ws + lay.off_slo),
                                                    reinterpret_cast<float4 *>(ws + lay.off_pair2),
                                                    reinterpret_cast<float2 *>(ws + lay.off_rows2),
                                                    reinterpret_cast<int32_t *>(ws + lay.off_tp));
    return cudaGetLastError();
}

}  // namespace dyn
