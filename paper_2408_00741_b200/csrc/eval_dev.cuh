// Device-side pieces of the candidate evaluation shared by the sweep kernels and the mixed-pool search
// (included by those translation units only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

// The table addresses of the threshold path are formed as subnormal floats (see units() below): a build that
// flushes subnormals to zero (-ftz=true, --use_fast_math) would turn every address into zero.  The compiler
// defines nothing a source file could test for this, so the build script refuses such flags and
// dyn_self_check() tests the arithmetic on the device.

namespace dyn {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr float kTwo23 = 8388608.0f;
constexpr uint32_t kTwo23Bits = 0x4b000000u;

// smallest value over the warp (no NaNs here)
__device__ __forceinline__ float warp_min(float v) {
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}

// smallest value over the lanes of `mask` (the caller's group; all its lanes call with the same mask)
__device__ __forceinline__ float group_min(float v, unsigned mask) {
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, %2;" : "=f"(r) : "f"(v), "r"(mask));
    return r;
}

// ---- table access -----------------------------------------------------------------------------
// General path: `base` is the byte address of the pair's row minus 16 * bits(2^23): the entry address is
// one multiply-add away from the bit pattern of y = 2^23 + floor(x).  Shared memory is addressed in 32 bits.
template <bool SMEM>
__device__ __forceinline__ float4 entry16(const char *__restrict__ ws, uint32_t base, float y) {
    uint32_t addr = __float_as_uint(y) * 16u + base;
    if (SMEM) {
        addr = DYN_SMEM_ADDR(addr, 16u);
        float4 r;
        asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(addr));
        return r;
    }
    return __ldg(reinterpret_cast<const float4 *>(ws + DYN_GLOBAL_OFF(addr, 16u)));
}
// 8-byte entry / 16-byte pair constants at byte address (shared) or byte offset (scratch block) `addr`
template <bool SMEM>
__device__ __forceinline__ float2 load8(const char *__restrict__ ws, uint32_t addr) {
    addr = SMEM ? DYN_SMEM_ADDR(addr, 8u) : DYN_GLOBAL_OFF(addr, 8u);
    if (SMEM) {
        float2 r;
        asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(r.x), "=f"(r.y) : "r"(addr));
        return r;
    }
    return __ldg(reinterpret_cast<const float2 *>(ws + addr));
}
template <bool SMEM>
__device__ __forceinline__ float4 load16(const char *__restrict__ ws, uint32_t addr) {
    addr = SMEM ? DYN_SMEM_ADDR(addr, 16u) : DYN_GLOBAL_OFF(addr, 16u);
    if (SMEM) {
        float4 r;
        asm("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(addr));
        return r;
    }
    return __ldg(reinterpret_cast<const float4 *>(ws + addr));
}
template <bool SMEM>
__device__ __forceinline__ uint32_t table_origin() {
    if (SMEM) {
        extern __shared__ float4 smem[];
        return uint32_t(__cvta_generic_to_shared(smem));
    }
    return 0u;
}

// best = min(best, E) if a <= b: one compare and one predicated min
__device__ __forceinline__ void min_if_le(float &best, float a, float b, float E) {
    asm("{\n\t.reg .pred p;\n\tsetp.le.f32 p, %1, %2;\n\t@p min.f32 %0, %0, %3;\n\t}"
        : "+f"(best) : "f"(a), "f"(b), "f"(E));
}

// ---- packed fp32 pairs held in 64-bit registers ---------------------------------------------------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float half_of(uint64_t v, int hi) {
    float lo, up;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(up) : "l"(v));
    return hi ? up : lo;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// A subnormal float with bit pattern k has the value k * 2^-149 ("k units").
__device__ __forceinline__ float units(uint32_t k) { return __uint_as_float(k); }

// (bytes - 2^26) units as a float.  Added to (2^23 + m) * 2^-146 = (2^26 + 8m) units it leaves bytes + 8m
// units, a subnormal number whose bit pattern is the integer bytes + 8m.  `bytes` is a multiple of 8
// below 2^23, so every value involved is exactly representable and the arithmetic is exact.
__device__ __forceinline__ float row_offset_units(uint32_t bytes) {
    return -float(int(67108864u - bytes)) * units(1u);
}

// ---- threshold path, tables in shared memory: two candidates of one (TP, f) pair ---------------------
// ln2 = per-instance loads {lA, lB}; icm2 = {icm, icm}; off2 = row offset in units, twice; limA/limB =
// load limit of the pair (or -1 where the GPU budget excludes the candidate).  Per candidate:
//   feasible = l <= lim;  y = rz(l*icm + 2^23);  z = y*2^-146 + off  (bits(z) = address of the entry);
//   if feasible: {a, b} = entry;  best = min(best, a + l*b).
#ifdef DYN_CHECK
// the checking build forms the two addresses with scalar instructions of the same rounding (bit-identical
// results) and tests them against the staged range before the lookups
__device__ __forceinline__ void fast_two_checked(uint64_t ln2, uint64_t icm2, uint64_t off2, float limA, float limB, float &eA,
                                                 float &eB, bool &okA, bool &okB) {
    float l[2], icm[2], off[2], e[2];
    bool ok[2];
    asm("mov.b64 {%0, %1}, %2;" : "=f"(l[0]), "=f"(l[1]) : "l"(ln2));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(icm[0]), "=f"(icm[1]) : "l"(icm2));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(off[0]), "=f"(off[1]) : "l"(off2));
    const float lim[2] = {limA, limB};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        ok[k] = l[k] <= lim[k];
        e[k] = 0.f;
        if (ok[k]) {
            const float y = __fmaf_rz(l[k], icm[k], 8388608.0f);
            const float z = __fmaf_rn(y, __uint_as_float(8u), off[k]);
            const uint32_t addr = DYN_SMEM_ADDR(__float_as_uint(z), 8u);
            float2 en;
            asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(en.x), "=f"(en.y) : "r"(addr));
            e[k] = fmaf(l[k], en.y, en.x);
        }
    }
    eA = e[0]; eB = e[1]; okA = ok[0]; okB = ok[1];
}
#endif

__device__ __forceinline__ void fast_two(uint64_t ln2, uint64_t icm2, uint64_t off2, uint64_t two23_2, uint64_t eight2,
                                         float limA, float limB, float &bestA, float &bestB) {
#ifdef DYN_CHECK
    float eA, eB;
    bool okA, okB;
    fast_two_checked(ln2, icm2, off2, limA, limB, eA, eB, okA, okB);
    if (okA) bestA = fminf(bestA, eA);
    if (okB) bestB = fminf(bestB, eB);
    return;
#endif
    // The lookups are predicated and land in the registers that held y and z: those are defined on every
    // path, so nothing stays live around the pair loop for the sake of a skipped load (an infeasible
    // candidate forms a meaningless energy from them, which its predicated min ignores).
    asm("{\n\t"
        ".reg .pred pA, pB;\n\t"
        ".reg .f32 lA, lB, a0, b0, a1, b1, eA, eB;\n\t"
        ".reg .b32 zA, zB;\n\t"
        ".reg .b64 y, z;\n\t"
        "mov.b64 {lA, lB}, %2;\n\t"
        "setp.le.f32 pA, lA, %7;\n\t"
        "setp.le.f32 pB, lB, %8;\n\t"
        "fma.rz.f32x2 y, %2, %3, %5;\n\t"
        "fma.rn.f32x2 z, y, %6, %4;\n\t"
        "mov.b64 {zA, zB}, z;\n\t"
        "@pA ld.shared.b64 y, [zA];\n\t"
        "@pB ld.shared.b64 z, [zB];\n\t"
        "mov.b64 {a0, b0}, y;\n\t"
        "mov.b64 {a1, b1}, z;\n\t"
        "fma.rn.f32 eA, lA, b0, a0;\n\t"
        "fma.rn.f32 eB, lB, b1, a1;\n\t"
        "@pA min.f32 %0, %0, eA;\n\t"
        "@pB min.f32 %1, %1, eB;\n\t"
        "}"
        : "+f"(bestA), "+f"(bestB)
        : "l"(ln2), "l"(icm2), "l"(off2), "l"(two23_2), "l"(eight2), "f"(limA), "f"(limB));
}

// fast_two for the evaluate-only kernel: the pool energies n*e of the two candidates, +inf where infeasible
__device__ __forceinline__ void fast_two_energy(uint64_t ln2, uint64_t icm2, uint64_t off2, uint64_t two23_2,
                                                uint64_t eight2, float limA, float limB, float nfA, float nfB,
                                                float &EA, float &EB) {
#ifdef DYN_CHECK
    float eA, eB;
    bool okA, okB;
    fast_two_checked(ln2, icm2, off2, limA, limB, eA, eB, okA, okB);
    EA = okA ? eA * nfA : __int_as_float(0x7f800000);
    EB = okB ? eB * nfB : __int_as_float(0x7f800000);
    return;
#endif
    asm("{\n\t"
        ".reg .pred pA, pB;\n\t"
        ".reg .f32 lA, lB, a0, b0, a1, b1, eA, eB;\n\t"
        ".reg .b32 zA, zB;\n\t"
        ".reg .b64 y, z;\n\t"
        "mov.b64 {lA, lB}, %2;\n\t"
        "setp.le.f32 pA, lA, %7;\n\t"
        "setp.le.f32 pB, lB, %8;\n\t"
        "fma.rz.f32x2 y, %2, %3, %5;\n\t"
        "fma.rn.f32x2 z, y, %6, %4;\n\t"
        "mov.b64 {zA, zB}, z;\n\t"
        "@pA ld.shared.b64 y, [zA];\n\t"
        "@pB ld.shared.b64 z, [zB];\n\t"
        "mov.b64 {a0, b0}, y;\n\t"
        "mov.b64 {a1, b1}, z;\n\t"
        "fma.rn.f32 eA, lA, b0, a0;\n\t"
        "fma.rn.f32 eB, lB, b1, a1;\n\t"
        "mul.rn.f32 eA, eA, %9;\n\t"
        "mul.rn.f32 eB, eB, %10;\n\t"
        "selp.f32 %0, eA, 0f7F800000, pA;\n\t"
        "selp.f32 %1, eB, 0f7F800000, pB;\n\t"
        "}"
        : "=f"(EA), "=f"(EB)
        : "l"(ln2), "l"(icm2), "l"(off2), "l"(two23_2), "l"(eight2), "f"(limA), "f"(limB), "f"(nfA), "f"(nfB));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// the same evaluation for one candidate with ordinary address arithmetic (tables in shared memory or
// read through L1), bit-identical to fast_two: e = a + l*b of segment floor(l*icm), ok = l <= lim.
// `row` is the byte address / offset of the pair's row.  An infeasible candidate reads entry 0.
template <bool SMEM>
__device__ __forceinline__ void fast_one(const char *__restrict__ ws, uint32_t row, float l, float icm, float lim,
                                         float &e, bool &ok) {
    ok = l <= lim;
    const float y = __fmaf_rz(l, icm, kTwo23);
    const uint32_t m = ok ? __float_as_uint(y) - kTwo23Bits : 0u;
    const float2 en = load8<SMEM>(ws, row + m * 8u);
    e = fmaf(l, en.y, en.x);
}

struct Consts2 {            // the same constant in both halves of a register pair
    float2 M, negM, two23, neg23;
};

// General path: two candidates of one (TP, f) pair.  ln = L/n per candidate, ic = (M-1)/(M*cap).
// v = sat(ln*ic) is the table position over M; y = 2^23 + floor(v*M); nnu = floor(v*M) - v*M.
// Entries {TBT, -slope, energy, -slope} at the segment's left knot, feasible iff TBT <= slo (u > 1 and
// never-feasible pairs read as TBT = huge or +inf through the sentinel entries).  The energy of one
// instance enters the running minimum of its chain when feasible.
template <bool SMEM>
__device__ __forceinline__ void general_two(const char *__restrict__ ws, uint32_t base, float lnA, float lnB, float ic,
                                            float slo, const Consts2 &k, bool allowA, bool allowB, float &bestA,
                                            float &bestB) {
    const float2 v = make_float2(__saturatef(lnA * ic), __saturatef(lnB * ic));   // NaN -> 0, > 1 -> 1
    const float2 y = __ffma2_rz(v, k.M, k.two23);
    const float2 fm = __fadd2_rn(y, k.neg23);
    const float2 nnu = __ffma2_rn(v, k.negM, fm);
    const float4 eA = entry16<SMEM>(ws, base, y.x);
    const float4 eB = entry16<SMEM>(ws, base, y.y);
    const float tbtA = fmaf(nnu.x, eA.y, eA.x), tbtB = fmaf(nnu.y, eB.y, eB.x);
    if (allowA) min_if_le(bestA, tbtA, slo, fmaf(nnu.x, eA.w, eA.z));     // allow*: GPU budget (always true without one)
    if (allowB) min_if_le(bestB, tbtB, slo, fmaf(nnu.y, eB.w, eB.z));
}

// scalar form of the same evaluation, bit-identical to general_two (evaluate-only kernel, pair recovery)
template <bool SMEM>
__device__ __forceinline__ void general_one(const char *__restrict__ ws, uint32_t base, float ln, float ic, float slo,
                                            float Mf, float &e, bool &ok) {
    const float v = __saturatef(ln * ic);
    const float y = __fmaf_rz(v, Mf, kTwo23);
    const float nnu = fmaf(v, -Mf, y + (-kTwo23));
    const float4 en = entry16<SMEM>(ws, base, y);
    ok = fmaf(nnu, en.y, en.x) <= slo;
    e = fmaf(nnu, en.w, en.z);
}

}  // namespace

}  // namespace dyn
