// Instrumentation (no counterpart in the paper): two small kernels that measure, on the GPU they run
// on and at the clock it runs at, the ceilings the sweep is judged against.
//
//   fma_probe_kernel          every thread advances 8 independent fp32 multiply-add chains: nothing but
//                             FMA instructions, one per scheduler and clock when the machine sustains it.
//                             Its rate is the fp32 peak (2 flop per lane and FMA) and, divided by 64, the
//                             issue ceiling in warp instructions per second.
//   sweep_inner_probe_kernel  the pair loop of the fused sweep on the threshold path exactly as the sweep
//                             runs it (the same device function on tables in shared memory, 8 candidates
//                             per lane and pair), with no tile around it: no loads of the load tensor, no
//                             reductions, no pair recovery, no stores.  Its rate is what the instruction
//                             mix of the inner loop reaches on this machine for a given share of
//                             feasible candidates (an infeasible candidate skips its table lookup); the
//                             sweep kernel's rate divided by it is the share of the inner loop in the
//                             sweep's time.
//
// The caller times the launches (events on the stream, or dyn_set_timing_events).
#define DYN_TU_ID 12
#include "dyn_internal.cuh"
#include "eval_dev.cuh"

#include <math_constants.h>

namespace dyn {

namespace {

constexpr int kProbeThreads = 256;
constexpr int kChains = 8;

__global__ void __launch_bounds__(kProbeThreads, 8)
fma_probe_kernel(const float a, const float b, const int iters, float *__restrict__ sink) {
    float x[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) x[k] = float(threadIdx.x) * 1e-3f + float(k);
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int k = 0; k < kChains; ++k) x[k] = fmaf(x[k], a, b);
        }
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) s += x[k];
    if (s == -1.2345e30f) *sink = s;             // never true for the values used: keeps the chains alive
}

constexpr int kProbeM = 8;                       // utilisation knots of the synthetic table
constexpr int kProbeP = 32;                      // (TP, f) pairs
constexpr int kProbeNCH = 8;                     // candidates per lane and pair (two instance counts x four tiles)

__global__ void __launch_bounds__(kProbeThreads, 4)
sweep_inner_probe_kernel(const int iters, const float scale, const float feasible_share, float *__restrict__ sink) {
    extern __shared__ float4 smem[];
    // pair2[P] float4 {icm, icm, llim, cap} | rows2[P][M+1] float2 {a, b}
    constexpr int RS = kProbeM + 1;
    float2 *rows2 = reinterpret_cast<float2 *>(smem + kProbeP);
    for (int p = threadIdx.x; p < kProbeP; p += blockDim.x) {
        const float icm = float(kProbeM - 1) / (1.0f + 0.01f * float(p));
        smem[p] = make_float4(icm, icm, feasible_share * scale, 1.0f);   // loads are uniform on [0, scale)
    }
    for (int i = threadIdx.x; i < kProbeP * RS; i += blockDim.x)
        rows2[i] = make_float2(1.0f + float(i % RS), 0.5f + 0.001f * float(i / RS));
    __syncthreads();
    DYN_SET_RANGES(uint32_t(__cvta_generic_to_shared(smem)),
                   uint32_t(__cvta_generic_to_shared(smem)) + uint32_t(kProbeP) * 16u + uint32_t(kProbeP * RS) * 8u, 0u);
    uint32_t origin = table_origin<true>();
    asm volatile("" : "+r"(origin) : : "memory");
    const uint32_t cpair = origin;
    const uint32_t crow = origin + uint32_t(kProbeP) * 16u;
    const uint32_t pstep = uint32_t(RS) * 8u;
    const uint64_t two23_2 = pack2(kTwo23, kTwo23);
    const uint64_t eight2 = pack2(units(8u), units(8u));
    const float off0 = row_offset_units(crow);
    const float offs = float(int(pstep)) * units(1u);
    const uint64_t off2_first = pack2(off0, off0), off2_step = pack2(offs, offs);

    const int lane = threadIdx.x & 31;
    float best[kProbeNCH];
    uint64_t ln2[kProbeNCH / 2];
#pragma unroll
    for (int q = 0; q < kProbeNCH; q += 2) {
        // per-instance loads spread over [0, scale): table positions l*icm stay inside the rows
        const float l0 = scale * float(lane * kProbeNCH + q) / float(32 * kProbeNCH);
        const float l1 = scale * float(lane * kProbeNCH + q + 1) / float(32 * kProbeNCH);
        ln2[q / 2] = pack2(l0, l1);
        best[q] = best[q + 1] = CUDART_INF_F;
    }
    const uint64_t shrink = pack2(0.999f, 0.999f), grow = pack2(1.015f, 1.015f);   // 0.999^15 * 1.015 = 1.0
    for (int it = 0; it < iters; ++it) {
        uint64_t off2 = off2_first;
#pragma unroll 8
        for (int p = 0; p < kProbeP; ++p) {
            uint64_t icm2, lim2;
            asm("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(icm2), "=l"(lim2) : "r"(cpair + uint32_t(p) * 16u));
            const float lim = __uint_as_float(uint32_t(lim2));
#pragma unroll
            for (int q = 0; q < kProbeNCH; q += 2)
                fast_two(ln2[q / 2], icm2, off2, two23_2, eight2, lim, lim, best[q], best[q + 1]);
            off2 = add2(off2, off2_step);
        }
        // other loads for the next round, as a new pass of tiles would bring (4 instructions per 256
        // candidates): shrink, and start again from the top once they have halved, so the share of
        // feasible candidates stays near the requested one
#pragma unroll
        for (int q = 0; q < kProbeNCH / 2; ++q) ln2[q] = mul2(ln2[q], (it & 15) == 15 ? grow : shrink);
    }
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < kProbeNCH; ++q) s += best[q];
    if (s == -1.2345e30f) *sink = s;
}

// 0 until the check has run; 1 = subnormal arithmetic is exact, 2 = it is not (flushed to zero)
__device__ int g_self_check;

// forms the shared-memory byte address of entry m of a row at byte offset `bytes` the way fast_two does, from
// values the compiler cannot fold, and compares with the integer arithmetic
__global__ void self_check_kernel(const float m_plus_two23, const uint32_t bytes, const uint32_t want) {
    const float off = row_offset_units(bytes);
    float z;
    asm volatile("fma.rn.f32 %0, %1, %2, %3;" : "=f"(z) : "f"(m_plus_two23), "f"(units(8u)), "f"(off));
    g_self_check = (__float_as_uint(z) == want) ? 1 : 2;
}

#ifdef DYN_CHECK
// a planted violation: index 5 into an array of 3, which the check records and replaces by 0
__global__ void check_selftest_kernel(int *out) {
    int a[3] = {7, 8, 9};
    const int i = DYN_IDX(5 + int(threadIdx.x), 3);
    *out = a[i];
}
#endif

}  // namespace

}  // namespace dyn

using namespace dyn;

extern "C" {

int dyn_debug_selftest(int32_t *d_out, void *stream) {
#ifdef DYN_CHECK
    if (!d_out) return DYN_EINVAL;
    check_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(d_out);
    DYN_CUDA_TRY(cudaGetLastError());
    return DYN_OK;
#else
    (void)d_out;
    (void)stream;
    return DYN_EUNSUPPORTED;
#endif
}

int dyn_self_check(void *stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t m = 5u, bytes = 4096u + 72u;
    self_check_kernel<<<1, 1, 0, st>>>(kTwo23 + float(m), bytes, bytes + 8u * m);
    DYN_CUDA_TRY(cudaGetLastError());
    DYN_CUDA_TRY(cudaStreamSynchronize(st));
    int got = 0;
    DYN_CUDA_TRY(cudaMemcpyFromSymbol(&got, g_self_check, sizeof(int)));
    return got == 1 ? DYN_OK : DYN_EUNSUPPORTED;
}

int dyn_probe_fma(int32_t iters, float *d_sink, double *fp32_ops, void *stream) {
    if (iters < 1 || !d_sink) return DYN_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = sm_count() * 8;
    DYN_CUDA_TRY(record_start(st));
    // a and b keep every chain finite: x -> 0.999 x + 0.001 converges to 1
    fma_probe_kernel<<<grid, kProbeThreads, 0, st>>>(0.999f, 0.001f, iters, d_sink);
    DYN_CUDA_TRY(cudaGetLastError());
    DYN_CUDA_TRY(record_stop(st));
    if (fp32_ops) *fp32_ops = 2.0 * double(grid) * kProbeThreads * double(iters) * 8.0 * kChains;
    return DYN_OK;
}

int dyn_probe_sweep_inner(int32_t iters, float feasible_share, float *d_sink, double *candidates, void *stream) {
    if (iters < 1 || !d_sink || !(feasible_share >= 0.f && feasible_share <= 1.f)) return DYN_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = sm_count() * 4;
    const size_t smem = size_t(kProbeP) * 16 + size_t(kProbeP) * (kProbeM + 1) * 8;
    DYN_CUDA_TRY(record_start(st));
    sweep_inner_probe_kernel<<<grid, kProbeThreads, smem, st>>>(iters, 1.0f, feasible_share, d_sink);
    DYN_CUDA_TRY(cudaGetLastError());
    DYN_CUDA_TRY(record_stop(st));
    if (candidates) *candidates = double(grid) * kProbeThreads * double(iters) * kProbeP * kProbeNCH;
    return DYN_OK;
}

}  // extern "C"
