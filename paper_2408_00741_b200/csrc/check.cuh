// Index checks of the checking build (-DDYN_CHECK; `python -m paper_2408_00741_b200.build --check` builds
// libdynamo_check.so with them).  In that build every computed index into a global array, a shared-memory
// bin or a table passes through DYN_IDX(index, extent): an index outside [0, extent) is recorded and replaced
// by 0, so the access stays in bounds and the kernel runs on; nothing traps and nothing waits.  Shared-memory
// addresses that are formed arithmetically (the sweep's table lookups) are checked against the range the
// kernel staged.  The first violation of a translation unit is kept as {count, site, index, extent}, site =
// translation unit number * 65536 + source line; dyn_debug_status() collects the records of all translation
// units.  In the ordinary build the macros cost nothing: DYN_IDX(i, n) is (i).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#ifdef DYN_CHECK

#include <type_traits>

#ifndef DYN_TU_ID
#error "define DYN_TU_ID (a small number, unique per translation unit) before including the library's headers"
#endif

namespace dyn {
namespace check {

struct Record {
    unsigned int count, site, index, extent;
};

// host side (abi.cu): every translation unit registers a function that reads (and clears) its record
typedef cudaError_t (*Reader)(Record *out);
void register_reader(Reader r);

namespace {

__device__ Record g_record;          // one per translation unit (internal linkage)

__device__ __noinline__ void fail(unsigned int site, unsigned long long i, unsigned long long n) {
    if (atomicAdd(&g_record.count, 1u) == 0u) {
        g_record.site = site;
        g_record.index = i > 0xffffffffull ? 0xffffffffu : (unsigned int)i;
        g_record.extent = n > 0xffffffffull ? 0xffffffffu : (unsigned int)n;
    }
}

template <class I, class N>
__device__ __forceinline__ I idx(I i, N n, unsigned int site) {
    bool nonneg = true;
    if constexpr (std::is_signed<I>::value) nonneg = i >= I(0);
    if (nonneg && (unsigned long long)(i) < (unsigned long long)(n)) return i;
    fail(site, (unsigned long long)(i), (unsigned long long)(n));
    return I(0);
}

// a pointer that must lie inside [base, base + n)
template <class T>
__device__ __forceinline__ const T *ptr(const T *p, const T *base, long long n, unsigned int site) {
    const long long i = p - base;
    if (i >= 0 && i < n) return p;
    fail(site, (unsigned long long)(i), (unsigned long long)(n));
    return base;
}

// ranges of arithmetically formed addresses, set by the kernel before it forms any: shared-memory byte
// addresses [lo, hi) of the staged tables, and the byte extent of the scratch block for tables read from it
struct Ranges {
    unsigned int smem_lo, smem_hi, global_bytes;
};
__device__ __forceinline__ Ranges &ranges() {
    __shared__ Ranges r;
    return r;
}
// called by every thread of the CTA, before the barrier that ends the staging (or followed by one)
__device__ __forceinline__ void set_ranges(unsigned int smem_lo, unsigned int smem_hi, unsigned int global_bytes) {
    if (threadIdx.x == 0) {
        ranges().smem_lo = smem_lo;
        ranges().smem_hi = smem_hi;
        ranges().global_bytes = global_bytes;
    }
    __syncthreads();
}
__device__ __forceinline__ unsigned int smem_addr(unsigned int addr, unsigned int bytes, unsigned int site) {
    const Ranges &r = ranges();
    if (addr >= r.smem_lo && addr + bytes <= r.smem_hi && (addr & (bytes - 1u)) == 0u) return addr;
    fail(site, addr, r.smem_hi);
    return r.smem_lo;
}
__device__ __forceinline__ unsigned int global_off(unsigned int off, unsigned int bytes, unsigned int site) {
    const Ranges &r = ranges();
    if (off + bytes <= r.global_bytes && (off & (bytes - 1u)) == 0u) return off;
    fail(site, off, r.global_bytes);
    return 0u;
}

cudaError_t read_record(Record *out) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_record, sizeof(Record));
    if (e != cudaSuccess) return e;
    const Record zero = {0u, 0u, 0u, 0u};
    return cudaMemcpyToSymbol(g_record, &zero, sizeof(Record));
}
struct Registrar {
    Registrar() { register_reader(&read_record); }
};
Registrar g_registrar;

}  // namespace
}  // namespace check
}  // namespace dyn

#define DYN_SITE (unsigned(DYN_TU_ID) * 65536u + unsigned(__LINE__))
#define DYN_IDX(i, n) (::dyn::check::idx((i), (n), DYN_SITE))
#define DYN_PTR(p, base, n) (::dyn::check::ptr((p), (base), (long long)(n), DYN_SITE))
#define DYN_SMEM_ADDR(addr, bytes) (::dyn::check::smem_addr((addr), (bytes), DYN_SITE))
#define DYN_GLOBAL_OFF(off, bytes) (::dyn::check::global_off((off), (bytes), DYN_SITE))
#define DYN_SET_RANGES(lo, hi, gbytes) ::dyn::check::set_ranges((lo), (hi), (gbytes))

#else  // ordinary build

#define DYN_IDX(i, n) (i)
#define DYN_PTR(p, base, n) (p)
#define DYN_SMEM_ADDR(addr, bytes) (addr)
#define DYN_GLOBAL_OFF(off, bytes) (off)
#define DYN_SET_RANGES(lo, hi, gbytes) ((void)0)

#endif
