// Checked global-memory access for the library's own loads and stores -- the stand-in for a memory sanitizer.
//
// Every kernel reaches global memory through the wrappers below (TMA boxes excepted: their extents are enforced by
// the tensor map in hardware).  In the regular build they are the plain intrinsics.  Built with -DDASS_BOUNDS_CHECK
// (python -m paper_2405_01943_b200.build --bounds-check: the whole library as ONE translation unit, so that the table
// below exists once), each entry point first registers the address ranges of the buffers it was given, and every
// access is tested against them: an access outside all ranges is SKIPPED (a load yields zero) and counted, with the
// first offender's address, width and source line kept for dass_bounds_report.  Nothing traps and nothing faults.
// Internal header.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dass {

#ifdef DASS_BOUNDS_CHECK

constexpr int BOUNDS_MAX_RANGES = 12;
struct BoundsTable {
    unsigned long long lo[BOUNDS_MAX_RANGES], hi[BOUNDS_MAX_RANGES];   // [lo, hi)
    int n;
};
struct BoundsReport {
    unsigned int violations;
    unsigned int first_bytes, first_line;
    unsigned long long first_addr;
};
static __device__ BoundsTable g_bounds;
static __device__ BoundsReport g_bounds_report;

__device__ __forceinline__ bool access_ok(const void *p, unsigned nbytes, unsigned line)
{
    const unsigned long long a = (unsigned long long)p;
    for (int i = 0; i < g_bounds.n; ++i)
        if (a >= g_bounds.lo[i] && a + nbytes <= g_bounds.hi[i]) return true;
    if (atomicAdd(&g_bounds_report.violations, 1u) == 0u) {
        g_bounds_report.first_addr = a;
        g_bounds_report.first_bytes = nbytes;
        g_bounds_report.first_line = line;
    }
    return false;
}
#define DASS_ACCESS_OK(p, n) dass::access_ok((p), (unsigned)(n), (unsigned)__LINE__)

// Host side: the ranges of one entry-point call, uploaded on the call's stream before its kernels.
inline size_t &bounds_shrink_next()
{
    static size_t bytes = 0;      // test hook: the next call registers every range this much shorter
    return bytes;
}
struct BoundsScope {
    BoundsTable t;
    size_t shrink;
    BoundsScope() : shrink(bounds_shrink_next()) { t.n = 0; bounds_shrink_next() = 0; }
    void add(const void *p, size_t bytes)
    {
        if (!p || bytes == 0 || t.n >= BOUNDS_MAX_RANGES) return;
        const size_t cut = shrink < bytes ? shrink : bytes;
        t.lo[t.n] = (unsigned long long)reinterpret_cast<uintptr_t>(p);
        t.hi[t.n] = t.lo[t.n] + (bytes - cut);
        ++t.n;
    }
    cudaError_t commit(cudaStream_t st) const
    {
        return cudaMemcpyToSymbolAsync(g_bounds, &t, sizeof(BoundsTable), 0, cudaMemcpyHostToDevice, st);
    }
};
#define DASS_BOUNDS_SCOPE(name) dass::BoundsScope name
#define DASS_BOUNDS_ADD(name, p, bytes) (name).add((p), (size_t)(bytes))
#define DASS_BOUNDS_COMMIT(name, st) \
    do { if ((name).commit(st) != cudaSuccess) return DASS_ERR_CUDA; } while (0)

#else

#define DASS_ACCESS_OK(p, n) true
#define DASS_BOUNDS_SCOPE(name) do { } while (0)
#define DASS_BOUNDS_ADD(name, p, bytes) do { } while (0)
#define DASS_BOUNDS_COMMIT(name, st) do { } while (0)

#endif

// ------------------------------------------------------------------ the access wrappers
template <typename T> __device__ __forceinline__ T zero_of() { return T(); }
template <> __device__ __forceinline__ uint4 zero_of<uint4>() { return make_uint4(0u, 0u, 0u, 0u); }
template <> __device__ __forceinline__ uint2 zero_of<uint2>() { return make_uint2(0u, 0u); }
template <> __device__ __forceinline__ float4 zero_of<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }

#define DASS_DEFINE_LOAD(name, expr)                                                            \
    template <typename T> __device__ __forceinline__ T name##_at(const T *p, unsigned line)    \
    {                                                                                           \
        (void)line;                                                                             \
        return DASS_ACCESS_OK_LINE(p, sizeof(T), line) ? (expr) : zero_of<T>();                 \
    }

#ifdef DASS_BOUNDS_CHECK
#define DASS_ACCESS_OK_LINE(p, n, line) dass::access_ok((p), (unsigned)(n), (line))
#else
#define DASS_ACCESS_OK_LINE(p, n, line) true
#endif

DASS_DEFINE_LOAD(ld_cs, __ldcs(p))      // streaming load (evict first)
DASS_DEFINE_LOAD(ld_g, __ldg(p))        // read-only cached load
DASS_DEFINE_LOAD(ld_plain, *p)          // ordinary load

template <typename T> __device__ __forceinline__ void st_cs_at(T *p, const T &v, unsigned line)
{
    (void)line;
    if (DASS_ACCESS_OK_LINE(p, sizeof(T), line)) __stcs(p, v);
}
template <typename T> __device__ __forceinline__ void st_plain_at(T *p, const T &v, unsigned line)
{
    (void)line;
    if (DASS_ACCESS_OK_LINE(p, sizeof(T), line)) *p = v;
}

// The forms kernels write: the source line of the access site is recorded with the first violation.
#define DASS_LD_CS(p) dass::ld_cs_at((p), (unsigned)__LINE__)
#define DASS_LD_G(p) dass::ld_g_at((p), (unsigned)__LINE__)
#define DASS_LD(p) dass::ld_plain_at((p), (unsigned)__LINE__)
#define DASS_ST_CS(p, v) dass::st_cs_at((p), (v), (unsigned)__LINE__)
#define DASS_ST(p, v) dass::st_plain_at((p), (v), (unsigned)__LINE__)

}  // namespace dass
