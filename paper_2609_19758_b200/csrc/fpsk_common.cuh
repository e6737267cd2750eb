// Shared declarations of the FP-Sketch CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>

#include "fpsk.h"

namespace fpsk {

extern std::atomic<unsigned long long> g_launches;   // kernels launched by this library
inline void count_launch(int n = 1) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

#define FPSK_CUDA_OK(expr)                         \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess) return FPSK_ERR_CUDA; \
    } while (0)

#define FPSK_LAUNCH_CHECK()                                    \
    do {                                                       \
        fpsk::count_launch();                                  \
        if (cudaPeekAtLastError() != cudaSuccess) return FPSK_ERR_CUDA; \
    } while (0)

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------- integer hash
// Section "Moment Sketches" draws hashes and signs without fixing a family; this is the
// library's: two multiply / xor-shift rounds on 32-bit words.
__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x)
{
    x ^= x >> 16;
    x *= 0x7FEB352Du;
    x ^= x >> 15;
    x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x;
}
constexpr uint32_t kGolden = 0x9E3779B9u;

__host__ __device__ __forceinline__ uint32_t round_key(uint64_t seed, int rnd, int side)
{
    uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
    return mix32(lo ^ mix32(hi + kGolden * (uint32_t)(2 * rnd + side + 1)));
}
// bucket in [0, m_b) and sign (+1 / -1) of index idx under key
__host__ __device__ __forceinline__ void hash_index(uint32_t key, uint32_t idx, uint32_t m_b,
                                                    int &bucket, int &sign)
{
    uint32_t h = mix32(idx ^ key);
    bucket = (int)(((uint64_t)h * (uint64_t)m_b) >> 32);
    sign = (mix32(h + kGolden) & 1u) ? -1 : 1;
}

// ---------------------------------------------------------------- half-precision loads
template <typename T> struct HalfTraits;
template <> struct HalfTraits<__half> {
    static __device__ __forceinline__ float to_f(__half x) { return __half2float(x); }
    // two packed values -> two floats
    static __device__ __forceinline__ float2 unpack2(uint32_t w)
    {
        __half2 h = *reinterpret_cast<__half2 *>(&w);
        return __half22float2(h);
    }
};
template <> struct HalfTraits<__nv_bfloat16> {
    static __device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
    static __device__ __forceinline__ float2 unpack2(uint32_t w)
    {
        float2 r;
        r.x = __uint_as_float(w << 16);
        r.y = __uint_as_float(w & 0xFFFF0000u);
        return r;
    }
};

// Running max of |x| over packed pairs of 16-bit floats, kept as a packed pair: one abs and
// one max instruction per two elements (native HMNMX2).  NaN operands are ignored by the max.
template <typename T> __device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t w);
template <> __device__ __forceinline__ uint32_t absmax2<__half>(uint32_t acc, uint32_t w)
{
    __half2 a = *reinterpret_cast<__half2 *>(&acc), b = *reinterpret_cast<__half2 *>(&w);
    a = __hmax2(a, __habs2(b));
    return *reinterpret_cast<uint32_t *>(&a);
}
template <> __device__ __forceinline__ uint32_t absmax2<__nv_bfloat16>(uint32_t acc, uint32_t w)
{
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&acc), b = *reinterpret_cast<__nv_bfloat162 *>(&w);
    a = __hmax2(a, __habs2(b));
    return *reinterpret_cast<uint32_t *>(&a);
}

template <typename T> __device__ __forceinline__ float bits16_to_float(uint32_t b);
template <> __device__ __forceinline__ float bits16_to_float<__half>(uint32_t b)
{
    return __half2float(__ushort_as_half((unsigned short)b));
}
template <> __device__ __forceinline__ float bits16_to_float<__nv_bfloat16>(uint32_t b)
{
    return __uint_as_float(b << 16);
}

__device__ __forceinline__ uint4 ldg_nc_v4(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// ---------------------------------------------------------------- bounds-checked build
// With -DFPSK_DEBUG_BOUNDS every index that a kernel takes from a table (a permutation entry, a bucket
// number, a decoded coordinate, a slot from a counter) is checked before it addresses memory: an index out of
// range is recorded (first one per source file: line, index, limit; and a count) and the access is skipped,
// so the kernel returns normally.  fpsk_debug_bounds_report (fpsk_test.h) reads the records.  In the product
// build the check compiles to `true`.
#ifdef FPSK_DEBUG_BOUNDS
struct BoundsRecord {
    unsigned int count;
    int line;
    long long index, limit;
};
static __device__ BoundsRecord g_bounds_tu;
__device__ __forceinline__ bool bounds_ok(long long idx, long long limit, int line)
{
    if (idx >= 0 && idx < limit) return true;
    if (atomicAdd(&g_bounds_tu.count, 1u) == 0u) {
        g_bounds_tu.line = line;
        g_bounds_tu.index = idx;
        g_bounds_tu.limit = limit;
    }
    return false;
}
#define FPSK_IN_BOUNDS(idx, limit) fpsk::bounds_ok((long long)(idx), (long long)(limit), __LINE__)
void bounds_register(const char *file, cudaError_t (*read)(BoundsRecord *), cudaError_t (*clear)());
namespace {
struct BoundsRegistration {
    BoundsRegistration()
    {
        bounds_register(__BASE_FILE__,
                        [](BoundsRecord *r) { return cudaMemcpyFromSymbol(r, g_bounds_tu, sizeof(*r)); },
                        []() { BoundsRecord z = {0u, 0, 0, 0}; return cudaMemcpyToSymbol(g_bounds_tu, &z, sizeof(z)); });
    }
} g_bounds_registration;
}  // namespace
#else
#define FPSK_IN_BOUNDS(idx, limit) true
#endif

// ---------------------------------------------------------------- bounded device-side wait
// Spin until *ctr >= target; gives up after a fixed number of polls and returns false, so
// that a kernel can flag FPSK_ERR_TIMEOUT and leave instead of hanging.
__device__ __forceinline__ bool bounded_wait_ge(const unsigned int *ctr, unsigned int target, unsigned int max_polls = 1u << 21)
{
    for (unsigned int it = 0; it < max_polls; ++it) {
        unsigned int v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr));
        if (v >= target) return true;
        __nanosleep(it < 64 ? 20 : 200);
    }
    return false;
}

// ---------------------------------------------------------------- internal launchers
struct ProbeDims {
    int64_t n1, n2, n3, lda, ldb, ldc;
};

fpsk_status probe_launch(const void *A, const void *B, const float *C, const ProbeDims &d,
                         fpsk_dtype dtype, double mu, void *ws, size_t ws_bytes, cudaStream_t st,
                         fpsk_probe_result *d_result, float *d_residual);
size_t probe_ws_bytes(int64_t n1, int64_t n2, int64_t n3);

}  // namespace fpsk
