// Device helpers shared by the streaming kernels: mbarrier waits with a time bound, bulk
// (TMA engine) global->shared copies, publication counters, and 16-bit-float lane helpers
// (mixed-precision FP32 accumulation, packed min/max tracking).
#pragma once
#include "fpsk_common.cuh"

namespace fpsk {

// Running min and max of packed pairs of 16-bit floats (two HMNMX2 per word, no integer work;
// NaN operands are ignored).  max|x| follows from both at the end.
template <typename T> struct MinMax2 {
    uint32_t mx, mn;
    __device__ __forceinline__ void init();
    __device__ __forceinline__ void upd(uint32_t w);
    __device__ __forceinline__ float absmax() const;   // >= 0; 0 when nothing was seen
};
template <> __device__ __forceinline__ void MinMax2<__half>::init() { mx = 0xFC00FC00u; mn = 0x7C007C00u; }
template <> __device__ __forceinline__ void MinMax2<__nv_bfloat16>::init() { mx = 0xFF80FF80u; mn = 0x7F807F80u; }
template <> __device__ __forceinline__ void MinMax2<__half>::upd(uint32_t w)
{
    __half2 a = *reinterpret_cast<__half2 *>(&mx), b = *reinterpret_cast<__half2 *>(&mn), x = *reinterpret_cast<__half2 *>(&w);
    a = __hmax2(a, x);
    b = __hmin2(b, x);
    mx = *reinterpret_cast<uint32_t *>(&a);
    mn = *reinterpret_cast<uint32_t *>(&b);
}
template <> __device__ __forceinline__ void MinMax2<__nv_bfloat16>::upd(uint32_t w)
{
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&mx), b = *reinterpret_cast<__nv_bfloat162 *>(&mn),
                   x = *reinterpret_cast<__nv_bfloat162 *>(&w);
    a = __hmax2(a, x);
    b = __hmin2(b, x);
    mx = *reinterpret_cast<uint32_t *>(&a);
    mn = *reinterpret_cast<uint32_t *>(&b);
}
template <typename T> __device__ __forceinline__ float MinMax2<T>::absmax() const
{
    const float a = fmaxf(bits16_to_float<T>(mx & 0xFFFFu), bits16_to_float<T>(mx >> 16));
    const float b = fminf(bits16_to_float<T>(mn & 0xFFFFu), bits16_to_float<T>(mn >> 16));
    return fmaxf(fmaxf(a, -b), 0.f);
}
// exact 16-bit pattern of a non-negative value that is representable in T
template <typename T> __device__ __forceinline__ unsigned int float_to_bits16(float x);
template <> __device__ __forceinline__ unsigned int float_to_bits16<__half>(float x)
{
    return (unsigned int)__half_as_ushort(__float2half_rn(x));
}
template <> __device__ __forceinline__ unsigned int float_to_bits16<__nv_bfloat16>(float x)
{
    return __float_as_uint(x) >> 16;
}

// acc[e] += x_e for the 8 half-precision values of a 16-byte vector, with the mixed-precision
// add of sm_100 (add.f32.f16 / add.f32.bf16: FP32 accumulate of a 16-bit operand, one FP
// instruction per element and no unpacking on the integer pipe).
template <typename T> __device__ __forceinline__ void madd2(float &a0, float &a1, uint32_t w);
template <> __device__ __forceinline__ void madd2<__half>(float &a0, float &a1, uint32_t w)
{
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.f32.f16 %0, lo, %0;\n\tadd.f32.f16 %1, hi, %1;\n\t}"
        : "+f"(a0), "+f"(a1) : "r"(w));
}
template <> __device__ __forceinline__ void madd2<__nv_bfloat16>(float &a0, float &a1, uint32_t w)
{
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.f32.bf16 %0, lo, %0;\n\tadd.f32.bf16 %1, hi, %1;\n\t}"
        : "+f"(a0), "+f"(a1) : "r"(w));
}
template <typename T>
__device__ __forceinline__ void add8m(float2 (&acc)[4], const uint4 &v, MinMax2<T> &mm)
{
    madd2<T>(acc[0].x, acc[0].y, v.x);
    madd2<T>(acc[1].x, acc[1].y, v.y);
    madd2<T>(acc[2].x, acc[2].y, v.z);
    madd2<T>(acc[3].x, acc[3].y, v.w);
    mm.upd(v.x); mm.upd(v.y); mm.upd(v.z); mm.upd(v.w);
}
template <typename T>
__device__ __forceinline__ void fma8m(float2 (&acc)[4], const uint4 &v, float u, MinMax2<T> &mm)
{
    const float2 uu = make_float2(u, u);
    acc[0] = __ffma2_rn(uu, HalfTraits<T>::unpack2(v.x), acc[0]);
    acc[1] = __ffma2_rn(uu, HalfTraits<T>::unpack2(v.y), acc[1]);
    acc[2] = __ffma2_rn(uu, HalfTraits<T>::unpack2(v.z), acc[2]);
    acc[3] = __ffma2_rn(uu, HalfTraits<T>::unpack2(v.w), acc[3]);
    mm.upd(v.x); mm.upd(v.y); mm.upd(v.z); mm.upd(v.w);
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on an mbarrier phase: gives up (returns false) after about a second of polling
// instead of spinning forever.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity)
{
    const long long t_end = clock64() + 2000000000LL;
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 1024; ++it)
            if (mbar_try(bar, parity)) return true;
        if (clock64() > t_end) return false;
    }
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    if (mbar_try(bar, parity)) return true;       // the common case: one instruction
    return mbar_wait_slow(bar, parity);
}
// The same for a whole warp: lane 0 polls, the outcome is broadcast, and __syncwarp orders the
// other lanes' later reads after lane 0's observation of the completed phase.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity)
{
    int w = 1;
    if ((threadIdx.x & 31) == 0) w = mbar_wait_bounded(bar, parity) ? 1 : 0;
    w = __shfl_sync(0xFFFFFFFFu, w, 0);
    __syncwarp();
    return w != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Publication counters: a release-add makes everything this thread has observed (its own writes
// and, through the preceding CTA barrier, its CTA's) visible before the count; the ticket is an
// acquire-release add, so the last arriver also sees what every earlier arriver published.
__device__ __forceinline__ void red_release_add(unsigned int *ctr)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(ctr), "r"(1u) : "memory");
}
__device__ __forceinline__ unsigned int atom_acq_rel_add(unsigned int *ctr)
{
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(ctr), "r"(1u) : "memory");
    return old;
}
// Cross-proxy fence between the generic proxy (ordinary loads/stores) and the async proxy (bulk
// copies): a thread that has observed a publication (acquire) executes it before it issues bulk
// copies of the published data.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

}  // namespace fpsk
