// Detection probe: s = (1^T A) B - 1^T C, its noise estimate, threshold and verdict in one
// persistent cooperative kernel (Eq. (S) with H1 = 1^T, H2 = I; Section "Thresholds";
// Algorithm 2, probe part; Section "Nonfinite").
//
// Every CTA streams a row block of A (column sums -> partial u), then a row block of C
// (column sums), then, once all partial u are published, a row block of B (the GEMV u.B).
// The C phase sits between the A phase and the wait on it, so the wait is normally free.
// Partial vectors are combined in a fixed order: the result is deterministic.
#include "fpsk_common.cuh"

#include <math.h>
#include <mutex>

namespace fpsk {

constexpr int kProbeThreads = 512;
constexpr int kMaxTpr = 128;      // threads that share one row segment (x8 halves / x4 floats)
constexpr int kUChunk = 2048;     // u values staged in shared memory per GEMV chunk
constexpr int kCtrlWords = 64;

struct Decomp {
    int cg;      // column groups
    int rg;      // row groups; cg*rg <= grid
    int gwv;     // vectors (8 halves or 4 floats) per column group
    int stride;  // floats per partial row = cg*gwv*vec
};

struct ProbeArgs {
    const void *A, *B;
    const float *C;
    long long n1, n2, n3, lda, ldb, ldc;
    Decomp dA, dB, dC;
    unsigned int *ctrl;       // [0] A published, [1] partials published, [2] ticket
    float *partA, *partP, *partC;
    unsigned int *maxA, *maxB;   // per-CTA max |.| as 16-bit patterns
    float *s;                 // n3 floats
    fpsk_probe_result *result;
    float mu;
};

template <bool VEC>
__device__ __forceinline__ uint4 load8h(const unsigned short *X, long long ld, long long row,
                                        long long col0, long long cols)
{
    if (VEC) return ldg_nc_v4(X + row * ld + col0);
    unsigned int w[4] = {0, 0, 0, 0};
    const unsigned short *p = X + row * ld;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (col0 + e < cols) w[e >> 1] |= (unsigned int)p[col0 + e] << ((e & 1) * 16);
    return make_uint4(w[0], w[1], w[2], w[3]);
}

template <bool VEC>
__device__ __forceinline__ float4 load4f(const float *X, long long ld, long long row,
                                         long long col0, long long cols)
{
    if (VEC) {
        uint4 v = ldg_nc_v4(X + row * ld + col0);
        return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z),
                           __uint_as_float(v.w));
    }
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    const float *p = X + row * ld;
    if (col0 + 0 < cols) r.x = p[col0 + 0];
    if (col0 + 1 < cols) r.y = p[col0 + 1];
    if (col0 + 2 < cols) r.z = p[col0 + 2];
    if (col0 + 3 < cols) r.w = p[col0 + 3];
    return r;
}

template <typename T>
__device__ __forceinline__ void add8(float (&acc)[8], const uint4 &v, unsigned int &mx)
{
    float2 f;
    f = HalfTraits<T>::unpack2(v.x); acc[0] += f.x; acc[1] += f.y;
    f = HalfTraits<T>::unpack2(v.y); acc[2] += f.x; acc[3] += f.y;
    f = HalfTraits<T>::unpack2(v.z); acc[4] += f.x; acc[5] += f.y;
    f = HalfTraits<T>::unpack2(v.w); acc[6] += f.x; acc[7] += f.y;
    mx = max2_u16(mx, max2_u16(max2_u16(abs2_bits(v.x), abs2_bits(v.y)),
                               max2_u16(abs2_bits(v.z), abs2_bits(v.w))));
}

template <typename T>
__device__ __forceinline__ void fma8(float (&acc)[8], const uint4 &v, float u, unsigned int &mx)
{
    float2 f;
    f = HalfTraits<T>::unpack2(v.x); acc[0] = fmaf(u, f.x, acc[0]); acc[1] = fmaf(u, f.y, acc[1]);
    f = HalfTraits<T>::unpack2(v.y); acc[2] = fmaf(u, f.x, acc[2]); acc[3] = fmaf(u, f.y, acc[3]);
    f = HalfTraits<T>::unpack2(v.z); acc[4] = fmaf(u, f.x, acc[4]); acc[5] = fmaf(u, f.y, acc[5]);
    f = HalfTraits<T>::unpack2(v.w); acc[6] = fmaf(u, f.x, acc[6]); acc[7] = fmaf(u, f.y, acc[7]);
    mx = max2_u16(mx, max2_u16(max2_u16(abs2_bits(v.x), abs2_bits(v.y)),
                               max2_u16(abs2_bits(v.z), abs2_bits(v.w))));
}

// Sum the per-row-lane accumulators of a CTA in lane order and store the partial vector.
template <int NV>
__device__ __forceinline__ void reduce_lanes_store(const float (&acc)[NV], float *red, int tc, int rl,
                                                   int RL, int tpr, bool active, float *dst)
{
    __syncthreads();   // red may still be read by the previous phase
    if (active) {
#pragma unroll
        for (int e = 0; e < NV; ++e) red[(rl * tpr + tc) * NV + e] = acc[e];
    }
    __syncthreads();
    if (active && rl == 0) {
        float t[NV];
#pragma unroll
        for (int e = 0; e < NV; ++e) t[e] = red[tc * NV + e];
        for (int l = 1; l < RL; ++l) {
#pragma unroll
            for (int e = 0; e < NV; ++e) t[e] += red[(l * tpr + tc) * NV + e];
        }
#pragma unroll
        for (int e = 0; e < NV; ++e) __stcg(dst + tc * NV + e, t[e]);
    }
}

__device__ __forceinline__ unsigned int block_max_u16(unsigned int packed, unsigned int *sm)
{
    unsigned int m = max(packed & 0xFFFFu, packed >> 16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
    __syncthreads();
    unsigned int r = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r = max(r, sm[w]);
    return r;
}

// Column sums of a row block of a half-precision matrix.
template <typename T, bool VEC>
__device__ void colsum_half_phase(const unsigned short *X, long long ld, long long rows, long long cols,
                                  const Decomp &d, int c, float *part, unsigned int *maxout,
                                  float *red, unsigned int *smx)
{
    const int tpr = d.gwv, RL = kProbeThreads / tpr;
    const int tc = threadIdx.x % tpr, rl = threadIdx.x / tpr;
    const int cg = c % d.cg, rg = c / d.cg;
    const bool has_piece = rg < d.rg;
    const long long col0 = ((long long)cg * d.gwv + tc) * 8;
    const bool active = has_piece && rl < RL && col0 < cols;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    unsigned int mx = 0;
    if (active) {
        const long long r0 = rows * rg / d.rg, r1 = rows * (rg + 1) / d.rg;
        long long r = r0 + rl;
        constexpr int U = 8;
        for (; r + (long long)(U - 1) * RL < r1; r += (long long)U * RL) {
            uint4 v[U];
#pragma unroll
            for (int q = 0; q < U; ++q) v[q] = load8h<VEC>(X, ld, r + (long long)q * RL, col0, cols);
#pragma unroll
            for (int q = 0; q < U; ++q) add8<T>(acc, v[q], mx);
        }
        for (; r < r1; r += RL) {
            uint4 v = load8h<VEC>(X, ld, r, col0, cols);
            add8<T>(acc, v, mx);
        }
    }
    if (has_piece)
        reduce_lanes_store<8>(acc, red, tc, rl, RL, tpr, active,
                              part + (long long)rg * d.stride + (long long)cg * d.gwv * 8);
    else {
        __syncthreads();
        __syncthreads();
    }
    unsigned int m = block_max_u16(mx, smx);
    if (threadIdx.x == 0) __stcg(maxout + c, m);
}

// Column sums of a row block of the FP32 matrix C.
template <bool VEC>
__device__ void colsum_f32_phase(const float *X, long long ld, long long rows, long long cols,
                                 const Decomp &d, int c, float *part, float *red)
{
    const int tpr = d.gwv, RL = kProbeThreads / tpr;
    const int tc = threadIdx.x % tpr, rl = threadIdx.x / tpr;
    const int cg = c % d.cg, rg = c / d.cg;
    const bool has_piece = rg < d.rg;
    const long long col0 = ((long long)cg * d.gwv + tc) * 4;
    const bool active = has_piece && rl < RL && col0 < cols;
    float acc[4] = {0, 0, 0, 0};
    if (active) {
        const long long r0 = rows * rg / d.rg, r1 = rows * (rg + 1) / d.rg;
        long long r = r0 + rl;
        constexpr int U = 8;
        for (; r + (long long)(U - 1) * RL < r1; r += (long long)U * RL) {
            float4 v[U];
#pragma unroll
            for (int q = 0; q < U; ++q) v[q] = load4f<VEC>(X, ld, r + (long long)q * RL, col0, cols);
#pragma unroll
            for (int q = 0; q < U; ++q) {
                acc[0] += v[q].x; acc[1] += v[q].y; acc[2] += v[q].z; acc[3] += v[q].w;
            }
        }
        for (; r < r1; r += RL) {
            float4 v = load4f<VEC>(X, ld, r, col0, cols);
            acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
        }
    }
    if (has_piece)
        reduce_lanes_store<4>(acc, red, tc, rl, RL, tpr, active,
                              part + (long long)rg * d.stride + (long long)cg * d.gwv * 4);
    else {
        __syncthreads();
        __syncthreads();
    }
}

// p-partial of a row block of B: sum_k u_k B_kj over the block's k range.
template <typename T, bool VEC>
__device__ void gemv_phase(const unsigned short *X, long long ld, long long rows, long long cols,
                           const Decomp &d, int c, const float *partA, const Decomp &dA,
                           float *part, unsigned int *maxout, float *red, float *us, unsigned int *smx)
{
    const int tpr = d.gwv, RL = kProbeThreads / tpr;
    const int tc = threadIdx.x % tpr, rl = threadIdx.x / tpr;
    const int cg = c % d.cg, rg = c / d.cg;
    const bool has_piece = rg < d.rg;
    const long long col0 = ((long long)cg * d.gwv + tc) * 8;
    const bool active = has_piece && rl < RL && col0 < cols;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    unsigned int mx = 0;
    const long long r0 = has_piece ? rows * rg / d.rg : 0, r1 = has_piece ? rows * (rg + 1) / d.rg : 0;
    for (long long base = r0; base < r1; base += kUChunk) {
        const int cnt = (int)min((long long)kUChunk, r1 - base);
        __syncthreads();
        // u_k = sum of the published partial column sums of A, in row-group order
        for (int t = threadIdx.x; t < cnt; t += kProbeThreads) {
            const float *src = partA + (base + t);
            float u = __ldcg(src);
            for (int g = 1; g < dA.rg; ++g) u += __ldcg(src + (long long)g * dA.stride);
            us[t] = u;
        }
        __syncthreads();
        if (active) {
            int t = rl;
            constexpr int U = 8;
            for (; t + (U - 1) * RL < cnt; t += U * RL) {
                uint4 v[U];
#pragma unroll
                for (int q = 0; q < U; ++q) v[q] = load8h<VEC>(X, ld, base + t + q * RL, col0, cols);
#pragma unroll
                for (int q = 0; q < U; ++q) fma8<T>(acc, v[q], us[t + q * RL], mx);
            }
            for (; t < cnt; t += RL) {
                uint4 v = load8h<VEC>(X, ld, base + t, col0, cols);
                fma8<T>(acc, v, us[t], mx);
            }
        }
    }
    if (has_piece)
        reduce_lanes_store<8>(acc, red, tc, rl, RL, tpr, active,
                              part + (long long)rg * d.stride + (long long)cg * d.gwv * 8);
    else {
        __syncthreads();
        __syncthreads();
    }
    unsigned int m = block_max_u16(mx, smx);
    if (threadIdx.x == 0) __stcg(maxout + c, m);
}

struct ArgMax {
    float v;
    int i;
};
__device__ __forceinline__ ArgMax amax(ArgMax a, ArgMax b)
{
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}

// Deterministic block sum: per-thread values combined by a fixed tree.
__device__ __forceinline__ float block_sum(float v, float *sm)
{
    __syncthreads();
    sm[threadIdx.x] = v;
    __syncthreads();
    for (int s = kProbeThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) sm[threadIdx.x] += sm[threadIdx.x + s];
        __syncthreads();
    }
    return sm[0];
}

template <typename T>
__device__ void verdict(const ProbeArgs &p, int grid, float *red, int status)
{
    const int n = (int)p.n3;
    float sum = 0.f;
    ArgMax am = {-1.f, 0x7FFFFFFF};
    int bad = 0;
    for (int j = threadIdx.x; j < n; j += kProbeThreads) {
        float a = fabsf(__ldcg(p.s + j));
        sum += a;
        if (!(a <= 3.402823466e38f)) bad = 1;          // Inf or NaN
        am = amax(am, ArgMax{(a != a) ? -1.f : a, j});
    }
    const float mean_abs = block_sum(sum, red) / (float)n;
    float csum = 0.f;
    const float clip = 5.f * mean_abs;
    for (int j = threadIdx.x; j < n; j += kProbeThreads) csum += fminf(fabsf(__ldcg(p.s + j)), clip);
    const float sigma = 1.2533f * (block_sum(csum, red) / (float)n);
    // arg max and flags
    __syncthreads();
    ArgMax *ams = reinterpret_cast<ArgMax *>(red);
    ams[threadIdx.x] = am;
    __syncthreads();
    for (int s = kProbeThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) ams[threadIdx.x] = amax(ams[threadIdx.x], ams[threadIdx.x + s]);
        __syncthreads();
    }
    am = ams[0];
    const int anybad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        unsigned int ma = 0, mb = 0;
        for (int c = 0; c < grid; ++c) {
            ma = max(ma, __ldcg(p.maxA + c));
            mb = max(mb, __ldcg(p.maxB + c));
        }
        const float tau = 100.f * (float)p.n2 * 1.1920928955078125e-07f * bits16_to_float<T>(ma) *
                          bits16_to_float<T>(mb);
        const float nb = (float)(n > 2 ? n : 2);
        const float thr = fminf(tau, p.mu * sqrtf(2.f * logf(nb)) * sigma);
        fpsk_probe_result r;
        r.nonfinite = anybad ? 1 : 0;
        r.fired = (anybad || am.v > thr) ? 1 : 0;
        r.argmax_col = am.i;
        r.status = status;
        r.max_abs = am.v;
        r.sigma_hat = sigma;
        r.thr = thr;
        r.tau = tau;
        *p.result = r;
    }
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(kProbeThreads, 2) probe_kernel(const ProbeArgs p)
{
    __shared__ __align__(16) float red[kProbeThreads * 8];
    __shared__ float us[kUChunk];
    __shared__ unsigned int smx[kProbeThreads / 32];
    __shared__ int s_flag;
    const int c = blockIdx.x, G = gridDim.x;
    const unsigned short *A = static_cast<const unsigned short *>(p.A);
    const unsigned short *B = static_cast<const unsigned short *>(p.B);

    colsum_half_phase<T, VEC>(A, p.lda, p.n1, p.n2, p.dA, c, p.partA, p.maxA, red, smx);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(p.ctrl + 0, 1u);
    }
    colsum_f32_phase<VEC>(p.C, p.ldc, p.n1, p.n3, p.dC, c, p.partC, red);

    if (threadIdx.x == 0) s_flag = bounded_wait_ge(p.ctrl + 0, (unsigned)G) ? 1 : 0;
    __syncthreads();
    int ok = s_flag;
    if (ok) gemv_phase<T, VEC>(B, p.ldb, p.n2, p.n3, p.dB, c, p.partA, p.dA, p.partP, p.maxB, red, us, smx);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(p.ctrl + 1, 1u);
        s_flag = (ok && bounded_wait_ge(p.ctrl + 1, (unsigned)G)) ? 1 : 0;
    }
    __syncthreads();
    ok = s_flag;
    if (ok) {
        // s_j for this CTA's slice of columns: partial p minus partial column sums of C
        const long long j0 = p.n3 * c / G, j1 = p.n3 * (c + 1) / G;
        for (long long j = j0 + threadIdx.x; j < j1; j += kProbeThreads) {
            float pj = __ldcg(p.partP + j);
            for (int g = 1; g < p.dB.rg; ++g) pj += __ldcg(p.partP + (long long)g * p.dB.stride + j);
            float cj = __ldcg(p.partC + j);
            for (int g = 1; g < p.dC.rg; ++g) cj += __ldcg(p.partC + (long long)g * p.dC.stride + j);
            __stcg(p.s + j, pj - cj);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (!ok) atomicOr(p.ctrl + 3, 1u);
        unsigned int t = atomicAdd(p.ctrl + 2, 1u);
        s_flag = (t == (unsigned)G - 1) ? 1 : 0;
    }
    __syncthreads();
    if (s_flag) {   // the last CTA through: everything is published
        __threadfence();
        const int failed = (int)__ldcg(p.ctrl + 3);
        verdict<T>(p, G, red, failed ? (int)FPSK_ERR_TIMEOUT : (int)FPSK_OK);
        __syncthreads();
        if (threadIdx.x == 0 && !failed) {
            // self-reset for the next launch (after a timeout the host must re-initialise)
            p.ctrl[0] = 0; p.ctrl[1] = 0; p.ctrl[2] = 0;
        }
    }
}

// ---------------------------------------------------------------- host side
struct DevInfo {
    int sms = 0;
    int grid = 0;
};
static DevInfo g_dev[64];
static std::mutex g_dev_mu;

static fpsk_status probe_grid(int &grid)
{
    int dev = 0;
    FPSK_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return FPSK_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_dev_mu);
    if (g_dev[dev].grid == 0) {
        int sms = 0, occ = 0, o2 = 0;
        FPSK_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        // the four instantiations have near-identical resource use; take the minimum
        FPSK_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, probe_kernel<__half, true>, kProbeThreads, 0));
        FPSK_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, probe_kernel<__nv_bfloat16, true>, kProbeThreads, 0));
        occ = occ < o2 ? occ : o2;
        FPSK_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, probe_kernel<__half, false>, kProbeThreads, 0));
        occ = occ < o2 ? occ : o2;
        FPSK_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, probe_kernel<__nv_bfloat16, false>, kProbeThreads, 0));
        occ = occ < o2 ? occ : o2;
        if (occ < 1 || sms < 1) return FPSK_ERR_CUDA;
        if (occ > 2) occ = 2;
        g_dev[dev].sms = sms;
        g_dev[dev].grid = sms * occ;
    }
    grid = g_dev[dev].grid;
    return FPSK_OK;
}

// Upper bound used for workspace sizing when no device is present / before the first launch.
constexpr int kMaxGrid = 1024;

static bool make_decomp(long long cols, int vec, int grid, Decomp &d)
{
    long long wv = (cols + vec - 1) / vec;
    long long cg = (wv + kMaxTpr - 1) / kMaxTpr;
    if (cg > grid) return false;
    d.cg = (int)cg;
    d.gwv = (int)((wv + cg - 1) / cg);
    d.rg = grid / d.cg;
    d.stride = d.cg * d.gwv * vec;
    return true;
}

static size_t part_floats(long long cols, int vec)
{
    // rows of partials <= kMaxGrid/cg; stride <= cols + cg*vec  ->  bounded by kMaxGrid*kMaxTpr*vec + slack
    long long wv = (cols + vec - 1) / vec;
    long long cg = (wv + kMaxTpr - 1) / kMaxTpr;
    long long gwv = (wv + cg - 1) / cg;
    long long rg = kMaxGrid / cg;
    if (rg < 1) rg = 1;
    return (size_t)(rg * cg * gwv * vec);
}

size_t probe_ws_bytes(int64_t n1, int64_t n2, int64_t n3)
{
    if (n1 < 1 || n2 < 1 || n3 < 1) return 0;
    size_t b = 256;                                      // control words
    b += align_up(part_floats(n2, 8) * 4, 256);          // partA
    b += align_up(part_floats(n3, 8) * 4, 256);          // partP
    b += align_up(part_floats(n3, 4) * 4, 256);          // partC
    b += align_up((size_t)kMaxGrid * 4, 256) * 2;        // maxA, maxB
    b += align_up((size_t)n3 * 4, 256);                  // s
    return b;
}

fpsk_status probe_launch(const void *A, const void *B, const float *C, const ProbeDims &d,
                         fpsk_dtype dtype, double mu, void *ws, size_t ws_bytes, cudaStream_t st,
                         fpsk_probe_result *d_result, float *d_residual)
{
    int grid = 0;
    fpsk_status rc = probe_grid(grid);
    if (rc != FPSK_OK) return rc;
    if (grid > kMaxGrid) grid = kMaxGrid;
    ProbeArgs p;
    p.A = A; p.B = B; p.C = C;
    p.n1 = d.n1; p.n2 = d.n2; p.n3 = d.n3; p.lda = d.lda; p.ldb = d.ldb; p.ldc = d.ldc;
    if (!make_decomp(d.n2, 8, grid, p.dA) || !make_decomp(d.n3, 8, grid, p.dB) ||
        !make_decomp(d.n3, 4, grid, p.dC))
        return FPSK_ERR_SHAPE;
    if (ws_bytes < probe_ws_bytes(d.n1, d.n2, d.n3)) return FPSK_ERR_WORKSPACE;
    char *w = static_cast<char *>(ws);
    p.ctrl = reinterpret_cast<unsigned int *>(w); w += 256;
    p.partA = reinterpret_cast<float *>(w); w += align_up(part_floats(d.n2, 8) * 4, 256);
    p.partP = reinterpret_cast<float *>(w); w += align_up(part_floats(d.n3, 8) * 4, 256);
    p.partC = reinterpret_cast<float *>(w); w += align_up(part_floats(d.n3, 4) * 4, 256);
    p.maxA = reinterpret_cast<unsigned int *>(w); w += align_up((size_t)kMaxGrid * 4, 256);
    p.maxB = reinterpret_cast<unsigned int *>(w); w += align_up((size_t)kMaxGrid * 4, 256);
    p.s = d_residual ? d_residual : reinterpret_cast<float *>(w);
    p.result = d_result;
    p.mu = (float)mu;

    const bool vec = ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) |
                       reinterpret_cast<uintptr_t>(C)) & 15) == 0 &&
                     d.lda % 8 == 0 && d.ldb % 8 == 0 && d.ldc % 4 == 0 && d.n2 % 8 == 0 &&
                     d.n3 % 8 == 0;
    void *args[] = {&p};
    const void *fn;
    if (dtype == FPSK_FP16)
        fn = vec ? (const void *)probe_kernel<__half, true> : (const void *)probe_kernel<__half, false>;
    else
        fn = vec ? (const void *)probe_kernel<__nv_bfloat16, true> : (const void *)probe_kernel<__nv_bfloat16, false>;
    FPSK_CUDA_OK(cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kProbeThreads), args, 0, st));
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

}  // namespace fpsk
