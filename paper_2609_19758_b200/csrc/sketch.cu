// Hashed moment sketches S, R, T of E = AB - C for one hash round, without forming AB
// (Section "Moment Sketches", Eq. (S)):  (H1 A)(B H2^T) - H1 C H2^T and the index-weighted
// forms.  All accumulation is FP32 in a fixed order: no float atomics anywhere, so results
// are bit-reproducible run to run.
//
//   hash_kernel / scan_kernel / place_kernel   hash tables and bucket-sorted permutations
//   compress_a_kernel   P = H1 A, Pw = H1 W1 A          (m_b x n2, rows grouped by bucket)
//   compress_b_kernel / compress_b8_kernel (B as k x n) / compress_wt_kernel (the weight W = B^T)
//                       Q = B H2^T, Qw = B W2 H2^T      (n2 x m_b)
//   sgemm_kernel        S_AB = P Q, R_AB = Pw Q, T_AB = P Qw   (FP32 SIMT, split-K partials); with the tensor-core
//                       contraction (tc_contract.cu) the compressions write scaled FP16 planes instead of P, Q
//   scatter_c_kernel / scatter_c2_kernel   S_C, R_C, T_C: one streaming pass over C per round
//   combine_kernel      S = sum of AB partials - sum of C partials
// The column side + B compression and the C scatter run on auxiliary streams when the caller provides them.
#include "sketch.cuh"
#include "stream_pipe.cuh"

#include <mutex>
#include <vector>

namespace fpsk {

// ---------------------------------------------------------------- hash tables
__global__ void hash_kernel(uint32_t key, int n, int m_b, int *bucket, int *sign, int *count)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    int b, s;
    hash_index(key, (uint32_t)idx, (uint32_t)m_b, b, s);
    bucket[idx] = b;
    sign[idx] = s;
    if (count) atomicAdd(count + b, 1);
}

// exclusive scan of count[0..m_b) into start[0..m_b]; single CTA
__global__ void scan_kernel(const int *count, int m_b, int *start)
{
    __shared__ int carry;
    __shared__ int buf[1024];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < m_b; base += 1024) {
        int i = base + threadIdx.x;
        int v = i < m_b ? count[i] : 0;
        buf[threadIdx.x] = v;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            int t = threadIdx.x >= o ? buf[threadIdx.x - o] : 0;
            __syncthreads();
            buf[threadIdx.x] += t;
            __syncthreads();
        }
        if (i < m_b) start[i] = carry + buf[threadIdx.x] - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry += buf[1023];
        __syncthreads();
    }
    if (threadIdx.x == 0) start[m_b] = carry;
}

// Stable placement: entry idx goes to start[b] + (number of idx' < idx in the same bucket).
// perm packs the index (low 31 bits) and the sign (bit 31 set = -1).  One warp per entry: the
// lanes share the scan over the earlier entries, so the O(n^2 / 2) comparisons spread over the
// whole GPU.
__global__ void __launch_bounds__(256) place_kernel(const int *bucket, const int *sign, const int *start, int n, uint32_t *perm,
                                                    uint32_t *pos)
{
    const int idx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (idx >= n) return;
    const int b = __ldg(bucket + idx);
    int cnt = 0;
    int j = lane;
    for (; j + 96 < idx; j += 128) {
        const int b0 = __ldg(bucket + j), b1 = __ldg(bucket + j + 32), b2 = __ldg(bucket + j + 64), b3 = __ldg(bucket + j + 96);
        cnt += (b0 == b) + (b1 == b) + (b2 == b) + (b3 == b);
    }
    for (; j < idx; j += 32) cnt += (__ldg(bucket + j) == b);
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if (lane == 0) {
        const uint32_t sbit = __ldg(sign + idx) < 0 ? 0x80000000u : 0u;
        const uint32_t where = (uint32_t)(__ldg(start + b) + cnt);
        if (FPSK_IN_BOUNDS(where, n)) perm[where] = (uint32_t)idx | sbit;
        if (pos) pos[idx] = where | sbit;        // the inverse: where entry idx sits in the sorted order (and its sign)
    }
}

fpsk_status build_hash_side(uint64_t seed, int rnd, int side, int n, int m_b, int *bucket, int *sign,
                            int *count, int *start, uint32_t *perm, cudaStream_t st, uint32_t *pos)
{
    const uint32_t key = round_key(seed, rnd, side);
    if (count) FPSK_CUDA_OK(cudaMemsetAsync(count, 0, sizeof(int) * (size_t)m_b, st));
    hash_kernel<<<(n + 255) / 256, 256, 0, st>>>(key, n, m_b, bucket, sign, count);
    FPSK_LAUNCH_CHECK();
    if (!perm) return FPSK_OK;
    scan_kernel<<<1, 1024, 0, st>>>(count, m_b, start);
    FPSK_LAUNCH_CHECK();
    place_kernel<<<(n + 7) / 8, 256, 0, st>>>(bucket, sign, start, n, perm, pos);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// Eight FP32 values, scaled by a power of two -> the 16-byte chunks of their two FP16 terms (x = hi + lo up to
// 2^-24 |x|: the remainder x - hi is exact in FP32 and lo rounds it to 11 bits).
__device__ __forceinline__ void split8_f16(const float (&x)[8], float scale, uint4 &hi, uint4 &lo)
{
    unsigned short h[8], l[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float xs = x[j] * scale;
        const __half bh = __float2half_rn(xs);
        const float r1 = xs - __half2float(bh);
        const __half bl = __float2half_rn(r1);
        h[j] = __half_as_ushort(bh); l[j] = __half_as_ushort(bl);
    }
    hi = make_uint4(h[0] | ((unsigned)h[1] << 16), h[2] | ((unsigned)h[3] << 16), h[4] | ((unsigned)h[5] << 16), h[6] | ((unsigned)h[7] << 16));
    lo = make_uint4(l[0] | ((unsigned)l[1] << 16), l[2] | ((unsigned)l[3] << 16), l[4] | ((unsigned)l[5] << 16), l[6] | ((unsigned)l[7] << 16));
}
// Where the chunk (row r, eight k starting at k0) of a tiled operand plane sits (layout of tc_contract.cu):
// tiles of R rows by 32 k, the planes of a tile back to back.
template <int R>
__device__ __forceinline__ size_t plane_chunk_offset(int r, int k0, int kblocks)
{
    const int rt = r / R, rr = r % R, kb = k0 >> 5, kc = (k0 & 31) >> 3;
    return ((size_t)rt * kblocks + kb) * kTcPlanes * (size_t)(R * 64) + (size_t)(kc * (R / 8) + rr / 8) * 128 + (size_t)(rr % 8) * 16;
}

__global__ void __launch_bounds__(256) tc_scale_kernel(const int *count, int m_b, const float *maxv, float *scale)
{
    __shared__ int wmax[8];
    int c = 0;
    for (int b = threadIdx.x; b < m_b; b += blockDim.x) c = max(c, count[b]);
    c = __reduce_max_sync(0xFFFFFFFFu, c);
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) c = max(c, wmax[w]);
        scale[0] = tc_scale_of(c, maxv[0]);
    }
}
fpsk_status tc_scale_launch(const int *count, int m_b, const float *maxv, float *scale, cudaStream_t st)
{
    tc_scale_kernel<<<1, 256, 0, st>>>(count, m_b, maxv, scale);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- A compression
// CTA (x: group of 8-column vectors, y: bucket a).  Thread owns 8 adjacent columns and walks
// the rows of bucket a in ascending row order.
// PLANES: the sums go out as tiled BF16 planes for the tensor-core contraction (K extent kblocks * 32,
// zero beyond n2) instead of FP32 rows of P, Pw.
template <typename T, bool VEC, bool MOM, bool PLANES>
__global__ void __launch_bounds__(128) compress_a_kernel(const unsigned short *A, long long lda, int n1, int n2,
                                                         int kpad, float inv_p1, const uint32_t *rowperm,
                                                         const int *rowstart, float *P, float *Pw, int kblocks,
                                                         unsigned char *planesP, unsigned char *planesPw, int m_b,
                                                         const float *tc_scale)
{
    // FP32 output: CTA = one bucket, consecutive threads = consecutive columns.  Plane output: a warp covers
    // eight consecutive buckets x four k-chunks, because the eight buckets of a k-chunk are one 128-byte
    // line of the tiled plane (lone 16-byte chunks, one bucket per CTA, take three times as long to store).
    const int a = PLANES ? (int)blockIdx.y * 8 + (int)(threadIdx.x & 7) : (int)blockIdx.y;
    const long long col0 = PLANES ? ((long long)blockIdx.x * (blockDim.x / 8) + (threadIdx.x >> 3)) * 8
                                  : ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 8;
    if (col0 >= (PLANES ? kblocks * 32 : kpad)) return;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, accw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (col0 < n2 && a < m_b) {
        const int s0 = rowstart[a], s1 = rowstart[a + 1];
        // eight rows in flight (a bucket of the noise measurement has a hundred rows: one load at a time is all latency);
        // the additions stay in row order
        for (int s = s0; s < s1; s += 8) {
            uint32_t e[8];
            uint4 v[8];
            bool ok[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                e[u] = s + u < s1 ? __ldg(rowperm + s + u) : 0u;
                const int i = (int)(e[u] & 0x7FFFFFFFu);
                ok[u] = s + u < s1 && FPSK_IN_BOUNDS(s + u, n1) && FPSK_IN_BOUNDS(i, n1);
                v[u] = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    if (VEC) v[u] = ldg_nc_v4(A + (long long)i * lda + col0);
                    else {
                        unsigned int w[4] = {0, 0, 0, 0};
                        for (int q = 0; q < 8; ++q)
                            if (col0 + q < n2) w[q >> 1] |= (unsigned int)A[(long long)i * lda + col0 + q] << ((q & 1) * 16);
                        v[u] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (!ok[u]) continue;
                const int i = (int)(e[u] & 0x7FFFFFFFu);
                const float sg = (e[u] >> 31) ? -1.f : 1.f;
                const float swi = sg * ((float)(i + 1) * inv_p1);
                const unsigned int ww[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float2 f = HalfTraits<T>::unpack2(ww[q]);
                    acc[2 * q] += sg * f.x;
                    acc[2 * q + 1] += sg * f.y;
                    if (MOM) {
                        accw[2 * q] = fmaf(swi, f.x, accw[2 * q]);
                        accw[2 * q + 1] = fmaf(swi, f.y, accw[2 * q + 1]);
                    }
                }
            }
        }
    }
    if (PLANES) {
        const size_t off = plane_chunk_offset<128>(a, (int)col0, kblocks);
        const float sc = __ldg(tc_scale);
        uint4 hi, lo;
        split8_f16(acc, sc, hi, lo);
        *reinterpret_cast<uint4 *>(planesP + off) = hi;
        *reinterpret_cast<uint4 *>(planesP + off + 128 * 64) = lo;
        if (MOM) {
            split8_f16(accw, sc, hi, lo);
            *reinterpret_cast<uint4 *>(planesPw + off) = hi;
            *reinterpret_cast<uint4 *>(planesPw + off + 128 * 64) = lo;
        }
        return;
    }
    float4 *dp = reinterpret_cast<float4 *>(P + (long long)a * kpad + col0);
    dp[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    dp[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    if (MOM) {
        float4 *dw = reinterpret_cast<float4 *>(Pw + (long long)a * kpad + col0);
        dw[0] = make_float4(accw[0], accw[1], accw[2], accw[3]);
        dw[1] = make_float4(accw[4], accw[5], accw[6], accw[7]);
    }
}

// ---------------------------------------------------------------- B compression
// One row of B at a time staged in shared memory; thread b folds the columns of bucket b in
// ascending column order.  Rows k >= n2 (padding of the contraction) are written as zeros.
template <typename T, bool MOM>
__global__ void __launch_bounds__(256) compress_b_kernel(const unsigned short *B, long long ldb, int n2, int n3,
                                                         int kpad, int m_b, int npad, float inv_p3,
                                                         const uint32_t *colperm, const int *colstart,
                                                         float *Q, float *Qw)
{
    extern __shared__ __align__(16) unsigned short rowbuf[];
    for (int k = blockIdx.x; k < kpad; k += gridDim.x) {
        if (k >= n2) {
            for (int b = threadIdx.x; b < npad; b += blockDim.x) {
                Q[(long long)k * npad + b] = 0.f;
                if (MOM) Qw[(long long)k * npad + b] = 0.f;
            }
            continue;
        }
        __syncthreads();
        const unsigned short *src = B + (long long)k * ldb;
        if (((reinterpret_cast<uintptr_t>(src) & 15) == 0) && (n3 % 8 == 0)) {
            for (int j = threadIdx.x * 8; j < n3; j += blockDim.x * 8)
                *reinterpret_cast<uint4 *>(rowbuf + j) = ldg_nc_v4(src + j);
        } else {
            for (int j = threadIdx.x; j < n3; j += blockDim.x) rowbuf[j] = src[j];
        }
        __syncthreads();
        for (int b = threadIdx.x; b < npad; b += blockDim.x) {
            float q = 0.f, qw = 0.f;
            if (b < m_b) {
                const int s0 = __ldg(colstart + b), s1 = __ldg(colstart + b + 1);
                for (int s = s0; s < s1; ++s) {
                    const uint32_t e = __ldg(colperm + s);
                    const int j = (int)(e & 0x7FFFFFFFu);
                    if (!FPSK_IN_BOUNDS(s, n3) || !FPSK_IN_BOUNDS(j, n3)) continue;
                    const float sg = (e >> 31) ? -1.f : 1.f;
                    const float x = bits16_to_float<T>(rowbuf[j]);
                    q += sg * x;
                    if (MOM) qw = fmaf(sg * ((float)(j + 1) * inv_p3), x, qw);
                }
            }
            Q[(long long)k * npad + b] = q;
            if (MOM) Qw[(long long)k * npad + b] = qw;
        }
    }
}

// ---------------------------------------------------------------- B compression from the transposed weight
// B given as W = B^T (n3 x n2, row-major: the x W^T layout of a linear layer).  Column j of B is row j of W, so
// the fold over the columns of bucket b is a sum of rows of W, the mirror image of the A compression: a thread
// owns eight adjacent k of one bucket and walks the bucket's rows in ascending j, which is the order of
// additions of the kernels above (same bits).  Lanes: eight consecutive buckets x four k-chunks per warp, so
// that a warp stores whole 128-byte lines of the tiled planes (32-byte runs of the FP32 rows of Q).  Writes the
// padding too: buckets up to bmax and k up to kend are zeros.
template <typename T, bool VEC, bool MOM, bool PLANES>
__global__ void __launch_bounds__(128) compress_wt_kernel(const unsigned short *Wt, long long ldw, int n2, int n3,
                                                          int kpad, int m_b, int npad, float inv_p3,
                                                          const uint32_t *colperm, const int *colstart, float *Q,
                                                          float *Qw, int kblocks, int btiles, unsigned char *planesQ,
                                                          unsigned char *planesQw, const float *tc_scale)
{
    const int b = (int)blockIdx.y * 8 + (int)(threadIdx.x & 7);
    const int k0 = ((int)blockIdx.x * (int)(blockDim.x / 8) + (int)(threadIdx.x >> 3)) * 8;
    const int kend = PLANES ? kblocks * 32 : kpad;
    const int bmax = PLANES ? btiles * 256 : npad;
    if (k0 >= kend || b >= bmax) return;
    float q[8] = {0, 0, 0, 0, 0, 0, 0, 0}, qw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (k0 < n2 && b < m_b) {
        const int s0 = colstart[b], s1 = colstart[b + 1];
        // eight rows of W in flight, the additions in row order (as in compress_a_kernel)
        for (int s = s0; s < s1; s += 8) {
            uint32_t e[8];
            uint4 v[8];
            bool ok[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                e[u] = s + u < s1 ? __ldg(colperm + s + u) : 0u;
                const int j = (int)(e[u] & 0x7FFFFFFFu);
                ok[u] = s + u < s1 && FPSK_IN_BOUNDS(s + u, n3) && FPSK_IN_BOUNDS(j, n3);
                v[u] = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    if (VEC) v[u] = ldg_nc_v4(Wt + (long long)j * ldw + k0);
                    else {
                        unsigned int w[4] = {0, 0, 0, 0};
                        for (int t = 0; t < 8; ++t)
                            if (k0 + t < n2) w[t >> 1] |= (unsigned int)Wt[(long long)j * ldw + k0 + t] << ((t & 1) * 16);
                        v[u] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (!ok[u]) continue;
                const int j = (int)(e[u] & 0x7FFFFFFFu);
                const float sg = (e[u] >> 31) ? -1.f : 1.f;
                const float swj = sg * ((float)(j + 1) * inv_p3);
                const unsigned int ww[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float2 f = HalfTraits<T>::unpack2(ww[t]);
                    q[2 * t] += sg * f.x;
                    q[2 * t + 1] += sg * f.y;
                    if (MOM) {
                        qw[2 * t] = fmaf(swj, f.x, qw[2 * t]);
                        qw[2 * t + 1] = fmaf(swj, f.y, qw[2 * t + 1]);
                    }
                }
            }
        }
    }
    if (PLANES) {
        const size_t off = plane_chunk_offset<256>(b, k0, kblocks);
        const float sc = __ldg(tc_scale);
        uint4 hi, lo;
        split8_f16(q, sc, hi, lo);
        *reinterpret_cast<uint4 *>(planesQ + off) = hi;
        *reinterpret_cast<uint4 *>(planesQ + off + 256 * 64) = lo;
        if (MOM) {
            split8_f16(qw, sc, hi, lo);
            *reinterpret_cast<uint4 *>(planesQw + off) = hi;
            *reinterpret_cast<uint4 *>(planesQw + off + 256 * 64) = lo;
        }
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            if (k0 + t < kpad) {
                Q[(long long)(k0 + t) * npad + b] = q[t];
                if (MOM) Qw[(long long)(k0 + t) * npad + b] = qw[t];
            }
        }
    }
}

// ---------------------------------------------------------------- compressions straight into the tiled planes
// Row-bucket sums of a row-major half-precision matrix X (rows of A grouped by h1, or rows of W = B^T grouped by
// h2), written as the scaled FP16 hi/lo planes of the tensor-core contraction (R-row tiles, see plane_chunk_offset).
// A CTA takes eight consecutive buckets and 256 consecutive k: warp w owns bucket 8 * blockIdx.y + w and its lanes
// run along k, so every row is read in one 512-byte piece (the kernels above give a warp eight buckets and read
// 64 bytes per row and warp); up to four rows of the bucket are in flight per thread.  The sums are split, turned
// through shared memory, and leave as full 128-byte lines: the eight buckets of a k-chunk are one line of the plane.
// Same additions in the same order as compress_a_kernel / compress_wt_kernel: same bits.
template <typename T, int R, bool VEC, bool MOM>
__global__ void __launch_bounds__(256, 6) compress_planes_kernel(const unsigned short *X, long long ld, int nrows, int n2,
                                                                 float inv_p, const uint32_t *perm, const int *start, int m_b,
                                                                 int kblocks, unsigned char *planes, unsigned char *planes_w,
                                                                 const float *tc_scale)
{
    __shared__ uint4 tile[MOM ? 4 : 2][32 * 9];          // [plane][k-chunk l][bucket w] as l * 9 + w (padded: no bank conflicts)
    const int w = (int)threadIdx.x >> 5, l = (int)threadIdx.x & 31;
    const int a = (int)blockIdx.y * 8 + w;
    const int k0 = ((int)blockIdx.x * 32 + l) * 8;
    const int kend = kblocks * 32;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, accw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (k0 < n2 && a < m_b) {
        const int s0 = start[a], s1 = start[a + 1];
        for (int sb = s0; sb < s1; sb += 4) {
            uint32_t e[4];
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) e[u] = sb + u < s1 ? __ldg(perm + sb + u) : 0u;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = (int)(e[u] & 0x7FFFFFFFu);
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (sb + u >= s1 || !FPSK_IN_BOUNDS(sb + u, nrows) || !FPSK_IN_BOUNDS(i, nrows)) continue;
                if (VEC) v[u] = ldg_nc_v4(X + (long long)i * ld + k0);
                else {
                    unsigned int ww[4] = {0, 0, 0, 0};
                    for (int q = 0; q < 8; ++q)
                        if (k0 + q < n2) ww[q >> 1] |= (unsigned int)X[(long long)i * ld + k0 + q] << ((q & 1) * 16);
                    v[u] = make_uint4(ww[0], ww[1], ww[2], ww[3]);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (sb + u >= s1) break;
                const int i = (int)(e[u] & 0x7FFFFFFFu);
                const float sg = (e[u] >> 31) ? -1.f : 1.f;
                const float swi = sg * ((float)(i + 1) * inv_p);
                const unsigned int ww[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float2 f = HalfTraits<T>::unpack2(ww[q]);
                    acc[2 * q] += sg * f.x;
                    acc[2 * q + 1] += sg * f.y;
                    if (MOM) {
                        accw[2 * q] = fmaf(swi, f.x, accw[2 * q]);
                        accw[2 * q + 1] = fmaf(swi, f.y, accw[2 * q + 1]);
                    }
                }
            }
        }
    }
    const float sc = __ldg(tc_scale);
    uint4 hi, lo;
    split8_f16(acc, sc, hi, lo);
    tile[0][l * 9 + w] = hi;
    tile[1][l * 9 + w] = lo;
    if (MOM) {
        split8_f16(accw, sc, hi, lo);
        tile[2][l * 9 + w] = hi;
        tile[3][l * 9 + w] = lo;
    }
    __syncthreads();
    // thread t stores 16-byte slot t & 7 of line t >> 3 (k-chunk): a warp writes four full lines
    const int t = (int)threadIdx.x, lc = t >> 3, slot = t & 7;
    const int kc0 = ((int)blockIdx.x * 32 + lc) * 8;
    const int ab = (int)blockIdx.y * 8 + slot;
    if (kc0 < kend) {
        const size_t off = plane_chunk_offset<R>(ab, kc0, kblocks);
        const int ti = lc * 9 + slot;
        *reinterpret_cast<uint4 *>(planes + off) = tile[0][ti];
        *reinterpret_cast<uint4 *>(planes + off + R * 64) = tile[1][ti];
        if (MOM) {
            *reinterpret_cast<uint4 *>(planes_w + off) = tile[2][ti];
            *reinterpret_cast<uint4 *>(planes_w + off + R * 64) = tile[3][ti];
        }
    }
}

// ---------------------------------------------------------------- C scatter
// CTA (x: bucket row a, y: split).  The rows of bucket a (ascending) are divided among the
// splits; each row of C is staged in shared memory and folded over its columns by bucket;
// the three accumulators of bucket row a live in shared memory, one owner thread per b.
// The same with eight consecutive rows of B per pass: the column lists are walked once for eight rows,
// the barriers are amortised, and the eight sums of a bucket are exactly one 16-byte chunk of the tiled
// BF16 planes (PLANES: emitted directly, K extent kblocks * 32 and bucket extent btiles * 256, zero
// padded; otherwise FP32 rows of Q, Qw as above).  Same order of additions per row as the kernel above.
template <typename T, bool MOM, bool PLANES>
__global__ void __launch_bounds__(1024) compress_b8_kernel(const unsigned short *B, long long ldb, int n2, int n3,
                                                          int kpad, int m_b, int npad, float inv_p3,
                                                          const uint32_t *colperm, const int *colstart, float *Q,
                                                          float *Qw, int kblocks, int btiles, unsigned char *planesQ,
                                                          unsigned char *planesQw, const float *tc_scale, const uint32_t *colpos)
{
    extern __shared__ __align__(16) unsigned short rowbuf8[];
    const int n3p = (n3 + 7) & ~7;
    const int kend = PLANES ? kblocks * 32 : kpad;
    const int bmax = PLANES ? btiles * 256 : npad;
    // S only into FP32 Q, aligned B (the noise measurement below the tensor cores' bucket count): the eight rows go into
    // shared memory in bucket-sorted column order, sign applied (colpos: position and sign of every column), and a
    // thread per (bucket, row) adds a contiguous run - the bucket's columns in ascending order, as below: the same
    // additions in the same order, without the gather through the column list and with every thread at work also
    // when the buckets are few.
    const bool sorted_rows = !PLANES && !MOM && n3 % 8 == 0 && ldb % 8 == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0;
    if (sorted_rows) {
        const int rs = n3p + 2;               // row stride in shared memory: the eight rows of a bucket's run fall into eight banks
        for (int k0 = blockIdx.x * 8; k0 < kend; k0 += gridDim.x * 8) {
            __syncthreads();
            for (int j = threadIdx.x * 8; j < n3; j += blockDim.x * 8) {
                const uint4 c0 = __ldg(reinterpret_cast<const uint4 *>(colpos + j)), c1 = __ldg(reinterpret_cast<const uint4 *>(colpos + j + 4));
                const uint32_t cp[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                uint4 v[8];
#pragma unroll
                for (int r = 0; r < 8; ++r) v[r] = k0 + r < n2 ? ldg_nc_v4(B + (long long)(k0 + r) * ldb + j) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const unsigned int ww[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint32_t pos = cp[q] & 0x7FFFFFFFu;
                        if (!FPSK_IN_BOUNDS(pos, n3)) continue;
                        const unsigned short h = (unsigned short)(ww[q >> 1] >> ((q & 1) * 16));
                        rowbuf8[(size_t)r * rs + pos] = (unsigned short)(h ^ ((cp[q] >> 31) ? 0x8000u : 0u));
                    }
                }
            }
            __syncthreads();
            for (int it = threadIdx.x; it < bmax * 8; it += blockDim.x) {
                const int b = it >> 3, r = it & 7;
                float q1 = 0.f;
                if (b < m_b) {
                    const int s0 = __ldg(colstart + b), s1 = __ldg(colstart + b + 1);
                    const unsigned short *rowp = rowbuf8 + (size_t)r * rs;
                    for (int sx = s0; sx < s1; sx += 8) {
                        unsigned short h[8];              // eight loads in flight, then added in order
#pragma unroll
                        for (int u = 0; u < 8; ++u) h[u] = sx + u < s1 ? rowp[sx + u] : (unsigned short)0;
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if (sx + u < s1) q1 += bits16_to_float<T>(h[u]);
                    }
                }
                if (k0 + r < kpad) Q[(long long)(k0 + r) * npad + b] = q1;
            }
        }
        return;
    }
    for (int k0 = blockIdx.x * 8; k0 < kend; k0 += gridDim.x * 8) {
        __syncthreads();
        for (int r = 0; r < 8; ++r) {
            unsigned short *dstrow = rowbuf8 + (size_t)r * n3p;
            if (k0 + r >= n2) {
                for (int j = threadIdx.x * 8; j < n3p; j += blockDim.x * 8) *reinterpret_cast<uint4 *>(dstrow + j) = make_uint4(0, 0, 0, 0);
                continue;
            }
            const unsigned short *src = B + (long long)(k0 + r) * ldb;
            if (((reinterpret_cast<uintptr_t>(src) & 15) == 0) && (n3 % 8 == 0)) {
                for (int j = threadIdx.x * 8; j < n3; j += blockDim.x * 8) *reinterpret_cast<uint4 *>(dstrow + j) = ldg_nc_v4(src + j);
            } else {
                for (int j = threadIdx.x; j < n3; j += blockDim.x) dstrow[j] = src[j];
            }
        }
        __syncthreads();
        for (int b = threadIdx.x; b < bmax; b += blockDim.x) {
            float q[8] = {0, 0, 0, 0, 0, 0, 0, 0}, qw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (b < m_b) {
                const int s0 = __ldg(colstart + b), s1 = __ldg(colstart + b + 1);
                for (int s = s0; s < s1; ++s) {
                    const uint32_t e = __ldg(colperm + s);
                    const int j = (int)(e & 0x7FFFFFFFu);
                    if (!FPSK_IN_BOUNDS(s, n3) || !FPSK_IN_BOUNDS(j, n3)) continue;
                    const float sg = (e >> 31) ? -1.f : 1.f;
                    const float swj = sg * ((float)(j + 1) * inv_p3);
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const float x = bits16_to_float<T>(rowbuf8[(size_t)r * n3p + j]);
                        q[r] += sg * x;
                        if (MOM) qw[r] = fmaf(swj, x, qw[r]);
                    }
                }
            }
            if (PLANES) {
                const size_t off = plane_chunk_offset<256>(b, k0, kblocks);
                const float sc = __ldg(tc_scale);
                uint4 hi, lo;
                split8_f16(q, sc, hi, lo);
                *reinterpret_cast<uint4 *>(planesQ + off) = hi;
                *reinterpret_cast<uint4 *>(planesQ + off + 256 * 64) = lo;
                if (MOM) {
                    split8_f16(qw, sc, hi, lo);
                    *reinterpret_cast<uint4 *>(planesQw + off) = hi;
                    *reinterpret_cast<uint4 *>(planesQw + off + 256 * 64) = lo;
                }
            } else {
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    if (k0 + r < kpad) {
                        Q[(long long)(k0 + r) * npad + b] = q[r];
                        if (MOM) Qw[(long long)(k0 + r) * npad + b] = qw[r];
                    }
                }
            }
        }
    }
}

// CTA (bucket a, row split).  Columns go in chunks of kScChunk: every thread sums the signed (and
// row-weighted) rows of the bucket for its own columns in registers - no barrier per row, sixteen
// independent loads per thread and row in flight - then the chunk's column sums go through shared
// memory once and thread b folds the columns of bucket b (ascending) into S, R, T.
constexpr int kScChunk = 4096;
template <bool MOM, bool VEC>
__global__ void __launch_bounds__(256) scatter_c_kernel(const float *C, long long ldc, int n1, int n3, int m_b,
                                                        float inv_p1, float inv_p3, const uint32_t *rowperm,
                                                        const int *rowstart, const uint32_t *colperm,
                                                        const int *colstart, int nsplit, float *part)
{
    extern __shared__ __align__(16) float sm[];
    float *tS = sm;                           // kScChunk
    float *tR = sm + kScChunk;                // kScChunk
    float *accS = sm + 2 * kScChunk;
    float *accR = accS + m_b;
    float *accT = accR + m_b;
    const int a = blockIdx.x, sp = blockIdx.y;
    for (int b = threadIdx.x; b < m_b; b += blockDim.x) {
        accS[b] = 0.f;
        if (MOM) { accR[b] = 0.f; accT[b] = 0.f; }
    }
    const int s0 = rowstart[a], s1 = rowstart[a + 1];
    const int cnt = s1 - s0;
    const int q0 = s0 + (int)((long long)cnt * sp / nsplit), q1 = s0 + (int)((long long)cnt * (sp + 1) / nsplit);
    for (int c0 = 0; c0 < n3; c0 += kScChunk) {
        const int cw = min(kScChunk, n3 - c0);
        float4 rs[4], rr[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { rs[q] = make_float4(0.f, 0.f, 0.f, 0.f); rr[q] = make_float4(0.f, 0.f, 0.f, 0.f); }
        for (int s = q0; s < q1; ++s) {
            const uint32_t e = __ldg(rowperm + s);
            const int i = (int)(e & 0x7FFFFFFFu);
            if (!FPSK_IN_BOUNDS(s, n1) || !FPSK_IN_BOUNDS(i, n1)) continue;
            const float v1 = (e >> 31) ? -1.f : 1.f;
            const float v1w = v1 * ((float)(i + 1) * inv_p1);
            const float *src = C + (long long)i * ldc + c0;
            float4 x[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int j = q * 1024 + threadIdx.x * 4;
                if (VEC) {
                    x[q] = j < cw ? __ldg(reinterpret_cast<const float4 *>(src + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
                } else {
                    x[q].x = j + 0 < cw ? src[j + 0] : 0.f;
                    x[q].y = j + 1 < cw ? src[j + 1] : 0.f;
                    x[q].z = j + 2 < cw ? src[j + 2] : 0.f;
                    x[q].w = j + 3 < cw ? src[j + 3] : 0.f;
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                rs[q].x = fmaf(v1, x[q].x, rs[q].x); rs[q].y = fmaf(v1, x[q].y, rs[q].y);
                rs[q].z = fmaf(v1, x[q].z, rs[q].z); rs[q].w = fmaf(v1, x[q].w, rs[q].w);
                if (MOM) {
                    rr[q].x = fmaf(v1w, x[q].x, rr[q].x); rr[q].y = fmaf(v1w, x[q].y, rr[q].y);
                    rr[q].z = fmaf(v1w, x[q].z, rr[q].z); rr[q].w = fmaf(v1w, x[q].w, rr[q].w);
                }
            }
        }
        __syncthreads();                      // the previous chunk's fold has finished reading tS, tR
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = q * 1024 + threadIdx.x * 4;
            *reinterpret_cast<float4 *>(tS + j) = rs[q];
            if (MOM) *reinterpret_cast<float4 *>(tR + j) = rr[q];
        }
        __syncthreads();
        for (int b = threadIdx.x; b < m_b; b += blockDim.x) {
            const int k0 = __ldg(colstart + b), k1 = __ldg(colstart + b + 1);
            float fs = 0.f, fr = 0.f, ft = 0.f;
            for (int c = k0; c < k1; ++c) {
                const uint32_t ce = __ldg(colperm + c);
                if (!FPSK_IN_BOUNDS(c, n3) || !FPSK_IN_BOUNDS(ce & 0x7FFFFFFFu, n3)) continue;
                const int j = (int)(ce & 0x7FFFFFFFu) - c0;
                if (j < 0 || j >= cw) continue;
                const float sg = (ce >> 31) ? -1.f : 1.f;
                const float x = tS[j];
                fs += sg * x;
                if (MOM) {
                    ft = fmaf(sg * ((float)(j + c0 + 1) * inv_p3), x, ft);
                    fr += sg * tR[j];
                }
            }
            accS[b] += fs;
            if (MOM) { accR[b] += fr; accT[b] += ft; }
        }
    }
    __syncthreads();
    const long long mm = (long long)m_b * m_b;
    float *dst = part + (long long)sp * 3 * mm + (long long)a * m_b;
    for (int b = threadIdx.x; b < m_b; b += blockDim.x) {
        dst[b] = accS[b];
        if (MOM) { dst[mm + b] = accR[b]; dst[2 * mm + b] = accT[b]; }
    }
}

// The same scatter for column counts whose three sorted column-sum vectors fit in shared memory
// (n3 <= kSc2MaxCols).  Four rows of the bucket are in flight per thread, and every thread writes its
// column sums, signed (and column-weighted for T), straight to the position its column has in the
// bucket-sorted order (colpos, the inverse permutation): a bucket's entries are then contiguous and the
// fold is a sum over a range, in the same ascending column order as the kernel above, with the bucket
// boundaries fetched into shared memory while the rows stream.  Measured at 1024 buckets on 4096^2 FP32:
// 34 us against 36 us; a CTA lives about 7 us (start 0.7, rows 2.5, scatter 1.0, fold 2.3) and two fit an SM.
constexpr int kSc2MaxCols = 16384;
template <bool MOM, bool VEC>
__global__ void __launch_bounds__(256, 2) scatter_c2_kernel(const float *C, long long ldc, int n1, int n3, int m_b,
                                                            float inv_p1, float inv_p3, const uint32_t *rowperm,
                                                            const int *rowstart, const uint32_t *colpos,
                                                            const int *colstart, int nsplit, float *part)
{
    extern __shared__ __align__(16) float sm2[];
    const int n3p = (n3 + 3) & ~3;
    float *ts = sm2;                          // sorted, signed column sums
    float *tt = sm2 + n3p;                    // ... times the column weight
    float *tr = sm2 + 2 * n3p;                // row-weighted
    int *cs = reinterpret_cast<int *>(sm2 + (MOM ? 3 : 1) * n3p);   // bucket boundaries, fetched while the rows stream
    for (int b = threadIdx.x; b <= m_b; b += blockDim.x) cs[b] = __ldg(colstart + b);
    const int a = blockIdx.x, sp = blockIdx.y;
    const int s0 = rowstart[a], s1 = rowstart[a + 1];
    const int cnt = s1 - s0;
    const int q0 = s0 + (int)((long long)cnt * sp / nsplit), q1 = s0 + (int)((long long)cnt * (sp + 1) / nsplit);
    for (int c0 = 0; c0 < n3; c0 += kScChunk) {
        const int cw = min(kScChunk, n3 - c0);
        // where my sixteen columns go (independent of the rows: in flight with them)
        uint4 cp[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = q * 1024 + threadIdx.x * 4;
            if (VEC) cp[q] = j < cw ? __ldg(reinterpret_cast<const uint4 *>(colpos + c0 + j)) : make_uint4(0, 0, 0, 0);
            else {
                cp[q].x = j + 0 < cw ? __ldg(colpos + c0 + j + 0) : 0u;
                cp[q].y = j + 1 < cw ? __ldg(colpos + c0 + j + 1) : 0u;
                cp[q].z = j + 2 < cw ? __ldg(colpos + c0 + j + 2) : 0u;
                cp[q].w = j + 3 < cw ? __ldg(colpos + c0 + j + 3) : 0u;
            }
        }
        float4 rs[4], rr[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { rs[q] = make_float4(0.f, 0.f, 0.f, 0.f); rr[q] = make_float4(0.f, 0.f, 0.f, 0.f); }
        for (int sb = q0; sb < q1; sb += 4) {
            uint32_t e4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) e4[u] = sb + u < q1 ? __ldg(rowperm + sb + u) : 0u;
            float4 x[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float *src = C + (long long)(e4[u] & 0x7FFFFFFFu) * ldc + c0;
                const bool live = sb + u < q1 && FPSK_IN_BOUNDS(sb + u, n1) && FPSK_IN_BOUNDS(e4[u] & 0x7FFFFFFFu, n1);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j = q * 1024 + threadIdx.x * 4;
                    if (!live || j >= cw) { x[u][q] = make_float4(0.f, 0.f, 0.f, 0.f); continue; }
                    if (VEC) x[u][q] = __ldg(reinterpret_cast<const float4 *>(src + j));
                    else {
                        x[u][q].x = src[j];
                        x[u][q].y = j + 1 < cw ? src[j + 1] : 0.f;
                        x[u][q].z = j + 2 < cw ? src[j + 2] : 0.f;
                        x[u][q].w = j + 3 < cw ? src[j + 3] : 0.f;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (sb + u >= q1) break;
                const int i = (int)(e4[u] & 0x7FFFFFFFu);
                const float v1 = (e4[u] >> 31) ? -1.f : 1.f;
                const float v1w = v1 * ((float)(i + 1) * inv_p1);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    rs[q].x = fmaf(v1, x[u][q].x, rs[q].x); rs[q].y = fmaf(v1, x[u][q].y, rs[q].y);
                    rs[q].z = fmaf(v1, x[u][q].z, rs[q].z); rs[q].w = fmaf(v1, x[u][q].w, rs[q].w);
                    if (MOM) {
                        rr[q].x = fmaf(v1w, x[u][q].x, rr[q].x); rr[q].y = fmaf(v1w, x[u][q].y, rr[q].y);
                        rr[q].z = fmaf(v1w, x[u][q].z, rr[q].z); rr[q].w = fmaf(v1w, x[u][q].w, rr[q].w);
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = q * 1024 + threadIdx.x * 4;
            const uint32_t cpe[4] = {cp[q].x, cp[q].y, cp[q].z, cp[q].w};
            const float rse[4] = {rs[q].x, rs[q].y, rs[q].z, rs[q].w};
            const float rre[4] = {rr[q].x, rr[q].y, rr[q].z, rr[q].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (j + e >= cw) continue;
                const uint32_t pos = cpe[e] & 0x7FFFFFFFu;
                if (!FPSK_IN_BOUNDS(pos, n3)) continue;
                const float sg = (cpe[e] >> 31) ? -1.f : 1.f;
                ts[pos] = sg * rse[e];
                if (MOM) {
                    tt[pos] = (sg * ((float)(c0 + j + e + 1) * inv_p3)) * rse[e];
                    tr[pos] = sg * rre[e];
                }
            }
        }
    }
    __syncthreads();
    const long long mm = (long long)m_b * m_b;
    float *dst = part + (long long)sp * 3 * mm + (long long)a * m_b;
    for (int b = threadIdx.x; b < m_b; b += blockDim.x) {
        const int k0 = cs[b], k1 = cs[b + 1];
        float fs = 0.f, fr = 0.f, ft = 0.f;
        for (int c = k0; c < k1; ++c) {
            fs += ts[c];
            if (MOM) { ft += tt[c]; fr += tr[c]; }
        }
        dst[b] = fs;
        if (MOM) { dst[mm + b] = fr; dst[2 * mm + b] = ft; }
    }
}

// ---------------------------------------------------------------- the C scatter as a producer/consumer ring
// The same reduction as scatter_c2_kernel<false, true> (S only, aligned C), same additions in the same order, as a
// persistent kernel: one CTA per SM; a producer warp that streams the rows of a unit (row bucket a, row split) with
// one bulk copy per 16 KB piece of a row into a ring of shared-memory stages of two rows; sixteen consumer warps that
// add the signed rows in registers and write the column sums of a unit to their bucket-sorted positions; and, where
// shared memory has room for two such buffers, eight folder warps that add them up by column bucket while the
// consumers are already on the next unit (with one buffer the consumers fold themselves).  The rows of the next
// units are in flight all the while (in the kernels above a CTA streams, scatters and folds in turn).  Units are
// handed out by a device counter, so CTAs that meet small buckets take more of them.  Every wait is bounded: a
// thread that gives up sets ctrl[1], which the caller reads after the launch.
constexpr int kSrStageBytes0 = 16384;
constexpr int kSrConsumers = 512;
struct SrSync {   // named barrier over the consumer warps of scatter_ring_kernel
    static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }
};
constexpr int kSrQ = kSrStageBytes0 / 16 / kSrConsumers;     // float4 per consumer thread and stage
constexpr int kSrFolders = 256;                // warps that fold a unit's sorted column sums while the next unit's rows are added
constexpr int kSrThreads = kSrConsumers + 32 + kSrFolders;
constexpr int kSrRowBytes = kSrStageBytes0;   // one row of a 4096-column chunk
constexpr int kSrRows = 2;                    // rows of a chunk per stage: the per-stage hand-over is paid once for both
constexpr int kSrStageBytes = kSrRows * kSrRowBytes;
constexpr int kSrStages = 4;                  // at most; fewer where the two buffers of column sums leave less room
struct SrUnit { int a, sp, flags, pad; };     // flags: 1 nothing was added (write zeros), 2 no more units
struct SrMeta {                               // what the consumers need to know about a stage
    int flags;                                // 1 first rows of a chunk, 2 last rows of a chunk, 4 last stage of the unit, 8 no more units
    int valid;                                // bit r: row r of the stage was copied
    float sign[kSrRows];
    int a, sp, c0, cw;
};
struct SrArgs {
    const float *C;
    long long ldc;
    int n1, n3, m_b, nsplit, n_units, nst;    // nst: ring stages in use
    const uint32_t *rowperm, *colpos;
    const int *rowstart, *colstart;
    float *part;
    unsigned int *ctrl;                       // [0] unit counter (zero before the launch), [1] set when a bounded wait gave up
};

// Bucket sums of one unit from its sorted column sums: thread per column bucket, the columns of a bucket added in
// their sorted order; two buckets per thread at a time, so that their loads are independent.
static __device__ __forceinline__ void sr_fold(const float *ts, const int *cs, float *dst, int m_b, int t, int nt, bool empty_unit)
{
    for (int b = t; b < m_b; b += 2 * nt) {
        const int b2 = b + nt;
        float fa = 0.f, fb = 0.f;
        if (!empty_unit) {
            int ca = cs[b], cb = 0, eb = 0;
            const int ea = cs[b + 1];
            if (b2 < m_b) { cb = cs[b2]; eb = cs[b2 + 1]; }
            while (ca < ea || cb < eb) {
                const float xa = ca < ea ? ts[ca] : 0.f;
                const float xb = cb < eb ? ts[cb] : 0.f;
                if (ca < ea) { fa += xa; ++ca; }
                if (cb < eb) { fb += xb; ++cb; }
            }
        }
        dst[b] = fa;
        if (b2 < m_b) dst[b2] = fb;
    }
}

template <bool FW>     // FW: a group of folder warps and two buffers of column sums; otherwise the consumers fold, one buffer
__global__ void __launch_bounds__(FW ? kSrThreads : kSrConsumers + 32, 1) scatter_ring_kernel(const SrArgs p)
{
    extern __shared__ __align__(128) unsigned char sr_smem[];
    unsigned char *ring = sr_smem;
    const int n3p = (p.n3 + 3) & ~3;
    float *ts0 = reinterpret_cast<float *>(sr_smem + (size_t)p.nst * kSrStageBytes);  // sorted, signed column sums of a unit, two buffers
    int *cs = reinterpret_cast<int *>(ts0 + (FW ? 2 : 1) * n3p);                               // bucket boundaries in the sorted order
    SrMeta *meta = reinterpret_cast<SrMeta *>(cs + ((p.m_b + 1 + 3) & ~3));
    SrUnit *umeta = reinterpret_cast<SrUnit *>(meta + kSrStages);
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(umeta + 2);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kSrStages);
    const uint32_t tsfull0 = smem_u32(bars + 2 * kSrStages), tsfree0 = smem_u32(bars + 2 * kSrStages + 2);
    const int tid = (int)threadIdx.x;
    if (tid == kSrConsumers) {
        for (int s = 0; s < kSrStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kSrConsumers / 32);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(tsfull0 + 8 * s, kSrConsumers);
            mbar_init(tsfree0 + 8 * s, kSrFolders);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (tid < kSrConsumers)
        for (int b = tid; b <= p.m_b; b += kSrConsumers) cs[b] = __ldg(p.colstart + b);
    __syncthreads();
    const long long mm = (long long)p.m_b * p.m_b;
    if (FW && tid >= kSrConsumers + 32) {
        // ------------------------------------------------------------ folder warps
        // Bucket sums of one unit: thread per column bucket, the columns of a bucket added in their sorted order.
        const int ft = tid - (kSrConsumers + 32);
        int fb = 0;
        uint32_t fph = 0;                     // bit b: parity of the next phase of buffer b
        for (;;) {
            if (!mbar_wait_warp(tsfull0 + 8 * fb, (fph >> fb) & 1u)) { if (ft == 0) atomicOr(p.ctrl + 1, 1u); break; }
            const SrUnit um = umeta[fb];
            if (um.flags & 2) break;
            const float *ts = ts0 + (size_t)fb * n3p;
            float *dst = p.part + (long long)um.sp * 3 * mm + (long long)um.a * p.m_b;
            const bool empty_unit = um.flags & 1;
            sr_fold(ts, cs, dst, p.m_b, ft, kSrFolders, empty_unit);
            mbar_arrive(tsfree0 + 8 * fb);    // every folder thread: its reads of the buffer are done
            fph ^= 1u << fb;
            fb ^= 1;
        }
        return;
    }
    if (tid >= kSrConsumers) {
        // ------------------------------------------------------------ producer warp
        // What a unit needs before its first copy can be issued is a chain of three dependent loads (unit counter,
        // bucket boundaries, row indices), about 2 us when taken one after the other - longer than the copies of the
        // unit take.  So the chain is a three-deep pipeline over the units: while the rows of unit k are issued, the
        // row indices of unit k + 1, the boundaries of unit k + 2 and the number of unit k + 3 are in flight.  Lane l
        // holds the index of row l of a unit (further groups of 32 rows are fetched in place); lane 0 issues.
        const int lane = tid & 31;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        auto next_stage = [&](const SrMeta &m, const float *src0, const float *src1, uint32_t bytes) {      // lane 0 only
            if (!mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u)) { ok = false; return; }
            meta[stage] = m;
            if (m.valid) {
                mbar_expect_tx(full0 + 8 * stage, bytes * (uint32_t)__popc(m.valid));
                const uint32_t dst = smem_u32(ring + (size_t)stage * kSrStageBytes);
                if (m.valid & 1) bulk_g2s(dst, src0, bytes, full0 + 8 * stage);
                if (m.valid & 2) bulk_g2s(dst + kSrRowBytes, src1, bytes, full0 + 8 * stage);
            } else {
                mbar_arrive(full0 + 8 * stage);
            }
            if (++stage == p.nst) { stage = 0; phase ^= 1u; }
        };
        auto take_unit = [&]() {
            int u = 0;
            if (lane == 0) u = (int)atomicAdd(p.ctrl, 1u);
            return __shfl_sync(0xFFFFFFFFu, u, 0);
        };
        auto bounds_of = [&](int u, int &q0, int &q1) {
            q0 = q1 = 0;
            if (u >= p.n_units) return;
            const int a = u % p.m_b, sp = u / p.m_b;
            const int s0 = __ldg(p.rowstart + a), s1 = __ldg(p.rowstart + a + 1);
            const int cnt = s1 - s0;
            q0 = s0 + (int)((long long)cnt * sp / p.nsplit);
            q1 = s0 + (int)((long long)cnt * (sp + 1) / p.nsplit);
        };
        // prologue: fill the pipeline
        int u_c = take_unit();                                  // unit whose rows are issued next
        int q0_c, q1_c;
        bounds_of(u_c, q0_c, q1_c);
        uint32_t e_c = q0_c + lane < q1_c ? __ldg(p.rowperm + q0_c + lane) : 0u;
        int u_b = take_unit();                                  // unit one behind: boundaries known
        int q0_b, q1_b;
        bounds_of(u_b, q0_b, q1_b);
        int u_a = take_unit();                                  // unit two behind: number known
        while (u_c < p.n_units) {
            // the loads of the following units first (independent of one another and of the copies below)
            const int u_new = take_unit();
            int q0_a, q1_a;
            bounds_of(u_a, q0_a, q1_a);
            const uint32_t e_b = q0_b + lane < q1_b ? __ldg(p.rowperm + q0_b + lane) : 0u;
            // ---- the rows of the present unit
            const int a = u_c % p.m_b, sp = u_c / p.m_b;
            if (q1_c <= q0_c) {
                if (lane == 0) {
                    SrMeta m = {1 | 2 | 4, 0, {0.f, 0.f}, a, sp, 0, 0};        // nothing to add: the consumers write zeros
                    next_stage(m, nullptr, nullptr, 0);
                }
            } else {
                for (int c0 = 0; c0 < p.n3; c0 += kSrRowBytes / 4) {
                    const int cw = min(kSrRowBytes / 4, p.n3 - c0);
                    const bool last_chunk = c0 + kSrRowBytes / 4 >= p.n3;
                    for (int base = q0_c; base < q1_c; base += 32) {
                        const uint32_t eg = base == q0_c ? e_c : (base + lane < q1_c ? __ldg(p.rowperm + base + lane) : 0u);
                        const int ng = min(32, q1_c - base);
                        for (int r = 0; r < ng; r += kSrRows) {
                            const uint32_t e0 = __shfl_sync(0xFFFFFFFFu, eg, r);
                            const uint32_t e1 = __shfl_sync(0xFFFFFFFFu, eg, (r + 1) & 31);
                            if (lane != 0 || !ok) continue;
                            const int sidx = base + r;
                            const bool two = r + 1 < ng;
                            const int last = sidx + (two ? 1 : 0);
                            const int i0 = (int)(e0 & 0x7FFFFFFFu), i1 = (int)(e1 & 0x7FFFFFFFu);
                            SrMeta m;
                            m.flags = (sidx == q0_c ? 1 : 0) | (last == q1_c - 1 ? 2 : 0) | ((last == q1_c - 1 && last_chunk) ? 4 : 0);
                            m.valid = 0;
                            if (FPSK_IN_BOUNDS(sidx, p.n1) && FPSK_IN_BOUNDS(i0, p.n1)) m.valid |= 1;
                            if (two && FPSK_IN_BOUNDS(last, p.n1) && FPSK_IN_BOUNDS(i1, p.n1)) m.valid |= 2;
                            m.sign[0] = (e0 >> 31) ? -1.f : 1.f;
                            m.sign[1] = (e1 >> 31) ? -1.f : 1.f;
                            m.a = a; m.sp = sp; m.c0 = c0; m.cw = cw;
                            next_stage(m, p.C + (long long)i0 * p.ldc + c0, p.C + (long long)i1 * p.ldc + c0, (uint32_t)cw * 4u);
                        }
                    }
                }
            }
            if (!__shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0)) break;
            // ---- rotate the pipeline
            u_c = u_b; q0_c = q0_b; q1_c = q1_b; e_c = e_b;
            u_b = u_a; q0_b = q0_a; q1_b = q1_a;
            u_a = u_new;
        }
        if (lane == 0) {
            if (ok) {
                SrMeta m = {8, 0, {0.f, 0.f}, 0, 0, 0, 0};
                next_stage(m, nullptr, nullptr, 0);
            }
            if (!ok) {
                atomicOr(p.ctrl + 1, 1u);
                // before the CTA can leave: copies that may still be landing in its shared memory (bounded)
                for (int s = 0; s < p.nst; ++s) {
                    mbar_wait_bounded(full0 + 8 * s, 0);
                    mbar_wait_bounded(full0 + 8 * s, 1);
                }
            }
        }
        return;
    }
    // ------------------------------------------------------------ consumer warps
    int stage = 0;
    uint32_t phase = 0;
    int buf = 0;                              // buffer of column sums the present unit is scattered to
    uint32_t aph = 0;                         // bit b: number of units handed over in buffer b, mod 2
    bool unit_open = false;                   // the present unit has its buffer
    float4 acc[kSrQ];
    uint4 cp[kSrQ];
    for (;;) {
        if (!mbar_wait_warp(full0 + 8 * stage, phase)) { if (tid == 0) atomicOr(p.ctrl + 1, 1u); break; }
        const SrMeta m = meta[stage];
        if (m.flags & 8) {
            if (!FW) break;
            // no more units: tell the folders through the next buffer
            if (!mbar_wait_warp(tsfree0 + 8 * buf, ((aph >> buf) & 1u) ^ 1u)) { if (tid == 0) atomicOr(p.ctrl + 1, 1u); break; }
            if (tid == 0) umeta[buf] = SrUnit{0, 0, 2, 0};
            mbar_arrive(tsfull0 + 8 * buf);
            break;
        }
        if (m.flags & 1) {
#pragma unroll
            for (int q = 0; q < kSrQ; ++q) {
                acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int j = q * (kSrConsumers * 4) + tid * 4;
                cp[q] = j < m.cw ? __ldg(reinterpret_cast<const uint4 *>(p.colpos + m.c0 + j)) : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int r = 0; r < kSrRows; ++r) {
            if (!((m.valid >> r) & 1)) continue;
            const float *row = reinterpret_cast<const float *>(ring + (size_t)stage * kSrStageBytes + (size_t)r * kSrRowBytes);
            const float sg = m.sign[r];
#pragma unroll
            for (int q = 0; q < kSrQ; ++q) {
                const int j = q * (kSrConsumers * 4) + tid * 4;
                if (j < m.cw) {
                    const float4 x = *reinterpret_cast<const float4 *>(row + j);
                    acc[q].x = fmaf(sg, x.x, acc[q].x); acc[q].y = fmaf(sg, x.y, acc[q].y);
                    acc[q].z = fmaf(sg, x.z, acc[q].z); acc[q].w = fmaf(sg, x.w, acc[q].w);
                }
            }
        }
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(empty0 + 8 * stage);
        if (++stage == p.nst) { stage = 0; phase ^= 1u; }
        if (m.flags & 2) {
            // the chunk's column sums, signed, to the positions their columns have in the bucket-sorted order; the
            // buffer must have been folded (two units ago) before the first of them is written
            if (FW && !unit_open) {
                if (!mbar_wait_warp(tsfree0 + 8 * buf, ((aph >> buf) & 1u) ^ 1u)) { if (tid == 0) atomicOr(p.ctrl + 1, 1u); break; }
                unit_open = true;
            }
            float *ts = ts0 + (size_t)buf * n3p;
#pragma unroll
            for (int q = 0; q < kSrQ; ++q) {
                const int j = q * (kSrConsumers * 4) + tid * 4;
                const uint32_t cpe[4] = {cp[q].x, cp[q].y, cp[q].z, cp[q].w};
                const float rse[4] = {acc[q].x, acc[q].y, acc[q].z, acc[q].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (j + e >= m.cw) continue;
                    const uint32_t pos = cpe[e] & 0x7FFFFFFFu;
                    if (!FPSK_IN_BOUNDS(pos, p.n3)) continue;
                    ts[pos] = ((cpe[e] >> 31) ? -1.f : 1.f) * rse[e];
                }
            }
        }
        if (m.flags & 4) {
            if (FW) {
                // hand the unit to the folders: every consumer thread arrives after its own writes
                if (tid == 0) umeta[buf] = SrUnit{m.a, m.sp, m.cw == 0 ? 1 : 0, 0};
                mbar_arrive(tsfull0 + 8 * buf);
                aph ^= 1u << buf;
                buf ^= 1;
                unit_open = false;
            } else {
                float *dst = p.part + (long long)m.sp * 3 * mm + (long long)m.a * p.m_b;
                SrSync::sync();
                sr_fold(ts0, cs, dst, p.m_b, tid, kSrConsumers, m.cw == 0);
                SrSync::sync();       // the buffer is rewritten by the next unit
            }
        }
    }
}

static size_t scatter_ring_fixed(int n3, int m_b, bool fw)
{
    return (size_t)(fw ? 2 : 1) * ((n3 + 3) & ~3) * 4 + (size_t)((m_b + 1 + 3) & ~3) * 4 + kSrStages * sizeof(SrMeta) + 2 * sizeof(SrUnit) +
           (2 * kSrStages + 4) * 8 + 128;
}
// Ring stages that fit beside the buffers of column sums (0: this form does not fit).
static int scatter_ring_stages(int n3, int m_b, bool fw)
{
    const size_t fixed = scatter_ring_fixed(n3, m_b, fw), budget = 224 * 1024;
    if (fixed + 2 * (size_t)kSrStageBytes > budget) return 0;
    const size_t nst = (budget - fixed) / kSrStageBytes;
    return (int)(nst > (size_t)kSrStages ? kSrStages : nst);
}

// ---------------------------------------------------------------- FP32 SIMT contraction
// C[M x N] = A[M x K] * B[K x N], all row-major, K a multiple of BK, FP32 FMA only (the
// sketch noise is the measured quantity, so no reduced-precision tensor-core path here).
// blockIdx.z = problem * ksplit + split; each split writes its own partial output.
struct GemmBatch {
    const float *P, *Pw;      // problems: 0 = P Q, 1 = Pw Q, 2 = P Qw
    const float *Q, *Qw;
    float *Cpart;     // [ksplit][nprob][M*N]
    int M, N, K, lda, ldb, ksplit, kchunk;
    int nprob;        // problems per split in Cpart
};

template <int BM, int BN, int T>   // T = 4 or 8 outputs per thread per dimension; 256 threads
__global__ void __launch_bounds__(256, 2) sgemm_kernel(const GemmBatch g)
{
    constexpr int BK = 16;
    constexpr int PADM = BM + 4, PADN = BN + 4;
    __shared__ __align__(16) float As[2][BK][PADM];
    __shared__ __align__(16) float Bs[2][BK][PADN];
    const int prob = blockIdx.z / g.ksplit, ks = blockIdx.z % g.ksplit;
    const float *__restrict__ A = prob == 1 ? g.Pw : g.P;
    const float *__restrict__ B = prob == 2 ? g.Qw : g.Q;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int k_begin = ks * g.kchunk, k_end = min(g.K, k_begin + g.kchunk);
    const int tid = threadIdx.x;
    constexpr int TX = BN / T;               // threads along N
    const int tx = tid % TX, ty = tid / TX;
    constexpr int HALF = T / 4;              // 1 or 2 groups of 4
    // global -> smem assignment
    constexpr int A_F4 = BM * BK / 4 / 256;  // float4 per thread for the A tile
    constexpr int B_F4 = BK * BN / 4 / 256;
    float4 ra[A_F4], rb[B_F4];
    float acc[T][T];
#pragma unroll
    for (int i = 0; i < T; ++i)
#pragma unroll
        for (int j = 0; j < T; ++j) acc[i][j] = 0.f;

    auto gload = [&](int k0) {
#pragma unroll
        for (int q = 0; q < A_F4; ++q) {
            int f = tid + q * 256;           // float4 index in tile: row = f / 4, kq = f % 4
            int row = f >> 2, kq = f & 3;
            int gr = m0 + row;
            ra[q] = (gr < g.M) ? *reinterpret_cast<const float4 *>(A + (long long)gr * g.lda + k0 + kq * 4)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int q = 0; q < B_F4; ++q) {
            int f = tid + q * 256;           // row k = f / (BN/4), c4 = f % (BN/4)
            int kr = f / (BN / 4), c4 = f % (BN / 4);
            int gc = n0 + c4 * 4;
            rb[q] = (gc < g.ldb) ? *reinterpret_cast<const float4 *>(B + (long long)(k0 + kr) * g.ldb + gc)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto sstore = [&](int buf) {
#pragma unroll
        for (int q = 0; q < A_F4; ++q) {
            int f = tid + q * 256;
            int row = f >> 2, kq = f & 3;
            As[buf][kq * 4 + 0][row] = ra[q].x;
            As[buf][kq * 4 + 1][row] = ra[q].y;
            As[buf][kq * 4 + 2][row] = ra[q].z;
            As[buf][kq * 4 + 3][row] = ra[q].w;
        }
#pragma unroll
        for (int q = 0; q < B_F4; ++q) {
            int f = tid + q * 256;
            int kr = f / (BN / 4), c4 = f % (BN / 4);
            *reinterpret_cast<float4 *>(&Bs[buf][kr][c4 * 4]) = rb[q];
        }
    };

    if (k_begin < k_end) {
        gload(k_begin);
        sstore(0);
        __syncthreads();
        int buf = 0;
        for (int k0 = k_begin; k0 < k_end; k0 += BK) {
            const bool more = (k0 + BK) < k_end;
            if (more) gload(k0 + BK);
#pragma unroll
            for (int kk = 0; kk < BK; ++kk) {
                float a[T], b[T];
#pragma unroll
                for (int h = 0; h < HALF; ++h) {
                    float4 va = *reinterpret_cast<const float4 *>(&As[buf][kk][h * (BM / 2) + ty * 4]);
                    float4 vb = *reinterpret_cast<const float4 *>(&Bs[buf][kk][h * (BN / 2) + tx * 4]);
                    a[h * 4 + 0] = va.x; a[h * 4 + 1] = va.y; a[h * 4 + 2] = va.z; a[h * 4 + 3] = va.w;
                    b[h * 4 + 0] = vb.x; b[h * 4 + 1] = vb.y; b[h * 4 + 2] = vb.z; b[h * 4 + 3] = vb.w;
                }
#pragma unroll
                for (int i = 0; i < T; ++i)
#pragma unroll
                    for (int j = 0; j < T; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            if (more) {
                sstore(buf ^ 1);
                __syncthreads();
                buf ^= 1;
            }
        }
    }
    float *Cout = g.Cpart + ((long long)ks * g.nprob + prob) * (long long)g.M * g.N;
#pragma unroll
    for (int i = 0; i < T; ++i) {
        const int row = m0 + (i / 4) * (BM / 2) * (HALF - 1) + (HALF == 1 ? ty * 4 + i : ty * 4 + (i & 3));
        if (row >= g.M) continue;
#pragma unroll
        for (int j = 0; j < T; ++j) {
            const int col = n0 + (j / 4) * (BN / 2) * (HALF - 1) + (HALF == 1 ? tx * 4 + j : tx * 4 + (j & 3));
            if (col < g.N) Cout[(long long)row * g.N + col] = acc[i][j];
        }
    }
}

// ---------------------------------------------------------------- combine
// tc_scale (tensor-core contraction only): the partials carry the two sides' powers of two, undone here.
__global__ void combine_kernel(const float *partAB, int ksplit, const float *partC, int nsplit, long long mm,
                               int nsk, float *S, float *R, float *T, const float *tc_scale)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= mm) return;
    const float unscale = tc_scale ? 1.f / (tc_scale[0] * tc_scale[1]) : 1.f;        // a power of two: exact
    for (int q = 0; q < nsk; ++q) {
        float ab = partAB[(long long)q * mm + idx];
        for (int s = 1; s < ksplit; ++s) ab += partAB[((long long)s * 3 + q) * mm + idx];
        ab *= unscale;
        float c = partC[(long long)q * mm + idx];
        for (int s = 1; s < nsplit; ++s) c += partC[((long long)s * 3 + q) * mm + idx];
        float *dst = q == 0 ? S : (q == 1 ? R : T);
        dst[idx] = ab - c;
    }
}
// The same for four consecutive buckets per thread (m_b^2 a multiple of 4, 16-byte aligned arrays): 16-byte loads,
// up to eight partials in flight per sum, added in split order.
__global__ void __launch_bounds__(256) combine4_kernel(const float *partAB, int ksplit, const float *partC, int nsplit,
                                                       long long mm, int nsk, float *S, float *R, float *T,
                                                       const float *tc_scale)
{
    const long long idx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (idx >= mm) return;
    const float unscale = tc_scale ? 1.f / (tc_scale[0] * tc_scale[1]) : 1.f;        // a power of two: exact
    for (int q = 0; q < nsk; ++q) {
        float4 ab = make_float4(0.f, 0.f, 0.f, 0.f), c = ab;
        for (int s0 = 0; s0 < ksplit; s0 += 8) {
            float4 v[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)
                v[t] = s0 + t < ksplit ? __ldcs(reinterpret_cast<const float4 *>(partAB + ((long long)(s0 + t) * 3 + q) * mm + idx))
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (s0 + t == 0) ab = v[t];            // the first partial starts the sum (no 0 + x: keeps -0 as it is)
                else if (s0 + t < ksplit) { ab.x += v[t].x; ab.y += v[t].y; ab.z += v[t].z; ab.w += v[t].w; }
            }
        }
        ab.x *= unscale; ab.y *= unscale; ab.z *= unscale; ab.w *= unscale;
        for (int s0 = 0; s0 < nsplit; s0 += 8) {
            float4 v[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)
                v[t] = s0 + t < nsplit ? __ldcs(reinterpret_cast<const float4 *>(partC + ((long long)(s0 + t) * 3 + q) * mm + idx))
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (s0 + t == 0) c = v[t];
                else if (s0 + t < nsplit) { c.x += v[t].x; c.y += v[t].y; c.z += v[t].z; c.w += v[t].w; }
            }
        }
        float *dst = q == 0 ? S : (q == 1 ? R : T);
        *reinterpret_cast<float4 *>(dst + idx) = make_float4(ab.x - c.x, ab.y - c.y, ab.z - c.z, ab.w - c.w);
    }
}

// Subtract every confirmed fault from its bucket (Algorithm 1, peeling loop).  One thread:
// the list is short and the order of subtractions is then fixed.
__global__ void peel_kernel(const PeelEntry *F, int nF_host, const int *d_nF, uint32_t key1, uint32_t key2, int m_b, float inv_p1,
                            float inv_p3, float *S, float *R, float *T)
{
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    const int nF = d_nF ? *d_nF : nF_host;
    for (int f = 0; f < nF; ++f) {
        int a, b, s1, s2;
        hash_index(key1, (uint32_t)F[f].i, (uint32_t)m_b, a, s1);
        hash_index(key2, (uint32_t)F[f].j, (uint32_t)m_b, b, s2);
        const double g = (double)(s1 * s2) * F[f].delta;
        const long long o = (long long)a * m_b + b;
        if (!FPSK_IN_BOUNDS(a, m_b) || !FPSK_IN_BOUNDS(b, m_b)) continue;
        S[o] = (float)((double)S[o] - g);
        if (R) R[o] = (float)((double)R[o] - g * ((double)(F[f].i + 1) * (double)inv_p1));
        if (T) T[o] = (float)((double)T[o] - g * ((double)(F[f].j + 1) * (double)inv_p3));
    }
}

// ---------------------------------------------------------------- hash tables of several rounds at once
static void sketch_use_set(SketchWs &w, int q)
{
    const HashSet &hs = w.sets[q];
    w.h1 = hs.h1; w.v1 = hs.v1; w.h2 = hs.h2; w.v2 = hs.v2;
    w.rowperm = hs.rowperm; w.colperm = hs.colperm; w.colpos = hs.colpos;
    w.rowcount = hs.rowcount; w.rowstart = hs.rowstart; w.colcount = hs.colcount; w.colstart = hs.colstart;
}

struct HashJob {                 // one side of one round
    uint32_t key;
    int n;
    int *bucket, *sign, *count, *start;
    uint32_t *perm, *pos;
};
struct HashBatch {
    HashJob job[2 * kHashSets];
};
// blockIdx.y = job: the three kernels of build_hash_side for all jobs of the batch in one launch each
__global__ void hash_batch_kernel(HashBatch hb, int m_b)
{
    const HashJob &j = hb.job[blockIdx.y];
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= j.n) return;
    int b, s;
    hash_index(j.key, (uint32_t)idx, (uint32_t)m_b, b, s);
    j.bucket[idx] = b;
    j.sign[idx] = s;
    atomicAdd(j.count + b, 1);
}
__global__ void scan_batch_kernel(HashBatch hb, int m_b)
{
    const HashJob &j = hb.job[blockIdx.x];
    __shared__ int carry;
    __shared__ int buf[1024];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < m_b; base += 1024) {
        const int i = base + threadIdx.x;
        const int v = i < m_b ? j.count[i] : 0;
        buf[threadIdx.x] = v;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const int t = threadIdx.x >= o ? buf[threadIdx.x - o] : 0;
            __syncthreads();
            buf[threadIdx.x] += t;
            __syncthreads();
        }
        if (i < m_b) j.start[i] = carry + buf[threadIdx.x] - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry += buf[1023];
        __syncthreads();
    }
    if (threadIdx.x == 0) j.start[m_b] = carry;
}
__global__ void __launch_bounds__(256) place_batch_kernel(HashBatch hb)
{
    const HashJob &jb = hb.job[blockIdx.y];
    const int idx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (idx >= jb.n) return;
    const int b = __ldg(jb.bucket + idx);
    int cnt = 0;
    int j = lane;
    for (; j + 96 < idx; j += 128) {
        const int b0 = __ldg(jb.bucket + j), b1 = __ldg(jb.bucket + j + 32), b2 = __ldg(jb.bucket + j + 64), b3 = __ldg(jb.bucket + j + 96);
        cnt += (b0 == b) + (b1 == b) + (b2 == b) + (b3 == b);
    }
    for (; j < idx; j += 32) cnt += (__ldg(jb.bucket + j) == b);
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if (lane == 0) {
        const uint32_t sbit = __ldg(jb.sign + idx) < 0 ? 0x80000000u : 0u;
        const uint32_t where = (uint32_t)(__ldg(jb.start + b) + cnt);
        if (FPSK_IN_BOUNDS(where, jb.n)) jb.perm[where] = (uint32_t)idx | sbit;
        if (jb.pos) jb.pos[idx] = where | sbit;
    }
}

fpsk_status prepare_hash_rounds(uint64_t seed, int first, int count, long long n1, long long n3, int m_b, SketchWs &w,
                                cudaStream_t st)
{
    if (count > kHashSets) count = kHashSets;
    w.prepared_count = 0;
    if (count < 1) return FPSK_OK;
    HashBatch hb;
    int nmax = 0;
    // the counts of sets 0 .. count - 1 are one contiguous block (see sketch_carve)
    FPSK_CUDA_OK(cudaMemsetAsync(w.sets[0].rowcount, 0, (size_t)count * 2 * align_up((size_t)(m_b + 1) * 4, 256), st));
    for (int q = 0; q < count; ++q) {
        const HashSet &hs = w.sets[q];
        hb.job[2 * q] = HashJob{round_key(seed, first + q, 0), (int)n1, hs.h1, hs.v1, hs.rowcount, hs.rowstart, hs.rowperm, nullptr};
        hb.job[2 * q + 1] = HashJob{round_key(seed, first + q, 1), (int)n3, hs.h2, hs.v2, hs.colcount, hs.colstart, hs.colperm, hs.colpos};
    }
    nmax = (int)(n1 > n3 ? n1 : n3);
    hash_batch_kernel<<<dim3((nmax + 255) / 256, 2 * count), 256, 0, st>>>(hb, m_b);
    FPSK_LAUNCH_CHECK();
    scan_batch_kernel<<<2 * count, 1024, 0, st>>>(hb, m_b);
    FPSK_LAUNCH_CHECK();
    place_batch_kernel<<<dim3((nmax + 7) / 8, 2 * count), 256, 0, st>>>(hb);
    FPSK_LAUNCH_CHECK();
    w.prepared_first = first;
    w.prepared_count = count;
    w.prepared_seed = seed;
    return FPSK_OK;
}

// ---------------------------------------------------------------- host orchestration
static int pow2_exp(long long n)
{
    int p = 0;
    while ((1LL << p) < n) ++p;
    return p;
}

void sketch_plan(long long n1, long long n2, long long n3, int m_b, SketchPlan &pl)
{
    pl.kpad = (int)((n2 + 15) / 16 * 16);
    pl.npad = (m_b + 3) / 4 * 4;
    int ns = (512 + m_b - 1) / m_b;
    if (ns > 16) ns = 16;
    long long avg_rows = n1 / m_b;
    if (ns > avg_rows) ns = (int)(avg_rows > 1 ? avg_rows : 1);
    pl.nsplit = ns < 1 ? 1 : ns;
    pl.tile = m_b <= 192 ? 64 : 128;
    const int tiles = ((m_b + pl.tile - 1) / pl.tile) * ((m_b + pl.tile - 1) / pl.tile) * 3;
    int ks = (600 + tiles - 1) / tiles;
    const int maxks = pl.kpad / 256 > 1 ? pl.kpad / 256 : 1;   // at least 256 of K per split
    if (ks > maxks) ks = maxks;
    if (ks > 32) ks = 32;
    if (ks < 1) ks = 1;
    int kchunk = ((pl.kpad + ks - 1) / ks + 15) / 16 * 16;
    ks = (pl.kpad + kchunk - 1) / kchunk;
    pl.ksplit = ks;
    pl.kchunk = kchunk;
}

static int sketch_sms()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return 148;
    return sms;
}

size_t sketch_ws_bytes(long long n1, long long n2, long long n3, int m_b, bool tc)
{
    SketchPlan pl;
    sketch_plan(n1, n2, n3, m_b, pl);
    const size_t mm = (size_t)m_b * m_b;
    tc = tc && m_b >= kTcMinBuckets;
    const int tcks = tc ? tc_plan_ksplit(m_b, m_b, pl.kpad, 3, sketch_sms()) : 0;
    size_t b = 0;
    b += kHashSets * align_up((size_t)n1 * 4, 256) * 3;          // h1, v1, rowperm           (per prepared hash round)
    b += kHashSets * align_up((size_t)n3 * 4, 256) * 4;          // h2, v2, colperm, colpos
    b += kHashSets * align_up((size_t)(m_b + 1) * 4, 256) * 4;   // rowcount, rowstart, colcount, colstart
    b += align_up((size_t)m_b * pl.kpad * 4, 256) * 2;       // P, Pw
    b += align_up((size_t)pl.kpad * pl.npad * 4, 256) * 2;   // Q, Qw
    b += align_up((size_t)(pl.ksplit > tcks ? pl.ksplit : tcks) * 3 * mm * 4, 256);      // AB partials
    if (tc) b += align_up(tc_planes_bytes(m_b, pl.kpad), 256) * 4 + 512;          // FP16 planes of P, Pw, Q^T, Qw^T; error word; scales
    b += align_up((size_t)pl.nsplit * 3 * mm * 4, 256);      // C partials
    b += 256;                                                // control words of the ring scatter
    return b;
}

bool sketch_carve(void *ws, size_t ws_bytes, long long n1, long long n2, long long n3, int m_b, SketchWs &w, bool tc)
{
    if (ws_bytes < sketch_ws_bytes(n1, n2, n3, m_b, tc)) return false;
    tc = tc && m_b >= kTcMinBuckets;
    sketch_plan(n1, n2, n3, m_b, w.pl);
    w.aux = nullptr;
    const size_t mm = (size_t)m_b * m_b;
    char *p = static_cast<char *>(ws);
    auto take = [&](size_t bytes) { void *r = p; p += align_up(bytes, 256); return r; };
    // the bucket counts of all sets side by side: one memset clears them when several rounds are prepared at once
    for (int q = 0; q < kHashSets; ++q) {
        w.sets[q].rowcount = (int *)take((size_t)(m_b + 1) * 4);
        w.sets[q].colcount = (int *)take((size_t)(m_b + 1) * 4);
    }
    for (int q = 0; q < kHashSets; ++q) {
        HashSet &hs = w.sets[q];
        hs.h1 = (int *)take((size_t)n1 * 4); hs.v1 = (int *)take((size_t)n1 * 4); hs.rowperm = (uint32_t *)take((size_t)n1 * 4);
        hs.h2 = (int *)take((size_t)n3 * 4); hs.v2 = (int *)take((size_t)n3 * 4); hs.colperm = (uint32_t *)take((size_t)n3 * 4);
        hs.colpos = (uint32_t *)take((size_t)n3 * 4);
        hs.rowstart = (int *)take((size_t)(m_b + 1) * 4);
        hs.colstart = (int *)take((size_t)(m_b + 1) * 4);
    }
    w.prepared_first = 0; w.prepared_count = 0; w.prepared_seed = 0;
    sketch_use_set(w, 0);
    w.P = (float *)take((size_t)m_b * w.pl.kpad * 4); w.Pw = (float *)take((size_t)m_b * w.pl.kpad * 4);
    w.Q = (float *)take((size_t)w.pl.kpad * w.pl.npad * 4); w.Qw = (float *)take((size_t)w.pl.kpad * w.pl.npad * 4);
    w.tc = tc;
    w.tc_ksplit = tc ? tc_plan_ksplit(m_b, m_b, w.pl.kpad, 3, sketch_sms()) : 0;
    w.partAB = (float *)take((size_t)(w.pl.ksplit > w.tc_ksplit ? w.pl.ksplit : w.tc_ksplit) * 3 * mm * 4);
    for (int i = 0; i < 4; ++i) w.planes[i] = tc ? (unsigned char *)take(tc_planes_bytes(m_b, w.pl.kpad)) : nullptr;
    w.tc_err = tc ? (unsigned int *)take(256) : nullptr;
    w.tc_scale = tc ? (float *)take(256) : nullptr;
    w.d_maxab = nullptr;
    w.partC = (float *)take((size_t)w.pl.nsplit * 3 * mm * 4);
    w.sc_ctrl = (unsigned int *)take(256);
    return true;
}

int sketch_max_buckets(long long n1, long long n2, long long n3)
{
    // scatter_c_kernel keeps two column-sum chunks and three m_b-vectors in shared memory
    (void)n3;
    const long long budget = 200 * 1024 - 2LL * kScChunk * 4;
    if (budget < 3 * 4) return 0;
    long long m = budget / 12;
    if (m > 16384) m = 16384;
    return (int)m;
}

// ---------------------------------------------------------------- B -> W = B^T (16-bit elements)
// 64 x 64 tiles through shared memory.  VEC (16-byte aligned rows on both sides, n2 and n3 multiples of 8): a thread
// reads 8 consecutive columns of a row of B with one load and writes 8 consecutive k of a row of W with one store.
template <bool VEC>
__global__ void __launch_bounds__(256) transpose16_kernel(const unsigned short *B, long long ldb, int n2, int n3,
                                                          unsigned short *W, long long ldw)
{
    __shared__ __align__(16) unsigned short tile[64][66];      // row pitch 33 words: rows 8 apart fall into different banks
    const int k0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    if (VEC) {
        for (int e = threadIdx.x; e < 64 * 8; e += 256) {
            const int r = e >> 3, c8 = (e & 7) * 8;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (k0 + r < n2 && j0 + c8 < n3) v = ldg_nc_v4(B + (long long)(k0 + r) * ldb + j0 + c8);
            uint32_t *dst = reinterpret_cast<uint32_t *>(&tile[r][c8]);
            dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
        }
        __syncthreads();
        for (int e = threadIdx.x; e < 64 * 8; e += 256) {
            const int r8 = (e & 7) * 8, c = e >> 3;            // eight consecutive lanes write 128 contiguous bytes of a row of W
            if (j0 + c >= n3 || k0 + r8 >= n2) continue;
            unsigned short x[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) x[t] = tile[r8 + t][c];
            *reinterpret_cast<uint4 *>(W + (long long)(j0 + c) * ldw + k0 + r8) =
                make_uint4(x[0] | ((unsigned)x[1] << 16), x[2] | ((unsigned)x[3] << 16), x[4] | ((unsigned)x[5] << 16),
                           x[6] | ((unsigned)x[7] << 16));
        }
    } else {
        for (int e = threadIdx.x; e < 64 * 64; e += 256) {
            const int r = e >> 6, c = e & 63;                  // a warp reads 32 consecutive columns of one row of B
            tile[r][c] = (k0 + r < n2 && j0 + c < n3) ? B[(long long)(k0 + r) * ldb + j0 + c] : (unsigned short)0;
        }
        __syncthreads();
        for (int e = threadIdx.x; e < 64 * 64; e += 256) {
            const int c = e >> 6, r = e & 63;                  // ... and writes 32 consecutive k of one row of W
            if (j0 + c < n3 && k0 + r < n2) W[(long long)(j0 + c) * ldw + k0 + r] = tile[r][c];
        }
    }
}

fpsk_status transpose_b_launch(const void *B, long long ldb, long long n2, long long n3, void *W, long long ldw,
                               cudaStream_t st)
{
    dim3 grid((unsigned)((n3 + 63) / 64), (unsigned)((n2 + 63) / 64));
    const bool vec = ((reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(W)) & 15) == 0 && ldb % 8 == 0 &&
                     ldw % 8 == 0 && n2 % 8 == 0 && n3 % 8 == 0;
    if (vec)
        transpose16_kernel<true><<<grid, 256, 0, st>>>(static_cast<const unsigned short *>(B), ldb, (int)n2, (int)n3,
                                                       static_cast<unsigned short *>(W), ldw);
    else
        transpose16_kernel<false><<<grid, 256, 0, st>>>(static_cast<const unsigned short *>(B), ldb, (int)n2, (int)n3,
                                                        static_cast<unsigned short *>(W), ldw);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- auxiliary streams
struct SketchAuxPool {
    std::mutex mu;
    std::vector<SketchAux *> free_list;
};
static SketchAuxPool &sketch_aux_pool()
{
    static SketchAuxPool *p = new SketchAuxPool;       // never destroyed: no CUDA calls at process exit
    return *p;
}
SketchAuxLease::~SketchAuxLease()
{
    if (!aux || borrowed) return;
    SketchAuxPool &pool = sketch_aux_pool();
    std::lock_guard<std::mutex> g(pool.mu);
    pool.free_list.push_back(aux);
}
fpsk_status sketch_aux_acquire(SketchAuxLease &lease)
{
    int dev = 0;
    FPSK_CUDA_OK(cudaGetDevice(&dev));
    SketchAuxPool &pool = sketch_aux_pool();
    {
        std::lock_guard<std::mutex> g(pool.mu);
        for (size_t i = 0; i < pool.free_list.size(); ++i) {
            if (pool.free_list[i]->device != dev) continue;
            lease.aux = pool.free_list[i];
            pool.free_list.erase(pool.free_list.begin() + (long)i);
            return FPSK_OK;
        }
    }
    SketchAux *a = new SketchAux;
    g_lazy_resources.fetch_add(1, std::memory_order_relaxed);
    lease.aux = a;                  // returned to the pool even when a creation below fails (unused handles stay null)
    return sketch_aux_create(*a);
}

fpsk_status sketch_aux_create(SketchAux &a)
{
    FPSK_CUDA_OK(cudaGetDevice(&a.device));
    FPSK_CUDA_OK(cudaStreamCreateWithFlags(&a.s1, cudaStreamNonBlocking));
    FPSK_CUDA_OK(cudaStreamCreateWithFlags(&a.s2, cudaStreamNonBlocking));
    {
        // the tails are short and latency-bound: their CTAs go ahead of the builds' in the queue for free SMs
        int lo = 0, hi = 0;
        FPSK_CUDA_OK(cudaDeviceGetStreamPriorityRange(&lo, &hi));
        FPSK_CUDA_OK(cudaStreamCreateWithPriority(&a.s3, cudaStreamNonBlocking, hi));
    }
    for (int e = 0; e < 5; ++e) FPSK_CUDA_OK(cudaEventCreateWithFlags(&a.ev[e], cudaEventDisableTiming));
    for (int e = 0; e < 3; ++e) FPSK_CUDA_OK(cudaEventCreateWithFlags(&a.evb[e], cudaEventDisableTiming));
    FPSK_CUDA_OK(cudaEventCreateWithFlags(&a.evt, cudaEventDisableTiming));
    return FPSK_OK;
}

bool sketch_aux_destroy(SketchAux &a)
{
    bool ok = true;
    if (a.s1) ok = (cudaStreamDestroy(a.s1) == cudaSuccess) && ok;
    if (a.s2) ok = (cudaStreamDestroy(a.s2) == cudaSuccess) && ok;
    if (a.s3) ok = (cudaStreamDestroy(a.s3) == cudaSuccess) && ok;
    for (int e = 0; e < 5; ++e)
        if (a.ev[e]) ok = (cudaEventDestroy(a.ev[e]) == cudaSuccess) && ok;
    for (int e = 0; e < 3; ++e)
        if (a.evb[e]) ok = (cudaEventDestroy(a.evb[e]) == cudaSuccess) && ok;
    if (a.evt) ok = (cudaEventDestroy(a.evt) == cudaSuccess) && ok;
    a = SketchAux();
    return ok;
}

bool sketch_select_round(SketchWs &w, uint64_t seed, int rnd)
{
    if (w.prepared_count > 0 && seed == w.prepared_seed && rnd >= w.prepared_first && rnd < w.prepared_first + w.prepared_count) {
        sketch_use_set(w, rnd - w.prepared_first);
        return true;
    }
    return false;
}

template <typename T>
static fpsk_status build_sketches_t(const SketchIn &in, uint64_t seed, int rnd, int m_b, bool mom, SketchWs &w,
                                    cudaStream_t st, float *S, float *R, float *Tt)
{
    const int n1 = (int)in.n1, n2 = (int)in.n2, n3 = (int)in.n3;
    const float inv_p1 = 1.0f / (float)(1LL << pow2_exp(n1));
    const float inv_p3 = 1.0f / (float)(1LL << pow2_exp(n3));
    fpsk_status rc;
    // st: row side, A compression, contraction, combine; sB: column side, B compression; sC: C scatter
    // (needs both sides).  Without auxiliary streams all three are st.
    SketchAux *ax = (w.aux && w.aux->s1 && w.aux->s2 && w.aux->ev[4]) ? w.aux : nullptr;
    cudaStream_t sB = ax ? ax->s1 : st, sC = ax ? ax->s2 : st;
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[0], st));             // everything queued before this build
        FPSK_CUDA_OK(cudaStreamWaitEvent(sB, ax->ev[0], 0));
        FPSK_CUDA_OK(cudaStreamWaitEvent(sC, ax->ev[0], 0));
    }
    if (w.prepared_count > 0 && seed == w.prepared_seed && rnd >= w.prepared_first && rnd < w.prepared_first + w.prepared_count) {
        sketch_use_set(w, rnd - w.prepared_first);         // tables prepared ahead (on st, before this point)
    } else {
        // built here, into the first set (whatever was prepared is overwritten: forget it)
        w.prepared_count = 0;
        sketch_use_set(w, 0);
        rc = build_hash_side(seed, rnd, 0, n1, m_b, w.h1, w.v1, w.rowcount, w.rowstart, w.rowperm, st);
        if (rc != FPSK_OK) return rc;
        rc = build_hash_side(seed, rnd, 1, n3, m_b, w.h2, w.v2, w.colcount, w.colstart, w.colperm, sB, w.colpos);
        if (rc != FPSK_OK) return rc;
    }
    const float *scA = w.tc ? w.tc_scale : nullptr, *scB = w.tc ? w.tc_scale + 1 : nullptr;
    if (w.tc) {
        if (!w.d_maxab) return FPSK_ERR_PARAM;
        rc = tc_scale_launch(w.rowcount, m_b, w.d_maxab, w.tc_scale, st);
        if (rc != FPSK_OK) return rc;
        rc = tc_scale_launch(w.colcount, m_b, w.d_maxab + 1, w.tc_scale + 1, sB);
        if (rc != FPSK_OK) return rc;
    }
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[1], st));             // row side ready
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[2], sB));             // column side ready
        FPSK_CUDA_OK(cudaStreamWaitEvent(sC, ax->ev[1], 0));
        FPSK_CUDA_OK(cudaStreamWaitEvent(sC, ax->ev[2], 0));
    }

    const unsigned short *A = static_cast<const unsigned short *>(in.A);
    const unsigned short *B = static_cast<const unsigned short *>(in.B);
    const SketchPlan &pl = w.pl;
    // With the tensor-core contraction the compressions emit the tiled BF16 planes themselves (no FP32 P, Q).
    const int kblocks = (pl.kpad + 31) / 32;
    const int btiles = (m_b + 255) / 256;
    const bool b8 = (size_t)16 * (((n3 + 7) & ~7) + 2) <= 160 * 1024;      // eight rows of B fit in shared memory
    {
        const bool vec = (reinterpret_cast<uintptr_t>(in.A) & 15) == 0 && in.lda % 8 == 0 && n2 % 8 == 0;
        const int kcols = w.tc ? kblocks * 32 : pl.kpad;
        dim3 grid = w.tc ? dim3((kcols / 8 + 15) / 16, (m_b + 7) / 8) : dim3((kcols / 8 + 127) / 128, m_b);
#define FPSK_CA(V, M, PL) compress_a_kernel<T, V, M, PL><<<grid, 128, 0, st>>>(A, in.lda, n1, n2, pl.kpad, inv_p1, w.rowperm, w.rowstart, w.P, w.Pw, kblocks, w.planes[0], w.planes[1], m_b, scA)
        if (w.tc) {
            dim3 gp((kblocks * 32 / 8 + 31) / 32, (m_b + 7) / 8);
#define FPSK_CP(V, M) compress_planes_kernel<T, 128, V, M><<<gp, 256, 0, st>>>(A, in.lda, n1, n2, inv_p1, w.rowperm, w.rowstart, m_b, kblocks, w.planes[0], w.planes[1], scA)
            if (vec) { if (mom) FPSK_CP(true, true); else FPSK_CP(true, false); }
            else     { if (mom) FPSK_CP(false, true); else FPSK_CP(false, false); }
#undef FPSK_CP
        } else {
            if (vec) { if (mom) FPSK_CA(true, true, false); else FPSK_CA(true, false, false); }
            else     { if (mom) FPSK_CA(false, true, false); else FPSK_CA(false, false, false); }
        }
#undef FPSK_CA
        FPSK_LAUNCH_CHECK();
    }
    if (in.bt) {
        const bool vec = (reinterpret_cast<uintptr_t>(in.B) & 15) == 0 && in.ldb % 8 == 0 && n2 % 8 == 0;
        const int kcols = w.tc ? kblocks * 32 : pl.kpad;
        const int bmax = w.tc ? btiles * 256 : pl.npad;
        dim3 grid((kcols / 8 + 15) / 16, (bmax + 7) / 8);
#define FPSK_CW(V, M, PL) compress_wt_kernel<T, V, M, PL><<<grid, 128, 0, sB>>>(B, in.ldb, n2, n3, pl.kpad, m_b, pl.npad, inv_p3, w.colperm, w.colstart, w.Q, w.Qw, kblocks, btiles, w.planes[2], w.planes[3], scB)
        if (w.tc) {
            // buckets up to the padded extent of the plane (btiles * 256): the ones beyond m_b are written as zeros
            dim3 gp((kblocks * 32 / 8 + 31) / 32, btiles * 256 / 8);
#define FPSK_CP(V, M) compress_planes_kernel<T, 256, V, M><<<gp, 256, 0, sB>>>(B, in.ldb, n3, n2, inv_p3, w.colperm, w.colstart, m_b, kblocks, w.planes[2], w.planes[3], scB)
            if (vec) { if (mom) FPSK_CP(true, true); else FPSK_CP(true, false); }
            else     { if (mom) FPSK_CP(false, true); else FPSK_CP(false, false); }
#undef FPSK_CP
        } else {
            if (vec) { if (mom) FPSK_CW(true, true, false); else FPSK_CW(true, false, false); }
            else     { if (mom) FPSK_CW(false, true, false); else FPSK_CW(false, false, false); }
        }
#undef FPSK_CW
        FPSK_LAUNCH_CHECK();
    } else if (b8) {
        const size_t smem = (size_t)16 * (((n3 + 7) & ~7) + 2);      // eight rows of 16-bit values (+ the padding of the sorted form)
        const int groups = (w.tc ? kblocks * 32 : pl.kpad) / 8;
        const int grid = groups < 888 ? groups : 888;
        // the sorted-row form (S only, FP32 Q, aligned B) is instruction-bound on its scattered 16-bit stores and holds one
        // CTA per SM at 8192 columns: 32 warps instead of 8
        const bool sorted8 = n3 % 8 == 0 && in.ldb % 8 == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0;
#define FPSK_CB8(M, PL)                                                                                                          \
    do {                                                                                                                         \
        FPSK_CUDA_OK(cudaFuncSetAttribute(compress_b8_kernel<T, M, PL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        compress_b8_kernel<T, M, PL><<<grid, (!PL && !M && sorted8) ? 1024 : 256, smem, sB>>>(B, in.ldb, n2, n3, pl.kpad, m_b, pl.npad, inv_p3, w.colperm,      \
                                                              w.colstart, w.Q, w.Qw, kblocks, btiles, w.planes[2], w.planes[3], scB, w.colpos); \
    } while (0)
        if (w.tc) { if (mom) FPSK_CB8(true, true); else FPSK_CB8(false, true); }
        else      { if (mom) FPSK_CB8(true, false); else FPSK_CB8(false, false); }
#undef FPSK_CB8
        FPSK_LAUNCH_CHECK();
    } else {
        const size_t smem = ((size_t)n3 * 2 + 15) / 16 * 16;
        int grid = pl.kpad < 1184 ? pl.kpad : 1184;
        if (mom) {
            FPSK_CUDA_OK(cudaFuncSetAttribute(compress_b_kernel<T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compress_b_kernel<T, true><<<grid, 256, smem, sB>>>(B, in.ldb, n2, n3, pl.kpad, m_b, pl.npad, inv_p3, w.colperm, w.colstart, w.Q, w.Qw);
        } else {
            FPSK_CUDA_OK(cudaFuncSetAttribute(compress_b_kernel<T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compress_b_kernel<T, false><<<grid, 256, smem, sB>>>(B, in.ldb, n2, n3, pl.kpad, m_b, pl.npad, inv_p3, w.colperm, w.colstart, w.Q, w.Qw);
        }
        FPSK_LAUNCH_CHECK();
    }
    if (w.tc && !b8 && !in.bt) {
        // wide B: Q, Qw came out as FP32 rows; split them here (row b of Q^T is column b of Q)
        rc = tc_split_launch(w.Q, scB, 1, pl.npad, m_b, pl.kpad, 1, w.planes[2], sB);
        if (rc != FPSK_OK) return rc;
        if (mom) {
            rc = tc_split_launch(w.Qw, scB, 1, pl.npad, m_b, pl.kpad, 1, w.planes[3], sB);
            if (rc != FPSK_OK) return rc;
        }
    }
    // ---- C scatter: independent of the compressions and of the contraction
    {
        const size_t smem = ((size_t)2 * kScChunk + 3 * (size_t)m_b) * 4;
        dim3 grid(m_b, pl.nsplit);
        const bool vec = (reinterpret_cast<uintptr_t>(in.C) & 15) == 0 && in.ldc % 4 == 0 && n3 % 4 == 0;
#define FPSK_SC(M, V)                                                                                                        \
    do {                                                                                                                     \
        FPSK_CUDA_OK(cudaFuncSetAttribute(scatter_c_kernel<M, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        scatter_c_kernel<M, V><<<grid, 256, smem, sC>>>(in.C, in.ldc, n1, n3, m_b, inv_p1, inv_p3, w.rowperm, w.rowstart,  \
                                                        w.colperm, w.colstart, pl.nsplit, w.partC);                          \
    } while (0)
        const size_t smem2 = (size_t)(mom ? 3 : 1) * ((n3 + 3) & ~3) * 4 + (size_t)(m_b + 1) * 4;
#define FPSK_SC2(M, V)                                                                                                        \
    do {                                                                                                                      \
        FPSK_CUDA_OK(cudaFuncSetAttribute(scatter_c2_kernel<M, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2)); \
        scatter_c2_kernel<M, V><<<grid, 256, smem2, sC>>>(in.C, in.ldc, n1, n3, m_b, inv_p1, inv_p3, w.rowperm, w.rowstart, \
                                                          w.colpos, w.colstart, pl.nsplit, w.partC);                          \
    } while (0)
        // the ring form with folder warps where both buffers leave room for the whole ring, with folding consumers where one does
        const bool ring_fw = scatter_ring_stages(n3, m_b, true) == kSrStages;
        const bool ring_fits = ring_fw || scatter_ring_stages(n3, m_b, false) == kSrStages;
        // measured: the ring form wins from about 150 MB of C (268 MB: 73 against 83 us, 1 GB: 233 against 302 us) and loses
        // below (67 MB: 30 against 27 us), where its longer start is not made up
        const bool ring_any = ring_fits && (long long)n1 * n3 >= (40LL << 20);
        FPSK_CUDA_OK(cudaMemsetAsync(w.sc_ctrl, 0, 8, sC));       // unit counter and give-up flag of the ring form (the flag is read whichever form runs)
        if (!mom && vec && n3 <= kSc2MaxCols && ring_any) {
            // S only, aligned C: the persistent producer/consumer form (same bits)
            static std::once_flag once;
            static cudaError_t attr_err = cudaSuccess;
            std::call_once(once, [] {
                attr_err = cudaFuncSetAttribute(scatter_ring_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
                if (attr_err == cudaSuccess)
                    attr_err = cudaFuncSetAttribute(scatter_ring_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
            });
            if (attr_err != cudaSuccess) return FPSK_ERR_CUDA;
            SrArgs sa;
            sa.C = in.C; sa.ldc = in.ldc; sa.n1 = n1; sa.n3 = n3; sa.m_b = m_b; sa.nsplit = pl.nsplit; sa.n_units = m_b * pl.nsplit; sa.nst = kSrStages;
            sa.rowperm = w.rowperm; sa.colpos = w.colpos; sa.rowstart = w.rowstart; sa.colstart = w.colstart;
            sa.part = w.partC; sa.ctrl = w.sc_ctrl;
            const int sms = sketch_sms();
            const size_t smem_ring = (size_t)kSrStages * kSrStageBytes + scatter_ring_fixed(n3, m_b, ring_fw);
            const int grid = sa.n_units < sms ? sa.n_units : sms;
            if (ring_fw) scatter_ring_kernel<true><<<grid, kSrThreads, smem_ring, sC>>>(sa);
            else scatter_ring_kernel<false><<<grid, kSrConsumers + 32, smem_ring, sC>>>(sa);
        } else if (n3 <= kSc2MaxCols) {
            if (mom) { if (vec) FPSK_SC2(true, true); else FPSK_SC2(true, false); }
            else     { if (vec) FPSK_SC2(false, true); else FPSK_SC2(false, false); }
        } else {
            if (mom) { if (vec) FPSK_SC(true, true); else FPSK_SC(true, false); }
            else     { if (vec) FPSK_SC(false, true); else FPSK_SC(false, false); }
        }
#undef FPSK_SC2
#undef FPSK_SC
        FPSK_LAUNCH_CHECK();
    }
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[3], sB));             // B side compressed
        FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->ev[3], 0));
    }
    int ab_splits = pl.ksplit;
    if (w.tc) {
        // split-BF16 contraction on the tensor cores, one launch for all problems
        FPSK_CUDA_OK(cudaMemsetAsync(w.tc_err, 0, 4, st));
        const unsigned char *pa[2] = {w.planes[0], w.planes[1]}, *pb[2] = {w.planes[2], w.planes[3]};
        const int selA[3] = {0, 1, 0}, selB[3] = {0, 0, 1};
        ab_splits = w.tc_ksplit;
        rc = tc_contract_launch(pa, pb, selA, selB, mom ? 3 : 1, 3, w.partAB, m_b, m_b, pl.kpad, ab_splits, w.tc_err, st);
        if (rc != FPSK_OK) return rc;
    } else
    {
        GemmBatch g;
        g.P = w.P; g.Pw = w.Pw; g.Q = w.Q; g.Qw = w.Qw;
        g.Cpart = w.partAB;
        g.M = m_b; g.N = m_b; g.K = pl.kpad; g.lda = pl.kpad; g.ldb = pl.npad;
        g.ksplit = pl.ksplit; g.kchunk = pl.kchunk;
        g.nprob = 3;          // combine_kernel reads a stride of three problems per split
        const int nprob = mom ? 3 : 1;
        if (pl.tile == 64) {
            dim3 grid((m_b + 63) / 64, (m_b + 63) / 64, nprob * pl.ksplit);
            sgemm_kernel<64, 64, 4><<<grid, 256, 0, st>>>(g);
        } else {
            dim3 grid((m_b + 127) / 128, (m_b + 127) / 128, nprob * pl.ksplit);
            sgemm_kernel<128, 128, 8><<<grid, 256, 0, st>>>(g);
        }
        FPSK_LAUNCH_CHECK();
    }
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[4], sC));             // C sketches ready
        FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->ev[4], 0));
    }
    {
        const long long mm = (long long)m_b * m_b;
        const bool al16 = ((reinterpret_cast<uintptr_t>(w.partAB) | reinterpret_cast<uintptr_t>(w.partC) | reinterpret_cast<uintptr_t>(S) |
                            reinterpret_cast<uintptr_t>(R) | reinterpret_cast<uintptr_t>(Tt)) & 15) == 0;
        if (mm % 4 == 0 && al16)
            combine4_kernel<<<(unsigned)((mm / 4 + 255) / 256), 256, 0, st>>>(w.partAB, ab_splits, w.partC, pl.nsplit, mm, mom ? 3 : 1, S, R, Tt, w.tc ? w.tc_scale : nullptr);
        else
            combine_kernel<<<(unsigned)((mm + 255) / 256), 256, 0, st>>>(w.partAB, ab_splits, w.partC, pl.nsplit, mm, mom ? 3 : 1, S, R, Tt, w.tc ? w.tc_scale : nullptr);
        FPSK_LAUNCH_CHECK();
    }
    return FPSK_OK;
}

fpsk_status exclusive_scan_launch(const int *count, int n, int *start, cudaStream_t st)
{
    scan_kernel<<<1, 1024, 0, st>>>(count, n, start);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status contraction_launch(const float *P, const float *Q, float *part, int M, int N, int K, int lda, int ldb,
                               int ksplit, int kchunk, int tile, cudaStream_t st)
{
    GemmBatch g;
    g.P = P; g.Pw = P; g.Q = Q; g.Qw = Q;
    g.Cpart = part;
    g.M = M; g.N = N; g.K = K; g.lda = lda; g.ldb = ldb;
    g.ksplit = ksplit; g.kchunk = kchunk; g.nprob = 1;
    if (tile == 64) {
        dim3 grid((N + 63) / 64, (M + 63) / 64, ksplit);
        sgemm_kernel<64, 64, 4><<<grid, 256, 0, st>>>(g);
    } else {
        dim3 grid((N + 127) / 128, (M + 127) / 128, ksplit);
        sgemm_kernel<128, 128, 8><<<grid, 256, 0, st>>>(g);
    }
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status build_b_side(const void *B, long long ldb, long long n2, long long n3, fpsk_dtype dtype, int m_b, int kpad,
                         int npad, const uint32_t *colperm, const int *colstart, float *Q, cudaStream_t st)
{
    const unsigned short *Bp = static_cast<const unsigned short *>(B);
    const size_t smem = ((size_t)n3 * 2 + 15) / 16 * 16;
    int grid = kpad < 1184 ? kpad : 1184;
    if (dtype == FPSK_FP16) {
        FPSK_CUDA_OK(cudaFuncSetAttribute(compress_b_kernel<__half, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        compress_b_kernel<__half, false><<<grid, 256, smem, st>>>(Bp, ldb, (int)n2, (int)n3, kpad, m_b, npad, 0.f, colperm, colstart, Q, nullptr);
    } else {
        FPSK_CUDA_OK(cudaFuncSetAttribute(compress_b_kernel<__nv_bfloat16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        compress_b_kernel<__nv_bfloat16, false><<<grid, 256, smem, st>>>(Bp, ldb, (int)n2, (int)n3, kpad, m_b, npad, 0.f, colperm, colstart, Q, nullptr);
    }
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status build_sketches(const SketchIn &in, fpsk_dtype dtype, uint64_t seed, int rnd, int m_b, bool mom,
                           SketchWs &w, cudaStream_t st, float *S, float *R, float *T)
{
    if (dtype == FPSK_FP16) return build_sketches_t<__half>(in, seed, rnd, m_b, mom, w, st, S, R, T);
    return build_sketches_t<__nv_bfloat16>(in, seed, rnd, m_b, mom, w, st, S, R, T);
}

fpsk_status peel_launch(const PeelEntry *dF, int nF, uint64_t seed, int rnd, long long n1, long long n3, int m_b,
                        float *S, float *R, float *T, cudaStream_t st, const int *d_nF)
{
    if (!d_nF && nF <= 0) return FPSK_OK;
    const float inv_p1 = 1.0f / (float)(1LL << pow2_exp(n1));
    const float inv_p3 = 1.0f / (float)(1LL << pow2_exp(n3));
    peel_kernel<<<1, 32, 0, st>>>(dF, nF, d_nF, round_key(seed, rnd, 0), round_key(seed, rnd, 1), m_b, inv_p1, inv_p3, S, R, T);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

}  // namespace fpsk
