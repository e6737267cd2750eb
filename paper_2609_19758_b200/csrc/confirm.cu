// Confirmation of candidates (Section "Validation"; Algorithm 1, neighbourhood search):
// for every candidate and every offset of its (2r+1)^2 window, gamma = A_i,* . B_*,j is
// recomputed in FP64 together with sum_k |A_ik||B_kj|, and the entry is a hit iff
// |gamma - C_ij| > c eps sum_k |A_ik||B_kj| (eps = 2^-23).  The acceptance test of an entry
// does not depend on the search state, so all window entries are tested in parallel and the
// ordered walk of Algorithm 1 is replayed afterwards over the (few) hits.
#include "sketch.cuh"

namespace fpsk {

constexpr int kConfirmThreads = 1024;     // many k slices per window entry: the dot products are load latency

// CTA (x: candidate, y: row offset d_i + r).  Thread (slice, d_j) accumulates every
// `slices`-th k of column j_hat + d_j; slices are then summed in slice order.  Adjacent lanes take adjacent
// columns when B is k x n (a row of B is contiguous in j) and adjacent slices when B comes as W = B^T (a row of W
// is contiguous in k).
template <typename T>
__global__ void __launch_bounds__(kConfirmThreads) confirm_kernel(
    const unsigned short *A, long long lda, const unsigned short *B, long long ldb, const float *C, long long ldc,
    long long n1, long long n2, long long n3, const Candidate *cand, const int *n_cand, int r, double c_valid, int force,
    Hit *hits, int *n_hits, int hit_cap, int bt)
{
    __shared__ double sg[kConfirmThreads];
    __shared__ double sa[kConfirmThreads];
    const int u = blockIdx.x;
    if (u >= *n_cand) return;
    const int W = 2 * r + 1;
    const int di = (int)blockIdx.y - r;
    const long long i = (long long)cand[u].ih + di;
    if (i < 0 || i >= n1) return;
    const int slices = kConfirmThreads / W;
    const int dj = bt ? (int)threadIdx.x / slices : (int)threadIdx.x % W;
    const int ks = bt ? (int)threadIdx.x % slices : (int)threadIdx.x / W;
    const long long j = (long long)cand[u].jh - r + dj;
    const bool active = ks < slices && dj < W && j >= 0 && j < n3;
    double g = 0.0, ab = 0.0;
    if (active) {
        const unsigned short *arow = A + i * lda;
        // column j of B: strided in B, or row j of the transposed weight
        const unsigned short *bcol = bt ? B + j * ldb : B + j;
        const long long bstep = bt ? 1 : ldb;
        // eight loads of each operand in flight per thread; the sums run in ascending k of the slice
        long long k = ks;
        for (; k + 7 * (long long)slices < n2; k += 8 * (long long)slices) {
            unsigned short av[8], bv[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                av[q] = arow[k + q * slices];
                bv[q] = bcol[(k + q * slices) * bstep];
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const double p = (double)bits16_to_float<T>(av[q]) * (double)bits16_to_float<T>(bv[q]);   // exact
                g += p;
                ab += fabs(p);
            }
        }
        for (; k < n2; k += slices) {
            const double a = (double)bits16_to_float<T>(arow[k]);
            const double b = (double)bits16_to_float<T>(bcol[k * bstep]);
            const double p = a * b;          // exact: two <= 11-bit significands
            g += p;
            ab += fabs(p);
        }
    }
    if (ks < slices && dj < W) {
        sg[ks * W + dj] = g;
        sa[ks * W + dj] = ab;
    }
    __syncthreads();
    if (active && ks == 0) {
        for (int s = 1; s < slices; ++s) {
            g += sg[s * W + dj];
            ab += sa[s * W + dj];
        }
        const float cij = C[i * ldc + j];
        const double tau_ij = c_valid * 1.1920928955078125e-07 * ab;
        if (force || fabs(g - (double)cij) > tau_ij) {
            const int slot = atomicAdd(n_hits, 1);
            if (slot < hit_cap) {
                Hit h;
                h.cand = u; h.di = di; h.dj = dj - r; h.i = (int)i; h.j = (int)j;
                h.c_value = cij; h.gamma = g;
                hits[slot] = h;
            }
        }
    }
}

// ---------------------------------------------------------------- first moments of the candidate buckets only
// Only the K buckets that the selection keeps ever have their R and T read (Eq. (recover)), so the two weighted
// sketches are not built whole: for a kept bucket (a, b)
//   R = sum_k Pw[a,k] Q[k,b] - sum_{i in a, j in b} v1 v2 w_i C_ij,    T = sum_k P[a,k] Qw[k,b] - sum v1 v2 w_j C_ij,
// with the compressed rows and columns formed on the fly from the bucket's rows of A and columns of B (same FP32
// order as the compressions), the products accumulated in FP64, and the peeled faults of the bucket subtracted.
// One CTA per collected key.
constexpr int kMomThreads = 1024;         // few CTAs do any work (one per kept bucket): wide ones
template <typename T>
__global__ void __launch_bounds__(kMomThreads) candidate_moments_kernel(
    const unsigned short *A, long long lda, const unsigned short *B, long long ldb, int bt, const float *C, long long ldc,
    int n1, int n2, int n3, int m_b, float inv_p1, float inv_p3, const uint32_t *rowperm, const int *rowstart, const uint32_t *colperm,
    const int *colstart, const unsigned long long *keys, const int *counts, int cap, const PeelEntry *peel, const int *d_n_peel,
    uint32_t key1, uint32_t key2, float *Rc, float *Tc, int vec)
{
    __shared__ double sr[kMomThreads], st_[kMomThreads];
    const int slot = blockIdx.x;
    int n = counts[1];
    if (n > cap) n = cap;
    if (slot >= n) return;
    const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(keys[slot] & 0xFFFFFFFFull);
    const int a = (int)(idx / (uint32_t)m_b), b = (int)(idx % (uint32_t)m_b);
    if (!FPSK_IN_BOUNDS(a, m_b)) return;          // a key that does not name a bucket
    const int r0 = rowstart[a], r1 = rowstart[a + 1], c0 = colstart[b], c1 = colstart[b + 1];
    double accR = 0.0, accT = 0.0;
    if (vec) {
        // eight consecutive k per thread, four rows (columns) of the bucket in flight: the walk is load latency
        for (int k0 = threadIdx.x * 8; k0 < n2; k0 += kMomThreads * 8) {
            float p[8] = {0, 0, 0, 0, 0, 0, 0, 0}, pw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            float q[8] = {0, 0, 0, 0, 0, 0, 0, 0}, qw[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int side = 0; side < 2; ++side) {
                const uint32_t *perm = side ? colperm : rowperm;
                const unsigned short *X = side ? B : A;
                const long long ld = side ? ldb : lda;
                const float inv_p = side ? inv_p3 : inv_p1;
                const int b0 = side ? c0 : r0, b1 = side ? c1 : r1;
                for (int sb = b0; sb < b1; sb += 4) {
                    uint32_t e4[4];
                    uint4 v4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) e4[u] = sb + u < b1 ? __ldg(perm + sb + u) : 0u;
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        v4[u] = sb + u < b1 ? ldg_nc_v4(X + (long long)(e4[u] & 0x7FFFFFFFu) * ld + k0) : make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (sb + u >= b1) break;
                        const int i = (int)(e4[u] & 0x7FFFFFFFu);
                        const float sg = (e4[u] >> 31) ? -1.f : 1.f;
                        const float sw = sg * ((float)(i + 1) * inv_p);
                        const unsigned int ww[4] = {v4[u].x, v4[u].y, v4[u].z, v4[u].w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const float2 f = HalfTraits<T>::unpack2(ww[t]);
                            if (side == 0) {
                                p[2 * t] += sg * f.x; p[2 * t + 1] += sg * f.y;
                                pw[2 * t] = fmaf(sw, f.x, pw[2 * t]); pw[2 * t + 1] = fmaf(sw, f.y, pw[2 * t + 1]);
                            } else {
                                q[2 * t] += sg * f.x; q[2 * t + 1] += sg * f.y;
                                qw[2 * t] = fmaf(sw, f.x, qw[2 * t]); qw[2 * t + 1] = fmaf(sw, f.y, qw[2 * t + 1]);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                accR += (double)pw[t] * (double)q[t];
                accT += (double)p[t] * (double)qw[t];
            }
        }
    } else {
        for (int k = threadIdx.x; k < n2; k += kMomThreads) {
            float p = 0.f, pw = 0.f, q = 0.f, qw = 0.f;
            for (int s = r0; s < r1; ++s) {
                const uint32_t e = __ldg(rowperm + s);
                const int i = (int)(e & 0x7FFFFFFFu);
                if (!FPSK_IN_BOUNDS(i, n1)) continue;
                const float sg = (e >> 31) ? -1.f : 1.f;
                const float x = bits16_to_float<T>(A[(long long)i * lda + k]);
                p += sg * x;
                pw = fmaf(sg * ((float)(i + 1) * inv_p1), x, pw);
            }
            for (int s = c0; s < c1; ++s) {
                const uint32_t e = __ldg(colperm + s);
                const int j = (int)(e & 0x7FFFFFFFu);
                if (!FPSK_IN_BOUNDS(j, n3)) continue;
                const float sg = (e >> 31) ? -1.f : 1.f;
                const float y = bits16_to_float<T>(bt ? B[(long long)j * ldb + k] : B[(long long)k * ldb + j]);
                q += sg * y;
                qw = fmaf(sg * ((float)(j + 1) * inv_p3), y, qw);
            }
            accR += (double)pw * (double)q;
            accT += (double)p * (double)qw;
        }
    }
    // the bucket's entries of C, one (row, column) pair per thread and step
    const int nr = r1 - r0, nc = c1 - c0;
    for (int e = threadIdx.x; e < nr * nc; e += kMomThreads) {
        const uint32_t er = __ldg(rowperm + r0 + e / nc), ec = __ldg(colperm + c0 + e % nc);
        const int i = (int)(er & 0x7FFFFFFFu), j = (int)(ec & 0x7FFFFFFFu);
        if (!FPSK_IN_BOUNDS(i, n1) || !FPSK_IN_BOUNDS(j, n3)) continue;
        const double v = ((er >> 31) != (ec >> 31)) ? -1.0 : 1.0;
        const double c = (double)C[(long long)i * ldc + j];
        accR -= v * (double)((float)(i + 1) * inv_p1) * c;
        accT -= v * (double)((float)(j + 1) * inv_p3) * c;
    }
    sr[threadIdx.x] = accR;
    st_[threadIdx.x] = accT;
    __syncthreads();
    for (int s = kMomThreads / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) { sr[threadIdx.x] += sr[threadIdx.x + s]; st_[threadIdx.x] += st_[threadIdx.x + s]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double R = sr[0], Tm = st_[0];
        // faults confirmed in earlier rounds that hash into this bucket (Algorithm 1, peeling)
        const int n_peel = d_n_peel ? *d_n_peel : 0;
        for (int f = 0; f < n_peel; ++f) {
            int a2, b2, s1, s2;
            hash_index(key1, (uint32_t)peel[f].i, (uint32_t)m_b, a2, s1);
            if (a2 != a) continue;
            hash_index(key2, (uint32_t)peel[f].j, (uint32_t)m_b, b2, s2);
            if (b2 != b) continue;
            const double g = (double)(s1 * s2) * peel[f].delta;
            R -= g * ((double)(peel[f].i + 1) * (double)inv_p1);
            Tm -= g * ((double)(peel[f].j + 1) * (double)inv_p3);
        }
        Rc[slot] = (float)R;
        Tc[slot] = (float)Tm;
    }
}

fpsk_status candidate_moments_launch(const SketchIn &in, fpsk_dtype dtype, const SketchWs &sk, int m_b, int K, SelectWs &sel,
                                     const PeelEntry *d_peel, const int *d_n_peel, uint64_t seed, int rnd, cudaStream_t st)
{
    if (K < 1) return FPSK_OK;
    int p1 = 0, p3 = 0;
    while ((1LL << p1) < in.n1) ++p1;
    while ((1LL << p3) < in.n3) ++p3;
    const float inv_p1 = 1.0f / (float)(1LL << p1), inv_p3 = 1.0f / (float)(1LL << p3);
    const unsigned short *A = static_cast<const unsigned short *>(in.A);
    const unsigned short *B = static_cast<const unsigned short *>(in.B);
    const uint32_t key1 = round_key(seed, rnd, 0), key2 = round_key(seed, rnd, 1);
    // 16-byte loads along k need both operands as rows contiguous in k (B as W = B^T) and aligned
    const int vec = (in.bt && ((reinterpret_cast<uintptr_t>(in.A) | reinterpret_cast<uintptr_t>(in.B)) & 15) == 0 && in.lda % 8 == 0 &&
                     in.ldb % 8 == 0 && in.n2 % 8 == 0) ? 1 : 0;
    if (dtype == FPSK_FP16)
        candidate_moments_kernel<__half><<<K, kMomThreads, 0, st>>>(A, in.lda, B, in.ldb, in.bt, in.C, in.ldc, (int)in.n1, (int)in.n2, (int)in.n3, m_b, inv_p1,
                                                            inv_p3, sk.rowperm, sk.rowstart, sk.colperm, sk.colstart, sel.keys,
                                                            sel.counts, kSelMaxK, d_peel, d_n_peel, key1, key2, sel.Rc, sel.Tc, vec);
    else
        candidate_moments_kernel<__nv_bfloat16><<<K, kMomThreads, 0, st>>>(A, in.lda, B, in.ldb, in.bt, in.C, in.ldc, (int)in.n1, (int)in.n2, (int)in.n3, m_b,
                                                                   inv_p1, inv_p3, sk.rowperm, sk.rowstart, sk.colperm,
                                                                   sk.colstart, sel.keys, sel.counts, kSelMaxK, d_peel, d_n_peel,
                                                                   key1, key2, sel.Rc, sel.Tc, vec);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status confirm_launch(const SketchIn &in, fpsk_dtype dtype, const Candidate *cand, const int *n_cand,
                           int max_cand, int radius, double c_valid, int force, Hit *hits, int *n_hits, int hit_cap,
                           cudaStream_t st, bool hits_cleared)
{
    if (radius < 0 || 2 * radius + 1 > kConfirmThreads) return FPSK_ERR_PARAM;
    if (!hits_cleared) FPSK_CUDA_OK(cudaMemsetAsync(n_hits, 0, sizeof(int), st));
    dim3 grid(max_cand, 2 * radius + 1);
    const unsigned short *A = static_cast<const unsigned short *>(in.A);
    const unsigned short *B = static_cast<const unsigned short *>(in.B);
    if (dtype == FPSK_FP16)
        confirm_kernel<__half><<<grid, kConfirmThreads, 0, st>>>(A, in.lda, B, in.ldb, in.C, in.ldc, in.n1, in.n2, in.n3,
                                                                 cand, n_cand, radius, c_valid, force, hits, n_hits, hit_cap, in.bt);
    else
        confirm_kernel<__nv_bfloat16><<<grid, kConfirmThreads, 0, st>>>(A, in.lda, B, in.ldb, in.C, in.ldc, in.n1, in.n2,
                                                                        in.n3, cand, n_cand, radius, c_valid, force, hits, n_hits,
                                                                        hit_cap, in.bt);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- ordered search over a round's hits, on the device
constexpr int kReplayThreads = 1024;
constexpr int kReplayMaxHits = 2048;

__device__ __forceinline__ unsigned int offset_rank(int di, int dj, int r)
{
    // Chebyshev, then Manhattan, then d_i, then d_j (all ascending) packed into one integer (< 2^23 for r <= 16)
    const int ch = max(abs(di), abs(dj)), mh = abs(di) + abs(dj);
    return (unsigned int)(((ch * 64 + mh) * 64 + (di + r)) * 64 + (dj + r));
}

__global__ void __launch_bounds__(kReplayThreads) replay_kernel(const Hit *hits, const int *n_hits, int hit_cap,
                                                               const Candidate *cand, const int *n_cand, int K, int radius,
                                                               int round, DevFault *F, int f_cap, PeelEntry *peel, int *rstate)
{
    __shared__ unsigned long long keys[kReplayMaxHits];       // (offset rank, candidate, hit index): all distinct
    __shared__ unsigned char in_f[kReplayMaxHits];            // the hit's entry was confirmed in an earlier round
    __shared__ unsigned char alive[kSelMaxK];
    const int tid = (int)threadIdx.x;
    int nh = *n_hits;
    const bool over = nh > hit_cap || nh > kReplayMaxHits;
    if (nh > hit_cap) nh = hit_cap;
    if (nh > kReplayMaxHits) nh = kReplayMaxHits;
    const int nU = min(*n_cand, K);
    const int nF0 = min(rstate[0], f_cap);
    int np2 = 1;
    while (np2 < nh) np2 <<= 1;
    for (int h = tid; h < np2; h += kReplayThreads) {
        unsigned long long key = ~0ull;
        unsigned char seen = 0;
        if (h < nh) {
            const Hit x = hits[h];
            key = ((unsigned long long)offset_rank(x.di, x.dj, radius) << 32) | ((unsigned long long)(unsigned int)(x.cand & 0xFFFF) << 16) |
                  (unsigned long long)h;
            for (int f = 0; f < nF0; ++f)
                if (F[f].i == x.i && F[f].j == x.j) { seen = 1; break; }
        }
        keys[h] = key;
        in_f[h] = seen;
    }
    for (int u = tid; u < kSelMaxK; u += kReplayThreads) alive[u] = 1;
    __syncthreads();
    // bitonic sort, ascending, over the next power of two of the hits present
    for (int k2 = 2; k2 <= np2; k2 <<= 1) {
        for (int j2 = k2 >> 1; j2 > 0; j2 >>= 1) {
            for (int t = tid; t < np2; t += kReplayThreads) {
                const int p = t ^ j2;
                if (p > t) {
                    const unsigned long long a = keys[t], b = keys[p];
                    const bool up = (t & k2) == 0;
                    if ((a > b) == up) { keys[t] = b; keys[p] = a; }
                }
            }
            __syncthreads();
        }
    }
    if (tid != 0) return;
    int nF = nF0, nP = rstate[1], trunc = over ? 1 : 0;
    for (int s = 0; s < nh; ++s) {
        const int h = (int)(keys[s] & 0xFFFFull);
        const Hit x = hits[h];
        if (x.cand < 0 || x.cand >= nU || !alive[x.cand] || in_f[h]) continue;
        bool dup = false;                       // the same entry reached through another bucket of this round
        for (int f = nF0; f < nF; ++f)
            if (F[f].i == x.i && F[f].j == x.j) { dup = true; break; }
        if (dup) continue;
        if (nF >= f_cap) { trunc = 1; break; }
        DevFault d;
        d.i = x.i; d.j = x.j; d.gamma = x.gamma; d.c_value = x.c_value; d.round = round; d.flat = cand[x.cand].flat; d.pad = 0;
        F[nF++] = d;
        const double delta = x.gamma - (double)x.c_value;
        // only finite faults are peeled (Section "Peeling Across Hash Rounds")
        if (isfinite(delta)) {
            PeelEntry e;
            e.i = x.i; e.j = x.j; e.delta = delta;
            peel[nP++] = e;                     // nP <= nF <= f_cap: the lists have the same capacity
        }
        alive[x.cand] = 0;
    }
    rstate[0] = nF;
    rstate[1] = nP;
    if (trunc) rstate[2] = 1;
}

fpsk_status replay_launch(const Hit *hits, const int *n_hits, int hit_cap, const Candidate *cand, const int *n_cand, int K,
                          int radius, int round, DevFault *F, int f_cap, PeelEntry *peel, int *rstate, cudaStream_t st)
{
    if (K > kSelMaxK) return FPSK_ERR_PARAM;
    replay_kernel<<<1, kReplayThreads, 0, st>>>(hits, n_hits, hit_cap, cand, n_cand, K, radius, round, F, f_cap, peel, rstate);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

}  // namespace fpsk
