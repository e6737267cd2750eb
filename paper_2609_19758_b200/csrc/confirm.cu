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

fpsk_status confirm_launch(const SketchIn &in, fpsk_dtype dtype, const Candidate *cand, const int *n_cand,
                           int max_cand, int radius, double c_valid, int force, Hit *hits, int *n_hits, int hit_cap,
                           cudaStream_t st)
{
    if (radius < 0 || 2 * radius + 1 > kConfirmThreads) return FPSK_ERR_PARAM;
    FPSK_CUDA_OK(cudaMemsetAsync(n_hits, 0, sizeof(int), st));
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

}  // namespace fpsk
