// Pieces of Algorithm 2 around the localizer (Section "Nonfinite and Out of Range Entries";
// Algorithm 2, lines "F_abs", "restore" and "Apply"): the exact elementwise scan for entries
// that are not finite or beyond fp32max/16, their recomputation as absolute values, and the
// small scatter that writes values into C (patch, restore, apply).
#include "sketch.cuh"

#include <vector>

namespace fpsk {

constexpr int kScanGrid = 1184;
constexpr int kScanThreads = 256;

__device__ __forceinline__ bool out_of_range(float x)
{
    // NaN and Inf fail the comparison as well
    return !(fabsf(x) <= 3.402823466e38f / 16.f);
}

// pass 1: flagged entries per CTA (each CTA owns a contiguous range of rows)
__global__ void __launch_bounds__(kScanThreads) scan_count_kernel(const float *C, long long ldc, long long n1, long long n3, int *counts)
{
    const long long r0 = n1 * blockIdx.x / gridDim.x, r1 = n1 * (blockIdx.x + 1) / gridDim.x;
    int c = 0;
    for (long long r = r0; r < r1; ++r) {
        const float *row = C + r * ldc;
        for (long long j = threadIdx.x; j < n3; j += kScanThreads) c += out_of_range(row[j]) ? 1 : 0;
    }
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    __shared__ int sh[kScanThreads / 32];
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < kScanThreads / 32; ++w) t += sh[w];
        counts[blockIdx.x] = t;
    }
}

// exclusive scan of the per-CTA counts; total in offsets[grid]
__global__ void scan_offsets_kernel(const int *counts, int grid, int *offsets)
{
    if (threadIdx.x != 0) return;
    int t = 0;
    for (int g = 0; g < grid; ++g) {
        offsets[g] = t;
        t += counts[g];
    }
    offsets[grid] = t;
}

// pass 2: CTAs that saw flagged entries walk their rows again in row-major order and write the
// coordinates at their offset, so that the list is in flat-index order and the first `cap`
// entries are the kept ones (deterministic).
__global__ void __launch_bounds__(kScanThreads) scan_collect_kernel(const float *C, long long ldc, long long n1, long long n3,
                                                                   const int *counts, const int *offsets, int cap, ScanEntry *out)
{
    if (counts[blockIdx.x] == 0) return;
    __shared__ int warp_cnt[kScanThreads / 32];
    __shared__ int base;
    if (threadIdx.x == 0) base = offsets[blockIdx.x];
    __syncthreads();
    const long long r0 = n1 * blockIdx.x / gridDim.x, r1 = n1 * (blockIdx.x + 1) / gridDim.x;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (long long r = r0; r < r1; ++r) {
        const float *row = C + r * ldc;
        for (long long j0 = 0; j0 < n3; j0 += kScanThreads) {
            const long long j = j0 + threadIdx.x;
            const bool f = j < n3 && out_of_range(row[j]);
            const unsigned int bal = __ballot_sync(0xFFFFFFFFu, f);
            if (lane == 0) warp_cnt[wid] = __popc(bal);
            __syncthreads();
            int before = 0, total = 0;
            for (int w = 0; w < kScanThreads / 32; ++w) {
                if (w < wid) before += warp_cnt[w];
                total += warp_cnt[w];
            }
            if (f) {
                const int pos = base + before + __popc(bal & ((1u << lane) - 1u));
                if (pos < cap) out[pos] = ScanEntry{(int)r, (int)j};
            }
            __syncthreads();
            if (threadIdx.x == 0) base += total;
            __syncthreads();
        }
    }
}

__global__ void patch_kernel(float *C, long long ldc, const PatchEntry *e, int n)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    float *dst = C + (long long)e[t].i * ldc + e[t].j;
    if (e[t].mode == PATCH_SET) *dst = (float)e[t].value;
    else if (e[t].mode == PATCH_ADD) *dst = (float)((double)*dst + e[t].value);
    else *dst = *reinterpret_cast<const float *>(&e[t].value);       // PATCH_SET_BITS: the stored bit pattern
}

size_t repair_scratch_bytes()
{
    return align_up((size_t)(kScanGrid + 1) * 4, 256) * 2 + align_up(sizeof(ScanEntry) * kRepairCap, 256) +
           align_up(sizeof(PatchEntry) * kRepairCap, 256) + align_up(sizeof(Candidate) * kRepairCap, 256) +
           align_up(sizeof(Hit) * kRepairCap, 256) + 256;
}

fpsk_status patch_launch(float *C, long long ldc, const PatchEntry *d_entries, int n, cudaStream_t st)
{
    if (n <= 0) return FPSK_OK;
    patch_kernel<<<(n + 127) / 128, 128, 0, st>>>(C, ldc, d_entries, n);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status scan_launch(const float *C, long long ldc, long long n1, long long n3, int cap, void *scratch, cudaStream_t st,
                        ScanEntry *h_entries, int *h_count)
{
    if (cap > kRepairCap) cap = kRepairCap;
    char *p = static_cast<char *>(scratch);
    int *counts = reinterpret_cast<int *>(p); p += align_up((size_t)(kScanGrid + 1) * 4, 256);
    int *offsets = reinterpret_cast<int *>(p); p += align_up((size_t)(kScanGrid + 1) * 4, 256);
    ScanEntry *ent = reinterpret_cast<ScanEntry *>(p);
    const int grid = (int)(n1 < kScanGrid ? n1 : kScanGrid);
    scan_count_kernel<<<grid, kScanThreads, 0, st>>>(C, ldc, n1, n3, counts);
    FPSK_LAUNCH_CHECK();
    scan_offsets_kernel<<<1, 32, 0, st>>>(counts, grid, offsets);
    FPSK_LAUNCH_CHECK();
    scan_collect_kernel<<<grid, kScanThreads, 0, st>>>(C, ldc, n1, n3, counts, offsets, cap, ent);
    FPSK_LAUNCH_CHECK();
    int total = 0;
    FPSK_CUDA_OK(cudaMemcpyAsync(&total, offsets + grid, 4, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    const int n = total < cap ? total : cap;
    if (n > 0) {
        FPSK_CUDA_OK(cudaMemcpyAsync(h_entries, ent, sizeof(ScanEntry) * n, cudaMemcpyDeviceToHost, st));
        FPSK_CUDA_OK(cudaStreamSynchronize(st));
    }
    *h_count = n;
    return FPSK_OK;
}

// gamma = A_i,* . B_*,j in FP64 for a list of entries (the confirmation kernel with radius 0,
// reporting every entry whatever its test says); also the entries' current values.
fpsk_status recompute_entries(const SketchIn &in, fpsk_dtype dtype, const ScanEntry *h_entries, int n, void *scratch,
                              cudaStream_t st, double *h_gamma, float *h_old)
{
    if (n <= 0) return FPSK_OK;
    if (n > kRepairCap) return FPSK_ERR_CAPACITY;
    char *p = static_cast<char *>(scratch);
    p += align_up((size_t)(kScanGrid + 1) * 4, 256) * 2 + align_up(sizeof(ScanEntry) * kRepairCap, 256) +
         align_up(sizeof(PatchEntry) * kRepairCap, 256);
    Candidate *d_cand = reinterpret_cast<Candidate *>(p); p += align_up(sizeof(Candidate) * kRepairCap, 256);
    Hit *d_hits = reinterpret_cast<Hit *>(p); p += align_up(sizeof(Hit) * kRepairCap, 256);
    int *d_cnt = reinterpret_cast<int *>(p);        // [0] number of candidates, [1] number of hits
    std::vector<Candidate> cand((size_t)n);
    for (int e = 0; e < n; ++e) cand[e] = Candidate{e, h_entries[e].i, h_entries[e].j, 0.f};
    FPSK_CUDA_OK(cudaMemcpyAsync(d_cand, cand.data(), sizeof(Candidate) * n, cudaMemcpyHostToDevice, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(d_cnt, &n, 4, cudaMemcpyHostToDevice, st));
    fpsk_status rc = confirm_launch(in, dtype, d_cand, d_cnt, n, 0, 100.0, 1, d_hits, d_cnt + 1, kRepairCap, st);
    if (rc != FPSK_OK) return rc;
    std::vector<Hit> hits((size_t)n);
    int nh = 0;
    FPSK_CUDA_OK(cudaMemcpyAsync(&nh, d_cnt + 1, 4, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(hits.data(), d_hits, sizeof(Hit) * n, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    if (nh != n) return FPSK_ERR_CAPACITY;
    for (int h = 0; h < n; ++h) {
        const int e = hits[h].cand;
        if (e < 0 || e >= n) return FPSK_ERR_CAPACITY;
        h_gamma[e] = hits[h].gamma;
        h_old[e] = hits[h].c_value;
    }
    return FPSK_OK;
}

}  // namespace fpsk
