// fpsk_probe_static: the detection probe for callers that cannot allocate device memory.
//
// Some callers may not call cudaMalloc (or any allocator) at the point where they verify a
// GEMM: code running inside a stream-capture region, a real-time or fault-handling path that
// must not take the allocator's locks, or a plug-in that is handed tensors but owns no memory
// pool.  fpsk_probe needs about 10 MB of scratch (partial sums, synchronisation words) that
// such a caller would have to allocate.  This variant keeps that scratch in a fixed array
// inside the library instead.  The kernel is the one fpsk_probe launches; only the origin of
// the scratch differs.
#include "fpsk_common.cuh"

#include <mutex>

namespace fpsk {

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_probe_scratch[FPSK_PROBE_STATIC_SCRATCH_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address, so the
// address is looked up once per device (with that device current) and cached here.
static void *g_scratch_addr[64];
static std::mutex g_scratch_mu;

static fpsk_status scratch_address(void **out)
{
    int dev = 0;
    FPSK_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return FPSK_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        FPSK_CUDA_OK(cudaGetSymbolAddress(&ptr, g_probe_scratch));
        if (!ptr) return FPSK_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return FPSK_OK;
}

}  // namespace fpsk

using namespace fpsk;

extern "C" fpsk_status fpsk_probe_static(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C,
                                         int64_t ldc, int64_t m, int64_t k, int64_t n, fpsk_dtype dtype,
                                         int c_is_fp32, const fpsk_params *p, void *stream,
                                         fpsk_probe_result *d_result, float *d_residual)
{
    if (!c_is_fp32) return FPSK_ERR_DTYPE;
    if (!A || !B || !C || !d_result) return FPSK_ERR_NULL;
    if (dtype != FPSK_FP16 && dtype != FPSK_BF16) return FPSK_ERR_DTYPE;
    if (m < 1 || k < 1 || n < 1 || lda < k || ldb < n || ldc < n) return FPSK_ERR_SHAPE;
    if (m >= (1LL << 30) || k >= (1LL << 30) || n >= (1LL << 30)) return FPSK_ERR_SHAPE;
    double mu = 4.0;
    if (p) {
        if (!(p->mu > 0) || p->b_transposed) return FPSK_ERR_PARAM;      // B is streamed as k x n here
        mu = p->mu;
    }
    // shapes whose scratch does not fit the built-in array are refused, never truncated
    if (probe_ws_bytes(m, k, n) > (size_t)FPSK_PROBE_STATIC_SCRATCH_BYTES) return FPSK_ERR_WORKSPACE;
    void *scratch = nullptr;
    fpsk_status rc = scratch_address(&scratch);
    if (rc != FPSK_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left.  Only the synchronisation words must
    // start at zero (a call that timed out leaves them dirty); everything else is overwritten
    // before it is read.
    FPSK_CUDA_OK(cudaMemsetAsync(scratch, 0, 256, st));
    ProbeDims d{m, k, n, lda, ldb, ldc};
    return probe_launch(A, B, C, d, dtype, mu, scratch, (size_t)FPSK_PROBE_STATIC_SCRATCH_BYTES, st, d_result,
                        d_residual);
}
