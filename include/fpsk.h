/*
 * fpsk.h - C ABI of the B200 FP-Sketch verifier.
 *
 * FP-Sketch verifies a half-precision tensor-core GEMM after the fact.  The GEMM under
 * test delivers its FP32 accumulator C (n1 x n3) un-narrowed; the verifier reads the
 * operands A (n1 x n2, FP16 or BF16) and B (n2 x n3, same type) and C and never forms AB
 * (paper: Introduction; Section "Mixed Precision GEMM and Where to Verify").
 *
 * Conventions for every entry point
 *   - All matrices are row-major.  lda, ldb, ldc are leading dimensions in ELEMENTS.
 *   - Pointers named d_* or documented "device" must be device memory of the current
 *     device; pointers named h_* are host memory.  A, B, C, workspace are device memory
 *     unless an entry point says otherwise.
 *   - The caller owns every buffer.  The library allocates no device memory and never writes
 *     to A or B; C is written only by fpsk_verify_repair and fpsk_apply_corrections (paper,
 *     Section "Overview": localization does not modify C; Algorithm 2, "Apply").
 *     fpsk_measure_noise, fpsk_localize and fpsk_verify_repair read their results back through a small
 *     pinned host buffer (about 16 KB) and run independent parts of their work on three auxiliary
 *     non-blocking streams, tied to `stream` by events on both sides (work queued on `stream` before the
 *     call is complete before any of it starts; everything is complete when the call returns, also when
 *     it returns an error).  These host resources are the caller's when it passes a context
 *     (fpsk_context_create, fpsk_params.context); otherwise they are created on first use, one set per
 *     concurrent call and device, and kept for the life of the process.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Indices are 0-based.  The 1-based index weights of the paper are internal.
 *   - Errors are return codes.  Nothing throws, aborts or resets the device.  After
 *     FPSK_ERR_CUDA the CUDA error is left for the caller to query.
 *   - Fast paths use 128-bit loads when the base pointers are 16-byte aligned and the
 *     leading dimensions are multiples of 8 (A, B) / 4 (C) elements; otherwise a scalar
 *     path with the same arithmetic order runs.
 */
#ifndef FPSK_H
#define FPSK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { FPSK_FP16 = 0, FPSK_BF16 = 1 } fpsk_dtype;   /* operand type of A and B */

typedef enum {
    FPSK_OK = 0,
    FPSK_ERR_NULL = 1,       /* a required pointer is NULL                                  */
    FPSK_ERR_SHAPE = 2,      /* a dimension < 1, a leading dimension too small, or too large */
    FPSK_ERR_DTYPE = 3,      /* unknown operand type, or C is not FP32                       */
    FPSK_ERR_ALIGN = 4,      /* workspace not 256-byte aligned                               */
    FPSK_ERR_WORKSPACE = 5,  /* workspace smaller than the matching *_workspace_bytes()      */
    FPSK_ERR_BUCKETS = 6,    /* bucket count < 1 or beyond what the kernels support          */
    FPSK_ERR_CAPACITY = 7,   /* fault list or an internal list was truncated                 */
    FPSK_ERR_CUDA = 8,       /* a CUDA call failed                                           */
    FPSK_ERR_TIMEOUT = 9,    /* a bounded device-side wait gave up                           */
    FPSK_ERR_PARAM = 10      /* a parameter is out of range                                  */
} fpsk_status;

/* Verdict of the probe; lives in device memory so that it can stay there until the caller
 * reads it once per step (paper, Section "The Cheap S Only Probe"). */
typedef struct {
    int32_t fired;       /* 1: dirty (max|s| > thr, or s not finite); 0: clean            */
    int32_t nonfinite;   /* 1: some sketch entry is Inf or NaN (Section "Nonfinite")       */
    int32_t argmax_col;  /* column with the largest |s_j|                                  */
    int32_t status;      /* fpsk_status set by the device (FPSK_ERR_TIMEOUT) else FPSK_OK  */
    float max_abs;       /* max_j |s_j| over the finite entries                            */
    float sigma_hat;     /* 1.2533 mean(min(|s|, 5 mean|s|))                               */
    float thr;           /* min(tau sqrt(n1), mu sqrt(2 ln N_b) sigma_hat), N_b = max(n3, 2) */
    float tau;           /* 100 n2 2^-23 max|A| max|B|                                     */
} fpsk_probe_result;

/* One confirmed fault (paper, Section "Validation"; Algorithm 1). */
typedef struct {
    int32_t i, j;        /* 0-based coordinate in C                                        */
    double delta;        /* correction gamma - C_ij, i.e. E_ij; an injected +d reads -d    */
    double recompute;    /* gamma = A_i,* . B_*,j accumulated in FP64                      */
    float c_value;       /* the delivered C_ij                                             */
    int32_t round;       /* hash round that found it                                       */
    int32_t bucket_a, bucket_b;   /* its bucket (h1(i), h2(j)) in that round               */
} fpsk_fault;

/* Engine parameters; fpsk_default_params() fills the paper's defaults
 * (Section "Methodology": k=3, rho_min=0.02, r*=4, r_max=16; Section "Validation": c=100;
 *  Section "Thresholds": mu=4; Section "Sketch Noise Sets the Bucket Count": B*=0.3, c=2). */
typedef struct {
    int32_t rounds;      /* k hash rounds, 1..8                                            */
    int32_t r_star;      /* target radius                                                  */
    int32_t r_max;       /* largest radius, <= 16                                          */
    int32_t radius;      /* search radius; -1 = derive it from the measured noise          */
    int32_t s_budget;    /* declared fault count s (sets K = max(64, 8 s) and m_comb)      */
    int32_t delta_max;   /* declared bound Delta on faults per row or column               */
    int32_t mad_of_abs;  /* 1: MAD of |S| as printed in the paper; 0: signed MAD of S      */
    int32_t tensor_cores;/* 0: FP32 FMA contraction; 1: tcgen05 contraction on two scaled FP16
                            terms per FP32 value (three products, FP32 accumulation in TMEM)   */
    int32_t b_transposed;/* fpsk_measure_noise, fpsk_localize: 1 = the B pointer is the weight
                            W = B^T (n x k, row-major, ldb >= k), i.e. C = A W^T; 0 = B is k x n.
                            Other entry points take B as k x n (fpsk_probe_hashed has its own
                            switch in fpsk_bside).                                          */
    int32_t scale_cap;   /* fpsk_probe_hashed only.  0 (default): thr = min(tau, ...) exactly as Section
                            "Thresholds" prints it; 1: the analytic cap enters as tau sqrt(m n / n_buckets^2)
                            (not in the paper: for sketches so coarse that a clean bucket, which sums
                            m n / n_buckets^2 entries of E, can exceed the bound on ONE inner product)     */
    double rho_min;      /* smallest fault to localize, in units of rms(C)                 */
    double c_valid;      /* c of tau_ij = c eps sum_k |A_ik||B_kj|                         */
    double mu;           /* probe margin                                                   */
    double b_star;       /* target index budget                                            */
    double c_coll;       /* collision constant of m_comb                                   */
    void *context;       /* fpsk_context* of the caller (see fpsk_context_create), or NULL: the library then
                            creates the auxiliary streams, events and pinned buffer itself on first use      */
} fpsk_params;

/* Result of the run-time noise measurement (Section "Fault Magnitude, Calibration, and the
 * Neighbourhood Search"). */
typedef struct {
    double sigma_clip;       /* clipped-mean estimate on S at m0                            */
    double sigma_mad;        /* MAD estimate on the same S                                  */
    double rms_c;            /* strided, clipped rms of C                                   */
    double c_hat;            /* sigma_clip m0 / (2^-24 sqrt(n1 n2 n3) rms_c)                */
    double index_budget_B;   /* B = max(n1,n3) sigma / (rho_min rms)                        */
    int32_t m0;              /* bucket count the measurement ran at                         */
    int32_t m_probe;         /* recalibrated probe bucket count m'                          */
    int32_t m_loc;           /* bucket count for localization                               */
    int32_t radius;          /* search radius r for localization                            */
} fpsk_noise;

const char *fpsk_status_string(fpsk_status s);
void fpsk_default_params(fpsk_params *p);

/* ---- host-only scalar planning (no device work) --------------------------------------- */

/* Starting bucket count of Eq. (mstart): min(max(m_comb, m_num, 16), max(m_comb, m_max)) with
 * m_num from Eq. (mnum) at delta = rms(C).  Returns the count, or -1 on bad arguments.
 * (m,k,n) = (n1,n2,n3). */
int32_t fpsk_law_m_start(int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, const fpsk_params *p);

/* Calibration plan of Section "Calibration": from a noise estimate sigma_hat measured at
 * bucket count m_cur and an rms estimate of C, the localization bucket count and radius.
 * A non-positive or non-finite estimate falls back to Eq. (sigma).  Outputs are host
 * pointers; index_budget may be NULL. */
fpsk_status fpsk_plan(int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, double sigma_hat,
                      double rms_c, int32_t m_cur, const fpsk_params *p,
                      int32_t *m_loc, int32_t *radius, double *index_budget);

/* ---- probe: detection on every call ------------------------------------------------------ */

/* Bytes of device workspace fpsk_probe needs for this shape (0 on bad arguments). */
size_t fpsk_probe_workspace_bytes(int64_t m, int64_t k, int64_t n);

/* One-time preparation of a probe workspace: zeroes its synchronisation words (async on
 * `stream`).  Call once after allocating the workspace, and again after a probe reported
 * FPSK_ERR_TIMEOUT in its result.  A workspace serves one probe at a time: probes sharing a
 * workspace must be ordered on one stream. */
fpsk_status fpsk_probe_init(void *workspace, size_t ws_bytes, void *stream);

/* The detection sketch (Eq. (S) with H1 = 1^T, H2 = I): s = (1^T A) B - 1^T C, its noise
 * estimate, threshold and one-bit verdict (Section "Thresholds"; Algorithm 2, probe part;
 * each entry of s sums n1 entries of E, so the analytic cap tau enters as tau sqrt(n1)),
 * in ONE kernel launch, asynchronous on `stream`, no host synchronisation.
 *   A, B       device, m x k and k x n, type `dtype`
 *   C          device, m x n FP32; c_is_fp32 must be 1: a narrowed C is rejected
 *              (Algorithm 2 line 1) with FPSK_ERR_DTYPE
 *   d_result   device, written by the kernel; valid once `stream` has been synchronised
 *   d_residual device, n floats receiving s, or NULL
 * Reads 2mk + 2kn + 4mn bytes.  Deterministic: fixed summation order, no float atomics. */
fpsk_status fpsk_probe(const void *A, int64_t lda, const void *B, int64_t ldb,
                       const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                       fpsk_dtype dtype, int c_is_fp32, const fpsk_params *p,
                       void *workspace, size_t ws_bytes, void *stream,
                       fpsk_probe_result *d_result, float *d_residual);

/* The same probe for operands in (pinned) HOST memory: copies A, B, C into staging space
 * inside the workspace, runs fpsk_probe, copies the verdict back and synchronises `stream`.
 * The workspace must hold fpsk_probe_workspace_bytes() + 2mk + 2kn + 4mn (+ 3*256) bytes;
 * host matrices are dense (leading dimension = column count). */
size_t fpsk_probe_host_workspace_bytes(int64_t m, int64_t k, int64_t n);
fpsk_status fpsk_probe_host(const void *hA, const void *hB, const float *hC,
                            int64_t m, int64_t k, int64_t n, fpsk_dtype dtype,
                            const fpsk_params *p, void *workspace, size_t ws_bytes,
                            void *stream, fpsk_probe_result *h_result);

/* The probe without caller-provided scratch.  (No counterpart in the paper: this is a
 * deployment convenience of this library.)
 *
 * For callers that cannot allocate device memory where they verify a GEMM - inside a
 * stream-capture region, on a latency-critical or fault-handling path that must not enter the
 * allocator, or in a plug-in that is handed tensors but owns no memory pool - the scratch
 * that fpsk_probe takes as `workspace` lives in a fixed array of
 * FPSK_PROBE_STATIC_SCRATCH_BYTES inside the library (held by every GPU that loads the
 * library, until the process exits).  Arguments and results are those of fpsk_probe, minus
 * the workspace; A, B, C and the outputs are still the caller's device buffers.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - Shapes whose scratch would not fit (fpsk_probe_workspace_bytes(m,k,n) >
 *     FPSK_PROBE_STATIC_SCRATCH_BYTES) are refused with FPSK_ERR_WORKSPACE; nothing is launched.
 *     12 MiB covers every shape up to 16384 x 16384 x 16384.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     call re-zeroes the words that must start at zero.  Two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them. */
#define FPSK_PROBE_STATIC_SCRATCH_BYTES (12u << 20)
fpsk_status fpsk_probe_static(const void *A, int64_t lda, const void *B, int64_t ldb,
                              const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                              fpsk_dtype dtype, int c_is_fp32, const fpsk_params *p, void *stream,
                              fpsk_probe_result *d_result, float *d_residual);

/* ---- the paper's own probe: S alone, B side cached ------------------------------------------ */

/* Host-side record of a cached B side (Section "Implementation": the sketch of the B side is
 * cached and keyed on tensor identity and version, so an in-place optimizer update invalidates
 * it).  Zero-initialise it once (valid = 0); fpsk_probe_hashed fills and checks it.  The key is
 * (B pointer, ldb, b_version, shape, dtype, seed, round, n_buckets, cache pointer, layout of B).
 * The record only says what was ENQUEUED: the (re)build runs asynchronously on the stream of the call
 * that missed, so a cache and its record belong to one stream (or to streams the caller orders after
 * that call). */
typedef struct {
    const void *B;
    void *cache;
    int64_t ldb, m, k, n;
    uint64_t seed, version;
    int32_t dtype, n_buckets, round;
    int32_t valid;        /* 0: nothing cached                                                 */
    int32_t rebuilds;     /* how many times the B side was (re)built through this record       */
    int32_t b_transposed; /* set by the caller before the first call: 0 = the B pointer is B (k x n, row-major);
                             1 = it is W = B^T (n x k, row-major, ldb >= k), the x W^T weight layout  */
    int32_t built_transposed; /* layout the cached B side was built from (part of the key; library-written) */
    int32_t reserved;
} fpsk_bside;

/* State of a probe across calls; see "what the probe keeps between calls" below. */
typedef struct {
    uint32_t calls;             /* probes accumulated since the reset                              */
    uint32_t clean_calls;       /* those that reported clean                                       */
    uint32_t fired_any;         /* OR of the verdicts since the reset                              */
    uint32_t first_fired_call;  /* 1-based index of the first dirty call since the reset, 0 = none */
    double sigma_sum;           /* sum of sigma_hat over the clean calls                           */
    double reserved;
} fpsk_probe_state;

/* Bytes of device memory for the cached B side (hash tables and bucket-sorted permutations of
 * rows and columns, Q = B H2^T as k x n_buckets FP32, max|B|) and for the per-call workspace
 * (P = H1 A, H1 C, split-K partials, S).  0 on bad arguments. */
size_t fpsk_probe_hashed_cache_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets);
size_t fpsk_probe_hashed_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets);

/* 1 when `side` already holds the B side for exactly this key (the call would read A and C only),
 * else 0.  Host only. */
int32_t fpsk_bside_matches(const fpsk_bside *side, const void *B, int64_t ldb, uint64_t b_version,
                           int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed,
                           int32_t round, int32_t n_buckets, const void *cache);

/* The S only probe (Section "The Cheap S Only Probe"): S = (H1 A)(B H2^T) - H1 C H2^T for hash
 * round `round` of `seed` at n_buckets buckets per side, sigma_hat = 1.2533 mean(min(|S|, 5 mean|S|))
 * over the n_buckets^2 buckets, thr = min(tau, mu sqrt(2 ln n_buckets^2) sigma_hat) (Section "Thresholds";
 * p->scale_cap = 1 widens the cap to tau sqrt(m n / n_buckets^2)), dirty iff max|S| > thr or S is not finite.
 *   B, ldb        B itself, or, with side->b_transposed = 1, the weight W = B^T as n x k row-major
 *                 (C = A W^T); only the (re)build of the B side reads it
 *   side, cache   the B side.  When `side` does not match the key (see fpsk_bside), it is rebuilt
 *                 into `cache` first (reads B once; side->rebuilds is incremented); on a match B
 *                 is not read: the call reads 2mk + 4mn bytes.  Bump b_version after every in-place
 *                 change of B.
 *   workspace     per-call scratch; its first 256 bytes must be zero before the first call
 *                 (fpsk_probe_init does that) and again after a result with status FPSK_ERR_TIMEOUT
 *   d_result      device; argmax_col holds the flat bucket index a * n_buckets + b
 *   d_S           device, n_buckets^2 floats receiving S, or NULL
 *   d_state       device, accumulated into by the last kernel of the call, or NULL
 * sigma_hat is the noise at this bucket count and feeds fpsk_plan directly.
 * Launches on a matching B side: three kernels (stream of A and C, contraction, combine and verdict).  With
 * p->tensor_cores = 1, n_buckets <= 256, A and C aligned to 16 bytes and k % 8 == 0, n % 4 == 0, lda % 8 == 0,
 * ldc % 4 == 0: one cooperative kernel (A streams first and leaves as FP16 planes scaled per bucket and column
 * segment, the first CTAs contract them with the cached planes of B H2^T on the tensor cores while the others
 * stream C, then all combine); S then differs from the three-kernel form by the rounding of the contraction only.
 * Asynchronous on `stream`, no host synchronisation; deterministic (bit-identical from call to call in either form). */
fpsk_status fpsk_probe_hashed(fpsk_bside *side, const void *A, int64_t lda, const void *B, int64_t ldb,
                              uint64_t b_version, const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                              fpsk_dtype dtype, int c_is_fp32, uint64_t seed, int32_t round, int32_t n_buckets,
                              const fpsk_params *p, void *cache, size_t cache_bytes, void *workspace,
                              size_t ws_bytes, void *stream, fpsk_probe_result *d_result, float *d_S,
                              fpsk_probe_state *d_state);

/* ---- what the probe keeps between calls ------------------------------------------------------ */

/* fpsk_probe_state (declared above, device memory, 32 bytes): the probe averages sigma_hat over the
 * calls it reports clean without a host synchronisation, and accumulates the verdicts into one flag,
 * so that a caller synchronises once per step instead of once per GEMM (Section "Calibration",
 * "Recalibrating the probe"; Section "Implementation").  fpsk_probe_hashed updates it inside its
 * last kernel when d_state is not NULL; fpsk_probe_accumulate does the same for the result of any
 * probe of this library (one single-thread kernel).  Updates are plain read-modify-writes: the calls
 * that share a state must be ordered on one stream.  Everything here can be captured into a CUDA
 * graph (first call of each entry point outside the capture) and replayed. */
fpsk_status fpsk_probe_state_reset(fpsk_probe_state *d_state, void *stream);
fpsk_status fpsk_probe_accumulate(const fpsk_probe_result *d_result, fpsk_probe_state *d_state, void *stream);

/* Cadence of the recalibration: 1 when `calls` is 16 or a later multiple of 1024 ("after 16 calls
 * and then every 1024"), else 0.  Host only. */
int32_t fpsk_recalibration_due(uint32_t calls);

/* m' = max(m_comb, 16, min(ceil(n_buckets B1 / B*), m_max)) with B1 = max(m, n) sigma_bar / rms_c, and
 * whether m' lies outside [n_buckets / 1.25, 1.25 n_buckets] (then the caller rebuilds its hashes,
 * buffers, caches and graphs at m').  sigma_bar = sigma_sum / clean_calls of a state read back by
 * the caller.  A sigma_bar or rms_c that is not a positive finite number leaves n_buckets unchanged.
 * Host only; outputs are host pointers. */
fpsk_status fpsk_probe_recalibrate(int64_t m, int64_t n, double sigma_bar, double rms_c, int32_t n_buckets,
                                   const fpsk_params *p, int32_t *m_new, int32_t *rebuild);

/* ---- hashed moment sketches --------------------------------------------------------------- */

/* Hash round `round` of `seed` (Section "Moment Sketches": h1, v1 for side 0 = rows,
 * h2, v2 for side 1 = columns): d_bucket[idx] in [0, n_buckets), d_sign[idx] = +1 or -1,
 * idx = 0..count-1.  Device outputs, asynchronous. */
fpsk_status fpsk_hash_tables(uint64_t seed, int32_t round, int32_t side, int64_t count,
                             int32_t n_buckets, int32_t *d_bucket, int32_t *d_sign, void *stream);

/* Bytes of device workspace for fpsk_sketches / fpsk_measure_noise / fpsk_localize with these parameters
 * (0 for a bad shape, bad parameters or a bucket count out of range).  Covers, with tensor_cores = 1 and at least
 * 384 buckets, the FP16 planes of the compressed operands, and, with b_transposed = 0, room for W = B^T
 * (n x k rounded up to 8, 16-bit): fpsk_localize transposes B into it once per call and runs its rounds on W. */
size_t fpsk_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets, const fpsk_params *p);

/* Largest bucket count the kernels accept for this shape (shared-memory limits). */
int32_t fpsk_max_buckets(int64_t m, int64_t k, int64_t n);

/* Sum and first-moment sketches of E = AB - C for one hash round (Eq. (S) and the weighted
 * forms R, T of Section "Moment Sketches"), from compressed operands
 * (H1 A)(B H2^T) - H1 C H2^T, without forming AB.  d_S, d_R, d_T: device, n_buckets^2 floats
 * each, row-major [a][b]; d_R and d_T may both be NULL for the S-only form.  p (NULL = defaults) selects the
 * contraction (p->tensor_cores, effective from 384 buckets) and the layout of B (p->b_transposed), as in
 * fpsk_localize; the workspace is the one fpsk_workspace_bytes sizes for these parameters.  Asynchronous. */
fpsk_status fpsk_sketches(const void *A, int64_t lda, const void *B, int64_t ldb,
                          const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                          fpsk_dtype dtype, uint64_t seed, int32_t round, int32_t n_buckets,
                          const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream,
                          float *d_S, float *d_R, float *d_T);

/* Run-time noise measurement on a (clean) product: S of round 0 at m0 buckets (m0 <= 0: the
 * law's starting count), both noise estimates, the strided clipped rms of C, the normalized
 * constant and the plan (Section "Calibration" and "Recalibrating the probe").
 * h_out is a host pointer; the call synchronises `stream`. */
fpsk_status fpsk_measure_noise(const void *A, int64_t lda, const void *B, int64_t ldb,
                               const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                               fpsk_dtype dtype, uint64_t seed, int32_t m0, const fpsk_params *p,
                               void *workspace, size_t ws_bytes, void *stream, fpsk_noise *h_out);

/* Localization (Algorithm 2 lines "Localize"; Algorithm 1 per round): p->rounds fresh hash
 * rounds at n_buckets, peeling confirmed faults across rounds, candidates from moment ratios
 * (Eq. (recover)), each confirmed by an FP64 recomputation of its inner product over the
 * (2r+1)^2 window, so no clean entry is ever reported (Lemma 1).
 *   n_buckets  bucket count m_loc used verbatim
 *   p->radius  search radius, or -1 to derive it from sigma_MAD of the first round's S
 *   h_faults   host array of `capacity` records, sorted by (i, j) on return
 *   h_count    host, number of faults found (may exceed capacity with FPSK_ERR_CAPACITY)
 * The call synchronises `stream` once per round. */
fpsk_status fpsk_localize(const void *A, int64_t lda, const void *B, int64_t ldb,
                          const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                          fpsk_dtype dtype, uint64_t seed, int32_t n_buckets, const fpsk_params *p,
                          void *workspace, size_t ws_bytes, void *stream,
                          fpsk_fault *h_faults, int32_t capacity, int32_t *h_count);

/* ---- Algorithm 2 complete: verify, localize, repair in place ------------------------------ */

typedef struct {
    int32_t state;        /* 0: clean (only the probe ran); 1: repaired, the second probe is clean;
                             2: the second probe still fires - the caller must recompute C = AB */
    int32_t n_faults;     /* faults found (absolute ones included)                              */
    int32_t n_absolute;   /* entries found by the exact scan (not finite, or |C_ij| > fp32max/16) */
    int32_t m_loc;        /* bucket count localization ran at                                   */
    int32_t radius;       /* search radius it used                                              */
    int32_t reserved;
    fpsk_probe_result first_probe, second_probe;
} fpsk_repair_report;

/* Bytes of workspace for fpsk_verify_repair (n_buckets <= 0: sized for any plan). */
size_t fpsk_repair_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets, const fpsk_params *p);

/* Algorithm 2: probe; on a dirty product the exact scan for entries that are not finite or
 * larger than fp32max/16 (at most K, recomputed as absolute values; C holds the recomputed
 * values while the sketches are built and gets them back afterwards - Section "Nonfinite and
 * Out of Range Entries"), the plan from the noise measured on this call (sigma_MAD of a fresh S
 * at the law's bucket count and the strided rms of C; n_buckets > 0 skips the plan), k rounds
 * of Algorithm 1, then Apply: C_ij <- delta for the absolute entries, C_ij <- C_ij + delta for
 * the others, and a second probe.  C is MODIFIED in place (device, m x n FP32).
 * Faults come back sorted by (i, j); absolute entries have round = -1, bucket_a = bucket_b = -1
 * and delta = recompute = the repaired value.  Host outputs; the call synchronises `stream`. */
fpsk_status fpsk_verify_repair(const void *A, int64_t lda, const void *B, int64_t ldb, float *C, int64_t ldc,
                               int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed,
                               int32_t n_buckets, const fpsk_params *p, void *workspace, size_t ws_bytes,
                               void *stream, fpsk_fault *h_faults, int32_t capacity,
                               fpsk_repair_report *h_report);

/* The Apply step alone (Algorithm 2, "Apply"): writes a fault list into C.  Entries with
 * round < 0 are absolute (C_ij <- delta), the others corrections (C_ij <- C_ij + delta).
 * h_faults is a host array; workspace needs 256 KiB; at most 4096 entries per call. */
fpsk_status fpsk_apply_corrections(float *C, int64_t ldc, int64_t m, int64_t n, const fpsk_fault *h_faults,
                                   int32_t count, void *workspace, size_t ws_bytes, void *stream);

/* ---- caller-owned host resources ------------------------------------------------------------
 * fpsk_measure_noise, fpsk_localize and fpsk_verify_repair need, besides the device workspace, three auxiliary
 * non-blocking streams, ten events and about 16 KB of pinned host memory (their results come back through it).
 * A caller that wants to own them (no creation inside those calls, release at a time of its choosing) creates a
 * context on the device it will run on, puts it into fpsk_params.context and destroys it when no call that uses
 * it is in flight.  A context serves one call at a time.  With context = NULL the library creates one such set
 * per concurrent call and device on first use and keeps it for the life of the process.  (The paper has no
 * counterpart: its engine runs under a framework that owns streams and staging memory.) */
typedef struct fpsk_context fpsk_context;
fpsk_status fpsk_context_create(fpsk_context **out);
fpsk_status fpsk_context_destroy(fpsk_context *ctx);

#ifdef __cplusplus
}
#endif
#endif /* FPSK_H */
