// Internal interfaces between the sketch builder, the selection / confirmation kernels and
// the C ABI layer.
#pragma once
#include "fpsk_common.cuh"

namespace fpsk {

struct PeelEntry {          // a confirmed fault as the peeling kernel needs it
    int i, j;
    double delta;
};

struct SketchPlan {
    int kpad;      // n2 rounded up to 16: K extent of the contraction
    int npad;      // m_b rounded up to 4: leading dimension of Q, Qw
    int nsplit;    // row splits per bucket row in the C scatter
    int ksplit;    // K splits of the contraction
    int kchunk;    // K extent per split (multiple of 16)
    int tile;      // 64 or 128
};

// Two more streams and the events that tie them to the caller's stream: the parts of a sketch build that do
// not depend on each other (row side + A compression, column side + B compression, C scatter) run side by
// side, and the C scatter hides under the contraction.  Created on first use, kept for the life of the process,
// one set per concurrent call and device.
struct SketchAux {
    int device = -1;
    cudaStream_t s1 = nullptr, s2 = nullptr;
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    // localization: the tail of a round (selection, decode, confirmation) runs on s3 behind the event of the
    // round's sketch build, beside the next round's build on the caller's stream
    cudaStream_t s3 = nullptr;
    cudaEvent_t evb[3] = {nullptr, nullptr, nullptr};       // build of prepared round q is complete
    cudaEvent_t evt = nullptr;                              // the tails are complete
};
fpsk_status sketch_aux_create(SketchAux &a);     // streams and events on the current device (a.device is set)
bool sketch_aux_destroy(SketchAux &a);
struct SketchAuxLease {          // returns the set to the pool when it goes out of scope (unless it is borrowed from a context)
    SketchAux *aux = nullptr;
    bool borrowed = false;
    ~SketchAuxLease();
};
extern std::atomic<unsigned long long> g_lazy_resources;      // stream sets and pinned buffers the library created by itself
fpsk_status sketch_aux_acquire(SketchAuxLease &lease);
struct SketchWs;
// host side only: point w at the tables of round rnd when they were prepared ahead (prepare_hash_rounds)
bool sketch_select_round(SketchWs &w, uint64_t seed, int rnd);

constexpr int kHashSets = 3;     // hash rounds whose tables can be prepared ahead in one batch
struct HashSet {                 // the tables of one hash round
    int *h1, *v1, *h2, *v2;
    uint32_t *rowperm, *colperm, *colpos;
    int *rowcount, *rowstart, *colcount, *colstart;
};
struct SketchWs {
    SketchPlan pl;
    SketchAux *aux;              // nullptr: everything on the caller's stream
    HashSet sets[kHashSets];
    int prepared_first, prepared_count;      // rounds whose tables sit in sets[0 .. prepared_count) (host side)
    unsigned long long prepared_seed;
    // the tables of the round in progress (one of the sets)
    int *h1, *v1, *h2, *v2;
    uint32_t *rowperm, *colperm;
    uint32_t *colpos;            // inverse of colperm: position (and sign) of every column in the bucket-sorted order
    int *rowcount, *rowstart, *colcount, *colstart;
    float *P, *Pw, *Q, *Qw, *partAB, *partC;
    bool tc;                     // split-BF16 tensor-core contraction
    int tc_ksplit;
    unsigned char *planes[4];    // P, Pw, Q^T, Qw^T as tiled FP16 planes (hi, lo)
    unsigned int *tc_err;        // set by the contraction when a wait gave up
    unsigned int *sc_ctrl;       // ring scatter: [0] unit counter, [1] set when a bounded wait gave up
    float *tc_scale;             // [0], [1]: powers of two that bring P, Pw and Q, Qw into FP16 range (device)
    const float *d_maxab;        // [0] max|A|, [1] max|B| (device; set by the caller before a tensor-core build)
};

struct SketchIn {
    const void *A, *B;
    const float *C;
    long long n1, n2, n3, lda, ldb, ldc;
    int bt = 0;      // 1: B points to W = B^T (n3 x n2, row-major, leading dimension ldb)
};

void sketch_plan(long long n1, long long n2, long long n3, int m_b, SketchPlan &pl);
size_t sketch_ws_bytes(long long n1, long long n2, long long n3, int m_b, bool tc = false);
bool sketch_carve(void *ws, size_t ws_bytes, long long n1, long long n2, long long n3, int m_b, SketchWs &w, bool tc = false);
int sketch_max_buckets(long long n1, long long n2, long long n3);

fpsk_status build_hash_side(uint64_t seed, int rnd, int side, int n, int m_b, int *bucket, int *sign,
                            int *count, int *start, uint32_t *perm, cudaStream_t st, uint32_t *pos = nullptr);
// W = B^T for 16-bit elements: W[j * ldw + k] = B[k * ldb + j], k < n2, j < n3 (ldw >= n2)
fpsk_status transpose_b_launch(const void *B, long long ldb, long long n2, long long n3, void *W, long long ldw,
                               cudaStream_t st);
// Hash tables and bucket-sorted permutations of rounds first .. first + count - 1 (count <= kHashSets), both sides, in
// three batched launches; build_sketches then finds them ready.
fpsk_status prepare_hash_rounds(uint64_t seed, int first, int count, long long n1, long long n3, int m_b, SketchWs &w,
                                cudaStream_t st);
fpsk_status build_sketches(const SketchIn &in, fpsk_dtype dtype, uint64_t seed, int rnd, int m_b, bool mom,
                           SketchWs &w, cudaStream_t st, float *S, float *R, float *T);
// start[0..n] = exclusive prefix sums of count[0..n)  (one CTA, any n)
fpsk_status exclusive_scan_launch(const int *count, int n, int *start, cudaStream_t st);
// one FP32 contraction part[ks] = P[:, ks-th K chunk] Q[ks-th K chunk, :]  (M x K by K x N, K a multiple of 16)
fpsk_status contraction_launch(const float *P, const float *Q, float *part, int M, int N, int K, int lda, int ldb,
                               int ksplit, int kchunk, int tile, cudaStream_t st);
// Q = B H2^T (kpad x npad, rows >= n2 zero) from the bucket-sorted column permutation
fpsk_status build_b_side(const void *B, long long ldb, long long n2, long long n3, fpsk_dtype dtype, int m_b, int kpad,
                         int npad, const uint32_t *colperm, const int *colstart, float *Q, cudaStream_t st);
fpsk_status peel_launch(const PeelEntry *dF, int nF, uint64_t seed, int rnd, long long n1, long long n3, int m_b,
                        float *S, float *R, float *T, cudaStream_t st,
                        const int *d_nF = nullptr);      // d_nF: the count is read on the device instead (nF is ignored)

// ---- selection (select.cu) -----------------------------------------------------------------
struct Candidate {          // one decoded bucket of the set U (Algorithm 1)
    int flat;               // a*m_b + b
    int ih, jh;             // rounded 0-based coordinate estimate
    float s_abs;
};

struct SelectWs {           // all device memory
    unsigned int *hist;     // histograms of the radix select (digits x two jobs x copies x 256 bins) + control words
    unsigned int *err;      // nonzero after a bounded grid-wide wait of a select gave up (the host reads it)
    unsigned long long *state;   // radix-select state
    float *scal;            // scalar results: [0] median, [1] sigma_mad, [2] mean|S|, [3] sigma_clip,
                            //                 [4] thr, [5] tau_c, [6] tau_d
    float *partial;         // per-CTA partial sums
    unsigned long long *keys;    // selected keys (<= kmax)
    int *counts;            // [0] valid samples of C, [1] collected, [2] n_U
    Candidate *cand;        // <= kmax
    float *Rc, *Tc;         // first moments of the collected keys' buckets (slot order of `keys`)
    bool hist_clean;        // host side: the histogram has been zeroed since this workspace was carved
};
constexpr int kSelMaxK = 1024;
size_t select_ws_bytes();
void select_carve(void *ws, SelectWs &w);

// clipped-mean estimate 1.2533 mean(min(|S|, 5 mean|S|)) -> scal[3]
fpsk_status sigma_clip_launch(const float *S, long long mm, SelectWs &w, cudaStream_t st);
// thresholds from scal[1] and tau, K largest |S| above max(tau_c, tau_d), decoded candidates.
// mad_mode >= 0: sigma_MAD of S (1: of |S|, 0: signed) is computed in the same launches first.
// the two halves of select_candidates_launch, for a caller that computes the moments of the collected keys in between
fpsk_status select_collect_launch(const float *S, int m_b, long long n1, long long n3, const float *d_tau, int radius, int K,
                                  int mad_mode, SelectWs &w, cudaStream_t st);
fpsk_status decode_launch(const float *S, const float *R, const float *T, const float *Rc, const float *Tc, long long n1,
                          long long n3, SelectWs &w, cudaStream_t st, int *zero_word = nullptr);   // zero_word: a counter cleared by the launch (the next confirmation's hits)
fpsk_status select_candidates_launch(const float *S, const float *R, const float *T, int m_b, long long n1,
                                     long long n3, const float *d_tau, int radius, int K, int mad_mode, SelectWs &w,
                                     cudaStream_t st);
// device max |X| of a half matrix -> out[0] (float)
fpsk_status max_abs_half_launch(const void *X, long long ld, long long rows, long long cols, fpsk_dtype dtype,
                                float *out, unsigned int *scratch, cudaStream_t st);
// sigma_MAD of S (mad_of_abs: of |S| as printed, else signed) -> scal[1], median -> scal[0]; and the strided,
// clipped rms of C (Section "Calibration") -> out[0]; the three medians share one launch
long long rms_c_samples(const float *C, long long ldc, long long n1, long long n3, float *samples, SelectWs &w,
                        cudaStream_t st);          // the samples alone (count -> w.counts[0]); returns how many, < 0 on a launch error
fpsk_status sigma_mad_rms_c_select_launch(const float *S, long long mm, int mad_of_abs, float *samples, long long nsamp,
                                          SelectWs &w, float *out, cudaStream_t st);      // the selects and the rms on samples taken before
fpsk_status sigma_mad_rms_c_launch(const float *S, long long mm, int mad_of_abs, const float *C, long long ldc,
                                   long long n1, long long n3, float *samples, SelectWs &w, float *out, cudaStream_t st);

// ---- confirmation (confirm.cu) ---------------------------------------------------------------
struct Hit {                // an accepted window entry
    int cand;               // index into the candidate list
    int di, dj;             // offset from the candidate's estimate
    int i, j;
    float c_value;
    double gamma;           // FP64 recomputation
};
// A confirmed fault as the device keeps it over the rounds of a localization (Algorithm 1's set F).
struct DevFault {
    int i, j;
    double gamma;           // FP64 recomputation
    float c_value;          // the delivered C_ij
    int round;              // hash round that found it; < 0: an absolute repair handed in by the caller (never peeled)
    int flat;               // its bucket a * m_b + b in that round
    int pad;
};
static_assert(sizeof(DevFault) == 32, "DevFault is 32 bytes");
// Replay of Algorithm 1's ordered search over a round's hits, on the device (one CTA): the hits sorted by offset
// (Chebyshev, Manhattan, d_i, d_j) and then by candidate; a bucket leaves U at its first accepted entry; an entry
// already in F is skipped.  Accepted entries are appended to F (count in rstate[0]) and, when their error is finite,
// to the peel list (count in rstate[1]); rstate[2] is set when a list overflowed (hits, F).
fpsk_status replay_launch(const Hit *hits, const int *n_hits, int hit_cap, const Candidate *cand, const int *n_cand, int K,
                          int radius, int round, DevFault *F, int f_cap, PeelEntry *peel, int *rstate, cudaStream_t st);
// force != 0: report every in-range window entry, whatever its test says
// R, T of Eq. (recover) for the collected keys only (w.keys, count w.counts[1]) -> w.Rc, w.Tc: per key, the dot
// products of the bucket's compressed rows of A and columns of B, the bucket's entries of C, and the peeled faults
// that fall into the bucket.  Uses the hash tables of the round held in `sk`.
fpsk_status candidate_moments_launch(const SketchIn &in, fpsk_dtype dtype, const SketchWs &sk, int m_b, int K, SelectWs &sel,
                                     const PeelEntry *d_peel, const int *d_n_peel, uint64_t seed, int rnd, cudaStream_t st);
fpsk_status confirm_launch(const SketchIn &in, fpsk_dtype dtype, const Candidate *cand, const int *n_cand,
                           int max_cand, int radius, double c_valid, int force, Hit *hits, int *n_hits, int hit_cap,
                           cudaStream_t st, bool hits_cleared = false);      // hits_cleared: *n_hits was zeroed by an earlier launch on st

// ---- scan / patch / apply (repair.cu) ----------------------------------------------------------
constexpr int kRepairCap = 4096;      // entries one call can scan out, patch or apply
struct ScanEntry {
    int i, j;
};
enum { PATCH_SET = 0, PATCH_ADD = 1, PATCH_SET_BITS = 2 };
struct PatchEntry {
    int i, j;
    int mode;          // PATCH_SET: C_ij = value; PATCH_ADD: C_ij += value; PATCH_SET_BITS: raw float bits in value
    double value;
};
size_t repair_scratch_bytes();
fpsk_status scan_launch(const float *C, long long ldc, long long n1, long long n3, int cap, void *scratch, cudaStream_t st,
                        ScanEntry *h_entries, int *h_count);
fpsk_status recompute_entries(const SketchIn &in, fpsk_dtype dtype, const ScanEntry *h_entries, int n, void *scratch,
                              cudaStream_t st, double *h_gamma, float *h_old);
fpsk_status patch_launch(float *C, long long ldc, const PatchEntry *d_entries, int n, cudaStream_t st);

// ---- split-precision tensor-core contraction (tc_contract.cu) -------------------------------------
// bytes of the three tiled BF16 planes of a rows x kk FP32 matrix
size_t tc_planes_bytes(int rows, int kk);
// planes of X(r, k) = src[r * ldr + k * ldk], tiled for the A side (b_side = 0) or the B side (1) of the contraction
fpsk_status tc_split_launch(const float *src, const float *d_scale, long long ldr, long long ldk, int rows, int kk, int b_side, unsigned char *planes,
                            cudaStream_t st);
// part[ks][prob] = A_selA[prob] (M x K) times B_selB[prob] (N x K) transposed, over the ks-th range of K
fpsk_status tc_contract_launch(const unsigned char *const *planesA, const unsigned char *const *planesB, const int *selA,
                               const int *selB, int nprob, int pstride, float *part, int M, int N, int K, int ksplit,
                               unsigned int *d_err, cudaStream_t st);
int tc_plan_ksplit(int M, int N, int K, int nprob, int sms);
constexpr int kTcPlanes = 2;            // FP16 terms per FP32 value (hi, lo)
// The power of two that brings the bucket sums of one side into FP16 range: |sum| <= (largest bucket) x max|X|
// is scaled below 2^14 (FP16 reaches 65504).  Exact to undo; elements more than 2^16 below the largest
// lose bits of their lo term, an absolute error below 2^-39 of the largest.
__device__ __forceinline__ float tc_scale_of(int max_count, float max_abs)
{
    if (!(max_abs > 0.f && max_abs <= 3.4028234663852886e38f) || max_count < 1) return 1.f;
    // max_abs < 2^(ilogb + 1), max_count < 2^(bits of max_count): exponents only, so nothing overflows here
    int e = 14 - (ilogbf(max_abs) + 1 + (32 - __clz(max_count)));
    e = e > 126 ? 126 : (e < -126 ? -126 : e);
    return ldexpf(1.f, e);
}
// scale[0] = tc_scale_of(max of count[0..m_b), maxv[0])   (all device)
fpsk_status tc_scale_launch(const int *count, int m_b, const float *maxv, float *scale, cudaStream_t st);
constexpr int kTcMinBuckets = 384;      // below this the FP32 FMA contraction is the faster one (measured)

// ---- the S only probe with a cached B side (hprobe.cu) ------------------------------------------
size_t hprobe_cache_bytes(long long n1, long long n2, long long n3, int m);
size_t hprobe_ws_bytes(long long n1, long long n2, long long n3, int m);
fpsk_status hprobe_prepare(const void *B, long long ldb, int b_transposed, long long n1, long long n2, long long n3, fpsk_dtype dtype,
                           uint64_t seed, int rnd, int m, void *cache, size_t cache_bytes, cudaStream_t st);
fpsk_status hprobe_launch(const void *A, long long lda, const float *C, long long ldc, long long n1, long long n2,
                          long long n3, fpsk_dtype dtype, int m, double mu, int scale_cap, int tensor_cores, void *cache, size_t cache_bytes, void *ws,
                          size_t ws_bytes, cudaStream_t st, fpsk_probe_result *d_result, float *d_S, fpsk_probe_state *d_state);
fpsk_status probe_accumulate_launch(const fpsk_probe_result *d_result, fpsk_probe_state *d_state, cudaStream_t st);

}  // namespace fpsk
