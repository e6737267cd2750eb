// C ABI of the FP-Sketch verifier: argument checks, workspace carving, the scalar planner
// (Sections "Sketch Noise Sets the Bucket Count" and "Calibration") and the round loop of
// Algorithm 2's localize part with the ordered replay of Algorithm 1's search over the hits.
#include "sketch.cuh"
#include "fpsk_test.h"

#include <math.h>
#include <string.h>
#include <algorithm>
#include <mutex>
#include <vector>

namespace fpsk {
std::atomic<unsigned long long> g_launches{0};
std::atomic<unsigned long long> g_lazy_resources{0};

#ifdef FPSK_DEBUG_BOUNDS
// the bounds records of the source files of the library (each registers its own at load)
struct BoundsSource {
    const char *file;
    cudaError_t (*read)(BoundsRecord *);
    cudaError_t (*clear)();
};
static std::vector<BoundsSource> &bounds_sources()
{
    static std::vector<BoundsSource> *v = new std::vector<BoundsSource>;
    return *v;
}
void bounds_register(const char *file, cudaError_t (*read)(BoundsRecord *), cudaError_t (*clear)())
{
    bounds_sources().push_back(BoundsSource{file, read, clear});
}
#endif

constexpr int kHitCap = 2048;
constexpr int kPeelCap = 4096;

// What the host needs from a localization, gathered on the device so that it is ONE copy at the end of the
// call: header and the first kPackFaults confirmed faults (more: a second copy).
constexpr int kPackFaults = 512;
struct FinalHeader {
    int n_faults, n_peel, truncated;
    unsigned int tc_err, sel_err;
    int pad[11];
};
static_assert(sizeof(FinalHeader) == 64, "FinalHeader is 64 bytes");
constexpr size_t kPackBytes = sizeof(FinalHeader) + (size_t)kPackFaults * sizeof(DevFault);

__global__ void pack_final_kernel(const int *rstate, const unsigned int *tc_err, const unsigned int *sc_err, const unsigned int *sel_err,
                                  const DevFault *F, unsigned char *pack)
{
    FinalHeader *h = reinterpret_cast<FinalHeader *>(pack);
    DevFault *pf = reinterpret_cast<DevFault *>(pack + sizeof(FinalHeader));
    const int nf = rstate[0];
    if (threadIdx.x == 0) {
        h->n_faults = nf;
        h->n_peel = rstate[1];
        h->truncated = rstate[2];
        h->tc_err = (tc_err ? *tc_err : 0u) | (sc_err ? *sc_err : 0u);
        h->sel_err = *sel_err;
    }
    const int np = nf < kPackFaults ? nf : kPackFaults;
    for (int t = threadIdx.x; t < np; t += blockDim.x) pf[t] = F[t];
}

// Pinned host staging for the results.  A pageable destination makes cudaMemcpyAsync block the host until the copy
// has run.  Buffers are created on
// first use (one per concurrent call) and kept for the life of the process.
struct PinnedPool {
    std::mutex mu;
    std::vector<void *> free_list;      // each kPackBytes
};
static PinnedPool &pinned_pool()
{
    static PinnedPool *p = new PinnedPool;      // never destroyed: no CUDA calls at process exit
    return *p;
}
struct PinnedLease {
    void *p = nullptr;
    bool borrowed = false;      // the buffer of a caller's context: not returned to the pool
    ~PinnedLease()
    {
        if (!p || borrowed) return;
        PinnedPool &pool = pinned_pool();
        std::lock_guard<std::mutex> g(pool.mu);
        pool.free_list.push_back(p);
    }
};
static fpsk_status pinned_acquire(PinnedLease &l)
{
    PinnedPool &pool = pinned_pool();
    {
        std::lock_guard<std::mutex> g(pool.mu);
        if (!pool.free_list.empty()) {
            l.p = pool.free_list.back();
            pool.free_list.pop_back();
            return FPSK_OK;
        }
    }
    g_lazy_resources.fetch_add(1, std::memory_order_relaxed);
    FPSK_CUDA_OK(cudaHostAlloc(&l.p, kPackBytes, cudaHostAllocPortable));
    return FPSK_OK;
}

}  // namespace fpsk

// What a caller's context holds: the host-side resources of one call at a time.
struct fpsk_context {
    fpsk::SketchAux aux;
    void *pinned = nullptr;           // kPackBytes
    cudaEvent_t round_done = nullptr;
};

namespace fpsk {

// The host-side resources of one call: from the caller's context when it passed one (nothing is created),
// else leased from the library's own pools (created on first use).
struct HostRes {
    SketchAuxLease aux;
    PinnedLease pin;
    cudaEvent_t round_done = nullptr;
    bool own_event = false;
    ~HostRes() { if (own_event && round_done) cudaEventDestroy(round_done); }
    fpsk_status acquire(const fpsk_params &q, bool need_event)
    {
        if (q.context) {
            fpsk_context *c = static_cast<fpsk_context *>(q.context);
            int dev = 0;
            FPSK_CUDA_OK(cudaGetDevice(&dev));
            if (c->aux.device != dev) return FPSK_ERR_PARAM;       // a context belongs to the device it was created on
            aux.aux = &c->aux; aux.borrowed = true;
            pin.p = c->pinned; pin.borrowed = true;
            round_done = c->round_done;
            return FPSK_OK;
        }
        fpsk_status rc = sketch_aux_acquire(aux);
        if (rc != FPSK_OK) return rc;
        rc = pinned_acquire(pin);
        if (rc != FPSK_OK) return rc;
        if (need_event) {
            FPSK_CUDA_OK(cudaEventCreateWithFlags(&round_done, cudaEventDisableTiming));
            own_event = true;
        }
        return FPSK_OK;
    }
    // Error exits: whatever was queued on the auxiliary streams and on the caller's stream is complete before
    // the call returns, as the header promises for every return.
    void drain(cudaStream_t st) const
    {
        if (aux.aux) {
            if (aux.aux->s1) cudaStreamSynchronize(aux.aux->s1);
            if (aux.aux->s2) cudaStreamSynchronize(aux.aux->s2);
            if (aux.aux->s3) cudaStreamSynchronize(aux.aux->s3);
        }
        cudaStreamSynchronize(st);
    }
};

// ---------------------------------------------------------------- scalar planner
static double cf_of(fpsk_dtype d) { return d == FPSK_BF16 ? 0.19 : 1.76 * 0.19; }

static double law_sigma(double n1, double n2, double n3, fpsk_dtype d, double rms, double m)
{
    return cf_of(d) * ldexp(1.0, -24) * sqrt(n1 * n3 * n2) * pow(n2 / 8192.0, 0.07) * rms / m;
}
static int m_comb_of(const fpsk_params &p)
{
    return (int)ceil(std::max(3.0 * p.c_coll * p.delta_max, sqrt(3.0 * p.c_coll * p.s_budget)));
}
static long long isqrt_ll(long long x)
{
    long long r = (long long)sqrt((double)x);
    while (r * r > x) --r;
    while ((r + 1) * (r + 1) <= x) ++r;
    return r;
}
static int m_max_of(long long n1, long long n3) { return (int)std::max(16LL, isqrt_ll((n1 * n3) / 16)); }
static int m_mem_of(long long n2)
{
    const long long lim = (1LL << 31) / 4;     // 3 m^2 + 6 m n2 <= lim
    long long m = (long long)((-6.0 * n2 + sqrt(36.0 * (double)n2 * n2 + 12.0 * lim)) / 6.0);
    while (3 * (m + 1) * (m + 1) + 6 * (m + 1) * n2 <= lim) ++m;
    while (m > 0 && 3 * m * m + 6 * m * n2 > lim) --m;
    return (int)std::min(m, 1LL << 30);
}
static int m_start_of(long long n1, long long n2, long long n3, fpsk_dtype d, const fpsk_params &p)
{
    const double x = (double)std::max(n1, n3) / p.b_star * law_sigma((double)n1, (double)n2, (double)n3, d, 1.0, 1.0);
    const double mnum = ceil(x);
    const int mc = m_comb_of(p);
    const double lo = std::max({(double)mc, mnum, 16.0});
    const double hi = (double)std::max(mc, m_max_of(n1, n3));
    return (int)std::min(lo, hi);
}
static int radius_of_budget(double B) { return B <= 0.05 ? 0 : std::max(2, (int)ceil(2.5 * B)); }

static void plan_of(long long n1, long long n2, long long n3, fpsk_dtype d, double sigma, double rms, int m_cur,
                    const fpsk_params &p, int &m_loc, int &radius, double &Bout)
{
    const bool ok = std::isfinite(sigma) && sigma > 0 && std::isfinite(rms) && rms > 0;
    if (!ok) {
        sigma = law_sigma((double)n1, (double)n2, (double)n3, d, 1.0, (double)m_cur);
        rms = 1.0;
    }
    const double B = (double)std::max(n1, n3) * sigma / (p.rho_min * rms);
    Bout = B;
    const int rB = radius_of_budget(B);
    if (rB <= p.r_star) {
        m_loc = m_cur;
        radius = rB;
        return;
    }
    const double grown = 16.0 * ceil(ceil((double)m_cur * rB / p.r_star) / 16.0);
    const double capped = std::min({grown, (double)m_max_of(n1, n3), (double)m_mem_of(n2)});
    m_loc = (int)std::max((double)m_cur, capped);
    const double Bp = B * m_cur / m_loc;
    radius = Bp <= 0.05 ? 0 : std::min(p.r_max, std::max(2, (int)ceil(2.5 * Bp)));
}

static bool params_ok(const fpsk_params &p)
{
    return p.rounds >= 1 && p.rounds <= 8 && p.r_star >= 0 && p.r_max >= 0 && p.r_max <= 16 && p.radius >= -1 &&
           p.radius <= 16 && p.s_budget >= 1 && p.delta_max >= 1 && p.rho_min > 0 && p.c_valid > 0 && p.mu > 0 &&
           p.b_star > 0 && p.c_coll > 1.0 - 1e-12 && (p.b_transposed == 0 || p.b_transposed == 1) &&
           (p.scale_cap == 0 || p.scale_cap == 1);
}

static fpsk_params resolve_params(const fpsk_params *p)
{
    fpsk_params q;
    if (p) q = *p;
    else fpsk_default_params(&q);
    return q;
}

static fpsk_status check_mats(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C, int64_t ldc,
                              int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, bool b_transposed = false)
{
    if (!A || !B || !C) return FPSK_ERR_NULL;
    if (dtype != FPSK_FP16 && dtype != FPSK_BF16) return FPSK_ERR_DTYPE;
    if (m < 1 || k < 1 || n < 1 || lda < k || ldb < (b_transposed ? k : n) || ldc < n) return FPSK_ERR_SHAPE;
    if (m >= (1LL << 30) || k >= (1LL << 30) || n >= (1LL << 30)) return FPSK_ERR_SHAPE;
    return FPSK_OK;
}

// ---------------------------------------------------------------- localize workspace
struct LocWs {
    SketchWs sk;
    float *S;                 // the sum sketch of the round (R, T exist only at the kept buckets: SelectWs::Rc, Tc)
    float *Sr[kHashSets];     // one S per round prepared ahead (Sr[0] == S): their builds run before the tails
    SelectWs sel;
    float *samples;
    float *misc;              // [0] max|A| [1] max|B| [2] tau [3] rms_c ; [8..] uint scratch
    PeelEntry *peel;          // confirmed finite faults, as the peeling needs them (device list, kPeelCap)
    DevFault *dfaults;        // Algorithm 1's set F on the device (kPeelCap)
    int *rstate;              // [0] faults in F, [1] entries of the peel list, [2] a list overflowed
    Hit *hits;
    int *n_hits;
    unsigned char *pack;      // kPackBytes: the call's results in one piece
    unsigned short *Wt;       // room for W = B^T (n3 x ldw) when B comes as k x n, else null
    long long ldw;
};

static size_t loc_ws_bytes(long long n1, long long n2, long long n3, int m_b, bool tc = false, bool wt = false)
{
    const size_t mm = (size_t)m_b * m_b;
    size_t b = sketch_ws_bytes(n1, n2, n3, m_b, tc);
    b += kHashSets * align_up(mm * 4, 256);
    b += align_up(select_ws_bytes(), 256);
    b += align_up((size_t)131072 * 4, 256);
    b += 256;
    b += align_up(sizeof(PeelEntry) * kPeelCap, 256);
    b += align_up(sizeof(DevFault) * kPeelCap, 256) + 256;
    b += align_up(sizeof(Hit) * kHitCap, 256);
    b += 256;
    b += align_up(kPackBytes, 256);
    if (wt) b += align_up((size_t)n3 * (size_t)((n2 + 7) & ~7LL) * 2, 256);
    return b;
}

static bool loc_carve(void *ws, size_t ws_bytes, long long n1, long long n2, long long n3, int m_b, LocWs &w, bool tc = false,
                      bool wt = false)
{
    if (ws_bytes < loc_ws_bytes(n1, n2, n3, m_b, tc, wt)) return false;
    const size_t mm = (size_t)m_b * m_b;
    const size_t skb = sketch_ws_bytes(n1, n2, n3, m_b, tc);
    if (!sketch_carve(ws, skb, n1, n2, n3, m_b, w.sk, tc)) return false;
    char *p = static_cast<char *>(ws) + skb;
    auto take = [&](size_t bytes) { void *r = p; p += align_up(bytes, 256); return r; };
    for (int q = 0; q < kHashSets; ++q) w.Sr[q] = (float *)take(mm * 4);
    w.S = w.Sr[0];
    select_carve(take(select_ws_bytes()), w.sel);
    w.samples = (float *)take((size_t)131072 * 4);
    w.misc = (float *)take(256);
    w.peel = (PeelEntry *)take(sizeof(PeelEntry) * kPeelCap);
    w.dfaults = (DevFault *)take(sizeof(DevFault) * kPeelCap);
    w.rstate = (int *)take(256);
    w.hits = (Hit *)take(sizeof(Hit) * kHitCap);
    w.n_hits = (int *)take(256);
    w.pack = (unsigned char *)take(kPackBytes);
    w.ldw = (n2 + 7) & ~7LL;
    w.Wt = wt ? (unsigned short *)take((size_t)n3 * (size_t)w.ldw * 2) : nullptr;
    return true;
}

// max|A| -> misc[0], max|B| -> misc[1] (device); the tensor-core contraction scales its planes by them
static fpsk_status loc_max_ab(const SketchIn &in, fpsk_dtype dtype, LocWs &w, cudaStream_t st)
{
    unsigned int *uscr = reinterpret_cast<unsigned int *>(w.misc + 8);
    fpsk_status rc = max_abs_half_launch(in.A, in.lda, in.n1, in.n2, dtype, w.misc + 0, uscr, st);
    if (rc != FPSK_OK) return rc;
    rc = in.bt ? max_abs_half_launch(in.B, in.ldb, in.n3, in.n2, dtype, w.misc + 1, uscr + 1, st)
               : max_abs_half_launch(in.B, in.ldb, in.n2, in.n3, dtype, w.misc + 1, uscr + 1, st);
    if (rc != FPSK_OK) return rc;
    w.sk.d_maxab = w.misc;
    return FPSK_OK;
}

// The scalars of a noise measurement (the select's eight scalars, rms(C), the select's error word) to the host
// through pinned staging: three small asynchronous copies and one wait (a pageable destination blocks per copy).
static fpsk_status read_noise_scalars(const LocWs &w, cudaStream_t st, float (&h_scal)[8], float &h_rms, void *pinned)
{
    char *h = static_cast<char *>(pinned);
    FPSK_CUDA_OK(cudaMemcpyAsync(h, w.sel.scal, 32, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(h + 32, w.misc + 3, 4, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(h + 36, w.sel.err, 4, cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    memcpy(h_scal, h, 32);
    memcpy(&h_rms, h + 32, 4);
    unsigned int err = 0;
    memcpy(&err, h + 36, 4);
    return err ? FPSK_ERR_TIMEOUT : FPSK_OK;
}

__global__ void tau_kernel(float *misc, float n2)
{
    if (threadIdx.x == 0) misc[2] = 100.f * n2 * 1.1920928955078125e-07f * misc[0] * misc[1];
}

// The localize part of Algorithm 2: p.rounds rounds of Algorithm 1 at m_b buckets, carrying F.
// Entries already in F with round < 0 are absolute repairs (Section "Nonfinite"): they count as
// found but are not peeled, their error is already absent from the sketches.
static fpsk_status localize_rounds(const SketchIn &in_caller, fpsk_dtype dtype, uint64_t seed, int m_b, const fpsk_params &q, LocWs &w,
                                   cudaStream_t st, HostRes &hr, std::vector<fpsk_fault> &F, bool &truncated, int &radius_used)
{
    SketchIn in = in_caller;
    const long long m = in.n1, k = in.n2, n = in.n3;
    const long long mm = (long long)m_b * m_b;
    const int K = std::min(std::max(64, 8 * q.s_budget), kSelMaxK);
    fpsk_status rc;
    SketchAuxLease &aux = hr.aux;
    w.sk.aux = aux.aux;
    // Once per call, side by side: max|A| and the hash tables of all rounds (they depend on the seed only) on the
    // caller's stream; max|B| and, for B given as k x n, its transpose on an auxiliary stream.  With W = B^T every round
    // reads rows of W: the B compression sums rows instead of gathering columns, the confirmation reads a row instead
    // of a strided column; same bits.
    SketchAux *ax = (aux.aux && aux.aux->s1 && aux.aux->s2 && aux.aux->ev[4]) ? aux.aux : nullptr;
    cudaStream_t sB0 = ax ? ax->s1 : st;
    unsigned int *uscr = reinterpret_cast<unsigned int *>(w.misc + 8);
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[0], st));             // whatever the caller queued before this call
        FPSK_CUDA_OK(cudaStreamWaitEvent(sB0, ax->ev[0], 0));
    }
    rc = max_abs_half_launch(in.A, in.lda, m, k, dtype, w.misc + 0, uscr, st);
    if (rc != FPSK_OK) return rc;
    rc = in.bt ? max_abs_half_launch(in.B, in.ldb, n, k, dtype, w.misc + 1, uscr + 1, sB0)
               : max_abs_half_launch(in.B, in.ldb, k, n, dtype, w.misc + 1, uscr + 1, sB0);
    if (rc != FPSK_OK) return rc;
    w.sk.d_maxab = w.misc;
    if (!in.bt && w.Wt) {
        rc = transpose_b_launch(in.B, in.ldb, k, n, w.Wt, w.ldw, sB0);
        if (rc != FPSK_OK) return rc;
        in.B = w.Wt;
        in.ldb = w.ldw;
        in.bt = 1;
    }
    rc = prepare_hash_rounds(seed, 0, std::min(q.rounds, (int)kHashSets), m, n, m_b, w.sk, st);
    if (rc != FPSK_OK) return rc;
    if (ax) {
        FPSK_CUDA_OK(cudaEventRecord(ax->ev[1], sB0));
        FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->ev[1], 0));
    }
    // tau = 100 n2 eps max|A| max|B| (device scalar misc[2])
    tau_kernel<<<1, 32, 0, st>>>(w.misc, (float)k);
    FPSK_LAUNCH_CHECK();

    int radius = q.radius;
    bool round0_built = false;
    if (radius < 0) {
        // no calibration handed in: sigma_MAD of the first round's S and the strided rms of C
        rc = build_sketches(in, dtype, seed, 0, m_b, false, w.sk, st, w.S, nullptr, nullptr);
        if (rc != FPSK_OK) return rc;
        round0_built = true;
        rc = sigma_mad_rms_c_launch(w.S, mm, q.mad_of_abs, in.C, in.ldc, m, n, w.samples, w.sel, w.misc + 3, st);
        if (rc != FPSK_OK) return rc;
        float h_scal[8], h_rms = 0.f;
        rc = read_noise_scalars(w, st, h_scal, h_rms, hr.pin.p);
        if (rc != FPSK_OK) return rc;
        double sig = h_scal[1], rms = h_rms;
        if (!(std::isfinite(sig) && sig > 0 && std::isfinite(rms) && rms > 0)) {
            sig = law_sigma((double)m, (double)k, (double)n, dtype, 1.0, (double)m_b);
            rms = 1.0;
        }
        radius = std::min(q.r_max, radius_of_budget((double)std::max(m, n) * sig / (q.rho_min * rms)));
    }
    radius_used = radius;

    PinnedLease &stage = hr.pin;
    // The sketches of a round do not depend on what earlier rounds find (only the peeling does; Section "Peeling
    // Across Hash Rounds"), and the tail of a round (peel, selection, moments of the kept buckets, decode,
    // confirmation, ordered search) touches none of a build's buffers but its S.  So the builds of all rounds whose
    // tables were prepared ahead are queued at once on the caller's stream, each into an S of its own, and every tail
    // runs on the auxiliary stream s3 behind its build's event: the GPU runs round t's tail beside round t + 1's
    // build.  The set F and the peel list live on the device (the ordered search of Algorithm 1 over a round's hits
    // is a one-CTA kernel), so the rounds chain on the stream and the host reads ONE packed result at the end of the
    // call.  Without auxiliary streams everything runs on the caller's stream in order.
    struct { cudaEvent_t e; } round_done{hr.round_done};
    // Only S is built whole.  The first moments R, T are read at the K buckets the selection keeps and nowhere else
    // (Eq. (recover)), so they are computed for those buckets alone once the keys are collected: a third of the
    // contraction, of the combine and of the plane writes.
    const bool overlap = ax && ax->s3 && ax->evb[0] && ax->evb[1] && ax->evb[2] && ax->evt;
    cudaStream_t ts = overlap ? ax->s3 : st;
    const int nprep = w.sk.prepared_count > 0 ? std::min(q.rounds, w.sk.prepared_count) : 0;
    // F as the caller hands it in (absolute repairs: found, never peeled) goes to the device first
    const int n_fixed = (int)std::min<size_t>(F.size(), kPeelCap);
    if ((int)F.size() > kPeelCap) truncated = true;
    std::vector<DevFault> fixed((size_t)n_fixed);
    for (int f = 0; f < n_fixed; ++f) {
        DevFault d;
        d.i = F[f].i; d.j = F[f].j; d.gamma = F[f].recompute; d.c_value = F[f].c_value; d.round = F[f].round; d.flat = -1; d.pad = 0;
        fixed[f] = d;
    }
    {
        // through the pinned staging (read again only at the end of the call, behind these copies in stream order),
        // so that nothing here waits for the device
        const int init[4] = {n_fixed, 0, 0, 0};
        const bool fits = sizeof(init) + sizeof(DevFault) * (size_t)n_fixed <= kPackBytes;
        char *hp = static_cast<char *>(stage.p);
        if (fits) {
            memcpy(hp, init, sizeof(init));
            if (n_fixed) memcpy(hp + sizeof(init), fixed.data(), sizeof(DevFault) * (size_t)n_fixed);
        }
        FPSK_CUDA_OK(cudaMemcpyAsync(w.rstate, fits ? (const void *)hp : (const void *)init, sizeof(init), cudaMemcpyHostToDevice, st));
        if (n_fixed)
            FPSK_CUDA_OK(cudaMemcpyAsync(w.dfaults, fits ? (const void *)(hp + sizeof(init)) : (const void *)fixed.data(),
                                         sizeof(DevFault) * (size_t)n_fixed, cudaMemcpyHostToDevice, st));
        if (!fits) FPSK_CUDA_OK(cudaStreamSynchronize(st));      // pageable sources are read by the copies until here
    }
    if (overlap) {
        if (round0_built) FPSK_CUDA_OK(cudaEventRecord(ax->evb[0], st));
        for (int t = round0_built ? 1 : 0; t < nprep; ++t) {
            rc = build_sketches(in, dtype, seed, t, m_b, false, w.sk, st, w.Sr[t], nullptr, nullptr);
            if (rc != FPSK_OK) return rc;
            FPSK_CUDA_OK(cudaEventRecord(ax->evb[t], st));
        }
    }
    for (int t = 0; t < q.rounds; ++t) {
        float *S = w.S;
        if (overlap) {
            if (t < nprep || (t == 0 && round0_built)) {
                S = w.Sr[t];
                FPSK_CUDA_OK(cudaStreamWaitEvent(ts, ax->evb[t], 0));
            } else {
                // a round beyond the prepared ones: its tables replace those of set 0, whose round must be finished
                FPSK_CUDA_OK(cudaEventRecord(ax->evt, ts));
                FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->evt, 0));
                rc = build_sketches(in, dtype, seed, t, m_b, false, w.sk, st, w.S, nullptr, nullptr);
                if (rc != FPSK_OK) return rc;
                FPSK_CUDA_OK(cudaEventRecord(ax->evb[0], st));
                FPSK_CUDA_OK(cudaStreamWaitEvent(ts, ax->evb[0], 0));
            }
            sketch_select_round(w.sk, seed, t);        // host side: the tables the kept buckets' moments are taken from
        } else if (!(t == 0 && round0_built)) {
            rc = build_sketches(in, dtype, seed, t, m_b, false, w.sk, st, w.S, nullptr, nullptr);
            if (rc != FPSK_OK) return rc;
        }
        if (t > 0) {
            rc = peel_launch(w.peel, 0, seed, t, m, n, m_b, S, nullptr, nullptr, ts, w.rstate + 1);
            if (rc != FPSK_OK) return rc;
        }
        // sigma_MAD of this round's S rides in the launches of the K-largest selection (round 0's is already
        // there when it was needed for the radius)
        const int mad_mode = (t == 0 && round0_built) ? -1 : (q.mad_of_abs ? 1 : 0);
        rc = select_collect_launch(S, m_b, m, n, w.misc + 2, radius, K, mad_mode, w.sel, ts);
        if (rc != FPSK_OK) return rc;
        rc = candidate_moments_launch(in, dtype, w.sk, m_b, K, w.sel, w.peel, w.rstate + 1, seed, t, ts);
        if (rc != FPSK_OK) return rc;
        rc = decode_launch(S, nullptr, nullptr, w.sel.Rc, w.sel.Tc, m, n, w.sel, ts, w.n_hits);
        if (rc != FPSK_OK) return rc;
        rc = confirm_launch(in, dtype, w.sel.cand, w.sel.counts + 2, K, radius, q.c_valid, 0, w.hits, w.n_hits, kHitCap, ts, true);
        if (rc != FPSK_OK) return rc;
        rc = replay_launch(w.hits, w.n_hits, kHitCap, w.sel.cand, w.sel.counts + 2, K, radius, t, w.dfaults, kPeelCap, w.peel,
                           w.rstate, ts);
        if (rc != FPSK_OK) return rc;
    }
    // ---- the one read of the call: header and the first kPackFaults faults
    pack_final_kernel<<<1, 256, 0, ts>>>(w.rstate, w.sk.tc ? w.sk.tc_err : nullptr, w.sk.sc_ctrl + 1, w.sel.err, w.dfaults, w.pack);
    FPSK_LAUNCH_CHECK();
    FPSK_CUDA_OK(cudaMemcpyAsync(stage.p, w.pack, kPackBytes, cudaMemcpyDeviceToHost, ts));
    FPSK_CUDA_OK(cudaEventRecord(round_done.e, ts));
    if (overlap) {
        // the caller's stream continues behind the last tail
        FPSK_CUDA_OK(cudaEventRecord(ax->evt, ts));
        FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->evt, 0));
    }
    FPSK_CUDA_OK(cudaEventSynchronize(round_done.e));
    const FinalHeader *hdr = static_cast<const FinalHeader *>(stage.p);
    if (hdr->tc_err || hdr->sel_err) return FPSK_ERR_TIMEOUT;        // a bounded wait (contraction, selects) gave up
    if (hdr->truncated) truncated = true;
    const int nF = std::min(hdr->n_faults, (int)kPeelCap);
    std::vector<DevFault> all((size_t)std::max(nF, 0));
    const DevFault *packed = reinterpret_cast<const DevFault *>(static_cast<const char *>(stage.p) + sizeof(FinalHeader));
    std::copy(packed, packed + std::min(nF, (int)kPackFaults), all.begin());
    if (nF > kPackFaults) {
        // more faults than travel with the header: fetch the rest of the list
        FPSK_CUDA_OK(cudaMemcpyAsync(all.data() + kPackFaults, w.dfaults + kPackFaults, sizeof(DevFault) * (size_t)(nF - kPackFaults),
                                     cudaMemcpyDeviceToHost, ts));
        FPSK_CUDA_OK(cudaStreamSynchronize(ts));
    }
    for (int f = n_fixed; f < nF; ++f) {
        const DevFault &d = all[f];
        fpsk_fault o;
        memset(&o, 0, sizeof(o));
        o.i = d.i; o.j = d.j;
        o.recompute = d.gamma;
        o.c_value = d.c_value;
        o.delta = d.gamma - (double)d.c_value;
        o.round = d.round;
        o.bucket_a = d.flat / m_b;
        o.bucket_b = d.flat % m_b;
        F.push_back(o);
    }
    return FPSK_OK;
}

static fpsk_status localize_core(const SketchIn &in, fpsk_dtype dtype, uint64_t seed, int m_b, const fpsk_params &q, LocWs &w,
                                 cudaStream_t st, HostRes &hr, std::vector<fpsk_fault> &F, bool &truncated, int &radius_used)
{
    const fpsk_status rc = localize_rounds(in, dtype, seed, m_b, q, w, st, hr, F, truncated, radius_used);
    // an error may leave a round's sketch build queued on the auxiliary streams: finish it before returning
    if (rc != FPSK_OK) hr.drain(st);
    return rc;
}

// Waits, with a short limit, for a flag that the caller leaves at zero: the wait gives up, the kernel
// reports FPSK_ERR_TIMEOUT in the result and returns normally, like every bounded wait of the library
// does after its (much longer) limit.
__global__ void selftest_wait_kernel(const unsigned int *flag, fpsk_probe_result *result)
{
    if (threadIdx.x != 0) return;
    const bool arrived = bounded_wait_ge(flag, 1u, 2048u);        // about half a millisecond
    fpsk_probe_result r;
    r.fired = 0; r.nonfinite = 0; r.argmax_col = -1;
    r.status = arrived ? (int)FPSK_OK : (int)FPSK_ERR_TIMEOUT;
    r.max_abs = 0.f; r.sigma_hat = 0.f; r.thr = 0.f; r.tau = 0.f;
    *result = r;
}

}  // namespace fpsk

using namespace fpsk;

extern "C" {

const char *fpsk_status_string(fpsk_status s)
{
    switch (s) {
    case FPSK_OK: return "ok";
    case FPSK_ERR_NULL: return "null pointer";
    case FPSK_ERR_SHAPE: return "bad shape or leading dimension";
    case FPSK_ERR_DTYPE: return "bad operand type, or C is not FP32";
    case FPSK_ERR_ALIGN: return "workspace not 256-byte aligned";
    case FPSK_ERR_WORKSPACE: return "workspace too small";
    case FPSK_ERR_BUCKETS: return "bucket count out of range";
    case FPSK_ERR_CAPACITY: return "list truncated";
    case FPSK_ERR_CUDA: return "CUDA error";
    case FPSK_ERR_TIMEOUT: return "bounded device wait gave up";
    case FPSK_ERR_PARAM: return "parameter out of range";
    }
    return "unknown";
}

void fpsk_default_params(fpsk_params *p)
{
    if (!p) return;
    memset(p, 0, sizeof(*p));
    p->rounds = 3; p->r_star = 4; p->r_max = 16; p->radius = -1;
    p->s_budget = 8; p->delta_max = 8; p->mad_of_abs = 1;
    p->rho_min = 0.02; p->c_valid = 100.0; p->mu = 4.0; p->b_star = 0.3; p->c_coll = 2.0;
}

int32_t fpsk_law_m_start(int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, const fpsk_params *p)
{
    const fpsk_params q = resolve_params(p);
    if (m < 1 || k < 1 || n < 1 || (dtype != FPSK_FP16 && dtype != FPSK_BF16) || !params_ok(q)) return -1;
    return m_start_of(m, k, n, dtype, q);
}

fpsk_status fpsk_plan(int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, double sigma_hat, double rms_c,
                      int32_t m_cur, const fpsk_params *p, int32_t *m_loc, int32_t *radius, double *index_budget)
{
    if (!m_loc || !radius) return FPSK_ERR_NULL;
    const fpsk_params q = resolve_params(p);
    if (m < 1 || k < 1 || n < 1 || m_cur < 1) return FPSK_ERR_SHAPE;
    if (dtype != FPSK_FP16 && dtype != FPSK_BF16) return FPSK_ERR_DTYPE;
    if (!params_ok(q)) return FPSK_ERR_PARAM;
    int ml, r;
    double B;
    plan_of(m, k, n, dtype, sigma_hat, rms_c, m_cur, q, ml, r, B);
    *m_loc = ml;
    *radius = r;
    if (index_budget) *index_budget = B;
    return FPSK_OK;
}

// ---------------------------------------------------------------- probe
size_t fpsk_probe_workspace_bytes(int64_t m, int64_t k, int64_t n) { return probe_ws_bytes(m, k, n); }

fpsk_status fpsk_probe_init(void *workspace, size_t ws_bytes, void *stream)
{
    if (!workspace) return FPSK_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    if (ws_bytes < 256) return FPSK_ERR_WORKSPACE;
    FPSK_CUDA_OK(cudaMemsetAsync(workspace, 0, 256, static_cast<cudaStream_t>(stream)));
    return FPSK_OK;
}

fpsk_status fpsk_probe(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C, int64_t ldc,
                       int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, int c_is_fp32, const fpsk_params *p,
                       void *workspace, size_t ws_bytes, void *stream, fpsk_probe_result *d_result,
                       float *d_residual)
{
    if (!c_is_fp32) return FPSK_ERR_DTYPE;      // a narrowed C is rejected, not tolerated
    fpsk_status rc = check_mats(A, lda, B, ldb, C, ldc, m, k, n, dtype);
    if (rc != FPSK_OK) return rc;
    if (!workspace || !d_result) return FPSK_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q) || q.b_transposed) return FPSK_ERR_PARAM;      // this probe streams B as k x n
    ProbeDims d{m, k, n, lda, ldb, ldc};
    return probe_launch(A, B, C, d, dtype, q.mu, workspace, ws_bytes, static_cast<cudaStream_t>(stream), d_result,
                        d_residual);
}

size_t fpsk_probe_host_workspace_bytes(int64_t m, int64_t k, int64_t n)
{
    const size_t base = probe_ws_bytes(m, k, n);
    if (!base) return 0;
    return align_up(base, 256) + align_up((size_t)m * k * 2, 256) + align_up((size_t)k * n * 2, 256) +
           align_up((size_t)m * n * 4, 256) + 256;
}

fpsk_status fpsk_probe_host(const void *hA, const void *hB, const float *hC, int64_t m, int64_t k, int64_t n,
                            fpsk_dtype dtype, const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream,
                            fpsk_probe_result *h_result)
{
    fpsk_status rc = check_mats(hA, k, hB, n, hC, n, m, k, n, dtype);
    if (rc != FPSK_OK) return rc;
    if (!workspace || !h_result) return FPSK_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    if (ws_bytes < fpsk_probe_host_workspace_bytes(m, k, n)) return FPSK_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *w = static_cast<char *>(workspace);
    const size_t base = align_up(probe_ws_bytes(m, k, n), 256);
    char *dA = w + base;
    char *dB = dA + align_up((size_t)m * k * 2, 256);
    char *dC = dB + align_up((size_t)k * n * 2, 256);
    char *dres = dC + align_up((size_t)m * n * 4, 256);
    FPSK_CUDA_OK(cudaMemcpyAsync(dA, hA, (size_t)m * k * 2, cudaMemcpyHostToDevice, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(dB, hB, (size_t)k * n * 2, cudaMemcpyHostToDevice, st));
    FPSK_CUDA_OK(cudaMemcpyAsync(dC, hC, (size_t)m * n * 4, cudaMemcpyHostToDevice, st));
    rc = fpsk_probe(dA, k, dB, n, reinterpret_cast<const float *>(dC), n, m, k, n, dtype, 1, p, workspace, base, stream,
                    reinterpret_cast<fpsk_probe_result *>(dres), nullptr);
    if (rc != FPSK_OK) return rc;
    FPSK_CUDA_OK(cudaMemcpyAsync(h_result, dres, sizeof(fpsk_probe_result), cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    return (fpsk_status)h_result->status;
}

// ---------------------------------------------------------------- sketches
// ---------------------------------------------------------------- S only probe, cached B side
size_t fpsk_probe_hashed_cache_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets)
{
    if (m < 1 || k < 1 || n < 1 || n_buckets < 1 || n_buckets > 4096) return 0;
    if (m >= (1LL << 30) || k >= (1LL << 30) || n >= (1LL << 30)) return 0;
    return hprobe_cache_bytes(m, k, n, n_buckets);
}

size_t fpsk_probe_hashed_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets)
{
    if (m < 1 || k < 1 || n < 1 || n_buckets < 1 || n_buckets > 4096) return 0;
    if (m >= (1LL << 30) || k >= (1LL << 30) || n >= (1LL << 30)) return 0;
    return hprobe_ws_bytes(m, k, n, n_buckets);
}

int32_t fpsk_bside_matches(const fpsk_bside *side, const void *B, int64_t ldb, uint64_t b_version, int64_t m,
                           int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed, int32_t round, int32_t n_buckets,
                           const void *cache)
{
    if (!side || !side->valid) return 0;
    return side->B == B && side->cache == cache && side->ldb == ldb && side->version == b_version && side->m == m &&
                   side->k == k && side->n == n && side->dtype == (int32_t)dtype && side->seed == seed &&
                   side->round == round && side->n_buckets == n_buckets
               ? 1 : 0;
}

fpsk_status fpsk_probe_hashed(fpsk_bside *side, const void *A, int64_t lda, const void *B, int64_t ldb,
                              uint64_t b_version, const float *C, int64_t ldc, int64_t m, int64_t k, int64_t n,
                              fpsk_dtype dtype, int c_is_fp32, uint64_t seed, int32_t round, int32_t n_buckets,
                              const fpsk_params *p, void *cache, size_t cache_bytes, void *workspace, size_t ws_bytes,
                              void *stream, fpsk_probe_result *d_result, float *d_S, fpsk_probe_state *d_state)
{
    if (!c_is_fp32) return FPSK_ERR_DTYPE;      // a narrowed C is rejected, not tolerated
    if (!side || !cache || !workspace || !d_result) return FPSK_ERR_NULL;
    const bool bt = side->b_transposed != 0;
    fpsk_status rc = check_mats(A, lda, B, bt ? n : ldb, C, ldc, m, k, n, dtype);      // W is n x k: its own check below
    if (rc != FPSK_OK) return rc;
    if (bt && ldb < k) return FPSK_ERR_SHAPE;
    if (n_buckets < 1 || n_buckets > 4096 || round < 0) return FPSK_ERR_BUCKETS;
    if ((reinterpret_cast<uintptr_t>(cache) & 255) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return FPSK_ERR_ALIGN;
    if (cache_bytes < hprobe_cache_bytes(m, k, n, n_buckets) || ws_bytes < hprobe_ws_bytes(m, k, n, n_buckets))
        return FPSK_ERR_WORKSPACE;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return FPSK_ERR_PARAM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (side->valid && side->built_transposed != side->b_transposed) side->valid = 0;      // the layout is part of the key
    if (!fpsk_bside_matches(side, B, ldb, b_version, m, k, n, dtype, seed, round, n_buckets, cache)) {
        side->valid = 0;
        rc = hprobe_prepare(B, ldb, bt ? 1 : 0, m, k, n, dtype, seed, round, n_buckets, cache, cache_bytes, st);
        if (rc != FPSK_OK) return rc;
        side->B = B; side->cache = cache; side->ldb = ldb; side->m = m; side->k = k; side->n = n;
        side->seed = seed; side->version = b_version; side->dtype = (int32_t)dtype; side->n_buckets = n_buckets;
        side->round = round; side->built_transposed = side->b_transposed; side->valid = 1; side->rebuilds += 1;
    }
    return hprobe_launch(A, lda, C, ldc, m, k, n, dtype, n_buckets, q.mu, q.scale_cap, q.tensor_cores, cache, cache_bytes, workspace, ws_bytes, st,
                         d_result, d_S, d_state);
}

// ---------------------------------------------------------------- give-up path of the device-side waits
fpsk_status fpsk_selftest_bounded_wait(uint32_t *d_flag, fpsk_probe_result *d_result, void *stream)
{
    if (!d_flag || !d_result) return FPSK_ERR_NULL;
    selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d_flag, d_result);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- stateful probe
fpsk_status fpsk_probe_state_reset(fpsk_probe_state *d_state, void *stream)
{
    if (!d_state) return FPSK_ERR_NULL;
    FPSK_CUDA_OK(cudaMemsetAsync(d_state, 0, sizeof(fpsk_probe_state), static_cast<cudaStream_t>(stream)));
    return FPSK_OK;
}

fpsk_status fpsk_probe_accumulate(const fpsk_probe_result *d_result, fpsk_probe_state *d_state, void *stream)
{
    if (!d_result || !d_state) return FPSK_ERR_NULL;
    return probe_accumulate_launch(d_result, d_state, static_cast<cudaStream_t>(stream));
}

int32_t fpsk_recalibration_due(uint32_t calls) { return (calls == 16u || (calls > 16u && calls % 1024u == 0u)) ? 1 : 0; }

fpsk_status fpsk_probe_recalibrate(int64_t m, int64_t n, double sigma_bar, double rms_c, int32_t n_buckets,
                                   const fpsk_params *p, int32_t *m_new, int32_t *rebuild)
{
    if (!m_new || !rebuild) return FPSK_ERR_NULL;
    if (m < 1 || n < 1) return FPSK_ERR_SHAPE;
    if (n_buckets < 1) return FPSK_ERR_BUCKETS;
    const fpsk_params q = resolve_params(p);
    *m_new = n_buckets;
    *rebuild = 0;
    if (!(std::isfinite(sigma_bar) && sigma_bar > 0 && std::isfinite(rms_c) && rms_c > 0)) return FPSK_OK;
    const double B1 = (double)std::max(m, n) * sigma_bar / rms_c;
    const double grown = std::min(ceil(n_buckets * B1 / q.b_star), (double)m_max_of(m, n));
    const int mn = (int)std::max({(double)m_comb_of(q), 16.0, grown});
    *m_new = mn;
    *rebuild = ((double)mn < n_buckets / 1.25 || (double)mn > 1.25 * n_buckets) ? 1 : 0;
    return FPSK_OK;
}

fpsk_status fpsk_hash_tables(uint64_t seed, int32_t round, int32_t side, int64_t count, int32_t n_buckets,
                             int32_t *d_bucket, int32_t *d_sign, void *stream)
{
    if (!d_bucket || !d_sign) return FPSK_ERR_NULL;
    if (count < 1 || count >= (1LL << 30)) return FPSK_ERR_SHAPE;
    if (n_buckets < 1) return FPSK_ERR_BUCKETS;
    if (round < 0 || side < 0 || side > 1) return FPSK_ERR_PARAM;
    return build_hash_side(seed, round, side, (int)count, n_buckets, d_bucket, d_sign, nullptr, nullptr, nullptr,
                           static_cast<cudaStream_t>(stream));
}

int32_t fpsk_max_buckets(int64_t m, int64_t k, int64_t n)
{
    if (m < 1 || k < 1 || n < 1) return 0;
    return sketch_max_buckets(m, k, n);
}

size_t fpsk_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets, const fpsk_params *p)
{
    if (m < 1 || k < 1 || n < 1) return 0;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return 0;
    // n_buckets <= 0: size for the law's starting count of either operand type
    if (n_buckets <= 0) n_buckets = std::max(m_start_of(m, k, n, FPSK_FP16, q), m_start_of(m, k, n, FPSK_BF16, q));
    if (n_buckets > sketch_max_buckets(m, k, n)) return 0;
    return loc_ws_bytes(m, k, n, n_buckets, q.tensor_cores != 0, !q.b_transposed);
}

fpsk_status fpsk_sketches(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C, int64_t ldc,
                          int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed, int32_t round,
                          int32_t n_buckets, const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream,
                          float *d_S, float *d_R, float *d_T)
{
    fpsk_status rc = check_mats(A, lda, B, ldb, C, ldc, m, k, n, dtype, p && p->b_transposed);
    if (rc != FPSK_OK) return rc;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return FPSK_ERR_PARAM;
    if (!workspace || !d_S) return FPSK_ERR_NULL;
    if ((d_R == nullptr) != (d_T == nullptr)) return FPSK_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    if (n_buckets < 1 || n_buckets > sketch_max_buckets(m, k, n)) return FPSK_ERR_BUCKETS;
    if (round < 0) return FPSK_ERR_PARAM;
    LocWs w;
    if (!loc_carve(workspace, ws_bytes, m, k, n, n_buckets, w, q.tensor_cores != 0)) return FPSK_ERR_WORKSPACE;
    SketchIn in{A, B, C, m, k, n, lda, ldb, ldc, q.b_transposed};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (w.sk.tc) {      // the tensor-core contraction scales its planes by max|A|, max|B|
        rc = loc_max_ab(in, dtype, w, st);
        if (rc != FPSK_OK) return rc;
    }
    return build_sketches(in, dtype, seed, round, n_buckets, d_R != nullptr, w.sk, st, d_S, d_R, d_T);
}

fpsk_status fpsk_measure_noise(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C, int64_t ldc,
                               int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed, int32_t m0,
                               const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream, fpsk_noise *h_out)
{
    fpsk_status rc = check_mats(A, lda, B, ldb, C, ldc, m, k, n, dtype, p && p->b_transposed);
    if (rc != FPSK_OK) return rc;
    if (!workspace || !h_out) return FPSK_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return FPSK_ERR_PARAM;
    if (m0 <= 0) m0 = m_start_of(m, k, n, dtype, q);
    if (m0 > sketch_max_buckets(m, k, n)) return FPSK_ERR_BUCKETS;
    LocWs w;
    // With the tensor-core contraction the B side is compressed from W = B^T (rows of W are contiguous along k):
    // a B that comes as k x n is transposed into the workspace first, when the workspace has the room that
    // fpsk_workspace_bytes sizes for it.  Same bits as the k x n kernels, a third less time at 16384^3.
    bool own_wt = q.tensor_cores != 0 && !q.b_transposed && loc_carve(workspace, ws_bytes, m, k, n, m0, w, true, true) && w.sk.tc;
    if (!own_wt && !loc_carve(workspace, ws_bytes, m, k, n, m0, w, q.tensor_cores != 0)) return FPSK_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SketchIn in{A, B, C, m, k, n, lda, ldb, ldc, q.b_transposed};
    HostRes hr;
    rc = hr.acquire(q, false);
    if (rc != FPSK_OK) return rc;
    SketchAuxLease &aux = hr.aux;
    w.sk.aux = aux.aux;
    float h_scal[8];
    float h_rms = 0.f;
    // one exit path: an error leaves nothing queued behind the call
    rc = [&]() -> fpsk_status {
        fpsk_status rc;
        if (w.sk.tc) {
            rc = loc_max_ab(in, dtype, w, st);
            if (rc != FPSK_OK) return rc;
        }
        if (own_wt && w.Wt) {
            rc = transpose_b_launch(in.B, in.ldb, k, n, w.Wt, w.ldw, st);
            if (rc != FPSK_OK) return rc;
            in.B = w.Wt;
            in.ldb = w.ldw;
            in.bt = 1;
        }
        // The samples of C need nothing from the sketch: they are taken on the stream that will run the C scatter, ahead of
        // the build (which joins that stream before its combine).  The clipped mean and the selects both only read S:
        // the two sums run on the other auxiliary stream beside the select launch.
        SketchAux *ax = (aux.aux && aux.aux->s1 && aux.aux->s2 && aux.aux->ev[4]) ? aux.aux : nullptr;
        if (ax) {
            FPSK_CUDA_OK(cudaEventRecord(ax->ev[0], st));             // whatever the caller queued before this call (the GEMM, say)
            FPSK_CUDA_OK(cudaStreamWaitEvent(ax->s2, ax->ev[0], 0));
        }
        const long long nsamp = rms_c_samples(C, ldc, m, n, w.samples, w.sel, ax ? ax->s2 : st);
        if (nsamp < 0) return FPSK_ERR_CUDA;
        rc = build_sketches(in, dtype, seed, 0, m0, false, w.sk, st, w.S, nullptr, nullptr);
        if (rc != FPSK_OK) return rc;
        const long long mm = (long long)m0 * m0;
        if (ax) {
            FPSK_CUDA_OK(cudaEventRecord(ax->ev[0], st));
            FPSK_CUDA_OK(cudaStreamWaitEvent(ax->s1, ax->ev[0], 0));
        }
        rc = sigma_clip_launch(w.S, mm, w.sel, ax ? ax->s1 : st);
        if (rc != FPSK_OK) return rc;
        if (ax) FPSK_CUDA_OK(cudaEventRecord(ax->ev[1], ax->s1));
        rc = sigma_mad_rms_c_select_launch(w.S, mm, q.mad_of_abs, w.samples, nsamp, w.sel, w.misc + 3, st);
        if (rc != FPSK_OK) return rc;
        if (ax) FPSK_CUDA_OK(cudaStreamWaitEvent(st, ax->ev[1], 0));
        return read_noise_scalars(w, st, h_scal, h_rms, hr.pin.p);
    }();
    if (rc != FPSK_OK) {
        hr.drain(st);
        return rc;
    }

    fpsk_noise out;
    memset(&out, 0, sizeof(out));
    out.sigma_clip = h_scal[3];
    out.sigma_mad = h_scal[1];
    out.rms_c = h_rms;
    out.m0 = m0;
    const bool rms_ok = std::isfinite(out.rms_c) && out.rms_c > 0;
    out.c_hat = rms_ok ? out.sigma_clip * m0 / (ldexp(1.0, -24) * sqrt((double)m * (double)k * (double)n) * out.rms_c)
                       : nan("");
    int ml, r;
    double B_;
    plan_of(m, k, n, dtype, out.sigma_clip, out.rms_c, m0, q, ml, r, B_);
    out.m_loc = ml;
    out.radius = r;
    out.index_budget_B = B_;
    if (rms_ok && std::isfinite(out.sigma_clip) && out.sigma_clip > 0) {
        const double B1 = (double)std::max(m, n) * out.sigma_clip / out.rms_c;
        const double grown = std::min(ceil(m0 * B1 / q.b_star), (double)m_max_of(m, n));
        out.m_probe = (int)std::max({(double)m_comb_of(q), 16.0, grown});
    } else {
        out.m_probe = m0;
    }
    *h_out = out;
    return FPSK_OK;
}

fpsk_status fpsk_localize(const void *A, int64_t lda, const void *B, int64_t ldb, const float *C, int64_t ldc,
                          int64_t m, int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed, int32_t n_buckets,
                          const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream, fpsk_fault *h_faults,
                          int32_t capacity, int32_t *h_count)
{
    fpsk_status rc = check_mats(A, lda, B, ldb, C, ldc, m, k, n, dtype, p && p->b_transposed);
    if (rc != FPSK_OK) return rc;
    if (!workspace || !h_count || (capacity > 0 && !h_faults)) return FPSK_ERR_NULL;
    if (capacity < 0) return FPSK_ERR_PARAM;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return FPSK_ERR_PARAM;
    if (n_buckets < 1 || n_buckets > sketch_max_buckets(m, k, n)) return FPSK_ERR_BUCKETS;
    LocWs w;
    if (!loc_carve(workspace, ws_bytes, m, k, n, n_buckets, w, q.tensor_cores != 0, !q.b_transposed)) return FPSK_ERR_WORKSPACE;
    SketchIn in{A, B, C, m, k, n, lda, ldb, ldc, q.b_transposed};
    *h_count = 0;
    std::vector<fpsk_fault> F;
    bool truncated = false;
    int radius_used = 0;
    HostRes hr;
    rc = hr.acquire(q, true);
    if (rc != FPSK_OK) return rc;
    rc = localize_core(in, dtype, seed, n_buckets, q, w, static_cast<cudaStream_t>(stream), hr, F, truncated, radius_used);
    if (rc != FPSK_OK) return rc;
    std::sort(F.begin(), F.end(), [](const fpsk_fault &x, const fpsk_fault &y) {
        return x.i != y.i ? x.i < y.i : x.j < y.j;
    });
    *h_count = (int32_t)F.size();
    const int ncopy = std::min<int>((int)F.size(), capacity);
    for (int f = 0; f < ncopy; ++f) h_faults[f] = F[f];
    if ((int)F.size() > capacity || truncated) return FPSK_ERR_CAPACITY;
    return FPSK_OK;
}

// ---------------------------------------------------------------- Algorithm 2, complete
size_t fpsk_repair_workspace_bytes(int64_t m, int64_t k, int64_t n, int32_t n_buckets, const fpsk_params *p)
{
    if (m < 1 || k < 1 || n < 1) return 0;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q)) return 0;
    int mb = n_buckets;
    if (mb <= 0) {   // calibrated on the call: size for the largest count the plan can ask for
        mb = std::max({m_start_of(m, k, n, FPSK_FP16, q), m_start_of(m, k, n, FPSK_BF16, q), m_max_of(m, n)});
        mb = std::min(mb, m_mem_of(k));
        mb = std::min(mb, sketch_max_buckets(m, k, n));
    }
    if (mb < 1 || mb > sketch_max_buckets(m, k, n)) return 0;
    return align_up(probe_ws_bytes(m, k, n), 256) + align_up(loc_ws_bytes(m, k, n, mb, q.tensor_cores != 0, true), 256) +
           align_up(repair_scratch_bytes(), 256) + 256;
}

fpsk_status fpsk_apply_corrections(float *C, int64_t ldc, int64_t m, int64_t n, const fpsk_fault *h_faults,
                                   int32_t count, void *workspace, size_t ws_bytes, void *stream)
{
    if (!C || (count > 0 && !h_faults) || !workspace) return FPSK_ERR_NULL;
    if (m < 1 || n < 1 || ldc < n || count < 0) return FPSK_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    if (count > kRepairCap) return FPSK_ERR_CAPACITY;
    if (ws_bytes < repair_scratch_bytes()) return FPSK_ERR_WORKSPACE;
    for (int f = 0; f < count; ++f)
        if (h_faults[f].i < 0 || h_faults[f].i >= m || h_faults[f].j < 0 || h_faults[f].j >= n) return FPSK_ERR_SHAPE;
    if (count == 0) return FPSK_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<PatchEntry> pe((size_t)count);
    for (int f = 0; f < count; ++f) {
        pe[f].i = h_faults[f].i;
        pe[f].j = h_faults[f].j;
        pe[f].value = h_faults[f].delta;
        pe[f].mode = h_faults[f].round < 0 ? PATCH_SET : PATCH_ADD;     // absolute entries carry the value itself
    }
    PatchEntry *d = static_cast<PatchEntry *>(workspace);
    FPSK_CUDA_OK(cudaMemcpyAsync(d, pe.data(), sizeof(PatchEntry) * count, cudaMemcpyHostToDevice, st));
    fpsk_status rc = patch_launch(C, ldc, d, count, st);
    if (rc != FPSK_OK) return rc;
    FPSK_CUDA_OK(cudaStreamSynchronize(st));      // pe is read by the copy until here
    return FPSK_OK;
}

fpsk_status fpsk_verify_repair(const void *A, int64_t lda, const void *B, int64_t ldb, float *C, int64_t ldc, int64_t m,
                               int64_t k, int64_t n, fpsk_dtype dtype, uint64_t seed, int32_t n_buckets,
                               const fpsk_params *p, void *workspace, size_t ws_bytes, void *stream, fpsk_fault *h_faults,
                               int32_t capacity, fpsk_repair_report *h_report)
{
    fpsk_status rc = check_mats(A, lda, B, ldb, C, ldc, m, k, n, dtype);
    if (rc != FPSK_OK) return rc;
    if (!workspace || !h_report || (capacity > 0 && !h_faults)) return FPSK_ERR_NULL;
    if (capacity < 0) return FPSK_ERR_PARAM;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return FPSK_ERR_ALIGN;
    const fpsk_params q = resolve_params(p);
    if (!params_ok(q) || q.b_transposed) return FPSK_ERR_PARAM;      // the repair path reads B as k x n
    if (n_buckets > sketch_max_buckets(m, k, n)) return FPSK_ERR_BUCKETS;
    if (ws_bytes < fpsk_repair_workspace_bytes(m, k, n, n_buckets, p) || fpsk_repair_workspace_bytes(m, k, n, n_buckets, p) == 0)
        return FPSK_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    memset(h_report, 0, sizeof(*h_report));

    // workspace: [probe | verdict | repair scratch | localize]
    char *wp = static_cast<char *>(workspace);
    void *probe_ws = wp;
    const size_t pws = align_up(probe_ws_bytes(m, k, n), 256);
    fpsk_probe_result *d_res = reinterpret_cast<fpsk_probe_result *>(wp + pws);
    void *rep_ws = wp + pws + 256;
    char *loc_ws = wp + pws + 256 + align_up(repair_scratch_bytes(), 256);
    const size_t loc_bytes = ws_bytes - (size_t)(loc_ws - wp);
    const int K = std::min(std::max(64, 8 * q.s_budget), kSelMaxK);

    // ---- S-only probe (every call)
    FPSK_CUDA_OK(cudaMemsetAsync(probe_ws, 0, 256, st));
    ProbeDims pd{m, k, n, lda, ldb, ldc};
    rc = probe_launch(A, B, C, pd, dtype, q.mu, probe_ws, pws, st, d_res, nullptr);
    if (rc != FPSK_OK) return rc;
    FPSK_CUDA_OK(cudaMemcpyAsync(&h_report->first_probe, d_res, sizeof(fpsk_probe_result), cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    if (h_report->first_probe.status != FPSK_OK) return (fpsk_status)h_report->first_probe.status;
    if (!h_report->first_probe.fired) {
        h_report->state = 0;       // clean: nothing else runs
        return FPSK_OK;
    }

    // ---- exact scan for nonfinite / out-of-range entries, recomputed as absolute values
    std::vector<fpsk_fault> F;
    std::vector<PatchEntry> restore;
    {
        int n_abs = 0;
        std::vector<ScanEntry> ent((size_t)K);
        rc = scan_launch(C, ldc, m, n, K, rep_ws, st, ent.data(), &n_abs);
        if (rc != FPSK_OK) return rc;
        if (n_abs > 0) {
            std::vector<double> gam((size_t)n_abs);
            std::vector<float> oldv((size_t)n_abs);
            SketchIn in0{A, B, C, m, k, n, lda, ldb, ldc};
            rc = recompute_entries(in0, dtype, ent.data(), n_abs, rep_ws, st, gam.data(), oldv.data());
            if (rc != FPSK_OK) return rc;
            std::vector<PatchEntry> pe((size_t)n_abs);
            for (int e = 0; e < n_abs; ++e) {
                fpsk_fault f;
                memset(&f, 0, sizeof(f));
                f.i = ent[e].i; f.j = ent[e].j;
                f.delta = gam[e];                 // absolute: the repaired value itself
                f.recompute = gam[e];
                f.c_value = oldv[e];
                f.round = -1; f.bucket_a = -1; f.bucket_b = -1;
                F.push_back(f);
                pe[e] = PatchEntry{f.i, f.j, PATCH_SET, gam[e]};
                restore.push_back(PatchEntry{f.i, f.j, PATCH_SET_BITS, 0.0});
                memcpy(&restore.back().value, &oldv[e], sizeof(float));      // exact bit pattern of the old entry
            }
            // C holds the recomputed values while the sketches are built
            PatchEntry *d = static_cast<PatchEntry *>(rep_ws);
            FPSK_CUDA_OK(cudaMemcpyAsync(d, pe.data(), sizeof(PatchEntry) * n_abs, cudaMemcpyHostToDevice, st));
            rc = patch_launch(C, ldc, d, n_abs, st);
            if (rc != FPSK_OK) return rc;
            FPSK_CUDA_OK(cudaStreamSynchronize(st));
        }
        h_report->n_absolute = n_abs;
    }

    // ---- plan from the noise measured on this call, then k rounds of Algorithm 1
    fpsk_params qq = q;
    int m_loc = n_buckets;
    bool truncated = false;
    int radius_used = 0;
    HostRes hr;
    rc = [&]() -> fpsk_status {
        fpsk_status rc = hr.acquire(q, true);
        if (rc != FPSK_OK) return rc;
        if (m_loc <= 0) {
            const int m0 = std::min(m_start_of(m, k, n, dtype, q), sketch_max_buckets(m, k, n));
            LocWs w0;
            if (!loc_carve(loc_ws, loc_bytes, m, k, n, m0, w0, q.tensor_cores != 0)) return FPSK_ERR_WORKSPACE;
            SketchIn in{A, B, C, m, k, n, lda, ldb, ldc};
            if (w0.sk.tc) {
                rc = loc_max_ab(in, dtype, w0, st);
                if (rc != FPSK_OK) return rc;
            }
            rc = build_sketches(in, dtype, seed, 0, m0, false, w0.sk, st, w0.S, nullptr, nullptr);
            if (rc != FPSK_OK) return rc;
            rc = sigma_mad_rms_c_launch(w0.S, (long long)m0 * m0, q.mad_of_abs, C, ldc, m, n, w0.samples, w0.sel, w0.misc + 3, st);
            if (rc != FPSK_OK) return rc;
            float h_scal[8], h_rms = 0.f;
            rc = read_noise_scalars(w0, st, h_scal, h_rms, hr.pin.p);
            if (rc != FPSK_OK) return rc;
            int r;
            double B_;
            plan_of(m, k, n, dtype, h_scal[1], h_rms, m0, q, m_loc, r, B_);
            m_loc = std::min(m_loc, sketch_max_buckets(m, k, n));
            if (qq.radius < 0) qq.radius = r;
        }
        LocWs w;
        if (!loc_carve(loc_ws, loc_bytes, m, k, n, m_loc, w, q.tensor_cores != 0, true)) return FPSK_ERR_WORKSPACE;
        SketchIn in{A, B, C, m, k, n, lda, ldb, ldc};
        return localize_core(in, dtype, seed, m_loc, qq, w, st, hr, F, truncated, radius_used);
    }();
    if (rc != FPSK_OK) hr.drain(st);
    // ---- the absolute entries go back into C whatever happened above
    if (!restore.empty()) {
        PatchEntry *d = static_cast<PatchEntry *>(rep_ws);
        fpsk_status rc2 = FPSK_OK;
        if (cudaMemcpyAsync(d, restore.data(), sizeof(PatchEntry) * restore.size(), cudaMemcpyHostToDevice, st) != cudaSuccess)
            rc2 = FPSK_ERR_CUDA;
        if (rc2 == FPSK_OK) rc2 = patch_launch(C, ldc, d, (int)restore.size(), st);
        if (cudaStreamSynchronize(st) != cudaSuccess && rc2 == FPSK_OK) rc2 = FPSK_ERR_CUDA;
        if (rc == FPSK_OK) rc = rc2;
    }
    if (rc != FPSK_OK) return rc;
    h_report->m_loc = m_loc;
    h_report->radius = radius_used;

    // ---- apply: C_ij <- delta for the absolute entries, C_ij <- C_ij + delta for the others
    std::sort(F.begin(), F.end(), [](const fpsk_fault &x, const fpsk_fault &y) {
        return x.i != y.i ? x.i < y.i : x.j < y.j;
    });
    h_report->n_faults = (int32_t)F.size();
    const int ncopy = std::min<int>((int)F.size(), capacity);
    for (int f = 0; f < ncopy; ++f) h_faults[f] = F[f];
    if ((int)F.size() > kRepairCap) truncated = true;
    rc = fpsk_apply_corrections(C, ldc, m, n, F.data(), (int)std::min<size_t>(F.size(), kRepairCap), rep_ws,
                                repair_scratch_bytes(), stream);
    if (rc != FPSK_OK) return rc;

    // ---- probe once more; if it still fires the caller must recompute the product
    rc = probe_launch(A, B, C, pd, dtype, q.mu, probe_ws, pws, st, d_res, nullptr);
    if (rc != FPSK_OK) return rc;
    FPSK_CUDA_OK(cudaMemcpyAsync(&h_report->second_probe, d_res, sizeof(fpsk_probe_result), cudaMemcpyDeviceToHost, st));
    FPSK_CUDA_OK(cudaStreamSynchronize(st));
    if (h_report->second_probe.status != FPSK_OK) return (fpsk_status)h_report->second_probe.status;
    h_report->state = h_report->second_probe.fired ? 2 : 1;
    if ((int)F.size() > capacity || truncated) return FPSK_ERR_CAPACITY;
    return FPSK_OK;
}

uint64_t fpsk_launch_count(void) { return g_launches.load(); }
uint64_t fpsk_lazy_resource_count(void) { return g_lazy_resources.load(); }

int32_t fpsk_debug_bounds_report(int64_t *violations, int32_t *line, int64_t *index, int64_t *limit, char *file, size_t file_cap)
{
#ifdef FPSK_DEBUG_BOUNDS
    long long total = 0;
    bool first = true;
    if (file && file_cap) file[0] = 0;
    for (const BoundsSource &src : bounds_sources()) {
        BoundsRecord r;
        if (src.read(&r) != cudaSuccess) return -1;
        total += r.count;
        if (r.count && first) {
            first = false;
            if (line) *line = r.line;
            if (index) *index = r.index;
            if (limit) *limit = r.limit;
            if (file && file_cap) {
                strncpy(file, src.file, file_cap - 1);
                file[file_cap - 1] = 0;
            }
        }
    }
    if (violations) *violations = total;
    return 1;
#else
    (void)line; (void)index; (void)limit; (void)file; (void)file_cap;
    if (violations) *violations = -1;
    return 0;
#endif
}

fpsk_status fpsk_debug_bounds_clear(void)
{
#ifdef FPSK_DEBUG_BOUNDS
    for (const BoundsSource &src : bounds_sources())
        if (src.clear() != cudaSuccess) return FPSK_ERR_CUDA;
#endif
    return FPSK_OK;
}

fpsk_status fpsk_context_create(fpsk_context **out)
{
    if (!out) return FPSK_ERR_NULL;
    *out = nullptr;
    fpsk_context *c = new fpsk_context;
    bool ok = sketch_aux_create(c->aux) == FPSK_OK;
    ok = ok && cudaEventCreateWithFlags(&c->round_done, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->pinned, kPackBytes, cudaHostAllocPortable) == cudaSuccess;
    if (!ok) {
        fpsk_context_destroy(c);
        return FPSK_ERR_CUDA;
    }
    *out = c;
    return FPSK_OK;
}

fpsk_status fpsk_context_destroy(fpsk_context *c)
{
    if (!c) return FPSK_OK;
    bool ok = sketch_aux_destroy(c->aux);
    if (c->round_done) ok = (cudaEventDestroy(c->round_done) == cudaSuccess) && ok;
    if (c->pinned) ok = (cudaFreeHost(c->pinned) == cudaSuccess) && ok;
    delete c;
    return ok ? FPSK_OK : FPSK_ERR_CUDA;
}

}  // extern "C"
