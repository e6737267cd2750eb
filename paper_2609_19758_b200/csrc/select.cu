// Noise estimates, thresholds and candidate selection on a sketch S (Section "Thresholds";
// Algorithm 1: MAD estimate, tau_c, tau_d, the K largest buckets, the set U and the moment
// ratios of Eq. (recover)).  Medians and the K-th largest key come from an exact radix select
// (integer histograms only), so every decision is deterministic.
#include "sketch.cuh"
#include "stream_pipe.cuh"

#include <math.h>

namespace fpsk {

enum SelMode {
    SEL_ABS = 0,        // key = bits(|S|)                         (median of |S|)
    SEL_SIGNED = 1,     // key = order-preserving bits of S        (median of S)
    SEL_DEV_ABS = 2,    // key = bits(||S| - med|)
    SEL_DEV_SIGNED = 3, // key = bits(|S - med|)
    SEL_TOPK = 4,       // key = bits(|S|) << 32 | ~idx (all keys distinct; a NaN sorts below everything)
    SEL_SAMPLE = 5      // valid iff S >= 0 (sentinel -1 marks dropped samples); key = bits(S)
};

// state words (per job slot)
enum { ST_PREFIX = 0, ST_K = 1, ST_SKIP = 2, ST_WORDS = 4 };
// scal slots
enum { SC_MED = 0, SC_MAD = 1, SC_MEAN = 2, SC_CLIP = 3, SC_THR = 4, SC_TAUC = 5, SC_TAUD = 6, SC_SMED = 7, SC_WORDS = 16 };
// Histogram words.  Every CTA adds its 256 counts to one of kHistCopies copies (CTA index modulo the copies),
// each copy in cache lines of its own, so that the CTAs' atomics do not all queue on the same eight lines.
// Digit d, job slot s, copy r: hist[kHistBase + ((d * 2 + s) * kHistCopies + r) * 256 ...].
enum { kHistCopies = 8, kHistBase = 64, kHistWords = 8 /*digits*/ * 2 * kHistCopies * 256,
       kHistErr = kHistBase + kHistWords, kSumTicket = kHistErr + 1, kHistBytes = (kHistBase + kHistWords + 64) * 4 };
// hist[0]: arrival counter of the running select launch (zeroed with the histograms before every launch);
// hist[kHistErr]: set when a bounded wait gave up (zeroed once per call of the library, read by the host);
// hist[kSumTicket]: ticket of the clipped-mean sums.

__device__ __forceinline__ uint32_t ordered_bits(float x)
{
    uint32_t b = __float_as_uint(x);
    return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t k)
{
    uint32_t b = (k >> 31) ? (k ^ 0x80000000u) : ~k;
    return __uint_as_float(b);
}

// key of the K-largest selection: descending |S|, ties by ascending flat index
__device__ __forceinline__ unsigned long long topk_key(float a, long long idx)
{
    const uint32_t hi = (a == a) ? __float_as_uint(a) : 0u;
    return ((unsigned long long)hi << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}

// key of element idx with value x (med: the median that the deviation keys are taken from)
__device__ __forceinline__ bool key_of(int mode, float x, long long idx, float med, unsigned long long &key)
{
    switch (mode) {
    case SEL_ABS: key = __float_as_uint(fabsf(x)); return true;
    case SEL_SIGNED: key = ordered_bits(x); return true;
    case SEL_DEV_ABS: key = __float_as_uint(fabsf(fabsf(x) - med)); return true;
    case SEL_DEV_SIGNED: key = __float_as_uint(fabsf(x - med)); return true;
    case SEL_TOPK: key = topk_key(fabsf(x), idx); return true;
    default:
        if (!(x >= 0.f)) return false;
        key = __float_as_uint(x);
        return true;
    }
}
__device__ __forceinline__ bool make_key(int mode, const float *S, long long idx, const float *scal,
                                         unsigned long long &key)
{
    return key_of(mode, S[idx], idx, scal[SC_MED], key);
}

// counts[0] = number of valid keys (SEL_SAMPLE)
__global__ void count_valid_kernel(int mode, const float *S, long long mm, const float *scal, int *counts)
{
    int c = 0;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < mm; i += (long long)gridDim.x * blockDim.x) {
        unsigned long long k;
        c += make_key(mode, S, i, scal, k) ? 1 : 0;
    }
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(counts, c);
}

constexpr int kSelThreads = 1024; // one CTA per SM
constexpr int kSelItems = 8;      // elements per thread and batch (their keys stay in registers over the digits when one
                                  // batch covers the source)

// One radix select in flight: its source, key kind, digit position.  Up to two run in one launch (slot 0, 1).
struct SelJob {
    const float *src;
    long long n;
    int mode, nbits, shift, K;
};

// rank to select: median of N keys, or (N - K) for the K largest
__device__ __forceinline__ void select_initial(const SelJob &j, const int *counts, bool &skip, unsigned long long &k)
{
    skip = false;
    k = 0;
    if (j.mode == SEL_TOPK) {
        // The K largest of all keys.  The buckets above the detection threshold are a top segment of this
        // order, so "the K largest above the threshold" is this selection cut at the threshold afterwards.
        if (j.n <= (long long)j.K) skip = true;
        else k = (unsigned long long)(j.n - j.K);
    } else if (j.mode == SEL_SAMPLE) {
        const int cnt = counts[0];
        if (cnt <= 0) skip = true;
        else k = (unsigned long long)((cnt - 1) / 2);
    } else {
        k = (unsigned long long)((j.n - 1) / 2);
    }
}

// what the selected key means, written once the last digit is known (or at once when nothing is selected)
__device__ __forceinline__ void select_result(int mode, unsigned long long key, bool skip, float *scal)
{
    if (mode == SEL_ABS) scal[SC_MED] = __uint_as_float((uint32_t)key);
    else if (mode == SEL_SIGNED) scal[SC_MED] = from_ordered_bits((uint32_t)key);
    else if (mode == SEL_DEV_ABS || mode == SEL_DEV_SIGNED) scal[SC_MAD] = 1.4826f * __uint_as_float((uint32_t)key);
    else if (mode == SEL_SAMPLE) scal[SC_SMED] = skip ? __uint_as_float(0x7FC00000u) : __uint_as_float((uint32_t)key);
}

// The digits of up to three radix selects in ONE cooperative launch: `a` in slot 0 and, beside it digit by
// digit, `b` and then `c` in slot 1 (independent sources, keys and ranks; one pass over memory when they
// share the source; c may take its deviations from b's result, which every CTA derives for itself).  A
// digit is: every CTA bins its keys in shared memory and adds the 256 counts to one of the copies of this
// digit's histogram; a grid-wide arrival counter (bounded wait); every CTA sums the copies and finds the
// bin of the k-th key by the same scan.  One CTA of 1024 threads per SM.  Measured at 10^6 keys: 5 us per
// digit (binning 1-2, arrival wait 2, copies + scan 1), against 9.5 us for a launch per digit with a
// last-CTA scan and the select state in global memory; the K-largest key needs only its upper four digits
// when the K-th value is unique, and the median of the samples of C and the two medians of the MAD ride in
// the same launches, so a localization round runs 8 digits in one launch instead of 16 launches.
struct SelChain {
    SelJob a, b, c;
    int have_b, have_c;
    // Epilogue of a localization round's launch (collect != 0; `a` is then the K-largest selection over S): the
    // thresholds tau_c, tau_d from sigma_MAD (just selected in slot 1, or already in scal) and the analytic cap, and
    // the keys at or above the K-th that exceed max(tau_c, tau_d) gathered into `keys` (unsorted, count in counts[1]).
    // Every CTA knows the K-th key and sigma_MAD when the digits are done, so this needs no further launch.
    int collect, cap;
    const float *taup;
    float nmax, rad;
    unsigned long long *keys;
    int *counts_out;
};
constexpr int kChainSteps = 8;                 // digits of the longest key (64 bits)

// For both select slots at once: inclusive scan of the 256 counts (thread t < 256 holds bin t) -> the bin whose
// running count passes k, and the number of keys below it; the same values in every thread of the CTA.  The first
// eight warps work among themselves (named barrier); the other warps only join the closing barrier.
__device__ __forceinline__ void pick_digits(const unsigned int (&h)[2], const unsigned long long (&k)[2], const bool (&on)[2],
                                            unsigned long long (*wsum)[8], int *s_bin, unsigned long long *s_before,
                                            int (&bin)[2], unsigned long long (&before_out)[2])
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (threadIdx.x < 256) {
        unsigned long long inc[2] = {h[0], h[1]};
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const unsigned long long v = __shfl_up_sync(0xFFFFFFFFu, inc[j], o);
                if (lane >= o) inc[j] += v;
            }
        }
        if (lane == 31) { wsum[0][wid] = inc[0]; wsum[1][wid] = inc[1]; }
        if (threadIdx.x < 2) { s_bin[threadIdx.x] = 255; s_before[threadIdx.x] = 0; }
        asm volatile("bar.sync 1, 256;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (!on[j]) continue;
            unsigned long long base = 0, total = 0;
            for (int w = 0; w < 8; ++w) {
                const unsigned long long v = wsum[j][w];
                if (w < wid) base += v;
                total += v;
            }
            const unsigned long long incl = inc[j] + base;          // keys in bins 0 .. threadIdx.x
            const unsigned long long before = incl - h[j];          // keys in bins below this one
            if (before <= k[j] && k[j] < incl) { s_bin[j] = (int)threadIdx.x; s_before[j] = before; }     // exactly one thread, when k < total
            if (threadIdx.x == 255 && k[j] >= total) { s_bin[j] = 255; s_before[j] = total; }              // k beyond the keys (not reached: k is clamped to the count)
        }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        bin[j] = s_bin[j];
        before_out[j] = s_before[j];
    }
}

__device__ __forceinline__ float median_value(int mode, unsigned long long key)
{
    return mode == SEL_SIGNED ? from_ordered_bits((uint32_t)key) : __uint_as_float((uint32_t)key);
}

// 32-bit part of a key that does not change over the digits (for the K-largest key: its upper half)
__device__ __forceinline__ uint32_t key_base(int mode, float x, float med)
{
    switch (mode) {
    case SEL_ABS: return __float_as_uint(fabsf(x));
    case SEL_SIGNED: return ordered_bits(x);
    case SEL_DEV_ABS: return __float_as_uint(fabsf(fabsf(x) - med));
    case SEL_DEV_SIGNED: return __float_as_uint(fabsf(x - med));
    case SEL_TOPK: { const float a = fabsf(x); return (a == a) ? __float_as_uint(a) : 0u; }
    default: return (x >= 0.f) ? __float_as_uint(x) : 0xFFFFFFFFu;      // dropped sample: no key
    }
}

// One digit of one select over the kSelItems elements of this thread (keys in registers): every lane whose
// key still carries the prefix adds one to its bin in shared memory.  Plain atomics: lanes of a warp that hit the
// same address cost no more than lanes that spread (measured on sketches of exact zeros), and combining equal bins
// first (match.any, a register cache of the last bins) only added instructions: 67 us per round against 43.
// LOW: the digit lies in the lower half of a 64-bit K-largest key (~element index) and the upper half must match.
template <bool LOW>
__device__ __forceinline__ void bin_items(const uint32_t (&kbj)[kSelItems], uint32_t ibase, uint32_t n32, bool sample,
                                          uint32_t pre_hi, uint32_t pre_lo, uint32_t fixed, int sh32, unsigned int *shj)
{
#pragma unroll
    for (int u = 0; u < kSelItems; ++u) {
        const uint32_t i32 = ibase + (uint32_t)(u * kSelThreads);
        const uint32_t kbu = kbj[u];
        bool valid = i32 < n32 && !(sample && kbu == 0xFFFFFFFFu);
        uint32_t word;
        if (LOW) {
            word = 0xFFFFFFFFu - i32;
            valid = valid && kbu == pre_hi && ((word ^ pre_lo) & fixed) == 0u;
        } else {
            word = kbu;
            valid = valid && ((word ^ pre_hi) & fixed) == 0u;
        }
        if (valid) atomicAdd(&shj[(word >> sh32) & 255u], 1u);
    }
}

__global__ void __launch_bounds__(kSelThreads, 1) select_chain_kernel(SelChain ch, float *scal, unsigned long long *state,
                                                              unsigned int *hist, const int *counts)
{
    __shared__ unsigned int sh[2][256];
    __shared__ unsigned long long wsum[2][8];
    __shared__ int s_bin[2], s_ok;
    __shared__ unsigned long long s_before[2];
    const int G = (int)gridDim.x, tid = (int)threadIdx.x;
    SelJob job[2] = {ch.a, ch.b};
    bool on[2] = {true, ch.have_b != 0};
    bool have_c = ch.have_c != 0;
    unsigned long long k[2] = {0, 0}, prefix[2] = {0, 0};
    float med = scal[SC_MED];
    const bool lead = blockIdx.x == 0 && tid == 0;
    // for the collect epilogue: sigma_MAD as it stands (replaced when this launch selects it) and the K-th key
    float mad_local = scal[SC_MAD];
    unsigned long long kth_local = 0ull;
    bool top_skipped = false;
    if (ch.collect && lead) {
        // cleared here, used after at least one grid-wide arrival: the lead's stores precede its release there
        ch.counts_out[0] = 0; ch.counts_out[1] = 0; ch.counts_out[2] = 0;
    }
    // a slot-1 job that has nothing to select makes room for its successor at once
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        for (int tries = 0; tries < 2 && on[j]; ++tries) {
            bool skip;
            select_initial(job[j], counts, skip, k[j]);
            job[j].shift = job[j].nbits - 8;
            if (!skip) break;
            if (j == 0) top_skipped = true;
            if (lead) {
                state[j * ST_WORDS + ST_SKIP] = 1;
                state[j * ST_WORDS + ST_PREFIX] = 0;
                select_result(job[j].mode, 0, true, scal);
            }
            if (j == 1 && have_c) { job[1] = ch.c; have_c = false; }
            else on[j] = false;
        }
    }
    const int steps1 = (ch.have_b ? ch.b.nbits / 8 : 0) + (ch.have_c ? ch.c.nbits / 8 : 0);
    const int nsteps = ch.a.nbits / 8 > steps1 ? ch.a.nbits / 8 : steps1;
    const long long per_grid = (long long)G * (kSelThreads * kSelItems);
    long long nall = ch.a.n;
    if (ch.have_b && ch.b.n > nall) nall = ch.b.n;
    if (ch.have_c && ch.c.n > nall) nall = ch.c.n;
    // When one batch covers the sources a thread derives the keys of its elements once per select and keeps
    // them (in registers) over the digits; otherwise it derives them again digit by digit.
    const bool one_batch = nall <= per_grid;
    uint32_t kb[2][kSelItems];                     // the keys of this thread's elements, in registers
    bool fresh[2] = {true, true};
    for (int step = 0; step < nsteps; ++step) {
        if (tid < 256) {
            sh[0][tid] = 0;
            sh[1][tid] = 0;
        }
        __syncthreads();
        long long nmax = 0;
#pragma unroll
        for (int j = 0; j < 2; ++j)
            if (on[j] && job[j].n > nmax) nmax = job[j].n;
        for (long long base = (long long)blockIdx.x * (kSelThreads * kSelItems); base < nmax; base += per_grid) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (!on[j] || !(fresh[j] || !one_batch)) continue;
#pragma unroll
                for (int u0 = 0; u0 < kSelItems; u0 += 8) {
                    float x[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const long long i = base + (u0 + u) * kSelThreads + tid;
                        x[u] = i < job[j].n ? __ldg(job[j].src + i) : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) kb[j][u0 + u] = key_base(job[j].mode, x[u], med);
                }
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (!on[j]) continue;
                const int shift = job[j].shift;
                const bool wide = job[j].nbits == 64;              // K-largest key: kb is the upper half, ~index the lower
                const bool low_half = wide && shift < 32;
                const bool sample = job[j].mode == SEL_SAMPLE;
                const uint32_t pre_hi = wide ? (uint32_t)(prefix[j] >> 32) : (uint32_t)prefix[j];
                const uint32_t pre_lo = (uint32_t)prefix[j];
                const int sh32 = low_half ? shift : (wide ? shift - 32 : shift);
                // bits of the 32-bit word in play that are already fixed by earlier digits
                const uint32_t fixed = sh32 + 8 >= 32 ? 0u : (0xFFFFFFFFu << (sh32 + 8));
                const uint32_t ibase = (uint32_t)base + (uint32_t)tid;      // element indices fit 32 bits (<= 2^24 buckets)
                if (low_half) bin_items<true>(kb[j], ibase, (uint32_t)job[j].n, sample, pre_hi, pre_lo, fixed, sh32, sh[j]);
                else bin_items<false>(kb[j], ibase, (uint32_t)job[j].n, sample, pre_hi, pre_lo, fixed, sh32, sh[j]);
            }
        }
        fresh[0] = false;
        fresh[1] = false;
        __syncthreads();
        unsigned int *hstep = hist + kHistBase + (size_t)step * (2 * kHistCopies * 256);
#pragma unroll
        for (int j = 0; j < 2; ++j)
            if (on[j] && tid < 256 && sh[j][tid]) atomicAdd(&hstep[(j * kHistCopies + (blockIdx.x % kHistCopies)) * 256 + tid], sh[j][tid]);
        // ---- all CTAs' counts are in: arrival counter, bounded wait
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            red_release_add(hist);
            s_ok = bounded_wait_ge(hist, (unsigned)(step + 1) * (unsigned)G) ? 1 : 0;
            if (!s_ok) atomicOr(hist + kHistErr, 1u);
        }
        __syncthreads();
        if (!s_ok) return;
        unsigned int hsum[2] = {0, 0};
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (!on[j]) continue;
#pragma unroll
            for (int r = 0; r < kHistCopies; ++r)
                if (tid < 256) hsum[j] += __ldcg(&hstep[(j * kHistCopies + r) * 256 + tid]);
        }
        int dbin[2];
        unsigned long long dbefore[2];
        {
            const bool on_now[2] = {on[0], on[1]};
            pick_digits(hsum, k, on_now, wsum, s_bin, s_before, dbin, dbefore);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (!on[j]) continue;
            k[j] -= dbefore[j];
            prefix[j] |= (unsigned long long)dbin[j] << job[j].shift;
            job[j].shift -= 8;
            // K-largest key: once the rank inside the remaining ties is 0, the lower digits cannot move the
            // cut (every key of the tie is at or above "upper half, zeros"), so they are left at zero
            if (job[j].nbits == 64 && job[j].shift < 32 && k[j] == 0) job[j].shift = -8;
            if (job[j].shift >= 0) continue;
            // the select in slot j is complete
            if (lead) {
                state[j * ST_WORDS + ST_SKIP] = 0;
                state[j * ST_WORDS + ST_PREFIX] = prefix[j];
                select_result(job[j].mode, prefix[j], false, scal);
            }
            if (job[j].mode == SEL_ABS || job[j].mode == SEL_SIGNED) med = median_value(job[j].mode, prefix[j]);
            if (job[j].mode == SEL_DEV_ABS || job[j].mode == SEL_DEV_SIGNED) mad_local = 1.4826f * __uint_as_float((uint32_t)prefix[j]);
            if (j == 0) kth_local = prefix[0];
            if (j == 1 && have_c) {
                job[1] = ch.c;
                have_c = false;
                fresh[1] = true;
                bool skip;
                select_initial(job[1], counts, skip, k[1]);
                job[1].shift = job[1].nbits - 8;
                prefix[1] = 0;
                if (skip) {
                    if (lead) {
                        state[ST_WORDS + ST_SKIP] = 1;
                        state[ST_WORDS + ST_PREFIX] = 0;
                        select_result(job[1].mode, 0, true, scal);
                    }
                    on[1] = false;
                }
            } else {
                on[j] = false;
            }
        }
        if (!on[0] && !on[1]) break;       // same decision in every CTA: nobody waits for a further digit
    }
    if (!ch.collect) return;
    // ---- thresholds (Section "Thresholds"; Algorithm 1) and the collection of the keys above them
    const float tau = __ldg(ch.taup);
    const float tau_c = fminf(tau, 2.f * mad_local);
    const float tau_d = ch.nmax * mad_local / fmaxf(ch.rad, 0.5f);
    const float thr = fmaxf(tau_c, tau_d);
    if (lead) {
        scal[SC_TAUC] = tau_c;
        scal[SC_TAUD] = tau_d;
        scal[SC_THR] = thr;
    }
    const unsigned long long kth = top_skipped ? 0ull : kth_local;
    for (long long i = (long long)blockIdx.x * kSelThreads + tid; i < ch.a.n; i += (long long)G * kSelThreads) {
        const float av = fabsf(__ldg(ch.a.src + i));
        if (!(av > thr)) continue;
        const unsigned long long key = topk_key(av, i);
        if (key < kth) continue;
        const int slot = atomicAdd(ch.counts_out + 1, 1);
        if (slot < ch.cap) ch.keys[slot] = key;
    }
}

static int select_capacity()
{
    static int cap = 0;            // co-resident CTAs of the cooperative select kernel on this device
    if (cap == 0) {
        int dev = 0, sms = 0, occ = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return 148;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, select_chain_kernel, kSelThreads, 0) != cudaSuccess || occ < 1) return sms;
        cap = sms;
    }
    return cap;
}

static int select_grid(long long n)
{
    const long long want = (n + kSelThreads * kSelItems - 1) / (kSelThreads * kSelItems);
    const int cap = select_capacity();
    return (int)(want < 1 ? 1 : (want > cap ? cap : want));
}

// Runs select `a` in slot 0 and, beside it, `b` and then `c` in slot 1.  One memset (this launch's histograms
// and arrival counter) and one cooperative launch.
struct SelCollect {
    const float *taup = nullptr;
    float nmax = 0.f, rad = 0.f;
};
static fpsk_status run_selects(SelJob a, SelJob b, bool have_b, SelJob c, bool have_c, SelectWs &w, cudaStream_t st,
                               const SelCollect *collect = nullptr)
{
    const int da = a.nbits / 8, db = have_b ? b.nbits / 8 : 0, dc = have_c ? c.nbits / 8 : 0;
    const int steps = da > db + dc ? da : db + dc;
    if (steps > kChainSteps || (have_c && !have_b)) return FPSK_ERR_PARAM;
    if (!w.hist_clean) {
        // the sticky error word only: the ticket next to it belongs to the clipped-mean sums, which may be running
        // on another stream at this moment
        FPSK_CUDA_OK(cudaMemsetAsync(w.hist + kHistErr, 0, sizeof(unsigned int), st));
        w.hist_clean = true;
    }
    FPSK_CUDA_OK(cudaMemsetAsync(w.hist, 0, (size_t)(kHistBase + steps * 2 * kHistCopies * 256) * sizeof(unsigned int), st));
    SelChain ch;
    ch.a = a; ch.b = b; ch.c = c; ch.have_b = have_b ? 1 : 0; ch.have_c = have_c ? 1 : 0;
    ch.collect = collect ? 1 : 0; ch.cap = kSelMaxK;
    ch.taup = collect ? collect->taup : nullptr; ch.nmax = collect ? collect->nmax : 0.f; ch.rad = collect ? collect->rad : 0.f;
    ch.keys = w.keys; ch.counts_out = w.counts;
    long long nmax = a.n;
    if (have_b && b.n > nmax) nmax = b.n;
    if (have_c && c.n > nmax) nmax = c.n;
    const int grid = select_grid(nmax);
    float *scal = w.scal;
    unsigned long long *state = w.state;
    unsigned int *hist = w.hist;
    const int *counts = w.counts;
    void *args[] = {(void *)&ch, (void *)&scal, (void *)&state, (void *)&hist, (void *)&counts};
    FPSK_CUDA_OK(cudaLaunchCooperativeKernel((const void *)select_chain_kernel, dim3(grid), dim3(kSelThreads), args, 0, st));
    count_launch();
    return FPSK_OK;
}

static SelJob sel_job(int mode, int nbits, const float *src, long long n, int K)
{
    SelJob j;
    j.src = src; j.n = n; j.mode = mode; j.nbits = nbits; j.shift = nbits - 8; j.K = K;
    return j;
}

// ---------------------------------------------------------------- clipped mean
// mode 0: sum |S| -> scal[SC_MEAN] = mean; mode 1: sum min(|S|, 5 mean) -> scal[SC_CLIP].
// Fixed grid, fixed per-CTA tree, partials summed in CTA order by the last CTA: deterministic.
constexpr int kSumGrid = 256;
__global__ void __launch_bounds__(256) abs_sum_kernel(int mode, const float *S, long long mm, float *scal, float *partial,
                                                      unsigned int *ticket)
{
    __shared__ float sh[256];
    __shared__ int last;
    const float clip = mode ? 5.f * scal[SC_MEAN] : 0.f;
    float acc = 0.f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < mm; i += (long long)gridDim.x * blockDim.x) {
        const float a = fabsf(S[i]);
        acc += mode ? fminf(a, clip) : a;
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        __stcg(partial + blockIdx.x, sh[0]);
        __threadfence();
        last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!last || threadIdx.x != 0) return;
    __threadfence();
    float tot = 0.f;
    for (int b = 0; b < (int)gridDim.x; ++b) tot += __ldcg(partial + b);
    const float mean = tot / (float)mm;
    if (mode) scal[SC_CLIP] = 1.2533f * mean;
    else scal[SC_MEAN] = mean;
    *ticket = 0;
}

fpsk_status sigma_clip_launch(const float *S, long long mm, SelectWs &w, cudaStream_t st)
{
    FPSK_CUDA_OK(cudaMemsetAsync(w.hist + kSumTicket, 0, 4, st));
    for (int mode = 0; mode < 2; ++mode) {
        abs_sum_kernel<<<kSumGrid, 256, 0, st>>>(mode, S, mm, w.scal, w.partial, w.hist + kSumTicket);
        FPSK_LAUNCH_CHECK();
    }
    return FPSK_OK;
}

// ---------------------------------------------------------------- thresholds and candidates
__global__ void thresholds_kernel(const float *taup, float nmax, float rad, float *scal, int *counts)
{
    if (threadIdx.x != 0) return;
    const float tau = *taup;
    const float sig = scal[SC_MAD];
    const float tau_c = fminf(tau, 2.f * sig);
    const float tau_d = nmax * sig / fmaxf(rad, 0.5f);
    scal[SC_TAUC] = tau_c;
    scal[SC_TAUD] = tau_d;
    scal[SC_THR] = fmaxf(tau_c, tau_d);
    counts[0] = 0; counts[1] = 0; counts[2] = 0;
}

__global__ void collect_kernel(const float *S, long long mm, const float *scal, const unsigned long long *state,
                               int cap, unsigned long long *keys, int *counts)
{
    // the K largest keys (slot 0 of the select state), cut at the detection threshold
    const unsigned long long kth = state[ST_SKIP] ? 0ull : state[ST_PREFIX];
    const float thr = scal[SC_THR];
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < mm; i += (long long)gridDim.x * blockDim.x) {
        const float a = fabsf(S[i]);
        if (!(a > thr)) continue;
        const unsigned long long k = topk_key(a, i);
        if (k < kth) continue;
        const int slot = atomicAdd(counts + 1, 1);
        if (slot < cap) keys[slot] = k;
    }
}

// Sort the selected keys (descending |S|, ties by ascending flat index), keep those with
// S != 0 and S, R, T finite (the set U), decode Eq. (recover) with 1-based -> 0-based indices.
// The moments come either from whole sketches R, T (indexed by bucket) or, when Rc is given, from the values
// computed for the collected keys only (Rc, Tc indexed by the key's slot in `keys`).
__global__ void __launch_bounds__(1024) decode_kernel(const float *S, const float *R, const float *T, const float *Rc,
                                                      const float *Tc, int p1, int p3, const unsigned long long *keys,
                                                      int *counts, int cap, Candidate *cand, int *zero_word)
{
    __shared__ unsigned long long sk[kSelMaxK];
    if (zero_word && threadIdx.x == 0) *zero_word = 0;       // the hit counter of the confirmation launched next
    __shared__ int flag[kSelMaxK];
    __shared__ unsigned short sl[kSelMaxK];           // the slot a key came from
    const int t = threadIdx.x;
    int n = counts[1];
    if (n > cap) n = cap;
    sk[t] = t < n ? keys[t] : 0ull;
    sl[t] = (unsigned short)t;
    __syncthreads();
    // the network only has to cover the keys that are there (a power of two; zeros fill the rest)
    int np2 = 2;
    while (np2 < n) np2 <<= 1;
    for (int k = 2; k <= np2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int ixj = t ^ j;
            if (ixj > t && ixj < np2) {
                const bool desc = (t & k) == 0;
                const unsigned long long a = sk[t], b = sk[ixj];
                if (desc ? (a < b) : (a > b)) {
                    sk[t] = b; sk[ixj] = a;
                    const unsigned short u = sl[t]; sl[t] = sl[ixj]; sl[ixj] = u;
                }
            }
            __syncthreads();
        }
    }
    Candidate c;
    c.flat = -1; c.ih = 0; c.jh = 0; c.s_abs = 0.f;
    int keep = 0;
    if (t < n) {
        const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(sk[t] & 0xFFFFFFFFull);
        const float s = S[idx], r = Rc ? Rc[sl[t]] : (R ? R[idx] : 0.f), q = Tc ? Tc[sl[t]] : (T ? T[idx] : 0.f);
        const bool fin = (fabsf(s) <= 3.402823466e38f) && (fabsf(r) <= 3.402823466e38f) && (fabsf(q) <= 3.402823466e38f);
        if (s != 0.f && fin) {
            float fi = rintf(ldexpf(r / s, p1)) - 1.f;
            float fj = rintf(ldexpf(q / s, p3)) - 1.f;
            const float lim = 1073741824.f;
            if (!(fabsf(fi) < lim)) fi = -lim;
            if (!(fabsf(fj) < lim)) fj = -lim;
            c.flat = (int)idx; c.ih = (int)fi; c.jh = (int)fj; c.s_abs = fabsf(s);
            keep = 1;
        }
    }
    flag[t] = keep;
    __syncthreads();
    // inclusive scan of the keep flags (order-preserving compaction)
    for (int o = 1; o < np2; o <<= 1) {
        const int v = t >= o ? flag[t - o] : 0;
        __syncthreads();
        flag[t] += v;
        __syncthreads();
    }
    if (keep && FPSK_IN_BOUNDS(flag[t] - 1, np2)) cand[flag[t] - 1] = c;
    if (t == np2 - 1) counts[2] = flag[t];
}

// Thresholds from scal[1] and tau, then the K largest |S| above max(tau_c, tau_d) into w.keys (unsorted; count in
// w.counts[1]).  mad_mode >= 0: sigma_MAD of S (1: of |S|, 0: signed) is computed in the same launch first.
fpsk_status select_collect_launch(const float *S, int m_b, long long n1, long long n3, const float *d_tau, int radius, int K,
                                  int mad_mode, SelectWs &w, cudaStream_t st)
{
    if (K > kSelMaxK) K = kSelMaxK;
    const long long mm = (long long)m_b * m_b;
    // The K-th largest key does not depend on the thresholds, so its eight digits run beside the four of
    // the median and the four of the MAD (mad_mode 1: of |S|, 0: signed; < 0: sigma_MAD is already in place).
    const SelJob top = sel_job(SEL_TOPK, 64, S, mm, K);
    const SelJob med = sel_job(mad_mode ? SEL_ABS : SEL_SIGNED, 32, S, mm, 0);
    const SelJob dev = sel_job(mad_mode ? SEL_DEV_ABS : SEL_DEV_SIGNED, 32, S, mm, 0);
    // thresholds and collection ride at the end of the same launch (every CTA knows the K-th key and sigma_MAD there)
    SelCollect col;
    col.taup = d_tau; col.nmax = (float)(n1 > n3 ? n1 : n3); col.rad = (float)radius;
    return run_selects(top, med, mad_mode >= 0, dev, mad_mode >= 0, w, st, &col);
}

// The collected keys sorted and decoded into w.cand (count in w.counts[2]); moments from the sketches R, T or, when
// Rc is given, from the per-key values Rc, Tc.
fpsk_status decode_launch(const float *S, const float *R, const float *T, const float *Rc, const float *Tc, long long n1,
                          long long n3, SelectWs &w, cudaStream_t st, int *zero_word)
{
    int p1 = 0, p3 = 0;
    while ((1LL << p1) < n1) ++p1;
    while ((1LL << p3) < n3) ++p3;
    decode_kernel<<<1, kSelMaxK, 0, st>>>(S, R, T, Rc, Tc, p1, p3, w.keys, w.counts, kSelMaxK, w.cand, zero_word);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

fpsk_status select_candidates_launch(const float *S, const float *R, const float *T, int m_b, long long n1,
                                     long long n3, const float *d_tau, int radius, int K, int mad_mode, SelectWs &w,
                                     cudaStream_t st)
{
    fpsk_status rc = select_collect_launch(S, m_b, n1, n3, d_tau, radius, K, mad_mode, w, st);
    if (rc != FPSK_OK) return rc;
    return decode_launch(S, R, T, nullptr, nullptr, n1, n3, w, st);
}

// ---------------------------------------------------------------- max |X| of a half matrix
// max |x| over a half-precision matrix as a 16-bit pattern (sign cleared; for finite values the
// unsigned order of the patterns is the order of the magnitudes in both formats).
template <typename T>
__global__ void __launch_bounds__(256) max_abs_half_kernel(const unsigned short *X, long long ld, long long rows, long long cols,
                                                           int vec_ok, unsigned int *out)
{
    unsigned int m = 0;
    if (vec_ok) {
        const long long cv = cols / 8;               // 16-byte vectors per row
        const long long total = rows * cv;
        // four independent 16-byte loads in flight per thread
        const long long stride = (long long)gridDim.x * blockDim.x;
        for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < total; i0 += 4 * stride) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long i = i0 + u * stride;
                long long off = i * 8;                   // rows back to back: no division
                if (ld != cols) {
                    const long long r = i / cv;
                    off = r * ld + (i - r * cv) * 8;
                }
                v[u] = i < total ? ldg_nc_v4(X + off) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const unsigned int w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    m = max(m, (w[q] >> 16) & 0x7FFFu);
                    m = max(m, w[q] & 0x7FFFu);
                }
            }
        }
    } else {
        for (long long r = blockIdx.x; r < rows; r += gridDim.x)
            for (long long c = threadIdx.x; c < cols; c += blockDim.x) m = max(m, (unsigned int)(X[r * ld + c] & 0x7FFFu));
    }
    // one atomic per CTA: thousands of atomics on the one word took longer than reading the matrix
    __shared__ unsigned int wmax[8];
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < 8; ++w) m = max(m, wmax[w]);
        if (m) atomicMax(out, m);
    }
}
template <typename T>
__global__ void max_abs_finish_kernel(const unsigned int *bits, float *out)
{
    if (threadIdx.x == 0) out[0] = bits16_to_float<T>(bits[0]);
}

fpsk_status max_abs_half_launch(const void *X, long long ld, long long rows, long long cols, fpsk_dtype dtype,
                                float *out, unsigned int *scratch, cudaStream_t st)
{
    FPSK_CUDA_OK(cudaMemsetAsync(scratch, 0, 4, st));
    const unsigned short *x = static_cast<const unsigned short *>(X);
    const int vec_ok = ((reinterpret_cast<uintptr_t>(X) & 15) == 0 && ld % 8 == 0 && cols % 8 == 0) ? 1 : 0;
    long long want = vec_ok ? (rows * (cols / 8) + 256 * 4 - 1) / (256 * 4) : rows;
    const int grid = (int)(want < 1 ? 1 : (want > 1184 ? 1184 : want));
    if (dtype == FPSK_FP16) {
        max_abs_half_kernel<__half><<<grid, 256, 0, st>>>(x, ld, rows, cols, vec_ok, scratch);
        FPSK_LAUNCH_CHECK();
        max_abs_finish_kernel<__half><<<1, 32, 0, st>>>(scratch, out);
    } else {
        max_abs_half_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(x, ld, rows, cols, vec_ok, scratch);
        FPSK_LAUNCH_CHECK();
        max_abs_finish_kernel<__nv_bfloat16><<<1, 32, 0, st>>>(scratch, out);
    }
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- strided, clipped rms of C
__global__ void sample_c_kernel(const float *C, long long ldc, long long n3, long long total, long long stride,
                                long long nsamp, float *samples)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= nsamp) return;
    const long long flat = t * stride;
    const long long r = flat / n3, c = flat - r * n3;
    const float a = fabsf(C[r * ldc + c]);
    samples[t] = (a <= 3.402823466e38f) ? a : -1.f;      // sentinel for Inf / NaN
}

// single CTA, FP64 accumulation in a fixed order
__global__ void __launch_bounds__(1024) clipped_rms_kernel(const float *samples, long long nsamp, const float *scal,
                                                           const int *counts, float *out)
{
    __shared__ double sh[1024];
    const float clip = 64.f * scal[SC_SMED];
    double acc = 0.0;
    for (long long i = threadIdx.x; i < nsamp; i += 1024) {
        const float a = samples[i];
        if (a >= 0.f) {
            const double v = (double)fminf(a, clip);
            acc += v * v;
        }
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 512; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int n = counts[0];
        out[0] = n > 0 ? (float)sqrt(sh[0] / (double)n) : __uint_as_float(0x7FC00000u);
    }
}

// Strided samples of |C| (-1 marks Inf / NaN) and the number of valid ones -> counts[0]; returns the sample count
// (< 0: a launch failed).
long long rms_c_samples(const float *C, long long ldc, long long n1, long long n3, float *samples, SelectWs &w,
                        cudaStream_t st)
{
    const long long total = n1 * n3;
    long long stride = total / 65536;
    if (stride < 1) stride = 1;
    const long long nsamp = (total + stride - 1) / stride;
    sample_c_kernel<<<(unsigned)((nsamp + 255) / 256), 256, 0, st>>>(C, ldc, n3, total, stride, nsamp, samples);
    if (cudaGetLastError() != cudaSuccess) return -1;
    if (cudaMemsetAsync(w.counts, 0, 4 * 4, st) != cudaSuccess) return -1;
    count_valid_kernel<<<64, 256, 0, st>>>(SEL_SAMPLE, samples, nsamp, w.scal, w.counts);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return nsamp;
}

// sigma_MAD of S (median -> scal[0], 1.4826 MAD -> scal[1]) and the strided, clipped rms of C (-> out[0]) from
// one launch: the median of the samples of C in one slot, the median of S and then the median of the
// deviations in the other.
fpsk_status sigma_mad_rms_c_launch(const float *S, long long mm, int mad_of_abs, const float *C, long long ldc,
                                   long long n1, long long n3, float *samples, SelectWs &w, float *out, cudaStream_t st)
{
    const long long nsamp = rms_c_samples(C, ldc, n1, n3, samples, w, st);
    if (nsamp < 0) return FPSK_ERR_CUDA;
    return sigma_mad_rms_c_select_launch(S, mm, mad_of_abs, samples, nsamp, w, out, st);
}

// The second half of the above, for a caller that took the samples earlier (on another stream, joined since).
fpsk_status sigma_mad_rms_c_select_launch(const float *S, long long mm, int mad_of_abs, float *samples, long long nsamp,
                                          SelectWs &w, float *out, cudaStream_t st)
{
    const SelJob med = sel_job(mad_of_abs ? SEL_ABS : SEL_SIGNED, 32, S, mm, 0);
    const SelJob dev = sel_job(mad_of_abs ? SEL_DEV_ABS : SEL_DEV_SIGNED, 32, S, mm, 0);
    const SelJob smp = sel_job(SEL_SAMPLE, 32, samples, nsamp, 0);
    fpsk_status rc = run_selects(smp, med, true, dev, true, w, st);
    if (rc != FPSK_OK) return rc;
    clipped_rms_kernel<<<1, 1024, 0, st>>>(samples, nsamp, w.scal, w.counts, out);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// ---------------------------------------------------------------- workspace
size_t select_ws_bytes()
{
    return align_up(kHistBytes, 256) /*hist+tickets*/ + 256 /*state*/ + 256 /*scal*/ + align_up(kSumGrid * 4, 256) +
           align_up(kSelMaxK * 8, 256) + 256 /*counts*/ + align_up(kSelMaxK * sizeof(Candidate), 256) +
           2 * align_up(kSelMaxK * 4, 256) /*moments of the collected keys*/;
}

void select_carve(void *ws, SelectWs &w)
{
    char *p = static_cast<char *>(ws);
    w.hist = (unsigned int *)p; p += align_up(kHistBytes, 256);
    w.err = w.hist + kHistErr;
    w.state = (unsigned long long *)p; p += 256;
    w.scal = (float *)p; p += 256;
    w.partial = (float *)p; p += align_up(kSumGrid * 4, 256);
    w.keys = (unsigned long long *)p; p += align_up(kSelMaxK * 8, 256);
    w.counts = (int *)p; p += 256;
    w.cand = (Candidate *)p; p += align_up(kSelMaxK * sizeof(Candidate), 256);
    w.Rc = (float *)p; p += align_up(kSelMaxK * 4, 256);
    w.Tc = (float *)p;
    w.hist_clean = false;
}

}  // namespace fpsk
