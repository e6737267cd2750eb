// The S only probe at the probe's own bucket count (Section "The Cheap S Only Probe"):
//   S = (H1 A)(B H2^T) - H1 C H2^T,   sigma_hat, threshold and one-bit verdict (Section "Thresholds").
// The B side (hash round, bucket-sorted permutations, Q = B H2^T, max|B|, and the work list of the
// streaming kernel, which depends on the hash round only) is built once per weight tensor and kept
// by the caller; a call on a cached B reads A once and C once.
//
//   hp_rank_kernel, hp_count_chunks_kernel, hp_fill_stages_kernel, hp_segment_lists_kernel
//                           once per B side: the work list (for every (matrix, column segment, row bucket)
//                           unit the ring stages (rows, signs) that stream it, largest buckets first) and
//                           the per-segment column lists of the fold
//   hp_stream_kernel        P = H1 A (m x n2) and H1 C H2^T per column segment: signed row-bucket sums
//                           (and the column fold for C), one persistent CTA per SM, rows gathered by
//                           bulk copies into shared-memory rings
//   hp_rowsum_plain_kernel, hp_fold_plain_kernel
//                           the same with plain loads (inputs that bulk copies cannot address)
//   sgemm (sketch.cu) or tc_contract (tc_contract.cu)
//                           P Q as split-K partials: FP32 FMA, or split-FP16 on the tensor cores
//   hp_combine_kernel       S = sum of split-K partials - sum of segment partials, statistics, verdict
//   hp_stream_kernel<T, true>
//                           all of the above in one cooperative launch (tensor cores asked for, at most 256 buckets,
//                           inputs the bulk copies can address): A streams first and leaves as FP16 planes, the first
//                           CTAs contract P Q on the tensor cores while the others stream C, then every CTA combines
// Every sum has a fixed order (no float atomics): results are bit-reproducible.
#include "tc_ops.cuh"

#include <math.h>
#include <stdlib.h>
#include <mutex>
#include <type_traits>

namespace fpsk {

constexpr int kHpConsumers = 512;
constexpr int kHpTeamThreads = 256;               // consumer threads of one team
constexpr int kHpThreads = kHpConsumers + 64;     // + one producer warp per team
constexpr int kHpStages = 6;                      // ring stages per team
constexpr int kHpStageBytes = 16384;
constexpr int kHpPieceBytes = 4096;               // one row of one column segment
constexpr int kHpPieces = kHpStageBytes / kHpPieceBytes;
static_assert(kHpPieces == 4, "a stage record's row indices sit in one 16-byte lane word");
constexpr int kHpBarBytes = 512;                  // barrier block: ring barriers of both teams, consumer and team barriers, and those of the fused contraction
static_assert(2 * 2 * kHpStages * 8 + 8 + 16 + (2 * 4 + 3) * 8 + 8 <= kHpBarBytes, "barrier block");
constexpr int kHpSegA = kHpPieceBytes / 2;        // columns of A per segment
constexpr int kHpSegC = kHpPieceBytes / 4;        // columns of C per segment
constexpr int kHpFoldBytes = 2 * 2 * kHpSegC * 4; // per team, two buffers of one segment of row-bucket sums of C
constexpr int kHpSmem = 2 * kHpStages * kHpStageBytes + kHpFoldBytes + kHpBarBytes + 2 * kHpStages * 16 /*stage records*/;
constexpr int kHpTcStages = 4;                    // operand stages of the fused contraction: they take the place of the rings
static_assert(kHpTcStages * kTcStageBytes <= 2 * kHpStages * kHpStageBytes, "the contraction's stages fit in the rings");

struct HpArgs {
    const unsigned short *A;
    long long lda;
    const float *C;
    long long ldc;
    int n1, n2, n3, m, kpad;
    int segsA, segsC;              // column segments of A and of C
    const uint32_t *rowperm;       // rows sorted by bucket; bit 31 = sign -1
    const int *rowstart;           // [m + 1]
    const int *stages;             // chunks of 8 stage records, 16 ints per record:
                                   //   [0] bucket | isC << 30   [1] segment   [2] pieces | last-of-unit << 8 | signs << 16
                                   //   [4 .. 4 + pieces) row indices;  [15] of the chunk's last record: next chunk of the unit
                                   // chunk k is the first chunk of the k-th unit handed out; longer units continue in chunks >= units
    const uint32_t *segperm;       // per column segment of C: its columns (local index, bit 31 = sign -1) sorted by bucket
    const int *segstart;           // [segsC][m + 1] bucket boundaries in segperm, relative to the segment
    float *P;                      // m x kpad
    float *Tc;                     // m x n3 (plain-load path only)
    float *partC;                  // [segsC][m*m]: H1 C H2^T restricted to the columns of one segment
    unsigned int *maxA;            // per CTA: bits of max|A| over what it streamed
    unsigned int *ctrl;            // [0] verdict ticket, [1] error flag, [2] next unit to hand out, [3] statistics published;
                                   // fused kernel: [4] CTAs done with A, [5] next unit of C, [6] CTAs done streaming
    // ---- the fused kernel (stream, contraction on the tensor cores, combine and verdict in one launch)
    unsigned char *Pplanes;        // P = H1 A as tiled FP16 planes (A side: tiles of 128 buckets x 32 k), every (bucket, column
                                   // segment of A) scaled by its own power of two
    float *scaleP;                 // [m][segsA] those powers of two
    const unsigned char *Qplanes;  // Q^T as tiled FP16 planes (B side), one scale
    float *partAB;                 // [segsA * nsub][m * m] partial products, scaled
    int gm;                        // CTAs that contract once A is in (the first gm)
    int nsub;                      // K ranges per column segment of A: a range never spans two scales
    int kblocks;                   // K blocks of 32 in the planes
    int trace_on;
    unsigned long long *trace;     // measurement build, when trace_on: 32 words per CTA - [0, 16 G) eight stamps per team (entry, first
                                   // copy, through with A, first stage, end, hand-over done, contraction done, units), [16 G, 24 G)
                                   // eight per CTA of the combine, [24 G, 32 G) per contracting CTA: K blocks landed, tile ready, rows stored
};

// Units are (matrix, column segment, row bucket); all units of A go out before those of C.  A unit's rows go
// out in ring stages of up to kHpPieces rows; a stage never mixes units; an empty bucket still gets
// one stage (its sums are written as zeros).  Stage records come in chunks of eight, so that one
// warp-wide 16-byte load brings a whole chunk.
constexpr int kHpChunk = 8;

// Buckets ranked by row count, largest first (ties by index).  Units are handed out in rank order, so
// the last units to go out are the smallest and all teams finish close together.
__global__ void hp_rank_kernel(const int *rowstart, int m, int *rank)
{
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= m) return;
    const int rows = __ldg(rowstart + a + 1) - __ldg(rowstart + a);
    int r = 0;
    for (int o = 0; o < m; ++o) {
        const int ro = __ldg(rowstart + o + 1) - __ldg(rowstart + o);
        r += (ro > rows) || (ro == rows && o < a);
    }
    rank[a] = r;
}

// position of unit (isC, seg, a) in the hand-out order
__device__ __forceinline__ int hp_unit_pos(const HpArgs &p, const int *rank, bool isC, int seg, int a)
{
    // all units of A first (the fused kernel contracts as soon as P is complete), each matrix largest buckets first
    const int r = __ldg(rank + a);
    return isC ? p.m * p.segsA + r * p.segsC + seg : r * p.segsA + seg;
}

__global__ void hp_count_chunks_kernel(HpArgs p, const int *rank, int *extra)
{
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    const int UA = p.m * p.segsA, U = UA + p.m * p.segsC;
    if (u >= U) return;
    const bool isC = u >= UA;
    const int v = isC ? u - UA : u;
    const int seg = v / p.m, a = v - seg * p.m;
    const int rows = __ldg(p.rowstart + a + 1) - __ldg(p.rowstart + a);
    const int nst = rows > 0 ? (rows + kHpPieces - 1) / kHpPieces : 1;
    extra[hp_unit_pos(p, rank, isC, seg, a)] = (nst + kHpChunk - 1) / kHpChunk - 1;        // chunks beyond the first
}

__global__ void hp_fill_stages_kernel(HpArgs p, const int *rank, const int *extra_start, int *stages)
{
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    const int UA = p.m * p.segsA, U = UA + p.m * p.segsC;
    if (u >= U) return;
    const bool isC = u >= UA;
    const int v = isC ? u - UA : u;
    const int seg = v / p.m, a = v - seg * p.m;
    const int s0 = __ldg(p.rowstart + a), s1 = __ldg(p.rowstart + a + 1);
    const int nst = s1 > s0 ? (s1 - s0 + kHpPieces - 1) / kHpPieces : 1;
    const int nchunk = (nst + kHpChunk - 1) / kHpChunk;
    const int up = hp_unit_pos(p, rank, isC, seg, a);
    int pos = s0;
    for (int k = 0; k < nchunk; ++k) {
        const int ci = k == 0 ? up : U + extra_start[up] + (k - 1);
        for (int j = 0; j < kHpChunk; ++j) {
            int *rec = stages + ((long long)ci * kHpChunk + j) * 16;
            const int st = k * kHpChunk + j;
            for (int q = 0; q < 16; ++q) rec[q] = 0;
            if (st < nst) {
                const int np = min(kHpPieces, s1 - pos);
                unsigned int signs = 0;
                for (int q = 0; q < np; ++q) {
                    const uint32_t e = __ldg(p.rowperm + pos + q);
                    rec[4 + q] = (int)(e & 0x7FFFFFFFu);
                    signs |= (e >> 31) << q;
                }
                rec[0] = a | (isC ? (1 << 30) : 0);
                rec[1] = seg;
                rec[2] = np | (st == nst - 1 ? 0x100 : 0) | (int)(signs << 16);
                pos += np;
            }
            if (j == kHpChunk - 1) rec[15] = k + 1 < nchunk ? U + extra_start[up] + k : -1;
        }
    }
}

// Column lists of one segment of C (CTA = segment): the segment's columns sorted by bucket, stable in
// the column index, so that a bucket's fold adds its columns in ascending order.
__global__ void __launch_bounds__(256) hp_segment_lists_kernel(const int *h2, const int *v2, int n3, int m, uint32_t *segperm,
                                                               int *segstart)
{
    __shared__ int sh[kHpSegC];
    extern __shared__ int cnt[];                // m + 1
    const int seg = blockIdx.x;
    const int c0 = seg * kHpSegC, w = min(kHpSegC, n3 - c0);
    for (int j = threadIdx.x; j < w; j += blockDim.x) sh[j] = h2[c0 + j];
    for (int b = threadIdx.x; b <= m; b += blockDim.x) cnt[b] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < w; j += blockDim.x) atomicAdd(&cnt[sh[j]], 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int b = 0; b < m; ++b) {
            const int n = cnt[b];
            cnt[b] = run;
            run += n;
        }
        cnt[m] = run;
    }
    __syncthreads();
    for (int b = threadIdx.x; b <= m; b += blockDim.x) segstart[(long long)seg * (m + 1) + b] = cnt[b];
    for (int j = threadIdx.x; j < w; j += blockDim.x) {
        const int b = sh[j];
        int rank = 0;
        for (int i = 0; i < j; ++i) rank += (sh[i] == b);
        segperm[c0 + cnt[b] + rank] = (uint32_t)j | (v2[c0 + j] < 0 ? 0x80000000u : 0u);
    }
}

// Barrier over the consumer warps on an mbarrier (one arrival per warp), so that this wait is
// bounded like every other wait of the kernel.  Returns false when it gave up.
__device__ __forceinline__ bool hp_consumer_sync(uint32_t cbar, uint32_t &cpar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(cbar);
    const bool w = mbar_wait_warp(cbar, cpar);
    cpar ^= 1u;
    return w;
}

// The same over the eight consumer warps of one team.
__device__ __forceinline__ bool hp_team_sync(uint32_t tbar, uint32_t &tpar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(tbar);
    const bool w = mbar_wait_warp(tbar, tpar);
    tpar ^= 1u;
    return w;
}

__device__ __forceinline__ unsigned long long hp_gtime()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---------------------------------------------------------------- combine + verdict
struct HvArgs {
    const float *partAB;     // [ksplit][m*m]
    int ksplit;
    const float *partC;      // [nseg][m*m]
    int nseg;
    int m, n1, n2, n3;
    const unsigned int *maxA;
    int n_maxA;
    const float *maxB;       // [0] max|B|, [1] scale of the Q planes
    const float *scaleA;     // scale of the P planes when the partials come from the tensor cores, else null
    float thr_scale;         // mu sqrt(2 ln max(m^2, 2))
    float cap_scale;         // 1 (the printed rule), or sqrt(n1 n3 / m^2) when the caller asked for the scaled cap
    float *S;                // m*m
    float4 *vstat;           // per CTA: sum|S|, nonfinite count, max, argmax (as int bits)
    float *cstat;            // per CTA: sum of min(|S|, clip)
    unsigned int *ctrl;      // [0] ticket, [1] error flag, [2] unit counter of the streaming kernel, [3] statistics published,
                             // [4 .. 6] the fused kernel's phase counters
    fpsk_probe_result *result;
    fpsk_probe_state *state; // accumulated into when not null
    unsigned long long *ctrace;   // time stamps per CTA when tracing (8 each), else null
};

struct HvMax {
    float v;
    int i;
};
__device__ __forceinline__ HvMax hv_better(HvMax a, HvMax b)
{
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}

// One probe result into the running state (single thread; calls sharing a state are stream-ordered).
__device__ __forceinline__ void state_accumulate(fpsk_probe_state *st, const fpsk_probe_result &r)
{
    fpsk_probe_state s = *st;
    s.calls += 1;
    if (r.fired) {
        if (!s.fired_any) s.first_fired_call = s.calls;
        s.fired_any = 1;
    } else {
        s.clean_calls += 1;
        s.sigma_sum += (double)r.sigma_hat;
    }
    *st = s;
}

__global__ void state_accumulate_kernel(const fpsk_probe_result *r, fpsk_probe_state *st)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) state_accumulate(st, *r);
}

fpsk_status probe_accumulate_launch(const fpsk_probe_result *d_result, fpsk_probe_state *d_state, cudaStream_t st)
{
    state_accumulate_kernel<<<1, 32, 0, st>>>(d_result, d_state);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

constexpr int kHvThreads = 512;
constexpr int kHvWarps = kHvThreads / 32;
constexpr int kHvMaxGrid = 512;

struct HvStat {
    float sum, bad;
    HvMax mx;
};
__device__ __forceinline__ HvStat hv_join(HvStat a, HvStat b)
{
    HvStat r;
    r.sum = a.sum + b.sum;
    r.bad = a.bad + b.bad;
    r.mx = hv_better(a.mx, b.mx);
    return r;
}
// Block-wide combination in a fixed shape (butterfly inside a warp, then the warps in order): every
// thread returns the same value.  `slot` must hold kHvWarps entries; two uses need two slot arrays
// or a barrier between them.  Sync::sync() is the barrier over the kHvThreads threads that take part.
struct HvSyncCta {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};
struct HvSyncConsumers {    // the 512 consumer threads of the fused kernel (its producer warps are elsewhere)
    static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }
};
template <typename Sync>
__device__ __forceinline__ HvStat hv_block_join(HvStat v, HvStat *slot)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        HvStat w;
        w.sum = __shfl_xor_sync(0xFFFFFFFFu, v.sum, o);
        w.bad = __shfl_xor_sync(0xFFFFFFFFu, v.bad, o);
        w.mx.v = __shfl_xor_sync(0xFFFFFFFFu, v.mx.v, o);
        w.mx.i = __shfl_xor_sync(0xFFFFFFFFu, v.mx.i, o);
        // lower lane first: the same operand order in both partners
        v = (threadIdx.x & o) ? hv_join(w, v) : hv_join(v, w);
    }
    if ((threadIdx.x & 31) == 0) slot[threadIdx.x >> 5] = v;
    Sync::sync();
    HvStat r = slot[0];
#pragma unroll
    for (int w = 1; w < kHvWarps; ++w) r = hv_join(r, slot[w]);
    return r;
}

// Cooperative grid, CTA c owns a contiguous range of the m^2 buckets.
//   1. S = (split-K partials, in split order) - (segment partials of H1 C H2^T, in segment order);
//      per-CTA sum|S|, count of non-finite entries, max and argmax; publish (release) and wait
//      (bounded) for all CTAs.
//   2. every CTA forms the same total in the same order, hence the same clip level 5 mean|S|; when
//      some bucket exceeds it, it re-reads its own range of S (still in L2) for the clipped sum.
//   3. the last CTA to finish (ticket) adds the clipped sums in CTA order and writes the verdict.
template <typename T, typename Sync>
__device__ __forceinline__ void hv_combine_body(const HvArgs &p)
{
    __shared__ HvStat slot0[kHvWarps], slot1[kHvWarps], slot2[kHvWarps], slot3[kHvWarps];
    __shared__ unsigned int sma[kHvWarps];
    __shared__ int s_flag;
    const int c = blockIdx.x, G = gridDim.x, tid = threadIdx.x;
    const long long mm = (long long)p.m * p.m;
    // time stamps for FPSK_HPROBE_TRACE (0 entry, 1 partials loaded, 2 joined, 3 all published, 4 totals,
    // 5 clipped sum, 6 ticket, 7 verdict)
#define CT(k) do { if (p.ctrace && tid == 0) p.ctrace[c * 8 + (k)] = hp_gtime(); } while (0)
    CT(0);
    // ranges in units of 4 buckets (the tail CTA takes the remainder of an m^2 that is not a multiple of 4)
    const long long q4 = (mm + 3) / 4;
    const long long i0 = 4 * (q4 * c / G), i1 = min(mm, 4 * (q4 * (c + 1) / G));
    HvStat l = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
    const float unscale = p.scaleA ? 1.f / (__ldcg(p.scaleA) * __ldcg(p.maxB + 1)) : 1.f;      // powers of two: exact
    for (long long i = i0 + tid; i < i1; i += kHvThreads) {
        float ab = 0.f;
        for (int s0 = 0; s0 < p.ksplit; s0 += 8) {
            float v[8];                 // eight partials in flight, then added in split order
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = s0 + q < p.ksplit ? __ldcg(p.partAB + (long long)(s0 + q) * mm + i) : 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) ab += v[q];
        }
        ab *= unscale;
        float cf = 0.f;
        for (int s0 = 0; s0 < p.nseg; s0 += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = s0 + q < p.nseg ? __ldcg(p.partC + (long long)(s0 + q) * mm + i) : 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) cf += v[q];
        }
        const float sv = ab - cf;
        __stcg(p.S + i, sv);
        const float av = fabsf(sv);
        l.sum += av;
        if (!(av <= 3.4028234663852886e38f)) l.bad += 1.f;          // Inf or NaN
        else l.mx = hv_better(l.mx, HvMax{av, (int)i});
    }
    CT(1);
    l = hv_block_join<Sync>(l, slot0);
    CT(2);
    if (tid == 0) {
        __stcg(p.vstat + c, make_float4(l.sum, l.bad, l.mx.v, __int_as_float(l.mx.i)));
        red_release_add(p.ctrl + 3);
        s_flag = bounded_wait_ge(p.ctrl + 3, (unsigned)G) ? 1 : 0;
        if (!s_flag) atomicOr(p.ctrl + 1, 1u);
    }
    Sync::sync();
    CT(3);
    const bool ok = s_flag != 0;
    // ---- the same totals in every CTA: records in CTA order, thread-strided, then the fixed shape
    HvStat t = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
    if (ok) {
        for (int r = tid; r < G; r += kHvThreads) {
            const float4 v = __ldcg(p.vstat + r);
            t = hv_join(t, HvStat{v.x, v.y, {v.z, __float_as_int(v.w)}});
        }
    }
    t = hv_block_join<Sync>(t, slot1);
    CT(4);
    const float mean = t.sum / (float)mm;
    const bool slow = !(t.mx.v <= 5.f * mean) || t.bad > 0.f;
    if (slow) {
        const float clip = 5.f * mean;
        HvStat cs = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
        for (long long i = i0 + tid; i < i1; i += kHvThreads) cs.sum += fminf(fabsf(__ldcg(p.S + i)), clip);
        cs = hv_block_join<Sync>(cs, slot2);
        if (tid == 0) __stcg(p.cstat + c, cs.sum);
    }
    CT(5);
    if (tid == 0) {
        __threadfence();
        const unsigned int tk = atom_acq_rel_add(p.ctrl + 0);
        s_flag = (tk == (unsigned int)(G - 1)) ? 1 : 0;
    }
    Sync::sync();
    CT(6);
    if (!s_flag) return;
    __threadfence();
    // ---- last CTA
    float clipped = t.sum;
    if (slow) {
        HvStat cs = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
        for (int r = tid; r < G; r += kHvThreads) cs.sum += __ldcg(p.cstat + r);
        cs = hv_block_join<Sync>(cs, slot3);
        clipped = cs.sum;
    }
    unsigned int ma = 0;
    for (int r = tid; r < p.n_maxA; r += kHvThreads) ma = max(ma, __ldcg(p.maxA + r));
    ma = __reduce_max_sync(0xFFFFFFFFu, ma);
    if ((tid & 31) == 0) sma[tid >> 5] = ma;
    Sync::sync();
    if (tid == 0) {
        ma = 0;
        for (int w = 0; w < kHvWarps; ++w) ma = max(ma, sma[w]);
        const float sigma = 1.2533f * (clipped / (float)mm);
        const float tau = 100.f * (float)p.n2 * 1.1920928955078125e-07f * bits16_to_float<T>(ma) * __ldcg(p.maxB);
        // a bucket sums n1 n3 / m^2 entries of E on average: the per-entry cap grows like the root of that
        const float thr = fminf(tau * p.cap_scale, p.thr_scale * sigma);
        fpsk_probe_result r;
        r.nonfinite = t.bad > 0.f ? 1 : 0;
        r.fired = (t.bad > 0.f || t.mx.v > thr) ? 1 : 0;
        r.argmax_col = t.mx.v >= 0.f ? t.mx.i : -1;
        r.status = (!ok || __ldcg(p.ctrl + 1)) ? (int)FPSK_ERR_TIMEOUT : (int)FPSK_OK;
        r.max_abs = t.mx.v >= 0.f ? t.mx.v : 0.f;
        r.sigma_hat = sigma;
        r.thr = thr;
        r.tau = tau;
        *p.result = r;
        if (p.ctrace) p.ctrace[c * 8 + 7] = hp_gtime();
        if (p.state) state_accumulate(p.state, r);
        // counters ready for the next call on this workspace
        for (int q = 0; q < 8; ++q) p.ctrl[q] = 0;
    }
#undef CT
}

template <typename T>
__global__ void __launch_bounds__(kHvThreads) hp_combine_kernel(const HvArgs p)
{
    hv_combine_body<T, HvSyncCta>(p);
}

// The combine of the fused kernel (its 512 consumer threads): one grid-wide step instead of two.
//   1. as above, with all partials of a bucket in flight at once (they arrive unscaled): S, per-CTA sum|S|, non-finite
//      count, max and argmax; then the ticket.
//   2. the last CTA forms the totals in CTA order.  If no bucket exceeds the clip level 5 mean|S| the clipped sum is the
//      sum; otherwise it re-reads all of S (m^2 values, still in L2) itself, with many loads in flight.
template <typename T>
__device__ __forceinline__ void hv_combine_fused(const HvArgs &p)
{
    typedef HvSyncConsumers Sync;
    __shared__ HvStat slot0[kHvWarps], slot1[kHvWarps], slot2[kHvWarps];
    __shared__ unsigned int sma[kHvWarps];
    __shared__ int s_last;
    const int c = blockIdx.x, G = gridDim.x, tid = threadIdx.x;
    const long long mm = (long long)p.m * p.m;
#define CT(k) do { if (p.ctrace && tid == 0) p.ctrace[c * 8 + (k)] = hp_gtime(); } while (0)
    CT(0);
    const long long q4 = (mm + 3) / 4;
    const long long i0 = 4 * (q4 * c / G), i1 = min(mm, 4 * (q4 * (c + 1) / G));
    HvStat l = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
    for (long long i = i0 + tid; i < i1; i += kHvThreads) {
        float ab = 0.f, cf = 0.f;
        for (int s0 = 0; s0 < p.ksplit || s0 < 2 * p.nseg; s0 += 16) {
            float v[16], u[8];          // all in flight, then added in split and in segment order
#pragma unroll
            for (int q = 0; q < 16; ++q) v[q] = s0 + q < p.ksplit ? __ldcg(p.partAB + (long long)(s0 + q) * mm + i) : 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) u[q] = s0 / 2 + q < p.nseg ? __ldcg(p.partC + (long long)(s0 / 2 + q) * mm + i) : 0.f;
#pragma unroll
            for (int q = 0; q < 16; ++q) ab += v[q];
#pragma unroll
            for (int q = 0; q < 8; ++q) cf += u[q];
        }
        const float sv = ab - cf;
        __stcg(p.S + i, sv);
        const float av = fabsf(sv);
        l.sum += av;
        if (!(av <= 3.4028234663852886e38f)) l.bad += 1.f;          // Inf or NaN
        else l.mx = hv_better(l.mx, HvMax{av, (int)i});
    }
    CT(1);
    l = hv_block_join<Sync>(l, slot0);
    CT(2);
    if (tid == 0) {
        __stcg(p.vstat + c, make_float4(l.sum, l.bad, l.mx.v, __int_as_float(l.mx.i)));
        __threadfence();
        const unsigned int tk = atom_acq_rel_add(p.ctrl + 0);
        s_last = (tk == (unsigned int)(G - 1)) ? 1 : 0;
    }
    Sync::sync();
    CT(6);
    if (!s_last) return;
    // ---- last CTA (thread 0's ticket was an acquire and the barrier above passes it on to the other threads; the
    // records and S were stored to L2 and are loaded from there): totals in CTA order (thread-strided, then the fixed
    // shape), max|A|
    HvStat t = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
    for (int r = tid; r < G; r += kHvThreads) {
        const float4 v = __ldcg(p.vstat + r);
        t = hv_join(t, HvStat{v.x, v.y, {v.z, __float_as_int(v.w)}});
    }
    unsigned int ma = 0;
    for (int r = tid; r < p.n_maxA; r += kHvThreads) ma = max(ma, __ldcg(p.maxA + r));
    t = hv_block_join<Sync>(t, slot1);
    CT(4);
    const float mean = t.sum / (float)mm;
    const bool slow = !(t.mx.v <= 5.f * mean) || t.bad > 0.f;
    float clipped = t.sum;
    if (slow) {
        // all of S again (m^2 values, still in L2), eight 16-byte loads in flight per thread
        const float clip = 5.f * mean;
        HvStat cs = {0.f, 0.f, {-1.f, 0x7FFFFFFF}};
        const long long nq = (reinterpret_cast<uintptr_t>(p.S) & 15) ? 0 : mm / 4;      // a caller's S may be aligned to 4 bytes only
        const float4 *S4 = reinterpret_cast<const float4 *>(p.S);
        for (long long q0 = tid; q0 < nq; q0 += 8 * kHvThreads) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = q0 + (long long)u * kHvThreads < nq ? __ldcg(S4 + q0 + (long long)u * kHvThreads) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 8; ++u)
                cs.sum += (fminf(fabsf(v[u].x), clip) + fminf(fabsf(v[u].y), clip)) + (fminf(fabsf(v[u].z), clip) + fminf(fabsf(v[u].w), clip));
        }
        for (long long i = 4 * nq + tid; i < mm; i += kHvThreads) cs.sum += fminf(fabsf(__ldcg(p.S + i)), clip);
        cs = hv_block_join<Sync>(cs, slot2);
        clipped = cs.sum;
    }
    CT(5);
    ma = __reduce_max_sync(0xFFFFFFFFu, ma);
    if ((tid & 31) == 0) sma[tid >> 5] = ma;
    Sync::sync();
    if (tid == 0) {
        ma = 0;
        for (int w = 0; w < kHvWarps; ++w) ma = max(ma, sma[w]);
        const float sigma = 1.2533f * (clipped / (float)mm);
        const float tau = 100.f * (float)p.n2 * 1.1920928955078125e-07f * bits16_to_float<T>(ma) * __ldcg(p.maxB);
        const float thr = fminf(tau * p.cap_scale, p.thr_scale * sigma);
        fpsk_probe_result r;
        r.nonfinite = t.bad > 0.f ? 1 : 0;
        r.fired = (t.bad > 0.f || t.mx.v > thr) ? 1 : 0;
        r.argmax_col = t.mx.v >= 0.f ? t.mx.i : -1;
        r.status = __ldcg(p.ctrl + 1) ? (int)FPSK_ERR_TIMEOUT : (int)FPSK_OK;
        r.max_abs = t.mx.v >= 0.f ? t.mx.v : 0.f;
        r.sigma_hat = sigma;
        r.thr = thr;
        r.tau = tau;
        *p.result = r;
        if (p.ctrace) p.ctrace[c * 8 + 7] = hp_gtime();
        if (p.state) state_accumulate(p.state, r);
        for (int q = 0; q < 8; ++q) p.ctrl[q] = 0;       // counters ready for the next call on this workspace
    }
#undef CT
}

// One CTA per SM, two independent teams per CTA.  A team is one producer warp, eight consumer warps
// (256 threads x 16 bytes = one row piece) and its own ring of kHpStages stages; it takes whole
// units, so nothing is shared between teams.  Two producer warps matter: one warp issues a bulk
// copy about every 90 ns, which at 4 KB per copy is just the SM's share of the memory bandwidth.
//
// Units are handed out by a counter (ctrl[2]): a team that streams faster takes more of them, so
// all teams finish together whatever their share of the memory system.  Which team sums a unit
// does not change the sum (fixed order inside the unit).  The producer asks the counter for the next unit when
// it starts one and sends for that unit's stage records half way through, so no round trip to L2 sits between
// two units and a team never holds more than the unit it streams and one more.
//
// FUSED (cooperative launch): the whole probe in this one kernel.
//   1. The units of A go out first; a finished unit of A is written as the two FP16 planes of the tensor-core
//      contraction, scaled by a power of two of its own (bucket, column segment), not as FP32.
//   2. When a CTA has no unit of A left it publishes (ctrl[4]).  The first gm CTAs then wait (bounded) for all CTAs,
//      i.e. for the whole of P, and contract: their rings become the operand stages, one producer warp brings the
//      plane tiles of P and of Q^T with bulk copies, the other issues the tcgen05 MMAs of a (row tile, K range)
//      item into TMEM, four consumer warps store the partial.  Meanwhile the other CTAs stream C; the gm CTAs
//      join them when their items are done.
//   3. When the units of C are exhausted every CTA publishes (ctrl[6]) and waits (bounded) for all others; the
//      consumer threads then run the combine (partials in K order, each undone by its scales, minus the segment
//      partials of H1 C H2^T; statistics; verdict by the last CTA) exactly as hp_combine_kernel does.
// The sums are the same whichever CTA does them: results stay bit-reproducible.
// Barrier over all 18 warps of the CTA on an mbarrier (one arrival per warp): bounded like every other wait.
__device__ __forceinline__ bool hp_cta_sync(uint32_t pbar, uint32_t &ppar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(pbar);
    const bool w = mbar_wait_warp(pbar, ppar);
    ppar ^= 1u;
    return w;
}

template <typename T, bool FUSED>
__global__ void __launch_bounds__(kHpThreads, 1) hp_stream_kernel(const HpArgs p, const HvArgs hv)
{
    extern __shared__ __align__(128) unsigned char smem[];
    float *fold_all = reinterpret_cast<float *>(smem + 2 * kHpStages * kHpStageBytes);
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + 2 * kHpStages * kHpStageBytes + kHpFoldBytes);
    int *recs_all = reinterpret_cast<int *>(smem + 2 * kHpStages * kHpStageBytes + kHpFoldBytes + kHpBarBytes);
    __shared__ unsigned int smx[kHpConsumers / 32];
    __shared__ float smxf[2 * (kHpConsumers / 32)];     // warp maxima of a finished unit of A, two buffers
    __shared__ int s_go;
    const int c = blockIdx.x;
    const int G = (int)gridDim.x;
    const int tid = threadIdx.x;
    const bool tr = p.trace_on != 0;
    const int team = tid < kHpConsumers ? tid >> 8 : (tid - kHpConsumers) >> 5;
    unsigned char *ring = smem + (size_t)team * kHpStages * kHpStageBytes;
    int *recs = recs_all + team * kHpStages * 4;
    const uint32_t full0 = smem_u32(bars) + team * (2 * kHpStages * 8), empty0 = full0 + kHpStages * 8;
    const uint32_t cbar = smem_u32(bars) + 2 * (2 * kHpStages * 8);
    const uint32_t tbar = cbar + 8 + 8 * team;           // barrier over the team's consumer warps
    // fused contraction: operand stages full / empty, accumulator ready / read, CTA barrier, TMEM address
    const uint32_t kfull0 = cbar + 24, kempty0 = kfull0 + 8 * kHpTcStages, accb = kempty0 + 8 * kHpTcStages, accfree = accb + 8,
                   pbar = accfree + 8;
    uint32_t *tslot = reinterpret_cast<uint32_t *>(bars) + (24 + 2 * (2 * kHpStages * 8) + (2 * kHpTcStages + 3) * 8) / 4;
    if (tid == 0) {
        for (int s = 0; s < 2 * kHpStages; ++s) {
            const int tm = s / kHpStages, ss = s % kHpStages;
            mbar_init(smem_u32(bars) + tm * (2 * kHpStages * 8) + 8 * ss, 1);
            mbar_init(smem_u32(bars) + tm * (2 * kHpStages * 8) + kHpStages * 8 + 8 * ss, kHpTeamThreads / 32);
        }
        mbar_init(cbar, kHpConsumers / 32);
        mbar_init(cbar + 8, kHpTeamThreads / 32);
        mbar_init(cbar + 16, kHpTeamThreads / 32);
        if (FUSED) {
            for (int s = 0; s < kHpTcStages; ++s) {
                mbar_init(kfull0 + 8 * s, 1);
                mbar_init(kempty0 + 8 * s, 1);
            }
            mbar_init(accb, 1);
            mbar_init(accfree, 4);
            mbar_init(pbar, kHpThreads / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tr && (tid == 0 || tid == kHpTeamThreads)) p.trace[(c * 2 + team) * 8 + 0] = hp_gtime();
    const int UA = p.m * p.segsA, U = UA + p.m * p.segsC;
    const bool contractor = FUSED && c < p.gm;
    uint32_t ppar = 0;

    if (tid >= kHpConsumers) {
        // ------------------------------------------------------------ producer warp of the team
        const int lane = tid & 31;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        bool first = true;
        const int4 *chunks = reinterpret_cast<const int4 *>(p.stages);
        const int4 zero4 = make_int4(0, 0, 0, 0);
        // One empty stage whose record is `mark` (-1: end of work, -2: no more units of A).
        auto send_mark = [&](int mark) {
            int w = 1;
            if (lane == 0) w = mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u) ? 1 : 0;
            w = __shfl_sync(0xFFFFFFFFu, w, 0);
            if (!w) { ok = false; return; }
            if (lane == 0) {
                recs[stage * 4] = mark;
                mbar_arrive(full0 + 8 * stage);
            }
            if (++stage == kHpStages) { stage = 0; phase ^= 1u; }
        };
        // Streams units below u_end, starting with uA; the unit after each is taken from the counter (base + old value)
        // when its predecessor starts, and its first chunk of stage records (lane l holds 16 bytes: ints 4 (l % 4) .. of
        // record l / 4) is sent for half way through the predecessor, when the counter's answer has long arrived.  So a
        // team holds the unit it streams and one more: what is left over when the counter runs out is one unit per team.
        auto stream_units = [&](int uA, int u_end, unsigned int *ctr, int base) {
            int4 RA = uA < u_end ? __ldg(chunks + (long long)uA * 32 + lane) : zero4;
            while (uA < u_end && ok) {
                int uB = 0;
                if (lane == 0) uB = base + (int)atomicAdd(ctr, 1u);
                int4 RB = zero4;
                bool haveB = false;
                int4 R = RA;
                for (;;) {
                    const unsigned int lastmask = __ballot_sync(0xFFFFFFFFu, (lane & 3) == 0 && (R.z & 0x100));
                    const int nxt = __shfl_sync(0xFFFFFFFFu, R.w, 31);
                    int4 Rn = zero4;
                    if (!lastmask && nxt >= 0) Rn = __ldg(chunks + (long long)nxt * 32 + lane);    // continuation, in flight meanwhile
                    const int jn = lastmask ? ((__ffs(lastmask) - 1) >> 2) + 1 : kHpChunk;
                    for (int j = 0; j < jn; ++j) {
                        if (!haveB && 2 * j >= jn) {
                            uB = __shfl_sync(0xFFFFFFFFu, uB, 0);
                            if (uB < u_end) RB = __ldg(chunks + (long long)uB * 32 + lane);
                            haveB = true;
                        }
                        const int h0 = __shfl_sync(0xFFFFFFFFu, R.x, 4 * j), h1 = __shfl_sync(0xFFFFFFFFu, R.y, 4 * j),
                                  h2 = __shfl_sync(0xFFFFFFFFu, R.z, 4 * j);
                        const int src = 4 * j + 1;                  // ints 4..7 of record j: the row indices
                        const int v0 = __shfl_sync(0xFFFFFFFFu, R.x, src), v1 = __shfl_sync(0xFFFFFFFFu, R.y, src),
                                  v2 = __shfl_sync(0xFFFFFFFFu, R.z, src), v3 = __shfl_sync(0xFFFFFFFFu, R.w, src);
                        const int row = (lane & 2) ? ((lane & 1) ? v3 : v2) : ((lane & 1) ? v1 : v0);
                        const int np = h2 & 0xFF;
                        const bool isC = (h0 >> 30) != 0;
                        const int seg = h1;
                        const int wbytes = isC ? 4 * min(kHpSegC, p.n3 - seg * kHpSegC) : 2 * min(kHpSegA, p.n2 - seg * kHpSegA);
                        const unsigned char *base_p = isC ? reinterpret_cast<const unsigned char *>(p.C + (long long)seg * kHpSegC)
                                                          : reinterpret_cast<const unsigned char *>(p.A + (long long)seg * kHpSegA);
                        const long long ldb = isC ? p.ldc * 4 : p.lda * 2;
                        int w = 1;
                        if (lane == 0) w = mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u) ? 1 : 0;
                        w = __shfl_sync(0xFFFFFFFFu, w, 0);
                        if (!w) { ok = false; break; }
                        if (lane == 0) {
                            *reinterpret_cast<int4 *>(recs + stage * 4) = make_int4(h0, h1, h2, 0);
                            if (np > 0) mbar_expect_tx(full0 + 8 * stage, (uint32_t)np * (uint32_t)wbytes);
                            else mbar_arrive(full0 + 8 * stage);
                        }
                        __syncwarp();
                        if (tr && lane == 0 && first) { p.trace[(c * 2 + team) * 8 + 1] = hp_gtime(); first = false; }
                        if (lane < np) {
                            // a row index or a segment out of range (bounds-checked build): row 0 of segment 0 is copied
                            // instead, so that the stage still completes
                            const bool in = FPSK_IN_BOUNDS(row, p.n1) && FPSK_IN_BOUNDS(seg, isC ? p.segsC : p.segsA);
                            const unsigned char *src = in ? base_p + (long long)row * ldb
                                                          : (isC ? reinterpret_cast<const unsigned char *>(p.C) : reinterpret_cast<const unsigned char *>(p.A));
                            bulk_g2s(smem_u32(ring + (size_t)stage * kHpStageBytes) + (uint32_t)lane * kHpPieceBytes, src, (uint32_t)wbytes,
                                     full0 + 8 * stage);
                        }
                        if (++stage == kHpStages) { stage = 0; phase ^= 1u; }
                    }
                    if (lastmask || !ok || nxt < 0) break;
                    R = Rn;
                }
                if (!haveB) {
                    uB = __shfl_sync(0xFFFFFFFFu, uB, 0);
                    if (uB < u_end) RB = __ldg(chunks + (long long)uB * 32 + lane);
                }
                uA = uB; RA = RB;
            }
        };
        // the first unit of every team is fixed (no round trip to the counter before the first copy);
        // the counter hands out the units after those
        const int nteams = 2 * G;
        // One call site of stream_units (it must stay inlined: its ring position lives in registers): the fused kernel
        // comes by twice, for A and for C, with the contraction in between on the first gm CTAs.
        int ph_u0 = 2 * c + team, ph_end = FUSED ? UA : U, ph_base = nteams;
        unsigned int *ph_ctr = p.ctrl + 2;
        for (int ph = 0; ph < (FUSED ? 2 : 1) && ok; ++ph) {
          if (FUSED && ph == 1) {
            send_mark(-2);
            if (!ok) break;
            const int nteamsB = 2 * (G - p.gm);            // teams that go straight on to C: their first unit is fixed
            ph_end = U; ph_ctr = p.ctrl + 5; ph_base = UA + nteamsB;
            if (contractor) {
                // ---- contraction: this warp is the operand producer (team 0) or the MMA issuer (team 1)
                __syncwarp();
                if (team == 1) {
                    tc_alloc(smem_u32(tslot), kTcCols);
                    tc_relinquish();
                    tc_fence_before();
                }
                bool live = hp_cta_sync(pbar, ppar);          // both teams of this CTA are through with A: the rings are free
                const int mtiles = (p.m + kTcBM - 1) / kTcBM;
                const int nitems = mtiles * p.segsA * p.nsub;
                const int kb_seg = kHpSegA / kTcBK;             // K blocks per column segment of A
                const int kb_sub = kb_seg / p.nsub;
                int kst = 0;
                uint32_t kph = 0;
                // While the other CTAs finish A: the Q^T tiles of the first K blocks, which do not depend on A
                int pre = 0;
                if (live && team == 0 && c < nitems) {
                    const int pl = c / mtiles;
                    const int kb0 = (pl / p.nsub) * kb_seg + (pl % p.nsub) * kb_sub, kb1 = min(p.kblocks, kb0 + kb_sub);
                    pre = max(0, min(kHpTcStages, kb1 - kb0));
                    for (int q = 0; q < pre; ++q) {
                        if (lane == 0) mbar_expect_tx(kfull0 + 8 * q, kTcStageBytes);
                        __syncwarp();
                        if (lane >= 2 && lane < 6)
                            bulk_g2s(smem_u32(smem + (size_t)q * kTcStageBytes + (size_t)lane * 8192),
                                     p.Qplanes + (size_t)(kb0 + q) * kTcPlanes * kTcTileB + (size_t)(lane - 2) * 8192, 8192, kfull0 + 8 * q);
                    }
                }
                live = hp_cta_sync(pbar, ppar) && live;       // P complete (the consumers' thread 0 has waited for it), TMEM address written
                tc_fence_after();
                const uint32_t tmem = *tslot;
                live = live && s_go != 0;
                if (live && team == 0) {
                    asm volatile("fence.proxy.async;" ::: "memory");      // the planes were written by ordinary stores of other CTAs
                    for (int it = c; it < nitems && live; it += p.gm) {
                        const int mt = it % mtiles, pl = it / mtiles;     // pl = seg * nsub + sub
                        const int kb0 = (pl / p.nsub) * kb_seg + (pl % p.nsub) * kb_sub, kb1 = min(p.kblocks, kb0 + kb_sub);
                        for (int kb = kb0; kb < kb1; ++kb) {
                            const bool early = it == c && kb - kb0 < pre;       // stage armed and Q^T on its way since before
                            if (!early) {
                                int w = 1;
                                if (lane == 0) w = mbar_wait_bounded(kempty0 + 8 * kst, kph ^ 1u) ? 1 : 0;
                                w = __shfl_sync(0xFFFFFFFFu, w, 0);
                                if (!w) { live = false; break; }
                                if (lane == 0) mbar_expect_tx(kfull0 + 8 * kst, kTcStageBytes);
                                __syncwarp();
                            }
                            if (lane < 6 && !(early && lane >= 2)) {
                                // six copies of 8 KB in flight: lanes 0, 1 the planes of the P tile, lanes 2 .. 5 those of the
                                // Q^T tile; both tiles are contiguous in memory in the order the stage holds them
                                const unsigned char *src = lane < 2 ? p.Pplanes + ((size_t)mt * p.kblocks + kb) * kTcPlanes * kTcTileA + (size_t)lane * 8192
                                                                    : p.Qplanes + (size_t)kb * kTcPlanes * kTcTileB + (size_t)(lane - 2) * 8192;
                                bulk_g2s(smem_u32(smem + (size_t)kst * kTcStageBytes + (size_t)lane * 8192), src, 8192, kfull0 + 8 * kst);
                            }
                            if (++kst == kHpTcStages) { kst = 0; kph ^= 1u; }
                        }
                    }
                    if (!live && lane == 0) atomicOr(p.ctrl + 1, 1u);
                } else if (live) {
                    // instruction descriptor: FP32 accumulator, FP16 x FP16, both K-major, N = 256, M = 128
                    const uint32_t idesc = (1u << 4) | ((uint32_t)(kTcBN >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
                    uint32_t fph = 0;
                    for (int it = c; it < nitems && live; it += p.gm) {
                        const int pl = it / mtiles;
                        const int kb0 = (pl / p.nsub) * kb_seg + (pl % p.nsub) * kb_sub, kb1 = min(p.kblocks, kb0 + kb_sub);
                        if (it != c) {
                            // the accumulator of the previous item has been read
                            int w = 1;
                            if (lane == 0) w = mbar_wait_bounded(accfree, fph) ? 1 : 0;
                            w = __shfl_sync(0xFFFFFFFFu, w, 0);
                            fph ^= 1u;
                            if (!w) { live = false; break; }
                            tc_fence_after();
                        }
                        uint32_t acc = 0;
                        for (int kb = kb0; kb < kb1; ++kb) {
                            int w = 1;
                            if (lane == 0) w = mbar_wait_bounded(kfull0 + 8 * kst, kph) ? 1 : 0;
                            w = __shfl_sync(0xFFFFFFFFu, w, 0);
                            if (!w) { live = false; break; }
                            tc_fence_after();
                            if (tr && lane == 0 && kb - kb0 < 8) p.trace[(size_t)G * 24 + c * 8 + (kb - kb0)] = hp_gtime();
                            if (lane == 0) {
                                const uint32_t sbase = smem_u32(smem + (size_t)kst * kTcStageBytes);
                                const int pairA[3] = {1, 0, 0}, pairB[3] = {0, 1, 0};      // (lo,hi) (hi,lo) (hi,hi): small weights first
#pragma unroll
                                for (int kstep = 0; kstep < kTcBK / 16; ++kstep) {
#pragma unroll
                                    for (int q = 0; q < 3; ++q) {
                                        const uint32_t sa = sbase + pairA[q] * kTcTileA + kstep * 2 * (kTcBM / 8) * 128;
                                        const uint32_t sb = sbase + kTcPlanes * kTcTileA + pairB[q] * kTcTileB + kstep * 2 * (kTcBN / 8) * 128;
                                        tc_mma(tmem, tc_smem_desc(sa, (kTcBM / 8) * 128, 128), tc_smem_desc(sb, (kTcBN / 8) * 128, 128), idesc, acc);
                                        acc = 1;
                                    }
                                }
                                tc_commit(kempty0 + 8 * kst);       // the stage is free once these MMAs have read it
                            }
                            __syncwarp();
                            if (++kst == kHpTcStages) { kst = 0; kph ^= 1u; }
                        }
                        if (tr && lane == 0) p.trace[(c * 2 + 1) * 8 + 3] = hp_gtime();
                        if (lane == 0) tc_commit(accb);             // arrives when every MMA issued above is complete
                        __syncwarp();
                    }
                    if (!live && lane == 0) atomicOr(p.ctrl + 1, 1u);
                }
                hp_cta_sync(pbar, ppar);                      // the tile of a single item stands in shared memory
                hp_cta_sync(pbar, ppar);                      // partials stored, operand stages idle: the rings are rings again
                if (team == 1) {
                    tc_fence_after();
                    tc_dealloc(tmem, kTcCols);
                }
                int u0 = 0;
                if (lane == 0) u0 = ph_base + (int)atomicAdd(p.ctrl + 5, 1u);
                ph_u0 = __shfl_sync(0xFFFFFFFFu, u0, 0);
            } else {
                ph_u0 = UA + 2 * (c - p.gm) + team;
            }
          }
          stream_units(ph_u0, ph_end, ph_ctr, ph_base);
        }
        if (ok) send_mark(-1);                                // end of work
        if (tr && lane == 0 && !FUSED) p.trace[(c * 2 + team) * 8 + 2] = hp_gtime();
        if (!ok && lane == 0) atomicOr(p.ctrl + 1, 1u);
    } else {
        // ------------------------------------------------------------ consumer warps of the team
        const int tc = tid & (kHpTeamThreads - 1);     // 256 x 16 B across a piece
        const int warp = tid >> 5, lane = tid & 31;
        int stage = 0;
        uint32_t phase = 0, cpar = 0, tpar = 0;
        unsigned int nunit = 0, ncunit = 0, naunit = 0;
        bool ok = true;
        bool first = true;
        float *fold = fold_all + team * (2 * kHpSegC);
        const long long mm2 = (long long)p.m * p.m;
        MinMax2<T> mm;
        mm.init();
        // The fused kernel runs the streaming loop twice, for A and for C, with the hand-over of P (and on the first gm
        // CTAs the contraction) in between; little is live across that, so the loop is compiled as it is without it.
        for (int ph = 0; ph < (FUSED ? 2 : 1) && ok; ++ph) {
          bool fresh = true;                             // the next stage opens a unit
          int fs0 = 0, fs1 = 0;                          // this thread's first bucket in the open C unit's segment list
          float2 acc[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
          bool switch_now = false;
          for (;;) {
            if (!mbar_wait_warp(full0 + 8 * stage, phase)) { ok = false; break; }
            if (tr && first && tc == 0) { p.trace[(c * 2 + team) * 8 + 3] = hp_gtime(); first = false; }
            const int4 r = *reinterpret_cast<const int4 *>(recs + stage * 4);
            if (r.x == -1) break;
            if (FUSED && r.x == -2) {
                // ---- no unit of A is left for this team
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (++stage == kHpStages) { stage = 0; phase ^= 1u; }
                switch_now = true;
                break;
            }
            const int a = r.x & 0x3FFFFFFF;
            const bool isC = (r.x >> 30) != 0;
            const int seg = r.y;
            const int np = r.z & 0xFF;
            const bool last = (r.z & 0x100) != 0;
            const unsigned int sg = ((unsigned int)r.z) >> 16;
            const int wbytes = isC ? 4 * min(kHpSegC, p.n3 - seg * kHpSegC) : 2 * min(kHpSegA, p.n2 - seg * kHpSegA);
            const bool active = tc * 16 < wbytes;
            if (fresh && isC && tc < p.m) {
                // needed when the unit is complete: in flight while its rows stream
                fs0 = __ldg(p.segstart + (long long)seg * (p.m + 1) + tc);
                fs1 = __ldg(p.segstart + (long long)seg * (p.m + 1) + tc + 1);
            }
            fresh = false;
            if (active) {
                const unsigned char *sb = ring + (size_t)stage * kHpStageBytes + tc * 16;
                if (np == kHpPieces) {
                    // full stage: all loads in flight before the first use
                    if (isC) {
                        float4 x[kHpPieces];
#pragma unroll
                        for (int q = 0; q < kHpPieces; ++q) x[q] = *reinterpret_cast<const float4 *>(sb + q * kHpPieceBytes);
#pragma unroll
                        for (int q = 0; q < kHpPieces; ++q) {
                            const float f = ((sg >> q) & 1u) ? -1.f : 1.f;
                            acc[0] = __ffma2_rn(make_float2(f, f), make_float2(x[q].x, x[q].y), acc[0]);
                            acc[1] = __ffma2_rn(make_float2(f, f), make_float2(x[q].z, x[q].w), acc[1]);
                        }
                    } else {
                        uint4 x[kHpPieces];
#pragma unroll
                        for (int q = 0; q < kHpPieces; ++q) x[q] = *reinterpret_cast<const uint4 *>(sb + q * kHpPieceBytes);
#pragma unroll
                        for (int q = 0; q < kHpPieces; ++q) {
                            const uint32_t flip = ((sg >> q) & 1u) ? 0x80008000u : 0u;
                            x[q].x ^= flip; x[q].y ^= flip; x[q].z ^= flip; x[q].w ^= flip;
                            add8m<T>(acc, x[q], mm);
                        }
                    }
                } else if (isC) {
#pragma unroll
                    for (int q = 0; q < kHpPieces; ++q) {
                        if (q < np) {
                            const float4 x = *reinterpret_cast<const float4 *>(sb + q * kHpPieceBytes);
                            const float f = ((sg >> q) & 1u) ? -1.f : 1.f;
                            acc[0] = __ffma2_rn(make_float2(f, f), make_float2(x.x, x.y), acc[0]);
                            acc[1] = __ffma2_rn(make_float2(f, f), make_float2(x.z, x.w), acc[1]);
                        }
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < kHpPieces; ++q) {
                        if (q < np) {
                            uint4 x = *reinterpret_cast<const uint4 *>(sb + q * kHpPieceBytes);
                            const uint32_t flip = ((sg >> q) & 1u) ? 0x80008000u : 0u;
                            x.x ^= flip; x.y ^= flip; x.z ^= flip; x.w ^= flip;
                            add8m<T>(acc, x, mm);
                        }
                    }
                }
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(empty0 + 8 * stage);
            if (++stage == kHpStages) { stage = 0; phase ^= 1u; }
            if (last) {
                // unit complete (a bucket or a segment out of range, bounds-checked build: its sums are dropped)
                const bool unit_ok = FPSK_IN_BOUNDS(a, p.m) && FPSK_IN_BOUNDS(seg, isC ? p.segsC : p.segsA);
                if (!unit_ok) {
                    if (isC) ++ncunit; else ++naunit;
                } else if (isC) {
                    // the segment's signed row-bucket sums go through shared memory; thread b then folds the
                    // columns of bucket b (ascending) into partC[seg][a][b].  Two buffers: the barrier of
                    // the next C unit separates this unit's reads from the writes of the one after.
                    float *tb = fold + (ncunit & 1u) * kHpSegC;
                    if (active) *reinterpret_cast<float4 *>(tb + tc * 4) = make_float4(acc[0].x, acc[0].y, acc[1].x, acc[1].y);
                    if (!hp_team_sync(tbar, tpar)) { ok = false; break; }
                    const uint32_t *sp = p.segperm + (long long)seg * kHpSegC;
                    float *dst = p.partC + (long long)seg * mm2 + (long long)a * p.m;
                    for (int b = tc; b < p.m; b += kHpTeamThreads) {
                        int s0 = fs0, s1 = fs1;
                        if (b != tc) {
                            s0 = __ldg(p.segstart + (long long)seg * (p.m + 1) + b);
                            s1 = __ldg(p.segstart + (long long)seg * (p.m + 1) + b + 1);
                        }
                        float cf = 0.f;
                        for (int s = s0; s < s1; s += 4) {
                            uint32_t e[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) e[q] = s + q < s1 ? __ldg(sp + s + q) : 0u;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t ci = e[q] & 0x7FFFFFFFu;
                                const float x = FPSK_IN_BOUNDS(ci, kHpSegC) ? tb[ci] : 0.f;
                                if (s + q < s1) cf += (e[q] >> 31) ? -x : x;
                            }
                        }
                        __stcg(dst + b, cf);
                    }
                    ++ncunit;
                } else if (FUSED) {
                    // the unit's sums as the two FP16 planes of the contraction, under the power of two that brings
                    // this (bucket, column segment) below 2^13; two buffers of warp maxima, as for the fold above
                    float mx = fmaxf(fmaxf(fmaxf(fabsf(acc[0].x), fabsf(acc[0].y)), fmaxf(fabsf(acc[1].x), fabsf(acc[1].y))),
                                     fmaxf(fmaxf(fabsf(acc[2].x), fabsf(acc[2].y)), fmaxf(fabsf(acc[3].x), fabsf(acc[3].y))));
                    bool bad = !(mx <= 3.4028234663852886e38f);          // NaN or Inf among this thread's sums
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
                    bad = __any_sync(0xFFFFFFFFu, bad);
                    float *wm = smxf + (naunit & 1u) * (kHpConsumers / 32);
                    if (lane == 0) wm[warp] = bad ? __int_as_float(0x7F800000) : mx;
                    if (!hp_team_sync(tbar, tpar)) { ok = false; break; }
                    float umax = 0.f;
#pragma unroll
                    for (int w = 0; w < kHpTeamThreads / 32; ++w) umax = fmaxf(umax, wm[team * (kHpTeamThreads / 32) + w]);
                    const float scale = tc_scale_of(1, umax);            // 1 for a zero or non-finite unit
                    const int col = seg * kHpSegA + tc * 8;
                    if (col < p.kblocks * kTcBK) {                       // inactive columns below that: zero padding of the K extent
                        const float x[8] = {acc[0].x, acc[0].y, acc[1].x, acc[1].y, acc[2].x, acc[2].y, acc[3].x, acc[3].y};
                        unsigned short h[8], l[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float xs = x[j] * scale;
                            const __half bh = __float2half_rn(xs);
                            const __half bl = __float2half_rn(xs - __half2float(bh));      // the remainder is exact in FP32
                            h[j] = __half_as_ushort(bh);
                            l[j] = __half_as_ushort(bl);
                        }
                        const int rt = a / kTcBM, rr = a % kTcBM, kbi = col / kTcBK, kc = (col % kTcBK) / 8;
                        unsigned char *out = p.Pplanes + ((size_t)rt * p.kblocks + kbi) * kTcPlanes * kTcTileA +
                                             (size_t)(kc * (kTcBM / 8) + rr / 8) * 128 + (size_t)(rr % 8) * 16;
                        __stcg(reinterpret_cast<uint4 *>(out), make_uint4(h[0] | ((unsigned)h[1] << 16), h[2] | ((unsigned)h[3] << 16),
                                                                          h[4] | ((unsigned)h[5] << 16), h[6] | ((unsigned)h[7] << 16)));
                        __stcg(reinterpret_cast<uint4 *>(out + kTcTileA), make_uint4(l[0] | ((unsigned)l[1] << 16), l[2] | ((unsigned)l[3] << 16),
                                                                                     l[4] | ((unsigned)l[5] << 16), l[6] | ((unsigned)l[7] << 16)));
                    }
                    if (tc == 0) __stcg(p.scaleP + (long long)a * p.segsA + seg, scale);
                    ++naunit;
                } else {
                    const int col = seg * kHpSegA + tc * 8;
                    if (active || col < p.kpad) {        // inactive columns below kpad: padding of the contraction's K extent (zeros)
                        float4 *dst = reinterpret_cast<float4 *>(p.P + (long long)a * p.kpad + col);
                        __stcg(dst, make_float4(acc[0].x, acc[0].y, acc[1].x, acc[1].y));
                        __stcg(dst + 1, make_float4(acc[2].x, acc[2].y, acc[3].x, acc[3].y));
                    }
                }
                ++nunit;
                fresh = true;
                acc[0] = acc[1] = acc[2] = acc[3] = make_float2(0.f, 0.f);
            }
          }
          if (!FUSED || !switch_now || !ok) break;
          {
                unsigned int mbits = float_to_bits16<T>(mm.absmax());
                mbits = __reduce_max_sync(0xFFFFFFFFu, mbits);
                if (lane == 0) smx[warp] = mbits;
                if (tr && tc == 0) p.trace[(c * 2 + team) * 8 + 2] = hp_gtime();      // this team is through with A
                if (!hp_consumer_sync(cbar, cpar)) { ok = false; break; }      // both teams: the CTA's share of P is written (break: leaves the phase loop)
                if (tid == 0) {
                    unsigned int r_ = 0;
                    for (int w = 0; w < kHpConsumers / 32; ++w) r_ = max(r_, smx[w]);
                    p.maxA[c] = r_;
                    __threadfence();
                    red_release_add(p.ctrl + 4);
                }
                if (contractor) {
                    bool live = hp_cta_sync(pbar, ppar);                 // the rings are free (the producer warp sends for Q^T tiles now)
                    if (tid == 0) {
                        s_go = bounded_wait_ge(p.ctrl + 4, (unsigned)G) ? 1 : 0;        // the whole of P
                        if (!s_go) atomicOr(p.ctrl + 1, 1u);
                        if (tr) p.trace[(c * 2 + 1) * 8 + 1] = hp_gtime();
                    }
                    live = hp_cta_sync(pbar, ppar) && live;
                    tc_fence_after();
                    const uint32_t tmem = *tslot;
                    live = live && s_go != 0;
                    const int mtiles = (p.m + kTcBM - 1) / kTcBM;
                    const int nitems = mtiles * p.segsA * p.nsub;
                    const int kb_seg = kHpSegA / kTcBK, kb_sub = kb_seg / p.nsub;
                    const bool single = nitems <= p.gm;                  // at most one item per CTA: its tile goes through shared memory
                    float *tile = reinterpret_cast<float *>(smem);       // [128][kTcBN + 1], in the idle operand stages
                    if (warp < 4 && live) {
                        // ---- the partial of every item: warp w owns TMEM lanes 32 w .., a thread one row of the tile
                        uint32_t aph = 0;
                        for (int it = c; it < nitems; it += p.gm) {
                            const int mt = it % mtiles, pl = it / mtiles;
                            const int kb0 = (pl / p.nsub) * kb_seg + (pl % p.nsub) * kb_sub, kb1 = min(p.kblocks, kb0 + kb_sub);
                            // the partial leaves unscaled: a row's factor is the power of two of its (bucket, column segment)
                            // times that of Q, so the product with its reciprocal is exact
                            const int row = mt * kTcBM + warp * 32 + lane;
                            float inv = 1.f;
                            if (row < p.m) inv = 1.f / (__ldcg(p.scaleP + (long long)row * p.segsA + pl / p.nsub) * __ldcg(hv.maxB + 1));
                            if (!mbar_wait_warp(accb, aph)) { if (lane == 0) atomicOr(p.ctrl + 1, 1u); break; }
                            aph ^= 1u;
                            tc_fence_after();
                            if (tr && tid == 0) p.trace[(c * 2 + 0) * 8 + 1] = hp_gtime();
                            float *dst0 = p.partAB + (long long)pl * mm2;
                            if (single) {
                                // one item per CTA: the operand stages are idle now, so the rows go through shared memory
                                // and out as full lines (thread = row on the way in, lane = column on the way out)
                                const int rloc = warp * 32 + lane;
#pragma unroll 1
                                for (int cc = 0; cc < kTcBN / 16; ++cc) {
                                    if (cc * 16 >= p.m) break;
                                    uint32_t v[16];
                                    if (kb1 > kb0) {
                                        tc_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(cc * 16), v);
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 16; ++j) v[j] = 0u;       // an empty K range: the partial is zero
                                    }
#pragma unroll
                                    for (int j = 0; j < 16; ++j) tile[rloc * (kTcBN + 1) + cc * 16 + j] = __uint_as_float(v[j]) * inv;
                                }
                            } else {
                                float *dst = dst0 + (long long)row * p.m;
#pragma unroll 1
                                for (int cc = 0; cc < kTcBN / 16; ++cc) {
                                    if (cc * 16 >= p.m) break;
                                    uint32_t v[16];
                                    if (kb1 > kb0) {
                                        tc_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(cc * 16), v);
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 16; ++j) v[j] = 0u;
                                    }
                                    if (row < p.m) {
#pragma unroll
                                        for (int j = 0; j < 16; ++j)
                                            if (cc * 16 + j < p.m) __stcg(dst + cc * 16 + j, __uint_as_float(v[j]) * inv);
                                    }
                                }
                            }
                            tc_fence_before();
                            __syncwarp();
                            if (tr && tid == 0) p.trace[(c * 2 + 0) * 8 + 3] = hp_gtime();
                            if (lane == 0) mbar_arrive(accfree);
                        }
                    }
                    tc_fence_before();
                    hp_cta_sync(pbar, ppar);                             // the tile of a single item stands in shared memory
                    if (tr && tid == 0) p.trace[(size_t)G * 24 + c * 8 + 6] = hp_gtime();
                    if (live && single && c < nitems) {
                        // all sixteen consumer warps: eight rows each, out as full lines (lane = column)
                        const int mt = c % mtiles, pl = c / mtiles;
                        float *dst0 = p.partAB + (long long)pl * mm2;
                        for (int r = warp * 8; r < warp * 8 + 8; ++r) {
                            const int rowg = mt * kTcBM + r;
                            if (rowg >= p.m) break;
                            float *dst = dst0 + (long long)rowg * p.m;
#pragma unroll
                            for (int q = 0; q < kTcBN / 32; ++q) {
                                const int col = q * 32 + lane;
                                if (col < p.m) __stcg(dst + col, tile[r * (kTcBN + 1) + col]);
                            }
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // bulk copies write here again later
                    }
                    if (tr && tid == 0) p.trace[(size_t)G * 24 + c * 8 + 7] = hp_gtime();
                    hp_cta_sync(pbar, ppar);                             // operand stages idle
                    if (tr && tc == 0) p.trace[(c * 2 + team) * 8 + 6] = hp_gtime();
                }
                if (tr && tc == 0) p.trace[(c * 2 + team) * 8 + 5] = hp_gtime();
          }
        }
        if (tr && tc == 0) { p.trace[(c * 2 + team) * 8 + 4] = hp_gtime(); p.trace[(c * 2 + team) * 8 + 7] = nunit; }
        if (!FUSED) {
            // max|A| over what this CTA streamed (for tau)
            unsigned int mbits = float_to_bits16<T>(mm.absmax());
            mbits = __reduce_max_sync(0xFFFFFFFFu, mbits);
            if ((tid & 31) == 0) {
                smx[tid >> 5] = mbits;
                if (!ok) atomicOr(p.ctrl + 1, 1u);
            }
            if (ok && hp_consumer_sync(cbar, cpar) && tid == 0) {
                unsigned int r_ = 0;
                for (int w = 0; w < kHpConsumers / 32; ++w) r_ = max(r_, smx[w]);
                p.maxA[c] = r_;
            }
        } else {
            // ---- every unit this CTA took is done: publish, wait (bounded) for all CTAs, then combine and verdict.
            // Every consumer thread comes here, also after a wait that gave up (the error word is set then), so the
            // barriers of the combine always see all 512 of them.
            if (!ok && lane == 0) atomicOr(p.ctrl + 1, 1u);
            hp_consumer_sync(cbar, cpar);
            if (tid == 0) {
                __threadfence();
                red_release_add(p.ctrl + 6);
                if (!bounded_wait_ge(p.ctrl + 6, (unsigned)G)) atomicOr(p.ctrl + 1, 1u);
                __threadfence();
            }
            HvSyncConsumers::sync();
            hv_combine_fused<T>(hv);
        }
    }
}

// The same signed row-bucket sums with plain loads, for inputs the bulk copies cannot address
// (base not 16-byte aligned, leading dimension or width not a multiple of 16 bytes).
// Thread (bucket a, column): rows of the bucket in ascending row order.
template <typename T>
__global__ void __launch_bounds__(256) hp_rowsum_plain_kernel(const HpArgs p)
{
    const int a = blockIdx.y;
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int s0 = __ldg(p.rowstart + a), s1 = __ldg(p.rowstart + a + 1);
    if (blockIdx.z == 0) {
        if (col >= p.kpad) return;
        constexpr unsigned int kInf = std::is_same<T, __half>::value ? 0x7C00u : 0x7F80u;
        float acc = 0.f;
        unsigned int mx = 0;
        if (col < p.n2) {
            for (int s = s0; s < s1; ++s) {
                const uint32_t e = __ldg(p.rowperm + s);
                const unsigned short h = p.A[(long long)(e & 0x7FFFFFFFu) * p.lda + col];
                const float x = bits16_to_float<T>(h);
                acc += (e >> 31) ? -x : x;
                const unsigned int mag = h & 0x7FFFu;       // |x| of a 16-bit float orders like its bit pattern
                if (mag <= kInf) mx = max(mx, mag);         // NaN operands are ignored, as in the streaming path
            }
        }
        p.P[(long long)a * p.kpad + col] = acc;
        mx = __reduce_max_sync(0xFFFFFFFFu, mx);
        if ((threadIdx.x & 31) == 0 && mx) atomicMax(p.maxA, mx);
    } else {
        if (col >= p.n3) return;
        float acc = 0.f;
        for (int s = s0; s < s1; ++s) {
            const uint32_t e = __ldg(p.rowperm + s);
            const float x = p.C[(long long)(e & 0x7FFFFFFFu) * p.ldc + col];
            acc += (e >> 31) ? -x : x;
        }
        p.Tc[(long long)a * p.n3 + col] = acc;
    }
}

// partC from Tc for the plain-load path: CTA (bucket row a, segment), thread b folds the segment's
// columns of bucket b in ascending order (same order as the streaming kernel).
__global__ void __launch_bounds__(256) hp_fold_plain_kernel(const HpArgs p)
{
    const int a = blockIdx.x, seg = blockIdx.y;
    const long long mm = (long long)p.m * p.m;
    const float *trow = p.Tc + (long long)a * p.n3 + (long long)seg * kHpSegC;
    const uint32_t *sp = p.segperm + (long long)seg * kHpSegC;
    for (int b = threadIdx.x; b < p.m; b += blockDim.x) {
        const int s0 = __ldg(p.segstart + (long long)seg * (p.m + 1) + b), s1 = __ldg(p.segstart + (long long)seg * (p.m + 1) + b + 1);
        float cf = 0.f;
        for (int s = s0; s < s1; ++s) {
            const uint32_t e = __ldg(sp + s);
            const float x = trow[e & 0x7FFFFFFFu];
            cf += (e >> 31) ? -x : x;
        }
        p.partC[(long long)seg * mm + (long long)a * p.m + b] = cf;
    }
}

// scale[0] = the power of two for the P planes, from the per-CTA maxima of |A| (16-bit patterns) and the
// largest row bucket
template <typename T>
__global__ void __launch_bounds__(256) hp_scale_a_kernel(const unsigned int *maxA, int n_maxA, const int *rowcount, int m, float *scale)
{
    __shared__ unsigned int wbits[8];
    __shared__ int wcnt[8];
    unsigned int mb = 0;
    int c = 0;
    for (int r = threadIdx.x; r < n_maxA; r += blockDim.x) mb = max(mb, maxA[r]);
    for (int b = threadIdx.x; b < m; b += blockDim.x) c = max(c, rowcount[b]);
    mb = __reduce_max_sync(0xFFFFFFFFu, mb);
    c = __reduce_max_sync(0xFFFFFFFFu, c);
    if ((threadIdx.x & 31) == 0) { wbits[threadIdx.x >> 5] = mb; wcnt[threadIdx.x >> 5] = c; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { mb = max(mb, wbits[w]); c = max(c, wcnt[w]); }
        scale[0] = tc_scale_of(c, bits16_to_float<T>((unsigned short)mb));
    }
}

// Q = B H2^T from the transposed weight W = B^T (n3 x n2, row-major): thread (bucket b, column k) adds the
// rows of W that fall in bucket b in ascending row order (the order in which the untransposed path adds
// the columns of B).  Runs once per B side; Q is kpad x npad with zero padding.
template <typename T>
__global__ void __launch_bounds__(256) hp_compress_wt_kernel(const unsigned short *W, long long ldw, int n2, int m_b, int kpad,
                                                             int npad, const uint32_t *colperm, const int *colstart, float *Q)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (k >= kpad) return;
    float q = 0.f;
    if (k < n2 && b < m_b) {
        const int s0 = __ldg(colstart + b), s1 = __ldg(colstart + b + 1);
        for (int s = s0; s < s1; ++s) {
            const uint32_t e = __ldg(colperm + s);
            const float x = bits16_to_float<T>(W[(long long)(e & 0x7FFFFFFFu) * ldw + k]);
            q += (e >> 31) ? -x : x;
        }
    }
    Q[(long long)k * npad + b] = q;
}

// ---------------------------------------------------------------- host side
struct HpPlan {
    int kpad, npad, segsA, segsC, tile, ksplit, kchunk;
    int tc_ksplit;     // K splits of the tensor-core contraction (128 x 128 tiles, K blocks of 64)
    // the fused kernel: K blocks of 32 in the planes, K ranges per column segment of A, contracting CTAs (0: not available)
    int kblocks, f_nsub, f_gm;
};

static void hp_plan(long long n2, long long n3, int m, int sms, HpPlan &pl)
{
    pl.kpad = (int)((n2 + 15) / 16 * 16);
    pl.npad = (m + 3) / 4 * 4;
    pl.segsA = (int)((n2 + kHpSegA - 1) / kHpSegA);
    pl.segsC = (int)((n3 + kHpSegC - 1) / kHpSegC);
    pl.tile = m <= 512 ? 64 : 128;
    const int t1 = (m + pl.tile - 1) / pl.tile;
    const int tiles = t1 * t1;
    int ks = (2 * sms + tiles - 1) / tiles;                     // two resident CTAs per SM
    const int maxks = pl.kpad / 128 > 1 ? pl.kpad / 128 : 1;    // at least 128 of K per split
    if (ks > maxks) ks = maxks;
    if (ks > 64) ks = 64;
    if (ks < 1) ks = 1;
    int kchunk = ((pl.kpad + ks - 1) / ks + 15) / 16 * 16;
    pl.ksplit = (pl.kpad + kchunk - 1) / kchunk;
    pl.kchunk = kchunk;
    pl.tc_ksplit = tc_plan_ksplit(m, m, pl.kpad, 1, sms);
    // Fused kernel: one column tile of 256 buckets, so m <= 256.  About 32 (row tile, K range) items, one per
    // contracting CTA: K ranges of at most 32 K blocks (the accumulation chain the sketches' noise was measured
    // with) that never span two column segments of A, because every segment of a bucket has its own scale.
    pl.kblocks = (pl.kpad + kTcBK - 1) / kTcBK;
    pl.f_nsub = 0; pl.f_gm = 0;
    if (m <= kTcBN) {
        const int mtiles = (m + kTcBM - 1) / kTcBM;
        int nsub = 2;
        while (nsub < 16 && mtiles * pl.segsA * nsub * 2 <= 32) nsub *= 2;
        const int items = mtiles * pl.segsA * nsub;
        const int gm = items < 32 ? items : 32;
        if (sms >= 2 * gm + 16) { pl.f_nsub = nsub; pl.f_gm = gm; }
    }
}

struct HpCache {          // the B side, device memory kept by the caller across calls
    int *h1, *v1, *rowcount, *rowstart;
    uint32_t *rowperm;
    int *h2, *v2, *colcount, *colstart;
    uint32_t *colperm;
    int *extra_count, *extra_start, *rank;
    int *stages;
    uint32_t *segperm;
    int *segstart;
    float *Q;
    unsigned char *Qplanes;   // Q^T as tiled FP16 planes (tensor-core contraction), scaled by maxB[1]
    float *maxB;          // [0] max|B|, [1] the power of two that brings Q into FP16 range
    unsigned int *scratch;
};

static size_t hp_cache_layout(void *base, long long n1, long long n2, long long n3, int m, int sms, HpCache *c)
{
    HpPlan pl;
    hp_plan(n2, n3, m, sms, pl);
    char *p = static_cast<char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) { void *r = p ? p + off : nullptr; off += align_up(bytes, 256); return r; };
    HpCache t;
    t.h1 = (int *)take((size_t)n1 * 4); t.v1 = (int *)take((size_t)n1 * 4); t.rowperm = (uint32_t *)take((size_t)n1 * 4);
    t.rowcount = (int *)take((size_t)(m + 1) * 4); t.rowstart = (int *)take((size_t)(m + 1) * 4);
    t.h2 = (int *)take((size_t)n3 * 4); t.v2 = (int *)take((size_t)n3 * 4); t.colperm = (uint32_t *)take((size_t)n3 * 4);
    t.colcount = (int *)take((size_t)(m + 1) * 4); t.colstart = (int *)take((size_t)(m + 1) * 4);
    const size_t units = (size_t)m * (pl.segsA + pl.segsC);
    t.extra_count = (int *)take((units + 1) * 4);
    t.extra_start = (int *)take((units + 1) * 4);
    t.rank = (int *)take((size_t)m * 4);
    // one chunk per unit, plus continuation chunks: at most (stages of all units) / 8 of them
    t.stages = (int *)take((units + (size_t)(pl.segsA + pl.segsC) * ((size_t)n1 / (kHpPieces * kHpChunk) + (size_t)m / kHpChunk + 1)) * kHpChunk * 64);
    t.segperm = (uint32_t *)take((size_t)n3 * 4);
    t.segstart = (int *)take((size_t)pl.segsC * (m + 1) * 4);
    t.Q = (float *)take((size_t)pl.kpad * pl.npad * 4);
    t.Qplanes = (unsigned char *)take(tc_planes_bytes(m, pl.kpad));
    t.maxB = (float *)take(256);
    t.scratch = (unsigned int *)take(256);
    if (c) *c = t;
    return off;
}

struct HpWork {           // per-call scratch
    unsigned int *ctrl;   // first 256 bytes: zero before the first call (fpsk_probe_init)
    unsigned int *maxA;
    float4 *vstat;
    float *P, *Tc, *partAB, *partC, *S, *cstat;
    unsigned char *Pplanes;
    float *scaleA;        // the power of two that brings P into FP16 range (tensor-core contraction)
    float *scaleP;        // fused kernel: one such power per (bucket, column segment of A)
    unsigned long long *trace;
};

static size_t hp_work_layout(void *base, long long n1, long long n2, long long n3, int m, int sms, HpWork *w)
{
    HpPlan pl;
    hp_plan(n2, n3, m, sms, pl);
    char *p = static_cast<char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) { void *r = p ? p + off : nullptr; off += align_up(bytes, 256); return r; };
    HpWork t;
    t.ctrl = (unsigned int *)take(256);
    t.maxA = (unsigned int *)take((size_t)(sms > 1 ? sms : 1) * 4);
    t.vstat = (float4 *)take((size_t)kHvMaxGrid * 16);
    t.cstat = (float *)take((size_t)kHvMaxGrid * 4);
    t.P = (float *)take((size_t)m * pl.kpad * 4);
    t.Tc = (float *)take((size_t)m * n3 * 4);
    int nparts = pl.ksplit > pl.tc_ksplit ? pl.ksplit : pl.tc_ksplit;
    if (pl.segsA * pl.f_nsub > nparts) nparts = pl.segsA * pl.f_nsub;
    t.partAB = (float *)take((size_t)nparts * m * m * 4);
    t.Pplanes = (unsigned char *)take(tc_planes_bytes(m, pl.kpad));
    t.scaleA = (float *)take(256);
    t.scaleP = (float *)take((size_t)m * pl.segsA * 4);
    t.partC = (float *)take((size_t)pl.segsC * m * m * 4);
    t.S = (float *)take((size_t)m * m * 4);
    t.trace = (unsigned long long *)take((size_t)(sms > 1 ? sms : 1) * 256);       // 32 words per CTA (see HpArgs::trace)
    if (w) *w = t;
    return off;
}

static int hp_sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return 148;
    return sms;
}

size_t hprobe_cache_bytes(long long n1, long long n2, long long n3, int m)
{
    return hp_cache_layout(nullptr, n1, n2, n3, m, hp_sm_count(), nullptr);
}

size_t hprobe_ws_bytes(long long n1, long long n2, long long n3, int m)
{
    return hp_work_layout(nullptr, n1, n2, n3, m, hp_sm_count(), nullptr);
}

static HpArgs hp_args(const void *A, long long lda, const float *C, long long ldc, long long n1, long long n2, long long n3,
                      int m, const HpPlan &pl, const HpCache &c, const HpWork *w)
{
    HpArgs a;
    a.A = static_cast<const unsigned short *>(A); a.lda = lda;
    a.C = C; a.ldc = ldc;
    a.n1 = (int)n1; a.n2 = (int)n2; a.n3 = (int)n3; a.m = m; a.kpad = pl.kpad;
    a.segsA = pl.segsA; a.segsC = pl.segsC;
    a.rowperm = c.rowperm; a.rowstart = c.rowstart; a.stages = c.stages;
    a.segperm = c.segperm; a.segstart = c.segstart;
    a.P = w ? w->P : nullptr; a.Tc = w ? w->Tc : nullptr; a.partC = w ? w->partC : nullptr;
    a.maxA = w ? w->maxA : nullptr; a.ctrl = w ? w->ctrl : nullptr;
    a.trace = w ? w->trace : nullptr;
    a.Pplanes = w ? w->Pplanes : nullptr; a.scaleP = w ? w->scaleP : nullptr; a.Qplanes = c.Qplanes;
    a.partAB = w ? w->partAB : nullptr;
    a.gm = pl.f_gm; a.nsub = pl.f_nsub > 0 ? pl.f_nsub : 1; a.kblocks = pl.kblocks;
    a.trace_on = 0;
#ifdef FPSK_MEASURE
    // measurement build only: FPSK_HPROBE_TRACE records per-team phase stamps in the workspace
    static const bool trace_env = getenv("FPSK_HPROBE_TRACE") != nullptr;
    a.trace_on = trace_env ? 1 : 0;
#endif
    return a;
}

// Build the B side: both hash tables of the round, Q = B H2^T, max|B| and the unit partition.
fpsk_status hprobe_prepare(const void *B, long long ldb, int b_transposed, long long n1, long long n2, long long n3, fpsk_dtype dtype,
                           uint64_t seed, int rnd, int m, void *cache, size_t cache_bytes, cudaStream_t st)
{
    const int sms = hp_sm_count();
    HpCache c;
    if (cache_bytes < hp_cache_layout(cache, n1, n2, n3, m, sms, &c)) return FPSK_ERR_WORKSPACE;
    HpPlan pl;
    hp_plan(n2, n3, m, sms, pl);
    fpsk_status rc = build_hash_side(seed, rnd, 0, (int)n1, m, c.h1, c.v1, c.rowcount, c.rowstart, c.rowperm, st);
    if (rc != FPSK_OK) return rc;
    rc = build_hash_side(seed, rnd, 1, (int)n3, m, c.h2, c.v2, c.colcount, c.colstart, c.colperm, st);
    if (rc != FPSK_OK) return rc;
    if (b_transposed) {
        // the weight as W = B^T (n3 x n2): bucket b of Q = B H2^T is the signed sum of the rows of W in bucket b
        dim3 grid((pl.kpad + 255) / 256, pl.npad);
        if (dtype == FPSK_FP16) hp_compress_wt_kernel<__half><<<grid, 256, 0, st>>>(static_cast<const unsigned short *>(B), ldb, (int)n2, m, pl.kpad, pl.npad, c.colperm, c.colstart, c.Q);
        else hp_compress_wt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const unsigned short *>(B), ldb, (int)n2, m, pl.kpad, pl.npad, c.colperm, c.colstart, c.Q);
        FPSK_LAUNCH_CHECK();
    } else {
        rc = build_b_side(B, ldb, n2, n3, dtype, m, pl.kpad, pl.npad, c.colperm, c.colstart, c.Q, st);
        if (rc != FPSK_OK) return rc;
    }
    rc = b_transposed ? max_abs_half_launch(B, ldb, n3, n2, dtype, c.maxB, c.scratch, st)
                      : max_abs_half_launch(B, ldb, n2, n3, dtype, c.maxB, c.scratch, st);
    if (rc != FPSK_OK) return rc;
    rc = tc_scale_launch(c.colcount, m, c.maxB, c.maxB + 1, st);
    if (rc != FPSK_OK) return rc;
    rc = tc_split_launch(c.Q, c.maxB + 1, 1, pl.npad, m, pl.kpad, 1, c.Qplanes, st);      // row b of Q^T is column b of Q
    if (rc != FPSK_OK) return rc;
    const HpArgs a = hp_args(nullptr, 0, nullptr, 0, n1, n2, n3, m, pl, c, nullptr);
    hp_segment_lists_kernel<<<pl.segsC, 256, (size_t)(m + 1) * 4, st>>>(c.h2, c.v2, (int)n3, m, c.segperm, c.segstart);
    FPSK_LAUNCH_CHECK();
    const int units = m * (pl.segsA + pl.segsC);
    hp_rank_kernel<<<(m + 127) / 128, 128, 0, st>>>(c.rowstart, m, c.rank);
    FPSK_LAUNCH_CHECK();
    hp_count_chunks_kernel<<<(units + 255) / 256, 256, 0, st>>>(a, c.rank, c.extra_count);
    FPSK_LAUNCH_CHECK();
    rc = exclusive_scan_launch(c.extra_count, units, c.extra_start, st);
    if (rc != FPSK_OK) return rc;
    hp_fill_stages_kernel<<<(units + 255) / 256, 256, 0, st>>>(a, c.rank, c.extra_start, c.stages);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// One probe on a prepared B side.  d_S may be NULL (S then stays in the workspace).
fpsk_status hprobe_launch(const void *A, long long lda, const float *C, long long ldc, long long n1, long long n2,
                          long long n3, fpsk_dtype dtype, int m, double mu, int scale_cap, int tensor_cores, void *cache, size_t cache_bytes, void *ws,
                          size_t ws_bytes, cudaStream_t st, fpsk_probe_result *d_result, float *d_S, fpsk_probe_state *d_state)
{
    const int sms = hp_sm_count();
    HpCache c;
    HpWork w;
    if (cache_bytes < hp_cache_layout(cache, n1, n2, n3, m, sms, &c)) return FPSK_ERR_WORKSPACE;
    if (ws_bytes < hp_work_layout(ws, n1, n2, n3, m, sms, &w)) return FPSK_ERR_WORKSPACE;
    HpPlan pl;
    hp_plan(n2, n3, m, sms, pl);
    const HpArgs a = hp_args(A, lda, C, ldc, n1, n2, n3, m, pl, c, &w);
    bool force_plain = false;
#ifdef FPSK_MEASURE
    // measurement build only: FPSK_HPROBE_PLAIN forces the plain-load kernels
    static const bool env_plain = getenv("FPSK_HPROBE_PLAIN") != nullptr;
    force_plain = env_plain;
#endif
    const bool bulk_ok = !force_plain && (reinterpret_cast<uintptr_t>(A) & 15) == 0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0 &&
                         lda % 8 == 0 && ldc % 4 == 0 && n2 % 8 == 0 && n3 % 4 == 0;
    int n_maxA = sms;
    HvArgs v;
    v.partAB = w.partAB; v.ksplit = 0; v.n_maxA = 0;
    v.partC = w.partC; v.nseg = pl.segsC;
    v.m = m; v.n1 = (int)n1; v.n2 = (int)n2; v.n3 = (int)n3;
    v.maxA = w.maxA; v.maxB = c.maxB;
    v.scaleA = nullptr;
    const double mm = (double)m * (double)m;
    v.thr_scale = (float)(mu * sqrt(2.0 * log(mm > 2.0 ? mm : 2.0)));
    v.cap_scale = scale_cap ? (float)sqrt((double)n1 * (double)n3 / mm) : 1.0f;
    v.S = d_S ? d_S : w.S;
    v.vstat = w.vstat; v.cstat = w.cstat; v.ctrl = w.ctrl; v.result = d_result; v.state = d_state;
    v.ctrace = a.trace_on ? w.trace + 8 * 2 * sms : nullptr;
    if (bulk_ok) {
        static std::once_flag once;
        static cudaError_t attr_err = cudaSuccess;
        std::call_once(once, [] {
            const void *fns[4] = {(const void *)hp_stream_kernel<__half, false>, (const void *)hp_stream_kernel<__nv_bfloat16, false>,
                                  (const void *)hp_stream_kernel<__half, true>, (const void *)hp_stream_kernel<__nv_bfloat16, true>};
            for (int i = 0; i < 4 && attr_err == cudaSuccess; ++i)
                attr_err = cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kHpSmem);
        });
        FPSK_CUDA_OK(attr_err);
        if (tensor_cores && pl.f_gm > 0 && sms <= kHvMaxGrid) {
            // the whole probe in one cooperative launch: stream, contraction on the tensor cores, combine, verdict
            v.partAB = w.partAB; v.ksplit = pl.segsA * pl.f_nsub; v.n_maxA = sms;
            void *args[] = {(void *)&a, (void *)&v};
            const void *fn = dtype == FPSK_FP16 ? (const void *)hp_stream_kernel<__half, true> : (const void *)hp_stream_kernel<__nv_bfloat16, true>;
            // (fn is hp_stream_kernel<T, true>)  Where the device cannot hold the whole grid at once (fewer SMs available to
            // this context than it reports), the launch is refused and the three-launch form below runs instead.
            const cudaError_t le = cudaLaunchCooperativeKernel(fn, dim3(sms), dim3(kHpThreads), args, kHpSmem, st);
            if (le == cudaSuccess) {
                count_launch();
                return FPSK_OK;
            }
            if (le != cudaErrorCooperativeLaunchTooLarge) return FPSK_ERR_CUDA;
            (void)cudaGetLastError();
            v.partAB = w.partAB; v.ksplit = 0; v.n_maxA = 0;
        }
        if (dtype == FPSK_FP16) hp_stream_kernel<__half, false><<<sms, kHpThreads, kHpSmem, st>>>(a, v);
        else hp_stream_kernel<__nv_bfloat16, false><<<sms, kHpThreads, kHpSmem, st>>>(a, v);
        FPSK_LAUNCH_CHECK();
    } else {
        n_maxA = 1;
        FPSK_CUDA_OK(cudaMemsetAsync(w.maxA, 0, 4, st));
        const int cols = pl.kpad > (int)n3 ? pl.kpad : (int)n3;
        dim3 grid((cols + 255) / 256, m, 2);
        if (dtype == FPSK_FP16) hp_rowsum_plain_kernel<__half><<<grid, 256, 0, st>>>(a);
        else hp_rowsum_plain_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(a);
        FPSK_LAUNCH_CHECK();
        hp_fold_plain_kernel<<<dim3(m, pl.segsC), 256, 0, st>>>(a);
        FPSK_LAUNCH_CHECK();
    }
    fpsk_status rc;
    int ksplit = pl.ksplit;
    if (tensor_cores) {
        if (dtype == FPSK_FP16) hp_scale_a_kernel<__half><<<1, 256, 0, st>>>(w.maxA, n_maxA, c.rowcount, m, w.scaleA);
        else hp_scale_a_kernel<__nv_bfloat16><<<1, 256, 0, st>>>(w.maxA, n_maxA, c.rowcount, m, w.scaleA);
        FPSK_LAUNCH_CHECK();
        rc = tc_split_launch(w.P, w.scaleA, pl.kpad, 1, m, pl.kpad, 0, w.Pplanes, st);
        if (rc != FPSK_OK) return rc;
        const unsigned char *pa[2] = {w.Pplanes, w.Pplanes}, *pb[2] = {c.Qplanes, c.Qplanes};
        const int sel[3] = {0, 0, 0};
        ksplit = pl.tc_ksplit;
        rc = tc_contract_launch(pa, pb, sel, sel, 1, 1, w.partAB, m, m, pl.kpad, ksplit, w.ctrl + 1, st);
    } else {
        rc = contraction_launch(w.P, c.Q, w.partAB, m, m, pl.kpad, pl.kpad, pl.npad, pl.ksplit, pl.kchunk, pl.tile, st);
    }
    if (rc != FPSK_OK) return rc;
    v.partAB = w.partAB; v.ksplit = ksplit; v.n_maxA = n_maxA;
    v.scaleA = tensor_cores ? w.scaleA : nullptr;
    {
        // cooperative: every CTA waits (bounded) for the statistics of all others
        int grid = sms < kHvMaxGrid ? sms : kHvMaxGrid;
        const long long q4 = ((long long)m * m + 3) / 4;
        if (grid > q4) grid = (int)q4;
        void *args[] = {(void *)&v};
        const void *fn = dtype == FPSK_FP16 ? (const void *)hp_combine_kernel<__half> : (const void *)hp_combine_kernel<__nv_bfloat16>;
        FPSK_CUDA_OK(cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kHvThreads), args, 0, st));
        count_launch();
    }
    return FPSK_OK;
}

}  // namespace fpsk
