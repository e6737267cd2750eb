// Split-precision contraction on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
// The sketches need S_AB = P Q (and the weighted forms) to FP32 accuracy: the sketch noise is the
// measured quantity, and a single-pass reduced-precision product raises it by orders of magnitude
// (Section "Implementation": TF32 raised the floor 419x).  An FP32 value, scaled by a power of two
// into FP16 range, is therefore split into two FP16 terms x = hi + lo (11 + 11 significand bits; the
// remainder x - hi is exact in FP32, so hi + lo misses x by at most 2^-24 |x|), and the product is formed
// from the three term pairs whose weight is above 2^-22:
//   (lo,hi) (hi,lo) (hi,hi),
// every pair one FP16 tcgen05.mma with FP32 accumulation into the same TMEM accumulator.  (Three BF16
// terms need six pairs for the same accuracy: twice the tensor-core work.)
//
//   tc_split_kernel      FP32 matrix -> two FP16 planes, laid out tile by tile exactly as the
//                        tensor core reads shared memory (K-major, no swizzle: 8 x 16-byte core
//                        matrices), so that the planes of an operand tile are one contiguous block
//   tc_contract_kernel   one 128 x 256 output tile per CTA and K split: a producer warp brings the operand
//                        tiles of a 32-deep K block with two bulk copies (mbarrier complete_tx), one
//                        thread issues the 6 MMAs of the block and commits them to the stage's
//                        "empty" barrier, four warps read the accumulator back (tcgen05.ld) and
//                        store the split-K partial.
// Every wait is bounded; on expiry the CTA flags the error word, frees its TMEM and leaves.
#include "tc_ops.cuh"

#include <mutex>

namespace fpsk {

constexpr int kTcStages = 4;
constexpr int kTcSmem = kTcStages * kTcStageBytes + 256;
constexpr int kTcThreads = 192;                          // warps 0-3 epilogue, warp 4 producer, warp 5 MMA
static_assert(kTcBM * (kTcBN + 1) * 4 <= kTcStages * kTcStageBytes, "epilogue tile fits in the operand stages");

// ---------------------------------------------------------------- FP32 -> two FP16 planes, tiled
// X(r, k) = scale * src[r * ldr + k * ldk] for r < rows, k < kk, else 0 (scale: a device scalar, a power of two).
// Tiles of R rows (128 for the A side, 256 for the B side) by 32 k.  Output: row tile rt, K block kb, plane p at
// ((rt * kblocks + kb) * 2 + p) * R * 64 bytes, so the planes of an operand tile are one contiguous block (one bulk copy); inside a plane
// tile the 16-byte chunk (row r, k chunk kc) sits at (kc * (R / 8) + r / 8) * 128 + (r % 8) * 16.
template <int R>
__global__ void __launch_bounds__(256) tc_split_kernel(const float *src, const float *d_scale, long long ldr, long long ldk,
                                                       int rows, int kk, int kblocks, unsigned char *planes)
{
    const float scale = d_scale ? __ldg(d_scale) : 1.f;
    __shared__ float tile[R][kTcBK + 1];
    constexpr int kTile = R * kTcBK * 2;
    const int kb = blockIdx.x, rt = blockIdx.y;
    const int r0 = rt * R, k0 = kb * kTcBK;
    if (ldk == 1) {
        // rows contiguous in k: a warp reads one row of 32 floats
        for (int e = threadIdx.x; e < R * kTcBK; e += 256) {
            const int r = e / kTcBK, k = e % kTcBK;
            tile[r][k] = (r0 + r < rows && k0 + k < kk) ? src[(long long)(r0 + r) * ldr + (k0 + k)] : 0.f;
        }
    } else {
        // columns contiguous in r: a warp reads 32 consecutive r of one k
        for (int e = threadIdx.x; e < R * kTcBK; e += 256) {
            const int k = e / R, r = e % R;
            tile[r][k] = (r0 + r < rows && k0 + k < kk) ? src[(long long)(r0 + r) * ldr + (long long)(k0 + k) * ldk] : 0.f;
        }
    }
    __syncthreads();
    unsigned char *out = planes + ((size_t)rt * kblocks + kb) * kTcPlanes * kTile;
    for (int id = threadIdx.x; id < R * (kTcBK / 8); id += 256) {
        const int kc = id / R, r = id % R;
        unsigned short h[8], l[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float x = tile[r][kc * 8 + j] * scale;
            const __half bh = __float2half_rn(x);
            const float r1 = x - __half2float(bh);               // exact
            const __half bl = __float2half_rn(r1);
            h[j] = __half_as_ushort(bh);
            l[j] = __half_as_ushort(bl);
        }
        const size_t off = (size_t)(kc * (R / 8) + r / 8) * 128 + (size_t)(r % 8) * 16;
        auto pack = [](const unsigned short *v) {
            return make_uint4(v[0] | ((unsigned)v[1] << 16), v[2] | ((unsigned)v[3] << 16), v[4] | ((unsigned)v[5] << 16),
                              v[6] | ((unsigned)v[7] << 16));
        };
        *reinterpret_cast<uint4 *>(out + off) = pack(h);
        *reinterpret_cast<uint4 *>(out + kTile + off) = pack(l);
    }
}

struct TcArgs {
    const unsigned char *planesA[2];   // operand matrices of the A side (P, Pw), tiled planes
    const unsigned char *planesB[2];   // of the B side (Q^T, Qw^T)
    int selA[3], selB[3];              // which matrix each problem multiplies
    float *Cpart;                      // [ksplit][nprob][M * N]
    int M, N;                          // valid extent of the output
    int mtiles, ntiles, kblocks;       // tiles of 128 rows of the A planes, of 256 rows of the B planes, K blocks of 32
    int ksplit, kb_per_split, nprob, pstride;   // partial (ks, prob) at (ks * pstride + prob) * M * N
    unsigned int *err;                 // set to 1 when a wait gave up
};

__global__ void __launch_bounds__(kTcThreads, 1) tc_contract_kernel(const TcArgs g)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + kTcStages * kTcStageBytes);
    uint32_t *tslot = reinterpret_cast<uint32_t *>(bars + 8);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kTcStages), accb = smem_u32(bars + 2 * kTcStages);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nt = blockIdx.x, mt = blockIdx.y;
    const int prob = blockIdx.z / g.ksplit, ks = blockIdx.z % g.ksplit;
    const int kb0 = ks * g.kb_per_split, kb1 = min(g.kblocks, kb0 + g.kb_per_split);
    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accb, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 5) {
        tc_alloc(smem_u32(tslot), kTcCols);
        tc_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tslot;

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        const unsigned char *pa = g.planesA[g.selA[prob]], *pb = g.planesB[g.selB[prob]];
        int stage = 0;
        uint32_t phase = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
            int w = 1;
            if (lane == 0) w = mbar_wait_bounded(empty0 + 8 * stage, phase ^ 1u) ? 1 : 0;
            w = __shfl_sync(0xFFFFFFFFu, w, 0);
            if (!w) { if (lane == 0) { atomicOr(g.err, 1u); } break; }
            if (lane == 0) mbar_expect_tx(full0 + 8 * stage, kTcStageBytes);
            __syncwarp();
            if (lane < 2) {
                // lane 0: the planes of the A tile (16 KB), lane 1: of the B tile (32 KB)
                const unsigned char *src = lane ? pb + ((size_t)nt * g.kblocks + kb) * kTcPlanes * kTcTileB
                                                : pa + ((size_t)mt * g.kblocks + kb) * kTcPlanes * kTcTileA;
                bulk_g2s(smem_u32(smem + (size_t)stage * kTcStageBytes + (size_t)lane * kTcPlanes * kTcTileA), src,
                         lane ? kTcPlanes * kTcTileB : kTcPlanes * kTcTileA, full0 + 8 * stage);
            }
            if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issue (one thread)
        // instruction descriptor: FP32 accumulator (bit 4), FP16 x FP16 (operand format fields 0), both K-major,
        // N = 256, M = 128
        const uint32_t idesc = (1u << 4) | ((uint32_t)(kTcBN >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        uint32_t acc = 0;
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
            int w = 1;
            if (lane == 0) w = mbar_wait_bounded(full0 + 8 * stage, phase) ? 1 : 0;
            w = __shfl_sync(0xFFFFFFFFu, w, 0);
            if (!w) { ok = false; break; }
            tc_fence_after();
            if (lane == 0) {
                const uint32_t sbase = smem_u32(smem + (size_t)stage * kTcStageBytes);
                // term pairs (A plane, B plane), small weights first
                const int pairA[3] = {1, 0, 0}, pairB[3] = {0, 1, 0};
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
                tc_commit(empty0 + 8 * stage);        // the stage is free once these MMAs have read it
            }
            __syncwarp();
            if (++stage == kTcStages) { stage = 0; phase ^= 1u; }
        }
        if (lane == 0) {
            if (!ok) atomicOr(g.err, 1u);
            tc_commit(accb);                          // arrives when every MMA issued above is complete
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue: warp w owns TMEM lanes 32 w ..
        const bool got = mbar_wait_warp(accb, 0);
        tc_fence_after();
        if (!got) { if (lane == 0) atomicOr(g.err, 1u); }
        else if (kb1 > kb0) {
            // accumulator rows through shared memory (the operand stages are free now), so that the partial
            // goes out as full 128-byte lines: thread = row on the way in, lane = column on the way out
            float *tile = reinterpret_cast<float *>(smem);                 // [128][kTcBN + 1]
            const int rloc = warp * 32 + lane;
#pragma unroll 1
            for (int c = 0; c < kTcBN / 32; ++c) {
                uint32_t v[32];
                tc_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), v);
#pragma unroll
                for (int j = 0; j < 32; ++j) tile[rloc * (kTcBN + 1) + c * 32 + j] = __uint_as_float(v[j]);
            }
            __syncwarp();                                                  // a warp reads back only the rows it wrote
            float *dst0 = g.Cpart + ((size_t)ks * g.pstride + prob) * (size_t)g.M * g.N;
            for (int r = 0; r < 32; ++r) {
                const int row = mt * kTcBM + warp * 32 + r;
                if (row >= g.M) break;
                float *dst = dst0 + (size_t)row * g.N + nt * kTcBN;
#pragma unroll
                for (int q = 0; q < kTcBN / 32; ++q) {
                    const int col = q * 32 + lane;
                    if (nt * kTcBN + col < g.N) dst[col] = tile[(warp * 32 + r) * (kTcBN + 1) + col];
                }
            }
        } else {
            // an empty K range (more splits than K blocks): the partial is zero
            const int row = mt * kTcBM + warp * 32 + lane;
            if (row < g.M) {
                float *dst = g.Cpart + ((size_t)ks * g.pstride + prob) * (size_t)g.M * g.N + (size_t)row * g.N;
                for (int j = 0; j < kTcBN; ++j)
                    if (nt * kTcBN + j < g.N) dst[nt * kTcBN + j] = 0.f;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tc_dealloc(tmem, kTcCols);
}

// ---------------------------------------------------------------- host side
size_t tc_planes_bytes(int rows, int kk)
{
    // sized for either side: rows rounded up to the B side's 256
    const size_t rt = (size_t)(rows + kTcBN - 1) / kTcBN, kb = (size_t)(kk + kTcBK - 1) / kTcBK;
    return kTcPlanes * rt * kb * kTcTileB;
}

fpsk_status tc_split_launch(const float *src, const float *d_scale, long long ldr, long long ldk, int rows, int kk, int b_side,
                            unsigned char *planes, cudaStream_t st)
{
    const int kb = (kk + kTcBK - 1) / kTcBK;
    if (b_side) tc_split_kernel<kTcBN><<<dim3(kb, (rows + kTcBN - 1) / kTcBN), 256, 0, st>>>(src, d_scale, ldr, ldk, rows, kk, kb, planes);
    else tc_split_kernel<kTcBM><<<dim3(kb, (rows + kTcBM - 1) / kTcBM), 256, 0, st>>>(src, d_scale, ldr, ldk, rows, kk, kb, planes);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

// K splits.  The tensor core's FP32 accumulation is not round-to-nearest: measured on sketches of clean
// products, chains of 1024 terms give the lowest noise, 2048 terms 9 % more, 8192 terms 2.4 times as much;
// shorter chains move the additions into the FP32 combine and approach its noise.  So no chain is longer than
// kTcMaxChain K blocks, and among the splits that respect this the one with the least estimated time wins:
// one CTA per SM, so the launch takes ceil(CTAs / SMs) rounds of (fixed cost + K blocks per CTA), the fixed
// cost (set-up, TMEM allocation, epilogue) being worth about nine K blocks of six MMAs; every split also adds a
// partial that the combine has to read.
constexpr int kTcMaxChain = 32;        // K blocks of 32: 1024 terms (chains of 1376 terms: 5 us less per round at
                                       // m = 1024, n2 = 4096, and a third more noise on a correctly rounded product)
constexpr int kTcFixedCost = 9;        // in K blocks
int tc_plan_ksplit(int M, int N, int K, int nprob, int sms)
{
    const int tiles = ((M + kTcBM - 1) / kTcBM) * ((N + kTcBN - 1) / kTcBN) * nprob;
    const int kblocks = (K + kTcBK - 1) / kTcBK;
    if (sms < 1) sms = 1;
    int best = 1;
    long long best_cost = -1;
    for (int s = 1; s <= kblocks && s <= 64; ++s) {
        const int per = (kblocks + s - 1) / s;
        if (per > kTcMaxChain) continue;
        if ((kblocks + per - 1) / per != s) continue;          // the same chains with fewer, empty splits
        const long long rounds = ((long long)tiles * s + sms - 1) / sms;
        // plus what a further partial costs the combine that follows (about 2.4e-6 K-block times per output element)
        const long long cost = 16 * rounds * (kTcFixedCost + per) + (long long)s * (1 + ((long long)M * N * nprob * 16) / 420000);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    if (best_cost < 0) best = (kblocks + kTcMaxChain - 1) / kTcMaxChain;     // more than 64 splits needed
    return best;
}

// part[ks][prob] = A_sel(prob) B_sel(prob)^T over the ks-th range of K blocks.  planesA[i] holds an M x K
// matrix (A-side planes of tc_split_launch), planesB[i] an N x K matrix (B-side planes).
fpsk_status tc_contract_launch(const unsigned char *const *planesA, const unsigned char *const *planesB, const int *selA,
                               const int *selB, int nprob, int pstride, float *part, int M, int N, int K, int ksplit,
                               unsigned int *d_err, cudaStream_t st)
{
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(tc_contract_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
    });
    FPSK_CUDA_OK(attr_err);
    TcArgs g;
    g.planesA[0] = planesA[0]; g.planesA[1] = planesA[1];
    g.planesB[0] = planesB[0]; g.planesB[1] = planesB[1];
    for (int i = 0; i < 3; ++i) { g.selA[i] = i < nprob ? selA[i] : 0; g.selB[i] = i < nprob ? selB[i] : 0; }
    g.Cpart = part; g.M = M; g.N = N;
    g.mtiles = (M + kTcBM - 1) / kTcBM; g.ntiles = (N + kTcBN - 1) / kTcBN; g.kblocks = (K + kTcBK - 1) / kTcBK;
    g.ksplit = ksplit; g.kb_per_split = (g.kblocks + ksplit - 1) / ksplit; g.nprob = nprob; g.pstride = pstride;
    g.err = d_err;
    tc_contract_kernel<<<dim3(g.ntiles, g.mtiles, nprob * ksplit), kTcThreads, kTcSmem, st>>>(g);
    FPSK_LAUNCH_CHECK();
    return FPSK_OK;
}

}  // namespace fpsk
