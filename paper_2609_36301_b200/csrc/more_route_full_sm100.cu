// Tensor-core path of the fused low-rank router for sm_100a: TMA-staged operands, tcgen05.mma with TMEM
// accumulators, a thread-per-token epilogue that keeps the running top-k (and, on request, the online
// (max, sum-of-exponentials) pair of Eq. app_online) in registers.
//
// One CTA routes one block of 256 tokens (two 128-row accumulators) over one contiguous range of expert tiles
// (Algorithm 1, with the token block additionally split over `msplit` CTAs along the expert dimension):
//
//   phase 1  z = X_blk R1            TMA streams 256x64 X tiles (128x64 and twice the stages for blocks of at most 128
//                                    tokens) and 64x64 R1 tiles (zero-filled beyond r), tcgen05.mma accumulates two
//                                    128 x 64 fp32 blocks in TMEM.
//   narrow   z -> bf16 hi + bf16 lo  written back to tensor memory (tcgen05.st) as the A operands [hi | lo] of phase 2:
//                                    TMEM lane = token, two K-elements per 32-bit column.  Carrying both parts keeps
//                                    the logits within ~3e-5 of exact arithmetic.
//   phase 2  y = z R2[:, block]      64 experts at a time: TMA brings the r x 64 block of R2 once for both
//                                    accumulators, tcgen05.mma with A from tensor memory (hi then lo into the same
//                                    accumulator) fills 64 TMEM columns, the epilogue drains them: each epilogue
//                                    thread owns one token and reads its logits 16 columns at a time.  The group hands
//                                    the accumulator back as soon as the last 32 columns are in registers, so the next
//                                    step's MMAs run while those are processed.
//   merge    running top-k           sorted (value, id) list in registers, fed through a per-token candidate buffer
//                                    in shared memory (see Selector).
//   finish   gates, ids, counts      written by the CTA itself (msplit == 1) or, after the partial lists have been
//                                    parked in scratch, by whichever CTA of the token block finishes last.
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM allocation + MMA issue (the whole warp stays converged and one
// elected lane issues; see tc_mma_bf16_ts_elect), warps 2..9 = epilogue (warp w reads TMEM lanes 32*(w%4).. of
// accumulator (w-2)/4).  Two CTAs are resident per SM (256 TMEM columns and ~112 KB of shared memory each): while one
// group's epilogue drains its accumulator the MMAs of the other three groups of the SM run.  The same kernel with
// FULL = true is the fused standard router (no z; every step contracts over all of h).
//
// Every mbarrier wait is bounded: when the budget runs out the thread records MORE_ERR_TIMEOUT in the device
// status word, raises the CTA's abort flag and all roles fall through to the common exit (TMEM is freed there).
#include "sm100_common.cuh"
#include "more_select.cuh"

#include <cuda_fp16.h>
#include <limits.h>

// -DMORE_STATS builds count epilogue events and clocks into KernelParams::stats (diagnostics only).
#ifdef MORE_STATS
#define STAT(...) __VA_ARGS__
#else
#define STAT(...)
#endif

namespace more {

namespace {

#ifndef MORE_CAND_CAP
#define MORE_CAND_CAP 8
#endif
// 1: the low-rank router keeps z (the A operand of phase 2) in shared memory, which frees tensor memory for a second
// accumulator per token group; 0: z in tensor memory, one accumulator per group
#ifndef MORE_PAIRED_DBL
#define MORE_PAIRED_DBL 1
#endif
// fused standard router: three stages of (256 x 64 X tile + 64 x 256 W tile) and six candidate slots per token
constexpr int kFullRingBytes = 3 * (kXTileBytes + 4 * 64 * 128) + 6 * kEpilogueThreads * 20;
constexpr int kFallbackSlots = 8;      // tokens re-routed per round of the filter's fallback (one per epilogue warp)

struct KernelParams {
    int T, h, r, M, k, gate_mode, msplit;
    int block_tokens;            // tokens routed per CTA: a multiple of 32, at most 256
    int x_rows;                  // rows of the X tile: 256, or 128 when block_tokens <= 128 (low-rank router only)
    int tiles_total;             // ceil(M / 128)
    int32_t* out_idx;
    float* out_gate;
    int32_t* out_counts;
    float* out_topval;
    float* out_lse;
    int* status;
    unsigned long long* stats;   // diagnostic event counters (only written by -DMORE_STATS builds)
    // scratch (msplit > 1): per token block an arrival counter, per (token, split) a partial list and (m, Z)
    unsigned* counters;
    float* part_val;
    int* part_id;
    float2* part_mz;
    // filter mode: transposed copy of R2 ([M][RPAD] bf16, ranks >= r zero); colnorm[0] = largest column norm of R2,
    // colnorm[1] = largest column norm of the error of its fp16 copy; R2 itself for the fallback sweep; the low halves
    // of z, [CTA][rank / 8][256 threads] x 16 B
    const __nv_bfloat16* r2t;
    const float* colnorm;
    const __nv_bfloat16* R2;
    uint4* zlo;
};

// Final outputs of one token from its sorted list and (m2, z): m2 is the running max in log2 units.
template <int KCAP>
__device__ __forceinline__ void write_token(const KernelParams& p, int64_t row, const TopList<KCAP>& L, float m2,
                                            float zsum, int* hist)
{
    constexpr float kLn2 = 0.6931471805599453f, kLog2e = 1.4426950408889634f;
    const int k = p.k;
    float denom = 0.f;
    if (p.gate_mode == MORE_GATE_TOPK_SOFTMAX) {
#pragma unroll
        for (int q = 0; q < KCAP; ++q)
            if (q < k) denom += ex2f((L.v[q] - L.v[0]) * kLog2e);
    } else {
        denom = zsum;
    }
    const float inv = 1.f / denom;
    const float ref2 = (p.gate_mode == MORE_GATE_TOPK_SOFTMAX) ? L.v[0] * kLog2e : m2;
#pragma unroll
    for (int q = 0; q < KCAP; ++q) {
        if (q < k) {
            p.out_idx[row * k + q] = L.id[q];
            p.out_gate[row * k + q] = ex2f(L.v[q] * kLog2e - ref2) * inv;
            if (p.out_topval) p.out_topval[row * k + q] = L.v[q];
            if ((unsigned)L.id[q] < (unsigned)p.M)            // (non-finite inputs can leave a slot unfilled)
                atomicAdd((hist ? hist : p.out_counts) + L.id[q], 1);
        }
    }
    if (p.out_lse) p.out_lse[row] = (m2 + log2f(zsum)) * kLn2;
}

// ------------------------------------------------------------------------------------------------- the kernel
// FULL = true is the fused STANDARD router (logits = X W with W [h][M], no low-rank bottleneck: Alg. 1 without z, the
// contraction running over K = h): there is no phase 1; every step accumulates 256 experts over all h/64 k-tiles of X
// (256 x 64) and W (64 x 256, four 64 x 64 boxes), so X is re-read from L2 once per 256 experts.  That takes all 512
// tensor-memory columns (two 128-token x 256-expert accumulators) and three 64 KB stages: one CTA per SM.  The epilogue
// is the same, run over four 64-column quarters per step.  map_r2 is then W's map (64 x 64 boxes), map_r1 is unused,
// RPAD is 64.
//
// FILTER = true (low-rank router, top-k-softmax gate, no log-sum-exp): the second contraction runs on one fp16 rounding
// of z (scaled per token by a power of two) against an fp16 copy of R2, i.e. half the MMAs; the selection keeps every
// expert within W = 2E of the running k-th approximate logit, E bounding what the rounding can change, and the
// survivors are rescored in fp32 from the full z and the transposed copy of R2; a token whose zone store overflows is
// routed again by a plain sweep.  The result is the exact top-k of the fp32 logits either way.
template <int RPAD, int KCAP, bool LSE, bool FULL = false, bool FILTER = false>
__global__ void __launch_bounds__(kThreads, 2)
route_tcgen05_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_r1,
                     const __grid_constant__ CUtensorMap map_r2, const KernelParams p)
{
    constexpr int kKSteps = RPAD / 16;                          // UMMA K = 16
    constexpr int kHalf = 64;                                   // experts per accumulator quarter: one 128-byte-wide block
    constexpr int kSubs = FULL ? 4 : 1;                         // quarters per step
    constexpr int kStep = kHalf * kSubs;                        // experts per step
    constexpr int kFullStages = 3, kWBoxBytes = 64 * 128, kFullStageBytes = kXTileBytes + 4 * kWBoxBytes;
    constexpr int kRing = FULL ? kFullRingBytes : kRingBytes;
    constexpr int kR2StageBytes = RPAD * 128;                   // RPAD rows x 64 experts
    // candidate slots per token (the standard router keeps the two 40 KB k-tile stages next to the buffers)
    // DBL (r <= 32): z is written to shared memory as one K-major 128 x 64 bf16 tile per token group (a row is
    // [hi | lo] of one token, the layout of an X tile) and read by the phase-2 MMAs from there, so each group has two
    // 64-column accumulators: the MMAs of step n + 1 run while the group still selects from step n, and a warp that
    // stops to fold its candidates no longer stalls the group's next accumulator.  (At r = 64 the tiles take 64 KB,
    // which leaves room for six candidate slots and two R2 stages only: measured slower, 390 against 375 us on c3, and
    // 380 with the overflow check run twice per chunk so that six slots fold as rarely as eight: the waits then move
    // from the accumulators to the two R2 stages;
    // so is keeping only the hi half in shared memory, lo in 32 tensor-memory columns and sweeping 48 experts per step
    // with two 48-column accumulators: 387 us, a third more steps with their hand-overs.
    // With the softmax sweep the epilogue is bound by its instructions, not by the hand-over: no gain, so not used.)
    constexpr bool DBL = !FULL && !FILTER && !LSE && RPAD <= 32 && (MORE_PAIRED_DBL != 0);
    constexpr int kZopTileBytes = 128 * 128;                    // 128 tokens x 64 bf16
    constexpr int kZopBytes = DBL ? 2 * kZopTileBytes : 0;      // [group]
    constexpr int kCandCap = FULL ? 6 : MORE_CAND_CAP;
    using Sel = Selector<KCAP, FILTER, kEpilogueThreads, kCandCap, 4>;
    STAT(constexpr int kCandValStride = Sel::kCandValStride;)
    constexpr int kCandValBytes = Sel::kCandValBytes;
    constexpr int kZoneOff = Sel::kCandBytes;                     // filter: the zone store follows the candidates
    constexpr int kCandBytes = Sel::kCandBytes + (FILTER ? Sel::kZoneBytes : 0);
    constexpr int kMmas2 = FILTER ? kKSteps : 2 * kKSteps;      // exact modes: hi then lo into one accumulator
    // R2 blocks in flight: what the ring has room for next to the candidate buffers, at most 8 (unused by FULL)
    constexpr int kStagesFit = (kRing - kZopBytes - kCandBytes) / kR2StageBytes;
    constexpr int kStagesP2 = FULL ? 1 : (kStagesFit < 8 ? kStagesFit : 8);
    static_assert(FULL || kStagesP2 >= 2, "no room for the R2 pipeline");
    constexpr int kCandOffset = FULL ? kFullStages * kFullStageBytes : kZopBytes;
    static_assert(kCandOffset + kCandBytes + (FULL ? 0 : kStagesP2 * kR2StageBytes) <= kRing, "phase-2 layout does not fit");
    // Tensor-memory columns of this CTA: [0, 128) the two 64-column fp32 accumulators (phase 1: z, phase 2: logits),
    // [128, 256) the two A operands of phase 2, z as bf16 [hi | lo], two K-elements per column.  FULL: two 256-column
    // accumulators, all 512 columns.
    constexpr uint32_t kAccCols = FULL ? 256 : 64, kZopCol0 = 128;
    constexpr uint32_t kAccStride = DBL ? 128 : kAccCols;       // columns between the two groups' accumulators
    constexpr int kAccBufs = DBL ? 2 : 1;                       // accumulators per group (64 columns apart)
    constexpr uint32_t kTmemAlloc = FULL ? 512 : kTmemCols;
    constexpr float kLog2e = 1.4426950408889634f;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;            // 1024-aligned: the 128-B swizzle repeats every 1 KB
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    uint8_t* ctl = ring_ptr + kRing;                         // control block
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctl);
    // barrier slots
    constexpr int kMaxStagesP1 = 4;
    constexpr int B_FULL1 = 0, B_EMPTY1 = B_FULL1 + kMaxStagesP1, B_ZACC = B_EMPTY1 + kMaxStagesP1, B_ZOP = B_ZACC + 1,
                  B_FULL2 = B_ZOP + 1, B_EMPTY2 = B_FULL2 + 8, B_ACCF = B_EMPTY2 + 8, B_ACCE = B_ACCF + 4,
                  B_COUNT = B_ACCE + 4;                  // accumulator barriers: [group * kAccBufs + buffer]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + B_COUNT * 8 + 4);
    int* last_flag = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 8);
    int* flagged = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 12);      // filter: tokens that need the fallback sweep
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    STAT(const long long st_top = clock64();)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int blk = blockIdx.x / p.msplit, split = blockIdx.x % p.msplit;
    const int tok0 = blk * p.block_tokens;
    // expert tiles of this CTA: an even share of ceil(M/128) tiles
    const int tile_lo = (int)(((long long)p.tiles_total * split) / p.msplit);
    const int tile_hi = (int)(((long long)p.tiles_total * (split + 1)) / p.msplit);
    const int ktiles1 = (p.h + 63) / 64;
    // phase-1 stages: a 128-row X tile (small token blocks) leaves room for four k-tiles in flight instead of two,
    // which matters when a CTA's projection is a chain of L2 round trips rather than a stream
    const int x_tile_bytes = p.x_rows * 128;
    const int st1_bytes = x_tile_bytes + kR1TileBytes;
    const int nst1 = (p.x_rows == 128) ? 4 : kStagesP1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kMaxStagesP1; ++i) { mbar_init(bar(B_FULL1 + i), 1); mbar_init(bar(B_EMPTY1 + i), 1); }
        mbar_init(bar(B_ZACC), 1);
        mbar_init(bar(B_ZOP), kEpilogueThreads);
        for (int i = 0; i < 8; ++i) { mbar_init(bar(B_FULL2 + i), 1); mbar_init(bar(B_EMPTY2 + i), 1); }
        for (int i = 0; i < 4; ++i) { mbar_init(bar(B_ACCF + i), 1); mbar_init(bar(B_ACCE + i), kEpilogueThreads / 2); }
        *abort_flag = 0;
        *last_flag = 0;
        *flagged = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemAlloc)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t cand = ring + kCandOffset;                   // phase 2: candidate buffers
    const uint32_t r2ring = ring + (FULL ? 0 : kCandOffset) + kCandBytes;     // phase 2: R2 stages
    // 64-expert steps of this CTA (the last one of the last tile is skipped when it lies wholly beyond M)
    constexpr int kTile = FULL ? kStep : kTileExperts;          // experts per tile of p.tiles_total
    const int e_lo = tile_lo * kTile;
    const int e_hi = min(tile_hi * kTile, p.M);
    const int nsteps = (e_hi - e_lo + kStep - 1) / kStep;

    if (warp == 0) {
        // ===================================================================================== TMA producer
        if (lane == 0 && FULL) {
            // standard router: for every 256-expert step, all k-tiles of X and of W[:, step]
            bool ok = true;
            const int total = nsteps * ktiles1;
            for (int g = 0; g < total && ok; ++g) {
                const int s = g % kFullStages, it = g / ktiles1, kt = g % ktiles1;
                if (g >= kFullStages) ok = mbar_wait(bar(B_EMPTY1 + s), ((g / kFullStages) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = ring + s * kFullStageBytes;
                mbar_expect_tx(bar(B_FULL1 + s), kFullStageBytes);
                tma_load_2d(dst, &map_x, bar(B_FULL1 + s), kt * 64, tok0);            // 256 token rows x 64 columns
                for (int j = 0; j < 4; ++j)                                           // 64 k-rows x 4 x 64 experts
                    tma_load_2d(dst + kXTileBytes + j * kWBoxBytes, &map_r2, bar(B_FULL1 + s), e_lo + it * kStep + j * kHalf,
                                kt * 64);
            }
        } else if (lane == 0) {
            bool ok = true;
            for (int kt = 0; kt < ktiles1 && ok; ++kt) {
                const int s = kt % nst1;
                if (kt >= nst1) ok = mbar_wait(bar(B_EMPTY1 + s), ((kt / nst1) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = ring + s * st1_bytes;
                mbar_expect_tx(bar(B_FULL1 + s), st1_bytes);
                tma_load_2d(dst, &map_x, bar(B_FULL1 + s), kt * 64, tok0);            // x_rows token rows x 64 columns
                tma_load_2d(dst + x_tile_bytes, &map_r1, bar(B_FULL1 + s), 0, kt * 64);
            }
            // the ring is reused by phase 2: wait until every phase-1 MMA has finished reading it
            ok = ok && mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
            for (int it = 0; it < nsteps && ok; ++it) {
                const int s = it % kStagesP2;
                if (it >= kStagesP2) ok = mbar_wait(bar(B_EMPTY2 + s), ((it / kStagesP2) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_FULL2 + s), kR2StageBytes);
                tma_load_2d(r2ring + s * kR2StageBytes, &map_r2, bar(B_FULL2 + s), e_lo + it * kHalf, 0);
            }
        }
    } else if (warp == 1) {
        // ======================================================================================= MMA issuer
        // The whole warp runs this code converged; one elected lane issues each tcgen05 instruction.
        bool ok = true;
        constexpr uint32_t idesc1 = umma_idesc(64);
        constexpr uint32_t idesc2 = FILTER ? umma_idesc_f16(kHalf) : umma_idesc(kHalf);
        if constexpr (FULL) {
            // standard router: per 256-expert step, K runs over all of h through the k-tile stages; each K = 16 slice
            // is four N = 64 instructions, one per 64-expert box of the W tile and accumulator quarter
            const uint64_t xd = umma_desc_sw128(ring, 16, 1024), wd = umma_desc_sw128(ring + kXTileBytes, 8192, 1024);
            const uint32_t x_lo0 = (uint32_t)xd, x_hi = (uint32_t)(xd >> 32), w_lo0 = (uint32_t)wd, w_hi = (uint32_t)(wd >> 32);
            int g = 0;
            for (int it = 0; it < nsteps && ok; ++it) {
                // both accumulators must have been read out (the k-tiles serve both token groups)
#pragma unroll
                for (int a = 0; a < 2; ++a)
                    if (a * 128 < p.block_tokens)
                        ok = __all_sync(kFullMask, ok && mbar_wait(bar(B_ACCE + a), (it & 1) ^ 1, abort_flag, p.status));
                if (!ok) break;
                for (int kt = 0; kt < ktiles1 && ok; ++kt, ++g) {
                    const int s = g % kFullStages;
                    ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL1 + s), (g / kFullStages) & 1, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t x_lo = x_lo0 + s * (kFullStageBytes >> 4), w_lo = w_lo0 + s * (kFullStageBytes >> 4);
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        if (a * 128 >= p.block_tokens) continue;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                tc_mma_bf16_ss_elect(tmem_base + a * kAccCols + j * kHalf, x_lo + a * (16384 >> 4) + kk * 2, x_hi,
                                                     w_lo + j * (kWBoxBytes >> 4) + kk * (2048 >> 4), w_hi, idesc1, (kt | kk) != 0);
                    }
                    tc_commit_elect(bar(B_EMPTY1 + s));
                }
                if (!ok) break;
#pragma unroll
                for (int a = 0; a < 2; ++a)
                    if (a * 128 < p.block_tokens) tc_commit_elect(bar(B_ACCF + a));
            }
        } else {
        {
            // descriptor words of stage 0: K-major X tile (A), MN-major R1 tile (B); +2 per 32 bytes of start address
            const uint64_t xd = umma_desc_sw128(ring, 16, 1024), rd = umma_desc_sw128(ring + x_tile_bytes, 8192, 1024);
            const uint32_t x_lo0 = (uint32_t)xd, x_hi = (uint32_t)(xd >> 32), r_lo0 = (uint32_t)rd, r_hi = (uint32_t)(rd >> 32);
            for (int kt = 0; kt < ktiles1 && ok; ++kt) {
                const int s = kt % nst1;
                ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL1 + s), (kt / nst1) & 1, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t x_lo = x_lo0 + s * (st1_bytes >> 4), r_lo = r_lo0 + s * (st1_bytes >> 4);
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    if (a * 128 >= p.x_rows) continue;      // a 128-row X tile has no second token group
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)      // A: +32 B per K = 16; B: 16 K-rows of 128 B
                        tc_mma_bf16_ss_elect(tmem_base + a * kAccStride, x_lo + a * (16384 >> 4) + kk * 2, x_hi,
                                             r_lo + kk * (2048 >> 4), r_hi, idesc1, (kt | kk) != 0);
                }
                tc_commit_elect(bar(B_EMPTY1 + s));
            }
        }
        if (ok) tc_commit_elect(bar(B_ZACC));
        ok = __all_sync(kFullMask, ok && mbar_wait(bar(B_ZOP), 0, abort_flag, p.status));
        tc_fence_after();
        const uint64_t bd0 = umma_desc_sw128(r2ring, 8192, 1024);
        const uint32_t b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
        const uint64_t zd0 = umma_desc_sw128(ring, 16, 1024);             // DBL: the z tiles, K-major like an X tile
        const uint32_t z_lo0 = (uint32_t)zd0, z_hi = (uint32_t)(zd0 >> 32);
        for (int it = 0; it < nsteps && ok; ++it) {
            const int s = it % kStagesP2;
            ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL2 + s), (it / kStagesP2) & 1, abort_flag, p.status));
            if (!ok) break;
            const uint32_t b_lo = b_lo0 + s * (kR2StageBytes >> 4);
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                if (a * 128 >= p.block_tokens) continue;     // a group without tokens takes no part in phase 2
                if constexpr (DBL) {
                    // accumulator (a, it & 1) is free once its 128 epilogue threads have read step it - 2 out of it
                    const int buf = it & 1;
                    ok = __all_sync(kFullMask, ok && mbar_wait(bar(B_ACCE + a * 2 + buf), ((it >> 1) & 1) ^ 1, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    // A from shared memory: K runs over the row [hi | lo], +32 B per K = 16
                    if constexpr (RPAD <= 32)
                        tc_mma_buffer_ss<kMmas2, kKSteps>(tmem_base + a * kAccStride + buf * kAccCols,
                                                          z_lo0 + a * (kZopTileBytes >> 4), z_hi, b_lo, b_hi, idesc2);
                    tc_commit_elect(bar(B_ACCF + a * 2 + buf));
                } else {
                    // accumulator a is free once its 128 epilogue threads have read the previous step out of it
                    ok = __all_sync(kFullMask, ok && mbar_wait(bar(B_ACCE + a), (it & 1) ^ 1, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    // K runs over [hi | lo]: 8 columns of A, 16 rows of B per instruction; one instruction sequence, one election
                    tc_mma_buffer_ts<kMmas2, kKSteps>(tmem_base + a * kAccCols, tmem_base + kZopCol0 + a * 64, b_lo, b_hi, idesc2);
                    tc_commit_elect(bar(B_ACCF + a));
                }
            }
            if (!ok) break;
            tc_commit_elect(bar(B_EMPTY2 + s));
        }
        }   // !FULL
    } else {
        // ========================================================================================= epilogue
        const int q = warp & 3;                              // TMEM lane group this warp may read
        const int acc = (warp - 2) >> 2;                     // which 128-token accumulator
        const int row_in_acc = q * 32 + lane;
        const int row_in_blk = acc * 128 + row_in_acc;
        const int64_t row = (int64_t)tok0 + row_in_blk;
        const bool row_live = row_in_blk < p.block_tokens && row < p.T;     // rows past the block belong to the next CTA
        const bool warp_live = acc * 128 + q * 32 < p.block_tokens;         // warp-uniform: block_tokens is a multiple of 32
        const uint32_t t_lane0 = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kAccStride;    // the group's (first) accumulator
        const uint32_t t_zop = tmem_base + ((uint32_t)(q * 32) << 16) + kZopCol0 + acc * 64;
        STAT(const long long st_k0 = clock64();)
        bool ok = FULL ? true : mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
        STAT(const long long st_k1 = clock64();)
        const int etid0 = threadIdx.x - 64;                  // 0..255 among the epilogue threads
        // filter: low half of this thread's z, 16 B per 8 ranks, in global scratch (read back once, for rescoring)
        uint4* zlo = FILTER ? p.zlo + (size_t)blockIdx.x * (RPAD / 8) * kEpilogueThreads + etid0 : nullptr;
        float zone_w = 0.f, zscale = 1.f;                    // filter: zone width; z = (hi + lo) * zscale
        if (ok && !FULL) {
            // ---- narrow z and store it to tensor memory as the A operand of phase 2: bf16 [hi | lo], or (filter) z
            // scaled by a power of two and rounded to fp16
            tc_fence_after();
            float lo2 = 0.f, z2 = 0.f, down = 1.f;
            if (FILTER) {
                // power of two that brings the token's largest |z| into [2^13, 2^14)
                float zmax = 0.f;
#pragma unroll
                for (int c = 0; c < RPAD / 16; ++c) {
                    float z[16];
                    tmem_ld16(t_lane0 + c * 16, z);
                    tmem_ld_wait16(z);
#pragma unroll
                    for (int e = 0; e < 16; ++e) zmax = fmaxf(zmax, fabsf(z[e]));
                }
                int ex = (int)((__float_as_uint(zmax) >> 23) & 0xffu) - 127;      // floor(log2 zmax) for normal zmax
                ex = (zmax > 0.f && zmax < INFINITY) ? max(-100, min(100, ex - 13)) : 0;
                zscale = __uint_as_float((uint32_t)(127 + ex) << 23);
                down = __uint_as_float((uint32_t)(127 - ex) << 23);
            }
#pragma unroll
            for (int c = 0; c < RPAD / 16; ++c) {
                float z[16];
                tmem_ld16(t_lane0 + c * 16, z);
                tmem_ld_wait16(z);
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    if (FILTER) {
                        const float z0 = z[2 * e] * down, z1 = z[2 * e + 1] * down;
                        const __half2 h = __floats2half2_rn(z0, z1);
                        const float2 hf = __half22float2(h);
                        const float d0 = z0 - hf.x, d1 = z1 - hf.y;
                        const __half2 l = __floats2half2_rn(d0, d1);
                        hi[e] = *reinterpret_cast<const uint32_t*>(&h);
                        lo[e] = *reinterpret_cast<const uint32_t*>(&l);
                        // the part of z the approximate logits do not see, and the size of z itself
                        lo2 = fmaf(d0, d0, lo2);
                        lo2 = fmaf(d1, d1, lo2);
                        z2 = fmaf(z0, z0, z2);
                        z2 = fmaf(z1, z1, z2);
                    } else {
                        const __nv_bfloat16 h0 = __float2bfloat16_rn(z[2 * e]), h1 = __float2bfloat16_rn(z[2 * e + 1]);
                        const __nv_bfloat16 l0 = __float2bfloat16_rn(z[2 * e] - __bfloat162float(h0));
                        const __nv_bfloat16 l1 = __float2bfloat16_rn(z[2 * e + 1] - __bfloat162float(h1));
                        hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                        lo[e] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
                    }
                }
                if constexpr (DBL) {
                    // row `row_in_acc` of the group's tile (128-byte rows, 1 KB per 8 rows): ranks 16c .. 16c+15 of hi are
                    // the 16-byte chunks 2c and 2c+1, those of lo follow the RPAD/8 chunks of hi; a chunk is stored at
                    // chunk index ^ (row % 8): the 128-byte swizzle
                    const uint32_t zrow = ring + acc * kZopTileBytes + (row_in_acc >> 3) * 1024 + (row_in_acc & 7) * 128;
                    const uint32_t x7 = row_in_acc & 7;
                    const uint32_t h0 = ((2 * c) ^ x7) * 16, h1 = ((2 * c + 1) ^ x7) * 16;
                    const uint32_t l0 = ((RPAD / 8 + 2 * c) ^ x7) * 16, l1 = ((RPAD / 8 + 2 * c + 1) ^ x7) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(zrow + h0), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(zrow + h1), "r"(hi[4]), "r"(hi[5]), "r"(hi[6]), "r"(hi[7]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(zrow + l0), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(zrow + l1), "r"(lo[4]), "r"(lo[5]), "r"(lo[6]), "r"(lo[7]) : "memory");
                } else {
                    tmem_st8(t_zop + c * 8, hi);
                    if (FILTER) {
                        zlo[(2 * c) * kEpilogueThreads] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                        zlo[(2 * c + 1) * kEpilogueThreads] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
                    } else {
                        tmem_st8(t_zop + RPAD / 2 + c * 8, lo);
                    }
                }
            }
            if constexpr (DBL) {
                fence_async_smem();              // the tiles are read by the tensor core (async proxy)
                tc_fence_before();               // ... and this thread's loads of z are complete
            } else {
                tmem_st_wait();
                tc_fence_before();
            }
            mbar_arrive(bar(B_ZOP));
            if (FILTER) {
                // |approximate - fp32 logit| (both in the scaled units of this token) <= |z - hi|_2 |R2_j|_2 for the
                // part of z the sweep does not see, + |z|_2 |R2_j - fp16(R2_j)|_2 for what the fp16 copy of R2 lost,
                // + the accumulation rounding of the two evaluations, bounded by 2^-18 |z|_2 |R2_j|_2 (a generous
                // multiple of fp32 epsilon).
                const float cn = __ldg(p.colnorm), cerr = __ldg(p.colnorm + 1);
                const float e_bound = sqrtf(lo2) * cn * 1.001f + sqrtf(z2) * (cn * 3.8147e-6f + cerr * 1.001f);
                // (e_bound is zero only for z = 0, where every logit is exactly zero either way)
                zone_w = (e_bound == e_bound) ? 2.f * e_bound * 1.001f : INFINITY;
            }
        }

        Sel S;
        S.init(cand + row_in_blk * 16, cand + kCandValBytes + row_in_blk * 4, cand + kZoneOff + row_in_blk * 4, zone_w);
        STAT(unsigned st_chunks = 0, st_hit = 0, st_app = 0, st_rcall = 0, st_riter = 0; long long st_twait = 0, st_tproc = 0, st_tref = 0;
             const long long st_t0 = clock64();)
        float m2 = -INFINITY, zsum = 0.f;                    // running max (log2 units) and sum of 2^(y - m2)

        // `ok` is kept warp-uniform from here on (tcgen05.ld, elect and the votes below need all 32 lanes).
        ok = __all_sync(kFullMask, ok);

        const bool group_live = acc * 128 < p.block_tokens;
        for (int it = 0; it < nsteps && ok && group_live; ++it) {
            int e0 = e_lo + it * kStep;
            bool ragged = e0 + kHalf > p.M;
            float va[16], vb[16];
            // ---- one 16-column chunk: group-of-four maxima, optional online softmax update, candidate scan
            auto process = [&](float (&v)[16], int col0) {
#ifdef MORE_EXP_NOPROC
                return;
#endif
                if (ragged) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (col0 + i >= p.M) v[i] = -INFINITY;
                }
                float t[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) t[i] = fmaxf(max3(v[4 * i], v[4 * i + 1], v[4 * i + 2]), v[4 * i + 3]);
                const float cmax = fmaxf(max3(t[0], t[1], t[2]), t[3]);
                if (LSE) {
                    const float c2 = cmax * kLog2e;
                    if (c2 > m2) { zsum *= ex2f(m2 - c2); m2 = c2; }
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        a0 += ex2f(fmaf(v[i], kLog2e, -m2));
                        a1 += ex2f(fmaf(v[i + 1], kLog2e, -m2));
                        a2 += ex2f(fmaf(v[i + 2], kLog2e, -m2));
                        a3 += ex2f(fmaf(v[i + 3], kLog2e, -m2));
                    }
                    zsum += (a0 + a1) + (a2 + a3);
                }
                // Append this chunk's candidate groups (a warp-uniform branch around predicated stores), then fold
                // the buffers into the lists if some token of the warp is running out of slots.
                STAT(st_chunks++;)
#ifdef MORE_EXP_NOSCAN
                m2 = fmaxf(m2, cmax);
                return;
#endif
                if (__any_sync(kFullMask, cmax > S.thr)) {
                    STAT(st_hit++; const uint32_t mark = S.ptr;)
                    S.scan(v, t, col0);
                    STAT(st_app += __reduce_add_sync(kFullMask, (S.ptr - mark) / kCandValStride);)
                    if (__any_sync(kFullMask, S.ptr >= S.warn)) {
                        // some token is about to run out of slots: fold now
                        STAT(st_rcall++; const long long tr0 = clock64();)
                        S.fold();
                        STAT(st_tref += clock64() - tr0;)
                    }
                }
            };
            STAT(const long long tw0 = clock64();)
            // the accumulator of this step: the group's only one, or (DBL) its buffer it & 1, in use every other step
            const int abuf = DBL ? (it & 1) : 0;
            const int abar = acc * kAccBufs + abuf;
            const uint32_t t_lane = t_lane0 + abuf * kAccCols;
            ok = __all_sync(kFullMask, mbar_wait(bar(B_ACCF + abar), (DBL ? (it >> 1) : it) & 1, abort_flag, p.status));
            STAT(const long long tw1 = clock64(); st_twait += tw1 - tw0;)
            if (!ok) break;
            if (!warp_live) {                                // nothing to select for these rows: just hand the buffer back
                mbar_arrive(bar(B_ACCE + abar));
                continue;
            }
            tc_fence_after();
#pragma unroll 1
            for (int sub = 0; sub < kSubs; ++sub, e0 += kHalf) {      // (one 64-column quarter unless FULL)
                const uint32_t t_sub = t_lane + sub * kHalf;
                ragged = e0 + kHalf > p.M;
                // columns 0-31: the load of the next 16 columns is in flight while the current 16 are processed
                tmem_ld16(t_sub, va);
                tmem_ld_wait16(va);
                tmem_ld16(t_sub + 16, vb);
                process(va, e0);
                tmem_ld_wait16(vb);
                tmem_ld16(t_sub + 32, va);
                process(vb, e0 + 16);
                // columns 32-63: both halves are brought into registers first; after the last quarter the accumulator
                // can then be handed back, and the next step's MMAs run while these 32 columns are processed
                tmem_ld_wait16(va);
                tmem_ld16(t_sub + 48, vb);
                tmem_ld_wait16(vb);
                if (sub == kSubs - 1) {
                    tc_fence_before();
                    mbar_arrive(bar(B_ACCE + abar));
                }
                process(va, e0 + 32);
                process(vb, e0 + 48);
            }
            STAT(st_tproc += clock64() - tw1;)
        }
        S.fold();
        TopList<KCAP>& L = S.L;

        if (FILTER && warp_live && group_live && ok) {
            // ---- rescoring: fp32 logits of the list and of the zone from the full z = (hi + lo) * zscale and the
            // experts' columns (rows of the transposed copy of R2); the exact values decide the final order
            S.prune();
            const int zcount = (int)((S.zptr - S.zbase) / Sel::kZoneStride);
            int zmax = zcount;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) zmax = max(zmax, __shfl_xor_sync(kFullMask, zmax, o));
            float acc[KCAP];
#pragma unroll
            for (int e = 0; e < KCAP; ++e) acc[e] = 0.f;
            auto z_chunk = [&](int c, float (&z8)[8]) {             // ranks 8c .. 8c+7 of this token's z
                uint32_t h4[4];
                tmem_ld4(t_zop + c * 4, h4);
                const uint4 lv = zlo[c * kEpilogueThreads];
                const uint32_t l4[4] = {lv.x, lv.y, lv.z, lv.w};
                tmem_ld_wait4(h4);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&h4[e]));
                    const float2 lf = __half22float2(*reinterpret_cast<const __half2*>(&l4[e]));
                    z8[2 * e] = (hf.x + lf.x) * zscale;
                    z8[2 * e + 1] = (hf.y + lf.y) * zscale;
                }
            };
            auto dot8 = [&](float a, const float (&z8)[8], const uint4& w) {
                a = fmaf(z8[0], bf_lo(w.x), a); a = fmaf(z8[1], bf_hi(w.x), a);
                a = fmaf(z8[2], bf_lo(w.y), a); a = fmaf(z8[3], bf_hi(w.y), a);
                a = fmaf(z8[4], bf_lo(w.z), a); a = fmaf(z8[5], bf_hi(w.z), a);
                a = fmaf(z8[6], bf_lo(w.w), a); a = fmaf(z8[7], bf_hi(w.w), a);
                return a;
            };
            const uint4* r2t = reinterpret_cast<const uint4*>(p.r2t);
            for (int c = 0; c < RPAD / 8; ++c) {
                float z8[8];
                z_chunk(c, z8);
#pragma unroll
                for (int e = 0; e < KCAP; ++e) {
                    if ((unsigned)L.id[e] < (unsigned)p.M) {
                        const uint4 w = __ldg(r2t + (size_t)L.id[e] * (RPAD / 8) + c);
                        acc[e] = dot8(acc[e], z8, w);
                    }
                }
            }
            TopList<KCAP> F;
            F.init();
#pragma unroll
            for (int e = 0; e < KCAP; ++e)
                if ((unsigned)L.id[e] < (unsigned)p.M) F.insert_ordered(acc[e], L.id[e]);
            for (int zi = 0; zi < zmax; ++zi) {
                const bool have = zi < zcount;
                const int id = have ? lds_s32(S.zbase + Sel::kZoneIdOff + zi * Sel::kZoneStride) : -1;
                float a = 0.f;
                for (int c = 0; c < RPAD / 8; ++c) {
                    float z8[8];
                    z_chunk(c, z8);
                    if ((unsigned)id < (unsigned)p.M) a = dot8(a, z8, __ldg(r2t + (size_t)id * (RPAD / 8) + c));
                }
                if ((unsigned)id < (unsigned)p.M) F.insert_ordered(a, id);
            }
            L = F;
        }
#ifdef MORE_STATS
        if (lane == 0 && p.stats) {
            atomicAdd(p.stats + 0, (unsigned long long)st_chunks);
            atomicAdd(p.stats + 1, (unsigned long long)st_hit);
            atomicAdd(p.stats + 3, (unsigned long long)st_app);
            atomicAdd(p.stats + 4, (unsigned long long)st_rcall);
            atomicAdd(p.stats + 5, (unsigned long long)st_riter);
            atomicAdd(p.stats + 8, (unsigned long long)st_twait);
            atomicAdd(p.stats + 9, (unsigned long long)st_tproc);
            atomicAdd(p.stats + 10, (unsigned long long)(clock64() - st_t0));
            atomicAdd(p.stats + 11, 1ull);
            atomicAdd(p.stats + 12, (unsigned long long)st_tref);
            atomicAdd(p.stats + 13, (unsigned long long)(st_k1 - st_k0));
            atomicAdd(p.stats + 14, (unsigned long long)(st_t0 - st_k1));
            atomicAdd(p.stats + 2, (unsigned long long)(st_k0 - st_top));
        }
#endif

        // ---- finish.  All 256 epilogue threads meet here, also after an abort, so the decision is uniform.
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // Expert histogram: when the M bins fit into the (now idle) ring, the CTA counts its tokens' ids in shared
        // memory and flushes only the non-zero bins with one global atomic each; otherwise straight to global memory
        // (with that many experts the bins hardly collide).  With few experts thousands of pairs hit each bin, and
        // same-address global atomics would serialise.
        const int etid = threadIdx.x - 64;                   // 0..255 among the epilogue threads
        if constexpr (FILTER) {
            // ---- fallback: tokens whose zone overflowed are routed again, exactly, over this CTA's experts; the result
            // replaces the token's list.  Rounds of kFallbackSlots tokens, one warp per token.
            auto epi_sync = [&]() { asm volatile("bar.sync 1, 256;" ::: "memory"); };
            if (S.overflow && row_live) atomicAdd(flagged, 1);
            epi_sync();
            const int nflag = (*abort_flag == 0) ? *flagged : 0;
            if (nflag > 0) {
                float* fz = reinterpret_cast<float*>(ring_ptr);                          // [slot][RPAD] z
                float* fv = fz + kFallbackSlots * RPAD;                                   // [slot][KCAP]
                int* fi = reinterpret_cast<int*>(fv + kFallbackSlots * KCAP);
                int* ticket = fi + kFallbackSlots * KCAP;
                if (etid == 0) *ticket = 0;
                epi_sync();
                bool mine = S.overflow && row_live;
                for (int done = 0; done < nflag; done += kFallbackSlots) {
                    int slot = -1;
                    if (mine) {
                        const int t = atomicAdd(ticket, 1);
                        if (t < done + kFallbackSlots) slot = t - done; else atomicSub(ticket, 1);
                    }
                    // the token's z: the high part comes from tensor memory, which only whole warps can read
                    if (warp_live && group_live && __any_sync(kFullMask, slot >= 0)) {
                        for (int c = 0; c < RPAD / 8; ++c) {
                            uint32_t h4[4];
                            tmem_ld4(t_zop + c * 4, h4);
                            const uint4 lv = zlo[c * kEpilogueThreads];
                            const uint32_t l4[4] = {lv.x, lv.y, lv.z, lv.w};
                            tmem_ld_wait4(h4);
                            if (slot >= 0) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&h4[e]));
                                    const float2 lf = __half22float2(*reinterpret_cast<const __half2*>(&l4[e]));
                                    fz[slot * RPAD + c * 8 + 2 * e] = (hf.x + lf.x) * zscale;
                                    fz[slot * RPAD + c * 8 + 2 * e + 1] = (hf.y + lf.y) * zscale;
                                }
                            }
                        }
                    }
                    epi_sync();
                    const int nslots = min(kFallbackSlots, nflag - done);
                    if (warp - 2 < nslots)
                        exact_topk_warp<KCAP>(fz + (warp - 2) * RPAD, p.R2, p.r, p.M, e_lo, e_hi, fv + (warp - 2) * KCAP,
                                              fi + (warp - 2) * KCAP, lane);
                    epi_sync();
                    if (slot >= 0) {
#pragma unroll
                        for (int e = 0; e < KCAP; ++e) { L.v[e] = fv[slot * KCAP + e]; L.id[e] = fi[slot * KCAP + e]; }
                        mine = false;
                    }
                    epi_sync();
                }
            }
        }
        int* hist = (p.M <= kRingBytes / 4) ? reinterpret_cast<int*>(ring_ptr) : nullptr;
        auto hist_clear = [&]() {
            if (hist) {
                for (int e = etid; e < p.M; e += kEpilogueThreads) hist[e] = 0;
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
        };
        auto hist_flush = [&]() {
            if (hist) {
                asm volatile("bar.sync 1, 256;" ::: "memory");
                for (int e = etid; e < p.M; e += kEpilogueThreads) {
                    const int c = hist[e];
                    if (c) atomicAdd(p.out_counts + e, c);
                }
            }
        };
        if (*abort_flag == 0) {
            if (p.msplit == 1) {
                hist_clear();
                if (row_live) write_token<KCAP>(p, row, L, m2, zsum, hist);
                hist_flush();
            } else {
                // park the partial list; the CTA that arrives last for this token block merges all of them
                const int64_t slot = ((int64_t)blk * kBlockTokens + row_in_blk) * p.msplit + split;
#pragma unroll
                for (int s = 0; s < KCAP; ++s) {
                    p.part_val[slot * KCAP + s] = L.v[s];
                    p.part_id[slot * KCAP + s] = L.id[s];
                }
                p.part_mz[slot] = make_float2(m2, zsum);
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (threadIdx.x == 64) {
                    const unsigned prev = atomicAdd(p.counters + blk, 1u);
                    *last_flag = (prev == (unsigned)p.msplit - 1u);
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (*last_flag) {
                    __threadfence();
                    const int64_t base = ((int64_t)blk * kBlockTokens + row_in_blk) * p.msplit;
                    TopList<KCAP> G;
                    G.init();
                    float gm = -INFINITY, gz = 0.f;
                    // A token's partial lists lie one after the other in scratch.  Each list's head (its four best
                    // entries, which is all most lists contribute) is fetched with two 16-byte loads, and the next
                    // list's head is requested before the current one is merged, so the L2 round trips overlap
                    // instead of adding up; the tail of a list is read only if its fourth entry still got in.
                    const float4* pv = reinterpret_cast<const float4*>(p.part_val + base * KCAP);
                    const int4* pi = reinterpret_cast<const int4*>(p.part_id + base * KCAP);
                    float4 hv = __ldcg(pv);
                    int4 hi = __ldcg(pi);
                    for (int sp = 0; sp < p.msplit; ++sp) {       // ascending expert ranges: ties keep the smaller id
                        const float4 cv = hv;
                        const int4 ci = hi;
                        if (sp + 1 < p.msplit) {
                            hv = __ldcg(pv + (size_t)(sp + 1) * (KCAP / 4));
                            hi = __ldcg(pi + (size_t)(sp + 1) * (KCAP / 4));
                        }
                        // each partial list is sorted: stop at the first entry that does not get in
                        bool more = cv.x > G.tau();
                        if (more) G.insert(cv.x, ci.x);
                        more = more && cv.y > G.tau();
                        if (more) G.insert(cv.y, ci.y);
                        more = more && cv.z > G.tau();
                        if (more) G.insert(cv.z, ci.z);
                        more = more && cv.w > G.tau();
                        if (more) G.insert(cv.w, ci.w);
                        for (int s = 4; s < KCAP && more; ++s) {
                            const float x = __ldcg(p.part_val + (base + sp) * KCAP + s);
                            const int j = __ldcg(p.part_id + (base + sp) * KCAP + s);
                            more = x > G.tau();
                            if (more) G.insert(x, j);
                        }
                        const float2 mz = __ldcg(p.part_mz + base + sp);
                        if (LSE && mz.x > -INFINITY) {
                            const float nm = fmaxf(gm, mz.x);
                            gz = gz * ex2f(gm - nm) + mz.y * ex2f(mz.x - nm);
                            gm = nm;
                        }
                    }
                    hist_clear();
                    if (row_live) write_token<KCAP>(p, row, G, gm, gz, hist);
                    hist_flush();
                    if (threadIdx.x == 64) p.counters[blk] = 0;   // ready for the next call
                }
            }
        }
    }

    // ---- common exit: everyone arrives here, also after an abort
    tc_fence_before();
    __syncthreads();
    STAT(if (threadIdx.x == 64 && p.stats) {
        atomicAdd(p.stats + 6, (unsigned long long)(clock64() - st_top));      // CTA lifetime, clk
        atomicMax(p.stats + 7, (unsigned long long)(clock64() - st_top));      // longest CTA
        atomicAdd(p.stats + 15, 1ull);
    })
    if (*abort_flag && threadIdx.x == 0) {
        // give bulk copies that may still be in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemAlloc) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// 2-D bf16 row-major tensor [rows][cols], box = box_cols x box_rows, 128-byte swizzle, zero fill out of bounds.
struct MapKey {
    const void* ptr;
    int rows, cols, box_rows, box_cols;
    bool operator==(const MapKey& o) const
    {
        return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows && box_cols == o.box_cols;
    }
};
constexpr int kMapCache = 128;
MapKey g_keys[kMapCache];
CUtensorMap g_maps[kMapCache];
int g_map_count = 0, g_map_next = 0;

}  // namespace

int get_tensor_map(const void* ptr, int rows, int cols, int box_rows, int box_cols, CUtensorMap* out)
{
    const MapKey key{ptr, rows, cols, box_rows, box_cols};
    for (int i = 0; i < g_map_count; ++i)
        if (g_keys[i] == key) { *out = g_maps[i]; return MORE_OK; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return MORE_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    CUresult res = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return MORE_ERR_CUDA;
    const int slot = (g_map_count < kMapCache) ? g_map_count++ : (g_map_next++ % kMapCache);
    g_keys[slot] = key;
    g_maps[slot] = m;
    *out = m;
    return MORE_OK;
}

namespace {

template <int RPAD, int KCAP, bool LSE, bool FULL, bool FILTER>
int launch_one(const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2, const KernelParams& kp, int ctas,
               cudaStream_t st, bool clear_counts)
{
    static unsigned long long configured = 0;   // one bit per device, per instantiation; guarded by the API mutex
    constexpr int smem_bytes = (FULL ? kFullRingBytes : kRingBytes) + 2048;    // + alignment slack + control block
    auto kern = route_tcgen05_kernel<RPAD, KCAP, LSE, FULL, FILTER>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!(configured >> (dev & 63) & 1ull)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess)
            return MORE_ERR_CUDA;
        configured |= 1ull << (dev & 63);
    }
    // every host-side step that can fail is behind us: only now is the first output touched
    if (clear_counts &&
        cudaMemsetAsync(kp.out_counts, 0, (size_t)kp.M * sizeof(int32_t), st) != cudaSuccess)
        return MORE_ERR_CUDA;
    kern<<<ctas, kThreads, smem_bytes, st>>>(mx, m1, m2, kp);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

// mode: 0 exact, 1 exact with the softmax sweep, 2 filter
template <int RPAD, int KCAP, bool FULL>
int launch_mode(int mode, const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2, const KernelParams& kp,
                int ctas, cudaStream_t st, bool clear_counts)
{
    if (mode == 1) return launch_one<RPAD, KCAP, true, FULL, false>(mx, m1, m2, kp, ctas, st, clear_counts);
    if (mode == 0) return launch_one<RPAD, KCAP, false, FULL, false>(mx, m1, m2, kp, ctas, st, clear_counts);
#ifdef MORE_WITH_FILTER
    if constexpr (!FULL && KCAP <= 16) return launch_one<RPAD, KCAP, false, false, true>(mx, m1, m2, kp, ctas, st, clear_counts);
#endif
    return MORE_ERR_SHAPE;
}

template <int RPAD, bool FULL>
int launch_kcap(int k, int mode, const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2,
                const KernelParams& kp, int ctas, cudaStream_t st, bool clear_counts)
{
    if (k <= 8) return launch_mode<RPAD, 8, FULL>(mode, mx, m1, m2, kp, ctas, st, clear_counts);
    if (k <= 16) return launch_mode<RPAD, 16, FULL>(mode, mx, m1, m2, kp, ctas, st, clear_counts);
    return launch_mode<RPAD, 32, FULL>(mode, mx, m1, m2, kp, ctas, st, clear_counts);
}

int kcap_of(int k) { return k <= 8 ? 8 : (k <= 16 ? 16 : 32); }
size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct PairedScratch {
    size_t counters, part_val, part_id, part_mz, r2t, r2h, partial, zlo, total;
};

PairedScratch paired_layout(const RouteArgs& a, const Plan& p)
{
    PairedScratch L{};
    size_t off = 0;
    if (p.msplit > 1) {
        const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
        const size_t slots = blocks * kBlockTokens * (size_t)p.msplit;
        const size_t kc = (size_t)kcap_of(a.k);
        L.counters = off; off += align_up(blocks * 4, 256);
        L.part_val = off; off += align_up(slots * kc * 4, 256);
        L.part_id = off; off += align_up(slots * kc * 4, 256);
        L.part_mz = off; off += align_up(slots * 8, 256);
    }
    if (p.filter) {
        const size_t rpad = a.r <= 16 ? 16 : (a.r <= 32 ? 32 : 64);
        L.r2t = off; off += align_up((size_t)a.M * rpad * 2, 256);
        L.r2h = off; off += align_up((size_t)a.M * a.r * 2, 256);
        L.partial = off; off += align_up((size_t)((a.M + 63) / 64) * 8, 256);
        L.zlo = off; off += align_up((size_t)p.ctas * (rpad / 8) * kEpilogueThreads * 16, 256);
    }
    L.total = off;
    return L;
}

}  // namespace

size_t full_scratch_bytes(const RouteArgs& a, const Plan& p) { return paired_layout(a, p).total; }
size_t paired_scratch_bytes(const RouteArgs& a, const Plan& p) { return paired_layout(a, p).total; }

// The kernel of this file for either router: the fused standard router (a.full) or the low-rank router with 256-token
// CTAs, two per SM ("paired": two 128-token groups per CTA).
int launch_paired(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch)
{
    const PairedScratch L = paired_layout(a, p);
    char* base = static_cast<char*>(scratch);
    const int rpad = a.full ? 64 : (a.r <= 16 ? 16 : (a.r <= 32 ? 32 : 64));
    const int x_rows = (!a.full && p.block_tokens <= 128) ? 128 : kBlockTokens;
    CUtensorMap mx, m1, m2;
    int rc = get_tensor_map(a.X, a.T, a.h, x_rows, 64, &mx);
    if (a.full) {
        // W [h][M]: its k-tiles are 64 x 64 boxes
        if (rc == MORE_OK) rc = get_tensor_map(a.R2, a.h, a.M, 64, 64, &m2);
        m1 = m2;
    } else {
        if (rc == MORE_OK) rc = get_tensor_map(a.R1, a.h, a.r, 64, 64, &m1);
        // the filter sweeps the fp16 copy of R2 in scratch (same shape; a 16-bit type either way as far as TMA cares)
        if (rc == MORE_OK)
            rc = get_tensor_map(p.filter ? static_cast<const void*>(base + L.r2h) : a.R2, a.r, a.M, rpad, 64, &m2);
    }
    if (rc != MORE_OK) return rc;

    KernelParams kp{};
    kp.T = a.T; kp.h = a.h; kp.r = a.r; kp.M = a.M; kp.k = a.k; kp.gate_mode = a.gate_mode; kp.msplit = p.msplit;
    kp.block_tokens = p.block_tokens;
    kp.x_rows = x_rows;
    kp.tiles_total = a.full ? (a.M + 255) / 256 : (a.M + kTileExperts - 1) / kTileExperts;
    kp.out_idx = a.out_idx; kp.out_gate = a.out_gate; kp.out_counts = a.out_counts;
    kp.out_topval = a.out_topval; kp.out_lse = a.out_lse;
    kp.status = ctx.status;
    kp.stats = ctx.stats;
    kp.R2 = a.R2;
    if (p.msplit > 1) {
        kp.counters = reinterpret_cast<unsigned*>(base + L.counters);
        kp.part_val = reinterpret_cast<float*>(base + L.part_val);
        kp.part_id = reinterpret_cast<int*>(base + L.part_id);
        kp.part_mz = reinterpret_cast<float2*>(base + L.part_mz);
        const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
        if (cudaMemsetAsync(kp.counters, 0, blocks * 4, a.stream) != cudaSuccess) return MORE_ERR_CUDA;
    }
    const bool lse = (a.gate_mode == MORE_GATE_FULL_SOFTMAX) || (a.out_lse != nullptr);
    int mode = lse ? 1 : 0;
    if (p.filter) {
        if (lse || a.k > 16 || a.full) return MORE_ERR_SHAPE;
        mode = 2;
        kp.r2t = reinterpret_cast<const __nv_bfloat16*>(base + L.r2t);
        kp.colnorm = ctx.colnorm;
        kp.zlo = reinterpret_cast<uint4*>(base + L.zlo);
        // the preparation kernel also clears out_counts
        rc = launch_route_prepare(a, rpad, base + L.r2h, base + L.r2t, base + L.partial, ctx);
        if (rc != MORE_OK) return rc;
    }
    const bool clear = !p.filter;
    if (a.full) return launch_kcap<64, true>(a.k, mode, mx, m1, m2, kp, p.ctas, a.stream, clear);
    switch (rpad) {
        case 16: return launch_kcap<16, false>(a.k, mode, mx, m1, m2, kp, p.ctas, a.stream, clear);
        case 32: return launch_kcap<32, false>(a.k, mode, mx, m1, m2, kp, p.ctas, a.stream, clear);
        default: return launch_kcap<64, false>(a.k, mode, mx, m1, m2, kp, p.ctas, a.stream, clear);
    }
}

int launch_full(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch) { return launch_paired(a, ctx, p, scratch); }

}  // namespace more
