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

#include <limits.h>

// -DMORE_STATS builds count epilogue events and clocks into KernelParams::stats (diagnostics only).
#ifdef MORE_STATS
#define STAT(...) __VA_ARGS__
#else
#define STAT(...)
#endif

namespace more {

namespace {

// Running top-k of one token.  Between refreshes the sorted list is left alone.  A chunk of 16 logits is looked at
// as four groups of four; every group whose maximum beats the cached threshold `tau` (the list's last entry as of
// the last refresh, hence never above the true threshold) is appended whole, in ascending column order, to this
// thread's column of a shared-memory candidate buffer: one predicated 16-byte store of the four values (they sit in
// four consecutive registers as loaded from tensor memory, so nothing is moved), one predicated 4-byte store of the
// group's first column into a parallel array, and no branch.  refresh() then inserts the buffered elements that beat
// the up-to-date threshold, so the inserts of several chunks of all 32 tokens of a warp are executed together.  A
// chunk appends at most 4 entries and the warp refreshes as soon as some token has fewer than 4 free slots left, so
// the buffer cannot overflow.
constexpr int kCandValStride = kEpilogueThreads * 16;     // bytes between successive value slots of one thread
constexpr int kCandColStride = kEpilogueThreads * 4;      // ... and between its column slots
#ifndef MORE_CAND_CAP
#define MORE_CAND_CAP 8
#endif
constexpr unsigned kFullMask = 0xffffffffu;

template <int KCAP, int CAP>
struct Selector {
    static constexpr int kWarnSlots = CAP - 4;            // a chunk must always find 4 free slots
    static_assert(kWarnSlots >= 1, "candidate buffer too small");
    TopList<KCAP> L;
    float tau;
    uint32_t ptr;     // shared-memory address of this thread's next free value slot
    uint32_t cptr;    // ... and of the matching column slot
    uint32_t base, cbase;
    uint32_t warn;    // at or beyond this fill level the warp refreshes after the chunk

    __device__ __forceinline__ void init(uint32_t first_val_slot, uint32_t first_col_slot)
    {
        L.init();
        tau = -INFINITY;
        base = ptr = first_val_slot;
        cbase = cptr = first_col_slot;
        warn = first_val_slot + kWarnSlots * kCandValStride;
    }
    // Called by all 32 lanes of a warp together.  Every round inserts at most one element per token: the maximum
    // of the token's current entry, which is then struck out of the entry; a token whose entry holds nothing above its
    // (rising) threshold any more moves on to its next entries.  The rounds end when no token has anything left, so
    // their number is the largest count of real insertions of any token of the warp, and the (select-only) insert
    // code is executed once per round.
    __device__ __forceinline__ void refresh()
    {
        uint32_t a = base, c = cbase;
        float x0 = -INFINITY, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
        int col = 0;
        for (;;) {
            float m = fmaxf(max3(x0, x1, x2), x3);
            while (!(m > L.tau()) && a < ptr) {
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=f"(x0), "=f"(x1), "=f"(x2), "=f"(x3) : "r"(a) : "memory");
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(col) : "r"(c) : "memory");
                a += kCandValStride;
                c += kCandColStride;
                m = fmaxf(max3(x0, x1, x2), x3);
            }
            const bool pass = m > L.tau();
            if (!__any_sync(kFullMask, pass)) break;
            // the maximum's lowest column on a tie, so that equal logits enter the list in ascending column order
            const int j = (x0 == m) ? 0 : ((x1 == m) ? 1 : ((x2 == m) ? 2 : 3));
            if (pass) L.insert(m, col + j);
            x0 = (j == 0) ? -INFINITY : x0;
            x1 = (j == 1) ? -INFINITY : x1;
            x2 = (j == 2) ? -INFINITY : x2;
            x3 = (j == 3) ? -INFINITY : x3;
        }
        ptr = base;
        cptr = cbase;
        tau = L.tau();
    }
    // if (t > tau) append {v0, v1, v2, v3} and col
    __device__ __forceinline__ void append4(float t, float v0, float v1, float v2, float v3, int col)
    {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.gt.f32 p, %2, %8;\n\t"
            "@p st.shared.v4.b32 [%0], {%3, %4, %5, %6};\n\t"
            "@p st.shared.b32 [%1], %7;\n\t"
            "@p add.u32 %0, %0, %9;\n\t"
            "@p add.u32 %1, %1, %10;\n\t}"
            : "+r"(ptr), "+r"(cptr)
            : "f"(t), "f"(v0), "f"(v1), "f"(v2), "f"(v3), "r"(col), "f"(tau), "n"(kCandValStride), "n"(kCandColStride)
            : "memory");
    }
    // v: 16 logits of columns col0.., t: maxima of the groups (v[4i] .. v[4i+3]).
    __device__ __forceinline__ void scan(const float (&v)[16], const float (&t)[4], int col0)
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) append4(t[i], v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3], col0 + 4 * i);
    }
};

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
// contraction running over K = h): there is no phase 1, every 64-expert step instead accumulates over all h/64 k-tiles
// of X (256 x 64, re-read per step) and W (64 x 64) with the phase-1 pipeline and stage layout, and the epilogue is
// the same.  map_r2 is then W's map (64 x 64 boxes), map_r1 is unused, RPAD is 64.
template <int RPAD, int KCAP, bool LSE, bool FULL = false>
__global__ void __launch_bounds__(kThreads, 2)
route_tcgen05_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_r1,
                     const __grid_constant__ CUtensorMap map_r2, const KernelParams p)
{
    constexpr int kKSteps = RPAD / 16;                          // UMMA K = 16
    constexpr int kHalf = 64;                                   // experts per phase-2 step: one 128-byte-wide R2 block
    constexpr int kR2StageBytes = RPAD * 128;                   // RPAD rows x 64 experts
    // candidate slots per token (the standard router keeps the two 40 KB k-tile stages next to the buffers)
    constexpr int kCandCap = FULL ? 6 : MORE_CAND_CAP;
    using Sel = Selector<KCAP, kCandCap>;
    constexpr int kCandValBytes = kCandCap * kCandValStride;
    constexpr int kCandBytes = kCandCap * (kCandValStride + kCandColStride);
    // R2 blocks in flight: what the ring has room for next to the candidate buffers, at most 8 (unused by FULL)
    constexpr int kStagesFit = (kRingBytes - kCandBytes) / kR2StageBytes;
    constexpr int kStagesP2 = FULL ? 1 : (kStagesFit < 8 ? kStagesFit : 8);
    static_assert(FULL || kStagesP2 >= 2, "no room for the R2 pipeline");
    constexpr int kCandOffset = FULL ? kStagesP1 * kP1StageBytes : 0;
    static_assert(kCandOffset + kCandBytes + (FULL ? 0 : kStagesP2 * kR2StageBytes) <= kRingBytes, "phase-2 layout does not fit");
    // Tensor-memory columns of this CTA: [0, 128) the two 64-column fp32 accumulators (phase 1: z, phase 2: logits),
    // [128, 256) the two A operands of phase 2, z as bf16 [hi | lo], two K-elements per column.
    constexpr uint32_t kAccCols = 64, kZopCol0 = 128;
    constexpr float kLog2e = 1.4426950408889634f;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;            // 1024-aligned: the 128-B swizzle repeats every 1 KB
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    uint8_t* ctl = ring_ptr + kRingBytes;                    // control block
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctl);
    // barrier slots
    constexpr int kMaxStagesP1 = 4;
    constexpr int B_FULL1 = 0, B_EMPTY1 = B_FULL1 + kMaxStagesP1, B_ZACC = B_EMPTY1 + kMaxStagesP1, B_ZOP = B_ZACC + 1,
                  B_FULL2 = B_ZOP + 1, B_EMPTY2 = B_FULL2 + 8, B_ACCF = B_EMPTY2 + 8, B_ACCE = B_ACCF + 2,
                  B_COUNT = B_ACCE + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + B_COUNT * 8 + 4);
    int* last_flag = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 8);
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
        for (int i = 0; i < 2; ++i) { mbar_init(bar(B_ACCF + i), 1); mbar_init(bar(B_ACCE + i), kEpilogueThreads / 2); }
        *abort_flag = 0;
        *last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t cand = ring + kCandOffset;                   // phase 2: candidate buffers
    const uint32_t r2ring = ring + kCandBytes;                  // phase 2: R2 stages
    // 64-expert steps of this CTA (the last one of the last tile is skipped when it lies wholly beyond M)
    const int e_lo = tile_lo * kTileExperts;
    const int e_hi = min(tile_hi * kTileExperts, p.M);
    const int nsteps = (e_hi - e_lo + kHalf - 1) / kHalf;

    if (warp == 0) {
        // ===================================================================================== TMA producer
        if (lane == 0 && FULL) {
            // standard router: for every 64-expert step, all k-tiles of X and of W[:, step]
            bool ok = true;
            const int total = nsteps * ktiles1;
            for (int g = 0; g < total && ok; ++g) {
                const int s = g % kStagesP1, it = g / ktiles1, kt = g % ktiles1;
                if (g >= kStagesP1) ok = mbar_wait(bar(B_EMPTY1 + s), ((g / kStagesP1) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = ring + s * kP1StageBytes;
                mbar_expect_tx(bar(B_FULL1 + s), kP1StageBytes);
                tma_load_2d(dst, &map_x, bar(B_FULL1 + s), kt * 64, tok0);            // 256 token rows x 64 columns
                tma_load_2d(dst + kXTileBytes, &map_r2, bar(B_FULL1 + s), e_lo + it * kHalf, kt * 64);
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
        constexpr uint32_t idesc2 = umma_idesc(kHalf);
        if constexpr (FULL) {
            // standard router: per 64-expert step, K runs over all of h through the two k-tile stages
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
                    const int s = g % kStagesP1;
                    ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL1 + s), (g / kStagesP1) & 1, abort_flag, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t x_lo = x_lo0 + s * (kP1StageBytes >> 4), w_lo = w_lo0 + s * (kP1StageBytes >> 4);
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        if (a * 128 >= p.block_tokens) continue;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            tc_mma_bf16_ss_elect(tmem_base + a * kAccCols, x_lo + a * (16384 >> 4) + kk * 2, x_hi,
                                                 w_lo + kk * (2048 >> 4), w_hi, idesc1, (kt | kk) != 0);
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
                        tc_mma_bf16_ss_elect(tmem_base + a * kAccCols, x_lo + a * (16384 >> 4) + kk * 2, x_hi,
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
        for (int it = 0; it < nsteps && ok; ++it) {
            const int s = it % kStagesP2;
            ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL2 + s), (it / kStagesP2) & 1, abort_flag, p.status));
            if (!ok) break;
            const uint32_t b_lo = b_lo0 + s * (kR2StageBytes >> 4);
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                if (a * 128 >= p.block_tokens) continue;     // a group without tokens takes no part in phase 2
                // accumulator a is free once its 128 epilogue threads have read the previous step out of it
                ok = __all_sync(kFullMask, ok && mbar_wait(bar(B_ACCE + a), (it & 1) ^ 1, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int j = 0; j < 2 * kKSteps; ++j)       // K runs over [hi | lo]: 8 columns of A, 16 rows of B per step
                    tc_mma_bf16_ts_elect(tmem_base + a * kAccCols, tmem_base + kZopCol0 + a * 64 + j * 8,
                                         b_lo + (j % kKSteps) * (2048 >> 4), b_hi, idesc2, j != 0);
                tc_commit_elect(bar(B_ACCF + a));
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
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kAccCols;
        const uint32_t t_zop = tmem_base + ((uint32_t)(q * 32) << 16) + kZopCol0 + acc * 64;
        STAT(const long long st_k0 = clock64();)
        bool ok = FULL ? true : mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
        STAT(const long long st_k1 = clock64();)
        if (ok && !FULL) {
            // ---- narrow z to bf16 [hi | lo] and store it to tensor memory as the A operand of phase 2
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < RPAD / 16; ++c) {
                float z[16];
                tmem_ld16(t_lane + c * 16, z);
                tmem_ld_wait16(z);
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const __nv_bfloat16 h0 = __float2bfloat16_rn(z[2 * e]), h1 = __float2bfloat16_rn(z[2 * e + 1]);
                    const __nv_bfloat16 l0 = __float2bfloat16_rn(z[2 * e] - __bfloat162float(h0));
                    const __nv_bfloat16 l1 = __float2bfloat16_rn(z[2 * e + 1] - __bfloat162float(h1));
                    hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                    lo[e] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
                }
                tmem_st8(t_zop + c * 8, hi);
                tmem_st8(t_zop + RPAD / 2 + c * 8, lo);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar(B_ZOP));
        }

        Sel S;
        S.init(cand + row_in_blk * 16, cand + kCandValBytes + row_in_blk * 4);
        STAT(unsigned st_chunks = 0, st_hit = 0, st_app = 0, st_rcall = 0, st_riter = 0; long long st_twait = 0, st_tproc = 0, st_tref = 0;
             const long long st_t0 = clock64();)
        float m2 = -INFINITY, zsum = 0.f;                    // running max (log2 units) and sum of 2^(y - m2)

        // `ok` is kept warp-uniform from here on (tcgen05.ld, elect and the votes below need all 32 lanes).
        ok = __all_sync(kFullMask, ok);

        const bool group_live = acc * 128 < p.block_tokens;
        for (int it = 0; it < nsteps && ok && group_live; ++it) {
            const int e0 = e_lo + it * kHalf;
            const bool ragged = e0 + kHalf > p.M;
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
                if (__any_sync(kFullMask, cmax > S.tau)) {
                    STAT(st_hit++; const uint32_t mark = S.ptr;)
                    S.scan(v, t, col0);
                    STAT(st_app += __reduce_add_sync(kFullMask, (S.ptr - mark) / kCandValStride);)
                    if (__any_sync(kFullMask, S.ptr >= S.warn)) {
                        // some token is about to run out of slots: fold now
                        STAT(st_rcall++; const long long tr0 = clock64();)
                        S.refresh();
                        STAT(st_tref += clock64() - tr0;)
                    }
                }
            };
            STAT(const long long tw0 = clock64();)
            ok = __all_sync(kFullMask, mbar_wait(bar(B_ACCF + acc), it & 1, abort_flag, p.status));
            STAT(const long long tw1 = clock64(); st_twait += tw1 - tw0;)
            if (!ok) break;
            if (!warp_live) {                                // nothing to select for these rows: just hand the buffer back
                mbar_arrive(bar(B_ACCE + acc));
                continue;
            }
            tc_fence_after();
            // columns 0-31: the load of the next 16 columns is in flight while the current 16 are processed
            tmem_ld16(t_lane, va);
            tmem_ld_wait16(va);
            tmem_ld16(t_lane + 16, vb);
            process(va, e0);
            tmem_ld_wait16(vb);
            tmem_ld16(t_lane + 32, va);
            process(vb, e0 + 16);
            // columns 32-63: both halves are brought into registers first; the accumulator can then be handed back,
            // and the next step's MMAs run while these 32 columns are processed
            tmem_ld_wait16(va);
            tmem_ld16(t_lane + 48, vb);
            tmem_ld_wait16(vb);
            tc_fence_before();
            mbar_arrive(bar(B_ACCE + acc));
            process(va, e0 + 32);
            process(vb, e0 + 48);
            STAT(st_tproc += clock64() - tw1;)
        }
        S.refresh();
        TopList<KCAP>& L = S.L;
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
        int* hist = (p.M * 4 <= kRingBytes) ? reinterpret_cast<int*>(ring_ptr) : nullptr;
        const int etid = threadIdx.x - 64;                   // 0..255 among the epilogue threads
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
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

template <int RPAD, int KCAP, bool LSE, bool FULL>
int launch_one(const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2, const KernelParams& kp, int ctas,
               cudaStream_t st)
{
    static unsigned long long configured = 0;   // one bit per device, per instantiation; guarded by the API mutex
    auto kern = route_tcgen05_kernel<RPAD, KCAP, LSE, FULL>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!(configured >> (dev & 63) & 1ull)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return MORE_ERR_CUDA;
        configured |= 1ull << (dev & 63);
    }
    // every host-side step that can fail is behind us: only now is the first output touched
    if (cudaMemsetAsync(kp.out_counts, 0, (size_t)kp.M * sizeof(int32_t), st) != cudaSuccess) return MORE_ERR_CUDA;
    kern<<<ctas, kThreads, kSmemBytes, st>>>(mx, m1, m2, kp);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

template <int RPAD, int KCAP, bool FULL>
int launch_lse(bool lse, const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2, const KernelParams& kp,
               int ctas, cudaStream_t st)
{
    return lse ? launch_one<RPAD, KCAP, true, FULL>(mx, m1, m2, kp, ctas, st)
               : launch_one<RPAD, KCAP, false, FULL>(mx, m1, m2, kp, ctas, st);
}

template <int RPAD, bool FULL>
int launch_kcap(int k, bool lse, const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2,
                const KernelParams& kp, int ctas, cudaStream_t st)
{
    if (k <= 8) return launch_lse<RPAD, 8, FULL>(lse, mx, m1, m2, kp, ctas, st);
    if (k <= 16) return launch_lse<RPAD, 16, FULL>(lse, mx, m1, m2, kp, ctas, st);
    return launch_lse<RPAD, 32, FULL>(lse, mx, m1, m2, kp, ctas, st);
}

int kcap_of(int k) { return k <= 8 ? 8 : (k <= 16 ? 16 : 32); }
size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

size_t full_scratch_bytes(const RouteArgs& a, const Plan& p)
{
    if (p.msplit <= 1) return 0;
    const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
    const size_t slots = blocks * kBlockTokens * (size_t)p.msplit;
    const size_t kc = (size_t)kcap_of(a.k);
    return align_up(blocks * 4, 256) + align_up(slots * kc * 4, 256) * 2 + align_up(slots * 8, 256);
}

int launch_full(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch)
{
    CUtensorMap mx, m2;
    int rc = get_tensor_map(a.X, a.T, a.h, kBlockTokens, 64, &mx);
    // W [h][M]: its k-tiles are 64 x 64 boxes
    if (rc == MORE_OK) rc = get_tensor_map(a.R2, a.h, a.M, 64, 64, &m2);
    if (rc != MORE_OK) return rc;

    KernelParams kp;
    kp.T = a.T; kp.h = a.h; kp.r = a.r; kp.M = a.M; kp.k = a.k; kp.gate_mode = a.gate_mode; kp.msplit = p.msplit;
    kp.block_tokens = p.block_tokens;
    kp.x_rows = kBlockTokens;
    kp.tiles_total = (a.M + kTileExperts - 1) / kTileExperts;
    kp.out_idx = a.out_idx; kp.out_gate = a.out_gate; kp.out_counts = a.out_counts;
    kp.out_topval = a.out_topval; kp.out_lse = a.out_lse;
    kp.status = ctx.status;
    kp.stats = ctx.stats;
    kp.counters = nullptr; kp.part_val = nullptr; kp.part_id = nullptr; kp.part_mz = nullptr;
    if (p.msplit > 1) {
        const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
        const size_t slots = blocks * kBlockTokens * (size_t)p.msplit;
        const size_t kc = (size_t)kcap_of(a.k);
        char* base = static_cast<char*>(scratch);
        kp.counters = reinterpret_cast<unsigned*>(base);
        base += align_up(blocks * 4, 256);
        kp.part_val = reinterpret_cast<float*>(base);
        base += align_up(slots * kc * 4, 256);
        kp.part_id = reinterpret_cast<int*>(base);
        base += align_up(slots * kc * 4, 256);
        kp.part_mz = reinterpret_cast<float2*>(base);
        if (cudaMemsetAsync(kp.counters, 0, blocks * 4, a.stream) != cudaSuccess) return MORE_ERR_CUDA;
    }
    const bool lse = (a.gate_mode == MORE_GATE_FULL_SOFTMAX) || (a.out_lse != nullptr);
    return launch_kcap<64, true>(a.k, lse, mx, m2, m2, kp, p.ctas, a.stream);
}

}  // namespace more
