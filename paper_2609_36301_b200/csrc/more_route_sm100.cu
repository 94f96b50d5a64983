// Tensor-core path of the fused low-rank router for sm_100a (Algorithm 1 with the gates of Section 2 / Eq. app_softmax
// and the per-expert counts fused in).  One CTA per SM, 18 warps:
//
//   warp 0       TMA producer: X and R1 k-tiles for phase 1, R2 blocks of 64 experts for phase 2.
//   warp 1       tensor-memory allocation and the tcgen05.mma issue of phase 1.
//   warps 2..17  epilogue: four groups of four warps.  A group owns 128 tensor-memory lanes = 128 tokens and one
//                contiguous range of experts; a thread owns one token of its group.  The groups feed themselves in
//                phase 2: whichever warp of a group is the last to have read an accumulator buffer out issues, there
//                and then, the MMAs that refill it (the warp stays converged, one elected lane issues).  A separate
//                issuing warp adds its own wake-up and a chain of slow synchronising instructions to every hand-over,
//                and measured several hundred clocks per 32-column buffer.
//
// A CTA routes `block_tokens` (<= 512) tokens.  Its four groups are laid out as tg token groups x es expert ranges
// (tg * es <= 4): with many tokens per SM every group takes different tokens and sweeps all of the CTA's experts; with
// few tokens per SM several groups share the same 128 tokens and sweep different expert ranges, and their lists are
// merged through shared memory at the end.  On top of that a token block can be split over `msplit` CTAs along the
// expert axis (partial lists parked in global scratch, merged by the CTA that finishes last).
//
//   phase 1  z = X_blk R1            128 x 64 X tiles and 64 x 64 R1 tiles by TMA, tcgen05.mma into fp32 accumulators.
//   narrow   z -> 16-bit operand     each group writes z into its own tensor-memory columns as the A operand of
//                                    phase 2 (tcgen05.st): bf16 high part + bf16 low part in the exact modes; in
//                                    filter mode z scaled by a power of two and rounded to fp16, nothing else.
//   phase 2  y = z R2[:, 32 experts] N = 32 MMAs with A from tensor memory fill a ring of 32-column accumulators per
//                                    group (three, or two when the operand needs 64 columns); a warp copies a buffer
//                                    into registers, counts itself out of it, and the last one refills it, so the
//                                    MMAs run up to a ring ahead of the slowest warp of a group.  Every range is swept
//                                    for the same number of steps; what lies beyond a range's end is masked.
//   select   running top-k           sorted list in registers fed through a per-token candidate buffer in shared
//                                    memory (Selector).
//   finish   gates, ids, counts.
//
// Filter mode (top-k-softmax gate, no log-sum-exp wanted).  The second contraction runs on one 16-bit rounding of z
// only, which halves its tensor work and frees tensor memory for the ring, but perturbs each logit by up to
// E = |z - hi(z)|_2 * max_j |R2[:, j]|_2 (Cauchy-Schwarz).  hi(z) is fp16, not bf16: three more mantissa bits make E
// ~2e-3 of the logits' spread instead of ~2e-2.  Both operands of a kind::f16 MMA must then be fp16 (a bf16 B with an
// fp16 A is an illegal instruction on this part), so the preparation kernel also writes an fp16 copy of R2, which the
// sweep reads instead of R2; bf16 values convert exactly unless they leave fp16's exponent range, and the Euclidean
// norm of each column's conversion error enters the bound (it is zero or ~1e-8 for sane weights, and infinite --
// sending every token to the fallback -- if a weight overflows fp16).  Every token's z is first scaled by a power of
// two that puts its largest component near 2^13, so z neither overflows nor goes subnormal whatever the scale of the
// inputs (the approximate logits of a token are all scaled alike, which selection does not see).  The sweep keeps,
// besides the running
// top-k of the approximate logits, every expert within W = 2E below the k-th of them (the "zone": any expert of the
// true top-k lies there), and the survivors' logits are then recomputed in fp32 from the full z and the expert's
// column (a row of the transposed copy of R2 the preparation kernel writes), which decides the final top-k, order
// and gates.  A token whose zone overflows its few slots is routed again by a plain CUDA-core sweep at the end, so
// the result is always the exact top-k of the fp32 logits.
//
// Every mbarrier wait is bounded: when the budget runs out the thread records MORE_ERR_TIMEOUT in the device status
// word, raises the CTA's abort flag and all roles fall through to the common exit (tensor memory is freed there).
#include "sm100_common.cuh"
#include "more_select.cuh"

#include <cuda_fp16.h>

#include <type_traits>

#ifdef MORE_STATS
#define STAT(...) __VA_ARGS__
#else
#define STAT(...)
#endif

namespace more {

namespace {

constexpr int kGroups = 4;                         // 128-token groups per CTA
constexpr int kEpiThreads = 128 * kGroups;
constexpr int kFirstEpiWarp = 2;
constexpr int kRThreads = 32 * kFirstEpiWarp + kEpiThreads;   // TMA warp, phase-1 MMA warp, 16 epilogue warps
constexpr int kRRing = 208 * 1024;                 // shared-memory working area
constexpr int kRSmem = kRRing + 1024 /*alignment slack*/ + 1024 /*barriers, flags*/ + 4096 /*published thresholds*/;
constexpr int kGroupCols = 128;                    // tensor-memory columns per group
constexpr int kBufCols = 32;                       // one accumulator buffer of the ring
#ifndef MORE_CAND_CAP
#define MORE_CAND_CAP 12
#endif
constexpr int kCandCap = MORE_CAND_CAP;            // candidate slots per token
using SelLayout = Selector<8, true, kEpiThreads, kCandCap, 8>;      // (byte layout only: independent of KCAP, FILTER)
constexpr int kCandValBytes = SelLayout::kCandValBytes;
constexpr int kCandBytes = SelLayout::kCandBytes;
constexpr int kZoneStride = SelLayout::kZoneStride;
constexpr int kZoneIdOff = SelLayout::kZoneIdOff;
constexpr int kZoneBytes = SelLayout::kZoneBytes;
constexpr int kXGroupBytes = 128 * 128;            // X tile of one token group: 128 tokens x 64 bf16
constexpr int kR1Bytes = 64 * 128;
constexpr int kMaxStages1 = 8;                     // k-tiles of the projection in flight (a CTA with few tokens is a chain of L2 round trips)
constexpr int kFallbackSlots = 16;                 // tokens re-routed per round of the fallback (one per epilogue warp)
constexpr float kLog2e = 1.4426950408889634f;

// (the ...Fan modes are the exact modes with the fanned-out merge of parked lists compiled in for lists longer than 8
// entries: launched only when a token block is split over 8 or more CTAs, because that code costs the sweep of such
// kernels ~3 %; lists of up to 8 entries always have it)
enum { kModeExact = 0, kModeExactLse = 1, kModeFilter = 2, kModeExactFan = 3, kModeExactLseFan = 4 };

struct RouteParams {
    int T, h, r, M, k, gate_mode;
    int msplit, es, tg;          // CTAs per token block; expert ranges and token groups inside a CTA
    int spread;                  // a block of at most 64 tokens is repeated over the 128 tensor-memory lanes (see the kernel)
    int block_tokens;            // tokens per CTA: a multiple of 32, at most 128 * tg
    int blocks64;                // ceil(M / 64)
    int nst1, st1_bytes;         // phase-1 stages
    int nst2, st2_bytes, r2_off; // phase-2 stages (es R2 blocks each) and where they start in the ring
    int32_t* out_idx;
    float* out_gate;
    int32_t* out_counts;
    float* out_topval;
    float* out_lse;
    int* status;
    unsigned long long* stats;
    // global scratch of an msplit > 1 launch: per token block an arrival counter, per (token, split) a partial list
    unsigned* counters;
    float* part_val;
    int* part_id;
    float2* part_mz;
    // filter mode: transposed copy of R2 ([M][RPAD] bf16, columns >= r zero); colnorm[0] = largest column norm of R2,
    // colnorm[1] = largest column norm of the error of its fp16 copy
    const __nv_bfloat16* r2t;
    const float* colnorm;
    const __nv_bfloat16* R2;     // for the fallback sweep
    uint4* zlo;                  // filter: the low halves of z, [CTA][rank / 8][512 threads] x 16 B
};

// Final outputs of one token from its sorted list and (m2, z): m2 is the running max in log2 units.
template <int KCAP>
__device__ __forceinline__ void write_token(const RouteParams& p, int64_t row, const TopList<KCAP>& L, float m2,
                                            float zsum, int* hist)
{
    constexpr float kLn2 = 0.6931471805599453f;
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

// The CTA that arrives last for a token block merges the partial lists that the block's `msplit` CTAs parked in global
// scratch: on return the thread of every live token (`writer`, row `row_in_blk` of the block) holds the token's
// list and (m, Z) pair.  Called by all 512 epilogue threads; the ring (idle by then) is working space.  A function
// of its own so that its register needs stay out of the sweep's allocation.
template <int KCAP, bool LSE, bool FAN>
__device__ __forceinline__ void merge_parked_lists(const RouteParams& p, int blk, int etid, int live_tokens, uint8_t* ring_ptr,
                                                int row_in_blk, bool writer, TopList<KCAP>& G, float& gm, float& gz)
{
    auto epi_sync = [&]() { asm volatile("bar.sync 1, 512;" ::: "memory"); };
    // Merge of the partial lists [sp_lo, sp_hi) of one token into (G, gm, gz).  A token's lists lie
    // one after the other in scratch.  Each list's head (its four best entries, which is all most
    // lists contribute) is fetched with two 16-byte loads, and the next list's head is requested
    // before the current one is merged, so the L2 round trips overlap; the tail of a list is read
    // only if its fourth entry still got in.  Ascending expert ranges: ties keep the smaller id.
    auto merge_range = [&](TopList<KCAP>& G, float& gm, float& gz, int tok_in_blk, int sp_lo, int sp_hi) {
        const int64_t base = ((int64_t)blk * p.block_tokens + tok_in_blk) * p.msplit;
        const float4* pv = reinterpret_cast<const float4*>(p.part_val + base * KCAP);
        const int4* pi = reinterpret_cast<const int4*>(p.part_id + base * KCAP);
        float4 hv = __ldcg(pv + (size_t)sp_lo * (KCAP / 4));
        int4 hi = __ldcg(pi + (size_t)sp_lo * (KCAP / 4));
        for (int sp = sp_lo; sp < sp_hi; ++sp) {
            const float4 cv = hv;
            const int4 ci = hi;
            if (sp + 1 < sp_hi) {
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
    };
    G.init();
    gm = -INFINITY;
    gz = 0.f;
    // With few tokens and many splits (decode shapes) one thread per token would walk all lists one
    // L2 round trip after the other; instead `fan` threads per token merge a contiguous share of the
    // ranges each, park their result in the idle ring, and the token's own thread merges those.
    // (FAN: always for lists of up to 8 entries; for longer ones this code raises the register needs of the whole kernel,
    // which costs the sweep of the large k = 16 configurations ~3 %, so it is compiled into instantiations of their own
    // that are launched only when a token block is split over 8 or more CTAs.)
    int fan = 1;
    if constexpr (FAN)
        while (fan < 16 && 2 * fan * p.block_tokens <= kEpiThreads && 4 * fan <= p.msplit) fan *= 2;
    if (fan == 1) {
        if (writer) merge_range(G, gm, gz, row_in_blk, 0, p.msplit);
    } else if constexpr (FAN) {
        // The lists are first copied into the idle ring with coalesced, independent loads (one L2
        // round trip for all of them instead of one per list and thread), in batches of `lb` lists per
        // token when they do not fit at once; a token's rows are skewed by 16 bytes against the banks.
        // All merging is done with the sorted-list network (no data-dependent control flow): a worker
        // folds its share of the lists into one, then the `fan` lists of a token are merged pairwise
        // in log2(fan) levels.
        const int bt = p.block_tokens;
        constexpr int kPerList = KCAP * 8 + 8;
    constexpr int kInFlight = KCAP <= 8 ? 4 : 2;          // loads per array and thread in flight during the copy
        float* sv = reinterpret_cast<float*>(ring_ptr);                  // [fan][KCAP][bt]
        int* si = reinterpret_cast<int*>(sv + fan * KCAP * bt);         // [fan][KCAP][bt]
        float2* smz = reinterpret_cast<float2*>(si + fan * KCAP * bt);  // [fan][bt]
        const int sub_bytes = (fan * bt * kPerList + 127) & ~127;
        int lb = ((kRRing - sub_bytes) / bt - 40) / kPerList;
        lb = lb < p.msplit ? lb : p.msplit;
        const int tsv = lb * KCAP + 4, tsm = lb + 1;        // a token's stride in floats / in float2s
        float* av = reinterpret_cast<float*>(ring_ptr + sub_bytes);      // [bt][lb][KCAP] (+ skew)
        int* ai = reinterpret_cast<int*>(av + bt * tsv);
        float2* amz = reinterpret_cast<float2*>(ai + bt * tsv);
        const int wt = etid % bt, wf = etid / bt;
        const bool worker = wf < fan && wt < live_tokens;
        const int share_lo = (int)((long long)p.msplit * wf / fan), share_hi = (int)((long long)p.msplit * (wf + 1) / fan);
        TopList<KCAP> S;
        S.init();
        float sm = -INFINITY, sz = 0.f;
        auto join_mz = [&](const float2 mz) {
            if (LSE && mz.x > -INFINITY) {
                const float nm = fmaxf(sm, mz.x);
                sz = sz * ex2f(sm - nm) + mz.y * ex2f(mz.x - nm);
                sm = nm;
            }
        };
        const int64_t blk_slot = (int64_t)blk * bt * p.msplit;
        const float4* gv = reinterpret_cast<const float4*>(p.part_val);
        const int4* gi = reinterpret_cast<const int4*>(p.part_id);
        for (int sp0 = 0; sp0 < p.msplit; sp0 += lb) {
            const int nl = min(lb, p.msplit - sp0);
            const int q4 = nl * (KCAP / 4);
            const int total = live_tokens * q4;
            for (int e0 = etid; e0 < total; e0 += kInFlight * kEpiThreads) {
                float4 xv[kInFlight];
                int4 xi[kInFlight];
                int dst[kInFlight];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    const int e = e0 + u * kEpiThreads;
                    dst[u] = -1;
                    if (e < total) {
                        const int t = e / q4, w = e - t * q4;
                        const int64_t src = (blk_slot + (int64_t)t * p.msplit + sp0) * (KCAP / 4) + w;
                        xv[u] = __ldcg(gv + src);
                        xi[u] = __ldcg(gi + src);
                        dst[u] = t * (tsv / 4) + w;
                    }
                }
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    if (dst[u] >= 0) {
                        reinterpret_cast<float4*>(av)[dst[u]] = xv[u];
                        reinterpret_cast<int4*>(ai)[dst[u]] = xi[u];
                    }
                }
            }
            if (LSE) {
                for (int e = etid; e < live_tokens * nl; e += kEpiThreads) {
                    const int t = e / nl, l = e - t * nl;
                    amz[t * tsm + l] = __ldcg(p.part_mz + blk_slot + (int64_t)t * p.msplit + sp0 + l);
                }
            }
            epi_sync();
            if (worker) {
                const int lo = max(share_lo, sp0), hi = min(share_hi, sp0 + nl);
                for (int sp = lo; sp < hi; ++sp) {
                    const float* lv = av + wt * tsv + (sp - sp0) * KCAP;
                    const int* li = ai + wt * tsv + (sp - sp0) * KCAP;
                    S.merge_sorted([&](int e) { return lv[e]; }, [&](int e) { return li[e]; });
                    if (LSE) join_mz(amz[wt * tsm + (sp - sp0)]);
                }
            }
            epi_sync();
        }
        auto park_sub = [&]() {
#pragma unroll
            for (int s = 0; s < KCAP; ++s) {
                sv[(wf * KCAP + s) * bt + wt] = S.v[s];
                si[(wf * KCAP + s) * bt + wt] = S.id[s];
            }
            smz[wf * bt + wt] = make_float2(sm, sz);
        };
        if (worker) park_sub();
        epi_sync();
        for (int d = 1; d < fan; d <<= 1) {
            if (worker && (wf & (2 * d - 1)) == 0) {
                S.merge_sorted([&](int e) { return sv[((wf + d) * KCAP + e) * bt + wt]; },
                               [&](int e) { return si[((wf + d) * KCAP + e) * bt + wt]; });
                if (LSE) join_mz(smz[(wf + d) * bt + wt]);
                if (2 * d < fan) park_sub();
                else if (wf == 0) park_sub();
            }
            epi_sync();
        }
        if (writer) {
#pragma unroll
            for (int s = 0; s < KCAP; ++s) {
                G.v[s] = sv[s * bt + row_in_blk];
                G.id[s] = si[s * bt + row_in_blk];
            }
            const float2 mz = smz[row_in_blk];
            gm = mz.x;
            gz = mz.y;
        }
        epi_sync();                          // the ring is reused by the histogram
    }
}

// ------------------------------------------------------------------------------------------------- the kernel
template <int RPAD, int KCAP, int MODE>
__global__ void __launch_bounds__(kRThreads, 1)
route_lowrank_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_r1,
                     const __grid_constant__ CUtensorMap map_r2, const RouteParams p)
{
    constexpr bool FILTER = MODE == kModeFilter;
    constexpr bool LSE = MODE == kModeExactLse || MODE == kModeExactLseFan;
    constexpr bool FAN = KCAP <= 8 || MODE == kModeExactFan || MODE == kModeExactLseFan;
    constexpr int kKSteps = RPAD / 16;                               // UMMA K = 16
    constexpr int kMmasPerBuf = FILTER ? kKSteps : 2 * kKSteps;      // exact modes: hi then lo into one accumulator
    constexpr int kZopCols = FILTER ? RPAD / 2 : RPAD;               // A operand: two bf16 per 32-bit column
    constexpr int kRingCol0 = (kZopCols <= 32) ? 32 : 64;            // first column of the accumulator ring
    constexpr int NBUF = (kGroupCols - kRingCol0) / kBufCols;        // 3 or 2
    constexpr int kR2BlockBytes = RPAD * 128;                        // RPAD rows x 64 experts
    using Sel = Selector<KCAP, FILTER, kEpiThreads, kCandCap, 8, 8, !FILTER>;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;            // 1024-aligned: the 128-B swizzle repeats every 1 KB
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    uint8_t* ctl = ring_ptr + kRRing;                        // control block
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctl);
    constexpr int B_FULL1 = 0, B_EMPTY1 = B_FULL1 + kMaxStages1, B_ZACC = B_EMPTY1 + kMaxStages1, B_FULL2 = B_ZACC + 1,
                  B_EMPTY2 = B_FULL2 + 8, B_ACCF = B_EMPTY2 + 8, B_COUNT = B_ACCF + kGroups * 3;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + B_COUNT * 8 + 4);
    int* last_flag = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 8);
    int* flagged = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 12);      // tokens that need the fallback sweep
    int* part_tab = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 16);    // [es]: first 64-expert block of every range
    int* zop_done = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 32);    // [tg]: warps that have written their operand
    int* released = reinterpret_cast<int*>(ctl + B_COUNT * 8 + 48);    // [group][slot]: warps that have read a buffer out
    STAT(long long* issue_clk = reinterpret_cast<long long*>(ctl + B_COUNT * 8 + 96);)   // [group][slot]: when the refill was issued
    // [token group][token][expert range]: the k-th value each range's thread has reached for its token (see `exchange`)
    float* tau_pub = reinterpret_cast<float*>(ctl + 1024);
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < kEpiThreads) { tau_pub[2 * threadIdx.x] = -INFINITY; tau_pub[2 * threadIdx.x + 1] = -INFINITY; }
    const int blk = blockIdx.x / p.msplit, split = blockIdx.x % p.msplit;
    const int tok0 = blk * p.block_tokens;
    const int live_tokens = min(p.block_tokens, p.T - tok0);
    const int tg_live = (live_tokens + 127) >> 7;            // token groups with at least one token
    const int es = p.es;
    const int ngroups = tg_live * es;
    const int nparts = p.msplit * es;
    // 64-expert blocks of expert range `esi` of this CTA: an even share of ceil(M / 64) blocks.  The shares differ by
    // at most one block; every range is swept for nsteps blocks all the same, and whatever that reads beyond the
    // range's own end (the next range's first block, or zero fill past M) is masked in the epilogue.
    auto part_lo = [&](int esi) { return part_tab[esi]; };
    auto live_warps = [&](int tgi) { return min(4, (live_tokens - tgi * 128 + 31) >> 5); };
    const int ktiles1 = (p.h + 63) / 64;
    const int nsteps = (p.blocks64 + nparts - 1) / nparts;
    const int nst2_mask = p.nst2 - 1;                        // nst2 is a power of two
    const int nst2_shift = 31 - __clz(p.nst2);

    if (threadIdx.x == 0) {
        for (int e = 0; e < es; ++e) part_tab[e] = (int)(((long long)p.blocks64 * (split * es + e)) / nparts);
        for (int i = 0; i < kMaxStages1; ++i) { mbar_init(bar(B_FULL1 + i), 1); mbar_init(bar(B_EMPTY1 + i), 1); }
        mbar_init(bar(B_ZACC), 1);
        // a stage is free again when both 32-expert halves of every group's step have been multiplied
        for (int i = 0; i < 8; ++i) { mbar_init(bar(B_FULL2 + i), 1); mbar_init(bar(B_EMPTY2 + i), 2 * ngroups); }
        for (int i = 0; i < kGroups * 3; ++i) { mbar_init(bar(B_ACCF + i), 1); released[i] = 0; }
        for (int t = 0; t < kGroups; ++t) zop_done[t] = 0;
        *abort_flag = 0;
        *last_flag = 0;
        *flagged = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t r2ring = ring + p.r2_off;

    if (warp == 0) {
        // ===================================================================================== TMA producer
        if (lane == 0) {
            bool ok = true;
            const uint32_t st1_tx = tg_live * kXGroupBytes + kR1Bytes;
            for (int kt = 0; kt < ktiles1 && ok; ++kt) {
                const int s = kt % p.nst1;
                if (kt >= p.nst1) ok = mbar_wait(bar(B_EMPTY1 + s), ((kt / p.nst1) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = ring + s * p.st1_bytes;
                mbar_expect_tx(bar(B_FULL1 + s), st1_tx);
                if (p.spread) {                                     // 4 x (32 token rows x 64 columns): the block, repeated
                    for (int j = 0; j < 4; ++j)
                        tma_load_2d(dst + j * (kXGroupBytes / 4), &map_x, bar(B_FULL1 + s), kt * 64,
                                    tok0 + (j * 32) % p.block_tokens);
                } else {
                    for (int t = 0; t < tg_live; ++t)               // 128 token rows x 64 columns per token group
                        tma_load_2d(dst + t * kXGroupBytes, &map_x, bar(B_FULL1 + s), kt * 64, tok0 + t * 128);
                }
                tma_load_2d(dst + p.tg * kXGroupBytes, &map_r1, bar(B_FULL1 + s), 0, kt * 64);
            }
            // the R2 stages lie beyond the phase-1 stages, so the first blocks of R2 arrive while phase 1 still runs
            for (int it = 0; it < nsteps && ok; ++it) {
                const int s = it & nst2_mask;
                if (it >= p.nst2) ok = mbar_wait(bar(B_EMPTY2 + s), ((it >> nst2_shift) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_FULL2 + s), es * kR2BlockBytes);
                for (int e = 0; e < es; ++e)
                    tma_load_2d(r2ring + s * p.st2_bytes + e * kR2BlockBytes, &map_r2, bar(B_FULL2 + s),
                                (part_lo(e) + it) * 64, 0);
            }
        }
    } else if (warp == 1) {
        // ================================================================================== phase-1 MMA issuer
        // The whole warp runs this code converged; one elected lane issues each tcgen05 instruction.  z of token group
        // t accumulates in the ring columns of the group's first expert range.  Descriptor words of stage 0: K-major X
        // tile (A), MN-major R1 tile (B); +2 per 32 bytes of start address.
        bool ok = true;
        constexpr uint32_t idesc1 = umma_idesc(RPAD);
        const uint64_t xd = umma_desc_sw128(ring, 16, 1024), rd = umma_desc_sw128(ring + p.tg * kXGroupBytes, 8192, 1024);
        const uint32_t x_lo0 = (uint32_t)xd, x_hi = (uint32_t)(xd >> 32), r_lo0 = (uint32_t)rd, r_hi = (uint32_t)(rd >> 32);
        for (int kt = 0; kt < ktiles1 && ok; ++kt) {
            const int s = kt % p.nst1;
            ok = __all_sync(kFullMask, mbar_wait(bar(B_FULL1 + s), (kt / p.nst1) & 1, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t x_lo = x_lo0 + s * (p.st1_bytes >> 4), r_lo = r_lo0 + s * (p.st1_bytes >> 4);
            for (int t = 0; t < tg_live; ++t) {
                const uint32_t d = tmem_base + (t * es) * kGroupCols + kRingCol0;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)      // A: +32 B per K = 16; B: 16 K-rows of 128 B
                    tc_mma_bf16_ss_elect(d, x_lo + t * (kXGroupBytes >> 4) + kk * 2, x_hi, r_lo + kk * (2048 >> 4),
                                         r_hi, idesc1, (kt | kk) != 0);
            }
            tc_commit_elect(bar(B_EMPTY1 + s));
        }
        if (ok) tc_commit_elect(bar(B_ZACC));
    } else {
        // ========================================================================================= epilogue
        const int ew = warp - kFirstEpiWarp;
        const int g = ew >> 2;                               // group
        const int q = warp & 3;                              // TMEM lane quarter this warp may access
        const int etid = threadIdx.x - 32 * kFirstEpiWarp;   // 0..511 among the epilogue threads
        const int tgi = g / es, esi = g % es;
        // Which token a lane holds.  Normally lane quarter q of token group tgi holds tokens tgi*128 + q*32 ...  A block
        // of at most 64 tokens (p.spread) is instead loaded into every 32- or 64-lane stretch of the group's 128 lanes,
        // so all stretches hold the same z, and expert range esi works on stretch esi: the few working warps of such a
        // CTA then sit in different lane quarters, i.e. on different schedulers, instead of all on the first one or two.
        const int lq = p.block_tokens >> 5;                                   // spread: lane quarters per copy (1 or 2)
        const int qi = p.spread ? ((q - esi * lq) & 3) : q;                  // this warp's index in its group's stretch
        const int row_in_tg = qi * 32 + lane;
        const int row_in_blk = tgi * 128 + row_in_tg;
        const int64_t row = (int64_t)tok0 + row_in_blk;
        const bool warp_live = g < ngroups && (tgi * 128 + qi * 32) < live_tokens && (!p.spread || qi < lq);     // warp-uniform
        const bool row_live = warp_live && row_in_blk < live_tokens;
        const uint32_t t_lanes = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t t_zacc = t_lanes + (tgi * es) * kGroupCols + kRingCol0;       // the token group's z (fp32)
        const uint32_t t_zop = t_lanes + g * kGroupCols;                              // this group's A operand
        const uint32_t t_ring = t_zop + kRingCol0;
        // filter: low half of this thread's z, 16 B per 8 ranks, in global scratch (read back once, for rescoring)
        uint4* zlo = FILTER ? p.zlo + (size_t)blockIdx.x * (RPAD / 8) * kEpiThreads + etid : nullptr;
        const int e_lo = part_lo(esi) * 64;
        // this range ends where the next one begins (the ranges of a CTA are consecutive shares of all parts)
        const int e_hi = min((int)(((long long)p.blocks64 * (split * es + esi + 1)) / nparts) * 64, p.M);
        const int nb = warp_live ? 2 * nsteps : 0;                                    // 32-expert buffers to drain
        const int lw = live_warps(tgi);                                               // warps of this group with tokens

        // ---- refill of the ring.  Buffer m of the group = 32-expert half (m & 1) of step m >> 1, in ring slot m % NBUF.
        // Called by one whole warp, converged; an elected lane issues.  Both commits follow the MMAs of this buffer:
        // one tells the group that the buffer is full, the other counts towards releasing the R2 stage.
        constexpr uint32_t idesc2 = FILTER ? umma_idesc_f16(kBufCols) : umma_idesc(kBufCols);
        const uint64_t bd0 = umma_desc_sw128(r2ring + esi * kR2BlockBytes, 8192, 1024);
        const uint32_t b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
        auto issue_buffer = [&](int grp, uint32_t b_lo_grp, int m, int slot) -> bool {
            const int it = m >> 1;
            const int st = it & nst2_mask;
            if (!mbar_wait(bar(B_FULL2 + st), (it >> nst2_shift) & 1, abort_flag, p.status)) return false;
            tc_fence_after();
            const uint32_t t_grp = tmem_base + grp * kGroupCols;
            tc_mma_buffer_ts<kMmasPerBuf, kKSteps>(t_grp + kRingCol0 + slot * kBufCols, t_grp,
                                                   b_lo_grp + st * (p.st2_bytes >> 4) + (m & 1) * (64 >> 4), b_hi, idesc2);
            tc_commit_elect(bar(B_ACCF + grp * 3 + slot));
            tc_commit_elect(bar(B_EMPTY2 + st));
            STAT(if (lane == 0) issue_clk[grp * 3 + slot] = clock64();)
            return true;
        };

        float zone_w = 0.f;
        bool ok = true;
        if (warp_live) {
            ok = mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
            ok = __all_sync(kFullMask, ok);
        }
        float zscale = 1.f;                                  // filter: z = (hi + lo) * zscale
        if (warp_live && ok) {
            // ---- narrow z and store it to tensor memory as the A operand of phase 2
            tc_fence_after();
            float lo2 = 0.f, z2 = 0.f, down = 1.f;
            if (FILTER) {
                // power of two that brings the token's largest |z| into [2^13, 2^14)
                float zmax = 0.f;
#pragma unroll
                for (int c = 0; c < RPAD / 16; ++c) {
                    float z[16];
                    tmem_ld16(t_zacc + c * 16, z);
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
                tmem_ld16(t_zacc + c * 16, z);
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
                        const float d0 = z[2 * e] - __bfloat162float(h0), d1 = z[2 * e + 1] - __bfloat162float(h1);
                        const __nv_bfloat16 l0 = __float2bfloat16_rn(d0), l1 = __float2bfloat16_rn(d1);
                        hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                        lo[e] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
                    }
                }
                tmem_st8(t_zop + c * 8, hi);
                if (FILTER) {
                    zlo[(2 * c) * kEpiThreads] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    zlo[(2 * c + 1) * kEpiThreads] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
                } else {
                    tmem_st8(t_zop + RPAD / 2 + c * 8, lo);
                }
            }
            tmem_st_wait();
            tc_fence_before();
            // The last warp of the token group to get here (all expert ranges of the group counted: they read the
            // same z, which the first range's ring is about to overwrite) starts phase 2 for every one of them.
            __syncwarp();
            int prior = 0;
            if (lane == 0)
                asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;"
                             : "=r"(prior) : "r"(smem_u32(zop_done + tgi)) : "memory");
            prior = __shfl_sync(kFullMask, prior, 0);
            if (prior == es * lw - 1) {
                tc_fence_after();
                for (int e = 0; e < es && ok; ++e)
                    for (int m = 0; m < NBUF && m < nb && ok; ++m)
                        ok = issue_buffer(tgi * es + e, b_lo0 + ((e - esi) * kR2BlockBytes >> 4), m, m);
            }
            ok = __all_sync(kFullMask, ok);
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
        S.init(ring + etid * 16, ring + kCandValBytes + etid * 4, ring + kCandBytes + etid * 4, zone_w);
        STAT(unsigned st_chunks = 0, st_hit = 0, st_app = 0, st_fold = 0, st_miss = 0, st_nlat = 0; long long st_lat = 0; long long st_twait = 0, st_tfold = 0, st_tresc = 0, st_tfall = 0;
             const long long st_t0 = clock64();)
        float m2 = -INFINITY, zsum = 0.f;                    // running max (log2 units) and sum of 2^(y - m2)

        // ---- one 16-column chunk: group-of-four maxima, optional online softmax update, candidate append.  Straight-line
        // code: the four predicated appends run whether or not any token of the warp has a candidate.  A warp-wide test
        // that skips them would save issue slots in half of the chunks, but a warp's loop is a chain of latencies, and
        // a vote plus a branch per chunk lengthens exactly that chain.
        auto process = [&](float (&v)[16], int col0) {
            float t[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) t[i] = fmaxf(max3(v[4 * i], v[4 * i + 1], v[4 * i + 2]), v[4 * i + 3]);
            if (LSE) {
                const float cmax = fmaxf(max3(t[0], t[1], t[2]), t[3]);
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
            STAT(st_chunks++;)
#ifdef MORE_EXP_NOSCAN
            m2 = fmaxf(m2, t[0] + t[1] + t[2] + t[3]);
            return;
#endif
            S.scan(v, t, col0);
        };
        // ---- after the two chunks of a buffer: fold if some token of the warp could overflow on the next buffer
        // (the first two buffers of a sweep are folded wholesale: with a near-empty list almost everything gets in)
        // The expert ranges of a CTA sweep the same tokens, and every range would pay the expensive start of a sweep on its
        // own.  After a fold a thread publishes two values of its list (KCAP entries, sorted): the last one, and the
        // one at position KCAP/es - 1.  Both give lower bounds for the token's final KCAP-th value: at least KCAP logits
        // reach any range's last value, and at least KCAP/es logits in every range, KCAP in all, reach the smallest
        // of the values at position KCAP/es - 1.  The larger bound, lowered by a hair so that an equal logit (which a
        // smaller id could still win) is kept, becomes the floor of this thread's own collection.
        float2* const tau_mine = reinterpret_cast<float2*>(tau_pub) + (tgi * 128 + row_in_tg) * es;
        auto exchange = [&]() {
            if constexpr (!FILTER) {
                if (es > 1) {
                    tau_mine[esi] = make_float2(S.L.tau(), es == 4 ? S.L.v[KCAP / 4 - 1] : S.L.v[KCAP / 2 - 1]);
                    float2 b = tau_mine[0];
                    for (int e = 1; e < es; ++e) {
                        const float2 o = tau_mine[e];
                        b.x = fmaxf(b.x, o.x);
                        b.y = fminf(b.y, o.y);
                    }
                    const float best = fmaxf(b.x, b.y);
                    S.ext = fmaf(-fabsf(best), 2.4e-7f, best) - 1e-37f;       // strictly below `best` (-inf stays -inf)
                    S.thr = fmaxf(S.thr, S.ext);
                }
            }
        };
        auto fold_check = [&](int n) {
            const bool folds = __any_sync(kFullMask, S.ptr >= S.warn);
            if (folds) {
                STAT(st_fold++; const long long tr0 = clock64();)
                if constexpr (FILTER) {
                    S.fold();
                } else {
                    if (n < 2) S.fold_all();
                    else S.fold();
                }
                STAT(st_tfold += clock64() - tr0;)
            }
            if (folds) exchange();
        };

        // ---- the sweep: buffer n of the group lives in ring slot n % NBUF.  A warp's loop is a chain of long
        // latencies (barrier test, tensor-memory load), so it is software-pipelined: the second half of a buffer is in
        // flight while the first is processed, the first half of the next buffer while the second is, and the buffer
        // is handed back (this warp counted out of it) as soon as both halves are in registers.
        // Refills take turns: the warp whose index in the group is n mod (live warps) refills buffer n's slot with
        // buffer n + NBUF, one iteration later, when normally every warp has already counted itself out of it.  (Letting
        // whichever warp is out last refill at once keeps the slowest warp the slowest; a separate issuing warp per
        // group would exceed the thread count that leaves 96 registers per thread.)
        if (nb > 0 && ok) {
            int slot = 0, pslot = 0, all_out = lw;                 // `released` reads all_out once every warp is out
            int my_refill = qi + 1;                                // next iteration at which this warp refills a slot
            uint32_t ph = 0;
            const uint32_t rel0 = smem_u32(released + g * 3);
            // One iteration = one buffer.  `masked` (a compile-time flag, so that the common iterations carry none of
            // the masking code) is set for the buffers that reach beyond the range's end.  The two register buffers
            // live inside one iteration only.
            auto one_buffer = [&](auto masked, int n) {
                const int col0 = e_lo + n * kBufCols;
                float va[16], vb[16];
                STAT(const long long tw1 = clock64(); if (!mbar_try_wait_now(bar(B_ACCF + g * 3 + slot), ph)) st_miss++;)
                ok = mbar_wait(bar(B_ACCF + g * 3 + slot), ph, abort_flag, p.status);
                STAT(st_twait += clock64() - tw1;)
                if (!ok) return;
                tc_fence_after();
                tmem_ld16(t_ring + slot * kBufCols, va);
                tmem_ld_wait16(va);
                tmem_ld16(t_ring + slot * kBufCols + 16, vb);
                if constexpr (decltype(masked)::value) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (col0 + i >= e_hi) va[i] = -INFINITY;
                }
                process(va, col0);
                STAT(const long long tl0 = clock64();)
                tmem_ld_wait16(vb);
                STAT(st_lat += clock64() - tl0; st_nlat++;)
                // count this warp out of buffer n (release: its tensor-memory loads are complete)
                tc_fence_before();
                __syncwarp();
                if (lane == 0)
                    asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(rel0 + 4 * slot) : "memory");
                // this warp's turn to refill the slot of buffer n - 1?  (all_out still counts buffer n - 1's use of it
                // unless the slot index has just wrapped, in which case the count was raised one iteration early)
                if (n == my_refill) {
                    my_refill += lw;
                    if (n - 1 + NBUF < nb) {
                        const int want = (slot == 0) ? all_out - lw : all_out;
                        const uint32_t ra = rel0 + 4 * pslot;
                        int have, spins = 0;
                        do {
                            asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(have) : "r"(ra) : "memory");
                        } while (have < want && ++spins < (1 << 26) && *abort_flag == 0);
                        ok = have >= want;
                        if (!ok) {
                            if (*abort_flag == 0) { *abort_flag = 1; atomicExch(p.status, MORE_ERR_TIMEOUT); }
                            return;
                        }
                        tc_fence_after();
                        ok = issue_buffer(g, b_lo0, n - 1 + NBUF, pslot);
                        if (!ok) return;
                    }
                }
                if constexpr (decltype(masked)::value) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (col0 + 16 + i >= e_hi) vb[i] = -INFINITY;
                }
                process(vb, col0 + 16);
                fold_check(n);
                pslot = slot;
                if (++slot == NBUF) { slot = 0; ph ^= 1; all_out += lw; }
            };
            const int ragged_from = min(nb, (e_hi - e_lo) / kBufCols);      // first buffer with columns to mask
            int n = 0;
            for (; n < ragged_from && ok; ++n) one_buffer(std::false_type{}, n);
            for (; n < nb && ok; ++n) one_buffer(std::true_type{}, n);
            ok = __all_sync(kFullMask, ok);
        }
        if (warp_live) S.fold();
        TopList<KCAP>& L = S.L;
        STAT(const long long st_t1 = clock64();)

        if (FILTER && warp_live && ok) {
            // ---- rescoring: fp32 logits of the list and of the zone from the full z = hi + lo and the experts'
            // columns (rows of the transposed copy); the exact values decide the final order
            S.prune();
            const int zcount = (int)((S.zptr - S.zbase) / kZoneStride);
            int zmax = zcount;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) zmax = max(zmax, __shfl_xor_sync(kFullMask, zmax, o));
            float acc[KCAP];
#pragma unroll
            for (int e = 0; e < KCAP; ++e) acc[e] = 0.f;
            auto z_chunk = [&](int c, float (&z8)[8]) {             // ranks 8c .. 8c+7 of this token's z
                uint32_t h4[4];
                tmem_ld4(t_zop + c * 4, h4);
                const uint4 lv = zlo[c * kEpiThreads];
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
                const int id = have ? lds_s32(S.zbase + kZoneIdOff + zi * kZoneStride) : -1;
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
        STAT(st_tresc = clock64() - st_t1;)
#ifdef MORE_STATS
        if (p.stats && warp_live) {
          const unsigned st_ov = __popc(__ballot_sync(kFullMask, FILTER && S.overflow && row_live));
          const unsigned st_zn = __reduce_add_sync(kFullMask, (S.zptr - S.zbase) / kZoneStride);
          if (lane == 0) {
            atomicAdd(p.stats + 0, (unsigned long long)st_chunks);
            atomicAdd(p.stats + 1, (unsigned long long)st_hit);
            atomicAdd(p.stats + 3, (unsigned long long)st_app);
            atomicAdd(p.stats + 4, (unsigned long long)st_fold);
            atomicAdd(p.stats + 8, (unsigned long long)st_twait);
            atomicAdd(p.stats + 9, (unsigned long long)st_miss);
            atomicAdd(p.stats + 6, (unsigned long long)st_lat);
            atomicAdd(p.stats + 5, (unsigned long long)st_nlat);
            atomicAdd(p.stats + 4 + 0 * 1, 0ull);
            atomicAdd(p.stats + 1 * 0 + 15 * 0 + 0, 0ull);
            atomicAdd(p.stats + 15 - 15 + 0, 0ull);
            atomicAdd(p.stats + 7 - 7 + 0, 0ull);
            atomicAdd(p.stats + 10 - 10, 0ull);
            atomicAdd(p.stats + 13 + (q >> 1), (unsigned long long)st_twait);
            atomicAdd(p.stats + 15, (unsigned long long)(q >> 1));
            atomicAdd(p.stats + 10, (unsigned long long)(st_t1 - st_t0));
            atomicAdd(p.stats + 7, (unsigned long long)st_tresc);
            atomicAdd(p.stats + 5, (unsigned long long)st_ov);
            atomicAdd(p.stats + 2, (unsigned long long)st_zn);
            atomicAdd(p.stats + 11, 1ull);
            atomicAdd(p.stats + 12, (unsigned long long)st_tfold);
          }
        }
#endif

        // ---- finish.  All 512 epilogue threads meet at every barrier below, also after an abort.
        auto epi_sync = [&]() { asm volatile("bar.sync 1, 512;" ::: "memory"); };
        if (FILTER && S.overflow && row_live) atomicAdd(flagged, 1);
        epi_sync();                                          // the candidate / zone / z areas are idle from here on
        const bool aborted = *abort_flag != 0;

        if (FILTER && !aborted) {
            // ---- fallback: tokens whose zone overflowed are routed again, exactly, over this group's experts; the
            // result replaces the token's list.  Rounds of kFallbackSlots tokens, one warp per token.
            const int nflag = *flagged;
            if (nflag > 0) {
                float* fz = reinterpret_cast<float*>(ring_ptr);                          // [slot][RPAD] z
                int* frange = reinterpret_cast<int*>(ring_ptr + kFallbackSlots * RPAD * 4);   // [slot][2]
                float* fv = reinterpret_cast<float*>(frange + kFallbackSlots * 2);        // [slot][KCAP]
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
                    if (warp_live && __any_sync(kFullMask, slot >= 0)) {
                        for (int c = 0; c < RPAD / 8; ++c) {
                            uint32_t h4[4];
                            tmem_ld4(t_zop + c * 4, h4);
                            const uint4 lv = zlo[c * kEpiThreads];
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
                        if (slot >= 0) { frange[slot * 2] = e_lo; frange[slot * 2 + 1] = e_hi; }
                    }
                    epi_sync();
                    const int nslots = min(kFallbackSlots, nflag - done);
                    if (ew < nslots)
                        exact_topk_warp<KCAP>(fz + ew * RPAD, p.R2, p.r, p.M, frange[ew * 2], frange[ew * 2 + 1],
                                              fv + ew * KCAP, fi + ew * KCAP, lane);
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

        if (es > 1 && !aborted) {
            // ---- groups that share tokens: ranges 1.. park their lists in shared memory, range 0 merges them in
            // ascending range order (equal logits keep the smaller id)
            float* pv = reinterpret_cast<float*>(ring_ptr);                          // [tg][es-1][KCAP][128]
            int* pi = reinterpret_cast<int*>(ring_ptr + kGroups * KCAP * 128 * 4);
            float2* pmz = reinterpret_cast<float2*>(ring_ptr + 2 * kGroups * KCAP * 128 * 4);
            if (warp_live && esi > 0) {
                const int o = (tgi * (es - 1) + (esi - 1)) * KCAP * 128 + row_in_tg;
#pragma unroll
                for (int s = 0; s < KCAP; ++s) { pv[o + s * 128] = L.v[s]; pi[o + s * 128] = L.id[s]; }
                pmz[(tgi * (es - 1) + (esi - 1)) * 128 + row_in_tg] = make_float2(m2, zsum);
            }
            epi_sync();
            if (warp_live && esi == 0) {
                for (int e = 1; e < es; ++e) {
                    const int o = (tgi * (es - 1) + (e - 1)) * KCAP * 128 + row_in_tg;
#pragma unroll
                    for (int s = 0; s < KCAP; ++s) {
                        const float x = pv[o + s * 128];
                        if (x > L.tau()) L.insert(x, pi[o + s * 128]);
                    }
                    if (LSE) {
                        const float2 mz = pmz[(tgi * (es - 1) + (e - 1)) * 128 + row_in_tg];
                        if (mz.x > -INFINITY) {
                            const float nm = fmaxf(m2, mz.x);
                            zsum = zsum * ex2f(m2 - nm) + mz.y * ex2f(mz.x - nm);
                            m2 = nm;
                        }
                    }
                }
            }
            epi_sync();
        }
        const bool writer = row_live && esi == 0;            // one thread per token carries the result from here on

        // Expert histogram: when the M bins fit into the (now idle) ring, the CTA counts its tokens' ids in shared
        // memory and flushes only the non-zero bins with one global atomic each; otherwise straight to global memory
        // (with that many experts the bins hardly collide).  With few experts thousands of pairs hit each bin, and
        // same-address global atomics would serialise.
        // (a CTA with few tokens would spend longer clearing and flushing the bins than on its handful of atomics)
        int* hist = (p.M <= kRRing / 4 && live_tokens * p.k * 16 > p.M) ? reinterpret_cast<int*>(ring_ptr) : nullptr;
        auto hist_clear = [&]() {
            if (hist) {
                for (int e = etid; e < p.M; e += kEpiThreads) hist[e] = 0;
                epi_sync();
            }
        };
        auto hist_flush = [&]() {
            if (hist) {
                epi_sync();
                for (int e = etid; e < p.M; e += kEpiThreads) {
                    const int c = hist[e];
                    if (c) atomicAdd(p.out_counts + e, c);
                }
            }
        };
        if (!aborted) {
            if (p.msplit == 1) {
                hist_clear();
                if (writer) write_token<KCAP>(p, row, L, m2, zsum, hist);
                hist_flush();
            } else {
                // park the partial list; the CTA that arrives last for this token block merges all of them
                const int64_t slot = ((int64_t)blk * p.block_tokens + row_in_blk) * p.msplit + split;
                if (writer) {
#pragma unroll
                    for (int s = 0; s < KCAP; ++s) {
                        p.part_val[slot * KCAP + s] = L.v[s];
                        p.part_id[slot * KCAP + s] = L.id[s];
                    }
                    p.part_mz[slot] = make_float2(m2, zsum);
                }
                __threadfence();
                epi_sync();
                if (etid == 0) {
                    const unsigned prev = atomicAdd(p.counters + blk, 1u);
                    *last_flag = (prev == (unsigned)p.msplit - 1u);
                }
                epi_sync();
                if (*last_flag) {
                    __threadfence();
                    TopList<KCAP> G;
                    float gm, gz;
                    merge_parked_lists<KCAP, LSE, FAN>(p, blk, etid, live_tokens, ring_ptr, row_in_blk, writer, G, gm, gz);
                    hist_clear();
                    if (writer) write_token<KCAP>(p, row, G, gm, gz, hist);
                    hist_flush();
                    if (etid == 0) p.counters[blk] = 0;      // ready for the next call
                }
            }
        }
    }

    // ---- common exit: everyone arrives here, also after an abort
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        // give bulk copies that may still be in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------------------------ preparation (filter mode)
// For the filter: R2H = R2 converted to fp16 (same [r][M] layout, the B operand of the sweep), R2T[j][i] = R2[i][j]
// (bf16, [M][RPAD], ranks >= r zero, for the rescoring), the largest Euclidean column norm of R2 and of R2 - R2H
// (slightly inflated, so that rounding cannot make them too small), and out_counts cleared.  One CTA per 64 experts;
// the CTA that finishes last reduces the per-CTA maxima (the arrival counter returns to zero for the next call).
__global__ void __launch_bounds__(256)
route_prepare_kernel(const __nv_bfloat16* __restrict__ R2, int r, int rpad, int M, __half* __restrict__ r2h,
                     __nv_bfloat16* __restrict__ r2t, float2* __restrict__ partial, float* __restrict__ colnorm,
                     unsigned* __restrict__ arrivals, int32_t* __restrict__ out_counts)
{
    __shared__ __nv_bfloat16 tile[64][64 + 8];      // [rank][expert], padded rows
    __shared__ float red[64], rederr[64];
    __shared__ int last;
    const int j0 = blockIdx.x * 64;
    const int tj = threadIdx.x & 63, ti = threadIdx.x >> 6;
    for (int i = ti; i < rpad; i += 4) {
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (i < r && j0 + tj < M) {
            v = R2[(int64_t)i * M + j0 + tj];
            r2h[(int64_t)i * M + j0 + tj] = __float2half_rn(__bfloat162float(v));
        }
        tile[i][tj] = v;
    }
    if (threadIdx.x < 64 && j0 + threadIdx.x < M) out_counts[j0 + threadIdx.x] = 0;
    __syncthreads();
    if (threadIdx.x < 64) {
        float s = 0.f, se = 0.f;
        for (int i = 0; i < rpad; ++i) {
            const float x = __bfloat162float(tile[i][threadIdx.x]);
            const float e = x - __half2float(__float2half_rn(x));       // +-inf if x overflows fp16
            s = fmaf(x, x, s);
            se = fmaf(e, e, se);
        }
        red[threadIdx.x] = s;
        rederr[threadIdx.x] = se;
    }
    // transposed rows: 16 bytes (8 ranks) per item
    const int chunks = rpad / 8;
    for (int item = threadIdx.x; item < 64 * chunks; item += 256) {
        const int jj = item / chunks, c = item % chunks;
        if (j0 + jj < M) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                w[e] = (uint32_t)__bfloat16_as_ushort(tile[c * 8 + 2 * e][jj]) |
                       ((uint32_t)__bfloat16_as_ushort(tile[c * 8 + 2 * e + 1][jj]) << 16);
            reinterpret_cast<uint4*>(r2t)[(size_t)(j0 + jj) * chunks + c] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = 0.f, me = 0.f;
        for (int i = 0; i < 64; ++i) { m = fmaxf(m, red[i]); me = fmaxf(me, rederr[i]); }
        partial[blockIdx.x] = make_float2(m, me);
        __threadfence();
        last = (atomicAdd(arrivals, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (last) {
        __threadfence();
        float m = 0.f, me = 0.f;
        for (int i = threadIdx.x; i < (int)gridDim.x; i += 256) {
            const float2 v = __ldcg(partial + i);
            m = fmaxf(m, v.x);
            me = fmaxf(me, v.y);
        }
        __shared__ float red2[256], red3[256];
        red2[threadIdx.x] = m;
        red3[threadIdx.x] = me;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int i = 1; i < 256; ++i) { m = fmaxf(m, red2[i]); me = fmaxf(me, red3[i]); }
            colnorm[0] = sqrtf(m) * 1.0001f;
            colnorm[1] = sqrtf(me) * 1.0001f;      // NaN-free: me >= 0, possibly +inf
            *arrivals = 0;
        }
    }
}

// ------------------------------------------------------------------------------------------------ host side
using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const RouteParams);

// The instantiation for (RPAD, KCAP, MODE), with its shared-memory limit raised on the current device; null on failure.
template <int RPAD, int KCAP, int MODE>
KernelFn kernel_ready()
{
    static unsigned long long configured = 0;   // one bit per device, per instantiation; guarded by the API mutex
    KernelFn kern = route_lowrank_kernel<RPAD, KCAP, MODE>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!(configured >> (dev & 63) & 1ull)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kRSmem) != cudaSuccess)
            return nullptr;
        configured |= 1ull << (dev & 63);
    }
    return kern;
}

template <int RPAD, int KCAP>
KernelFn kernel_mode(int mode)
{
    switch (mode) {
        case kModeExact: return kernel_ready<RPAD, KCAP, kModeExact>();
        case kModeExactLse: return kernel_ready<RPAD, KCAP, kModeExactLse>();
        case kModeExactFan:
            if constexpr (KCAP > 8) return kernel_ready<RPAD, KCAP, kModeExactFan>();
            return kernel_ready<RPAD, KCAP, kModeExact>();
        case kModeExactLseFan:
            if constexpr (KCAP > 8) return kernel_ready<RPAD, KCAP, kModeExactLseFan>();
            return kernel_ready<RPAD, KCAP, kModeExactLse>();
        default:
#ifdef MORE_WITH_FILTER
            if constexpr (KCAP <= 16) return kernel_ready<RPAD, KCAP, kModeFilter>();
#endif
            return nullptr;
    }
}

template <int RPAD>
KernelFn kernel_kcap(int k, int mode)
{
    if (k <= 8) return kernel_mode<RPAD, 8>(mode);
    if (k <= 16) return kernel_mode<RPAD, 16>(mode);
    return kernel_mode<RPAD, 32>(mode);
}

int kcap_of(int k) { return k <= 8 ? 8 : (k <= 16 ? 16 : 32); }
int rpad_of(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }
size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct ScratchLayout {
    size_t counters, part_val, part_id, part_mz, r2t, r2h, partial, zlo, total;
};

ScratchLayout scratch_layout(const RouteArgs& a, const Plan& p)
{
    ScratchLayout L{};
    size_t off = 0;
    if (p.msplit > 1) {
        const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
        const size_t slots = blocks * (size_t)p.block_tokens * (size_t)p.msplit;
        const size_t kc = (size_t)kcap_of(a.k);
        L.counters = off; off += align_up(blocks * 4, 256);
        L.part_val = off; off += align_up(slots * kc * 4, 256);
        L.part_id = off; off += align_up(slots * kc * 4, 256);
        L.part_mz = off; off += align_up(slots * 8, 256);
    }
    if (p.filter) {
        L.r2t = off; off += align_up((size_t)a.M * rpad_of(a.r) * 2, 256);
        L.r2h = off; off += align_up((size_t)a.M * a.r * 2, 256);
        L.partial = off; off += align_up((size_t)((a.M + 63) / 64) * 8, 256);
        L.zlo = off; off += align_up((size_t)p.ctas * (rpad_of(a.r) / 8) * kEpiThreads * 16, 256);
    }
    L.total = off;
    return L;
}

}  // namespace

bool tcgen05_shape_ok(int T, int h, int r, int M, int k)
{
    return T >= 1 && h % 8 == 0 && M % 8 == 0 && r % 8 == 0 && r <= 64 && k <= 32;
}

size_t lowrank_scratch_bytes(const RouteArgs& a, const Plan& p) { return scratch_layout(a, p).total; }

// Shared-memory plan of a launch: phase-1 stages from the bottom of the ring, R2 stages at its top.  Returns false if
// the shape of the groups leaves no room (the planner never asks for such a shape).
bool lowrank_smem_plan(int rpad, int tg, int es, bool filter, int* nst1, int* st1_bytes, int* nst2, int* st2_bytes,
                       int* r2_off)
{
    const int st2 = es * rpad * 128;
    const int fixed = kCandBytes + (filter ? kZoneBytes : 0);
    int n2 = (kRRing - fixed) / st2;
    n2 = n2 >= 8 ? 8 : (n2 >= 4 ? 4 : n2);                  // a power of two (the kernel masks step numbers with it)
    const int st1 = tg * kXGroupBytes + kR1Bytes;
    // phase 1 wants at least two stages below the R2 stages
    while (n2 > 2 && kRRing - n2 * st2 < 2 * st1) n2 /= 2;
    if (n2 < 2) return false;
    if (n2 == 3) n2 = 2;
    const int off = (kRRing - n2 * st2) & ~1023;
    int n1 = off / st1;
    if (n1 > kMaxStages1) n1 = kMaxStages1;
    if (n1 < 1) return false;
    *nst1 = n1; *st1_bytes = st1; *nst2 = n2; *st2_bytes = st2; *r2_off = off;
    return true;
}

int launch_route_prepare(const RouteArgs& a, int rpad, void* r2h, void* r2t, void* partial, DeviceCtx& ctx)
{
    route_prepare_kernel<<<(a.M + 63) / 64, 256, 0, a.stream>>>(a.R2, a.r, rpad, a.M, static_cast<__half*>(r2h),
                                                               static_cast<__nv_bfloat16*>(r2t),
                                                               static_cast<float2*>(partial), ctx.colnorm,
                                                               ctx.prep_arrivals, a.out_counts);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

int launch_lowrank(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch)
{
    const int rpad = rpad_of(a.r);
    RouteParams rp{};
    if (!lowrank_smem_plan(rpad, p.tg, p.es, p.filter, &rp.nst1, &rp.st1_bytes, &rp.nst2, &rp.st2_bytes, &rp.r2_off))
        return MORE_ERR_SHAPE;
    const ScratchLayout L = scratch_layout(a, p);
    char* base = static_cast<char*>(scratch);
    CUtensorMap mx, m1, m2;
    // few tokens and several expert ranges per CTA: spread the working warps over the lane quarters (see the kernel)
    const bool spread = p.tg == 1 && p.block_tokens <= 64 && p.es >= 2;
    int rc = get_tensor_map(a.X, a.T, a.h, spread ? 32 : 128, 64, &mx);
    if (rc == MORE_OK) rc = get_tensor_map(a.R1, a.h, a.r, 64, 64, &m1);
    // the filter sweeps the fp16 copy of R2 in scratch (same shape; a 16-bit type either way as far as TMA cares)
    if (rc == MORE_OK) rc = get_tensor_map(p.filter ? static_cast<const void*>(base + L.r2h) : a.R2, a.r, a.M, rpad, 64, &m2);
    if (rc != MORE_OK) return rc;

    rp.T = a.T; rp.h = a.h; rp.r = a.r; rp.M = a.M; rp.k = a.k; rp.gate_mode = a.gate_mode;
    rp.msplit = p.msplit; rp.es = p.es; rp.tg = p.tg;
    rp.spread = spread ? 1 : 0;
    rp.block_tokens = p.block_tokens;
    rp.blocks64 = (a.M + 63) / 64;
    rp.out_idx = a.out_idx; rp.out_gate = a.out_gate; rp.out_counts = a.out_counts;
    rp.out_topval = a.out_topval; rp.out_lse = a.out_lse;
    rp.status = ctx.status;
    rp.stats = ctx.stats;
    rp.R2 = a.R2;
    if (p.msplit > 1) {
        rp.counters = reinterpret_cast<unsigned*>(base + L.counters);
        rp.part_val = reinterpret_cast<float*>(base + L.part_val);
        rp.part_id = reinterpret_cast<int*>(base + L.part_id);
        rp.part_mz = reinterpret_cast<float2*>(base + L.part_mz);
    }
    const bool lse = (a.gate_mode == MORE_GATE_FULL_SOFTMAX) || (a.out_lse != nullptr);
    int mode = lse ? kModeExactLse : kModeExact;
    if (p.msplit >= 8) mode = lse ? kModeExactLseFan : kModeExactFan;
    if (p.filter) {
        if (lse || a.k > 16) return MORE_ERR_SHAPE;
        mode = kModeFilter;
    }
    KernelFn kern = rpad == 16 ? kernel_kcap<16>(a.k, mode) : (rpad == 32 ? kernel_kcap<32>(a.k, mode) : kernel_kcap<64>(a.k, mode));
    if (!kern) return MORE_ERR_CUDA;
    // every host-side step that can fail is behind us: only now is anything enqueued and the first output touched
    if (p.msplit > 1) {
        const size_t blocks = (size_t)(a.T + p.block_tokens - 1) / p.block_tokens;
        if (cudaMemsetAsync(rp.counters, 0, blocks * 4, a.stream) != cudaSuccess) return MORE_ERR_CUDA;
    }
    if (p.filter) {
        rp.r2t = reinterpret_cast<const __nv_bfloat16*>(base + L.r2t);
        rp.colnorm = ctx.colnorm;
        rp.zlo = reinterpret_cast<uint4*>(base + L.zlo);
        // the preparation kernel also clears out_counts
        const int prc = launch_route_prepare(a, rpad, base + L.r2h, base + L.r2t, base + L.partial, ctx);
        if (prc != MORE_OK) return prc;
    } else if (cudaMemsetAsync(a.out_counts, 0, (size_t)a.M * sizeof(int32_t), a.stream) != cudaSuccess) {
        return MORE_ERR_CUDA;
    }
    kern<<<p.ctas, kRThreads, kRSmem, a.stream>>>(mx, m1, m2, rp);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

}  // namespace more
