// Per-token running top-k of the router kernels: the sorted register list, the candidate buffer in shared memory that
// defers the inserts, the zone store of the filter mode, and the plain CUDA-core sweep that re-routes a token exactly.
// Internal; every translation unit gets its own copy.
#pragma once

#include "sm100_common.cuh"

#include <cuda_bf16.h>
#include <limits.h>
#include <math.h>
#include <stdint.h>

namespace more {

namespace {

constexpr unsigned kFullMask = 0xffffffffu;

// ---------------------------------------------------------------------------------------------- running top-k
// Sorted (value, id) list of one token, held in registers.
template <int KCAP>
struct TopList {
    float v[KCAP];
    int id[KCAP];
    __device__ __forceinline__ void init()
    {
#pragma unroll
        for (int s = 0; s < KCAP; ++s) { v[s] = -INFINITY; id[s] = INT_MAX; }
    }
    __device__ __forceinline__ float tau() const { return v[KCAP - 1]; }
    // Insert (x, j) with x > tau().  Equal values keep the earlier (smaller-id) entry ahead.
    __device__ __forceinline__ void insert(float x, int j)
    {
#pragma unroll
        for (int s = KCAP - 1; s > 0; --s) {
            const bool above_prev = x > v[s - 1];
            const bool above_this = x > v[s];
            v[s] = above_prev ? v[s - 1] : (above_this ? x : v[s]);
            id[s] = above_prev ? id[s - 1] : (above_this ? j : id[s]);
        }
        const bool top = x > v[0];
        v[0] = top ? x : v[0];
        id[0] = top ? j : id[0];
    }
    // Replace this list by the KCAP best of it and of another sorted list under the full order (value descending, id
    // ascending); other_v(s) / other_id(s) return entry s of the other list (read where it lies: no second list in
    // registers).  Entry s against the other list's entry KCAP-1-s keeps the KCAP best of the union as a bitonic
    // sequence, which log2(KCAP) stages of compare-exchanges sort: straight-line code, the same work whatever the data.
    template <class FV, class FI>
    __device__ __forceinline__ void merge_sorted(FV other_v, FI other_id)
    {
#pragma unroll
        for (int s = 0; s < KCAP; ++s) {
            const float x = other_v(KCAP - 1 - s);
            const int j = other_id(KCAP - 1 - s);
            const bool take = x > v[s] || (x == v[s] && j < id[s]);
            v[s] = take ? x : v[s];
            id[s] = take ? j : id[s];
        }
#pragma unroll
        for (int stride = KCAP / 2; stride > 0; stride >>= 1) {
#pragma unroll
            for (int s = 0; s < KCAP; ++s) {
                if ((s & stride) == 0) {
                    const int t = s + stride;
                    const bool swap = v[t] > v[s] || (v[t] == v[s] && id[t] < id[s]);
                    const float hv = swap ? v[t] : v[s], lv = swap ? v[s] : v[t];
                    const int hi = swap ? id[t] : id[s], li = swap ? id[s] : id[t];
                    v[s] = hv; v[t] = lv; id[s] = hi; id[t] = li;
                }
            }
        }
    }
    // Insert with the full order (value descending, id ascending): for merging lists whose ids interleave.
    __device__ __forceinline__ void insert_ordered(float x, int j)
    {
        auto ahead = [&](int s) { return x > v[s] || (x == v[s] && j < id[s]); };
#pragma unroll
        for (int s = KCAP - 1; s > 0; --s) {
            const bool above_prev = ahead(s - 1);
            const bool above_this = ahead(s);
            v[s] = above_prev ? v[s - 1] : (above_this ? x : v[s]);
            id[s] = above_prev ? id[s - 1] : (above_this ? j : id[s]);
        }
        const bool top = ahead(0);
        v[0] = top ? x : v[0];
        id[0] = top ? j : id[0];
    }
};

// ---------------------------------------------------------------------------------------- shared-memory access
__device__ __forceinline__ float lds_f32(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ int lds_s32(uint32_t a)
{
    int v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t a, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory"); }
__device__ __forceinline__ void sts_s32(uint32_t a, int v) { asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Running top-k of one token.  Between folds the sorted list is left alone.  A chunk of 16 logits is looked at as four
// groups of four; every group whose maximum beats the cached threshold `thr` (never above the true one) is appended
// whole, in ascending column order, to this thread's column of a shared-memory candidate buffer: one predicated
// 16-byte store of the four values (they sit in four consecutive registers as loaded from tensor memory), one
// predicated 4-byte store of the group's first column, no branch.  fold() then inserts the buffered elements that beat
// the up-to-date threshold, so the inserts of several chunks of all 32 tokens of a warp are executed together.  A chunk
// appends at most 4 entries and the warp folds as soon as some token has fewer than 4 free slots left, so the buffer
// cannot overflow.
//
// FILTER: the logits are approximate to within E; thr sits W = 2E below the list's last value, elements that land in
// that zone (directly, or pushed out of the list) are kept in a second small per-token store, pruned when it fills
// up; a token whose zone still overflows is flagged for the fallback.
template <int KCAP, bool FILTER, int NT, int CAP, int PER_CHECK, int ZCAP = 8, bool EXT = false>
struct Selector {
    static constexpr int kCandValStride = NT * 16;   // bytes between successive value slots of one thread
    static constexpr int kCandColStride = NT * 4;    // ... and between its column slots
    static constexpr int kCandValBytes = CAP * kCandValStride;
    static constexpr int kCandBytes = CAP * (kCandValStride + kCandColStride);
    static constexpr int kZoneStride = NT * 4;
    static constexpr int kZoneIdOff = ZCAP * kZoneStride;
    static constexpr int kZoneBytes = 2 * kZoneIdOff;
    static_assert(CAP > PER_CHECK, "candidate buffer too small");
    TopList<KCAP> L;
    float thr;
    float W;
    float ext;        // EXT: a lower bound on the final k-th value known from elsewhere (strictly below it)
    uint32_t ptr, cptr, base, cbase, warn;
    uint32_t zptr, zbase;
    bool overflow;

    __device__ __forceinline__ void init(uint32_t first_val_slot, uint32_t first_col_slot, uint32_t first_zone_slot, float w)
    {
        L.init();
        thr = -INFINITY;
        ext = -INFINITY;
        W = w;
        base = ptr = first_val_slot;
        cbase = cptr = first_col_slot;
        warn = first_val_slot + (CAP - PER_CHECK) * kCandValStride;   // PER_CHECK entries can arrive between two checks
        zbase = zptr = first_zone_slot;
        overflow = false;
    }
    __device__ __forceinline__ float limit() const { return FILTER ? L.tau() - W : (EXT ? fmaxf(L.tau(), ext) : L.tau()); }

    // Drop the zone entries that have fallen more than W below the list; flag the token if the zone is still full.
    __device__ __forceinline__ void prune()
    {
        const float lim = limit();
        uint32_t rd = zbase, wr = zbase;
        while (__any_sync(kFullMask, rd < zptr)) {
            const bool act = rd < zptr;
            float v = -INFINITY;
            int id = 0;
            if (act) { v = lds_f32(rd); id = lds_s32(rd + kZoneIdOff); }
            if (act && v > lim) {
                sts_f32(wr, v);
                sts_s32(wr + kZoneIdOff, id);
                wr += kZoneStride;
            }
            rd += kZoneStride;
        }
        zptr = wr;
        if (zptr >= zbase + ZCAP * kZoneStride) {
            // more near-ties than the store holds: the token goes to the fallback, and from here on nothing of it is
            // collected any more (an infinite list admits no candidate), so that it cannot slow its warp down
            overflow = true;
            zptr = zbase;
#pragma unroll
            for (int s = 0; s < KCAP; ++s) L.v[s] = INFINITY;
        }
    }

    // Called by all 32 lanes of a warp together.  Every round handles at most one element per token: the maximum of
    // the token's current entry, which is then struck out of the entry; a token whose entry holds nothing above its
    // (rising) limit any more moves on to its next entries.  The rounds end when no token has anything left.
    __device__ __forceinline__ void fold()
    {
#ifdef MORE_EXP_NOFOLD
        ptr = base; cptr = cbase; thr = 3.2f; return;      // timing experiment: what the scan alone costs
#endif
        uint32_t a = base, c = cbase;
        float x0 = -INFINITY, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
        int col = 0;
        for (;;) {
            float m = fmaxf(max3(x0, x1, x2), x3);
            while (!(m > limit()) && a < ptr) {
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=f"(x0), "=f"(x1), "=f"(x2), "=f"(x3) : "r"(a) : "memory");
                col = lds_s32(c);
                a += kCandValStride;
                c += kCandColStride;
                m = fmaxf(max3(x0, x1, x2), x3);
            }
            const bool pass = m > limit();
            if (!__any_sync(kFullMask, pass)) break;
            // the maximum's lowest column on a tie, so that equal logits enter the list in ascending column order
            const int j = (x0 == m) ? 0 : ((x1 == m) ? 1 : ((x2 == m) ? 2 : 3));
            if constexpr (FILTER) {
                const bool ins = pass && (m > L.tau());
                const float ev = ins ? L.v[KCAP - 1] : m;          // what may belong into the zone: the entry pushed
                const int ei = ins ? L.id[KCAP - 1] : col + j;     // out of the list, or the element itself
                if (ins) L.insert(m, col + j);
                if (pass && ev > limit()) {
                    sts_f32(zptr, ev);
                    sts_s32(zptr + kZoneIdOff, ei);
                    zptr += kZoneStride;
                }
                if (__any_sync(kFullMask, zptr >= zbase + ZCAP * kZoneStride)) prune();
            } else {
                if (pass) L.insert(m, col + j);
            }
            x0 = (j == 0) ? -INFINITY : x0;
            x1 = (j == 1) ? -INFINITY : x1;
            x2 = (j == 2) ? -INFINITY : x2;
            x3 = (j == 3) ? -INFINITY : x3;
        }
        ptr = base;
        cptr = cbase;
        thr = limit();
    }
    // The same result as fold() for the start of a sweep, when nearly every buffered element still gets in: every
    // element of every entry is offered to the list in column order (an insert changes nothing for a value at or
    // below the list's last), straight-line code instead of one data-dependent round per element.  Not for FILTER.
    __device__ __forceinline__ void fold_all()
    {
        static_assert(!FILTER, "the zone store needs fold()");
        uint32_t a = base, c = cbase;
        while (__any_sync(kFullMask, a < ptr)) {
            float x0 = -INFINITY, x1 = -INFINITY, x2 = -INFINITY, x3 = -INFINITY;
            int col = 0;
            if (a < ptr) {
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=f"(x0), "=f"(x1), "=f"(x2), "=f"(x3) : "r"(a) : "memory");
                col = lds_s32(c);
            }
            L.insert(x0, col);
            L.insert(x1, col + 1);
            L.insert(x2, col + 2);
            L.insert(x3, col + 3);
            a += kCandValStride;
            c += kCandColStride;
        }
        ptr = base;
        cptr = cbase;
        thr = limit();
    }
    // if (t > thr) append {v0, v1, v2, v3} and col
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
            : "f"(t), "f"(v0), "f"(v1), "f"(v2), "f"(v3), "r"(col), "f"(thr), "n"(kCandValStride), "n"(kCandColStride)
            : "memory");
    }
    // v: 16 logits of columns col0.., t: maxima of the groups (v[4i] .. v[4i+3]).
    __device__ __forceinline__ void scan(const float (&v)[16], const float (&t)[4], int col0)
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) append4(t[i], v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3], col0 + 4 * i);
    }
};

// Exact top-KCAP of one token over experts [e_lo, e_hi) by a plain CUDA-core sweep, run by one warp: lane j takes the
// experts e_lo + j, e_lo + j + 32, ..., computes each logit as the fp32 chain l = fma(z[i], R2[i][e], l) over i
// ascending (the same chain the rescoring of the filter uses), keeps a lane-local sorted list, and the 32 lists are
// merged by KCAP rounds of a warp-wide argmax under the full order (value descending, id ascending).  zs: the token's
// z in shared memory (r floats); the result goes to out_v / out_id (shared memory, KCAP entries).
template <int KCAP>
__device__ __noinline__ void exact_topk_warp(const float* zs, const __nv_bfloat16* __restrict__ R2, int r, int M,
                                             int e_lo, int e_hi, float* out_v, int* out_id, int lane)
{
    TopList<KCAP> L;
    L.init();
    for (int e = e_lo + lane; e < e_hi; e += 32) {
        float l = 0.f;
        for (int i = 0; i < r; ++i) l = fmaf(zs[i], __bfloat162float(R2[(int64_t)i * M + e]), l);
        if (l > L.tau()) L.insert(l, e);
    }
    for (int q = 0; q < KCAP; ++q) {
        float bv = L.v[0];
        int bi = L.id[0];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(kFullMask, bv, o);
            const int oi = __shfl_xor_sync(kFullMask, bi, o);
            const bool take = ov > bv || (ov == bv && oi < bi);
            bv = take ? ov : bv;
            bi = take ? oi : bi;
        }
        if (lane == 0) { out_v[q] = bv; out_id[q] = bi; }
        if (L.id[0] == bi && L.v[0] == bv && bi != INT_MAX) {      // the winning lane pops its head
#pragma unroll
            for (int s = 0; s + 1 < KCAP; ++s) { L.v[s] = L.v[s + 1]; L.id[s] = L.id[s + 1]; }
            L.v[KCAP - 1] = -INFINITY;
            L.id[KCAP - 1] = INT_MAX;
        }
    }
}

}  // namespace

}  // namespace more
