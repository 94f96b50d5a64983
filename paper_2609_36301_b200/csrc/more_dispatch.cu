// Dispatch bookkeeping after routing: the "Sort + Count" box of the layer's forward flowchart ((N,k) -> (Nk) sorted
// indices + offsets).  Given the selected expert ids and their per-expert counts it produces, for the grouped expert
// GEMMs that follow, where each expert's run of (token, slot) pairs starts and the list of pairs grouped by expert.
//
//   dispatch_scan     one CTA: exclusive prefix sum of counts[M] -> offsets[M+1], and a copy that serves as the
//                     per-expert write cursor.
//   dispatch_scatter  one thread per (token, slot) pair p = n*k + j: claims the next place of its expert's run with
//                     an atomic add on the cursor and writes p there.
//
// The order of pairs inside one expert's run depends on the order in which the atomics land; everything else is
// deterministic (counts and offsets are exact integers).
#include "more_internal.h"

namespace more {

namespace {

constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(kScanThreads)
dispatch_scan(const int32_t* __restrict__ counts, int M, int32_t* __restrict__ offsets, int32_t* __restrict__ cursor)
{
    __shared__ int warp_tot[kScanThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (M + kScanThreads - 1) / kScanThreads;        // contiguous run of experts per thread
    const int lo = min(tid * per, M), hi = min(lo + per, M);
    int sum = 0;
    for (int e = lo; e < hi; ++e) sum += counts[e];
    int incl = sum;                                               // inclusive scan of the per-thread sums
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += up;
        }
        warp_tot[lane] = w;                                       // inclusive totals of the warps
    }
    __syncthreads();
    int run = incl - sum + (warp > 0 ? warp_tot[warp - 1] : 0);  // exclusive prefix of this thread's first expert
    for (int e = lo; e < hi; ++e) {
        offsets[e] = run;
        cursor[e] = run;
        run += counts[e];
    }
    if (tid == kScanThreads - 1) offsets[M] = warp_tot[kScanThreads / 32 - 1];
}

__global__ void dispatch_scatter(const int32_t* __restrict__ idx, long long pairs, int M, int32_t* __restrict__ cursor,
                                 int32_t* __restrict__ sorted_pairs)
{
    const int lane = threadIdx.x & 31;
    const long long stride = (long long)gridDim.x * blockDim.x;
    // whole warps iterate together (the loop bound is rounded up per warp) so that lanes routed to the same expert
    // can share one atomic: with skewed loads thousands of pairs hit the same cursor
    const long long first = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    for (long long base = first - lane; base < pairs; base += stride) {
        const long long p = base + lane;
        const int e = (p < pairs) ? idx[p] : -1;
        const bool live = (unsigned)e < (unsigned)M;
        const unsigned peers = __match_any_sync(0xffffffffu, live ? e : -1 - lane);   // lanes with my expert id
        int place = 0;
        if (live) {
            const int leader = __ffs(peers) - 1;
            if (lane == leader) place = atomicAdd(cursor + e, __popc(peers));
            place = __shfl_sync(peers, place, leader) + __popc(peers & ((1u << lane) - 1u));
            sorted_pairs[place] = (int32_t)p;
        }
    }
}

}  // namespace

size_t dispatch_scratch_bytes(int M) { return (size_t)M * sizeof(int32_t); }

int launch_dispatch(const int32_t* idx, const int32_t* counts, int T, int k, int M, int32_t* offsets,
                    int32_t* sorted_pairs, void* scratch, cudaStream_t stream)
{
    int32_t* cursor = static_cast<int32_t*>(scratch);
    dispatch_scan<<<1, kScanThreads, 0, stream>>>(counts, M, offsets, cursor);
    count_launch(1);
    const long long pairs = (long long)T * k;
    if (pairs > 0) {
        const int threads = 256;
        long long blocks = (pairs + threads - 1) / threads;
        if (blocks > 148 * 16) blocks = 148 * 16;
        dispatch_scatter<<<(int)blocks, threads, 0, stream>>>(idx, pairs, M, cursor, sorted_pairs);
        count_launch(1);
    }
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

}  // namespace more
