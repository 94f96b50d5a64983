// Hierarchical top-k for a router whose expert dimension is sharded (the paper leaves "local top-k per device, then
// global top-k" to future work; the combination of the per-shard softmax statistics is Eq. app_online applied to whole
// shards).  Every shard has routed the same T tokens over its own experts with more_route_ex and reports its k best
// (id, logit) pairs per token and its log-sum-exp; once the shards' reports sit side by side in this GPU's memory
// (an all-gather of k pairs per token and shard -- nothing of size M crosses a link), one thread per token merges
// them: a sorted list of k (value, id) pairs in registers, each candidate inserted with the full order (value
// descending, id ascending), then gates, ids and the expert histogram as in the router's own finish.
#include "more_internal.h"

#include <limits.h>

namespace more {

namespace {

constexpr int kMergeThreads = 128;

struct MergeParams {
    const int32_t* idx;      // [S][T][k]
    const float* val;        // [S][T][k]
    const float* lse;        // [S][T] or nullptr
    int S, T, k, M, gate_mode;
    int base[MORE_MERGE_MAX_SHARDS];   // added to the ids of each shard
    int32_t* out_idx;
    float* out_gate;
    float* out_val;          // nullable
    float* out_lse;          // nullable
    int32_t* out_counts;
};

template <int KCAP>
__global__ void __launch_bounds__(kMergeThreads) merge_shards_kernel(const MergeParams p)
{
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    const int t = blockIdx.x * kMergeThreads + threadIdx.x;
    if (t >= p.T) return;
    float v[KCAP];
    int id[KCAP];
#pragma unroll
    for (int s = 0; s < KCAP; ++s) { v[s] = -INFINITY; id[s] = INT_MAX; }
    const int k = p.k;
    for (int sh = 0; sh < p.S; ++sh) {
        const size_t row = ((size_t)sh * (size_t)p.T + (size_t)t) * (size_t)k;
        for (int j = 0; j < k; ++j) {
            const int raw = p.idx[row + j];
            const int e = raw + p.base[sh];
            const float x = p.val[row + j];
            if (raw < 0 || e >= p.M || !(x > -INFINITY)) continue;              // unused slot
            // skip what cannot enter: below the last entry, or equal to it with a larger id
            if (!(x > v[KCAP - 1] || (x == v[KCAP - 1] && e < id[KCAP - 1]))) continue;
            auto ahead = [&](int s) { return x > v[s] || (x == v[s] && e < id[s]); };
#pragma unroll
            for (int s = KCAP - 1; s > 0; --s) {
                const bool above_prev = ahead(s - 1);
                const bool above_this = ahead(s);
                v[s] = above_prev ? v[s - 1] : (above_this ? x : v[s]);
                id[s] = above_prev ? id[s - 1] : (above_this ? e : id[s]);
            }
            const bool top = ahead(0);
            v[0] = top ? x : v[0];
            id[0] = top ? e : id[0];
        }
    }
    // KCAP >= k: with fewer than KCAP slots wanted the list simply holds more than needed; only the first k count
    float lse2 = 0.f;                                     // log2-domain log-sum-exp over all shards
    if (p.lse) {
        float m = -INFINITY;
        for (int sh = 0; sh < p.S; ++sh) m = fmaxf(m, p.lse[(size_t)sh * p.T + t]);
        float z = 0.f;
        for (int sh = 0; sh < p.S; ++sh) z += exp2f((p.lse[(size_t)sh * p.T + t] - m) * kLog2e);
        lse2 = m * kLog2e + log2f(z);
        if (p.out_lse) p.out_lse[t] = lse2 * kLn2;
    }
    float denom = 0.f;
    if (p.gate_mode == MORE_GATE_TOPK_SOFTMAX) {
#pragma unroll
        for (int q = 0; q < KCAP; ++q)
            if (q < k && id[q] != INT_MAX) denom += exp2f((v[q] - v[0]) * kLog2e);
    }
    const float inv = (p.gate_mode == MORE_GATE_TOPK_SOFTMAX) ? 1.f / denom : 1.f;
    const float ref2 = (p.gate_mode == MORE_GATE_TOPK_SOFTMAX) ? v[0] * kLog2e : lse2;
#pragma unroll
    for (int q = 0; q < KCAP; ++q) {
        if (q < k) {
            const size_t o = (size_t)t * (size_t)k + (size_t)q;
            const bool used = id[q] != INT_MAX;
            p.out_idx[o] = used ? id[q] : -1;
            p.out_gate[o] = used ? exp2f(v[q] * kLog2e - ref2) * inv : 0.f;
            if (p.out_val) p.out_val[o] = v[q];
            if (used) atomicAdd(p.out_counts + id[q], 1);
        }
    }
}

}  // namespace

}  // namespace more

using namespace more;

extern "C" int more_merge_shards(const int32_t* idx, const float* topval, const float* lse, const int32_t* shard_base,
                                 int S, int T, int k, int M, int gate_mode, int32_t* out_idx, float* out_gate,
                                 float* out_topval, float* out_lse, int32_t* out_counts, void* stream)
{
    if (S < 1 || S > MORE_MERGE_MAX_SHARDS || T < 0 || k < 1 || k > MORE_K_MAX || M < 1) return MORE_ERR_SHAPE;
    if (gate_mode != MORE_GATE_TOPK_SOFTMAX && gate_mode != MORE_GATE_FULL_SOFTMAX) return MORE_ERR_MODE;
    if (!out_counts) return MORE_ERR_NULL;
    if (T > 0 && (!idx || !topval || !out_idx || !out_gate)) return MORE_ERR_NULL;
    if (gate_mode == MORE_GATE_FULL_SOFTMAX && !lse) return MORE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(out_counts, 0, (size_t)M * sizeof(int32_t), st) != cudaSuccess) return MORE_ERR_CUDA;
    if (T == 0) return MORE_OK;
    MergeParams p;
    p.idx = idx; p.val = topval; p.lse = lse;
    p.S = S; p.T = T; p.k = k; p.M = M; p.gate_mode = gate_mode;
    for (int s = 0; s < MORE_MERGE_MAX_SHARDS; ++s) p.base[s] = (shard_base && s < S) ? shard_base[s] : 0;
    p.out_idx = out_idx; p.out_gate = out_gate; p.out_val = out_topval; p.out_lse = out_lse; p.out_counts = out_counts;
    const int blocks = (T + kMergeThreads - 1) / kMergeThreads;
    if (k <= 8) merge_shards_kernel<8><<<blocks, kMergeThreads, 0, st>>>(p);
    else if (k <= 16) merge_shards_kernel<16><<<blocks, kMergeThreads, 0, st>>>(p);
    else merge_shards_kernel<32><<<blocks, kMergeThreads, 0, st>>>(p);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}
