// Generic (CUDA-core) path of the low-rank router: any shape within MORE_K_MAX / MORE_R_MAX.
//
// Two kernels.  generic_project_z computes z = X R1 in fp32 (Algorithm 1, phase 1) into scratch;
// generic_route_tokens gives one warp per token: the 32 lanes sweep the experts 32 at a time
// (logit = z . R2[:, j] in fp32, Algorithm 1 phase 2), keep the running top-k as a sorted list held one
// entry per lane, and carry a lane-local online (max, sum-of-exponentials) pair (Eq. app_online) that is
// merged across lanes at the end.  Slow next to the tensor-core path; it exists for shapes that path
// cannot take and as an independent on-device cross-check.
#include "more_internal.h"

#include <float.h>
#include <limits.h>

namespace more {

namespace {

constexpr int kWarpsPerBlock = 8;

__global__ void generic_project_z(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ R1,
                                  float* __restrict__ Z, int h, int r)
{
    const int64_t n = blockIdx.x;
    const __nv_bfloat16* x = X + n * (int64_t)h;
    for (int i = threadIdx.x; i < r; i += blockDim.x) {
        float acc = 0.f;
        for (int c = 0; c < h; ++c)
            acc = fmaf(__bfloat162float(x[c]), __bfloat162float(R1[(int64_t)c * r + i]), acc);
        Z[n * (int64_t)r + i] = acc;
    }
}

__global__ void generic_route_tokens(const float* __restrict__ Z, const __nv_bfloat16* __restrict__ R2,
                                     int T, int r, int M, int k, int gate_mode, int want_lse,
                                     int32_t* __restrict__ out_idx, float* __restrict__ out_gate,
                                     int32_t* __restrict__ out_counts, float* __restrict__ out_topval,
                                     float* __restrict__ out_lse)
{
    extern __shared__ float zs_all[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * kWarpsPerBlock + warp;
    if (n >= T) return;                       // whole warp leaves together
    float* zs = zs_all + (size_t)warp * r;
    for (int i = lane; i < r; i += 32) zs[i] = Z[n * (int64_t)r + i];
    __syncwarp();

    // Sorted list, entry q in lane q (q < k): larger logit first, equal logits by smaller id.
    float lv = -INFINITY;
    int li = INT_MAX;
    float tau = -INFINITY;                    // logit of entry k-1
    float m_run = -INFINITY, z_run = 0.f;     // lane-local online softmax state

    for (int j0 = 0; j0 < M; j0 += 32) {
        const int j = j0 + lane;
        float l = -INFINITY;
        if (j < M) {
            l = 0.f;
            for (int i = 0; i < r; ++i) l = fmaf(zs[i], __bfloat162float(R2[(int64_t)i * M + j]), l);
            if (want_lse) {
                float m_new = fmaxf(m_run, l);
                z_run = z_run * expf(m_run - m_new) + expf(l - m_new);   // exp(-inf) = 0 on the first element
                m_run = m_new;
            }
        }
        unsigned cand = __ballot_sync(0xffffffffu, l > tau);
        while (cand) {
            const int src = __ffs(cand) - 1;
            cand &= cand - 1;
            const float cv = __shfl_sync(0xffffffffu, l, src);
            const int cj = j0 + src;
            const bool better = (lane < k) && (lv > cv || (lv == cv && li < cj));
            const int pos = __popc(__ballot_sync(0xffffffffu, better));   // entries ahead of the candidate
            const float up_v = __shfl_up_sync(0xffffffffu, lv, 1);
            const int up_i = __shfl_up_sync(0xffffffffu, li, 1);
            if (pos < k) {
                if (lane > pos && lane < k) { lv = up_v; li = up_i; }
                if (lane == pos) { lv = cv; li = cj; }
            }
            tau = __shfl_sync(0xffffffffu, lv, k - 1);
        }
    }

    // (m, Z) over all experts: merge the 32 lane-local pairs.
    float m_all = m_run, z_all = z_run;
    if (want_lse) {
        for (int o = 16; o > 0; o >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, o));
        z_all = (m_run == -INFINITY) ? 0.f : z_run * expf(m_run - m_all);
        for (int o = 16; o > 0; o >>= 1) z_all += __shfl_xor_sync(0xffffffffu, z_all, o);
    }
    const float v0 = __shfl_sync(0xffffffffu, lv, 0);
    float e = (lane < k) ? expf(lv - v0) : 0.f;
    float s = e;
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane < k) {
        const float g = (gate_mode == MORE_GATE_TOPK_SOFTMAX) ? e / s : expf(lv - m_all) / z_all;
        out_idx[n * k + lane] = li;
        out_gate[n * k + lane] = g;
        if (out_topval) out_topval[n * k + lane] = lv;
        if ((unsigned)li < (unsigned)M) atomicAdd(out_counts + li, 1);   // (non-finite inputs can leave a slot unfilled)
    }
    if (out_lse && lane == 0) out_lse[n] = m_all + logf(z_all);
}

// psum[j] += sum over a chunk of tokens of exp(l_{n,j} - lse_n): thread per expert, 256 tokens per block row.
__global__ void generic_psum_kernel(const float* __restrict__ Z, const __nv_bfloat16* __restrict__ R2,
                                    const float* __restrict__ lse, int T, int r, int M, float* __restrict__ psum)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int n0 = blockIdx.y * 256, n1 = min(T, n0 + 256);
    if (j >= M) return;
    float acc = 0.f;
    for (int n = n0; n < n1; ++n) {
        const float* z = Z + (int64_t)n * r;
        float l = 0.f;
        for (int i = 0; i < r; ++i) l = fmaf(z[i], __bfloat162float(R2[(int64_t)i * M + j]), l);
        acc += expf(l - lse[n]);
    }
    atomicAdd(psum + j, acc);
}

}  // namespace

int launch_generic_psum(const __nv_bfloat16* X, const __nv_bfloat16* R1, const __nv_bfloat16* R2, int T, int h, int r,
                        int M, const float* lse, float* psum, void* scratch, cudaStream_t stream)
{
    float* Z = static_cast<float*>(scratch);
    generic_project_z<<<T, 128, 0, stream>>>(X, R1, Z, h, r);
    dim3 grid((M + 127) / 128, (T + 255) / 256);
    generic_psum_kernel<<<grid, 128, 0, stream>>>(Z, R2, lse, T, r, M, psum);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

size_t generic_scratch_bytes(const RouteArgs& a) { return (size_t)a.T * (size_t)a.r * sizeof(float); }

int launch_generic(const RouteArgs& a, DeviceCtx& ctx, void* scratch)
{
    (void)ctx;
    if (a.T == 0) return MORE_OK;
    float* Z = static_cast<float*>(scratch);
    const int want_lse = (a.gate_mode == MORE_GATE_FULL_SOFTMAX) || (a.out_lse != nullptr);
    generic_project_z<<<a.T, 128, 0, a.stream>>>(a.X, a.R1, Z, a.h, a.r);
    const int blocks = (a.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const size_t smem = (size_t)kWarpsPerBlock * a.r * sizeof(float);
    generic_route_tokens<<<blocks, kWarpsPerBlock * 32, smem, a.stream>>>(
        Z, a.R2, a.T, a.r, a.M, a.k, a.gate_mode, want_lse, a.out_idx, a.out_gate, a.out_counts, a.out_topval,
        a.out_lse);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

}  // namespace more
