// Training-forward statistic of Algorithm 2 on sm_100a: psum[i] = sum_n P_{n,i}, the column sums of the row-wise
// softmax over all M experts (Eq. app_softmax, Eq. app_psum), given each token's log-sum-exp from the routing sweep.
// This is Algorithm 2's second sweep: the logit tiles are produced again and reduced along the TOKEN axis, and the
// T x M probabilities never exist in memory.
//
// The first half of the kernel is the router's: TMA streams X and R1, tcgen05.mma accumulates z = X_blk R1 for a
// block of 256 tokens in TMEM, the epilogue threads narrow it to bf16 hi + lo in shared memory.  The second
// contraction is issued TRANSPOSED, D[expert][token] = R2[:, tile]^T z^T: the R2 tile is the (MN-major) A operand,
// z the (K-major) B operand, so a TMEM lane is an expert and its columns are tokens.  Each epilogue thread then owns
// one expert of the tile and adds exp(y - lse_token) over the 128 token columns of its half in registers -- a column
// sum with no cross-lane traffic -- and finishes with one atomic add into psum.  (In the router the lanes are tokens,
// because there the reduction runs along the expert axis.)
//
// Warp roles, shared-memory ring, barriers and the bounded waits are those of the router kernel.
#include "sm100_common.cuh"

#include <math.h>

namespace more {

namespace {

struct PsumParams {
    int T, h, r, M, msplit, tiles_total;
    const float* lse;    // [T] natural-log log-sum-exp of every token's logits
    float* psum;         // [M], zeroed before the launch
    int* status;
};

template <int RPAD>
__global__ void __launch_bounds__(kThreads, 2)
psum_tcgen05_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_r1,
                    const __grid_constant__ CUtensorMap map_r2, const PsumParams p)
{
    constexpr int kKSteps = RPAD / 16;
    constexpr int kZopOne = (RPAD == 64) ? 32768 : 16384;       // [hi | lo] operand of one 128-token half
    constexpr int kZopBytes = 2 * kZopOne;
    constexpr int kLseBytes = 1024;                              // 256 floats: log2-scaled lse of the block's tokens
    constexpr int kR2StageBytes = RPAD * 256;
    constexpr int kStagesP2 = (RPAD == 64) ? 2 : 4;
    static_assert(kZopBytes + kLseBytes + kStagesP2 * kR2StageBytes <= kRingBytes, "phase-2 layout does not fit");
    constexpr float kLog2e = 1.4426950408889634f;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    uint8_t* ctl = ring_ptr + kRingBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctl);
    constexpr int B_FULL1 = 0, B_EMPTY1 = B_FULL1 + kStagesP1, B_ZACC = B_EMPTY1 + kStagesP1, B_ZOP = B_ZACC + 1,
                  B_FULL2 = B_ZOP + 1, B_EMPTY2 = B_FULL2 + 8, B_ACCF = B_EMPTY2 + 8, B_ACCE = B_ACCF + 2,
                  B_COUNT = B_ACCE + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + B_COUNT * 8 + 4);
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int blk = blockIdx.x / p.msplit, split = blockIdx.x % p.msplit;
    const int tok0 = blk * kBlockTokens;
    const int tile_lo = (int)(((long long)p.tiles_total * split) / p.msplit);
    const int tile_hi = (int)(((long long)p.tiles_total * (split + 1)) / p.msplit);
    const int ntiles = tile_hi - tile_lo;
    const int ktiles1 = (p.h + 63) / 64;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStagesP1; ++i) { mbar_init(bar(B_FULL1 + i), 1); mbar_init(bar(B_EMPTY1 + i), 1); }
        mbar_init(bar(B_ZACC), 1);
        mbar_init(bar(B_ZOP), kEpilogueThreads);
        for (int i = 0; i < 8; ++i) { mbar_init(bar(B_FULL2 + i), 1); mbar_init(bar(B_EMPTY2 + i), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(B_ACCF + i), 1); mbar_init(bar(B_ACCE + i), kEpilogueThreads / 2); }
        *abort_flag = 0;
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
    const uint32_t zop = ring;
    float* lse2 = reinterpret_cast<float*>(ring_ptr + kZopBytes);
    const uint32_t r2ring = ring + kZopBytes + kLseBytes;

    if (warp == 0) {
        // ===================================================================================== TMA producer
        if (lane == 0) {
            bool ok = true;
            for (int kt = 0; kt < ktiles1 && ok; ++kt) {
                const int s = kt % kStagesP1;
                if (kt >= kStagesP1) ok = mbar_wait(bar(B_EMPTY1 + s), ((kt / kStagesP1) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = ring + s * kP1StageBytes;
                mbar_expect_tx(bar(B_FULL1 + s), kP1StageBytes);
                tma_load_2d(dst, &map_x, bar(B_FULL1 + s), kt * 64, tok0);
                tma_load_2d(dst + kXTileBytes, &map_r1, bar(B_FULL1 + s), 0, kt * 64);
            }
            ok = ok && mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
            for (int it = 0; it < ntiles && ok; ++it) {
                const int s = it % kStagesP2;
                if (it >= kStagesP2) ok = mbar_wait(bar(B_EMPTY2 + s), ((it / kStagesP2) - 1) & 1, abort_flag, p.status);
                if (!ok) break;
                const uint32_t dst = r2ring + s * kR2StageBytes;
                const int e0 = (tile_lo + it) * kTileExperts;
                mbar_expect_tx(bar(B_FULL2 + s), kR2StageBytes);
                tma_load_2d(dst, &map_r2, bar(B_FULL2 + s), e0, 0);
                tma_load_2d(dst + RPAD * 128, &map_r2, bar(B_FULL2 + s), e0 + 64, 0);
            }
        }
    } else if (warp == 1) {
        // ======================================================================================= MMA issuer
        // The whole warp runs this code converged and one elected lane issues each instruction; the descriptors are
        // words computed once plus integer offsets (see tc_mma_bf16_ss_elect).
        constexpr unsigned kFull = 0xffffffffu;
        bool ok = true;
        constexpr uint32_t idesc1 = umma_idesc(64);
        // second contraction transposed: A = R2 tile (MN-major), B = z operand (K-major), 128 experts x 128 tokens
        constexpr uint32_t idesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (0u << 16) |
                                    ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        {
            const uint64_t xd = umma_desc_sw128(ring, 16, 1024), rd = umma_desc_sw128(ring + kXTileBytes, 8192, 1024);
            const uint32_t x_lo0 = (uint32_t)xd, x_hi = (uint32_t)(xd >> 32), r_lo0 = (uint32_t)rd, r_hi = (uint32_t)(rd >> 32);
            for (int kt = 0; kt < ktiles1 && ok; ++kt) {
                const int s = kt % kStagesP1;
                ok = __all_sync(kFull, mbar_wait(bar(B_FULL1 + s), (kt / kStagesP1) & 1, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t x_lo = x_lo0 + s * (kP1StageBytes >> 4), r_lo = r_lo0 + s * (kP1StageBytes >> 4);
#pragma unroll
                for (int a = 0; a < 2; ++a) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma_bf16_ss_elect(tmem_base + a * kTileExperts, x_lo + a * (16384 >> 4) + kk * 2, x_hi,
                                             r_lo + kk * (2048 >> 4), r_hi, idesc1, (kt | kk) != 0);
                }
                tc_commit_elect(bar(B_EMPTY1 + s));
            }
        }
        if (ok) tc_commit_elect(bar(B_ZACC));
        ok = __all_sync(kFull, ok && mbar_wait(bar(B_ZOP), 0, abort_flag, p.status));
        tc_fence_after();
        const uint64_t ad0 = umma_desc_sw128(r2ring, RPAD * 128, 1024), zd0 = umma_desc_sw128(zop, 16, 1024);
        const uint32_t a_lo0 = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32), z_lo0 = (uint32_t)zd0, z_hi = (uint32_t)(zd0 >> 32);
        for (int it = 0; it < ntiles && ok; ++it) {
            const int s = it % kStagesP2;
            ok = __all_sync(kFull, mbar_wait(bar(B_FULL2 + s), (it / kStagesP2) & 1, abort_flag, p.status));
            if (!ok) break;
            const uint32_t a_lo = a_lo0 + s * (kR2StageBytes >> 4);
#pragma unroll
            for (int a = 0; a < 2; ++a) {            // token half a -> TMEM columns a*128 ..
                ok = __all_sync(kFull, ok && mbar_wait(bar(B_ACCE + a), (it & 1) ^ 1, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int j = 0; j < 2 * kKSteps; ++j) {
                    const uint32_t zbyte = j * 32;                                       // K offset in [hi | lo]
                    tc_mma_bf16_ss_elect(tmem_base + a * 128, a_lo + (j % kKSteps) * (2048 >> 4), a_hi,
                                         z_lo0 + ((a * kZopOne + (zbyte >> 7) * 16384 + (zbyte & 127)) >> 4), z_hi, idesc2,
                                         j != 0);
                }
                tc_commit_elect(bar(B_ACCF + a));
            }
            if (!ok) break;
            tc_commit_elect(bar(B_EMPTY2 + s));
        }
    } else {
        // ========================================================================================= epilogue
        const int q = warp & 3;                              // TMEM lane group: token rows (phase 1), experts (phase 2)
        const int half = (warp - 2) >> 2;                    // which 128-token half
        const int row_in_half = q * 32 + lane;
        const int row_in_blk = half * 128 + row_in_half;
        const int64_t row = (int64_t)tok0 + row_in_blk;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + half * 128;
        bool ok = mbar_wait(bar(B_ZACC), 0, abort_flag, p.status);
        if (ok) {
            tc_fence_after();
            // (the phase-1 ring is free now) log2-scaled log-sum-exp of my token; +inf for rows past T, whose
            // zero-filled logits then contribute exp(-inf) = 0
            lse2[row_in_blk] = (row < p.T) ? p.lse[row] * kLog2e : INFINITY;
            uint8_t* zrow = ring_ptr + half * kZopOne + row_in_half * 128;
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
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int ch_hi = c * 2 + hf, ch_lo = RPAD / 8 + c * 2 + hf;
                    const int slab_hi = ch_hi >> 3, slab_lo = ch_lo >> 3;
                    uint4 vh = make_uint4(hi[hf * 4], hi[hf * 4 + 1], hi[hf * 4 + 2], hi[hf * 4 + 3]);
                    uint4 vl = make_uint4(lo[hf * 4], lo[hf * 4 + 1], lo[hf * 4 + 2], lo[hf * 4 + 3]);
                    *reinterpret_cast<uint4*>(zrow + slab_hi * 16384 + (((ch_hi & 7) ^ (row_in_half & 7)) << 4)) = vh;
                    *reinterpret_cast<uint4*>(zrow + slab_lo * 16384 + (((ch_lo & 7) ^ (row_in_half & 7)) << 4)) = vl;
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bar(B_ZOP));
        }
        // all 256 lse2 entries must be visible before anyone reads them in the sweep
        asm volatile("bar.sync 1, 256;" ::: "memory");

        ok = __all_sync(0xffffffffu, ok);
        const float4* lse4 = reinterpret_cast<const float4*>(lse2 + half * 128);
        for (int it = 0; it < ntiles && ok; ++it) {
            const int expert = (tile_lo + it) * kTileExperts + q * 32 + lane;     // my lane's expert in this tile
            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_ACCF + half), it & 1, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            float va[16], vb[16];
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
            auto add16 = [&](const float (&v)[16], int c16) {        // token columns c16*16 .. +15 of my half
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const float4 l = lse4[c16 * 4 + g];              // same address in every lane: a broadcast
                    acc0 += ex2f(fmaf(v[4 * g], kLog2e, -l.x));
                    acc1 += ex2f(fmaf(v[4 * g + 1], kLog2e, -l.y));
                    acc2 += ex2f(fmaf(v[4 * g + 2], kLog2e, -l.z));
                    // (one exponential in four on the FMA pipe: the special-function unit's 16 results per clock per SM
                    // are this loop's narrowest resource; more than one in four costs more issue slots than it frees)
                    acc3 += ex2_poly(fmaf(v[4 * g + 3], kLog2e, -l.w));
                }
            };
            tmem_ld16(t_lane, va);
#pragma unroll
            for (int c = 0; c < 8; c += 2) {
                tmem_ld_wait16(va);
                tmem_ld16(t_lane + (c + 1) * 16, vb);
                add16(va, c);
                tmem_ld_wait16(vb);
                if (c + 2 < 8) tmem_ld16(t_lane + (c + 2) * 16, va);
                add16(vb, c + 1);
            }
            tc_fence_before();
            mbar_arrive(bar(B_ACCE + half));
            if (expert < p.M) atomicAdd(p.psum + expert, (acc0 + acc1) + (acc2 + acc3));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <int RPAD>
int launch_psum_rpad(const CUtensorMap& mx, const CUtensorMap& m1, const CUtensorMap& m2, const PsumParams& pp, int ctas,
                     cudaStream_t st)
{
    static unsigned long long configured = 0;
    auto kern = psum_tcgen05_kernel<RPAD>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!(configured >> (dev & 63) & 1ull)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return MORE_ERR_CUDA;
        configured |= 1ull << (dev & 63);
    }
    kern<<<ctas, kThreads, kSmemBytes, st>>>(mx, m1, m2, pp);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

}  // namespace

int launch_psum_tcgen05(const __nv_bfloat16* X, const __nv_bfloat16* R1, const __nv_bfloat16* R2, int T, int h, int r,
                        int M, const float* lse, float* psum, DeviceCtx& ctx, cudaStream_t stream)
{
    CUtensorMap mx, m1, m2;
    const int rpad = (r <= 16) ? 16 : (r <= 32 ? 32 : 64);
    int rc = get_tensor_map(X, T, h, kBlockTokens, 64, &mx);
    if (rc == MORE_OK) rc = get_tensor_map(R1, h, r, 64, 64, &m1);
    if (rc == MORE_OK) rc = get_tensor_map(R2, r, M, rpad, 64, &m2);
    if (rc != MORE_OK) return rc;
    PsumParams pp;
    pp.T = T; pp.h = h; pp.r = r; pp.M = M;
    pp.tiles_total = (M + kTileExperts - 1) / kTileExperts;
    pp.lse = lse; pp.psum = psum; pp.status = ctx.status;
    const int blocks = (T + kBlockTokens - 1) / kBlockTokens;
    const int slots = 2 * (ctx.sm_count > 0 ? ctx.sm_count : 148);
    int s = slots / blocks;                       // fill one wave of resident CTAs; each keeps >= 4 expert tiles
    if (s > pp.tiles_total / 4) s = pp.tiles_total / 4;
    if (s < 1) s = 1;
    if (s > 64) s = 64;
    pp.msplit = s;
    switch (rpad) {
        case 16: return launch_psum_rpad<16>(mx, m1, m2, pp, blocks * s, stream);
        case 32: return launch_psum_rpad<32>(mx, m1, m2, pp, blocks * s, stream);
        default: return launch_psum_rpad<64>(mx, m1, m2, pp, blocks * s, stream);
    }
}

}  // namespace more
