// PTX wrappers, UMMA descriptors and pipeline constants shared by the sm_100a kernels of this library
// (the router and the softmax column-sum kernel).  Internal; every translation unit gets its own copy.
#pragma once

#include <cuda.h>   // CUtensorMap and the driver entry-point typedef only; libcuda is resolved at run time
#include <cuda_runtime.h>
#include <limits.h>
#include <math.h>
#include <stdint.h>

#include "more_internal.h"

namespace more {

namespace {

constexpr int kThreads = 320;                      // warps 0, 1: TMA / MMA; warps 2..9: epilogue
constexpr int kEpilogueThreads = 256;              // one thread per token of the block
constexpr int kStagesP1 = 2;                       // phase-1 ring: 32 KB of X + 8 KB of R1 per stage
constexpr int kXTileBytes = kBlockTokens * 128;    // 256 tokens x 64 bf16
constexpr int kR1TileBytes = 64 * 128;             // 64 K-rows x 64 bf16 (columns >= r are zero-filled by TMA)
constexpr int kP1StageBytes = kXTileBytes + kR1TileBytes;
constexpr int kRingBytes = 110 * 1024;             // phase 1: the two stages; phase 2: A operands, candidates, R2 stages
static_assert(kStagesP1 * kP1StageBytes <= kRingBytes, "phase-1 ring does not fit");
constexpr int kSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 1024 /*barriers, flags*/;
constexpr int kTmemCols = 256;                     // tensor-memory columns per CTA (two CTAs share the 512 of an SM)
constexpr long long kWaitBudgetCycles = 4000000000LL;   // ~2 s
#ifndef MORE_SUSPEND_NS
#define MORE_SUSPEND_NS 20000
#endif
constexpr uint32_t kSuspendHintNs = MORE_SUSPEND_NS;             // a waiting thread may be parked this long per try

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"   // may suspend up to the hinted time
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok;
}

// Non-blocking test of a phase.
__device__ __forceinline__ uint32_t mbar_try_wait_now(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out of budget).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long budget = kWaitBudgetCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 15u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > budget) {
                *abort_flag = 1;
                atomicExch(status, MORE_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Same, with the A operand read from tensor memory: lane = row of A, each 32-bit column holds two consecutive
// bf16 K-elements (the lower index in the lower half), so one K = 16 step spans 8 columns.
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Warp-converged issue: all 32 lanes of the issuing warp execute these; elect.sync picks the one lane (the same on
// every call) that issues the instruction.  Keeping the warp converged and passing the shared-memory descriptors as
// two 32-bit words (low word = start address, advanced with one integer add per K step) keeps the issuing code short
// enough that it does not limit the tensor pipe: with descriptors rebuilt per instruction inside a one-lane branch
// the issue alone took 50-80 clocks per instruction, more than the 32 clocks a 128 x 64 x 16 MMA computes for.
__device__ __forceinline__ void tc_mma_bf16_ts_elect(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                                     uint32_t idesc, bool accumulate)
{
    if (accumulate)
        asm volatile(
            "{\n\t.reg .pred p, pe;\n\t.reg .b64 bd;\n\t"
            "setp.eq.u32 p, 0, 0;\n\tmov.b64 bd, {%2, %3};\n\telect.sync _|pe, 0xffffffff;\n\t"
            "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p, pe;\n\t.reg .b64 bd;\n\t"
            "setp.ne.u32 p, 0, 0;\n\tmov.b64 bd, {%2, %3};\n\telect.sync _|pe, 0xffffffff;\n\t"
            "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_ss_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                     uint32_t b_hi, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t.reg .b64 ad, bd;\n\t"
        "setp.ne.b32 p, %6, 0;\n\tmov.b64 ad, {%1, %2};\n\tmov.b64 bd, {%3, %4};\n\telect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_elect(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}

// 2^x for x <= 0 without the special-function unit: x = n + f with n = round(x) (the 1.5 * 2^23 trick leaves n in
// the low mantissa bits of t), 2^f by a degree-4 polynomial on [-0.5, 0.5] (relative error < 5e-5), and the exponent
// added as an integer.  Seven of its nine instructions run on the FMA pipe.
__device__ __forceinline__ float ex2_poly(float x)
{
    x = fmaxf(x, -125.f);
    const float t = x + 12582912.f;
    const float f = x - (t - 12582912.f);
    float p = 0.00961813f;
    p = fmaf(p, f, 0.0555041f);
    p = fmaf(p, f, 0.240227f);
    p = fmaf(p, f, 0.693147f);
    p = fmaf(p, f, 1.0f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// Store 8 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&u)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t* u = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
          "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
        : "r"(taddr)
        : "memory");
}
// Wait for outstanding TMEM loads and tie the 16 destination registers to the wait, so that no use of them can be
// scheduled ahead of it.
__device__ __forceinline__ void tmem_ld_wait16(float (&v)[16])
{
    uint32_t* u = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]),
                   "+r"(u[8]), "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15])
                 :
                 : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 4 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&u)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait4(uint32_t (&u)[4])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]) : : "memory");
}

// One arrival for the whole (converged) warp: the lanes' own tensor-memory accesses have completed (wait::ld /
// wait::st are warp-wide), the warp synchronises, lane 0 arrives.  The barrier counts warps, not threads.
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

// ------------------------------------------------------------------------------------------- UMMA descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
//   K-major operand  (rows = M/N index, 128-byte rows of 64 bf16 along K): SBO = 1024 B between 8-row groups.
//   MN-major operand (rows = K index, 128-byte rows of 64 bf16 along M/N): SBO = 1024 B between 8-K-row groups,
//                     LBO = distance between successive 64-element column blocks.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;     // descriptor version
    d |= (uint64_t)2 << 61;     // SWIZZLE_128B
    return d;
}
// Instruction descriptor: D = fp32, A = B = bf16, A K-major, B MN-major, M = 128, given N.
__host__ __device__ constexpr uint32_t umma_idesc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}
// The same with A = B = fp16 (format code 0).
__host__ __device__ constexpr uint32_t umma_idesc_f16(int n)
{
    return (1u << 4) | (0u << 7) | (0u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}

// All MMAs of one accumulator buffer in a single instruction sequence: D[128 x N] = sum over NM K-steps of
// A (tensor memory, 8 columns per K = 16 step) x B (shared memory, MN-major, 16 K-rows = 2048 bytes per step; the B
// offset wraps after KS steps, which is how a [hi | lo] operand pair reuses the same B rows).  The warp executes it
// converged; one elected lane issues.  b_lo / b_hi are the two words of the B descriptor.
#define MORE_MMA_STEP(AOFF, BOFF, PRED)                                                              \
    "add.u32 a, %1, " #AOFF ";\n\tadd.u32 bl, %2, " #BOFF ";\n\tmov.b64 bd, {bl, %3};\n\t"        \
    "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %4, " #PRED ";\n\t"
#define MORE_MMA_OPEN                                                                                \
    "{\n\t.reg .pred pe, pt, pf;\n\t.reg .b64 bd;\n\t.reg .b32 a, bl;\n\t"                        \
    "setp.eq.u32 pt, 0, 0;\n\tsetp.ne.u32 pf, 0, 0;\n\telect.sync _|pe, 0xffffffff;\n\t"
template <int NM, int KS>
__device__ __forceinline__ void tc_mma_buffer_ts(uint32_t d, uint32_t a0, uint32_t b_lo, uint32_t b_hi, uint32_t idesc)
{
    static_assert((NM == 1 && KS == 1) || (NM == 2 && (KS == 1 || KS == 2)) || (NM == 4 && (KS == 2 || KS == 4)) ||
                  (NM == 8 && KS == 4), "unsupported MMA sequence");
    if constexpr (NM == 1)
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) "}" ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else if constexpr (NM == 2 && KS == 2)
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) MORE_MMA_STEP(8, 128, pt) "}"
                     ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else if constexpr (NM == 2 && KS == 1)
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) MORE_MMA_STEP(8, 0, pt) "}"
                     ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else if constexpr (NM == 4 && KS == 4)
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) MORE_MMA_STEP(8, 128, pt) MORE_MMA_STEP(16, 256, pt)
                     MORE_MMA_STEP(24, 384, pt) "}" ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else if constexpr (NM == 4 && KS == 2)
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) MORE_MMA_STEP(8, 128, pt) MORE_MMA_STEP(16, 0, pt)
                     MORE_MMA_STEP(24, 128, pt) "}" ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else
        asm volatile(MORE_MMA_OPEN MORE_MMA_STEP(0, 0, pf) MORE_MMA_STEP(8, 128, pt) MORE_MMA_STEP(16, 256, pt)
                     MORE_MMA_STEP(24, 384, pt) MORE_MMA_STEP(32, 0, pt) MORE_MMA_STEP(40, 128, pt)
                     MORE_MMA_STEP(48, 256, pt) MORE_MMA_STEP(56, 384, pt) "}"
                     ::"r"(d), "r"(a0), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
}
#undef MORE_MMA_STEP
#undef MORE_MMA_OPEN

// The same with the A operand in shared memory (K-major, 32 bytes per K = 16 step): a_lo / a_hi are the two words of
// the A descriptor of the first step.  NM = 2 K-steps wrapping after 1, or 4 wrapping after 2.
#define MORE_MMA_STEP_SS(AOFF, BOFF, PRED)                                                           \
    "add.u32 al, %1, " #AOFF ";\n\tmov.b64 ad, {al, %2};\n\tadd.u32 bl, %3, " #BOFF ";\n\tmov.b64 bd, {bl, %4};\n\t" \
    "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, " #PRED ";\n\t"
#define MORE_MMA_OPEN_SS                                                                             \
    "{\n\t.reg .pred pe, pt, pf;\n\t.reg .b64 ad, bd;\n\t.reg .b32 al, bl;\n\t"                  \
    "setp.eq.u32 pt, 0, 0;\n\tsetp.ne.u32 pf, 0, 0;\n\telect.sync _|pe, 0xffffffff;\n\t"
template <int NM, int KS>
__device__ __forceinline__ void tc_mma_buffer_ss(uint32_t d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                 uint32_t idesc)
{
    static_assert((NM == 2 && KS == 1) || (NM == 4 && KS == 2), "unsupported MMA sequence");
    if constexpr (NM == 2)
        asm volatile(MORE_MMA_OPEN_SS MORE_MMA_STEP_SS(0, 0, pf) MORE_MMA_STEP_SS(2, 0, pt) "}"
                     ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    else
        asm volatile(MORE_MMA_OPEN_SS MORE_MMA_STEP_SS(0, 0, pf) MORE_MMA_STEP_SS(2, 128, pt) MORE_MMA_STEP_SS(4, 0, pt)
                     MORE_MMA_STEP_SS(6, 128, pt) "}"
                     ::"r"(d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
}
#undef MORE_MMA_STEP_SS
#undef MORE_MMA_OPEN_SS

}  // namespace

// 2-D bf16 row-major tensor [rows][cols] -> TMA descriptor with box = box_cols x box_rows, 128-byte swizzle, zero
// fill out of bounds.  Descriptors are cached (host side, guarded by the API mutex).
int get_tensor_map(const void* ptr, int rows, int cols, int box_rows, int box_cols, CUtensorMap* out);

}  // namespace more
