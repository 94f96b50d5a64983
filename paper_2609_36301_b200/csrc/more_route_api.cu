// Host side of libmore_route.so: argument checks, per-device state, launch planning, the extern "C" entry points.
#include "more_internal.h"
#include "more_debug.h"
#include "sm100_common.cuh"

#include <atomic>
#include <mutex>
#include <new>
#include <stdio.h>
#include <stdlib.h>

namespace more {

namespace {

std::mutex g_mutex;
std::atomic<long long> g_launches{0};
constexpr int kMaxDevices = 64;
DeviceCtx g_ctx[kMaxDevices];

int get_ctx(DeviceCtx** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MORE_ERR_CUDA;
    DeviceCtx& c = g_ctx[dev];
    if (c.dev != dev) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MORE_ERR_CUDA;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MORE_ERR_CUDA;
        c.cc_major = major;
        c.sm_count = sms;
        if (major != 10) return MORE_ERR_ARCH;
        void* blk = nullptr;                   // status word, the filter's two words, 16 diagnostic counters
        if (cudaMalloc(&blk, 256) != cudaSuccess) return MORE_ERR_CUDA;
        if (cudaMemset(blk, 0, 256) != cudaSuccess) return MORE_ERR_CUDA;
        c.status = static_cast<int*>(blk);
        c.colnorm = reinterpret_cast<float*>(static_cast<char*>(blk) + 64);
        c.prep_arrivals = reinterpret_cast<unsigned*>(static_cast<char*>(blk) + 72);
        c.stats = reinterpret_cast<unsigned long long*>(static_cast<char*>(blk) + 128);
        c.dev = dev;
    }
    if (c.cc_major != 10) return MORE_ERR_ARCH;
    *out = &c;
    return MORE_OK;
}

int ensure_bytes(void** buf, size_t* have, size_t need)
{
    if (need <= *have) return MORE_OK;
    if (*buf) {
        if (cudaDeviceSynchronize() != cudaSuccess) return MORE_ERR_CUDA;   // nothing may still be using it
        cudaFree(*buf);
        *buf = nullptr;
        *have = 0;
    }
    size_t bytes = (need + ((size_t)1 << 20) - 1) & ~(((size_t)1 << 20) - 1);
    if (cudaMalloc(buf, bytes) != cudaSuccess) { cudaGetLastError(); return MORE_ERR_CUDA; }
    *have = bytes;
    return MORE_OK;
}

// The scratch allocation always has room for a guard region behind the bytes a plan needs: kGuardBytes of a fixed
// pattern, written on the caller's stream ahead of the kernels, so that a kernel running past its scratch is caught
// by more_debug_scratch_guard instead of corrupting whatever lies behind.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardPattern = 0x5a;

int ensure_scratch(DeviceCtx* ctx, size_t need, cudaStream_t st)
{
    const size_t used = (need + 255) & ~(size_t)255;
    void* const before = ctx->scratch;
    int rc = ensure_bytes(&ctx->scratch, &ctx->scratch_bytes, used + kGuardBytes);
    if (rc != MORE_OK) return rc;
    if (ctx->scratch != before || used != ctx->scratch_used) {       // (the pattern stays put between calls otherwise)
        ctx->scratch_used = used;
        if (cudaMemsetAsync(static_cast<char*>(ctx->scratch) + used, kGuardPattern, kGuardBytes, st) != cudaSuccess)
            return MORE_ERR_CUDA;
    }
    return MORE_OK;
}

__global__ void expire_wait_kernel(long long budget, int* status)
{
    __shared__ uint64_t bar_storage;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // nobody arrives: the wait gives up after `budget` clocks, records the time-out and returns false
    (void)mbar_wait(bar, 0, &abort_flag, status, budget);
}

int check_shape(int T, int h, int r, int M, int k, int gate_mode, int path)
{
    if (gate_mode != MORE_GATE_TOPK_SOFTMAX && gate_mode != MORE_GATE_FULL_SOFTMAX) return MORE_ERR_MODE;
    if (path != MORE_PATH_AUTO && path != MORE_PATH_GENERIC && path != MORE_PATH_TCGEN05) return MORE_ERR_MODE;
    if (T < 0 || h < 1 || r < 1 || M < 1 || k < 1 || k > M || k > MORE_K_MAX || r > MORE_R_MAX) return MORE_ERR_SHAPE;
    if (M > MORE_M_MAX) return MORE_ERR_SHAPE;             // expert ids and column counters are 32-bit in the kernels
    return MORE_OK;
}

bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// The body of every routing entry point.  The caller holds g_mutex.
int route_device_locked(const RouteArgs& a, int path, int msplit)
{
    int rc = check_shape(a.T, a.h, a.r, a.M, a.k, a.gate_mode, path);
    if (rc != MORE_OK) return rc;
    if (!a.out_counts) return MORE_ERR_NULL;
    if (a.T > 0 && (!a.X || (!a.R1 && !a.full) || !a.R2 || !a.out_idx || !a.out_gate)) return MORE_ERR_NULL;
    if (!aligned(a.X, 16) || !aligned(a.R1, 16) || !aligned(a.R2, 16)) return MORE_ERR_ALIGN;
    if (!aligned(a.out_idx, 4) || !aligned(a.out_gate, 4) || !aligned(a.out_counts, 4) || !aligned(a.out_topval, 4) ||
        !aligned(a.out_lse, 4))
        return MORE_ERR_ALIGN;

    DeviceCtx* ctx = nullptr;
    rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    Plan plan;
    const bool want_lse = a.gate_mode == MORE_GATE_FULL_SOFTMAX || a.out_lse != nullptr;
    {
        // The planner walks a few thousand candidates for a decode-sized shape (tens of microseconds, comparable with
        // the kernel it plans); repeated calls with the same shape take the plan from a small cache.  Guarded by the
        // API mutex like everything here.
        struct PlanKey {
            int T, h, r, M, k, gate_mode, want_lse, full, path, msplit, sm_count;
            bool operator==(const PlanKey& o) const
            {
                return T == o.T && h == o.h && r == o.r && M == o.M && k == o.k && gate_mode == o.gate_mode &&
                       want_lse == o.want_lse && full == o.full && path == o.path && msplit == o.msplit && sm_count == o.sm_count;
            }
        };
        constexpr int kPlanCache = 16;
        static PlanKey keys[kPlanCache];
        static Plan plans[kPlanCache];
        static int used = 0, next = 0;
        const PlanKey key{a.T, a.h, a.r, a.M, a.k, a.gate_mode, want_lse ? 1 : 0, a.full ? 1 : 0, path, msplit, ctx->sm_count};
        int hit = -1;
        for (int i = 0; i < used; ++i)
            if (keys[i] == key) { hit = i; break; }
#ifdef MORE_DEV
        hit = -1;                                  // development builds re-plan every call (MORE_PLAN / MORE_KERNEL overrides)
#endif
        if (hit >= 0) {
            plan = plans[hit];
        } else {
            rc = make_plan(a.T, a.h, a.r, a.M, a.k, a.gate_mode, want_lse, a.full, path, msplit, ctx->sm_count, &plan);
            if (rc != MORE_OK) return rc;
            keys[next] = key;
            plans[next] = plan;
            next = (next + 1) % kPlanCache;
            if (used < kPlanCache) ++used;
        }
    }
    const size_t need = plan.path != MORE_PATH_TCGEN05
                            ? generic_scratch_bytes(a)
                            : (a.full ? full_scratch_bytes(a, plan)
                                      : (plan.paired ? paired_scratch_bytes(a, plan) : lowrank_scratch_bytes(a, plan)));
    rc = ensure_scratch(ctx, need, a.stream);
    if (rc != MORE_OK) return rc;
    if (a.T == 0 || plan.path != MORE_PATH_TCGEN05) {
        // (the tensor-core launchers clear out_counts themselves, after their last step that can fail)
        if (cudaMemsetAsync(a.out_counts, 0, (size_t)a.M * sizeof(int32_t), a.stream) != cudaSuccess) return MORE_ERR_CUDA;
        if (a.T == 0) return MORE_OK;
        return launch_generic(a, *ctx, ctx->scratch);
    }
    if (a.full) return launch_full(a, *ctx, plan, ctx->scratch);
    return plan.paired ? launch_paired(a, *ctx, plan, ctx->scratch) : launch_lowrank(a, *ctx, plan, ctx->scratch);
}

int route_device(const RouteArgs& a, int path, int msplit)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    return route_device_locked(a, path, msplit);
}

}  // namespace

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

namespace {

// Launch plan of the paired low-rank kernel (256-token CTAs, two per SM).
void plan_paired(int T, int h, int M, int msplit, int sm_count, Plan* p)
{
    const int slots = 2 * sm_count;                       // two CTAs are resident per SM
    const int tiles = (M + kTileExperts - 1) / kTileExperts;
    double best = 1e300;
    int best_bt = kBlockTokens, best_s = 1;
    for (int bt = kBlockTokens; bt >= 128; bt -= 32) {
        const int blocks = (T + bt - 1) / bt;
        int s = msplit;
        if (s == 0) {
            s = slots / blocks;
            if (s > tiles / 8) s = tiles / 8;
            if ((long long)blocks * s > sm_count) {
                int dense = s < tiles / 16 ? s : tiles / 16;
                const int one_per_sm = sm_count / blocks;
                s = dense > one_per_sm ? dense : one_per_sm;
                if (s > tiles / 8) s = tiles / 8;
            }
            if (s < 1) s = 1;
            if (s > 64) s = 64;
        }
        if (s > tiles) s = tiles;
        const long long ctas = (long long)blocks * s;
        const double per_sm = (double)((ctas + sm_count - 1) / sm_count);
        const double per_cta = 256.0 * (h / 8.0) + (double)bt * ((double)tiles / s) * 16.0 + 256.0 * 256.0;
        const double cost = per_sm * per_cta;
        if (cost < best * 0.999) { best = cost; best_bt = bt; best_s = s; }
    }
    p->block_tokens = best_bt;
    p->msplit = best_s;
    p->ctas = ((T + best_bt - 1) / best_bt) * best_s;
}

// Launch plan of the fused standard router: one CTA per SM, 256-expert steps that each run over all h/64 k-tiles.  A
// step costs the same whatever the block's fill (the MMAs are 128 tokens tall regardless), so what counts is waves x
// steps per CTA; splitting the experts over a few CTAs per token block evens out the last wave.
void plan_dense(int T, int h, int M, int msplit, int sm_count, Plan* p)
{
    const int tiles = (M + 255) / 256;
    const double ktiles = (h + 63) / 64;
    double best = 1e300;
    int best_bt = kBlockTokens, best_s = 1;
    for (int bt = kBlockTokens; bt >= 128; bt -= 32) {
        const int blocks = (T + bt - 1) / bt;
        const int s_lo = msplit > 0 ? (msplit < tiles ? msplit : tiles) : 1;
        const int s_hi = msplit > 0 ? s_lo : (tiles < 16 ? tiles : 16);
        for (int s = s_lo; s <= s_hi; ++s) {
            const long long ctas = (long long)blocks * s;
            const double waves = (double)((ctas + sm_count - 1) / sm_count);
            const double steps = (double)((tiles + s - 1) / s);
            // microseconds, fitted to B200 measurements: 1.2 per k-tile of a step (the L2 -> SM traffic of the
            // stages), 2.1 for its epilogue, 8 per CTA for start and pipeline fill, 25 more when the lists are
            // parked and merged
            double cost = waves * (steps * (1.2 * ktiles + 2.1) + 8.0 + (s > 1 ? 25.0 : 0.0));
            cost *= 1.0 + 0.02 * (kBlockTokens - bt) / 32.0;          // prefer full blocks on a tie
            if (cost < best * 0.999) { best = cost; best_bt = bt; best_s = s; }
        }
    }
    p->block_tokens = best_bt;
    p->msplit = best_s;
    p->ctas = ((T + best_bt - 1) / best_bt) * best_s;
}

// Launch plan of the low-rank router: one CTA per SM with four 128-lane groups, laid out as tg token groups x es expert
// ranges; msplit CTAs per token block.  A rough cycle model picks among the candidates: a sweep's time per 16-column
// chunk is the larger of one warp's latency chain and the issue slots of the warps that share a scheduler, every sweep
// pays a start-up (nearly every early logit is a candidate), the projection is bounded by the SM's share of HBM
// bandwidth, and a second wave of CTAs costs a whole CTA time.  Measured on B200 the candidates of a small shape lie
// within ~10 % of each other; what the model must avoid are the outliers (a lone warp sweeping thousands of experts,
// dozens of partial lists for hundreds of tokens).
void plan_lowrank(int T, int h, int r, int M, int k, bool want_lse, int msplit, int sm_count, Plan* p)
{
    const int blocks64 = (M + 63) / 64;
    const int rpad = r <= 16 ? 16 : (r <= 32 ? 32 : 64);
    // The filter mode (sweep on an fp16 rounding of z, exact rescoring of the survivors) is correct but not faster on any
    // measured shape; it is compiled and planned only in -DMORE_WITH_FILTER builds, which exist to reproduce that.
#ifdef MORE_WITH_FILTER
    const bool filter_ok = !want_lse && k <= 16 && M >= 4096;
#else
    const bool filter_ok = false;
#endif
    const double c_lat = want_lse ? 260.0 : 190.0, c_iss = want_lse ? 76.0 : 56.0;
    double best = 1e300;
    Plan bp = *p;
    for (int bt = 512; bt >= 32; bt -= 32) {
        const int blocks = (T + bt - 1) / bt;
        const int tg = (bt + 127) / 128;
        for (int es = 1; es * tg <= 4; es *= 2) {
            if (blocks64 < es) continue;                       // a range is at least one 64-expert block
            int n1, b1, n2, b2, off;
            if (!lowrank_smem_plan(rpad, tg, es, filter_ok, &n1, &b1, &n2, &b2, &off)) continue;
            int s_lo = 1, s_hi = 1;
            if (msplit > 0) {
                s_lo = s_hi = msplit < blocks64 / es ? msplit : (blocks64 / es > 0 ? blocks64 / es : 1);   // at most one CTA per 64-expert block
            } else {
                s_hi = sm_count / blocks;                      // never more CTAs than one wave
                if (s_hi > blocks64 / es) s_hi = blocks64 / es;
                if (s_hi > 64) s_hi = 64;
                if (s_hi < 1) s_hi = 1;
            }
            for (int s = s_lo; s <= s_hi; ++s) {
                if ((long long)s * es > blocks64) continue;
                const long long ctas = (long long)blocks * s;
                const double waves = (double)((ctas + sm_count - 1) / sm_count);
                // a sweep starts with an empty list, so nearly every early logit is a candidate: worth ~160 chunks on a
                // long range, about ten times its own length on a short one
                const double range_chunks = 4.0 * ((blocks64 + es * s - 1) / (es * s));     // whole 64-expert steps
                // (the expert ranges of a CTA share their thresholds, so together they pay one start, not es)
                const double all_chunks = range_chunks * es;
                const double chunks = range_chunks + (all_chunks < 16.0 ? 10.0 * all_chunks : 160.0) / es;
                // warps per scheduler: one per group, except that a block of at most 64 tokens is spread over the
                // lane quarters, one or two quarters per expert range (credited only to small problems: on long
                // sweeps the latency term of this model is too optimistic for two warps per scheduler)
                double groups = (double)tg * es;
                if (tg == 1 && bt <= 64 && es >= 2 && blocks * 8 <= sm_count) groups = bt <= 32 ? 1.0 : (es == 4 ? 2.0 : 1.0);
                const double per_chunk = c_lat > groups * c_iss ? c_lat : groups * c_iss;
                const double ktile = bt * 128.0 / 23.0 > 300.0 ? bt * 128.0 / 23.0 : 300.0;
                double t = 9000.0 + ((h + 63) / 64) * ktile + chunks * per_chunk;
                if (es > 1) t += 1500.0;
                if (s > 1) t += 7000.0 + 30.0 * s + 0.75 * s * bt;     // park, last arriver, its merge of s lists per token
                const double cost = waves * t;
                if (cost < best * 0.999) {
                    best = cost;
                    bp.block_tokens = bt; bp.tg = tg; bp.es = es; bp.msplit = s; bp.ctas = (int)ctas;
                }
            }
        }
    }
    *p = bp;
    p->filter = filter_ok;
}

}  // namespace

int make_plan(int T, int h, int r, int M, int k, int gate_mode, bool want_lse, bool full, int path, int msplit,
              int sm_count, Plan* out)
{
    (void)gate_mode;
    const bool fast_ok = tcgen05_shape_ok(T, h, r, M, k);
    if (path == MORE_PATH_TCGEN05 && !fast_ok) return MORE_ERR_SHAPE;
    if (msplit < 0 || msplit > 64) return MORE_ERR_SHAPE;
    Plan p;
    p.rpad = (r + 15) / 16 * 16;
    if (path == MORE_PATH_GENERIC || !fast_ok) {
        p.path = MORE_PATH_GENERIC;
        p.block_tokens = 8;
        p.msplit = 1;
        p.ctas = (T + 7) / 8;
        *out = p;
        return MORE_OK;
    }
    p.path = MORE_PATH_TCGEN05;
    if (sm_count <= 0) sm_count = 148;
    if (full) {
        plan_dense(T, h, M, msplit, sm_count, &p);
    } else {
        // Two kernels serve the low-rank router.  Measured on B200 over T = 2 k ... 64 k tokens, M = 1 k ... 64 k
        // experts, r = 16, 32, 64 and both gates: the grouped kernel (one CTA per SM, up to four token groups / expert
        // ranges side by side) wins while an SM has fewer than ~120 tokens; between that and ~260 tokens per SM it
        // wins for up to ~8 k experts, and with the softmax sweep (whose epilogue is bound by its own instructions
        // rather than by the accumulator hand-over) up to ~250 tokens per SM for any expert count when its 128-token
        // groups fill evenly; the paired kernel
        // (256-token CTAs, two per SM, 64-expert steps, two accumulators per group at r <= 32) wins on the rest.
        p.block_tokens = 0;
        const long long per_sm = ((long long)T + sm_count - 1) / sm_count;
        // (a CTA of the grouped kernel holds its tokens in groups of 128: with, say, 167 tokens per SM the second
        // group of every CTA is two thirds empty, and the kernel loses what it otherwise gains)
        const bool even_fill = per_sm % 128 == 0 || per_sm % 128 >= 80;
        bool grouped;
        if (per_sm < 120) grouped = true;
        else if (M <= 8192) grouped = per_sm < (want_lse ? 320 : 260);
        else grouped = (want_lse || M <= 16384) && per_sm < 250 && even_fill;      // (M = 16 k with the top-k gate: a tie)
#ifdef MORE_DEV
        if (const char* kk = getenv("MORE_KERNEL")) grouped = kk[0] == 'g';
#endif
        if (grouped) {
            plan_lowrank(T, h, r, M, k, want_lse, msplit, sm_count, &p);
        } else {
            plan_paired(T, h, M, msplit, sm_count, &p);
            p.paired = true;
        }
        if (p.block_tokens == 0) return MORE_ERR_SHAPE;
#ifdef MORE_DEV
        // development builds only: MORE_PLAN="block_tokens,es,msplit,filter[,paired]" overrides the planner
        if (const char* e = getenv("MORE_PLAN")) {
            int bt = 0, es = 0, s = 0, f = 0, pr = 0;
            if (sscanf(e, "%d,%d,%d,%d,%d", &bt, &es, &s, &f, &pr) >= 4) {
                p.block_tokens = bt; p.tg = (bt + 127) / 128; p.es = es; p.msplit = s;
                p.filter = f != 0 && !want_lse && k <= 16;
                p.paired = pr != 0;
                p.ctas = ((T + bt - 1) / bt) * s;
            }
        }
#endif
    }
    *out = p;
    return MORE_OK;
}

}  // namespace more

using namespace more;

extern "C" {

int more_route_ex(const void* X, const void* R1, const void* R2, int T, int h, int r, int M, int k, int gate_mode,
                  int32_t* out_idx, float* out_gate, int32_t* out_counts, float* out_topval, float* out_lse, int path,
                  int msplit, void* stream)
{
    RouteArgs a;
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.R1 = static_cast<const __nv_bfloat16*>(R1);
    a.R2 = static_cast<const __nv_bfloat16*>(R2);
    a.T = T; a.h = h; a.r = r; a.M = M; a.k = k; a.gate_mode = gate_mode;
    a.out_idx = out_idx; a.out_gate = out_gate; a.out_counts = out_counts;
    a.out_topval = out_topval; a.out_lse = out_lse;
    a.stream = static_cast<cudaStream_t>(stream);
    return route_device(a, path, msplit);
}

int more_route_full(const void* X, const void* W, int T, int h, int M, int k, int gate_mode, int32_t* out_idx,
                    float* out_gate, int32_t* out_counts, float* out_topval, float* out_lse, int msplit, void* stream)
{
    // the standard router has only the tensor-core path: say so instead of silently doing something else
    if (h < 1 || M < 1 || h % 8 != 0 || M % 8 != 0) return MORE_ERR_SHAPE;
    RouteArgs a;
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.R1 = nullptr;
    a.R2 = static_cast<const __nv_bfloat16*>(W);
    a.T = T; a.h = h; a.r = 64; a.M = M; a.k = k; a.gate_mode = gate_mode;   // r: the plan's cost model only
    a.out_idx = out_idx; a.out_gate = out_gate; a.out_counts = out_counts;
    a.out_topval = out_topval; a.out_lse = out_lse;
    a.stream = static_cast<cudaStream_t>(stream);
    a.full = true;
    return route_device(a, MORE_PATH_TCGEN05, msplit);
}

int more_route(const void* X, const void* R1, const void* R2, int T, int h, int r, int M, int k, int gate_mode,
               int32_t* out_idx, float* out_gate, int32_t* out_counts, void* stream)
{
    return more_route_ex(X, R1, R2, T, h, r, M, k, gate_mode, out_idx, out_gate, out_counts, nullptr, nullptr,
                         MORE_PATH_AUTO, 0, stream);
}

int more_route_host(const void* Xh, const void* R1h, const void* R2h, int T, int h, int r, int M, int k, int gate_mode,
                    int32_t* idx_h, float* gate_h, int32_t* counts_h, void* stream)
{
    int rc = check_shape(T, h, r, M, k, gate_mode, MORE_PATH_AUTO);
    if (rc != MORE_OK) return rc;
    if (!counts_h) return MORE_ERR_NULL;
    if (T > 0 && (!Xh || !R1h || !R2h || !idx_h || !gate_h)) return MORE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t bX = up((size_t)T * h * 2), bR1 = up((size_t)h * r * 2), bR2 = up((size_t)r * M * 2);
    const size_t bI = up((size_t)T * k * 4), bG = up((size_t)T * k * 4), bC = up((size_t)M * 4);
    // The staging buffer is shared by every call on the device and may be reallocated by a larger one, so the mutex
    // is held until this call's copies and kernels have finished with it (the call synchronises the stream anyway).
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    rc = ensure_bytes(&ctx->staging, &ctx->staging_bytes, bX + bR1 + bR2 + bI + bG + bC);
    if (rc != MORE_OK) return rc;
    char* base = static_cast<char*>(ctx->staging);
    char* dX = base; char* dR1 = dX + bX; char* dR2 = dR1 + bR1;
    char* dI = dR2 + bR2; char* dG = dI + bI; char* dC = dG + bG;
    bool ok = true;
    if (T > 0) {
        ok = ok && cudaMemcpyAsync(dX, Xh, (size_t)T * h * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(dR1, R1h, (size_t)h * r * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(dR2, R2h, (size_t)r * M * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
    }
    if (!ok) return MORE_ERR_CUDA;
    RouteArgs a;
    a.X = reinterpret_cast<const __nv_bfloat16*>(dX);
    a.R1 = reinterpret_cast<const __nv_bfloat16*>(dR1);
    a.R2 = reinterpret_cast<const __nv_bfloat16*>(dR2);
    a.T = T; a.h = h; a.r = r; a.M = M; a.k = k; a.gate_mode = gate_mode;
    a.out_idx = reinterpret_cast<int32_t*>(dI); a.out_gate = reinterpret_cast<float*>(dG);
    a.out_counts = reinterpret_cast<int32_t*>(dC);
    a.out_topval = nullptr; a.out_lse = nullptr;
    a.stream = st;
    rc = route_device_locked(a, MORE_PATH_AUTO, 0);
    if (rc != MORE_OK) return rc;
    if (T > 0) {
        ok = ok && cudaMemcpyAsync(idx_h, dI, (size_t)T * k * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(gate_h, dG, (size_t)T * k * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    }
    ok = ok && cudaMemcpyAsync(counts_h, dC, (size_t)M * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    return ok ? MORE_OK : MORE_ERR_CUDA;
}

int more_route_psum(const void* X, const void* R1, const void* R2, int T, int h, int r, int M, const float* lse,
                    float* out_psum, int path, void* stream)
{
    if (path != MORE_PATH_AUTO && path != MORE_PATH_GENERIC && path != MORE_PATH_TCGEN05) return MORE_ERR_MODE;
    if (T < 0 || h < 1 || r < 1 || M < 1 || r > MORE_R_MAX) return MORE_ERR_SHAPE;
    if (!out_psum) return MORE_ERR_NULL;
    if (T > 0 && (!X || !R1 || !R2 || !lse)) return MORE_ERR_NULL;
    if (!aligned(X, 16) || !aligned(R1, 16) || !aligned(R2, 16) || !aligned(lse, 4) || !aligned(out_psum, 4))
        return MORE_ERR_ALIGN;
    const bool fast_ok = tcgen05_shape_ok(T, h, r, M, 1);
    if (path == MORE_PATH_TCGEN05 && !fast_ok) return MORE_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool fast = fast_ok && path != MORE_PATH_GENERIC;
    if (!fast) {
        rc = ensure_scratch(ctx, (size_t)T * r * sizeof(float), st);
        if (rc != MORE_OK) return rc;
    }
    if (cudaMemsetAsync(out_psum, 0, (size_t)M * sizeof(float), st) != cudaSuccess) return MORE_ERR_CUDA;
    if (T == 0) return MORE_OK;
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(X);
    const __nv_bfloat16* r1 = static_cast<const __nv_bfloat16*>(R1);
    const __nv_bfloat16* r2 = static_cast<const __nv_bfloat16*>(R2);
    return fast ? launch_psum_tcgen05(x, r1, r2, T, h, r, M, lse, out_psum, *ctx, st)
                : launch_generic_psum(x, r1, r2, T, h, r, M, lse, out_psum, ctx->scratch, st);
}

int more_dispatch(const int32_t* idx, const int32_t* counts, int T, int k, int M, int32_t* out_offsets,
                  int32_t* out_sorted_pairs, void* stream)
{
    if (T < 0 || k < 1 || M < 1 || k > MORE_K_MAX) return MORE_ERR_SHAPE;
    if ((long long)T * k > 0x7fffffffLL) return MORE_ERR_TOO_LARGE;            // pairs are named by int32 positions
    if (!counts || !out_offsets) return MORE_ERR_NULL;
    if (T > 0 && (!idx || !out_sorted_pairs)) return MORE_ERR_NULL;
    if (!aligned(idx, 4) || !aligned(counts, 4) || !aligned(out_offsets, 4) || !aligned(out_sorted_pairs, 4))
        return MORE_ERR_ALIGN;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    rc = ensure_scratch(ctx, dispatch_scratch_bytes(M), static_cast<cudaStream_t>(stream));
    if (rc != MORE_OK) return rc;
    return launch_dispatch(idx, counts, T, k, M, out_offsets, out_sorted_pairs, ctx->scratch,
                           static_cast<cudaStream_t>(stream));
}

int more_route_plan_ex(int T, int h, int r, int M, int k, int gate_mode, int want_lse, int path, int msplit,
                       int* out8)
{
    int rc = check_shape(T, h, r, M, k, gate_mode, path);
    if (rc != MORE_OK) return rc;
    if (!out8) return MORE_ERR_NULL;
    Plan p;
    rc = make_plan(T, h, r, M, k, gate_mode, want_lse != 0 || gate_mode == MORE_GATE_FULL_SOFTMAX, false, path, msplit,
                   148, &p);
    if (rc != MORE_OK) return rc;
    out8[0] = p.path; out8[1] = p.msplit; out8[2] = p.ctas; out8[3] = p.block_tokens;
    out8[4] = p.tg; out8[5] = p.es; out8[6] = p.filter ? 1 : 0; out8[7] = p.paired ? 1 : 0;
    return MORE_OK;
}

int more_route_plan(int T, int h, int r, int M, int k, int gate_mode, int path, int msplit, int* path_out,
                    int* msplit_out, int* ctas_out)
{
    int o[8];
    const int rc = more_route_plan_ex(T, h, r, M, k, gate_mode, 0, path, msplit, o);
    if (rc != MORE_OK) return rc;
    if (path_out) *path_out = o[0];
    if (msplit_out) *msplit_out = o[1];
    if (ctas_out) *ctas_out = o[2];
    return MORE_OK;
}

int more_route_status(void* stream)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int host = 0;
    if (cudaMemcpyAsync(&host, ctx->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MORE_ERR_CUDA;
    if (cudaMemsetAsync(ctx->status, 0, sizeof(int), st) != cudaSuccess) return MORE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MORE_ERR_CUDA;
    return host == 0 ? MORE_OK : MORE_ERR_TIMEOUT;
}

long long more_route_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int more_route_debug_counters(unsigned long long* out16, void* stream)
{
    if (!out16) return MORE_ERR_NULL;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(out16, ctx->stats, 16 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MORE_ERR_CUDA;
    if (cudaMemsetAsync(ctx->stats, 0, 16 * sizeof(unsigned long long), st) != cudaSuccess) return MORE_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

int more_debug_expire_wait(long long budget_cycles, void* stream)
{
    if (budget_cycles < 0 || budget_cycles > 2000000000LL) return MORE_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    expire_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(budget_cycles, ctx->status);
    return cudaGetLastError() == cudaSuccess ? MORE_OK : MORE_ERR_CUDA;
}

int more_debug_scratch_guard(void* stream)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != MORE_OK) return rc;
    if (!ctx->scratch) return 1;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char host[kGuardBytes];
    if (cudaMemcpyAsync(host, static_cast<char*>(ctx->scratch) + ctx->scratch_used, kGuardBytes, cudaMemcpyDeviceToHost,
                        st) != cudaSuccess)
        return MORE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MORE_ERR_CUDA;
    for (size_t i = 0; i < kGuardBytes; ++i)
        if (host[i] != kGuardPattern) return 0;
    return 1;
}

const char* more_strerror(int code)
{
    switch (code) {
        case MORE_OK: return "ok";
        case MORE_ERR_NULL: return "a required pointer is NULL";
        case MORE_ERR_SHAPE: return "unsupported shape (sizes out of range, k > M, or the forced path cannot run it)";
        case MORE_ERR_ALIGN: return "misaligned pointer (inputs need 16 bytes, outputs 4)";
        case MORE_ERR_MODE: return "unknown gate_mode or path";
        case MORE_ERR_ARCH: return "the current device is not compute capability 10.x (B200)";
        case MORE_ERR_CUDA: return "a CUDA call failed";
        case MORE_ERR_TIMEOUT: return "a bounded on-device wait gave up";
        case MORE_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of this entry point";
        default: return "unknown error code";
    }
}

int more_version(void) { return 100; }

}  // extern "C"
