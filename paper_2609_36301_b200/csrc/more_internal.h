// Internal declarations shared by the translation units of libmore_route.so (not installed).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/more_route.h"

namespace more {

struct RouteArgs {
    const __nv_bfloat16* X;
    const __nv_bfloat16* R1;
    const __nv_bfloat16* R2;
    int T, h, r, M, k, gate_mode;
    int32_t* out_idx;
    float* out_gate;
    int32_t* out_counts;
    float* out_topval;  // nullable
    float* out_lse;     // nullable
    cudaStream_t stream;
    bool full = false;  // standard (full-rank) router: R1 unused, R2 is W [h][M], r only sizes the plan
};

// Per-device state: one cached scratch allocation, the sticky status word, device facts.
struct DeviceCtx {
    int dev = -1;
    int cc_major = 0;
    int sm_count = 0;
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
    size_t scratch_used = 0;      // bytes the last plan asked for; the guard region starts there
    int* status = nullptr;        // device int: 0 = ok, else a MORE_ERR_* code written by a kernel
    unsigned long long* stats = nullptr;   // 16 diagnostic counters, next to the status word
    void* staging = nullptr;      // device staging of more_route_host
    size_t staging_bytes = 0;
    float* colnorm = nullptr;           // device float[2]: column-norm maxima written by the filter's preparation
    unsigned* prep_arrivals = nullptr;  // device counter of that kernel (returns to zero after every launch)
};

// Largest number of tokens per CTA of the tensor-core path (rows of one X tile), and the expert-tile width.
constexpr int kBlockTokens = 256;
constexpr int kTileExperts = 128;

// Launch plan (host-only logic, testable without a device).
struct Plan {
    int path;     // MORE_PATH_GENERIC or MORE_PATH_TCGEN05
    int msplit;   // CTAs per token block
    int ctas;     // CTAs of the main kernel
    int rpad;     // r rounded up to a multiple of 16 (tensor-core path)
    int block_tokens;   // tokens per CTA (tensor-core path): a multiple of 32
    int tg = 1;   // low-rank router: 128-token groups per CTA ...
    int es = 1;   // ... and expert ranges swept side by side inside a CTA (tg * es <= 4)
    bool filter = false;   // low-rank router: approximate sweep + exact rescoring of the survivors
    bool paired = false;   // low-rank router: the kernel with 256-token CTAs, two per SM, instead of one CTA per SM
};

bool tcgen05_shape_ok(int T, int h, int r, int M, int k);
// want_lse: the caller asked for out_lse or the full-softmax gate; full: the standard (full-rank) router.
int make_plan(int T, int h, int r, int M, int k, int gate_mode, bool want_lse, bool full, int path, int msplit,
              int sm_count, Plan* out);
bool lowrank_smem_plan(int rpad, int tg, int es, bool filter, int* nst1, int* st1_bytes, int* nst2, int* st2_bytes,
                       int* r2_off);

// Scratch bytes each path needs for a problem.
size_t generic_scratch_bytes(const RouteArgs& a);
size_t lowrank_scratch_bytes(const RouteArgs& a, const Plan& p);
size_t full_scratch_bytes(const RouteArgs& a, const Plan& p);
size_t paired_scratch_bytes(const RouteArgs& a, const Plan& p);

// Launchers: enqueue on a.stream, return MORE_OK / MORE_ERR_*.  `scratch` is at least *_scratch_bytes().
int launch_generic(const RouteArgs& a, DeviceCtx& ctx, void* scratch);
// Both tensor-core launchers clear out_counts on the stream themselves, after every host-side step that can fail.
int launch_lowrank(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch);
int launch_full(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch);
int launch_paired(const RouteArgs& a, DeviceCtx& ctx, const Plan& p, void* scratch);
// Filter mode's preparation: fp16 copy and transposed copy of R2, column-norm maxima, out_counts cleared.
int launch_route_prepare(const RouteArgs& a, int rpad, void* r2h, void* r2t, void* partial, DeviceCtx& ctx);

int launch_generic_psum(const __nv_bfloat16* X, const __nv_bfloat16* R1, const __nv_bfloat16* R2, int T, int h, int r,
                        int M, const float* lse, float* psum, void* scratch, cudaStream_t stream);
int launch_psum_tcgen05(const __nv_bfloat16* X, const __nv_bfloat16* R1, const __nv_bfloat16* R2, int T, int h, int r,
                        int M, const float* lse, float* psum, DeviceCtx& ctx, cudaStream_t stream);

size_t dispatch_scratch_bytes(int M);
int launch_dispatch(const int32_t* idx, const int32_t* counts, int T, int k, int M, int32_t* offsets,
                    int32_t* sorted_pairs, void* scratch, cudaStream_t stream);

void count_launch(int n = 1);

}  // namespace more
