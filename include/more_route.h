/*
 * more_route.h -- C interface of the fused low-rank MoE router for NVIDIA B200 (sm_100a).
 *
 * The router scores M experts through an r-dimensional bottleneck and keeps the k best per token
 * (MoRE layer, Section 2:  g(x) = softmax(TopK(R_1 R_2 x)) ).  Operand names follow this interface, which
 * stores the paper's factors transposed:
 *
 *      X  [T][h]  token activations            (the paper's N = B*T tokens is this T)
 *      R1 [h][r]  down-projection              (= the paper's R_2 transposed;  z = X R1, Section 3.1 Setup)
 *      R2 [r][M]  expert vectors as columns    (= the paper's R_1 transposed;  logits l = z R2, Eq. app_logits)
 *
 * All three are bfloat16, row-major, contiguous, in DEVICE memory unless an entry point says otherwise.
 * The logits are produced tile by tile over M and reduced on chip to a per-token running top-k (and, in
 * full-softmax mode, a running max / sum of exponentials, Eq. app_online), so the T x M logit matrix is never
 * written to memory (Algorithm 1).  Accumulation is fp32; z is carried into the second contraction as a
 * bfloat16 high part plus a bfloat16 low part, so the logits are accurate to about 1e-5 rather than to the
 * 1e-2 a single bfloat16 z would give.
 *
 * Every function returns MORE_OK (0) or a negative MORE_ERR_* code.  On an error detected before launch
 * nothing is launched and no output is touched.  Calls are asynchronous on the given stream unless stated.
 * Buffers are owned by the caller; the library keeps, per device, one cached scratch allocation (grown on
 * demand by cudaMalloc, which may synchronise the device the first time a larger problem is seen) and a
 * small cache of TMA descriptors.  Calls on different host threads are serialised internally; two calls
 * whose kernels may overlap on the GPU (different streams) must not be issued for the same device, because
 * they share that scratch.
 */
#ifndef MORE_ROUTE_H_
#define MORE_ROUTE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* gate_mode */
enum {
    MORE_GATE_TOPK_SOFTMAX = 0, /* softmax over the k selected logits (Section 2); each row of gates sums to 1 */
    MORE_GATE_FULL_SOFTMAX = 1  /* P_{n,j} = exp(l_{n,j} - m_n) / Z_n over all M experts (Eq. app_softmax), carried
                                   across expert tiles by the online recurrence Eq. app_online; the k reported
                                   entries are NOT renormalised, so a row sums to less than 1 */
};

/* path selector of more_route_ex */
enum {
    MORE_PATH_AUTO = 0,    /* tensor-core path when the shape allows it, otherwise the generic path */
    MORE_PATH_GENERIC = 1, /* CUDA-core kernels, any shape within the limits below */
    MORE_PATH_TCGEN05 = 2  /* TMA + tcgen05/TMEM kernel; needs h % 8 == 0, M % 8 == 0, r % 8 == 0, r <= 64, k <= 32 */
};

/* error codes */
enum {
    MORE_OK = 0,
    MORE_ERR_NULL = -1,    /* a required pointer is NULL */
    MORE_ERR_SHAPE = -2,   /* T < 0; h, r, M or k < 1; k > M; k > MORE_K_MAX; r > MORE_R_MAX; M > MORE_M_MAX; msplit outside 0..64;
                              or the forced path cannot run the shape */
    MORE_ERR_ALIGN = -3,   /* X, R1 or R2 not 16-byte aligned, or an output not 4-byte aligned */
    MORE_ERR_MODE = -4,    /* unknown gate_mode or path */
    MORE_ERR_ARCH = -5,    /* the current device is not compute capability 10.x */
    MORE_ERR_CUDA = -6,    /* a CUDA runtime/driver call failed (allocation, descriptor encode, launch) */
    MORE_ERR_TIMEOUT = -7, /* a bounded on-device wait gave up; outputs of that call are undefined (more_route_status) */
    MORE_ERR_TOO_LARGE = -8 /* problem exceeds a fixed capacity of the chosen entry point */
};

#define MORE_K_MAX 32     /* largest k */
#define MORE_R_MAX 1024   /* largest r (generic path); the tensor-core path takes r <= 64 */
#define MORE_M_MAX (1 << 30) /* largest M: expert ids, and the kernels' column arithmetic, are 32-bit */

/*
 * more_route -- route T tokens (Algorithm 1 plus the gates of Section 2 / Eq. app_softmax and the per-expert
 * counts, the bincount of Eq. app_lbal without its 1/(Nk) factor).
 *
 *   X, R1, R2   device, bf16, layouts above, 16-byte aligned, read only.  Values must be finite.
 *   T,h,r,M,k   sizes; 1 <= k <= min(M, MORE_K_MAX).  T == 0 is allowed (only out_counts is written).
 *   gate_mode   MORE_GATE_*.
 *   out_idx     device int32 [T][k]: expert ids in [0, M), distinct within a row, ordered by descending logit,
 *               equal logits by ascending id.
 *   out_gate    device fp32 [T][k]: gate weights in the same order.
 *   out_counts  device int32 [M]: OVERWRITTEN with the number of (token, slot) pairs that selected each expert;
 *               sums to T*k.  (The library zeroes it on `stream` before accumulating.)
 *   stream      a cudaStream_t (NULL = the legacy default stream).  Outputs are valid once it has been synchronised.
 */
int more_route(const void* X, const void* R1, const void* R2,
               int T, int h, int r, int M, int k, int gate_mode,
               int32_t* out_idx, float* out_gate, int32_t* out_counts, void* stream);

/*
 * more_route_ex -- more_route with two optional extra outputs and explicit control of the launch plan.
 *
 *   out_topval  device fp32 [T][k] or NULL: the selected logits (Algorithm 1's TopVals), same order as out_idx.
 *   out_lse     device fp32 [T] or NULL: m_n + log Z_n over all M experts (Eq. app_softmax); computed in either
 *               gate mode when requested (it forces the full-softmax sweep).
 *   path        MORE_PATH_*; a forced path that cannot run the shape gives MORE_ERR_SHAPE.
 *   msplit      tensor-core path only: number of CTAs (at most 64) that share one token block by splitting the expert
 *               range (partial top-k lists and (m, Z) pairs are merged by the last CTA to finish);
 *               0 = chosen by the library.  Results do not depend on it.
 */
int more_route_ex(const void* X, const void* R1, const void* R2,
                  int T, int h, int r, int M, int k, int gate_mode,
                  int32_t* out_idx, float* out_gate, int32_t* out_counts,
                  float* out_topval, float* out_lse, int path, int msplit, void* stream);

/*
 * more_route_host -- the same computation for callers whose buffers live in HOST memory (pinned memory makes
 * the copies asynchronous and faster, pageable memory also works).  The library copies X, R1, R2 to device
 * staging buffers it owns, runs more_route on `stream`, copies out_idx / out_gate / out_counts back and
 * SYNCHRONISES the stream before returning, so the outputs are valid on return.
 * All pointers are host pointers; shapes, modes and errors as for more_route.
 */
int more_route_host(const void* X_host, const void* R1_host, const void* R2_host,
                    int T, int h, int r, int M, int k, int gate_mode,
                    int32_t* out_idx_host, float* out_gate_host, int32_t* out_counts_host, void* stream);

/*
 * more_route_noalloc -- more_route for callers that must not allocate device memory.  (The paper has no counterpart;
 * this is a property of the library, not of the method.)
 *
 * Who needs it: a process whose device memory is owned by its own pool and that may not call the CUDA allocator; code
 * for which a device allocation is unacceptable because it can synchronise the device and stall unrelated streams;
 * an environment that denies cudaMalloc outright.  This entry point calls no cudaMalloc, cudaFree or any other
 * allocating routine, ever.  It runs the generic (CUDA-core) kernels, for any shape they accept, and keeps their
 * only scratch, z = X R1 in fp32, in a fixed 4 MiB array that is part of the library image: every GPU that loads the
 * library holds that array until the process exits.
 *
 *   Limit      T * r <= more_route_noalloc_capacity() (= 1,048,576); beyond it the call returns MORE_ERR_TOO_LARGE
 *              and does nothing.
 *   Set-up     the first call on each device looks up the array's device address (cudaGetSymbolAddress) with that
 *              device current; make that first call before any stream capture begins.
 *   Sharing    all calls on a device use the same array, which keeps whatever the last call left in it.  Every call
 *              overwrites what it reads, and clears out_counts on `stream` itself, so no stale data can leak; but two
 *              calls whose kernels may overlap on the GPU race on the array and must be serialised by the caller.
 *   Otherwise  arguments, outputs, ordering, errors and asynchrony exactly as more_route.
 */
int more_route_noalloc(const void* X, const void* R1, const void* R2,
                       int T, int h, int r, int M, int k, int gate_mode,
                       int32_t* out_idx, float* out_gate, int32_t* out_counts, void* stream);

/* more_route_noalloc_capacity -- the largest T * r more_route_noalloc accepts. */
long long more_route_noalloc_capacity(void);

/*
 * more_route_psum -- the training-forward statistic of Algorithm 2: psum[i] = sum_n P_{n,i}, the column sums of the
 * row-wise softmax over all M experts (Eq. app_softmax, Eq. app_psum), from which the Switch balancing loss is
 * L_bal = (M/N) f . psum with f = counts / (N k) (Eq. app_lbal).  This is Algorithm 2's second sweep: the logit tiles
 * are produced again (z is recomputed from X, the second contraction runs transposed so that a tensor-memory lane is
 * an expert) and reduced over the tokens on chip; nothing of size T x M is written.
 *
 *   X, R1, R2, T, h, r, M   as for more_route (device, bf16).
 *   lse        device fp32 [T]: every token's log-sum-exp over all M logits, as written to out_lse by more_route_ex
 *              for the same inputs (P_{n,i} = exp(l_{n,i} - lse_n)).
 *   out_psum   device fp32 [M]: OVERWRITTEN (zeroed on `stream`, then accumulated with floating-point atomics, so the
 *              last bits depend on the order in which the adds land; the sum over all experts is T up to rounding).
 *   path       MORE_PATH_*, as for more_route_ex (the tensor-core path needs h, r, M multiples of 8 and r <= 64).
 */
int more_route_psum(const void* X, const void* R1, const void* R2, int T, int h, int r, int M,
                    const float* lse, float* out_psum, int path, void* stream);

/*
 * more_route_full -- the fused STANDARD (full-rank) router, g(x) = softmax(TopK(R x)): the same sweep without the
 * low-rank bottleneck (Algorithm 1 with the contraction running over K = h instead of r; the paper's "fused standard
 * MoE" comparison).  Logits l = X W with W = R^T stored [h][M] row-major; they are produced 256 experts at a time by
 * accumulating over all of h on the tensor cores, and selected, gated and counted exactly as in more_route.  The
 * T x M logits never reach memory, but X is re-read (from L2) once per 256-expert step, so unlike the low-rank router
 * this one does a full T x h x M contraction.
 *
 *   X           device bf16 [T][h];  W  device bf16 [h][M];  both 16-byte aligned; h and M multiples of 8, k <= 32
 *               (other shapes: MORE_ERR_SHAPE -- this entry point has the tensor-core path only).
 *   gate_mode, out_idx, out_gate, out_counts, out_topval, out_lse, msplit, stream: as for more_route_ex.
 * The products of bf16 inputs are exact in fp32 and only the fp32 accumulation rounds, so the logits agree with exact
 * arithmetic to ~1e-6 relative.
 */
int more_route_full(const void* X, const void* W, int T, int h, int M, int k, int gate_mode, int32_t* out_idx,
                    float* out_gate, int32_t* out_counts, float* out_topval, float* out_lse, int msplit, void* stream);

/*
 * more_merge_shards -- global top-k for a router whose EXPERT dimension is sharded (over GPUs, or over calls): the
 * hierarchical top-k the paper's discussion of sharded routers leaves to future work ("each device computes a local
 * top-k, then a global top-k"), with the shards' softmax statistics combined as in Eq. app_online.  Shard s has run
 * more_route_ex on the same T tokens with its own slice R2[:, lo_s:hi_s] and reports out_idx, out_topval (and out_lse);
 * after the reports of all S shards have been gathered into one buffer on this device (k pairs per token and shard),
 * this call produces what an unsharded more_route would have: a global top-k member is always a top-k member of its
 * own shard.
 *
 *   idx         device int32 [S][T][k]: expert ids as reported by the shards; shard_base[s] is added to those of shard s.
 *               Slots with a negative id, with id + base >= M, or with a logit of -inf are unused (a shard with fewer
 *               than k experts pads that way).
 *   topval      device fp32 [S][T][k]: the logits of those ids (any order inside a row).
 *   lse         device fp32 [S][T], or NULL: each shard's log-sum-exp over its own experts.  Required for
 *               MORE_GATE_FULL_SOFTMAX; if given, out_lse = log sum_s exp(lse_s).
 *   shard_base  HOST int32 [S], or NULL for all zeros (ids already global): first expert id of every shard.
 *   S           1 .. MORE_MERGE_MAX_SHARDS;  k <= MORE_K_MAX.
 *   out_idx, out_gate   device [T][k], as more_route: descending logit, ties by ascending global id; gates by gate_mode.
 *               A token with fewer than k usable pairs gets id -1 and gate 0 in the remaining places.
 *   out_topval  device fp32 [T][k] or NULL;  out_lse  device fp32 [T] or NULL.
 *   out_counts  device int32 [M]: OVERWRITTEN with the histogram of out_idx.
 * Asynchronous on `stream`; allocates nothing.  The selected logits are compared exactly as reported (no arithmetic
 * on them before the comparison), so the result does not depend on how the experts were split.
 */
#define MORE_MERGE_MAX_SHARDS 64
int more_merge_shards(const int32_t* idx, const float* topval, const float* lse, const int32_t* shard_base,
                      int S, int T, int k, int M, int gate_mode, int32_t* out_idx, float* out_gate,
                      float* out_topval, float* out_lse, int32_t* out_counts, void* stream);

/*
 * more_dispatch -- dispatch bookkeeping for the grouped expert GEMMs that follow the router: the "Sort + Count" box
 * of the layer's forward flowchart ((N,k) -> (Nk) sorted indices + offsets).
 *
 *   idx               device int32 [T][k]: more_route's out_idx.
 *   counts            device int32 [M]: more_route's out_counts for the same call.
 *   out_offsets       device int32 [M+1]: out_offsets[e] = number of (token, slot) pairs routed to experts < e, i.e. the
 *                     exclusive prefix sum of counts; out_offsets[M] = sum of counts (= T*k for finite inputs).
 *   out_sorted_pairs  device int32 [T*k]: the pairs, named by their flat position p = token*k + slot in idx, grouped by
 *                     expert: entries out_offsets[e] .. out_offsets[e+1]-1 are exactly the pairs whose id is e.  The
 *                     order inside one expert's run is unspecified (it depends on the order in which atomic
 *                     increments land) and may differ from call to call.  Pairs whose id is outside [0, M) (only
 *                     possible with non-finite inputs) are left out; entries past out_offsets[M] are not written.
 *   T*k must fit in int32.  Asynchronous on `stream`; uses M*4 bytes of the library's cached scratch, so it must not
 *   overlap on the GPU with another call of this library on the same device.
 */
int more_dispatch(const int32_t* idx, const int32_t* counts, int T, int k, int M,
                  int32_t* out_offsets, int32_t* out_sorted_pairs, void* stream);

/*
 * more_route_plan -- report, without launching, what more_route_ex would do for a shape:
 *   *path_out   MORE_PATH_GENERIC or MORE_PATH_TCGEN05
 *   *msplit_out CTAs per token block (1 on the generic path)
 *   *ctas_out   total CTAs of the main kernel
 * Any of the three may be NULL.  Host-only; needs no device.
 */
int more_route_plan(int T, int h, int r, int M, int k, int gate_mode, int path, int msplit,
                    int* path_out, int* msplit_out, int* ctas_out);

/*
 * more_route_plan_ex -- the same report with the whole launch plan of the tensor-core path (Algorithm 1 leaves the
 * block sizes B_N, B_M free; this is how the library chooses them).  want_lse: non-zero if out_lse will be requested.
 *   out8[0] path   out8[1] CTAs per token block   out8[2] total CTAs   out8[3] tokens per CTA
 *   out8[4] 128-token groups per CTA   out8[5] expert ranges swept side by side inside a CTA
 *   out8[6] reserved (0)
 *   out8[7] which of the two kernels: 1 = 256-token CTAs, two per SM, 64-expert steps (many tokens per SM);
 *           0 = one CTA per SM holding up to four token groups / expert ranges (few tokens per SM)
 * Host-only; needs no device.
 */
int more_route_plan_ex(int T, int h, int r, int M, int k, int gate_mode, int want_lse, int path, int msplit,
                       int* out8);

/*
 * more_route_status -- synchronise `stream` and return the sticky device-side status of the current device:
 * MORE_OK, or MORE_ERR_TIMEOUT if any kernel since the last call gave up on a bounded wait (an mbarrier that
 * never completed).  Reading the status clears it.
 */
int more_route_status(void* stream);

/* more_route_launches -- number of kernels this library has launched in this process (all devices). */
long long more_route_launches(void);

/* more_strerror -- a static, human-readable string for a MORE_* code. */
const char* more_strerror(int code);

/* more_version -- interface version, major*100 + minor. */
int more_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MORE_ROUTE_H_ */
