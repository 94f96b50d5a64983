// more_route_noalloc: the generic (CUDA-core) router for callers that must not allocate device memory.
//
// The ordinary entry points keep a per-device scratch buffer that they grow with cudaMalloc when a larger problem
// arrives.  Some callers cannot live with that: a serving process whose device memory is handed out entirely by its
// own pool, a component that is forbidden to call the CUDA allocator because an allocation may synchronise the whole
// device and stall unrelated streams, or a sandbox that simply denies cudaMalloc.  For them this file provides one
// entry point whose only scratch is a fixed array that is part of the library image itself.
//
// The array lives in device memory of every GPU that loads the library, from load until the process exits, whether
// or not the entry point is ever called.  It is never cleared: each call overwrites the part it needs before reading
// it, so nothing in it has to start at zero (the one output that must start at zero, out_counts, is cleared on the
// caller's stream by every call).  All calls on one device share the array; two calls whose kernels can overlap on
// the GPU (for instance on two streams) race on it and must be serialised by the caller.
#include "more_internal.h"

#include <mutex>

namespace {

// z = X R1 for up to this many (token, rank) pairs, fp32: 4 MiB per GPU.
constexpr long long kNoAllocMaxZ = 1 << 20;
static __device__ __align__(256) float g_noalloc_z[kNoAllocMaxZ];

std::mutex g_noalloc_mutex;
constexpr int kMaxDev = 64;
float* g_noalloc_ptr[kMaxDev];    // device address of g_noalloc_z on each device, filled on first use
bool g_noalloc_ready[kMaxDev];

// In host code `g_noalloc_z` is only a handle for the symbol, not an address a kernel could use; the device
// address has to be asked for, once per device, while that device is current.
int noalloc_setup(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return MORE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ready[dev]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MORE_ERR_CUDA;
        if (major != 10) return MORE_ERR_ARCH;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_z) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return MORE_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = static_cast<float*>(p);
        g_noalloc_ready[dev] = true;
    }
    *out = g_noalloc_ptr[dev];
    return MORE_OK;
}

bool aligned_to(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

extern "C" int more_route_noalloc(const void* X, const void* R1, const void* R2, int T, int h, int r, int M, int k,
                                  int gate_mode, int32_t* out_idx, float* out_gate, int32_t* out_counts, void* stream)
{
    if (gate_mode != MORE_GATE_TOPK_SOFTMAX && gate_mode != MORE_GATE_FULL_SOFTMAX) return MORE_ERR_MODE;
    if (T < 0 || h < 1 || r < 1 || M < 1 || k < 1 || k > M || k > MORE_K_MAX || r > MORE_R_MAX) return MORE_ERR_SHAPE;
    if ((long long)T * (long long)r > kNoAllocMaxZ) return MORE_ERR_TOO_LARGE;    // T*r beyond the built-in scratch
    if (!out_counts) return MORE_ERR_NULL;
    if (T > 0 && (!X || !R1 || !R2 || !out_idx || !out_gate)) return MORE_ERR_NULL;
    if (!aligned_to(X, 16) || !aligned_to(R1, 16) || !aligned_to(R2, 16)) return MORE_ERR_ALIGN;
    if (!aligned_to(out_idx, 4) || !aligned_to(out_gate, 4) || !aligned_to(out_counts, 4)) return MORE_ERR_ALIGN;

    float* z = nullptr;
    const int rc = noalloc_setup(&z);
    if (rc != MORE_OK) return rc;

    more::RouteArgs a;
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.R1 = static_cast<const __nv_bfloat16*>(R1);
    a.R2 = static_cast<const __nv_bfloat16*>(R2);
    a.T = T; a.h = h; a.r = r; a.M = M; a.k = k; a.gate_mode = gate_mode;
    a.out_idx = out_idx; a.out_gate = out_gate; a.out_counts = out_counts;
    a.out_topval = nullptr; a.out_lse = nullptr;
    a.stream = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(out_counts, 0, (size_t)M * sizeof(int32_t), a.stream) != cudaSuccess) return MORE_ERR_CUDA;
    if (T == 0) return MORE_OK;
    more::DeviceCtx unused;                     // the generic launcher takes its scratch as a plain pointer
    return more::launch_generic(a, unused, z);
}

extern "C" long long more_route_noalloc_capacity(void) { return kNoAllocMaxZ; }
