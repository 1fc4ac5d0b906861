// still_hybrid_attn_fwd_static: the prefill for callers that may not allocate device memory.
//
// still_hybrid_attn_fwd keeps its intermediate results (scores, selection, NP-Map features, the
// linear branch's numerator / denominator, the compacted salient K/V rows, a status block) in a
// workspace the caller allocates.  Some callers cannot do that: a plug-in that runs inside
// another runtime's memory plan, a serving loop whose memory was fixed at start-up, code that runs
// where cudaMalloc would synchronise the device or is forbidden outright.  For them the workspace
// lives here, in a fixed array in the library's own device image.  The price: the array has a
// fixed, modest size; every GPU that loads the library carries it until the process exits; and all
// calls share it.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/still.h"

namespace {

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// not a device address and must never be handed to a kernel or to still_hybrid_attn_fwd.
static __device__ __align__(256) unsigned char g_static_workspace[STILL_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_addr[kMaxDevices] = {};  // device address of the array, per device ordinal

// Device address of the scratch array on the current device (looked up once per device, with that
// device current).  Returns nullptr if the look-up fails.
void *static_workspace_ptr() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_addr[dev] = ptr;
    }
    return g_addr[dev];
}

}  // namespace

extern "C" int still_hybrid_attn_fwd_static(const still_params_t *p, int64_t N, const void *Q, const void *K,
                                            const void *V, const void *G, const void *Wq, const void *bq,
                                            const void *Wk, const void *bk, void *Y, float *scores,
                                            int32_t *sel_idx, void *cuda_stream) {
    if (!p || N < 0) return STILL_ERR_INVALID_ARG;
    const size_t need = still_workspace_bytes(p, N);
    if (need == 0) return STILL_ERR_INVALID_ARG;  // parameters the prefill would reject as well
    if (N == 0) return STILL_OK;
    if (need > (size_t)STILL_STATIC_WORKSPACE_BYTES) return STILL_ERR_WORKSPACE_TOO_SMALL;
    void *ws = static_workspace_ptr();
    if (!ws) return STILL_ERR_CUDA;
    // Everything the prefill expects to find zeroed (its status block) it clears itself at the start
    // of every call, on the caller's stream; the rest of the workspace is written before it is read.
    return still_hybrid_attn_fwd(p, N, Q, K, V, G, Wq, bq, Wk, bk, Y, scores, sel_idx, /*state_out=*/nullptr, 0, ws,
                                 (size_t)STILL_STATIC_WORKSPACE_BYTES, cuda_stream);
}
