// LAMB update for callers that cannot hand the library a workspace.
//
// Some users of this library have no way to obtain device scratch memory at the
// moment they need the update: an optimizer plug-in running under a training
// framework whose caching allocator has already reserved the whole GPU, a
// latency-critical step loop that must not enter the CUDA allocator (cudaMalloc
// may synchronise the device), or a host language binding that can pass
// tensors but not create them.  For them the scratch that ws_shard_update
// expects from the caller (trust ratios, squared norms, per-tile partial sums)
// lives in a fixed array inside the library image.
//
// The array is part of every GPU context that loads libws.so and stays
// resident until the process exits, so its size is kept modest.
#include <mutex>

#include "ws_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = WS_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime's symbol table, not
// an address a kernel could use; the device address is looked up below.
static __device__ __align__(256) unsigned char g_lamb_scratch[kStaticScratchBytes];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device, resolved once
// per device (with that device current) and cached.
ws_status scratch_for_current_device(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_lamb_update_static_scratch(cudaGetDevice)");
    if (dev < 0 || dev >= kMaxDevices) return WS_ERR_TOO_LARGE;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_lamb_scratch);
        if (e != cudaSuccess) return ws_cuda_fail(e, "ws_lamb_update_static_scratch(cudaGetSymbolAddress)");
        if (!p) return WS_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return WS_OK;
}

}  // namespace

extern "C" size_t ws_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" ws_status ws_lamb_update_static_scratch(const ws_plan* plan, const ws_grads* grads, const ws_state* state,
                                                   const ws_hyper* hyper, const ws_out* out, void* stream) {
    WsRange range_("ws_lamb_update_static_scratch");
    if (!plan || !hyper) return WS_ERR_INVALID_ARG;
    if (hyper->opt != WS_LAMB) return WS_ERR_INVALID_ARG;
    const size_t need = ws_workspace_bytes(plan, WS_LAMB);
    if (need > kStaticScratchBytes) return WS_ERR_TOO_LARGE;   // refuse before touching the device
    // all three launches' arguments are checked before the first one
    ws_status s = ws_lamb_check_apply_args(plan, state, hyper, out);
    if (s != WS_OK) return s;
    void* scratch = nullptr;
    if ((s = scratch_for_current_device(&scratch)) != WS_OK) return s;
    // The update itself is ws_shard_update's all-shard LAMB with the library's array as its workspace:
    // three launches, or one when the plan carries its one-launch schedule.  What has to start at zero
    // (the one-launch route's counters, flags, ticket and status word) is cleared on the stream by that
    // route itself; everything else in the scratch is overwritten before it is read.
    return ws_shard_update(plan, -1, grads, state, hyper, out, scratch, kStaticScratchBytes, stream);
}
