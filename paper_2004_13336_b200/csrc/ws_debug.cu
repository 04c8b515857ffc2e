// Bounds-checking debug build: the status word and the calls that read it.
//
// A library compiled with -DWS_DEBUG_BOUNDS makes every kernel compare the range of each work item
// with the extents of the buffers it was given before it touches them.  A range outside them ORs a
// bit into the status word below and the item is skipped: the error becomes a value the caller can
// read, never a trap, a failed assert or a wild access.  The regular build has none of this code; its
// three calls below only report that the checks are not compiled in.
#include "ws_internal.h"

#ifdef WS_DEBUG_BOUNDS
namespace {
// In host code this name is a handle for the runtime's symbol table, not a device address.
__device__ unsigned g_ws_bounds_status = 0;

__global__ void bounds_selftest_kernel(unsigned* word, long long index, long long extent) {
    // the check every kernel makes, on an index that lies outside on purpose; nothing is accessed
    if (index < 0 || index >= extent) atomicOr(word, (unsigned)WS_BOUNDS_SELFTEST);
}
}  // namespace

unsigned* ws_bounds_word() {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_ws_bounds_status) != cudaSuccess) return nullptr;
    return (unsigned*)p;
}
#endif

extern "C" int32_t ws_debug_bounds_enabled(void) {
#ifdef WS_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

extern "C" ws_status ws_debug_bounds_read(uint32_t* bits, int32_t clear) {
    if (!bits) return WS_ERR_INVALID_ARG;
    *bits = 0;
#ifdef WS_DEBUG_BOUNDS
    unsigned* w = ws_bounds_word();
    if (!w) return WS_ERR_CUDA;
    cudaError_t e = cudaDeviceSynchronize();
    unsigned v = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&v, w, sizeof(v), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && clear) e = cudaMemset(w, 0, sizeof(v));
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_debug_bounds_read");
    *bits = v;
    return WS_OK;
#else
    (void)clear;
    return WS_ERR_INVALID_ARG;
#endif
}

extern "C" ws_status ws_debug_bounds_selftest(void* stream) {
#ifdef WS_DEBUG_BOUNDS
    unsigned* w = ws_bounds_word();
    if (!w) return WS_ERR_CUDA;
    bounds_selftest_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(w, 10, 10);
    return ws_check_launch("ws_debug_bounds_selftest");
#else
    (void)stream;
    return WS_ERR_INVALID_ARG;
#endif
}
