// Host-buffer form of one whole step: host gradients in, host weights out.
// Pure orchestration of the other entry points plus cudaMemcpyAsync; every
// arithmetic and formatting step still runs in the kernels.
#include "ws_internal.h"

extern "C" int64_t ws_plan_arena_elems(const ws_plan* p) { return p ? p->arena_elems : 0; }

extern "C" ws_status ws_plan_arena_offsets(const ws_plan* p, const int64_t** offsets, int32_t* T) {
    if (!p || !offsets || !T) return WS_ERR_INVALID_ARG;
    *offsets = (const int64_t*)p->arena_off.data();
    *T = p->T;
    return WS_OK;
}

extern "C" ws_status ws_step_host(const ws_plan* p, const ws_host_io* io, const ws_state* state,
                                  const ws_hyper* hyper, const ws_out* out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    WsRange range_("ws_step_host");
    if (!p || !io || !state || !hyper) return WS_ERR_INVALID_ARG;
    if (!io->host_grads || !io->dev_grad_arena || !io->dev_packed_grads || !io->dev_weight_arena ||
        !io->host_weights)
        return WS_ERR_INVALID_ARG;
    if (io->grad_dtype != WS_F32 && io->grad_dtype != WS_BF16) return WS_ERR_DTYPE;
    if (!ws_aligned16(io->dev_grad_arena) || !ws_aligned16(io->dev_weight_arena)) return WS_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t geb = io->grad_dtype == WS_BF16 ? 2 : 4;
    std::vector<const void*> tptr(p->T);
    for (int t = 0; t < p->T; ++t) tptr[t] = (const char*)io->dev_grad_arena + (size_t)p->arena_off[t] * geb;
    for (int k = 0; k < p->R; ++k) {
        if (!io->host_grads[k] || !io->dev_packed_grads[k]) return WS_ERR_INVALID_ARG;
        cudaError_t e = cudaMemcpyAsync(io->dev_grad_arena, io->host_grads[k], (size_t)p->arena_elems * geb,
                                        cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return ws_cuda_fail(e, "ws_step_host(gradients to device)");
        ws_status s = ws_pack(p, tptr.data(), io->grad_dtype, io->dev_packed_grads[k], stream);
        if (s != WS_OK) return s;
    }
    ws_grads g;
    g.ptrs = (const void* const*)io->dev_packed_grads;
    g.R = p->R;
    g.dtype = io->grad_dtype;
    g.slice_mode = 0;
    ws_status s = ws_shard_update(p, -1, &g, state, hyper, out, workspace, workspace_bytes, stream);
    if (s != WS_OK) return s;
    const bool from_out = out && out->gathered;
    const ws_dtype wdt = from_out ? out->dtype : WS_F32;
    const size_t web = wdt == WS_BF16 ? 2 : 4;
    std::vector<void*> wptr(p->T);
    for (int t = 0; t < p->T; ++t) wptr[t] = (char*)io->dev_weight_arena + (size_t)p->arena_off[t] * web;
    s = ws_unpack(p, from_out ? out->gathered : state->w, wdt, wptr.data(), stream);
    if (s != WS_OK) return s;
    cudaError_t e = cudaMemcpyAsync(io->host_weights, io->dev_weight_arena, (size_t)p->arena_elems * web,
                                    cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_step_host(weights to host)");
    return WS_OK;
}
